"""CPU-side checks of the boundary: the library loads, exports every symbol the header declares,
and rejects bad configurations before touching the device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hivis.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hivis_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2509_23928_b200 as pkg
    syms = declared_symbols()
    assert "hivis_init" in syms and "hivis_draft" in syms and "hivis_verify" in syms and "hivis_prefill" in syms
    for s in syms:
        assert hasattr(pkg.lib, s), f"{s} is declared in hivis.h but not exported"
    assert set(syms) == set(pkg.EXPORTS) | {s for s in syms if s not in pkg.EXPORTS}
    for s in pkg.EXPORTS:
        assert s in syms, f"binding names {s}, which the header does not declare"


def _cfg(**kw):
    from paper_2509_23928_b200.binding import hivis_config
    base = dict(struct_size=C.sizeof(hivis_config), dtype=1, d=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                ffn=688, vocab=1024, rms_eps=1e-5, rope_base=1e4, max_batch=1, max_len=64, max_k=4)
    base.update(kw)
    return hivis_config(**base)


@pytest.mark.parametrize("kw,code", [
    (dict(struct_size=8), -1), (dict(dtype=7), -3), (dict(d=100), -2), (dict(head_dim=96), -2),
    (dict(n_q_heads=6, n_kv_heads=4), -2), (dict(ffn=690), -2), (dict(vocab=0), -2),
    (dict(max_batch=0), -5), (dict(max_batch=65), -5), (dict(max_k=17), -5), (dict(max_len=0), -5),
    (dict(rope_base=0.0), -1),
])
def test_init_rejects_bad_config_without_a_device(kw, code):
    from paper_2509_23928_b200.binding import hivis_weights, lib
    out = C.c_void_p()
    fake = hivis_weights(*([0x1000] * 7 + [None] * 3 + [0x1000] * 5 + [None]))
    rc = lib.hivis_init(C.byref(out), C.byref(_cfg(**kw)), C.byref(fake), None)
    assert rc == code and not out.value


def test_init_rejects_null_and_misaligned_weights():
    from paper_2509_23928_b200.binding import hivis_weights, lib
    out = C.c_void_p()
    assert lib.hivis_init(C.byref(out), C.byref(_cfg()), C.byref(hivis_weights()), None) == -1
    bad = hivis_weights(*([0x1008] * 7 + [None] * 3 + [0x1000] * 5 + [None]))
    assert lib.hivis_init(C.byref(out), C.byref(_cfg()), C.byref(bad), None) == -1
    partial_bias = hivis_weights(*([0x1000] * 7 + [0x1000, None, None] + [0x1000] * 5 + [None]))
    assert lib.hivis_init(C.byref(out), C.byref(_cfg()), C.byref(partial_bias), None) == -1
    assert lib.hivis_init(None, None, None, None) == -1
    assert lib.hivis_destroy(None) == 0


def test_null_context_is_an_argument_error():
    from paper_2509_23928_b200.binding import lib
    assert lib.hivis_draft(None, 1, None, 1, None, 0, None, None, None, None) == -1
    assert lib.hivis_verify(None, 1, None, 1, None, None, 0, None, None, None, None) == -1
    assert lib.hivis_prefill(None, 1, None, None, None, None, None, None, None) == -1
    assert lib.hivis_step_bytes(None, 0, None) == 0
    assert lib.hivis_draft_sampled(None, 1, None, 1, None, 0, 1.0, None, None, None, None) == -1
    assert lib.hivis_set_kv_len_batch(None, 1, None, None, 0, None) == -1


def test_product_package_does_not_import_the_oracle():
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2509_23928_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("# no oracle", ""), f"{f} mentions the oracle"
