"""HiViS drafter step on B200: thin Python binding over the C-ABI library `libhivis.so`.

Everything on the path (fusion FC + step residual, RMSNorm, QKV, RoPE, split-KV attention over
the text-only cache, O projection, SwiGLU MLP, LM head + argmax, greedy verification and KV
rollback) runs in the library's CUDA kernels; this package only marshals arguments.  PyTorch is
used for device memory and streams.  There is no CPU fallback: importing `binding` raises if the
library cannot be loaded.
"""
from .binding import (Drafter, HivisError, lib, hivis_init, hivis_destroy, hivis_prefill, hivis_draft,
                      hivis_verify, hivis_reset, hivis_get_kv_len, hivis_set_kv_len, hivis_read_kv,
                      hivis_debug_tap, hivis_step_bytes, hivis_launch_count, hivis_last_error, hivis_profile_begin, hivis_profile_end, PROFILE_CLASSES,
                      hivis_set_option, hivis_status, hivis_verify_noalloc, hivis_read_phase_times, hivis_draft_tree, hivis_verify_tree, hivis_verify_sampled, hivis_draft_sampled, hivis_set_kv_len_batch, HIVIS_OPT_CHAIN_KERNEL, HIVIS_OPT_TC_KERNEL,
                      HIVIS_F32, HIVIS_BF16, EXPORTS, LIB_PATH)

__all__ = ["Drafter", "HivisError", "lib", "hivis_init", "hivis_destroy", "hivis_prefill", "hivis_draft",
           "hivis_verify", "hivis_reset", "hivis_get_kv_len", "hivis_set_kv_len", "hivis_read_kv",
           "hivis_debug_tap", "hivis_step_bytes", "hivis_launch_count", "hivis_last_error", "hivis_profile_begin", "hivis_profile_end", "PROFILE_CLASSES", "hivis_set_option", "hivis_status", "hivis_verify_noalloc", "hivis_read_phase_times", "hivis_draft_tree", "hivis_verify_tree", "hivis_verify_sampled", "hivis_draft_sampled", "hivis_set_kv_len_batch", "HIVIS_OPT_CHAIN_KERNEL", "HIVIS_OPT_TC_KERNEL",
           "HIVIS_F32", "HIVIS_BF16", "EXPORTS", "LIB_PATH"]
