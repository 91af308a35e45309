"""The N > 1 path of the benchmark on CPU: replicas only (no collective on the hot path), so what the ranks
share is the timing reduction.  Two gloo ranks check it."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import hivis_inputs as hi
    ms = 10.0 + 5.0 * rank                                  # rank 1 is the slower replica
    slowest = bench.max_over_ranks(ms, dist, "cpu")
    wl = bench.replica_workload(hi.workload("c1_tiny_f32_b1"), rank, world)
    ids, _, _ = hi.make_prompt(wl)
    gathered = [None] * world
    dist.all_gather_object(gathered, (slowest, wl.seed, int(ids[0]), wl.dims.d, wl.batch, wl.k))
    dist.barrier()
    if rank == 0:
        json.dump({"gathered": gathered, "value": bench.job_throughput(world, 4, wl.k, slowest)}, open(out, "w"))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_replica_and_aggregate(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, 29517, out), nprocs=2, join=True)
    r = json.load(open(out))
    g = r["gathered"]
    assert g[0][0] == g[1][0] == 15.0                        # both ranks see the slowest time
    assert g[0][1] != g[1][1]                                # independent replicas: different seeds ...
    assert g[0][3:] == g[1][3:]                              # ... same shapes
    assert abs(r["value"] - 2 * 4 * 4 / 15e-3) < 1e-6        # 2 replicas x 4 steps x k=4 draft steps / 15 ms


def test_reference_arm_prints_one_line_from_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_plain_launch_with_gpus_2_starts_two_ranks_itself():
    """`python bench.py --gpus 2` outside torchrun: the script starts its own two ranks (here on gloo with the device
    work stubbed), both go through the rank reduction, rank 0 prints one line with n_gpus = 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    env["HIVIS_BENCH_STUB"] = "1"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "4"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["config"]["parallelism"].startswith("replicas x2")
    assert line["stub_slowest_ms"] == 15.0 and line["value"] is None and "stub" in line["data"]


def test_fewer_ranks_than_gpus_is_refused():
    """--gpus 8 with a single started rank must not print a line that claims eight replicas."""
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", HIVIS_BENCH_STUB="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "8"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert p.returncode != 0 and p.stdout.strip() == "" and "refusing" in p.stderr


def test_traffic_figure_is_dropped_when_the_kernels_changed(tmp_path, monkeypatch):
    import bench
    f = tmp_path / "t.json"
    good = {"captures": {"w": {"dram_bytes_read": 10, "dram_bytes_write": 5, "source_hash": bench.kernel_source_hash()}}}
    f.write_text(json.dumps(good))
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    assert bench.captured_traffic("w") == 15
    assert bench.captured_traffic("other") is None
    good["captures"]["w"]["source_hash"] = "0" * 16
    f.write_text(json.dumps(good))
    assert bench.captured_traffic("w") is None
