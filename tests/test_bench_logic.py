"""Host logic of bench.py: the multi-rank reduction (max of the times, sum of the work) under
gloo with world_size 2, the clock-sample parser, and the rank gating of the reference arm."""
import json
import os
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, flops = bench.reduce_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist, None)
    out.put((rank, ms, flops))
    dist.barrier()
    dist.destroy_process_group()


def test_reduce_over_ranks_gloo_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 300.0), (1, 15.0, 300.0)]          # max of times, sum of work, same on every rank


def test_single_rank_passthrough():
    assert bench.reduce_over_ranks(3.5, 7.0) == (3.5, 7.0)


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    out0 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--size", "512",
                           "--steps", "1", "--warmup", "0"], env=env0, capture_output=True, text=True, timeout=300)
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["n_gpus"] == 2
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def test_workload_name_mentions_the_config():
    assert "16384" in bench.workload_name(16384, 19, 1.0) and "19 moduli" in bench.workload_name(16384, 19, 1.0)


def test_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it must run two ranks (here on CPU, gloo, no kernels)."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--launcher-selftest"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2
    assert lines[0]["ms_per_step"] == 11.0 and abs(lines[0]["value"] - 2e12 / 11e-3 / 1e12) < 1e-9   # max of times, sum of work


def test_recorded_traffic_needs_a_capture_of_the_current_source(tmp_path, monkeypatch):
    rec = {"captures": [{"M": 64, "N": 64, "K": 64, "moduli": 19, "dram_read_bytes": 10, "dram_write_bytes": 5,
                         "gemm_source_sha256": "not the current source", "command": "x"}]}
    path = tmp_path / "t.json"
    path.write_text(json.dumps(rec))
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(path))
    assert bench.recorded_traffic(64, 64, 64, 19)[0] is None
    assert bench.recorded_traffic(128, 64, 64, 19)[0] is None
    rec["captures"][0]["gemm_source_sha256"] = bench.gemm_source_hash()
    path.write_text(json.dumps(rec))
    assert bench.recorded_traffic(64, 64, 64, 19)[0] == 15.0
