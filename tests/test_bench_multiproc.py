"""The multi-rank plumbing of bench.py on CPU: two gloo ranks on 127.0.0.1.

The GEMM itself shards on M with no collective, so what N > 1 adds is only:
rank-specific shards of A, the MAX reduction of the per-rank step time, the
whole-job aggregate, and the reference arm running on rank 0 alone."""
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    import nk_inputs
    bench.init_distributed(world, None)
    my_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    ms = bench.max_over_ranks(my_ms, world, None)
    a = nk_inputs.fill(bench.shard_seed(17, rank), nk_inputs.TENSOR_A, 64, dtype="bf16")
    b = nk_inputs.fill(17, nk_inputs.TENSOR_B, 64, dtype="bf16")
    out.put((rank, ms, bench.whole_job_tflops(2e12, world, ms), a.tolist(), b.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, v0, a0, b0), (r1, ms1, v1, a1, b1) = res
    assert ms0 == ms1 == 15.0                      # the slowest rank sets the time
    assert v0 == v1 and abs(v0 - 2 * 2e12 / 15e-3 / 1e12) < 1e-9
    assert a0 != a1 and b0 == b1                   # own rows of A, replicated B


def test_reference_arm_is_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_bare_gpus_2_starts_two_ranks_itself():
    """`bench.py --gpus 2` run bare (no WORLD_SIZE in the environment) must start two ranks on its own.
    --dry-run leaves the GEMM out (no device here): what is checked is that two ranks met, that rank 0
    alone printed the JSON line, that it says n_gpus = 2, and that the slower rank set the time."""
    import json
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "5",
                        "--warmup", "0", "--dry-run"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["dry_run"] is True
    assert "rank 0 of 2" in r.stderr and "rank 1 of 2" in r.stderr
    # rank 1 sleeps 4 ms per step, rank 0 only 2 ms: the maximum over the ranks is reported
    assert out["ms_per_step"] >= 4.0
    assert "x2" in out["config"]["parallelism"]


def test_recorded_traffic_is_dropped_when_the_sources_change(tmp_path, monkeypatch):
    """The DRAM-traffic figure of the bench line comes from a committed capture that names the kernel,
    the shape and the hash of the kernel sources it was taken from; any mismatch must give null."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    from paper_2511_13764_b200 import _build
    rec = {"kernel": "k", "shape": [8, 8, 8], "dram_read_bytes": 10.0, "dram_write_bytes": 5.0,
           "source_hash": _build.source_hash(), "captured": "today"}
    path = tmp_path / "t.json"
    path.write_text(json.dumps(rec))
    monkeypatch.setattr(bench, "TRAFFIC_JSON", str(path))
    assert bench.recorded_traffic("k", (8, 8, 8))[0] == 15.0
    assert bench.recorded_traffic("other", (8, 8, 8))[0] is None
    assert bench.recorded_traffic("k", (8, 8, 16))[0] is None
    rec["source_hash"] = "0" * 64
    path.write_text(json.dumps(rec))
    assert bench.recorded_traffic("k", (8, 8, 8))[0] is None
