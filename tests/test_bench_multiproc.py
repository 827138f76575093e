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
