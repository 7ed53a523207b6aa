"""The benchmark's N > 1 logic on CPU: two gloo ranks, no GPU.  Covers the per-rank batches, the
max-over-ranks of the step time, the whole-job aggregate, and the reference arm's rule that only
rank 0 works and prints."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2602_14293_b200.ranks import Ranks
    from fc_inputs import workloads as wl
    rk = Ranks("gloo")
    rk.barrier()
    ch = wl.affine_gelu_residual_lse(4, 16)
    x = wl.make_inputs(ch, rk.batch_seed(0))[0]
    ms = rk.max_over_ranks(1.0 + rank)            # rank 1 is the slow one: 2.0 ms
    q.put((rank, int(x.astype("int64").sum()), ms, rk.aggregate(10.0, ms)))
    rk.finish()


def test_two_gloo_ranks_max_time_and_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, sum0, ms0, agg0), (r1, sum1, ms1, agg1) = res
    assert (r0, r1) == (0, 1)
    assert sum0 != sum1                                 # each rank drew its own batch
    assert ms0 == ms1 == 2.0                            # max over ranks, seen by both
    assert agg0 == agg1 == 2 * 10.0 / 2.0e-3            # all ranks' units over the slowest time


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "C1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "C1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
