"""The N > 1 path of bench.py is N independent replicas: per-rank batches, a barrier, the
slowest rank's time, aggregate tokens/s.  Its host logic is exercised here with two gloo
ranks on CPU (the data path itself has no collective)."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    import torch.distributed as dist

    import bench
    from paper_2404_13528_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # each rank draws a different batch of the same shape
        x = synth.swin_inputs(bench.shard_seed(3, rank), 1, 7, 7, 8, 1, 7, 0, "bf16")["x"]
        dist.barrier()
        ms = bench.max_over_ranks(dist, 10.0 + 5.0 * rank, "cpu")           # rank 1 is the slow one
        out.put((rank, ms, int(np.asarray(x, dtype=np.uint16).sum())))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_distinct_shards():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]            # max over ranks, seen by both
    assert res[0][2] != res[1][2]                          # the two ranks hold different data
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job_tokens_per_s(100352, 2, 10, 15.0) == 2 * 100352 * 10 / 0.015
    assert bench.max_over_ranks(None, 3.0, "cpu") == 3.0


def test_gpus_flag_must_match_the_launched_ranks():
    """`bench.py --gpus N` started without N ranks refuses (it never silently runs one rank and calls it N)."""
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "8"], capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode != 0
    assert "needs 8 ranks" in r.stderr and "torch.distributed.run" in r.stderr
