"""Host logic of the multi-GPU benchmark path on CPU ranks (gloo, world size 2)."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2502_11417_b200 import synth
    w = synth.make_workload(1, n=500, n_budgets=3, replica=rank)       # every rank draws its own trace
    mine = 10.0 * (rank + 1)                                           # rank 1 is the slow one
    total = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    q.put((rank, total, int(w.prompt_len.sum()), w.n, w.n_policies))
    dist.destroy_process_group()


def test_max_over_ranks_and_independent_traces():
    world, port = 2, 29500 + os.getpid() % 1000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [20.0, 20.0]                         # both ranks see the slowest rank's time
    assert got[0][2] != got[1][2]                                      # different traces ...
    assert got[0][3:] == got[1][3:] == (500, 3)                        # ... of the same shape
    import bench
    # whole-job rate: units of all ranks over the slowest rank's time
    assert bench.whole_job_rate(1500, world, steps=4, total_ms=20.0) == 1500 * 2 * 4 / 0.020
    assert bench.max_over_ranks(7.0, None, "cpu") == 7.0


def test_replica_zero_is_the_reference_trace():
    from paper_2502_11417_b200 import synth
    a, b = synth.make_workload(1, n=300), synth.make_workload(1, n=300, replica=0)
    assert (a.prompt_len == b.prompt_len).all() and (a.server_ttft_s == b.server_ttft_s).all()
    c = synth.make_workload(1, n=300, replica=3)
    assert not np.array_equal(a.output_len, c.output_len)


def test_never_clamps_follows_the_tick_arithmetic():
    """bench.never_clamps decides which algorithmic instruction count the play-out is held against: true iff
    every policy paces delivery and tau >= T + J for every endpoint, in microsecond ticks."""
    import bench
    from paper_2502_11417_b200 import synth
    for cfg in range(6):
        assert bench.never_clamps(synth.make_workload(cfg, n=64))
    w = synth.make_workload(3, n=64, n_budgets=2)                      # phone-class device: T = 100,000, J = 5,000
    w.policies = [synth.policy(0.5, r_c=1e6 / 105000.0)]
    assert bench.never_clamps(w)                                       # tau = T + J exactly
    w.policies = [synth.policy(0.5, r_c=1e6 / 104999.0)]
    assert not bench.never_clamps(w)
    w.policies = [synth.policy(0.5, flags=synth.FLAG_MIGRATION)]       # pacing off
    assert not bench.never_clamps(w)
