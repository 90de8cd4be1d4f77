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


def _shard_rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import Oracle
    from paper_2502_11417_b200 import synth
    w = synth.make_workload(4, n=3001, n_budgets=2)                    # every rank holds a range of ONE trace
    b = bench.shard_bounds(w.n, world)
    lo, hi = b[rank], b[rank + 1]
    part = Oracle(w.prompt_len[lo:hi], w.output_len[lo:hi], w.server_ttft_s[lo:hi], w.server_profile[lo:hi],
                  w.device_profile[lo:hi], w.servers, w.devices)
    G = part.n_groups
    tabs = [part.group_tables(g) for g in range(G)]
    cnt = np.stack([t[0] for t in tabs])
    mine = [torch.from_numpy(t[1].astype(np.int32)) for t in tabs]
    tcnt, ticks, n_ticks = bench.exchange_group_tables(cnt, mine, dist, "cpu")
    words = torch.arange(10, dtype=torch.int64) * (rank + 1)           # accumulators add up: one all-reduce
    dist.all_reduce(words, op=dist.ReduceOp.SUM)
    q.put((rank, lo, hi, tcnt, ticks.numpy(), n_ticks, words.numpy()))
    dist.destroy_process_group()


def test_request_range_shards_exchange_whole_trace_tables():
    """Two CPU ranks hold halves of one trace; after the exchange each has the length histogram and, group by
    group, the TTFT ticks of the whole trace (checked against the oracle's tables of the whole trace)."""
    from oracle import Oracle
    from paper_2502_11417_b200 import synth
    world, port = 2, 30500 + os.getpid() % 1000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_shard_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=120) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = synth.make_workload(4, n=3001, n_budgets=2)
    whole = Oracle.from_workload(w)
    assert [(g[1], g[2]) for g in got] == [(0, 1500), (1500, 3001)]    # contiguous, disjoint, covering
    for _, _, _, tcnt, ticks, n_ticks, words in got:
        off = 0
        for g in range(whole.n_groups):
            cnt, srt, _ = whole.group_tables(g)
            assert (tcnt[g] == cnt).all() and int(n_ticks[g]) == len(srt)
            assert (np.sort(ticks[off:off + len(srt)]) == srt).all()   # the group's ticks, the ranks' runs in turn
            off += len(srt)
        assert off == len(ticks) == w.n
        assert (words == np.arange(10) * 3).all()
    import bench
    assert bench.shard_bounds(10, 4) == [0, 2, 5, 7, 10]


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
