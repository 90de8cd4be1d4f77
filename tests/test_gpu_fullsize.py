"""Full-size workloads, in the launch configuration the benchmark times: sampled pairs against the oracle
(request ranges it can play one by one), whole-grid statistics against the oracle run on the host's threads,
and properties that hold at any size (needs a GPU)."""
import os

import numpy as np
import pytest

from oracle import Oracle
from paper_2502_11417_b200 import synth, Trace
from parity import rel_close, EXACT_PAIR, FLOAT_PAIR, REL_TOL

pytestmark = pytest.mark.gpu


def _sampled_ranges(n, k, width, seed):
    rng = np.random.default_rng(seed)
    starts = np.sort(rng.integers(0, n - width, size=k))
    return [(int(s), int(s) + width) for s in starts] + [(0, width), (n - width, n)]


def _check(w, policies, ranges, tag):
    tr = Trace.from_workload(w)
    P = len(policies)
    out = tr.alloc_pair_outputs(P)
    tr.eval_policies(policies, w.seed, out)
    gs = tr.reduce_stats()
    orc = Oracle.from_workload(w)
    from parity import check_tables
    check_tables(tr, orc, tag)             # length histograms, sorted TTFT ticks and knots at full size
    host = {f: out[f].cpu().numpy() for f in out}
    oout = orc.eval_columns(policies, w.seed, ranges)
    cols = np.concatenate([np.arange(i0, i1) for i0, i1 in ranges])
    for f in EXACT_PAIR:
        assert (host[f][:, cols] == oout[f]).all(), (tag, f)
    for f in FLOAT_PAIR:
        assert rel_close(host[f][:, cols], oout[f], REL_TOL).all(), (tag, f)
    # properties at full size
    sum_n, N = int(w.output_len.sum()), w.n
    for p in range(P):
        s = gs[p]
        th, bh = tr.histograms(p)
        assert s.n_requests == N and s.n_intervals == sum_n - N
        assert int(th.sum()) == N and int(bh.sum()) == sum_n - N          # no histogram update was lost
        assert s.n_server_only + s.n_device_only + s.n_race == N
        assert s.tok_server + s.tok_device == sum_n
        assert s.tok_device == int(host["tok_device"][p].sum(dtype=np.int64))
        assert s.n_migrations == int((host["mig_at"][p] > 0).sum()) and s.delayed_tokens == int(host["delayed"][p].sum(dtype=np.int64))
        assert s.n_device_only == int((host["decision"][p] == 1).sum()) and s.n_race == int((host["decision"][p] == 2).sum())
        assert rel_close(s.total_cost, host["cost"][p].sum(dtype=np.float64), 1e-5)
        assert rel_close(s.mean_ttft_s, host["ttft_s"][p].mean(dtype=np.float64), 1e-5)
        assert (host["tok_server"][p].astype(np.int64) + host["tok_device"][p] == w.output_len).all()
    tr.close()
    return gs


def test_workload1_full():
    w = synth.make_workload(1)
    gs = _check(w, w.policies, _sampled_ranges(w.n, 12, 150, 1), "workload1")
    dev_only = [s.n_device_only for s in gs]
    assert all(b <= a for a, b in zip(dev_only, dev_only[1:]))               # a larger budget races more prompts
    assert dev_only[0] == w.n and dev_only[-1] == 0


def test_workload3_full_long_outputs():
    w = synth.make_workload(3)
    _check(w, w.policies[::5], _sampled_ranges(w.n, 6, 40, 3), "workload3")


def test_workload4_full_six_groups_policy_subset():
    w = synth.make_workload(4)
    pols = [w.policies[k] for k in (0, 37, 127, 128 + 64, 3 * 128 + 100, 7 * 128 + 127)]
    _check(w, pols, _sampled_ranges(w.n, 6, 40, 4), "workload4")


# ---- the whole policy grid with reductions only: the launch configuration of workloads 2 and 4 ---------------

def _oracle_stats_threaded(orc, policies, seed, threads=None):
    """The oracle over disjoint request ranges on several host threads (its C library releases the GIL); the
    integer accumulators and histograms merge exactly."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle.binding import merge_stats
    threads = threads or max(1, os.cpu_count() or 1)
    bounds = [orc.n * k // threads for k in range(threads + 1)]
    with ThreadPoolExecutor(threads) as ex:
        parts = list(ex.map(lambda k: orc.eval(policies, seed, bounds[k], bounds[k + 1], finish=False)[0],
                            range(threads)))
    tot = merge_stats(parts)
    orc.finish(tot)
    return tot


@pytest.mark.parametrize("cfg,n", [(2, 6000), (4, 9000)])
def test_whole_policy_grid_against_oracle_on_a_short_trace(cfg, n):
    # all 1024 policies (32 full policy tiles), no per-pair arrays: every statistic and histogram, and the selection
    from parity import check_stats
    w = synth.make_workload(cfg, n=n)
    assert len(w.policies) == 1024
    tr = Trace.from_workload(w)
    tr.eval_policies(w.policies, w.seed)
    gs = tr.reduce_stats()
    orc = Oracle.from_workload(w)
    ostats = _oracle_stats_threaded(orc, w.policies, w.seed)
    check_stats(gs, ostats, tr.histograms, f"grid-config{cfg}")
    cheapest = min(s.total_cost for s in ostats)
    for cap, slo in [(1.25 * cheapest, 0.25), (1.05 * cheapest, 0.25), (1e30, 1e-3)]:
        assert tr.select_policy(cap, slo) == orc.select(ostats, cap, float(np.float32(slo))), (cfg, cap, slo)
    tr.close()


def _select_by_definition(st, cap, slo):
    """Sec. 4.1's objective as this library reads it, written out on the host: feasible = cost within the cap and
    P99 TBT within the objective; best = lowest P99 TTFT bin, then mean TTFT, cost, index; none feasible = cheapest."""
    feas = [p for p in range(len(st)) if st[p].total_cost <= cap and st[p].p99_tbt_s <= np.float32(slo)]
    if feas:
        return 0, min(feas, key=lambda p: (st[p].bin_p99_ttft, st[p].mean_ttft_s, st[p].total_cost, p))
    return -4, min(range(len(st)), key=lambda p: (st[p].total_cost, p))


def test_workload2_full_size_whole_grid_properties():
    w = synth.make_workload(2)
    P, N, sum_n = len(w.policies), w.n, int(w.output_len.sum())
    assert (N, P) == (1_000_000, 1024)
    tr = Trace.from_workload(w)
    tr.eval_policies(w.policies, w.seed)
    st = tr.reduce_stats()
    nb = 256
    for p in range(P):
        s = st[p]
        assert s.n_requests == N and s.n_intervals == sum_n - N
        assert s.n_server_only + s.n_device_only + s.n_race == N
        assert s.tok_server + s.tok_device == sum_n
        assert s.n_device_won <= s.n_device_started and s.n_migrations <= s.n_race
    for p in range(0, P, 37):                                              # no histogram update was lost
        th, bh = tr.histograms(p)
        assert int(th.sum()) == N and int(bh.sum()) == sum_n - N
    for t in range(4):                                                     # per threshold: budgets ascending
        blk = [st[t * nb + k] for k in range(nb)]
        dev_only = [s.n_device_only for s in blk]
        assert all(b <= a for a, b in zip(dev_only, dev_only[1:])) and dev_only[0] == N and dev_only[-1] == 0
        pre_srv = [s.prefill_tok_server for s in blk]
        assert all(b >= a for a, b in zip(pre_srv, pre_srv[1:]))           # the server's input tokens grow with b
        share = [s.prefill_tok_server / float(w.prompt_len.sum()) for s in blk]
        budgets = [w.policies[t * nb + k]["budget"] for k in range(nb)]
        assert all(sh <= b + 1e-12 for sh, b in zip(share, budgets))       # Eq. 3: the share stays within the budget
    # a threshold of +inf never migrates; a lower threshold migrates at least as often
    for k in range(nb):
        migs = [st[t * nb + k].n_migrations for t in range(4)]
        assert migs[3] == 0 and all(b <= a for a, b in zip(migs, migs[1:]))
    cheapest = min(s.total_cost for s in st)
    for cap, slo in [(1.25 * cheapest, 0.25), (1.02 * cheapest, 0.25), (0.5 * cheapest, 0.25), (1e30, 1e-3)]:
        assert tr.select_policy(cap, slo) == _select_by_definition(st, cap, slo), (cap, slo)
    tr.close()


def test_workload2_full_size_against_the_oracle():
    # 10^6 requests x 1024 policies: every counter, both histograms of every policy and the selection against the
    # oracle (about 2e11 token-steps of it, on all host threads), then every field of the pairs of each 64th
    # request under policies that span all four thresholds
    from parity import check_stats
    w = synth.make_workload(2)
    P, N = len(w.policies), w.n
    assert (N, P) == (1_000_000, 1024)
    tr = Trace.from_workload(w)
    tr.eval_policies(w.policies, w.seed)
    gs = tr.reduce_stats()
    orc = Oracle.from_workload(w)
    ostats = _oracle_stats_threaded(orc, w.policies, w.seed)
    check_stats(gs, ostats, tr.histograms, "config2-full")
    cheapest = min(s.total_cost for s in ostats)
    from paper_2502_11417_b200.api import select_policy
    for cap, slo in [(1.25 * cheapest, 0.25), (1.02 * cheapest, 0.25), (0.5 * cheapest, 0.25), (1e30, 1e-3)]:
        want = orc.select(ostats, cap, float(np.float32(slo)))
        assert tr.select_policy(cap, slo) == want and select_policy(gs, cap, slo) == want, (cap, slo)
    sub = [t * 256 + k for t in range(4) for k in (0, 37, 100, 128, 200, 255)]
    pols = [w.policies[p] for p in sub]
    out = tr.alloc_pair_outputs(len(pols))
    tr.eval_policies(pols, w.seed, out)
    tr.reduce_stats()
    cols = np.arange(0, N, 64)
    oout = orc.eval_columns(pols, w.seed, [(int(i), int(i) + 1) for i in cols])
    for f in EXACT_PAIR:
        assert (out[f][:, ::64].cpu().numpy() == oout[f]).all(), f
    for f in FLOAT_PAIR:
        assert rel_close(out[f][:, ::64].cpu().numpy(), oout[f], REL_TOL).all(), f
    assert (oout["mig_at"] > 0).any() and (oout["decision"] == 1).any() and (oout["decision"] == 2).any()
    tr.close()


def test_pair_arrays_beyond_2_32_elements():
    # 4.3 M requests x 1024 policies = 4.4e9 pairs: element indices no longer fit 32 bits, so the row writer runs
    # with 64-bit indices.  Its rows must equal those of two half-grid runs, whose indices do fit ...
    import torch
    w = synth.make_workload(2, n=4_300_000)
    P = len(w.policies)
    assert P * w.n > 2 ** 32 and (P // 2) * w.n < 2 ** 32
    tr = Trace.from_workload(w)
    # ... and the oracle's, every field, on sampled request ranges under all 1024 policies (the arrays are
    # written a few fields at a time: all nine at once would take 136 GB)
    orc = Oracle.from_workload(w)
    ranges = _sampled_ranges(w.n, 6, 24, 12)
    cols = np.concatenate([np.arange(i0, i1) for i0, i1 in ranges])
    oout = orc.eval_columns(w.policies, w.seed, ranges)
    for fields in (["ttft_s", "decision"], ["tbt_mean_s", "delayed"], ["tbt_max_s"], ["cost"], ["tok_server"],
                   ["tok_device"], ["mig_at"]):
        part = tr.alloc_pair_outputs(P, fields=fields)
        tr.eval_policies(w.policies, w.seed, part)
        tr.reduce_stats()
        for f in fields:
            got = torch.stack([part[f][:, i0:i1] for i0, i1 in ranges], 0).permute(1, 0, 2).reshape(P, -1).cpu().numpy()
            assert got.shape == oout[f].shape
            if f in EXACT_PAIR:
                assert (got == oout[f]).all(), f
            else:
                assert rel_close(got, oout[f], REL_TOL).all(), f
        del part
        torch.cuda.empty_cache()
    assert (oout["mig_at"] > 0).any()
    full = tr.alloc_pair_outputs(P, fields=["decision"])
    tr.eval_policies(w.policies, w.seed, full)
    tr.reduce_stats()
    half = tr.alloc_pair_outputs(P // 2, fields=["decision"])
    for lo in (0, P // 2):
        tr.eval_policies(w.policies[lo:lo + P // 2], w.seed, half)
        tr.reduce_stats()
        assert torch.equal(full["decision"][lo:lo + P // 2], half["decision"]), lo
    # and the rows are not trivially constant: budgets 0 and 1 decide differently
    assert int(full["decision"][0].max()) == 1 and int(full["decision"][255].min()) != 1
    tr.close()


@pytest.mark.parametrize("cfg,policy_step", [(3, 1), (4, 1)])
def test_aggregates_on_262144_requests(cfg, policy_step):
    # traces of 2^18 requests with the shape of workloads 3 and 4 under ALL their policies (many chunks, several
    # waves of blocks, six groups and 32 full policy tiles for workload 4): tables, every statistic and histogram
    # against the oracle run on host threads
    from parity import check_stats, check_tables
    w = synth.make_workload(cfg, n=1 << 18)
    pols = w.policies[::policy_step]
    tr = Trace.from_workload(w)
    orc = Oracle.from_workload(w)
    check_tables(tr, orc, f"sub-config{cfg}")
    tr.eval_policies(pols, w.seed)
    gs = tr.reduce_stats()
    ostats = _oracle_stats_threaded(orc, pols, w.seed)
    check_stats(gs, ostats, tr.histograms, f"sub-config{cfg}")
    cheapest = min(s.total_cost for s in ostats)
    assert tr.select_policy(1.25 * cheapest, 0.25) == orc.select(ostats, 1.25 * cheapest, float(np.float32(0.25)))
    tr.close()
