"""One trace evaluated as request-range shards in several contexts on one GPU: the shards' accumulators add up
to exactly what a single context holding the whole trace produces, and to the oracle's numbers (needs a GPU)."""
import numpy as np
import pytest

from oracle import Oracle
from paper_2502_11417_b200 import synth, Trace, DiscoError
from paper_2502_11417_b200.api import select_policy
from parity import check_stats, check_pairs, check_tables, check_prep

pytestmark = pytest.mark.gpu

MIG, PACE = synth.FLAG_MIGRATION, synth.FLAG_PACING


def _load_shard(w, i0, i1):
    return Trace().load_trace(w.prompt_len[i0:i1], w.output_len[i0:i1], w.server_ttft_s[i0:i1],
                              w.server_profile[i0:i1], w.device_profile[i0:i1], w.servers, w.devices,
                              first_index=i0)


def _whole_tables(shards, G):
    """Sum of the shards' length histograms; their sorted ticks one after the other, group by group."""
    cnt = np.zeros((G, 4097), np.int64)
    ticks, n_ticks = [], np.zeros(G, np.uint64)
    for g in range(G):
        for t in shards:
            c, _, s = t.group_tables(g)
            cnt[g] += c
            ticks.append(s)
            n_ticks[g] += len(s)
    return cnt, np.concatenate(ticks).astype(np.int32), n_ticks


def _policies():
    pols = [synth.policy(b, mig_threshold=th) for th in (0.0, 0.05, synth.INF) for b in synth.budget_grid(9)]
    pols += [synth.policy(b, flags=synth.FLAG_STOCHASTIC | PACE | md) for b in (0.3, 0.8)
             for md in (synth.MODE_AUTO, synth.MODE_DEVICE_CONSTRAINED)]        # routing draw keyed by the global index
    pols += [synth.policy(0.4, flags=synth.FLAG_BETA_RULE | MIG | PACE, l_immediate=30),
             synth.policy(0.6, r_c=30.0, t_m_s=0.3), synth.policy(0.7, flags=MIG)]   # a second and third timeline class
    return pols


@pytest.mark.parametrize("cuts", [(0.5,), (0.13, 0.61, 0.62)])
def test_shards_add_up_to_the_single_context_run(cuts):
    w = synth.make_workload(4, n=30_011, n_budgets=5)
    pols = _policies()
    P, G = len(pols), len(w.servers) * len(w.devices)
    bounds = [0] + [int(c * w.n) for c in cuts] + [w.n]
    whole = Trace.from_workload(w)
    whole_out = whole.alloc_pair_outputs(P)
    whole.eval_policies(pols, w.seed, whole_out)
    ws = whole.reduce_stats()

    shards = [_load_shard(w, a, b) for a, b in zip(bounds, bounds[1:])]
    cnt, ticks, n_ticks = _whole_tables(shards, G)
    words = None
    for k, (t, a, b) in enumerate(zip(shards, bounds, bounds[1:])):
        t.set_group_tables(cnt, ticks, n_ticks)
        out = t.alloc_pair_outputs(P)
        t.eval_policies(pols, w.seed, out)
        for f in out:                                  # a shard's pairs are the whole run's columns a..b
            assert (out[f].cpu().numpy() == whole_out[f][:, a:b].cpu().numpy()).all(), (k, f)
        part = t.export_accumulators()
        assert part.size == t.accumulator_words() == P * G * 12 + 2 * P * 864 + 2 * G
        words = part if words is None else words + part
    first = shards[0]
    first.import_accumulators(words)
    ms = first.reduce_stats()
    for p in range(P):
        assert bytes(ms[p]) == bytes(ws[p]), p          # bit for bit the single context's records
    # ... and the oracle's
    orc = Oracle.from_workload(w)
    check_tables(first, orc, "shards")                  # the tables a shard was given are the whole trace's
    check_prep(first, orc, pols, "shards")
    ostats, oout = orc.eval(pols, w.seed, pairs=True)
    check_stats(ms, ostats, first.histograms, "shards")
    check_pairs(whole_out, oout, tag="whole")
    cheapest = min(s.total_cost for s in ostats)
    for cap, slo in [(1.25 * cheapest, 0.25), (0.5 * cheapest, 0.25), (1e30, 1e-3)]:
        assert select_policy(ms, cap, slo) == orc.select(ostats, cap, float(np.float32(slo)))
    # a later evaluation in the context that took the import refers to its own requests again
    first.eval_policies(pols[:3], w.seed)
    again = first.reduce_stats()
    assert again[0].n_requests == bounds[1] and again[0].n_intervals == int(w.output_len[:bounds[1]].sum()) - bounds[1]
    for t in shards + [whole]:
        t.close()


def test_device_resident_ticks_and_words():
    import torch
    w = synth.make_workload(1, n=20_000, n_budgets=6)
    whole = Trace.from_workload(w)
    whole.eval_policies(w.policies, 3)
    ws = whole.reduce_stats()
    k = 7_777
    a, b = _load_shard(w, 0, k), _load_shard(w, k, w.n)
    cnt, ticks, n_ticks = _whole_tables([a, b], 1)
    dev_ticks = torch.from_numpy(ticks).cuda()
    total = None
    for t in (a, b):
        t.set_group_tables(cnt, dev_ticks, n_ticks)
        t.eval_policies(w.policies, 3)
        buf = torch.empty(t.accumulator_words(), dtype=torch.int64, device="cuda")
        t.export_accumulators(buf)
        total = buf if total is None else total + buf          # what an all-reduce (sum) would leave on every rank
    b.import_accumulators(total)
    ms = b.reduce_stats()
    for p in range(len(w.policies)):
        assert bytes(ms[p]) == bytes(ws[p]), p


def test_tables_are_checked():
    w = synth.make_workload(1, n=2_000, n_budgets=2)
    t = Trace.from_workload(w)
    cnt, _, srt = t.group_tables(0)
    n = np.array([len(srt)], np.uint64)
    bad = cnt.copy(); bad[17] += 1
    with pytest.raises(DiscoError) as ei:
        t.set_group_tables(bad[None, :], srt, n)
    assert ei.value.code == -1
    neg = srt.copy(); neg[5] = -3
    with pytest.raises(DiscoError) as ei:
        t.set_group_tables(cnt[None, :], neg, n)
    assert ei.value.code == -1
    with pytest.raises(DiscoError):
        t.eval_policies(w.policies, 0)                 # the context must be reloaded after a refused table
    t2 = Trace.from_workload(w)
    t2.set_group_tables(cnt[None, :], srt[::-1].copy(), n)      # any order within the group
    t2.eval_policies(w.policies, 1)
    s2 = t2.reduce_stats()
    t3 = Trace.from_workload(w)
    t3.eval_policies(w.policies, 1)
    s3 = t3.reduce_stats()
    assert bytes(s2[0]) == bytes(s3[0]) and bytes(s2[1]) == bytes(s3[1])
    with pytest.raises(DiscoError):
        Trace().load_trace(w.prompt_len, w.output_len, w.server_ttft_s, None, None, w.servers, w.devices,
                           first_index=(1 << 32) - 100)
