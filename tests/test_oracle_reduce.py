"""Pins for the oracle's reductions and policy selection."""
import ctypes as C

import numpy as np
import pytest

from oracle import lib, OracleStats, NBINS
from oracle.binding import merge_stats
from paper_2502_11417_b200 import synth
from helpers import oracle_of

L = lib()


def test_histogram_totals_and_exact_quantiles():
    w = synth.make_workload(1, n=6000)
    o = oracle_of(vars(w))
    pols = [synth.policy(b, flags=f) for b in (0.0, 0.4, 1.0)
            for f in (synth.FLAG_MIGRATION | synth.FLAG_PACING, synth.FLAG_MIGRATION)]
    st, out = o.eval(pols, w.seed, pairs=True, exact=True)
    n_int = int((w.output_len - 1).sum())
    for p in range(len(pols)):
        s = st[p]
        th, bh = np.ctypeslib.as_array(s.ttft_hist), np.ctypeslib.as_array(s.tbt_hist)
        assert th.sum() == w.n == s.n_requests and bh.sum() == n_int == s.n_intervals
        t = np.rint(out["ttft_s"][p] * 1e6).astype(np.int64)
        assert (th == np.bincount([L.orc_bin(int(v)) for v in t], minlength=NBINS)).all()
        srt = np.sort(t)
        for q, b, v, ex in [(0.5, s.bin_p50_ttft, s.p50_ttft_s, s.exact_p50_ttft_s),
                            (0.95, s.bin_p95_ttft, s.p95_ttft_s, s.exact_p95_ttft_s),
                            (0.99, s.bin_p99_ttft, s.p99_ttft_s, s.exact_p99_ttft_s)]:
            want = srt[int(np.ceil(q * w.n)) - 1]               # nearest rank
            assert abs(ex - want * 1e-6) < 1e-12
            assert L.orc_bin(int(want)) == b                    # the exact order statistic lies in the reported bin
            assert v == L.orc_bin_lower_edge(b) * 1e-6 and v <= ex < v * (1 + 1 / 32) + 32e-6
        assert L.orc_bin(int(round(s.exact_p99_tbt_s * 1e6))) == s.bin_p99_tbt
        assert abs(s.mean_ttft_s - (t * 1e-6).mean()) < 1e-12
        assert s.n_server_only + s.n_device_only + s.n_race == w.n
        assert s.tok_server + s.tok_device == int(w.output_len.sum())
        assert s.tok_server == int(out["tok_server"][p].sum()) and s.delayed_tokens == int(out["delayed"][p].sum())
        assert s.n_migrations == int((out["mig_at"][p] > 0).sum())
    # with pacing at 5 tokens/s and both endpoints faster than that, the pooled P99 TBT sits at 1/r_c
    assert st[0].exact_p99_tbt_s == pytest.approx(0.2, abs=1e-9)
    # without pacing the TBTs are the generation intervals
    assert st[1].exact_p99_tbt_s < 0.2


def test_nearest_rank_at_a_bin_boundary():
    # four requests, each alone in its TTFT bin, all served by the server (device-constrained, b = 0): rank
    # ceil(0.5 * 4) = 2 is reached exactly at the end of the second bin, ceil(0.95 * 4) = ceil(0.99 * 4) = 4 at the last
    from helpers import constructed
    ttft = np.array([0.008, 0.001, 0.004, 0.002], dtype=np.float32)
    tr = constructed([50, 60, 70, 80], [3, 4, 5, 6], ttft)
    o = oracle_of(tr)
    st, _ = o.eval([synth.policy(0.0, flags=synth.FLAG_PACING | synth.MODE_DEVICE_CONSTRAINED)], 1)
    s = st[0]
    assert s.n_server_only == 4
    assert (s.bin_p50_ttft, s.bin_p95_ttft, s.bin_p99_ttft) == (L.orc_bin(2000), L.orc_bin(8000), L.orc_bin(8000))
    assert s.p50_ttft_s == L.orc_bin_lower_edge(L.orc_bin(2000)) * 1e-6
    # pooled TBTs: 3 + 4 + 5 + 2 = 14 intervals of exactly tau = 200,000 ticks
    assert s.n_intervals == 14 and s.bin_p99_tbt == L.orc_bin(200000)


def test_range_split_merges_exactly():
    w = synth.make_workload(1, n=2000)
    o = oracle_of(vars(w))
    pols = [synth.policy(b) for b in (0.2, 0.8)]
    full, _ = o.eval(pols, 3)
    a, _ = o.eval(pols, 3, 0, 700, finish=False)
    b, _ = o.eval(pols, 3, 700, 2000, finish=False)
    tot = merge_stats([a, b])
    o.finish(tot)
    for p in range(2):
        for f, _t in OracleStats._fields_:
            x, y = getattr(full[p], f), getattr(tot[p], f)
            if f.endswith("_hist"):
                assert list(x) == list(y)
            elif f.startswith("exact"):
                continue
            elif isinstance(x, float):
                assert x == pytest.approx(y, rel=1e-12)
            else:
                assert x == y, f


def _brute_select(rows, cap, slo):
    feas = [(r[0], r[1], r[2], k) for k, r in enumerate(rows) if r[2] <= cap and r[3] <= slo]
    if feas:
        return 0, min(feas)[3]
    return -4, min((r[2], k) for k, r in enumerate(rows))[1]


@pytest.mark.parametrize("seed", range(10))
def test_selection_brute_force_with_ties(seed):
    rng = np.random.default_rng(seed)
    P = int(rng.integers(1, 17))
    # few distinct values per column so that ties occur at every level
    rows = [(float(rng.choice([1.0, 1.5, 2.0])), float(rng.choice([0.4, 0.5])), float(rng.choice([10.0, 20.0, 30.0])),
             float(rng.choice([0.19, 0.3]))) for _ in range(P)]
    st = (OracleStats * P)()
    for k, (p99, mean, cost, tbt) in enumerate(rows):
        st[k].p99_ttft_s, st[k].mean_ttft_s, st[k].total_cost, st[k].p99_tbt_s = p99, mean, cost, tbt
    for cap, slo in [(25.0, 0.25), (5.0, 0.25), (100.0, 0.1), (100.0, 1.0), (10.0, 0.19)]:
        best = C.c_int32(-1)
        rc = L.orc_select(C.cast(st, C.c_void_p), P, cap, slo, C.byref(best))
        assert (rc, best.value) == _brute_select(rows, cap, slo)
