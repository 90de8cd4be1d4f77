"""Pins for the oracle's dispatch controller: Algorithms 1-3, Eq. 3, the wait-then-race rule (Sec. 4.2)."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import SERVER_ONLY, DEVICE_ONLY, RACE
from paper_2502_11417_b200 import synth
from helpers import constructed, oracle_of

F32 = np.float32
S_MODE = synth.FLAG_MIGRATION | synth.FLAG_PACING | synth.MODE_SERVER_CONSTRAINED
D_MODE = synth.FLAG_MIGRATION | synth.FLAG_PACING | synth.MODE_DEVICE_CONSTRAINED


def test_algorithm1_mode_from_costs():
    tr = constructed([10, 20], [5, 5], [0.3, 0.4])
    cases = [  # (c_s prefill, decode, c_d prefill, decode, lambda) -> device-constrained?
        (1e-3, 1e-3, 0.2e-3, 0.2e-3, 1.0, False),
        (1e-3, 1e-3, 5e-3, 5e-3, 1.0, True),
        (1e-3, 2e-3, 3e-3, 1.5e-3, 1.0, False),      # min device 1.5e-3 is not above max server 2e-3
        (1e-3, 2e-3, 3e-3, 2.5e-3, 1.0, True),
        (1e-3, 1e-3, 0.2e-3, 0.2e-3, 10.0, True),    # the exchange rate prices the device above the server
        (1e-3, 1e-3, 1e-3, 1e-3, 1.0, False),        # equality is not "greater"
    ]
    for cps, cds, cpd, cdd, lam, want in cases:
        tr["servers"] = [synth.server(c_prefill=cps, c_decode=cds)]
        tr["devices"] = [synth.device(500.0, 20.0, c_prefill=cpd, c_decode=cdd, lam=lam)]
        o = oracle_of(tr)
        assert bool(o.prep(synth.policy(0.5)).device_constrained) == want
        assert o.prep(synth.policy(0.5, flags=D_MODE)).device_constrained == 1
        assert o.prep(synth.policy(0.5, flags=S_MODE)).device_constrained == 0


def _brute_l_th(lengths, b):
    """Smallest threshold whose concurrent (server) share of input tokens is at most b (exact rationals)."""
    total = sum(lengths)
    for L in range(0, 4098):
        server_share = sum(l for l in lengths if l >= L)
        if Fraction(server_share) <= Fraction(b) * total:
            return L
    raise AssertionError


@pytest.mark.parametrize("seed", range(6))
def test_algorithm3_threshold_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 9))
    lengths = [int(v) for v in rng.integers(1, 30, size=n)]
    o = oracle_of(constructed(lengths, [4] * n, [0.5] * n))
    for b in [0.0, 0.125, 0.25, 0.375, 0.5, 0.625, 0.75, 0.875, 1.0]:
        pr = o.prep(synth.policy(b, flags=S_MODE))
        want = _brute_l_th(lengths, Fraction(b))
        # thresholds between two occupied lengths route identically: compare the routing
        for l in lengths:
            assert (l < pr.l_th) == (l < want), (lengths, b, pr.l_th, want)


def test_algorithm3_limits_and_share():
    w = synth.make_workload(1, n=5000)
    o = oracle_of(vars(w))
    total = int(w.prompt_len.sum())
    prev = -1
    for b in synth.budget_grid(17):
        st, out = o.eval([synth.policy(b, flags=S_MODE)], 0, pairs=True)
        dec = out["decision"][0]
        assert not (dec == SERVER_ONLY).any() or b > 0      # with w = 0 the device always starts unless S = 0
        server_tokens = int(w.prompt_len[dec != DEVICE_ONLY].sum())
        assert st[0].prefill_tok_server >= server_tokens   # migrations to the server may add re-prefills
        assert Fraction(server_tokens) <= Fraction(float(F32(b))) * total       # share <= b exactly
        assert server_tokens >= prev                                          # non-decreasing in b
        prev = server_tokens
        if b == 0.0:
            assert (dec == DEVICE_ONLY).all()          # all-device limit (the llama.cpp baseline)
        if b == 1.0:
            assert (dec != DEVICE_ONLY).all()
        # Algorithm 3 routes by length only
        l_th = o.prep(synth.policy(b, flags=S_MODE)).l_th
        assert ((w.prompt_len < l_th) == (dec == DEVICE_ONLY)).all()


def test_algorithm2_tail_phase_and_limits():
    w = synth.make_workload(1, n=4000)
    tr = vars(w)
    tr["devices"] = [synth.device(500.0, 20.0, c_prefill=5e-3, c_decode=5e-3)]
    o = oracle_of(tr)
    cnt, srt, kn = o.group_tables(0)
    N = len(srt)
    alpha = 0.05
    for b in [0.0, 0.01, 0.03, 0.05]:
        pr = o.prep(synth.policy(b, alpha=alpha))
        assert pr.device_constrained == 1
        # b <= alpha: every length waits F^-1(1 - b)
        rank = int(np.ceil((1.0 - float(F32(b))) * N)) - 1
        assert pr.w_tail == srt[min(max(rank, 0), N - 1)]
        assert pr.l_star == 0 and pr.w_star == pr.w_tail
    # b = 0: the wait is the largest server TTFT, the device never starts: the all-server baseline (vLLM)
    st, out = o.eval([synth.policy(0.0)], 0, pairs=True)
    assert (out["decision"][0] == SERVER_ONLY).all() and st[0].n_device_started == 0
    assert st[0].tok_device == 0 and st[0].tok_server == int(w.output_len.sum())
    ticks = np.rint(w.server_ttft_s.astype(np.float64) * 1e6)
    assert np.allclose(out["ttft_s"][0], ticks * 1e-6, rtol=0, atol=1e-12)
    # b = 1: every wait is zero
    pr = o.prep(synth.policy(1.0))
    assert pr.l_star == 4097
    st, out = o.eval([synth.policy(1.0)], 0, pairs=True)
    assert (out["decision"][0] == RACE).all()


def test_algorithm2_funding_identity_and_monotone_waits():
    w = synth.make_workload(1, n=3000)
    tr = vars(w)
    tr["devices"] = [synth.device(500.0, 20.0, c_prefill=5e-3, c_decode=5e-3)]
    o = oracle_of(tr)
    cnt, srt, kn = o.group_tables(0)
    total = int((np.arange(4097) * cnt).sum())
    alpha = 0.05
    lens = np.unique(w.prompt_len)
    prev_wait = None
    for b in synth.budget_grid(33):
        pr = o.prep(synth.policy(b, alpha=alpha))
        waits = np.where(lens < pr.l_star, 0, np.where(lens == pr.l_star, pr.w_star, pr.w_tail))
        if prev_wait is not None:
            assert (waits <= prev_wait).all()        # a larger budget never lengthens a wait
        prev_wait = waits
        if float(F32(b)) > float(F32(alpha)) and pr.l_star <= 4096:
            ls = pr.l_star
            below = int((np.arange(ls) * cnt[:ls]).sum())
            A = (float(F32(b)) - float(F32(alpha))) / (1.0 - float(F32(alpha))) * total
            assert cnt[ls] > 0
            assert below <= A < below + ls * cnt[ls]
            assert 0.0 <= pr.funded_fraction < 1.0
            assert abs(below + pr.funded_fraction * ls * cnt[ls] - A) <= 1e-6 * max(A, 1.0)
            # F(w*) = (1 - alpha)(1 - f): the partly funded class starts the device with probability alpha + f(1 - alpha)
            q = (1.0 - float(F32(alpha))) * (1.0 - pr.funded_fraction)
            assert pr.w_star == srt[min(max(int(np.ceil(q * len(srt))) - 1, 0), len(srt) - 1)]
            assert 0 <= pr.w_star <= pr.w_tail


def test_algorithm2_wait_map_as_played():
    # three length classes of 200 requests: every request must wait W[l] (0 below l*, w* in the partly funded class,
    # w_tail above), i.e. the device starts exactly when the server's first token comes later than that
    from helpers import constructed
    rng = np.random.default_rng(12)
    lens = np.repeat([64, 128, 256], 200)
    ttft = rng.lognormal(-1.0, 0.6, size=600).astype(np.float32)
    tr = constructed(lens, rng.integers(2, 40, size=600), ttft,
                     devices=[synth.device(500.0, 20.0, c_prefill=5e-3, c_decode=5e-3)])
    o = oracle_of(tr)
    ticks = np.rint(ttft.astype(np.float64) * 1e6).astype(np.int64)
    partly = 0
    for b in (0.1, 0.3, 0.5, 0.7, 0.9):
        pol = synth.policy(b, flags=synth.FLAG_PACING)
        pr = o.prep(pol)
        assert pr.device_constrained and pr.l_star in (64, 128, 256)
        wait = np.where(lens < pr.l_star, 0, np.where(lens == pr.l_star, pr.w_star, pr.w_tail))
        st, out = o.eval([pol], 0, pairs=True)
        started = out["decision"][0] == RACE
        assert (started == (ticks > wait)).all() and not (out["decision"][0] == 1).any()
        in_class = lens == pr.l_star
        if 0 < pr.w_star < pr.w_tail and started[in_class].any() and (~started[in_class]).any():
            partly += 1
            # with the tail wait instead of w*, fewer of this class would have started
            assert (ticks[in_class] > pr.w_star).sum() > (ticks[in_class] > pr.w_tail).sum()
    assert partly >= 3


def test_algorithm2_realised_device_share_tracks_budget():
    # E[I_d(l) l] <= b E[l] (Sec. 4.2): statistical, since the wait is set from the trace's own TTFT quantiles
    w = synth.make_workload(1, n=40000)
    tr = vars(w)
    tr["devices"] = [synth.device(500.0, 20.0, c_prefill=5e-3, c_decode=5e-3)]
    o = oracle_of(tr)
    total = float(w.prompt_len.sum())
    for b in [0.02, 0.05, 0.2, 0.5, 0.8]:
        st, _ = o.eval([synth.policy(b, flags=synth.FLAG_PACING)], 0)    # migration off: prefill tokens = started only
        share = st[0].prefill_tok_device / total
        assert abs(share - b) < 0.02, (b, share)


def test_profile_ids_select_their_own_endpoints():
    # 2 server x 3 device profiles, no jitter, no pacing: a request's device TTFT and its inter-token interval are
    # those of the profiles it names (group = server id * number of devices + device id)
    srv = [synth.server(tbt_s=0.030), synth.server(tbt_s=0.045)]
    dev = [synth.device(500.0, 20.0), synth.device(250.0, 10.0, ttft_intercept_s=0.02), synth.device(1000.0, 40.0)]
    sp = np.array([0, 0, 0, 1, 1, 1] * 2, np.uint8)
    dp = np.array([0, 1, 2, 0, 1, 2] * 2, np.uint8)
    ttft = np.array([1e-6] * 6 + [100.0] * 6, np.float32)              # the server wins the first six races, the device the others
    tr = constructed([100] * 12, [11] * 12, ttft, servers=srv, devices=dev, sprof=sp, dprof=dp)
    o = oracle_of(tr)
    _, out = o.eval([synth.policy(1.0, flags=synth.MODE_SERVER_CONSTRAINED)], 0, pairs=True)
    kappa, c0 = np.array([2000, 4000, 1000]), np.array([0, 20000, 0])
    T_srv, T_dev = np.array([30000, 45000]), np.array([50000, 100000, 25000])
    assert (out["decision"][0] == RACE).all()
    assert np.allclose(out["ttft_s"][0][6:], (kappa[dp[6:]] * 100 + c0[dp[6:]]) * 1e-6, rtol=0, atol=1e-12)
    assert np.allclose(out["tbt_mean_s"][0][:6], T_srv[sp[:6]] * 1e-6, rtol=0, atol=1e-12)
    assert np.allclose(out["tbt_mean_s"][0][6:], T_dev[dp[6:]] * 1e-6, rtol=0, atol=1e-12)


def test_race_rule_and_tie():
    # device: 2000 ticks per prompt token + 10000 intercept; prompt 45 -> Td = 100000 ticks
    dev = [synth.device(500.0, 20.0, ttft_intercept_s=0.01)]
    S = [0.099999, 0.1, 0.100001, 0.05, 0.5]
    o = oracle_of(constructed([45] * 5, [3] * 5, S, devices=dev))
    pol = synth.policy(1.0, flags=S_MODE)                 # all race, w = 0
    for i, s in enumerate(S):
        r = o.play(pol, 0, i)
        st = int(round(s * 1e6))
        assert r["decision"] == RACE
        assert r["ttft"] == min(st, 100000)
        assert r["winner_is_device"] == (st > 100000)     # a tie at exactly 100000 goes to the server
    # wait-then-race in the device-constrained mode with a known wait
    n = 200
    rng = np.random.default_rng(3)
    ttft = rng.uniform(0.05, 2.0, size=n)
    dev = [synth.device(500.0, 20.0, c_prefill=5e-3, c_decode=5e-3)]
    tr = constructed(rng.integers(1, 400, size=n), [4] * n, ttft, devices=dev)
    o = oracle_of(tr)
    for b in [0.03, 0.3, 0.7]:
        pol = synth.policy(b)
        pr = o.prep(pol)
        st, out = o.eval([pol], 0, pairs=True)
        Sx = np.rint(tr["server_ttft_s"].astype(np.float64) * 1e6).astype(np.int64)
        l = tr["prompt_len"].astype(np.int64)
        wv = np.where(l < pr.l_star, 0, np.where(l == pr.l_star, pr.w_star, pr.w_tail))
        Td = 2000 * l
        started = Sx > wv
        want = np.where(started, np.minimum(Sx, wv + Td), Sx)
        assert (np.rint(out["ttft_s"][0] * 1e6).astype(np.int64) == want).all()
        assert ((out["decision"][0] == RACE) == started).all()
        # TTFT never exceeds the better endpoint's TTFT plus the wait
        assert (want <= np.minimum(Sx, Td) + wv).all()
        assert st[0].n_device_started == int(started.sum())
        assert st[0].n_device_won == int((started & (Sx > wv + Td)).sum())


def test_inverse_cdf_nearest_rank():
    # F^-1(q) = smallest sample whose empirical CDF reaches q
    S = [0.4, 0.1, 0.3, 0.2]
    o = oracle_of(constructed([5] * 4, [3] * 4, S))
    ticks = [100000, 200000, 300000, 400000]
    for q, want in [(0.0, 0), (0.1, 0), (0.25, 0), (0.26, 1), (0.5, 1), (0.51, 2), (0.75, 2), (0.76, 3), (1.0, 3)]:
        assert o.inverse_cdf(0, q) == ticks[want], q
    for q in np.linspace(0, 1, 41):
        v = o.inverse_cdf(0, float(q))
        assert sum(t <= v for t in ticks) / 4 >= q - 1e-12            # F(F^-1(q)) >= q ...
        assert all(sum(t <= u for t in ticks) / 4 < q for u in ticks if u < v)   # ... and no smaller sample does
