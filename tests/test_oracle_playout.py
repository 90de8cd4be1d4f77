"""Pins for the oracle's token play-out: paced delivery, buffer-based migration (Sec. 4.3, Eq. 4-6), cost (Eq. 8)."""
import math

import numpy as np
import pytest

from oracle import lib, RACE
from paper_2502_11417_b200 import synth
from helpers import constructed, oracle_of, read_golden

L = lib()
S_MODE = synth.MODE_SERVER_CONSTRAINED
D_MODE = synth.MODE_DEVICE_CONSTRAINED
MIG, PACE = synth.FLAG_MIGRATION, synth.FLAG_PACING


def fifo_delivery(g, tau):
    """Event-driven delivery buffer: generated tokens queue up in a FIFO; the reader takes the head token as soon
    as one is queued and at least tau has passed since its previous token."""
    import collections
    fifo, out, arrived, ready = collections.deque(), [], 0, None
    while len(out) < len(g):
        if not fifo:                                   # reader idles until the next token is generated
            fifo.append(g[arrived]); arrived += 1
        t = fifo[0] if ready is None else max(fifo[0], ready)
        while arrived < len(g) and g[arrived] <= t:    # tokens generated meanwhile join the queue
            fifo.append(g[arrived]); arrived += 1
        fifo.popleft()
        out.append(t)
        ready = t + tau
    return out


@pytest.mark.parametrize("T_s,r_c", [(0.030, 5.0), (0.150, 5.0), (0.200, 5.0), (0.350, 5.0)])
def test_constant_rate_closed_forms(T_s, r_c):
    n = 40
    o = oracle_of(constructed([100], [n], [0.1], servers=[synth.server(tbt_s=T_s)],
                              devices=[synth.device(1.0, 20.0)]))      # device far too slow: server wins
    T, tau = int(round(T_s * 1e6)), int(round(1e6 / r_c))
    r = o.play(synth.policy(1.0, flags=S_MODE), 0, 0)                   # pacing off
    assert not r["winner_is_device"]
    assert list(r["g"][1:]) == [j * T for j in range(n)] and list(r["d"][1:]) == list(r["g"][1:])
    r = o.play(synth.policy(1.0, r_c=r_c, flags=S_MODE | PACE), 0, 0)    # pacing on
    if T <= tau:
        assert list(r["d"][1:]) == [j * tau for j in range(n)]          # every TBT = 1/r_c (Table 3's constant P99)
    else:
        assert list(r["d"][1:]) == list(r["g"][1:])                     # generation is the bottleneck


@pytest.mark.parametrize("seed", range(5))
def test_delivery_against_max_plus_and_fifo(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(2, 60))
    tbt = float(rng.choice([0.03, 0.18, 0.21, 0.3]))
    o = oracle_of(constructed([50], [n], [0.1], servers=[synth.server(tbt_s=tbt, jitter=0.6)],
                              devices=[synth.device(1.0, 20.0)]))
    tau = 200000
    r = o.play(synth.policy(1.0, flags=S_MODE | PACE), seed, 0)
    g, d = [int(v) for v in r["g"][1:]], [int(v) for v in r["d"][1:]]
    T, J = int(round(tbt * 1e6)), int(round(tbt * 1e6 * float(np.float32(0.6))))
    # the generation times are the prefix sums of T + jitter(hash(seed, request, token))
    want_g = [0]
    for j in range(2, n + 1):
        want_g.append(want_g[-1] + T + L.orc_jitter(L.orc_hash(seed, 0, j), J))
    assert g == want_g
    # max-plus closed form of the paced recurrence
    assert d == [j * tau + max(g[k] - k * tau for k in range(j + 1)) for j in range(n)]
    assert d == fifo_delivery(g, tau)


def test_buffer_migration_worked_example():
    dev = [synth.device(200.0, 10.0)]                                  # phone: 5000 ticks/prompt token, 100000/token
    for l, m, M, delayed, tbt_max in read_golden("buffer_worked_example.txt"):
        # S = 1 tick < Td: the (dearer) server wins the race at once
        o = oracle_of(constructed([int(l)], [60], [1e-6], devices=dev))
        pol = synth.policy(1.0, t_m_s=1.0, r_c=5.0, flags=S_MODE | MIG | PACE)
        assert o.prep(pol).B == 5
        r = o.play(pol, 0, 0)
        assert r["decision"] == RACE and not r["winner_is_device"]
        assert r["mig_at"] == int(m) and r["mig_latency"] == int(M) and r["delayed"] == int(delayed)
        d = r["d"]
        assert max(int(d[j] - d[j - 1]) for j in range(2, 61)) == int(tbt_max)
        st, out = o.eval([pol], 0, pairs=True)
        assert out["mig_at"][0, 0] == int(m) and out["delayed"][0, 0] == int(delayed)
        assert out["tok_server"][0, 0] == int(m) and out["tok_device"][0, 0] == 60 - int(m)
        assert abs(out["tbt_max_s"][0, 0] - int(tbt_max) * 1e-6) < 1e-12


def test_per_request_tbt_mean_and_max_at_constant_rate():
    # no jitter, no migration: paced delivery at tau = 200,000 ticks gives every interval tau (Table 3's constant
    # TBT); unpaced delivery gives the winner's generation interval.  The mean is over the n - 1 intervals.
    tr = constructed([100, 100, 3000, 3000], [2, 9, 2, 33], [1e-6, 1e-6, 10.0, 10.0])   # the server wins the short prompts' race, the device (6 s) the long ones'
    o = oracle_of(tr)
    for flags, want in ((PACE | S_MODE, (0.2, 0.2, 0.2, 0.2)), (S_MODE, (0.03, 0.03, 0.05, 0.05))):
        _, out = o.eval([synth.policy(1.0, flags=flags)], 0, pairs=True)
        assert list(out["decision"][0]) == [RACE] * 4
        assert np.allclose(out["tbt_mean_s"][0], want, rtol=0, atol=1e-12)
        assert np.allclose(out["tbt_max_s"][0], want, rtol=0, atol=1e-12)
    one = oracle_of(constructed([100], [1], [1e-6]))
    _, out = one.eval([synth.policy(1.0, flags=PACE | S_MODE)], 0, pairs=True)
    assert out["tbt_mean_s"][0, 0] == 0.0 and out["tbt_max_s"][0, 0] == 0.0      # a single token has no interval


def test_migration_invariants_over_modes_and_flags():
    # only a raced request with at least two tokens may hand over; without pacing there is no slot to be late for
    # and delivery is generation, before and after a hand-off
    for dear in (False, True):
        w = synth.tiny_workload(23 + dear, 400, n_servers=2, n_devices=2, max_prompt=300, max_out=30, device_dearer=dear)
        w.output_len[::7] = 1
        o = oracle_of(vars(w))
        pols = [synth.policy(b, flags=f | md, expected_len=E, t_m_s=tm)
                for b in (0.0, 0.5, 1.0) for f in (MIG, MIG | PACE) for md in (S_MODE, D_MODE) for E in (0, 128)
                for tm in (0.0, 1.0)]
        st, out = o.eval(pols, 5, pairs=True)
        some = 0
        for p, pol in enumerate(pols):
            mig = out["mig_at"][p] > 0
            some += int(mig.sum())
            assert (out["decision"][p][mig] == RACE).all()
            assert not mig[w.output_len == 1].any()
            if not pol["flags"] & PACE:
                assert (out["delayed"][p] == 0).all() and st[p].delayed_tokens == 0
                for i in np.flatnonzero(mig)[:5]:
                    r = o.play(pol, 5, int(i))
                    assert r["mig_at"] == 1 and list(r["d"][1:]) == list(r["g"][1:])
        assert some > 100


def test_handoff_at_the_last_token_that_leaves_one_to_generate():
    # the worked example's stream fills its buffer of 5 at token 6: an output of 7 tokens still hands over (one
    # token is left for the device), an output of 6 tokens does not (nothing would remain)
    dev = [synth.device(200.0, 10.0)]
    pol = synth.policy(1.0, t_m_s=1.0, r_c=5.0, flags=S_MODE | MIG | PACE)
    for n, want_m in ((8, 6), (7, 6), (6, 0), (5, 0)):
        o = oracle_of(constructed([100], [n], [1e-6], devices=dev))
        r = o.play(pol, 0, 0)
        assert r["decision"] == RACE and not r["winner_is_device"]
        assert r["mig_at"] == want_m, (n, r["mig_at"])
        st, out = o.eval([pol], 0, pairs=True)
        assert out["tok_server"][0, 0] == (want_m or n) and out["tok_device"][0, 0] == n - (want_m or n)


@pytest.mark.parametrize("T,tau,t_m,T_tgt,kappa,l,n", [
    (30000, 200000, 1_000_000, 100000, 5000, 100, 50), (30000, 200000, 1_000_000, 100000, 5000, 400, 50),
    (30000, 200000, 1_000_000, 100000, 5000, 400, 12), (50000, 100000, 700_000, 20000, 2000, 300, 80),
    (150000, 200000, 400_000, 50000, 667, 2000, 64), (30000, 200000, 0, 100000, 5000, 50, 9)])
def test_migration_closed_form_without_jitter(T, tau, t_m, T_tgt, kappa, l, n):
    srv = [synth.server(tbt_s=T * 1e-6)]
    dev = [synth.device(1e6 / kappa, 1e6 / T_tgt)]
    o = oracle_of(constructed([l], [n], [1e-6], servers=srv, devices=dev))
    pol = synth.policy(1.0, t_m_s=t_m * 1e-6, r_c=1e6 / tau, flags=S_MODE | MIG | PACE)
    B = -(-t_m // tau)
    assert o.prep(pol).B == B
    r = o.play(pol, 0, 0)
    # occupancy when token j is generated: j tokens generated, 1 + floor(g_j / tau) delivered
    m = 1 if B == 0 else next((j for j in range(B, n) if j - 1 - ((j - 1) * T) // tau >= B), 0)
    assert r["mig_at"] == m
    if m:
        M = kappa * (l + m)
        D0 = (m - 1) * T + M - m * tau           # how far past its slot the first target token is generated
        d = r["d"]
        tbts = [int(d[j] - d[j - 1]) for j in range(2, n + 1)]
        if D0 <= 0:
            assert r["delayed"] == 0 and max(tbts) == tau
        else:
            assert max(tbts) == tau + D0
            assert r["delayed"] == min(n - m, math.ceil(D0 / (tau - T_tgt)))
        assert int(d[n]) == (n - 1) * tau + max(D0, 0)


@pytest.mark.parametrize("seed", range(8))
def test_handoff_index_brute_force_occupancy(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(2, 70))
    tbt = float(rng.choice([0.03, 0.1, 0.19, 0.25]))
    t_m = float(rng.choice([0.0, 0.3, 1.0, 2.2]))
    o = oracle_of(constructed([30], [n], [1e-6], servers=[synth.server(tbt_s=tbt, jitter=0.5)],
                              devices=[synth.device(500.0, 20.0, jitter=0.05)]))
    pol_nomig = synth.policy(1.0, t_m_s=t_m, flags=S_MODE | PACE)
    pol = synth.policy(1.0, t_m_s=t_m, flags=S_MODE | PACE | MIG)
    base = o.play(pol_nomig, seed, 0)
    g, d = base["g"], base["d"]
    B = o.prep(pol).B
    assert B == math.ceil(round(t_m * 1e6) / 200000)
    want = 0
    if B == 0:
        want = 1
    else:
        for j in range(B, n):          # tokens generated by g_j: j; delivered: those with d_k <= g_j
            if j - sum(1 for k in range(1, n + 1) if d[k] <= g[j]) >= B:
                want = j
                break
    r = o.play(pol, seed, 0)
    assert r["mig_at"] == want
    if want:
        # the stream before the hand-off is untouched; the source stops after token m
        assert list(r["g"][1:want + 1]) == list(g[1:want + 1]) and list(r["d"][1:want + 1]) == list(d[1:want + 1])
        assert r["g"][want + 1] == g[want] + r["mig_latency"] == g[want] + 2000 * (30 + want)
        gm, dm = r["g"], r["d"]
        assert all(dm[j] == max(gm[j], dm[j - 1] + 200000) for j in range(2, n + 1))
        assert r["delayed"] == sum(1 for j in range(want + 1, n + 1) if gm[j] > dm[want] + (j - want) * 200000)


def test_migration_trigger_and_threshold():
    # Eq. 4: migrate iff delta_c * remaining > overhead; delta_c = |1e-3 - 0.2e-3|
    n = 60
    o = oracle_of(constructed([100], [n], [1e-6], devices=[synth.device(200.0, 10.0)]))
    m = 6
    saving = float(np.float32(abs(float(np.float32(1e-3)) - float(np.float32(0.2e-3)))) * np.float32(n - m))
    for theta, want in [(0.0, m), (saving * 0.999, m), (saving, 0), (saving * 1.001, 0), (float("inf"), 0)]:
        r = o.play(synth.policy(1.0, mig_threshold=theta, flags=S_MODE | MIG | PACE), 0, 0)
        assert r["mig_at"] == want, theta
    # no migration when the flag is off, when the winner is the cheaper endpoint, or when nothing would remain
    assert o.play(synth.policy(1.0, flags=S_MODE | PACE), 0, 0)["mig_at"] == 0
    o2 = oracle_of(constructed([100], [n], [30.0], devices=[synth.device(200.0, 10.0)]))   # device wins, cheaper
    r = o2.play(synth.policy(1.0, flags=S_MODE | MIG | PACE), 0, 0)
    assert r["winner_is_device"] and r["mig_at"] == 0
    o3 = oracle_of(constructed([100], [6], [1e-6], devices=[synth.device(200.0, 10.0)]))   # n - 1 = 5 < first fill at 6
    assert o3.play(synth.policy(1.0, flags=S_MODE | MIG | PACE), 0, 0)["mig_at"] == 0
    o4 = oracle_of(constructed([100], [1], [1e-6], devices=[synth.device(200.0, 10.0)]))
    assert o4.play(synth.policy(1.0, t_m_s=0.0, flags=S_MODE | MIG | PACE), 0, 0)["mig_at"] == 0


def test_migration_to_server_draws_from_the_ttft_distribution():
    n = 400
    rng = np.random.default_rng(5)
    ttft = rng.uniform(0.2, 3.0, size=n)
    dev = [synth.device(5000.0, 20.0, c_prefill=5e-3, c_decode=5e-3)]     # dear device that wins most races
    tr = constructed(rng.integers(1, 40, size=n), rng.integers(20, 60, size=n), ttft, devices=dev)
    o = oracle_of(tr)
    cnt, srt, kn = o.group_tables(0)
    assert list(kn) == [srt[(k * (n - 1)) // 256] for k in range(257)]
    pol = synth.policy(1.0, flags=D_MODE | MIG | PACE)
    lat = []
    for i in range(n):
        r = o.play(pol, 9, i)
        if r["mig_at"]:
            assert r["winner_is_device"]
            u = L.orc_hash(9, i, 0)
            k, fr = u >> 24, (u >> 8) & 0xFFFF
            assert r["mig_latency"] == kn[k] + (((kn[k + 1] - kn[k]) * fr) >> 16)
            assert srt[0] <= r["mig_latency"] <= srt[-1]
            lat.append(r["mig_latency"])
    assert len(lat) > 200
    # the draws follow the group's own TTFT distribution
    assert abs(np.median(lat) - np.median(srt)) < 0.15 * np.median(srt)


def test_tokens_and_cost_eq8():
    w = synth.tiny_workload(4, 300, n_servers=2, n_devices=2, max_prompt=300, max_out=120)
    w.devices[0]["lam"], w.devices[1]["lam"] = 0.5, 3.0        # Eq. 8's exchange rate, not one
    o = oracle_of(vars(w))
    pols = [synth.policy(b, flags=f) for b in (0.0, 0.3, 1.0) for f in (S_MODE | MIG | PACE, D_MODE | MIG | PACE, PACE)]
    st, out = o.eval(pols, 4, pairs=True)
    for p, pol in enumerate(pols):
        assert (out["tok_server"][p] + out["tok_device"][p] == w.output_len).all()
        cps = np.array([s["c_prefill"] for s in w.servers], np.float32)[w.server_profile].astype(np.float64)
        cds = np.array([s["c_decode"] for s in w.servers], np.float32)[w.server_profile].astype(np.float64)
        cpd = np.array([d["c_prefill"] for d in w.devices], np.float32)[w.device_profile].astype(np.float64)
        cdd = np.array([d["c_decode"] for d in w.devices], np.float32)[w.device_profile].astype(np.float64)
        dec, mig = out["decision"][p], out["mig_at"][p].astype(np.int64)
        l = w.prompt_len.astype(np.int64)
        pre_s = np.where(dec != 1, l, 0)
        pre_d = np.where(dec != 0, l, 0)
        to_dev = (mig > 0) & (out["tok_server"][p] == mig)      # source was the server
        to_srv = (mig > 0) & ~to_dev
        pre_d = pre_d + np.where(to_dev, l + mig, 0)
        pre_s = pre_s + np.where(to_srv, l + mig, 0)
        lam = np.array([d["lam"] for d in w.devices], np.float32)[w.device_profile].astype(np.float64)
        want = cps * pre_s + cds * out["tok_server"][p] + lam * (cpd * pre_d + cdd * out["tok_device"][p])
        assert np.allclose(out["cost"][p], want, rtol=1e-12)
        assert st[p].prefill_tok_server == int(pre_s.sum()) and st[p].prefill_tok_device == int(pre_d.sum())
        assert abs(st[p].total_cost - want.sum()) < 1e-9 * want.sum()


def test_cost_monotone_in_budget_without_migration():
    # the constrained endpoint is the dearer one; a larger budget only adds work on it
    w = synth.make_workload(1, n=3000)
    for dev_dear in (False, True):
        tr = dict(vars(w))
        if dev_dear:
            tr["devices"] = [synth.device(500.0, 20.0, jitter=0.05, c_prefill=5e-3, c_decode=5e-3)]
        o = oracle_of(tr)
        pols = [synth.policy(b, flags=PACE) for b in synth.budget_grid(21)]
        st, _ = o.eval(pols, 1)
        if dev_dear:
            tok = [s.prefill_tok_device for s in st]
        else:
            tok = [s.prefill_tok_server for s in st]
        assert all(b >= a for a, b in zip(tok, tok[1:]))
        cost = [s.total_cost for s in st]                # cost is monotone in the budget
        assert all(b >= a - 1e-9 for a, b in zip(cost, cost[1:]))
