"""Pins for the oracle's Stoch-S / Stoch-D baselines (Sec. 5.1) and the expected-length migration trigger (Eq. 4)."""
import numpy as np
import pytest

from oracle import lib, SERVER_ONLY, DEVICE_ONLY, RACE
from paper_2502_11417_b200 import synth
from helpers import constructed, oracle_of

L = lib()
STOCH, MIG, PACE = synth.FLAG_STOCHASTIC, synth.FLAG_MIGRATION, synth.FLAG_PACING
S_MODE, D_MODE = synth.MODE_SERVER_CONSTRAINED, synth.MODE_DEVICE_CONSTRAINED


@pytest.mark.parametrize("mode", [S_MODE, D_MODE])
def test_stochastic_routing(mode):
    w = synth.make_workload(1, n=20000)
    o = oracle_of(vars(w))
    constrained, other = (SERVER_ONLY, DEVICE_ONLY) if mode == S_MODE else (DEVICE_ONLY, SERVER_ONLY)
    total = float(w.prompt_len.sum())
    S = np.rint(w.server_ttft_s.astype(np.float64) * 1e6).astype(np.int64)
    Td = 2000 * w.prompt_len.astype(np.int64)
    for b in [0.0, 0.1, 0.5, 0.9, 1.0]:
        pol = synth.policy(b, flags=STOCH | MIG | PACE | mode)
        st, out = o.eval([pol], 7, pairs=True)
        dec = out["decision"][0]
        # one endpoint per request: no race, no migration, all tokens on the routed endpoint
        assert not (dec == RACE).any() and st[0].n_migrations == 0 and st[0].n_device_won == 0
        assert (out["tok_device"][0][dec == DEVICE_ONLY] == w.output_len[dec == DEVICE_ONLY]).all()
        assert (out["tok_server"][0][dec == SERVER_ONLY] == w.output_len[dec == SERVER_ONLY]).all()
        t = np.rint(out["ttft_s"][0] * 1e6).astype(np.int64)
        assert (t == np.where(dec == DEVICE_ONLY, Td, S)).all()
        # the draw: request i goes to the constrained endpoint iff hash(seed, i, 2^32-1) < floor(b 2^32)
        u = np.array([L.orc_hash(7, i, 0xFFFFFFFF) for i in range(w.n)], dtype=np.float64)
        want = np.where((u < np.floor(float(np.float32(b)) * 2.0 ** 32)) | (b >= 1.0), constrained, other)
        assert (dec == want).all()
        frac = (dec == constrained).mean()
        assert abs(frac - b) < 4 * np.sqrt(max(b * (1 - b), 1e-9) / w.n) + 1e-12      # binomial
        share = w.prompt_len[dec == constrained].sum() / total                         # the budget's own measure
        assert abs(share - b) < 0.03
        if b == 0.0:
            assert (dec == other).all()
        if b == 1.0:
            assert (dec == constrained).all()


def test_disco_tail_ttft_is_not_worse_than_stochastic_routing():
    # Table 2's comparison, on a synthetic trace: at equal budgets the length-aware dispatch has the lower tail TTFT
    w = synth.make_workload(1, n=20000)
    o = oracle_of(vars(w))
    for b in [0.2, 0.4, 0.6, 0.8]:
        st, _ = o.eval([synth.policy(b, flags=PACE | S_MODE), synth.policy(b, flags=STOCH | PACE | S_MODE)], 3, exact=True)
        assert st[0].exact_p99_ttft_s <= st[1].exact_p99_ttft_s
        assert st[0].mean_ttft_s <= st[1].mean_ttft_s
        assert st[0].prefill_tok_server <= b * w.prompt_len.sum() + 1                 # same cap on the server's share


def test_expected_length_trigger():
    # server wins at once and is the dearer decoder; the buffer of 5 tokens fills at m = 6
    n = 60
    o = oracle_of(constructed([100], [n], [1e-6], devices=[synth.device(200.0, 10.0)]))
    dc = float(np.float32(abs(float(np.float32(1e-3)) - float(np.float32(0.2e-3)))))
    base = o.play(synth.policy(1.0, flags=S_MODE | MIG | PACE), 0, 0)
    assert base["mig_at"] == 6
    for E, theta, want in [(0, 0.0, 6), (128, 0.0, 6), (6, 0.0, 0), (5, 0.0, 0), (7, 0.0, 6),
                           (128, float(np.float32(dc) * np.float32(122)) * 0.999, 6),
                           (128, float(np.float32(dc) * np.float32(122)), 0),
                           (30, float(np.float32(dc) * np.float32(54)) * 0.999, 0),    # true remainder 54 would trigger
                           (128, float(np.float32(dc) * np.float32(54)) * 1.001, 6)]:  # true remainder would not
        r = o.play(synth.policy(1.0, mig_threshold=theta, flags=S_MODE | MIG | PACE, expected_len=E), 0, 0)
        assert r["mig_at"] == want, (E, theta)
        if want:        # the estimate only decides; the stream after the hand-off is the trace's
            assert list(r["g"]) == list(base["g"]) and list(r["d"]) == list(base["d"])
    st, out = o.eval([synth.policy(1.0, flags=S_MODE | MIG | PACE, expected_len=128)], 0, pairs=True)
    assert out["tok_server"][0, 0] == 6 and out["tok_device"][0, 0] == n - 6


def _started_tokens(lens, cnt, srt, l_imm, beta, w_tail):
    """sum_l l cnt[l] #{S > w(l)} with w(l) = 0 for l <= l_imm, min(beta l, w_tail) above (exact integers)."""
    acc = 0
    for l in lens:
        w = 0 if l <= l_imm else min(beta * int(l), w_tail)
        acc += int(l) * int(cnt[l]) * int(len(srt) - np.searchsorted(srt, w, side="right"))
    return acc


@pytest.mark.parametrize("l_imm", [0, 40])
def test_beta_rule_of_eq_1_2(l_imm):
    BETA = synth.FLAG_BETA_RULE
    w = synth.make_workload(1, n=3000)
    tr = vars(w)
    tr["devices"] = [synth.device(500.0, 20.0, jitter=0.05, c_prefill=5e-3, c_decode=5e-3)]     # device-constrained
    o = oracle_of(tr)
    cnt, srt, kn = o.group_tables(0)
    lens = np.nonzero(cnt)[0]
    total, N = int((np.arange(4097) * cnt).sum()), len(srt)
    prev = None
    for b in [0.0, 0.03, 0.05, 0.1, 0.3, 0.6, 0.9, 1.0]:
        pol = synth.policy(b, flags=BETA | PACE | D_MODE, l_immediate=l_imm)
        pr = o.prep(pol)
        ref = o.prep(synth.policy(b, flags=PACE | D_MODE))
        assert pr.beta_rule == 1 and pr.device_constrained == 1 and pr.w_tail == ref.w_tail     # phase 1 is shared
        bf = float(np.float32(b))
        if bf <= float(np.float32(0.05)):
            assert pr.beta == pr.w_tail + 1 and pr.l_immediate == 0      # b <= alpha: every prompt waits w_tail
        else:
            limit = bf * total * N
            got = _started_tokens(lens, cnt, srt, l_imm, pr.beta, pr.w_tail)
            floor_share = _started_tokens(lens, cnt, srt, l_imm, pr.w_tail + 1, pr.w_tail)
            if floor_share > limit:
                assert pr.beta == pr.w_tail + 1                          # even the longest waits exceed the budget
            else:
                assert got <= limit                                      # the budget holds ...
                assert pr.beta == 0 or _started_tokens(lens, cnt, srt, l_imm, pr.beta - 1, pr.w_tail) > limit   # ... tightly
        if prev is not None:
            assert pr.beta <= prev                                       # more budget, shorter waits
        prev = pr.beta
        # the rule as played: wait 0 up to l_immediate, min(beta l, w_tail) above; device starts iff S > w
        st, out = o.eval([pol], 0, pairs=True)
        S = np.rint(w.server_ttft_s.astype(np.float64) * 1e6).astype(np.int64)
        l = w.prompt_len.astype(np.int64)
        wait = np.where(l <= pr.l_immediate, 0, np.minimum(pr.beta * l, pr.w_tail))
        assert ((out["decision"][0] == RACE) == (S > wait)).all()
        assert st[0].prefill_tok_device == int(l[S > wait].sum())
        if bf > 0.05:
            # realised share tracks the expectation the rule budgets (S is independent of l in this trace)
            assert abs(st[0].prefill_tok_device - _started_tokens(lens, cnt, srt, l_imm, pr.beta, pr.w_tail) / N) < 0.03 * total
    assert o.prep(synth.policy(1.0, flags=BETA | PACE | D_MODE, l_immediate=l_imm)).beta == 0
    # in the server-constrained mode the flag changes nothing
    a = o.prep(synth.policy(0.4, flags=BETA | PACE | S_MODE))
    b_ = o.prep(synth.policy(0.4, flags=PACE | S_MODE))
    assert a.beta_rule == 0 and a.l_th == b_.l_th
