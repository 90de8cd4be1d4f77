"""Full-size workloads, in the launch configuration the benchmark times: sampled pairs against the oracle
(request ranges it can play one by one) and properties that hold at any size (needs a GPU)."""
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
    host = {f: out[f].cpu().numpy() for f in out}
    for i0, i1 in ranges:
        _, oout = orc.eval(policies, w.seed, i0, i1, pairs=True, finish=False)
        for f in EXACT_PAIR:
            assert (host[f][:, i0:i1] == oout[f][:, i0:i1]).all(), (tag, f, i0)
        for f in FLOAT_PAIR:
            assert rel_close(host[f][:, i0:i1], oout[f][:, i0:i1], REL_TOL).all(), (tag, f, i0)
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
