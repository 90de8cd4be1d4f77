"""Element-by-element comparison of the CUDA library with the CPU oracle on the same seeded inputs."""
import numpy as np

from oracle import Oracle
from paper_2502_11417_b200 import Trace

REL_TOL = 1e-5          # per-request fp32 latencies and costs
INT_STATS = ["n_requests", "n_intervals", "n_server_only", "n_device_only", "n_race", "n_device_started",
             "n_device_won", "n_migrations", "tok_server", "tok_device", "prefill_tok_server",
             "prefill_tok_device", "delayed_tokens"]
EXACT_PAIR = ["decision", "tok_server", "tok_device", "mig_at", "delayed"]
FLOAT_PAIR = ["ttft_s", "tbt_mean_s", "tbt_max_s", "cost"]


def rel_close(a, b, tol):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    return np.abs(a - b) <= tol * np.maximum(np.abs(b), 1e-30)


def check_stats(gs, os_, hists, tag=""):
    """gs: library stats; os_: oracle stats; hists: callable p -> (ttft_hist, tbt_hist) of the library."""
    for p in range(len(gs)):
        g, o = gs[p], os_[p]
        for f in INT_STATS:
            assert getattr(g, f) == getattr(o, f), (tag, p, f, getattr(g, f), getattr(o, f))
        th, bh = hists(p)
        assert (th == np.ctypeslib.as_array(o.ttft_hist)).all(), (tag, p, "ttft histogram")
        assert (bh == np.ctypeslib.as_array(o.tbt_hist)).all(), (tag, p, "tbt histogram")
        for f in ["bin_p50_ttft", "bin_p95_ttft", "bin_p99_ttft", "bin_p99_tbt"]:
            assert abs(getattr(g, f) - getattr(o, f)) <= 1, (tag, p, f)       # quantiles within one bin
            assert getattr(g, f) == getattr(o, f), (tag, p, f)                # and in fact identical
        for f in ["p50_ttft_s", "p95_ttft_s", "p99_ttft_s", "p99_tbt_s"]:
            assert rel_close(getattr(g, f), getattr(o, f), 1e-6), (tag, p, f)
        assert rel_close(g.mean_ttft_s, o.mean_ttft_s, 1e-9), (tag, p, g.mean_ttft_s, o.mean_ttft_s)
        assert rel_close(g.total_cost, o.total_cost, REL_TOL), (tag, p, g.total_cost, o.total_cost)


def check_pairs(gout, oout, rows=None, tag=""):
    for f in EXACT_PAIR:
        a = gout[f].cpu().numpy() if hasattr(gout[f], "cpu") else gout[f]
        b = oout[f]
        if rows is not None:
            a, b = a[:, rows], b[:, rows]
        bad = np.argwhere(a != b)
        assert bad.size == 0, (tag, f, bad[:5], a[tuple(bad[0])], b[tuple(bad[0])])
    for f in FLOAT_PAIR:
        a = gout[f].cpu().numpy() if hasattr(gout[f], "cpu") else gout[f]
        b = oout[f]
        if rows is not None:
            a, b = a[:, rows], b[:, rows]
        ok = rel_close(a, b, REL_TOL)
        bad = np.argwhere(~ok)
        assert bad.size == 0, (tag, f, bad[:5], a[tuple(bad[0])], b[tuple(bad[0])])


def check_prep(tr, orc, policies, tag=""):
    for g in range(orc.n_groups):
        for p, pol in enumerate(policies):
            a, b = tr.prep(g, p), orc.prep(pol, g)
            assert a.device_constrained == b.device_constrained, (tag, g, p)
            assert a.tau == b.tau and a.B == min(b.B, 8192), (tag, g, p)
            if a.device_constrained:
                assert (a.l_star, a.w_star, a.w_tail) == (b.l_star, b.w_star, b.w_tail), (tag, g, p)
                assert (a.beta_rule, a.l_immediate, a.beta) == (b.beta_rule, b.l_immediate, b.beta), \
                    (tag, g, p, (a.beta_rule, a.l_immediate, a.beta), (b.beta_rule, b.l_immediate, b.beta))
            else:
                assert a.l_th == b.l_th, (tag, g, p, a.l_th, b.l_th)


def check_tables(tr, orc, tag=""):
    for g in range(orc.n_groups):
        cnt, srt, kn = orc.group_tables(g)
        gcnt, gkn, gsrt = tr.group_tables(g)
        assert (cnt == gcnt).all(), (tag, g, "length histogram")
        assert (srt == gsrt).all(), (tag, g, "sorted TTFT ticks")
        if len(srt):
            assert (kn == gkn).all(), (tag, g, "knots")


def full_parity(w, policies=None, select=True, tag="", seed=None):
    """Loads w into both, compares tables, prep, every pair, every statistic, and the selection."""
    policies = w.policies if policies is None else policies
    seed = w.seed if seed is None else seed
    orc = Oracle.from_workload(w)
    tr = Trace.from_workload(w)
    check_tables(tr, orc, tag)
    out = tr.alloc_pair_outputs(len(policies))
    tr.eval_policies(policies, seed, out)
    gs = tr.reduce_stats()
    ostats, oout = orc.eval(policies, seed, pairs=True)
    check_prep(tr, orc, policies, tag)
    check_pairs(out, oout, tag=tag)
    check_stats(gs, ostats, tr.histograms, tag)
    if select:
        cheapest = min(s.total_cost for s in ostats)
        for cap, slo in [(1.25 * cheapest, 0.25), (0.5 * cheapest, 0.25), (1e30, 1e-3), (1e30, 10.0)]:
            assert tr.select_policy(cap, slo) == orc.select(ostats, cap, float(np.float32(slo))), (tag, cap, slo)
    tr.close()
    return gs, ostats
