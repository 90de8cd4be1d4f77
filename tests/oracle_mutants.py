"""Mutation check of the oracle's pins: plants one plausible mistake at a time in a COPY of the oracle's source
(a wrong comparison, index, sign, shift or a swapped endpoint), builds it, and runs the CPU pin tests against the
broken library.  A pin set that bites fails for every mutant.  Nothing here touches the CUDA path.
Left out because no input can tell them from the original: starting the hand-off search at j = B + 1 (at j = B the
test reads d_1 = 0 > g_B, never true) and running it up to j = n (the saving on zero remaining tokens is zero).

    python tests/oracle_mutants.py            # all mutants; prints the survivors, exit status 1 if there are any
    python tests/oracle_mutants.py 3 7        # only these
    python tests/oracle_mutants.py --gpu 3 7  # on a GPU machine: the parity tests (tests/test_gpu_parity.py) against the
                                              # broken oracle instead of the pins; they must fail too, which shows
                                              # that they would catch the same mistake made on the CUDA side
"""
import os
import subprocess
import sys
import tempfile

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "disco_oracle.cpp")

# (what the mistake is, exact text in the source, replacement)
MUTANTS = [
    ("hash: first shift 16 -> 15", "    x ^= x >> 16; x *= MUL1;", "    x ^= x >> 15; x *= MUL1;"),
    ("hash: multipliers swapped", "    x ^= x >> 15; x *= MUL2;", "    x ^= x >> 15; x *= MUL1;"),
    ("Eq. 3: >= becomes >", "if ((double)mass >= target) break;", "if ((double)mass > target) break;"),
    ("inverse CDF: rank off by one", "std::ceil(q * (double)G.N) - 1.0;", "std::ceil(q * (double)G.N);"),
    ("race: device starts on a tie", "R->device_started = S > w;", "R->device_started = S >= w;"),
    ("race: tie goes to the device", "R->winner_device = !(S <= w + Td);", "R->winner_device = !(S < w + Td);"),
    ("race: wait dropped from the device's TTFT", "R->ttft = std::min(S, w + Td);", "R->ttft = std::min(S, Td);"),
    ("jitter amplitude of the other endpoint", "const int64_t J = R->winner_device ? dv.J : sv.J;",
     "const int64_t J = R->winner_device ? sv.J : dv.J;"),
    ("pacing: max becomes the generation time",
     "for (int32_t j = 2; j <= n; ++j) d[j] = pacing ? std::max(g[j], d[j - 1] + tau) : g[j];",
     "for (int32_t j = 2; j <= n; ++j) d[j] = pacing ? std::max(g[j], d[j - 1]) : g[j];"),
    ("buffer test: index off by one", "if (d[j - pr.B + 1] > g[j]) { m = j; break; }",
     "if (d[j - pr.B] > g[j]) { m = j; break; }"),
    ("buffer test: > becomes >=", "if (d[j - pr.B + 1] > g[j]) { m = j; break; }",
     "if (d[j - pr.B + 1] >= g[j]) { m = j; break; }"),
    ("trigger: > becomes >=", "if (saving > pol.mig_threshold) {", "if (saving >= pol.mig_threshold) {"),
    ("hand-off latency: generated tokens not re-prefilled", "M = dv.kappa * (int64_t)(l + m) + dv.c0;",
     "M = dv.kappa * (int64_t)(l) + dv.c0;"),
    ("knot interpolation: fraction shift", "(int64_t)fr) >> 16);", "(int64_t)fr) >> 15);"),
    ("target stream keeps the source's interval", "Tt = dv.T; Jt = dv.J;", "Tt = sv.T; Jt = dv.J;"),
    ("delayed tokens: slot origin off by one", "if (g[j] > d[m] + (int64_t)(j - m) * tau) ++R->delayed;",
     "if (g[j] > d[m] + (int64_t)(j - m - 1) * tau) ++R->delayed;"),
    ("tokens: endpoints swapped", "R->tok_server = R->winner_device ? tgt : src;",
     "R->tok_server = R->winner_device ? src : tgt;"),
    ("prefill billing: loser's prefill not billed", "R->pre_device = R->device_started ? l : 0;",
     "R->pre_device = (R->device_started && R->winner_device) ? l : 0;"),
    ("Algorithm 2: tail quantile uses max instead of min", "const double q_tail = 1.0 - std::min(alpha, b);",
     "const double q_tail = 1.0 - std::max(alpha, b);"),
    ("Algorithm 2: budget not normalised by 1 - alpha", "const double A = ((b - alpha) / (1.0 - alpha)) * (double)G.Total;",
     "const double A = (b - alpha) * (double)G.Total;"),
    ("Algorithm 2: class funded on a strict comparison", "if ((double)with_l <= A) { funded = with_l; continue; }",
     "if ((double)with_l < A) { funded = with_l; continue; }"),
    ("Algorithm 2: w* from f instead of 1 - f", "out->w_star = inverse_cdf(G, (1.0 - alpha) * (1.0 - f));",
     "out->w_star = inverse_cdf(G, (1.0 - alpha) * f);"),
    ("Eq. 5: candidate endpoints swapped", "out->candidate_winner = (sv.cd > dcd) ? 1 : (dcd > sv.cd) ? 2 : 0;",
     "out->candidate_winner = (sv.cd > dcd) ? 2 : (dcd > sv.cd) ? 1 : 0;"),
    ("bins: octave offset", "int64_t b = 32 * (int64_t)(e - 4) + ((t >> (e - 5)) & 31);",
     "int64_t b = 32 * (int64_t)(e - 5) + ((t >> (e - 5)) & 31);"),
    ("quantile: rank reached on a strict comparison", "acc += hist[b]; if (acc >= rank) return b; }",
     "acc += hist[b]; if (acc > rank) return b; }"),
    ("jitter: range 2J instead of 2J + 1", "(uint64_t)(2 * J + 1)) >> 32) - J;", "(uint64_t)(2 * J)) >> 32) - J;"),
    ("ticks: truncated instead of rounded", "int64_t ticks_of_seconds(float s) { return llrint((double)s * 1e6); }",
     "int64_t ticks_of_seconds(float s) { return (int64_t)((double)s * 1e6); }"),
    ("device TTFT: intercept dropped", "const int64_t Td = dv.kappa * (int64_t)l + dv.c0;",
     "const int64_t Td = dv.kappa * (int64_t)l;"),
    ("Algorithm 3: threshold inclusive", "if (l < pr.l_th) device_only = true;", "if (l <= pr.l_th) device_only = true;"),
    ("Algorithm 2: wait map, l* class gets the tail wait",
     "else w = (l < pr.l_star) ? 0 : (l == pr.l_star) ? pr.w_star : pr.w_tail;",
     "else w = (l < pr.l_star) ? 0 : pr.w_tail;"),
    ("Eq. 1: immediate-start threshold exclusive", "if (pr.beta_rule) w = l <= pr.l_immediate ? 0 :",
     "if (pr.beta_rule) w = l < pr.l_immediate ? 0 :"),
    ("stochastic routing: endpoints swapped", "const bool to_device = pr.device_constrained ? constrained : !constrained;",
     "const bool to_device = pr.device_constrained ? !constrained : constrained;"),
    ("expected length: tokens already generated not subtracted",
     "std::max<int32_t>((int32_t)pol.expected_len - m, 0) : n - m;",
     "std::max<int32_t>((int32_t)pol.expected_len, 0) : n - m;"),
    ("pooled TBTs: first interval left out", "for (int32_t j = 2; j <= n; ++j) {\n                const int64_t tbt = d[j] - d[j - 1];",
     "for (int32_t j = 3; j <= n; ++j) {\n                const int64_t tbt = d[j] - d[j - 1];"),
    ("device wins counted for device-only requests too", "st.n_device_won += (R.decision == ORC_RACE && R.winner_device);",
     "st.n_device_won += R.winner_device;"),
    ("selection: mean TTFT before the tail", "if (x.p99_ttft_s != y.p99_ttft_s) { if (x.p99_ttft_s < y.p99_ttft_s) b = (int32_t)p; continue; }\n        if (x.mean_ttft_s != y.mean_ttft_s) { if (x.mean_ttft_s < y.mean_ttft_s) b = (int32_t)p; continue; }",
     "if (x.mean_ttft_s != y.mean_ttft_s) { if (x.mean_ttft_s < y.mean_ttft_s) b = (int32_t)p; continue; }\n        if (x.p99_ttft_s != y.p99_ttft_s) { if (x.p99_ttft_s < y.p99_ttft_s) b = (int32_t)p; continue; }"),
    ("selection: TBT objective ignored", "if (!(st[p].total_cost <= cost_cap) || !(st[p].p99_tbt_s <= tbt_slo_s)) continue;",
     "if (!(st[p].total_cost <= cost_cap)) continue;"),
    ("hash: request and token constants swapped", "    return mix(k0 + i * C_REQ);", "    return mix(k0 + i * C_TOK);"),
    ("Eq. 6: buffer size rounded down", "std::min<int64_t>((o->t_m + o->tau - 1) / o->tau, 1 << 30) : 0;",
     "std::min<int64_t>(o->t_m / o->tau, 1 << 30) : 0;"),
    ("Algorithm 1: max of the device costs", "bool device_constrained = std::min(dcp, dcd) > std::max(sv.cp, sv.cd);",
     "bool device_constrained = std::max(dcp, dcd) > std::max(sv.cp, sv.cd);"),
    ("Algorithm 1: exchange rate left out", "const double dcp = dv.lambda * dv.cp, dcd = dv.lambda * dv.cd;",
     "const double dcp = dv.cp, dcd = dv.lambda * dv.cd;"),
    ("knots: k N / 256 instead of k (N - 1) / 256", "G.sorted[(size_t)(((int64_t)k * (G.N - 1)) / 256)] : 0;",
     "G.sorted[(size_t)std::min<int64_t>(((int64_t)k * G.N) / 256, G.N - 1)] : 0;"),
    ("device-only requests billed a server prefill",
     "R->decision = ORC_DEVICE_ONLY; R->server_dispatched = false; R->device_started = true;",
     "R->decision = ORC_DEVICE_ONLY; R->server_dispatched = true; R->device_started = true;"),
    ("hand-off search runs one token short", "for (int32_t j = pr.B; j <= n - 1; ++j) {", "for (int32_t j = pr.B; j < n - 1; ++j) {"),
    ("migration of the cheaper winner", "const bool winner_dearer = R->winner_device ? (pr.candidate_winner == 2) : (pr.candidate_winner == 1);",
     "const bool winner_dearer = R->winner_device ? (pr.candidate_winner == 1) : (pr.candidate_winner == 2);"),
    ("stochastic routing: draw compared with b 2^31", "(double)u < std::floor(b * 4294967296.0);", "(double)u < std::floor(b * 2147483648.0);"),
    ("hash: high seed word ignored", "    uint32_t k0 = mix(lo ^ C_SEED) ^ hi;", "    uint32_t k0 = mix(lo ^ C_SEED);"),
    ("per-request mean TBT over n instead of n - 1", "((double)(d[n] - d[1]) * 1e-6) / (double)(n - 1) : 0.0;",
     "((double)(d[n] - d[1]) * 1e-6) / (double)(n) : 0.0;"),
    ("device starts counted for winners only", "st.n_device_started += R.device_started;",
     "st.n_device_started += (R.device_started && R.winner_device);"),
    ("P95 computed at 0.90", "const double qs[3] = {0.50, 0.95, 0.99};", "const double qs[3] = {0.50, 0.90, 0.99};"),
    ("P99 TBT over the requests instead of the intervals", "uint64_t r = (uint64_t)quantile_rank(0.99, st.n_intervals);",
     "uint64_t r = (uint64_t)quantile_rank(0.99, st.n_requests);"),
    ("quantile value: upper instead of lower bin edge", "*vals[k] = (double)bin_edge(*bins[k]) * 1e-6;",
     "*vals[k] = (double)bin_edge(*bins[k] + 1) * 1e-6;"),
    ("Eq. 1: wait not capped by the tail wait", "w = l <= pr.l_immediate ? 0 : std::min(pr.beta * (int64_t)l, pr.w_tail);",
     "w = l <= pr.l_immediate ? 0 : pr.beta * (int64_t)l;"),
    ("Eq. 2: slope search accepts one step too early", "if ((double)started_tokens(mid) <= limit) hi = mid; else lo = mid + 1;",
     "if ((double)started_tokens(mid) <= limit) hi = mid; else lo = mid;\n            if (hi - lo == 1) { lo = hi - 1; break; }"),
    ("migrated stream: late tokens counted on delivery times", "if (g[j] > d[m] + (int64_t)(j - m) * tau) ++R->delayed;",
     "if (d[j] > d[m] + (int64_t)(j - m) * tau) ++R->delayed;"),
    ("selection without a feasible policy: first instead of cheapest", "if (st[p].total_cost < st[c].total_cost) c = (int32_t)p;",
     "if (false && st[p].total_cost < st[c].total_cost) c = (int32_t)p;"),
    ("bins: linear region one too short", "    if (t < 32) return (int32_t)t;", "    if (t < 31) return (int32_t)t;"),
    ("bins: mantissa bits taken one place off", "+ ((t >> (e - 5)) & 31);", "+ ((t >> (e - 4)) & 31);"),
    ("groups: server and device index swapped", "const ServerTicks& sv = tr.srv[grp / tr.dev.size()];",
     "const ServerTicks& sv = tr.srv[grp % tr.srv.size()];"),
    ("Algorithm 2: b = alpha treated as above alpha", "    if (b <= alpha) {                 /* every length keeps the maximum wait */",
     "    if (b < alpha) {                 /* every length keeps the maximum wait */"),
    ("knot draw: index from the low byte", "const uint32_t k = u >> 24, fr = (u >> 8) & 0xFFFFu;",
     "const uint32_t k = u & 0xFFu, fr = (u >> 8) & 0xFFFFu;"),
    ("migration latency draw uses the token-1 hash", "const uint32_t u = token_hash(key, 0);\n                    const uint32_t k = u >> 24",
     "const uint32_t u = token_hash(key, 1);\n                    const uint32_t k = u >> 24"),
    ("target stream: first token not delayed by the hand-off", "g[m + 1] = g[m] + M;", "g[m + 1] = g[m] + Tt;"),
    ("server-constrained race keeps a wait", "if (l < pr.l_th) device_only = true;           /* Algorithm 3: short prompts stay on the device */",
     "if (l < pr.l_th) device_only = true; else w = 1000;"),
    ("no buffer: hand-off after the second token", "        if (pr.B == 0) {\n            m = 1;", "        if (pr.B == 0) {\n            m = 2;"),
    ("unpaced migrated stream delivered at the paced times", "                    d[j] = pacing ? std::max(g[j], d[j - 1] + tau) : g[j];",
     "                    d[j] = std::max(g[j], d[j - 1] + tau);"),
    ("late tokens counted without pacing too", "                if (pacing)\n                    for (int32_t j = m + 1; j <= n; ++j)",
     "                if (true)\n                    for (int32_t j = m + 1; j <= n; ++j)"),
    ("single-token outputs may hand over", "if (mig_on && R->decision == ORC_RACE && winner_dearer && n >= 2) {",
     "if (mig_on && R->decision == ORC_RACE && winner_dearer && n >= 1) {"),
    ("intervals counted as n instead of n - 1", "st.n_intervals += (uint64_t)(n - 1);", "st.n_intervals += (uint64_t)n;"),
    ("device-only requests may migrate", "if (mig_on && R->decision == ORC_RACE && winner_dearer && n >= 2) {",
     "if (mig_on && R->decision != ORC_SERVER_ONLY && winner_dearer && n >= 2) {"),
    ("cost: exchange rate dropped",
     "+ dv.lambda * (dv.cp * (double)R->pre_device + dv.cd * (double)R->tok_device);",
     "+ (dv.cp * (double)R->pre_device + dv.cd * (double)R->tok_device);"),
]


def run(ids=None, verbose=True, gpu=False):
    src = open(SRC).read()
    survivors = []
    with tempfile.TemporaryDirectory() as tmp:
        for k, (what, old, new) in enumerate(MUTANTS):
            if ids and k not in ids:
                continue
            if src.count(old) != 1:
                raise SystemExit("mutant %d: its text occurs %d times in the source" % (k, src.count(old)))
            cpp, so = os.path.join(tmp, "m%d.cpp" % k), os.path.join(tmp, "m%d.so" % k)
            with open(cpp, "w") as f:
                f.write(src.replace(old, new))
            subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-w",
                                   "-I", os.path.dirname(SRC), "-o", so, cpp])
            env = dict(os.environ, DISCO_ORACLE_LIB=so, DISCO_ORACLE_MUTATION_CHECK="1")
            select = ["-m", "gpu", os.path.join(ROOT, "tests", "test_gpu_parity.py")] if gpu else \
                     ["-m", "not gpu", "-k", "oracle and not mutant", os.path.join(ROOT, "tests")]
            r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] + select,
                               env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
            killed = r.returncode != 0
            if verbose:
                print("%2d %-55s %s" % (k, what, "killed" if killed else "SURVIVED"))
            if not killed:
                survivors.append((k, what))
    return survivors


if __name__ == "__main__":
    args = [a for a in sys.argv[1:] if a != "--gpu"]
    left = run([int(a) for a in args] or None, gpu="--gpu" in sys.argv[1:])
    sys.exit(1 if left else 0)
