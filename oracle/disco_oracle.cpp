/*
 * CPU oracle: plain restatement of DiSCo's dispatch + migration policy played
 * out on a trace (arXiv 2502.11417, Sec. 4; Appendix F, Algorithms 1-3;
 * Appendix E, Eq. 8).  TEST INFRASTRUCTURE ONLY -- see disco_oracle.h.
 *
 * Structure: for every policy, for every request, for every token.  Nothing is
 * shared between policies, nothing is blocked, fused or reordered, and no
 * closed form is used (closed forms are what the tests check this against).
 *
 * Compile with -ffp-contract=off so that every double expression is evaluated
 * exactly as written.
 */
#include "disco_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

namespace {

thread_local std::string g_err;
int fail(const char* msg) { g_err = msg; return -1; }

/* ---- per-token jitter: a counter hash of (seed, request, token) --------- */
/* Constants: first 32 fractional bits of sqrt(2), sqrt(3), sqrt(5) and two
 * odd multipliers from sqrt(7), sqrt(11).  The paper only says server TBT is
 * noisier than device TBT (Sec. 3); the generator itself is this library's. */
const uint32_t C_SEED = 0x6A09E667u, C_REQ = 0xBB67AE85u, C_TOK = 0x3C6EF373u;
const uint32_t MUL1 = 0xA54FF53Bu, MUL2 = 0x510E527Fu;

uint32_t mix(uint32_t x) {
    x ^= x >> 16; x *= MUL1;
    x ^= x >> 15; x *= MUL2;
    x ^= x >> 16;
    return x;
}
uint32_t request_key(uint64_t seed, uint32_t i) {
    uint32_t lo = (uint32_t)(seed & 0xFFFFFFFFu), hi = (uint32_t)(seed >> 32);
    uint32_t k0 = mix(lo ^ C_SEED) ^ hi;
    return mix(k0 + i * C_REQ);
}
uint32_t token_hash(uint32_t key, uint32_t j) { return mix(key + j * C_TOK); }
/* uniform integer in [-J, +J] */
int64_t jitter(uint32_t h, int64_t J) {
    return (int64_t)(((uint64_t)h * (uint64_t)(2 * J + 1)) >> 32) - J;
}

/* ---- ticks: 1 tick = 1 microsecond ------------------------------------- */
int64_t ticks_of_seconds(float s) { return llrint((double)s * 1e6); }
int64_t ticks_of_rate(float per_s) { return llrint(1e6 / (double)per_s); }

/* ---- histogram bins: 32 per octave ------------------------------------- */
int32_t bin_of(int64_t t) {
    if (t < 0) t = 0;
    if (t < 32) return (int32_t)t;
    int e = 0;
    for (int64_t v = t; v > 1; v >>= 1) ++e;           /* e = floor(log2 t) */
    int64_t b = 32 * (int64_t)(e - 4) + ((t >> (e - 5)) & 31);
    return (int32_t)std::min<int64_t>(b, ORC_NBINS - 1);
}
int64_t bin_edge(int32_t b) {
    if (b < 32) return b;
    int e = b / 32 + 4;
    return (int64_t)(32 + b % 32) << (e - 5);
}

struct ServerTicks { int64_t T, J; double cp, cd; };
struct DeviceTicks { int64_t T, J, kappa, c0; double cp, cd, lambda; };

struct Group {
    std::vector<int64_t> cnt;      /* requests per prompt length, [0..4096] */
    int64_t N = 0, Total = 0;      /* requests, input tokens */
    std::vector<int64_t> sorted;   /* ascending server-TTFT ticks: the empirical F */
    int64_t K[ORC_NKNOTS];         /* 257 equally spaced order statistics of F */
};

}  // namespace

struct orc_trace {
    uint64_t n = 0;
    std::vector<int32_t> l, nout, grp;
    std::vector<int64_t> S;
    std::vector<ServerTicks> srv;
    std::vector<DeviceTicks> dev;
    std::vector<Group> groups;     /* g = server_profile * n_devices + device_profile */
};

namespace {

/* F^{-1}(q) of the group's empirical TTFT distribution, nearest rank. */
int64_t inverse_cdf(const Group& G, double q) {
    if (G.N == 0) return 0;
    double r = std::ceil(q * (double)G.N) - 1.0;
    int64_t k = (int64_t)r;
    if (k < 0) k = 0;
    if (k > G.N - 1) k = G.N - 1;
    return G.sorted[(size_t)k];
}

struct PolicyTicks { int64_t tau, t_m; int32_t B; bool mig, pacing; int mode; };

int policy_ticks(const orc_policy_t& p, PolicyTicks* o) {
    if (!(p.budget >= 0.0f && p.budget <= 1.0f)) return fail("budget outside [0,1]");
    if (!(p.alpha > 0.0f && p.alpha < 1.0f)) return fail("alpha outside (0,1)");
    if (!(p.mig_threshold >= 0.0f)) return fail("migration threshold negative or NaN");
    if (!(p.r_c > 0.0f) || !std::isfinite(p.r_c)) return fail("consumption rate must be positive");
    if (!(p.t_m_s >= 0.0f) || !std::isfinite(p.t_m_s)) return fail("migration time must be >= 0");
    o->tau = ticks_of_rate(p.r_c);
    if (o->tau < 1) return fail("consumption interval below one tick");
    o->t_m = ticks_of_seconds(p.t_m_s);
    o->mig = (p.flags & ORC_FLAG_MIGRATION) != 0;
    o->pacing = (p.flags & ORC_FLAG_PACING) != 0;
    o->mode = (int)((p.flags >> 2) & 3);
    if (o->mode == 3 || (p.flags >> 6)) return fail("unknown flags");
    if (p.l_immediate > ORC_MAX_PROMPT) return fail("l_immediate above the longest prompt");
    /* Eq. 6: B = r_c * t_m tokens, rounded up; nothing to fill without a buffer */
    o->B = o->pacing ? (int32_t)std::min<int64_t>((o->t_m + o->tau - 1) / o->tau, 1 << 30) : 0;
    return 0;
}

int prep_group(const orc_trace& tr, const orc_policy_t& p, uint32_t g, orc_prep_t* out) {
    PolicyTicks pt;
    if (policy_ticks(p, &pt)) return -1;
    const Group& G = tr.groups[g];
    const ServerTicks& sv = tr.srv[g / tr.dev.size()];
    const DeviceTicks& dv = tr.dev[g % tr.dev.size()];
    const double b = (double)p.budget, alpha = (double)p.alpha;

    std::memset(out, 0, sizeof *out);
    out->tau = pt.tau; out->t_m = pt.t_m; out->B = pt.B;

    /* Algorithm 1, with the device costs expressed in money through lambda (Eq. 8) */
    const double dcp = dv.lambda * dv.cp, dcd = dv.lambda * dv.cd;
    bool device_constrained = std::min(dcp, dcd) > std::max(sv.cp, sv.cd);
    if (pt.mode == 1) device_constrained = true;
    if (pt.mode == 2) device_constrained = false;
    out->device_constrained = device_constrained ? 1 : 0;

    /* migration controller constants (Sec. 4.3, Eq. 4-5) */
    out->delta_c = (float)std::fabs(sv.cd - dcd);
    out->candidate_winner = (sv.cd > dcd) ? 1 : (dcd > sv.cd) ? 2 : 0;

    if (!device_constrained) {
        /* Algorithm 3 / Eq. 3: device-only mass below l_th is (1-b) of all input tokens */
        const double target = (1.0 - b) * (double)G.Total;
        int64_t mass = 0;
        int32_t L = 0;
        for (;;) {
            if ((double)mass >= target) break;       /* mass = sum_{l<L} l*cnt[l] */
            if (L > ORC_MAX_PROMPT) break;           /* cannot happen: mass == Total here */
            mass += (int64_t)L * G.cnt[L];
            ++L;
        }
        out->l_th = L;
        out->l_star = 0; out->w_star = 0; out->w_tail = 0;
        return 0;
    }

    /* Algorithm 2, phase 1: tail protection */
    const double q_tail = 1.0 - std::min(alpha, b);
    out->w_tail = inverse_cdf(G, q_tail);
    out->l_th = 0;
    if (p.flags & ORC_FLAG_BETA_RULE) {
        /* Phase 2 as in the body text (Eq. 1-2): w(l) = 0 for l <= l_immediate, min(beta l, w_tail) above.
         * beta (whole ticks per prompt token) is the smallest one under which the device's expected share
         * of input tokens, sum_l l cnt[l] P(S > w(l)), stays within b Total.  Counts are kept exact:
         * share * N = sum_l l cnt[l] #{S > w(l)}. */
        out->beta_rule = 1;
        out->l_star = 0; out->w_star = 0;
        const int64_t beta_hi = out->w_tail + 1;             /* from here on every wait is w_tail */
        if (b <= alpha) { out->l_immediate = 0; out->beta = beta_hi; return 0; }
        out->l_immediate = (int32_t)p.l_immediate;
        const double limit = (b * (double)G.Total) * (double)G.N;
        auto started_tokens = [&](int64_t beta) {
            int64_t acc = 0;
            for (int32_t l = 1; l <= ORC_MAX_PROMPT; ++l) {
                if (G.cnt[l] == 0) continue;
                const int64_t w = l <= out->l_immediate ? 0 : std::min(beta * (int64_t)l, out->w_tail);
                const int64_t later = G.N - (std::upper_bound(G.sorted.begin(), G.sorted.end(), w) - G.sorted.begin());
                acc += (int64_t)l * G.cnt[l] * later;
            }
            return acc;
        };
        int64_t lo = 0, hi = beta_hi;                        /* smallest beta in [0, beta_hi] within the limit */
        if ((double)started_tokens(hi) > limit) { out->beta = beta_hi; return 0; }   /* not even the longest waits fit */
        while (lo < hi) {
            const int64_t mid = lo + (hi - lo) / 2;
            if ((double)started_tokens(mid) <= limit) hi = mid; else lo = mid + 1;
        }
        out->beta = lo;
        return 0;
    }
    if (b <= alpha) {                 /* every length keeps the maximum wait */
        out->l_star = 0;
        out->w_star = out->w_tail;
        return 0;
    }
    /* phase 2: spend the remaining budget on the shortest prompts first.
     * A = input tokens that may start the device at once, beyond the tail share. */
    const double A = ((b - alpha) / (1.0 - alpha)) * (double)G.Total;
    out->budget_A = A;
    int64_t funded = 0;
    out->l_star = ORC_MAX_PROMPT + 1;
    out->w_star = 0;
    for (int32_t l = 0; l <= ORC_MAX_PROMPT; ++l) {
        if (G.cnt[l] == 0) continue;                         /* support of p(l) only */
        const int64_t with_l = funded + (int64_t)l * G.cnt[l];
        if ((double)with_l <= A) { funded = with_l; continue; }
        /* first class that does not fit: fund the fraction f of it */
        const double f = (A - (double)funded) / ((double)l * (double)G.cnt[l]);
        out->funded_fraction = f;
        out->l_star = l;
        out->w_star = inverse_cdf(G, (1.0 - alpha) * (1.0 - f));
        break;
    }
    return 0;
}

/* Everything one (request, policy) pair produces. */
struct PairResult {
    int decision; bool device_started, server_dispatched, winner_device;
    int64_t ttft;
    int32_t mig_at, delayed;
    int64_t mig_latency;
    int64_t tok_server, tok_device, pre_server, pre_device;
    double cost;
};

/* Plays request i under (pol, prep).  g, d must hold n+1 entries. */
void play(const orc_trace& tr, const orc_policy_t& pol, const orc_prep_t& pr, uint64_t seed,
          uint64_t i, int64_t* g, int64_t* d, PairResult* R) {
    const int32_t l = tr.l[i], n = tr.nout[i];
    const int64_t S = tr.S[i];
    const uint32_t grp = (uint32_t)tr.grp[i];
    const Group& G = tr.groups[grp];
    const ServerTicks& sv = tr.srv[grp / tr.dev.size()];
    const DeviceTicks& dv = tr.dev[grp % tr.dev.size()];
    const bool mig_on = (pol.flags & ORC_FLAG_MIGRATION) != 0;
    const bool pacing = (pol.flags & ORC_FLAG_PACING) != 0;
    const int64_t tau = pr.tau;
    const uint32_t key = request_key(seed, (uint32_t)i);

    /* ---- dispatch (Sec. 4.2): device TTFT is linear in the prompt length */
    const int64_t Td = dv.kappa * (int64_t)l + dv.c0;
    R->server_dispatched = true;
    int64_t w = 0;
    bool device_only = false;
    bool server_only = false;
    if (pol.flags & ORC_FLAG_STOCHASTIC) {
        /* Stoch-S / Stoch-D baselines (Sec. 5.1): each request goes to the constrained endpoint with
         * probability b, otherwise to the other one; one endpoint only, no race, no migration. */
        const uint32_t u = token_hash(key, 0xFFFFFFFFu);
        const double b = (double)pol.budget;
        const bool constrained = b >= 1.0 || (double)u < std::floor(b * 4294967296.0);
        const bool to_device = pr.device_constrained ? constrained : !constrained;
        device_only = to_device; server_only = !to_device;
    } else if (!pr.device_constrained) {
        if (l < pr.l_th) device_only = true;           /* Algorithm 3: short prompts stay on the device */
    } else {
        if (pr.beta_rule) w = l <= pr.l_immediate ? 0 : std::min(pr.beta * (int64_t)l, pr.w_tail);      /* Eq. 1 */
        else w = (l < pr.l_star) ? 0 : (l == pr.l_star) ? pr.w_star : pr.w_tail;   /* Algorithm 2's map W */
    }
    if (device_only) {
        R->decision = ORC_DEVICE_ONLY; R->server_dispatched = false; R->device_started = true;
        R->winner_device = true; R->ttft = Td;
    } else if (server_only) {
        R->decision = ORC_SERVER_ONLY; R->device_started = false; R->winner_device = false; R->ttft = S;
    } else {
        /* server first; the device starts after w if no server token has arrived; first token wins */
        R->device_started = S > w;
        if (!R->device_started) {
            R->decision = ORC_SERVER_ONLY; R->winner_device = false; R->ttft = S;
        } else {
            R->decision = ORC_RACE;
            R->winner_device = !(S <= w + Td);          /* tie goes to the server */
            R->ttft = std::min(S, w + Td);
        }
    }

    /* ---- generation and paced delivery, time origin = first token */
    const int64_t T = R->winner_device ? dv.T : sv.T;
    const int64_t J = R->winner_device ? dv.J : sv.J;
    g[1] = 0;
    for (int32_t j = 2; j <= n; ++j) g[j] = g[j - 1] + T + jitter(token_hash(key, (uint32_t)j), J);
    d[1] = 0;
    for (int32_t j = 2; j <= n; ++j) d[j] = pacing ? std::max(g[j], d[j - 1] + tau) : g[j];

    /* ---- migration (Sec. 4.3) */
    R->mig_at = 0; R->delayed = 0; R->mig_latency = 0;
    const bool winner_dearer = R->winner_device ? (pr.candidate_winner == 2) : (pr.candidate_winner == 1);
    if (mig_on && R->decision == ORC_RACE && winner_dearer && n >= 2) {
        /* hand-off index: first generated token at whose generation time the
         * buffer (generated but not yet delivered) holds B tokens */
        int32_t m = 0;
        if (pr.B == 0) {
            m = 1;
        } else {
            for (int32_t j = pr.B; j <= n - 1; ++j) {
                if (d[j - pr.B + 1] > g[j]) { m = j; break; }
            }
        }
        if (m > 0) {
            /* Eq. 4: projected saving on the remaining length against the overhead; the remainder is the
             * trace's true one, or what is left of an expected total length when the policy gives one */
            const int32_t remaining = pol.expected_len ? std::max<int32_t>((int32_t)pol.expected_len - m, 0) : n - m;
            const float saving = pr.delta_c * (float)remaining;
            if (saving > pol.mig_threshold) {
                int64_t M;
                int64_t Tt, Jt;
                if (!R->winner_device) {              /* target = device: re-prefill prompt + generated */
                    M = dv.kappa * (int64_t)(l + m) + dv.c0;
                    Tt = dv.T; Jt = dv.J;
                } else {                               /* target = server: a fresh TTFT draw from F */
                    const uint32_t u = token_hash(key, 0);
                    const uint32_t k = u >> 24, fr = (u >> 8) & 0xFFFFu;
                    M = G.K[k] + (((G.K[k + 1] - G.K[k]) * (int64_t)fr) >> 16);
                    Tt = sv.T; Jt = sv.J;
                }
                g[m + 1] = g[m] + M;
                for (int32_t j = m + 2; j <= n; ++j)
                    g[j] = g[j - 1] + Tt + jitter(token_hash(key, (uint32_t)j), Jt);
                for (int32_t j = m + 1; j <= n; ++j)
                    d[j] = pacing ? std::max(g[j], d[j - 1] + tau) : g[j];
                if (pacing)
                    for (int32_t j = m + 1; j <= n; ++j)
                        if (g[j] > d[m] + (int64_t)(j - m) * tau) ++R->delayed;   /* generated after its slot */
                R->mig_at = m; R->mig_latency = M;
            }
        }
    }

    /* ---- tokens and cost (Eq. 8) */
    const int64_t src = R->mig_at ? R->mig_at : n, tgt = n - src;
    R->tok_server = R->winner_device ? tgt : src;
    R->tok_device = R->winner_device ? src : tgt;
    R->pre_server = R->server_dispatched ? l : 0;
    R->pre_device = R->device_started ? l : 0;
    if (R->mig_at) {
        if (R->winner_device) R->pre_server += l + R->mig_at; else R->pre_device += l + R->mig_at;
    }
    R->cost = sv.cp * (double)R->pre_server + sv.cd * (double)R->tok_server
            + dv.lambda * (dv.cp * (double)R->pre_device + dv.cd * (double)R->tok_device);
}

double quantile_rank(double q, uint64_t M) { return std::ceil(q * (double)M); }

int32_t bin_of_rank(const uint64_t* hist, uint64_t rank) {
    uint64_t acc = 0;
    for (int32_t b = 0; b < ORC_NBINS; ++b) { acc += hist[b]; if (acc >= rank) return b; }
    return ORC_NBINS - 1;
}

double exact_quantile(std::vector<int64_t>& v, double q) {
    if (v.empty()) return 0.0;
    uint64_t r = (uint64_t)quantile_rank(q, v.size());
    if (r < 1) r = 1;
    std::nth_element(v.begin(), v.begin() + (r - 1), v.end());
    return (double)v[r - 1] * 1e-6;
}

}  // namespace

extern "C" {

uint32_t orc_mix(uint32_t x) { return mix(x); }
uint32_t orc_hash(uint64_t seed, uint32_t i, uint32_t j) { return token_hash(request_key(seed, i), j); }
int64_t orc_jitter(uint32_t h, int64_t J) { return jitter(h, J); }
int32_t orc_bin(int64_t t) { return bin_of(t); }
int64_t orc_bin_lower_edge(int32_t b) { return bin_edge(b); }
int64_t orc_seconds_to_ticks(float s) { return ticks_of_seconds(s); }
int64_t orc_rate_to_ticks(float r) { return ticks_of_rate(r); }
const char* orc_last_error(void) { return g_err.c_str(); }

orc_trace_t* orc_load(uint64_t n, const int32_t* prompt_len, const int32_t* output_len,
                      const float* ttft_s, const uint8_t* sprof, const uint8_t* dprof,
                      const orc_server_t* servers, uint32_t ns, const orc_device_t* devices, uint32_t nd) {
    if (!servers || !devices || ns == 0 || nd == 0 || ns > 255 || nd > 255) { fail("bad profile tables"); return nullptr; }
    if (n && (!prompt_len || !output_len || !ttft_s)) { fail("null trace array"); return nullptr; }
    orc_trace* tr = new orc_trace;
    tr->n = n;
    for (uint32_t s = 0; s < ns; ++s) {
        const orc_server_t& a = servers[s];
        if (!(a.tbt_s > 0) || !(a.jitter >= 0 && a.jitter <= 1)) { delete tr; fail("bad server profile"); return nullptr; }
        ServerTicks t;
        t.T = ticks_of_seconds(a.tbt_s);
        t.J = llrint((double)t.T * (double)a.jitter);
        t.cp = (double)a.c_prefill; t.cd = (double)a.c_decode;
        tr->srv.push_back(t);
    }
    for (uint32_t k = 0; k < nd; ++k) {
        const orc_device_t& a = devices[k];
        if (!(a.prefill_tps > 0) || !(a.decode_tps > 0) || !(a.jitter >= 0 && a.jitter <= 1) || !(a.ttft_intercept_s >= 0)) {
            delete tr; fail("bad device profile"); return nullptr;
        }
        DeviceTicks t;
        t.T = ticks_of_rate(a.decode_tps);
        t.J = llrint((double)t.T * (double)a.jitter);
        t.kappa = ticks_of_rate(a.prefill_tps);
        t.c0 = ticks_of_seconds(a.ttft_intercept_s);
        t.cp = (double)a.c_prefill; t.cd = (double)a.c_decode; t.lambda = (double)a.lambda;
        tr->dev.push_back(t);
    }
    tr->groups.resize((size_t)ns * nd);
    for (auto& G : tr->groups) G.cnt.assign(ORC_MAX_PROMPT + 1, 0);
    tr->l.resize(n); tr->nout.resize(n); tr->grp.resize(n); tr->S.resize(n);
    for (uint64_t i = 0; i < n; ++i) {
        const uint32_t s = sprof ? sprof[i] : 0, k = dprof ? dprof[i] : 0;
        if (s >= ns || k >= nd) { delete tr; fail("profile id out of range"); return nullptr; }
        if (prompt_len[i] < 1 || prompt_len[i] > ORC_MAX_PROMPT) { delete tr; fail("prompt length out of range"); return nullptr; }
        if (output_len[i] < 1 || output_len[i] > ORC_MAX_OUTPUT) { delete tr; fail("output length out of range"); return nullptr; }
        if (!(ttft_s[i] > 0) || !std::isfinite(ttft_s[i]) || ttft_s[i] > 2000.0f) { delete tr; fail("server TTFT out of range"); return nullptr; }
        tr->l[i] = prompt_len[i]; tr->nout[i] = output_len[i];
        tr->S[i] = ticks_of_seconds(ttft_s[i]);
        const uint32_t g = s * nd + k;
        tr->grp[i] = (int32_t)g;
        Group& G = tr->groups[g];
        G.cnt[prompt_len[i]] += 1; G.N += 1; G.Total += prompt_len[i];
        G.sorted.push_back(tr->S[i]);
    }
    for (auto& G : tr->groups) {
        std::sort(G.sorted.begin(), G.sorted.end());
        for (int k = 0; k < ORC_NKNOTS; ++k)
            G.K[k] = G.N ? G.sorted[(size_t)(((int64_t)k * (G.N - 1)) / 256)] : 0;
    }
    return tr;
}

void orc_free(orc_trace_t* t) { delete t; }
uint32_t orc_n_groups(const orc_trace_t* t) { return (uint32_t)t->groups.size(); }

int64_t orc_group_tables(const orc_trace_t* t, uint32_t g, int64_t* cnt, int64_t* sorted, int64_t* knots) {
    if (g >= t->groups.size()) return -1;
    const Group& G = t->groups[g];
    if (cnt) std::copy(G.cnt.begin(), G.cnt.end(), cnt);
    if (sorted) std::copy(G.sorted.begin(), G.sorted.end(), sorted);
    if (knots) std::copy(G.K, G.K + ORC_NKNOTS, knots);
    return G.N;
}

int64_t orc_inverse_cdf(const orc_trace_t* t, uint32_t g, double q) { return inverse_cdf(t->groups[g], q); }

int orc_prep(const orc_trace_t* t, const orc_policy_t* pol, uint32_t g, orc_prep_t* out) {
    if (!t || !pol || !out || g >= t->groups.size()) return fail("bad argument");
    return prep_group(*t, *pol, g, out);
}

int orc_play(const orc_trace_t* t, const orc_policy_t* pol, uint64_t seed, uint64_t i, int64_t* g, int64_t* d,
             int64_t* ttft, int32_t* winner_is_device, int32_t* mig_at, int64_t* mig_latency, int32_t* delayed) {
    if (!t || !pol || i >= t->n) return fail("bad argument");
    orc_prep_t pr;
    if (prep_group(*t, *pol, (uint32_t)t->grp[i], &pr)) return -1;
    PairResult R;
    play(*t, *pol, pr, seed, i, g, d, &R);
    if (ttft) *ttft = R.ttft;
    if (winner_is_device) *winner_is_device = R.winner_device;
    if (mig_at) *mig_at = R.mig_at;
    if (mig_latency) *mig_latency = R.mig_latency;
    if (delayed) *delayed = R.delayed;
    return R.decision;
}

int orc_eval(const orc_trace_t* t, const orc_policy_t* pols, uint32_t P, uint64_t seed, uint64_t i0, uint64_t i1,
             const orc_pair_out_t* out, orc_stats_t* stats, int want_exact) {
    return orc_eval_cols(t, pols, P, seed, i0, i1, out, t ? t->n : 0, 0, stats, want_exact);
}

int orc_eval_cols(const orc_trace_t* t, const orc_policy_t* pols, uint32_t P, uint64_t seed, uint64_t i0, uint64_t i1,
                  const orc_pair_out_t* out, uint64_t out_stride, uint64_t out_first, orc_stats_t* stats,
                  int want_exact) {
    if (!t || !pols || !stats || i0 > i1 || i1 > t->n) return fail("bad argument");
    if (out && (out_first > i0 || i1 - out_first > out_stride)) return fail("per-pair columns do not cover the range");
    const orc_trace& tr = *t;
    std::vector<int64_t> g(ORC_MAX_OUTPUT + 2), d(ORC_MAX_OUTPUT + 2);
    std::vector<orc_prep_t> prep(tr.groups.size());
    std::vector<int64_t> all_ttft, all_tbt;
    for (uint32_t p = 0; p < P; ++p) {
        const orc_policy_t& pol = pols[p];
        for (uint32_t gi = 0; gi < tr.groups.size(); ++gi)
            if (prep_group(tr, pol, gi, &prep[gi])) return -1;
        orc_stats_t& st = stats[p];
        all_ttft.clear(); all_tbt.clear();
        for (uint64_t i = i0; i < i1; ++i) {
            PairResult R;
            play(tr, pol, prep[(size_t)tr.grp[i]], seed, i, g.data(), d.data(), &R);
            const int32_t n = tr.nout[i];
            int64_t tbt_max = 0;
            for (int32_t j = 2; j <= n; ++j) {
                const int64_t tbt = d[j] - d[j - 1];
                tbt_max = std::max(tbt_max, tbt);
                st.tbt_hist[bin_of(tbt)] += 1;
                if (want_exact) all_tbt.push_back(tbt);
            }
            const double tbt_mean_s = n > 1 ? ((double)(d[n] - d[1]) * 1e-6) / (double)(n - 1) : 0.0;
            const double ttft_s = (double)R.ttft * 1e-6;
            st.n_requests += 1; st.n_intervals += (uint64_t)(n - 1);
            st.sum_ttft_s += ttft_s; st.total_cost += R.cost;
            st.ttft_hist[bin_of(R.ttft)] += 1;
            if (want_exact) all_ttft.push_back(R.ttft);
            st.n_server_only += R.decision == ORC_SERVER_ONLY;
            st.n_device_only += R.decision == ORC_DEVICE_ONLY;
            st.n_race += R.decision == ORC_RACE;
            st.n_device_started += R.device_started;
            st.n_device_won += (R.decision == ORC_RACE && R.winner_device);
            st.n_migrations += R.mig_at != 0;
            st.tok_server += (uint64_t)R.tok_server; st.tok_device += (uint64_t)R.tok_device;
            st.prefill_tok_server += (uint64_t)R.pre_server; st.prefill_tok_device += (uint64_t)R.pre_device;
            st.delayed_tokens += (uint64_t)R.delayed;
            if (out) {
                const size_t o = (size_t)p * out_stride + (size_t)(i - out_first);   /* row p, column of request i */
                if (out->ttft_s) out->ttft_s[o] = ttft_s;
                if (out->tbt_mean_s) out->tbt_mean_s[o] = tbt_mean_s;
                if (out->tbt_max_s) out->tbt_max_s[o] = (double)tbt_max * 1e-6;
                if (out->cost) out->cost[o] = R.cost;
                if (out->tok_server) out->tok_server[o] = (uint32_t)R.tok_server;
                if (out->tok_device) out->tok_device[o] = (uint32_t)R.tok_device;
                if (out->mig_at) out->mig_at[o] = (uint32_t)R.mig_at;
                if (out->delayed) out->delayed[o] = (uint16_t)R.delayed;
                if (out->decision) out->decision[o] = (uint8_t)R.decision;
            }
        }
        if (want_exact) {
            st.exact_p50_ttft_s = exact_quantile(all_ttft, 0.50);
            st.exact_p95_ttft_s = exact_quantile(all_ttft, 0.95);
            st.exact_p99_ttft_s = exact_quantile(all_ttft, 0.99);
            st.exact_p99_tbt_s = exact_quantile(all_tbt, 0.99);
        }
    }
    return 0;
}

void orc_finish(orc_stats_t* stats, uint32_t P) {
    for (uint32_t p = 0; p < P; ++p) {
        orc_stats_t& st = stats[p];
        st.mean_ttft_s = st.n_requests ? st.sum_ttft_s / (double)st.n_requests : 0.0;
        const double qs[3] = {0.50, 0.95, 0.99};
        int32_t* bins[3] = {&st.bin_p50_ttft, &st.bin_p95_ttft, &st.bin_p99_ttft};
        double* vals[3] = {&st.p50_ttft_s, &st.p95_ttft_s, &st.p99_ttft_s};
        for (int k = 0; k < 3; ++k) {
            uint64_t r = (uint64_t)quantile_rank(qs[k], st.n_requests);
            if (r < 1) r = 1;
            *bins[k] = st.n_requests ? bin_of_rank(st.ttft_hist, r) : 0;
            *vals[k] = (double)bin_edge(*bins[k]) * 1e-6;
        }
        uint64_t r = (uint64_t)quantile_rank(0.99, st.n_intervals);
        if (r < 1) r = 1;
        st.bin_p99_tbt = st.n_intervals ? bin_of_rank(st.tbt_hist, r) : 0;
        st.p99_tbt_s = (double)bin_edge(st.bin_p99_tbt) * 1e-6;
    }
}

/* Feasible = within the cost cap and the TBT objective; best = smallest tail
 * TTFT, then mean TTFT, then cost, then index (objectives of Sec. 4.1). */
int orc_select(const orc_stats_t* st, uint32_t P, double cost_cap, double tbt_slo_s, int32_t* best) {
    if (!st || !best || P == 0) return fail("bad argument");
    int32_t b = -1;
    for (uint32_t p = 0; p < P; ++p) {
        if (!(st[p].total_cost <= cost_cap) || !(st[p].p99_tbt_s <= tbt_slo_s)) continue;
        if (b < 0) { b = (int32_t)p; continue; }
        const orc_stats_t &x = st[p], &y = st[b];
        if (x.p99_ttft_s != y.p99_ttft_s) { if (x.p99_ttft_s < y.p99_ttft_s) b = (int32_t)p; continue; }
        if (x.mean_ttft_s != y.mean_ttft_s) { if (x.mean_ttft_s < y.mean_ttft_s) b = (int32_t)p; continue; }
        if (x.total_cost < y.total_cost) b = (int32_t)p;
    }
    if (b >= 0) { *best = b; return 0; }
    int32_t c = 0;
    for (uint32_t p = 1; p < P; ++p) if (st[p].total_cost < st[c].total_cost) c = (int32_t)p;
    *best = c;
    return -4;
}

}  // extern "C"
