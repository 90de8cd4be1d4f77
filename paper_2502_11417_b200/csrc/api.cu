// Host side of the C ABI: argument checks, device memory, launch order.  No arithmetic of the method runs
// here apart from turning the handful of profile and policy parameters into ticks.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "disco_internal.cuh"
#include "load.cuh"
#include "tile.cuh"

using namespace disco;

namespace {

thread_local std::string g_err;
std::atomic<uint64_t> g_launches{0};   // kernels launched by this library, all contexts

int fail(int code, const std::string& msg) { g_err = msg; return code; }
int fail_cuda(cudaError_t e, const char* what) {
    g_err = std::string(what) + ": " + cudaGetErrorString(e);
    return e == cudaErrorMemoryAllocation ? DISCO_ENOMEM : DISCO_ECUDA;
}
#define CU(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail_cuda(e_, #call); } while (0)

// A growable device buffer.
struct DevBuf {
    void* p = nullptr;
    size_t cap = 0;
    cudaError_t reserve(size_t bytes) {
        if (bytes <= cap && p) return cudaSuccess;
        if (p) { cudaFree(p); p = nullptr; cap = 0; }
        if (bytes < 16) bytes = 16;
        cudaError_t e = cudaMalloc(&p, bytes);
        if (e == cudaSuccess) cap = bytes;
        return e;
    }
    void release() { if (p) cudaFree(p); p = nullptr; cap = 0; }
    template <class T> T* as() const { return (T*)p; }
};

struct DevBufView { size_t off = 0; };

int64_t ticks_of_seconds(float s) { return llrint((double)s * 1e6); }
int64_t ticks_of_rate(float per_s) { return llrint(1e6 / (double)per_s); }

using HostReadback = LoadReadback;   // pinned host mirror of the load's read-back block

}  // namespace

namespace disco {
int set_error(int code, const char* msg) { return fail(code, msg); }

#ifdef DISCO_DEBUG
namespace {
std::vector<cudaError_t (*)(int32_t*)>& dbg_readers() { static std::vector<cudaError_t (*)(int32_t*)> v; return v; }
}  // namespace
void dbg_register(cudaError_t (*reader)(int32_t*)) { dbg_readers().push_back(reader); }
#endif
}  // namespace disco

namespace {
// Checked build: after a call has synchronised, asks every translation unit for an index its kernels refused.
// Returns 0, or DISCO_ECUDA with the kernel and the index in the error string.
int debug_check() {
#ifdef DISCO_DEBUG
    static const char* kernels[DBG_K_COUNT] = {"", "k_ingest", "radix sort", "k_scatter_by_length", "group tables", "k_prep",
                                               "k_playout_fast", "k_playout", "k_pairs_acc", "k_pairs_zones", "k_pairs_rows",
                                               "k_finalize", "k_select", "self-test"};
    static const char* whats[DBG_WHAT_COUNT] = {"", "request", "policy", "group", "chunk", "knot", "histogram bin",
                                                "window slot", "staging slot", "table entry", "counter", "element"};
    for (auto reader : disco::dbg_readers()) {
        int32_t w[4] = {0, 0, 0, 0};
        const cudaError_t e = reader(w);
        if (e != cudaSuccess) return fail_cuda(e, "reading the checked build's record");
        if (w[0]) {
            const char* k = w[0] > 0 && w[0] < DBG_K_COUNT ? kernels[w[0]] : "?";
            const char* t = w[1] > 0 && w[1] < DBG_WHAT_COUNT ? whats[w[1]] : "?";
            return fail(DISCO_ECUDA, std::string("checked build: ") + k + " refused " + t + " index " + std::to_string(w[2]) +
                                         " (bound " + std::to_string(w[3]) + ")");
        }
    }
#endif
    return 0;
}
}  // namespace

struct disco_ctx {
    uint32_t n = 0, ns = 0, nd = 0;
    int G = 0;
    bool loaded = false;
    std::vector<GroupConst> gc;
    std::vector<GroupConst> gc_dev;   // what d_gc holds (a reload with the same profiles skips the copy)
    const void* gc_dev_at = nullptr;
    // trace
    DevBuf in_prompt, in_out, in_ttft, in_sp, in_dp;      // staging of host inputs
    DevBuf keys_a, keys_b, tmp_idx, tmp_ln, cursors, inv, placed;
    DevBuf S, l, nout, orig, sorted;
    DevBuf zero, cum_mass, ng_exact, grp_off, knots, d_gc;   // `zero`: every table a load must clear, contiguous
    DevBuf fin_totals;                 // [2G] u64: output tokens and requests per group that the accumulators cover
    uint64_t first_index = 0;          // index of request 0 in the whole trace (hash key base)
    int sms = 0;                       // multiprocessors of the context's device
    // F as Algorithms 1-3 read it: the trace's own sorted ticks, or a whole trace's given by the caller
    DevBuf F_sorted_imp, F_off_imp;
    const int32_t* F_sorted = nullptr;
    const uint32_t* F_off = nullptr;
    bool tables_imported = false;
    std::vector<uint64_t> F_n;         // requests per group behind F (the group's own count unless imported)
    bool fin_imported = false;         // fin_totals holds a caller's merged totals, not this trace's
    std::vector<uint64_t> fin_own;     // this trace's totals, to put back before the next evaluation
    uint32_t *cnt = nullptr, *ng = nullptr, *max_n = nullptr, *radix_counts = nullptr;
    uint64_t* grp_sum_n = nullptr;
    int32_t* err = nullptr;
    size_t zero_bytes = 0;
    HostReadback* rb = nullptr;
    // evaluation
    uint32_t P = 0;
    bool evaluated = false, reduced = false;
    std::vector<PolicyConst> pol;
    DevBuf d_prep, d_accum, d_stats, d_tables, d_todo, d_left;
    struct View { void* p = nullptr; template <class T> T* as() const { return (T*)p; } };
    View d_acc, d_hist_ttft, d_hist_tbt, d_work;       // regions of d_accum (cleared by one memset)
    View d_pol, d_classes, d_pol_list, d_chunks;       // four regions of d_tables (filled by one copy)
    DevBuf rec_u32[7], rec_u16[2], rec_win[3];
    void* stage = nullptr;       // pinned staging for the small host->device tables
    size_t stage_cap = 0;
    cudaEvent_t stage_free = nullptr;
    int32_t* sel_host = nullptr; // pinned [2]
    void* stats_host = nullptr;  // pinned mirror of the statistics
    size_t stats_host_cap = 0;
    bool timing = false;         // record events around the play-out and pair kernels
    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    float ms[4] = {0.f, 0.f, 0.f, 0.f};   // clamp-free play-out, general play-out, pair reductions, pair rows
    bool timing_valid = false;

    ~disco_ctx() {
        DevBuf* all[] = {&in_prompt, &in_out, &in_ttft, &in_sp, &in_dp, &keys_a, &keys_b, &tmp_idx, &tmp_ln, &cursors, &inv, &placed,
                         &S, &l, &nout, &orig, &sorted, &zero, &cum_mass, &ng_exact, &grp_off, &knots, &d_gc, &d_prep, &d_accum, &d_stats, &d_tables, &d_todo,
                         &fin_totals, &F_sorted_imp, &F_off_imp, &d_left};
        for (DevBuf* b : all) b->release();
        for (auto& b : rec_u32) b.release();
        for (auto& b : rec_u16) b.release();
        for (auto& b : rec_win) b.release();
        if (rb) cudaFreeHost(rb);
        if (stage) cudaFreeHost(stage);
        if (sel_host) cudaFreeHost(sel_host);
        if (stats_host) cudaFreeHost(stats_host);
        if (stage_free) cudaEventDestroy(stage_free);
        for (auto& e : ev) if (e) cudaEventDestroy(e);
    }
};

namespace {

int check_profiles(const disco_trace_desc_t* d, std::vector<GroupConst>* out) {
    if (!d->servers || !d->devices || d->n_servers == 0 || d->n_devices == 0 ||
        (uint64_t)d->n_servers * d->n_devices > kMaxGroups)
        return fail(DISCO_EINVAL, "profile tables: need at least one server and one device and at most 64 groups");
    out->clear();
    for (uint32_t s = 0; s < d->n_servers; ++s) {
        const disco_server_profile_t& sv = d->servers[s];
        if (!(sv.tbt_s > 0.0f) || !std::isfinite(sv.tbt_s) || !(sv.jitter >= 0.0f && sv.jitter <= 1.0f) ||
            !std::isfinite(sv.c_prefill) || !std::isfinite(sv.c_decode))
            return fail(DISCO_EINVAL, "server profile " + std::to_string(s) + " is invalid");
        for (uint32_t k = 0; k < d->n_devices; ++k) {
            const disco_device_profile_t& dv = d->devices[k];
            if (!(dv.prefill_tps > 0.0f) || !(dv.decode_tps > 0.0f) || !std::isfinite(dv.prefill_tps) ||
                !std::isfinite(dv.decode_tps) || !(dv.jitter >= 0.0f && dv.jitter <= 1.0f) ||
                !(dv.ttft_intercept_s >= 0.0f) || !std::isfinite(dv.ttft_intercept_s) ||
                !std::isfinite(dv.c_prefill) || !std::isfinite(dv.c_decode) || !std::isfinite(dv.lambda))
                return fail(DISCO_EINVAL, "device profile " + std::to_string(k) + " is invalid");
            const int64_t Ts = ticks_of_seconds(sv.tbt_s), Tdv = ticks_of_rate(dv.decode_tps);
            const int64_t Js = llrint((double)Ts * (double)sv.jitter), Jd = llrint((double)Tdv * (double)dv.jitter);
            const int64_t kappa = ticks_of_rate(dv.prefill_tps), c0 = ticks_of_seconds(dv.ttft_intercept_s);
            if (Ts + Js >= (1 << 30) || Tdv + Jd >= (1 << 30) || kappa * (kMaxPrompt + kMaxOutput) + c0 >= (1LL << 31))
                return fail(DISCO_EINVAL, "profile too slow: a token interval or device TTFT exceeds the 32-bit tick range");
            GroupConst g;
            std::memset(&g, 0, sizeof g);
            g.T_srv = (int32_t)Ts; g.J_srv = (int32_t)Js; g.T_dev = (int32_t)Tdv; g.J_dev = (int32_t)Jd;
            g.kappa = (int32_t)kappa; g.c0 = (int32_t)c0;
            const double cps = sv.c_prefill, cds = sv.c_decode, lam = dv.lambda;
            const double dcp = lam * (double)dv.c_prefill, dcd = lam * (double)dv.c_decode;
            g.auto_device_constrained = std::fmin(dcp, dcd) > std::fmax(cps, cds) ? 1 : 0;   // Algorithm 1
            g.candidate = cds > dcd ? 1 : (dcd > cds ? 2 : 0);
            g.delta_c = (float)std::fabs(cds - dcd);
            g.cps = (float)cps; g.cds = (float)cds; g.lcpd = (float)dcp; g.lcdd = (float)dcd;
            g.cps_d = cps; g.cds_d = cds; g.cpd_d = dv.c_prefill; g.cdd_d = dv.c_decode; g.lambda_d = lam;
            out->push_back(g);
        }
    }
    return 0;
}

cudaError_t reserve_trace(disco_ctx* c, uint32_t n, bool host_inputs, bool has_sp, bool has_dp) {
    cudaError_t e;
    const size_t N = n ? n : 1;
    const int G = c->G;
#define R(buf, bytes) if ((e = c->buf.reserve(bytes)) != cudaSuccess) return e
    if (host_inputs) {
        R(in_prompt, N * 4); R(in_out, N * 4); R(in_ttft, N * 4);
        if (has_sp) R(in_sp, N);
        if (has_dp) R(in_dp, N);
    }
    R(keys_a, N * 8); R(keys_b, N * 8);
    R(tmp_ln, N * 4); R(cursors, (size_t)G * (kMaxPrompt + 1) * 4); R(inv, N * 4); R(placed, N * 16);
    R(S, N * 4); R(l, N * 2); R(nout, N * 2); R(orig, N * 4); R(sorted, N * 4);
    // one block for everything a load clears: cnt | grp_sum_n | ng | max_n | err | first radix counter buffer,
    // followed by the second counter buffer
    const size_t cnt_bytes = ((size_t)G * (kMaxPrompt + 1) * 4 + 15) / 16 * 16;
    const size_t counts_bytes = (size_t)256 * kRadixMaxBlocks * 4;
    const size_t head = cnt_bytes + kMaxGroups * 8 + kMaxGroups * 4 + 16 + 16;
    R(zero, head + 5 * counts_bytes + 1024);                    // + the 256 digit totals
    char* z = (char*)c->zero.p;
    c->cnt = (uint32_t*)z; c->grp_sum_n = (uint64_t*)(z + cnt_bytes); c->ng = (uint32_t*)(z + cnt_bytes + kMaxGroups * 8);
    c->max_n = (uint32_t*)(z + cnt_bytes + kMaxGroups * 12); c->err = (int32_t*)(z + cnt_bytes + kMaxGroups * 12 + 16);
    c->radix_counts = (uint32_t*)(z + head);
    c->zero_bytes = head;
    R(cum_mass, (size_t)G * (kMaxPrompt + 2) * 8); R(ng_exact, kMaxGroups * 4);
    R(grp_off, (kMaxGroups + 1) * 4); R(knots, (size_t)G * kNKnots * 4);
    R(d_gc, (size_t)G * sizeof(GroupConst));
    R(fin_totals, (size_t)2 * kMaxGroups * 8);
#undef R
    return cudaSuccess;
}

}  // namespace

namespace disco {
int check_debug_record() { return debug_check(); }
}  // namespace disco

extern "C" {

const char* disco_last_error(void) { return g_err.c_str(); }

void disco_free_trace(disco_ctx_t* ctx) { delete ctx; }

int disco_load_trace(disco_ctx_t** pctx, const disco_trace_desc_t* d, void* stream) {
    if (!pctx || !d) return fail(DISCO_EINVAL, "null argument");
    if (d->n >= (1ull << 31)) return fail(DISCO_EINVAL, "too many requests");
    if (d->n && (!d->prompt_len || !d->output_len || !d->server_ttft_s)) return fail(DISCO_EINVAL, "null trace array");
    if (d->arrays_on_device > 2) return fail(DISCO_EINVAL, "arrays_on_device must be 0, 1 or 2");
    if (d->first_index + d->n > (1ull << 32)) return fail(DISCO_EINVAL, "first_index + n exceeds 2^32");
    std::vector<GroupConst> gc;
    if (int rc = check_profiles(d, &gc)) return rc;
    cudaStream_t st = (cudaStream_t)stream;

    disco_ctx* c = *pctx;
    const bool fresh = c == nullptr;
    if (fresh) {
        c = new (std::nothrow) disco_ctx;
        if (!c) return fail(DISCO_ENOMEM, "out of host memory");
    }
    auto bail = [&](int rc) { if (fresh) delete c; else c->loaded = false; return rc; };
    c->loaded = c->evaluated = c->reduced = false;
    c->n = (uint32_t)d->n; c->ns = d->n_servers; c->nd = d->n_devices; c->G = (int)gc.size(); c->gc = gc;
    c->first_index = d->first_index;
    c->tables_imported = false;
    c->fin_imported = false;
    if (!c->sms) {
        int dev = 0;
        cudaError_t e0 = cudaGetDevice(&dev);
        if (e0 == cudaSuccess) e0 = cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, dev);
        if (e0 != cudaSuccess || c->sms < 1) return bail(fail_cuda(e0, "multiprocessor count of the current device"));
    }
    const uint32_t n = c->n;
    bool host_in = d->arrays_on_device != 1;
    cudaError_t e;
    // Host arrays that are page-locked and mapped (cudaHostAlloc, cudaHostRegister, a pinned tensor) are read by
    // the ingestion kernel in place (it reads every element exactly once): no staging copies.  Pageable arrays are
    // copied first.
    const void* in_place[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    bool zero_copy = host_in && n != 0 && d->arrays_on_device == 0;
    if (zero_copy) {
        const void* host[5] = {d->prompt_len, d->output_len, d->server_ttft_s, d->server_profile, d->device_profile};
        for (int k = 0; k < 5 && zero_copy; ++k) {
            if (!host[k]) continue;
            cudaPointerAttributes attr;
            if (cudaPointerGetAttributes(&attr, host[k]) != cudaSuccess) { cudaGetLastError(); zero_copy = false; break; }
            if (attr.type != cudaMemoryTypeHost || !attr.devicePointer) zero_copy = false;
            else in_place[k] = attr.devicePointer;
        }
    }
    if (zero_copy) host_in = false;
    if (!c->rb && (e = cudaMallocHost((void**)&c->rb, sizeof(HostReadback))) != cudaSuccess)
        return bail(fail_cuda(e, "cudaMallocHost"));
    if ((e = reserve_trace(c, n, host_in, d->server_profile != nullptr, d->device_profile != nullptr)) != cudaSuccess)
        return bail(fail_cuda(e, "device allocation for the trace"));

    LoadArgs a;
    std::memset(&a, 0, sizeof a);
    a.n = n; a.ns = c->ns; a.nd = c->nd;
    if (host_in && n) {
#define H2D(dst, src, bytes) if ((e = cudaMemcpyAsync(c->dst.p, src, bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return bail(fail_cuda(e, "host to device copy"))
        H2D(in_prompt, d->prompt_len, (size_t)n * 4); H2D(in_out, d->output_len, (size_t)n * 4);
        H2D(in_ttft, d->server_ttft_s, (size_t)n * 4);
        if (d->server_profile) H2D(in_sp, d->server_profile, (size_t)n);
        if (d->device_profile) H2D(in_dp, d->device_profile, (size_t)n);
#undef H2D
        a.prompt = c->in_prompt.as<int32_t>(); a.outlen = c->in_out.as<int32_t>(); a.ttft = c->in_ttft.as<float>();
        a.sp = d->server_profile ? c->in_sp.as<uint8_t>() : nullptr;
        a.dp = d->device_profile ? c->in_dp.as<uint8_t>() : nullptr;
    } else if (zero_copy) {
        a.prompt = (const int32_t*)in_place[0]; a.outlen = (const int32_t*)in_place[1]; a.ttft = (const float*)in_place[2];
        a.sp = (const uint8_t*)in_place[3]; a.dp = (const uint8_t*)in_place[4];
    } else {
        a.prompt = d->prompt_len; a.outlen = d->output_len; a.ttft = d->server_ttft_s;
        a.sp = d->server_profile; a.dp = d->device_profile;
    }
    a.keys_a = c->keys_a.as<uint64_t>(); a.keys_b = c->keys_b.as<uint64_t>(); a.cursors = c->cursors.as<uint32_t>(); a.inv = c->inv.as<uint32_t>(); a.placed = c->placed.as<uint4>();
    a.l_tmp = c->tmp_ln.as<uint16_t>(); a.n_tmp = c->tmp_ln.as<uint16_t>() + (n ? n : 1);
    a.radix_counts = c->radix_counts; a.zero_block = c->zero.p; a.zero_bytes = c->zero_bytes;
    a.ng_exact = c->ng_exact.as<uint32_t>(); a.readback = c->rb;     // pinned host memory, written by the last kernel
    a.S = c->S.as<int32_t>(); a.l = c->l.as<uint16_t>(); a.nout = c->nout.as<uint16_t>(); a.orig = c->orig.as<uint32_t>();
    a.sorted = c->sorted.as<int32_t>(); a.cnt = c->cnt; a.cum_mass = c->cum_mass.as<int64_t>();
    a.ng = c->ng; a.grp_off = c->grp_off.as<uint32_t>(); a.knots = c->knots.as<int32_t>();
    a.grp_sum_n = c->grp_sum_n; a.max_n = c->max_n; a.err = c->err;
    a.fin_totals = c->fin_totals.as<uint64_t>(); a.sms = c->sms;
    // the profile table is read from pageable memory: this copy returns once it has been staged
    const bool same_profiles = c->gc_dev_at == c->d_gc.p && c->gc_dev.size() == c->gc.size() &&
                               std::memcmp(c->gc_dev.data(), c->gc.data(), c->gc.size() * sizeof(GroupConst)) == 0;
    if (!same_profiles) {
        c->gc_dev_at = nullptr;
        if ((e = cudaMemcpyAsync(c->d_gc.p, c->gc.data(), c->gc.size() * sizeof(GroupConst), cudaMemcpyHostToDevice, st)) != cudaSuccess)
            return bail(fail_cuda(e, "profile copy"));
    }
    if ((e = run_load(a, st)) != cudaSuccess) return bail(fail_cuda(e, "trace ingestion kernels"));
    g_launches += load_kernel_launches(n, c->G);
    // the few numbers the host needs (error word, group sizes, longest output, largest TTFT per group) are in rb
    HostReadback* rb = c->rb;
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return bail(fail_cuda(e, "trace ingestion"));
    if (int rc = debug_check()) return bail(rc);
    if (!same_profiles) { c->gc_dev = c->gc; c->gc_dev_at = c->d_gc.p; }      // the copy has landed
    if (rb->err[0]) {
        static const char* what[] = {"", "prompt length outside 1..4096", "output length outside 1..8192",
                                     "server TTFT not finite, not positive or above 2000 s", "profile id out of range"};
        return bail(fail(DISCO_EINVAL, std::string(what[rb->err[0]]) + " at request " + std::to_string(rb->err[1])));
    }
    c->F_sorted = c->sorted.as<int32_t>(); c->F_off = c->grp_off.as<uint32_t>();
    c->F_n.assign(rb->ng, rb->ng + c->G);
    c->loaded = true;
    *pctx = c;
    return 0;
}

int disco_eval_policies(disco_ctx_t* c, const disco_policy_t* pol, uint32_t P, uint64_t seed,
                        const disco_pair_out_t* out, void* stream) {
    if (!c || !pol || P == 0) return fail(DISCO_EINVAL, "null context, null policies or P = 0");
    if (!c->loaded) return fail(DISCO_EINVAL, "no trace loaded");
    if (P > (1u << 19)) return fail(DISCO_EINVAL, "too many policies");
    cudaStream_t st = (cudaStream_t)stream;
    const int G = c->G;
    const uint32_t n = c->n;
    c->evaluated = c->reduced = false;

    // ---- policy constants and timeline classes
    std::vector<PolicyConst> pc(P);
    std::vector<ClassConst> classes;
    bool any_beta = false;                // some policy uses the Eq. 1-2 wait rule
    bool cls_extras_pending = false;      // some policy routes at random or triggers on an expected length
    for (uint32_t p = 0; p < P; ++p) {
        const disco_policy_t& q = pol[p];
        auto at = [p] { return " (policy " + std::to_string(p) + ")"; };
        if (!(q.budget >= 0.0f && q.budget <= 1.0f)) return fail(DISCO_EINVAL, "budget outside [0,1]" + at());
        if (!(q.alpha > 0.0f && q.alpha < 1.0f)) return fail(DISCO_EINVAL, "alpha outside (0,1)" + at());
        if (!(q.mig_threshold >= 0.0f)) return fail(DISCO_EINVAL, "migration threshold negative or NaN" + at());
        if (!(q.r_c > 0.0f) || !std::isfinite(q.r_c)) return fail(DISCO_EINVAL, "consumption rate must be positive" + at());
        if (!(q.t_m_s >= 0.0f) || !std::isfinite(q.t_m_s)) return fail(DISCO_EINVAL, "migration time must be >= 0" + at());
        const uint32_t mode = (q.flags >> 2) & 3u;
        if (mode == 3 || (q.flags >> 6)) return fail(DISCO_EINVAL, "unknown flags" + at());
        if (q.expected_len > (1u << 20)) return fail(DISCO_EINVAL, "expected length too large" + at());
        if (q.l_immediate > (uint32_t)kMaxPrompt) return fail(DISCO_EINVAL, "l_immediate above the longest prompt" + at());
        const int64_t tau = ticks_of_rate(q.r_c), t_m = ticks_of_seconds(q.t_m_s);
        if (tau < 1 || tau >= (1 << 30)) return fail(DISCO_EINVAL, "consumption interval outside 1 .. 2^30 ticks" + at());
        const bool pacing = (q.flags & DISCO_FLAG_PACING) != 0, mig = (q.flags & DISCO_FLAG_MIGRATION) != 0;
        int64_t B = pacing ? (t_m + tau - 1) / tau : 0;               // Eq. 6, rounded up
        if (B > kMaxOutput) B = kMaxOutput;                            // a buffer no stream can fill
        PolicyConst& o = pc[p];
        o.budget = q.budget; o.alpha = q.alpha; o.theta = q.mig_threshold; o.flags = q.flags;
        o.tau = (int32_t)tau; o.B = (int32_t)B; o.mode = (int32_t)mode;
        o.expected_len = q.expected_len; o.l_immediate = q.l_immediate;
        if (q.flags & DISCO_FLAG_BETA_RULE) any_beta = true;
        o.route_all = q.budget >= 1.0f ? 1 : 0;
        o.route_thr = o.route_all ? 0xFFFFFFFFu : (uint32_t)std::floor((double)q.budget * 4294967296.0);
        if ((q.flags & (DISCO_FLAG_STOCHASTIC | DISCO_FLAG_BETA_RULE)) || q.expected_len) cls_extras_pending = true;
        int cls = -1;
        for (size_t k = 0; k < classes.size(); ++k)
            if (classes[k].tau == o.tau && classes[k].B == o.B && classes[k].pacing == (int)pacing) { cls = (int)k; break; }
        if (cls < 0) {
            ClassConst cc;
            std::memset(&cc, 0, sizeof cc);
            cc.tau = o.tau; cc.tau_eff = pacing ? o.tau : 0; cc.B = o.B; cc.pacing = pacing;
            classes.push_back(cc);
            cls = (int)classes.size() - 1;
        }
        classes[cls].mig_any |= mig ? 1 : 0;
        o.cls = cls;
    }
    // ---- per class: 32-bit range proof and histogram windows of the regular TBTs
    const HostReadback& rb = *c->rb;
    const int64_t n_max = rb.max_n;
    for (ClassConst& cc : classes) {
        int Wmax[3] = {1, 1, 1};
        for (int g = 0; g < G; ++g) {
            const GroupConst& gc = c->gc[g];
            const int64_t xs = gc.T_srv + (int64_t)gc.J_srv, xd = gc.T_dev + (int64_t)gc.J_dev;
            if (rb.ng[g]) {
                const int64_t step = std::max<int64_t>(cc.tau_eff, std::max(xs, xd));
                const int64_t Mmax = std::max<int64_t>(rb.knot_max[g], (int64_t)gc.kappa * (kMaxPrompt + n_max) + gc.c0);
                if ((n_max - 1) * step + Mmax >= (1LL << 31))
                    return fail(DISCO_EINVAL, "a decode stream could outlast 2^31 ticks (about 35 minutes)");
            }
            int64_t lo_v[3], hi_v[3];
            lo_v[0] = cc.pacing ? cc.tau : gc.T_srv - (int64_t)gc.J_srv; hi_v[0] = cc.pacing ? std::max<int64_t>(cc.tau, xs) : xs;
            lo_v[1] = cc.pacing ? cc.tau : gc.T_dev - (int64_t)gc.J_dev; hi_v[1] = cc.pacing ? std::max<int64_t>(cc.tau, xd) : xd;
            lo_v[2] = std::min(lo_v[0], lo_v[1]); hi_v[2] = std::max(hi_v[0], hi_v[1]);
            for (int k = 0; k < 3; ++k) {
                const int lo = host_bin_of_ticks(lo_v[k]), hi = host_bin_of_ticks(hi_v[k]);
                cc.lo[g][k] = lo;
                cc.ktau[g][k] = cc.pacing ? host_bin_of_ticks(cc.tau) - lo : -1;
                Wmax[k] = std::max(Wmax[k], hi - lo + 1);
            }
        }
        for (int k = 0; k < 3; ++k) cc.W[k] = Wmax[k];
        const size_t win_bytes = (size_t)n * (Wmax[0] + Wmax[1] + Wmax[2]) * 4;
        if (win_bytes > (48ull << 30)) return fail(DISCO_ENOMEM, "per-request TBT windows would exceed 48 GB");
    }

    // ---- device buffers
    cudaError_t e;
    const size_t N1 = n ? n : 1;
    size_t wmax[3] = {1, 1, 1};
    for (const ClassConst& cc : classes) for (int k = 0; k < 3; ++k) wmax[k] = std::max<size_t>(wmax[k], cc.W[k]);
#define R(buf, bytes) if ((e = c->buf.reserve(bytes)) != cudaSuccess) return fail_cuda(e, "device allocation for the evaluation")
    R(d_prep, (size_t)G * P * sizeof(Prep));
    const size_t acc_bytes = (size_t)P * G * kNAcc * 8, hist_bytes = (size_t)P * kNBins * 8;
    // a to-do counter and a ticket counter per class, the work counters of the pair kernels (four words), and a
    // ticket counter per class for the zone kernel
    const size_t cls_cnt_bytes = (classes.size() * 8 + 15) / 16 * 16;
    const size_t cnt_bytes = cls_cnt_bytes + 32 + (classes.size() * 4 + 15) / 16 * 16;
    R(d_accum, acc_bytes + 2 * hist_bytes + cnt_bytes);
    R(d_todo, N1 * 4);
    c->d_acc.p = c->d_accum.p; c->d_hist_ttft.p = (char*)c->d_accum.p + acc_bytes;
    c->d_hist_tbt.p = (char*)c->d_accum.p + acc_bytes + hist_bytes;
    R(d_stats, P * sizeof(disco_policy_stats_t) + 16);
    for (int k = 0; k < 7; ++k) R(rec_u32[k], N1 * 4);
    for (int k = 0; k < 2; ++k) R(rec_u16[k], N1 * 2);
    for (int k = 0; k < 3; ++k) R(rec_win[k], N1 * wmax[k] * 4);

    if (c->fin_imported) {            // an import replaced the totals the final reductions refer to: back to the trace's own
        c->fin_own.assign((size_t)2 * G, 0);
        for (int g = 0; g < G; ++g) { c->fin_own[g] = rb.grp_sum_n[g]; c->fin_own[G + g] = rb.ng[g]; }
        CU(cudaMemcpyAsync(c->fin_totals.p, c->fin_own.data(), c->fin_own.size() * 8, cudaMemcpyHostToDevice, st));
        c->fin_imported = false;
    }
    // the accumulators are cleared while the host lays out the chunks and tables below
    CU(cudaMemsetAsync(c->d_accum.p, 0, acc_bytes + 2 * hist_bytes + cnt_bytes, st));

    // ---- policies grouped by class; request chunks (one group each) sized so that chunks x policy tiles
    //      fill the GPU about once
    std::vector<uint32_t> pol_list;
    std::vector<std::pair<uint32_t, uint32_t>> cls_range;       // [begin, end) in pol_list per class
    for (size_t k = 0; k < classes.size(); ++k) {
        const uint32_t b = (uint32_t)pol_list.size();
        for (uint32_t p = 0; p < P; ++p) if (pc[p].cls == (int)k) pol_list.push_back(p);
        // Within a class the policies are taken in an order that puts like policies side by side with their budgets
        // ascending, whatever order the caller gave them in: along such a run Algorithm 3's l_th does not increase
        // and Algorithm 2's l* does not decrease, which is what the zone-by-zone reduction needs of a tile.
        std::stable_sort(pol_list.begin() + b, pol_list.end(), [&](uint32_t x, uint32_t y) {
            const PolicyConst &a = pc[x], &c2 = pc[y];
            if (a.flags != c2.flags) return a.flags < c2.flags;
            if (a.expected_len != c2.expected_len) return a.expected_len < c2.expected_len;
            if (a.l_immediate != c2.l_immediate) return a.l_immediate < c2.l_immediate;
            if (a.alpha != c2.alpha) return a.alpha < c2.alpha;
            if (a.theta != c2.theta) return a.theta < c2.theta;
            return a.budget < c2.budget;
        });
        cls_range.push_back({b, (uint32_t)pol_list.size()});
    }
    const uint32_t tiles = (P + 31) / 32;
    // the zone kernel's blocks take (chunk, family of four policy tiles) items; the pair kernel works a chunk in
    // passes of at most 65,280 requests
    const uint32_t kMaxChunk = 65280;
    const uint32_t sms = (uint32_t)c->sms;
    const uint32_t fams = (tiles + 3) / 4;
    // about two items a block (the blocks draw them from a counter, so uneven items even out), chunks of 2,048
    // requests or more
    uint32_t want_chunks = std::max<uint32_t>(1, (2 * sms + fams - 1) / fams);
    const uint32_t min_chunks = (uint32_t)((N1 + kMaxChunk - 1) / kMaxChunk);
    if (min_chunks > want_chunks) {
        // several waves of blocks: the fewest chunks whose last wave is nearly full (long chunks spread a block's
        // set-up and flush over more requests), else the count near the minimum whose last wave is fullest
        double best = 0.0;
        for (uint32_t k = min_chunks; k < min_chunks + sms; ++k) {
            const uint64_t blocks = (uint64_t)k * fams, waves = (blocks + sms - 1) / sms;
            const double fill = (double)blocks / (double)(waves * sms);
            if (fill > best + 1e-9) { best = fill; want_chunks = k; }
            if (fill >= 0.94) break;
        }
    }
    uint32_t CH = (uint32_t)((N1 + want_chunks - 1) / want_chunks);
    CH = (CH + 255) / 256 * 256;
    CH = std::min<uint32_t>(std::max<uint32_t>(CH, 2048), kMaxChunk);
    // the chunks of the groups that Algorithm 1 finds device-constrained come first: Algorithm 2's wait map costs the
    // zone kernel more sweeps per chunk, and its blocks draw their work in list order, so the items drawn last (when
    // some blocks already idle) should be the cheap ones
    std::vector<Chunk> chunks;
    for (int dear = 1; dear >= 0; --dear)
        for (int g = 0; g < G; ++g) {
            if ((c->gc[g].auto_device_constrained != 0) != (dear != 0)) continue;
            for (uint32_t s = rb.grp_off[g]; s < rb.grp_off[g + 1]; s += CH)
                chunks.push_back({s, std::min(CH, rb.grp_off[g + 1] - s), g, 0});
        }
#undef R

    // scratch of the pair kernels: a bit per (request, policy tile), a counter per (chunk, policy tile)
    const size_t left_mask_words = (size_t)N1 * ((tiles + 31) / 32);
    // ... and, while that stays below 1 GB, a short list of flagged requests per (chunk, tile)
    const size_t left_cells = chunks.size() * (size_t)tiles;
    const size_t left_list_words = left_cells * kLeftList * 4 <= (1ull << 30) ? left_cells * kLeftList : 0;
    if ((e = c->d_left.reserve((left_mask_words + left_cells + left_list_words + 4) * 4)) != cudaSuccess)
        return fail_cuda(e, "device allocation for the evaluation");

    // ---- small tables to the device through pinned staging
    const size_t need = P * sizeof(PolicyConst) + classes.size() * sizeof(ClassConst) + P * 4 +
                        chunks.size() * sizeof(Chunk) + 64;
    if (c->stage_free) CU(cudaEventSynchronize(c->stage_free));     // an earlier call's copies may still read it
    else CU(cudaEventCreateWithFlags(&c->stage_free, cudaEventDisableTiming));
    if (need > c->stage_cap) {
        if (c->stage) cudaFreeHost(c->stage);
        c->stage = nullptr; c->stage_cap = 0;
        CU(cudaMallocHost(&c->stage, need));
        c->stage_cap = need;
    }
    // one staging block, one copy: policies | classes | policy list | chunks (16-byte aligned regions)
    char* sp = (char*)c->stage;
    size_t off = 0;
    auto put = [&](DevBufView& v, const void* src, size_t bytes) {
        std::memcpy(sp + off, src, bytes);
        v.off = off;
        off += (bytes + 15) / 16 * 16;
    };
    DevBufView v_pol, v_cls, v_list, v_chunks;
    put(v_pol, pc.data(), P * sizeof(PolicyConst));
    put(v_cls, classes.data(), classes.size() * sizeof(ClassConst));
    put(v_list, pol_list.data(), P * 4);
    put(v_chunks, chunks.data(), chunks.size() * sizeof(Chunk));
    if ((e = c->d_tables.reserve(off + 16)) != cudaSuccess) return fail_cuda(e, "device allocation for the evaluation");
    char* dt = (char*)c->d_tables.p;
    c->d_pol.p = dt + v_pol.off; c->d_classes.p = dt + v_cls.off; c->d_pol_list.p = dt + v_list.off;
    c->d_chunks.p = dt + v_chunks.off;
    CU(cudaMemcpyAsync(dt, sp, off, cudaMemcpyHostToDevice, st));
    CU(cudaEventRecord(c->stage_free, st));

    uint32_t* todo_counts = (uint32_t*)((char*)c->d_accum.p + acc_bytes + 2 * hist_bytes);
    c->d_work.p = (char*)c->d_accum.p + acc_bytes + 2 * hist_bytes + cls_cnt_bytes;

    // ---- Algorithms 1-3 for every (group, policy)
    CU(launch_prep(c->d_pol.as<PolicyConst>(), P, G, c->d_gc.as<GroupConst>(), c->cum_mass.as<int64_t>(),
                   c->cnt, c->F_sorted, c->F_off, c->d_prep.as<Prep>(), st));
    if (any_beta) {
        CU(launch_prep_beta(c->d_pol.as<PolicyConst>(), P, G, c->cum_mass.as<int64_t>(), c->cnt, c->F_sorted,
                            c->F_off, c->d_prep.as<Prep>(), st));
        g_launches += 1;
    }

    TraceDev tr;
    tr.n = n; tr.n_groups = G; tr.S = c->S.as<int32_t>(); tr.l = c->l.as<uint16_t>(); tr.nout = c->nout.as<uint16_t>();
    tr.orig = c->orig.as<uint32_t>(); tr.inv = c->inv.as<uint32_t>(); tr.len_end = c->cursors.as<uint32_t>(); tr.grp_off = c->grp_off.as<uint32_t>();
    TimelineRec rec;
    for (int k = 0; k < 3; ++k) {
        rec.sum[k] = c->rec_u32[2 * k].as<uint32_t>(); rec.max[k] = c->rec_u32[2 * k + 1].as<uint32_t>();
        rec.win[k] = c->rec_win[k].as<uint32_t>();
    }
    rec.stall = c->rec_u32[6].as<uint32_t>();
    rec.m = c->rec_u16[0].as<uint16_t>(); rec.delayed = c->rec_u16[1].as<uint16_t>();
    disco_pair_out_t po;
    std::memset(&po, 0, sizeof po);
    if (out) po = *out;

    uint64_t out_tokens = 0;
    for (int g = 0; g < G; ++g) out_tokens += rb.grp_sum_n[g];
    const bool long_outputs = out_tokens >= 512ull * n;
    // the hash is keyed by the request's index in the whole trace: key = mix(k0 + (first_index + i) * C_REQ)
    const uint32_t k0 = seed_key(seed) + (uint32_t)c->first_index * kHashReq;
    // ---- per timeline class: play every request out, then evaluate the class's policies on the summaries
    g_launches += 1;
    c->timing_valid = false;
    const bool timed = c->timing && classes.size() == 1;
    for (size_t k = 0; k < classes.size(); ++k) {
        const ClassConst* dcc = c->d_classes.as<ClassConst>() + k;
        if (timed) CU(cudaEventRecord(c->ev[0], st));
        // with pacing on, a stream whose slowest interval T + J is within tau never falls behind its reader
        bool never_clamps = classes[k].pacing != 0;
        for (int g = 0; g < G; ++g)
            never_clamps = never_clamps && (int64_t)c->gc[g].T_srv + c->gc[g].J_srv <= classes[k].tau &&
                           (int64_t)c->gc[g].T_dev + c->gc[g].J_dev <= classes[k].tau;
        CU(launch_timeline(tr, c->d_gc.as<GroupConst>(), dcc, classes[k].pacing != 0, c->knots.as<int32_t>(), k0, rec,
                           c->err, c->d_todo.as<uint32_t>(), todo_counts + 2 * k, never_clamps, long_outputs,
                           timed ? c->ev[1] : nullptr, c->sms, st));
        if (timed) CU(cudaEventRecord(c->ev[2], st));
        CU(launch_pairs(tr, c->d_gc.as<GroupConst>(), dcc, c->d_prep.as<Prep>(), P,
                        c->d_pol_list.as<uint32_t>() + cls_range[k].first, cls_range[k].second - cls_range[k].first,
                        c->d_chunks.as<Chunk>(), (uint32_t)chunks.size(), rec, po, c->d_acc.as<uint64_t>(),
                        c->d_hist_ttft.as<uint64_t>(), c->d_hist_tbt.as<uint64_t>(), c->d_left.as<uint32_t>(),
                        c->d_left.as<uint32_t>() + left_mask_words,
                        left_list_words ? c->d_left.as<uint32_t>() + left_mask_words + left_cells : nullptr,
                        sms, (uint32_t*)(c->d_work.as<uint64_t>() + 4) + k, c->d_work.as<uint64_t>(), k0, cls_extras_pending,
                        !classes[k].pacing || classes[k].W[0] > 1 || classes[k].W[1] > 1 || classes[k].W[2] > 1,
                        timed ? c->ev[3] : nullptr, st));
        if (timed) CU(cudaEventRecord(c->ev[4], st));
        const bool wide_k = !classes[k].pacing || classes[k].W[0] > 1 || classes[k].W[1] > 1 || classes[k].W[2] > 1;
        g_launches += (n ? ((classes[k].pacing && !never_clamps) ? 2 : 1) : 0) +
                      ((n && !chunks.empty()) ? (out ? 2 : 1) + (wide_k ? 0 : 1) : 0);
    }
    c->timing_valid = timed && n != 0;
    c->P = P; c->pol = pc;
    c->evaluated = true;
    return 0;
}

int disco_reduce_stats(disco_ctx_t* c, disco_policy_stats_t* stats, void* stream) {
    if (!c || !stats) return fail(DISCO_EINVAL, "null argument");
    if (!c->evaluated) return fail(DISCO_EINVAL, "no evaluation to reduce");
    cudaStream_t st = (cudaStream_t)stream;
    // statistics and the error word land in pinned host memory straight from the kernel
    const size_t bytes = c->P * sizeof(disco_policy_stats_t) + 16;
    if (bytes > c->stats_host_cap) {
        if (c->stats_host) cudaFreeHost(c->stats_host);
        c->stats_host = nullptr; c->stats_host_cap = 0;
        CU(cudaMallocHost(&c->stats_host, bytes));
        c->stats_host_cap = bytes;
    }
    CU(launch_finalize(c->P, c->G, c->d_gc.as<GroupConst>(), c->d_acc.as<uint64_t>(), c->d_hist_ttft.as<uint64_t>(),
                       c->d_hist_tbt.as<uint64_t>(), c->fin_totals.as<uint64_t>(),
                       c->d_stats.as<disco_policy_stats_t>(), (disco_policy_stats_t*)c->stats_host, c->err, st));
    CU(cudaStreamSynchronize(st));
    if (int rc = debug_check()) return rc;
    std::memcpy(stats, c->stats_host, c->P * sizeof(disco_policy_stats_t));
    std::memcpy(c->rb->err, (char*)c->stats_host + c->P * sizeof(disco_policy_stats_t), 16);
    g_launches += 1;
    if (c->timing_valid) {
        for (int k = 0; k < 4; ++k) CU(cudaEventElapsedTime(&c->ms[k], c->ev[k], c->ev[k + 1]));
    }
    if (c->rb->err[2]) return fail(DISCO_ECUDA, "internal error: an inter-token interval fell outside its histogram window");
    c->reduced = true;
    return 0;
}

int disco_select_policy(const disco_policy_stats_t* stats, uint32_t P, double cost_cap, float tbt_slo_s,
                        int32_t* best) {
    if (!stats || !best || P == 0) return fail(DISCO_EINVAL, "null argument or P = 0");
    if (P > (1u << 19)) return fail(DISCO_EINVAL, "too many policies");
    // lexicographic objective: feasible first; then (P99 TTFT bin, mean TTFT, cost, index); none feasible: cheapest
    const double slo = (double)tbt_slo_s;
    int64_t pick = -1;
    bool pick_ok = false;
    for (uint32_t p = 0; p < P; ++p) {
        const disco_policy_stats_t& s = stats[p];
        if (s.bin_p99_tbt < 0 || s.bin_p99_tbt >= kNBins || s.bin_p99_ttft < 0 || s.bin_p99_ttft >= kNBins)
            return fail(DISCO_EINVAL, "histogram bin out of range (policy " + std::to_string(p) + ")");
        const bool ok = s.total_cost <= cost_cap && (double)host_bin_edge_ticks(s.bin_p99_tbt) * 1e-6 <= slo;
        bool take;
        if (pick < 0) take = true;
        else if (ok != pick_ok) take = ok;
        else {
            const disco_policy_stats_t& b = stats[pick];
            if (ok) {
                if (s.bin_p99_ttft != b.bin_p99_ttft) take = s.bin_p99_ttft < b.bin_p99_ttft;
                else if (s.mean_ttft_s != b.mean_ttft_s) take = s.mean_ttft_s < b.mean_ttft_s;
                else take = s.total_cost < b.total_cost;
            } else {
                take = s.total_cost < b.total_cost;
            }
        }
        if (take) { pick = p; pick_ok = ok; }
    }
    *best = (int32_t)pick;
    if (!pick_ok) return fail(DISCO_EINFEASIBLE, "no policy meets the cost cap and the TBT objective");
    return 0;
}

int disco_select_policy_device(disco_ctx_t* c, double cost_cap, float tbt_slo_s, int32_t* best, void* stream) {
    if (!c || !best) return fail(DISCO_EINVAL, "null argument");
    if (!c->reduced) return fail(DISCO_EINVAL, "reduce the statistics before selecting");
    cudaStream_t st = (cudaStream_t)stream;
    if (!c->sel_host) CU(cudaMallocHost((void**)&c->sel_host, 8));
    g_launches += 1;
    CU(launch_select(c->d_stats.as<disco_policy_stats_t>(), c->P, cost_cap, tbt_slo_s, c->sel_host, st));   // writes the pinned pair
    CU(cudaStreamSynchronize(st));
    if (int rc = debug_check()) return rc;
    *best = c->sel_host[1];
    if (c->sel_host[0] != 0) return fail(DISCO_EINFEASIBLE, "no policy meets the cost cap and the TBT objective");
    return 0;
}

uint64_t disco_kernel_launch_count(void) { return g_launches.load(); }

int disco_set_timing(disco_ctx_t* c, int on) {
    if (!c) return fail(DISCO_EINVAL, "null context");
    if (on) for (auto& e : c->ev) if (!e) CU(cudaEventCreate(&e));
    c->timing = on != 0;
    c->timing_valid = false;
    return 0;
}

int disco_get_timing(disco_ctx_t* c, float* ms4) {
    if (!c || !ms4) return fail(DISCO_EINVAL, "null argument");
    if (!c->timing_valid || !c->reduced) return fail(DISCO_EINVAL, "no timed evaluation has been reduced");
    for (int k = 0; k < 4; ++k) ms4[k] = c->ms[k];
    return 0;
}

int disco_get_work_counts(disco_ctx_t* c, uint64_t* counts4, void* stream) {
    if (!c || !counts4) return fail(DISCO_EINVAL, "null argument");
    if (!c->evaluated) return fail(DISCO_EINVAL, "no evaluation");
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaMemcpyAsync(counts4, c->d_work.p, 32, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return 0;
}

int disco_get_histograms(disco_ctx_t* c, uint32_t p, uint64_t* ttft_hist, uint64_t* tbt_hist, void* stream) {
    if (!c || !c->evaluated || p >= c->P) return fail(DISCO_EINVAL, "no evaluation or policy index out of range");
    cudaStream_t st = (cudaStream_t)stream;
    if (ttft_hist) CU(cudaMemcpyAsync(ttft_hist, c->d_hist_ttft.as<uint64_t>() + (size_t)p * kNBins, kNBins * 8, cudaMemcpyDeviceToHost, st));
    if (tbt_hist) CU(cudaMemcpyAsync(tbt_hist, c->d_hist_tbt.as<uint64_t>() + (size_t)p * kNBins, kNBins * 8, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return 0;
}

int disco_get_prep(disco_ctx_t* c, uint32_t g, uint32_t p, disco_prep_t* out, void* stream) {
    if (!c || !out || !c->evaluated || p >= c->P || g >= (uint32_t)c->G) return fail(DISCO_EINVAL, "bad argument");
    cudaStream_t st = (cudaStream_t)stream;
    Prep pr;
    CU(cudaMemcpyAsync(&pr, c->d_prep.as<Prep>() + (size_t)g * c->P + p, sizeof pr, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    out->device_constrained = pr.device_constrained; out->l_th = pr.l_th; out->l_star = pr.l_star;
    out->B = c->pol[p].B; out->w_star = pr.w_star; out->w_tail = pr.w_tail; out->tau = c->pol[p].tau;
    out->beta_rule = pr.beta_rule; out->l_immediate = pr.beta_rule ? pr.l_star : 0; out->beta = pr.beta_rule ? pr.w_star : 0;
    if (pr.beta_rule) { out->l_star = 0; out->w_star = 0; }
    return 0;
}

int64_t disco_get_group_tables(disco_ctx_t* c, uint32_t g, int64_t* cnt, int32_t* knots, int32_t* sorted_ticks,
                               uint64_t n_sorted, void* stream) {
    if (!c || !c->loaded || g >= (uint32_t)c->G) return fail(DISCO_EINVAL, "bad argument");
    cudaStream_t st = (cudaStream_t)stream;
    // the tables Algorithms 1-3 read: the trace's own, or the whole trace's a caller has set
    const uint64_t ng = c->F_n[g];
    uint64_t off = c->rb->grp_off[g];
    if (c->tables_imported) { off = 0; for (uint32_t k = 0; k < g; ++k) off += c->F_n[k]; }
    if (cnt) {
        std::vector<uint32_t> tmp(kMaxPrompt + 1);
        CU(cudaMemcpyAsync(tmp.data(), c->cnt + (size_t)g * (kMaxPrompt + 1), tmp.size() * 4, cudaMemcpyDeviceToHost, st));
        CU(cudaStreamSynchronize(st));
        for (size_t i = 0; i < tmp.size(); ++i) cnt[i] = tmp[i];
    }
    if (knots) CU(cudaMemcpyAsync(knots, c->knots.as<int32_t>() + (size_t)g * kNKnots, kNKnots * 4, cudaMemcpyDefault, st));
    const uint64_t k = std::min<uint64_t>(n_sorted, ng);
    if (sorted_ticks && k) CU(cudaMemcpyAsync(sorted_ticks, c->F_sorted + off, k * 4, cudaMemcpyDefault, st));
    CU(cudaStreamSynchronize(st));
    return (int64_t)ng;
}

int disco_set_group_tables(disco_ctx_t* c, const int64_t* cnt, const int32_t* ticks, const uint64_t* n_ticks,
                           void* stream) {
    if (!c || !cnt || !n_ticks) return fail(DISCO_EINVAL, "null argument");
    if (!c->loaded) return fail(DISCO_EINVAL, "no trace loaded");
    cudaStream_t st = (cudaStream_t)stream;
    const int G = c->G;
    const size_t L = kMaxPrompt + 1;
    uint64_t total = 0;
    std::vector<uint32_t> off(G + 1, 0), cnt32((size_t)G * L);
    for (int g = 0; g < G; ++g) {
        uint64_t by_length = 0;
        for (size_t l = 0; l < L; ++l) {
            const int64_t v = cnt[(size_t)g * L + l];
            if (v < 0 || v > 0xFFFFFFFFll || (l == 0 && v != 0))
                return fail(DISCO_EINVAL, "length count negative, above 2^32 - 1 or at length 0 (group " + std::to_string(g) + ")");
            by_length += (uint64_t)v;
            cnt32[(size_t)g * L + l] = (uint32_t)v;
        }
        if (by_length != n_ticks[g])
            return fail(DISCO_EINVAL, "length counts do not add up to the number of TTFT ticks (group " + std::to_string(g) + ")");
        total += n_ticks[g];
        if (total > 0xFFFFFFFFull) return fail(DISCO_EINVAL, "more than 2^32 - 1 requests behind the tables");
        off[g + 1] = (uint32_t)total;
    }
    if (total && !ticks) return fail(DISCO_EINVAL, "null argument");
    cudaError_t e;
    const size_t T1 = (size_t)std::max<uint64_t>(total, 1);
    // the sort's scratch: the key buffers of the load (free between loads), grown if the whole trace is larger
    if ((e = c->F_sorted_imp.reserve(T1 * 4)) != cudaSuccess || (e = c->F_off_imp.reserve((size_t)(kMaxGroups + 1) * 4)) != cudaSuccess ||
        (e = c->keys_a.reserve(T1 * 8)) != cudaSuccess || (e = c->keys_b.reserve(T1 * 8)) != cudaSuccess ||
        (e = c->tmp_idx.reserve(T1 * 4)) != cudaSuccess)
        return fail_cuda(e, "device allocation for the tables");
    CU(cudaMemsetAsync(c->err, 0, 16, st));
    if (total) CU(cudaMemcpyAsync(c->tmp_idx.p, ticks, (size_t)total * 4, cudaMemcpyDefault, st));
    CU(cudaMemcpyAsync(c->F_off_imp.p, off.data(), (size_t)(G + 1) * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(c->cnt, cnt32.data(), cnt32.size() * 4, cudaMemcpyHostToDevice, st));
    uint32_t* counts = c->radix_counts + (size_t)4 * 256u * kRadixMaxBlocks;
    CU(sort_grouped_ticks(c->tmp_idx.as<int32_t>(), c->F_off_imp.as<uint32_t>(), G, (uint32_t)total, c->keys_a.as<uint64_t>(),
                          c->keys_b.as<uint64_t>(), counts, c->err, c->F_sorted_imp.as<int32_t>(), c->sms, st));
    CU(launch_tables_imported(G, c->cnt, c->cum_mass.as<int64_t>(), c->ng_exact.as<uint32_t>(),
                              c->F_sorted_imp.as<int32_t>(), c->F_off_imp.as<uint32_t>(), c->knots.as<int32_t>(), st));
    if (total) g_launches += 2 + 3 * (G > 1 ? 5 : 4);
    g_launches += 1;
    // error word and each group's largest tick (the largest hand-off latency a draw from F can give)
    int32_t err_host[4] = {0, 0, 0, 0};
    std::vector<int32_t> top(G, 0);
    CU(cudaMemcpyAsync(err_host, c->err, 16, cudaMemcpyDeviceToHost, st));
    for (int g = 0; g < G; ++g)
        if (n_ticks[g]) CU(cudaMemcpyAsync(&top[g], c->F_sorted_imp.as<int32_t>() + off[g + 1] - 1, 4, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));          // the host vectors above are read by the copies until here
    if (int rc = debug_check()) { c->loaded = false; return rc; }
    c->evaluated = c->reduced = false;
    if (err_host[0]) {
        c->loaded = false;                  // the length counts have been overwritten: the context must be reloaded
        return fail(DISCO_EINVAL, "negative TTFT tick at position " + std::to_string(err_host[1]) + "; reload the trace");
    }
    c->F_sorted = c->F_sorted_imp.as<int32_t>(); c->F_off = c->F_off_imp.as<uint32_t>();
    c->tables_imported = true;
    for (int g = 0; g < G; ++g) { c->F_n[g] = n_ticks[g]; c->rb->knot_max[g] = top[g]; }
    return 0;
}

uint64_t disco_accumulator_words(disco_ctx_t* c) {
    if (!c || !c->evaluated) return 0;
    return (uint64_t)c->P * c->G * kNAcc + 2ull * c->P * kNBins + 2ull * c->G;
}

int disco_export_accumulators(disco_ctx_t* c, uint64_t* words, void* stream) {
    if (!c || !words) return fail(DISCO_EINVAL, "null argument");
    if (!c->evaluated) return fail(DISCO_EINVAL, "no evaluation to export");
    cudaStream_t st = (cudaStream_t)stream;
    const size_t head = (size_t)c->P * c->G * kNAcc + 2 * (size_t)c->P * kNBins;      // one block of d_accum
    CU(cudaMemcpyAsync(words, c->d_accum.p, head * 8, cudaMemcpyDefault, st));
    CU(cudaMemcpyAsync(words + head, c->fin_totals.p, (size_t)2 * c->G * 8, cudaMemcpyDefault, st));
    CU(cudaStreamSynchronize(st));
    return 0;
}

int disco_import_accumulators(disco_ctx_t* c, const uint64_t* words, void* stream) {
    if (!c || !words) return fail(DISCO_EINVAL, "null argument");
    if (!c->evaluated) return fail(DISCO_EINVAL, "evaluate the policies first: the accumulators take their shape from it");
    cudaStream_t st = (cudaStream_t)stream;
    const size_t head = (size_t)c->P * c->G * kNAcc + 2 * (size_t)c->P * kNBins;
    CU(cudaMemcpyAsync(c->d_accum.p, words, head * 8, cudaMemcpyDefault, st));
    CU(cudaMemcpyAsync(c->fin_totals.p, words + head, (size_t)2 * c->G * 8, cudaMemcpyDefault, st));
    CU(cudaStreamSynchronize(st));
    c->reduced = false;
    c->fin_imported = true;
    return 0;
}

int disco_debug_selftest(void* stream) {
#ifdef DISCO_DEBUG
    // a kernel offers an index beyond its bound to the check: the access is skipped, the record comes back as an error
    CU(run_debug_selftest((cudaStream_t)stream));
    CU(cudaStreamSynchronize((cudaStream_t)stream));
    g_launches += 1;
    return debug_check();
#else
    (void)stream;
    return fail(DISCO_EINVAL, "not a checked build (compile with -DDISCO_DEBUG)");
#endif
}

int disco_measure_alu_peak(double* lane_instr_per_s, double* token_steps_per_s, void* stream) {
    if (!lane_instr_per_s) return fail(DISCO_EINVAL, "null argument");
    int dev = 0, sms = 0;
    CU(cudaGetDevice(&dev));
    CU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    double rate = 0.0;
    CU(run_alu_peak(sms, &rate, (cudaStream_t)stream));
    g_launches += 3;
    *lane_instr_per_s = rate * 13.0;
    if (token_steps_per_s) *token_steps_per_s = rate;
    return 0;
}

}  // extern "C"
