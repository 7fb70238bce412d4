// C ABI of the library: argument validation, workspace carving and kernel sequencing.
// Nothing here allocates, synchronises (except natsl_device_status) or touches the CPU oracle.
#include <cstring>

#include "natsl_internal.h"

#include <atomic>
#include <mutex>

using namespace natsl;

namespace natsl {
// Test hooks (natsl_debug_set_wait_limit): a bound for the device-side waits of the following
// launches, and whether the scan withholds the per-chunk flags the softmax kernel waits for.
static std::atomic<uint32_t> g_debug_wait_kcycles{0};
static std::atomic<int> g_debug_withhold_flags{0};
int debug_wait_kcycles() { return (int)g_debug_wait_kcycles.load(std::memory_order_relaxed); }
static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
}  // namespace natsl

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kStatusBytes = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Carver {
    char *base;
    size_t off = 0;
    explicit Carver(void *b) : base(static_cast<char *>(b)) {}
    template <typename T> T *take(size_t n) {
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += align_up(n * sizeof(T));
        return p;
    }
};

int check_params(const natsl_params *p, bool needs_L) {
    if (!p) return NATSL_ERR_NULL;
    if (p->dtype != NATSL_F32 && p->dtype != NATSL_BF16) return NATSL_ERR_DTYPE;
    if (p->B <= 0 || p->H <= 0) return NATSL_ERR_SHAPE;
    if (p->d != 64 && p->d != 128) return NATSL_ERR_SHAPE;
    if (p->C != kC) return NATSL_ERR_SHAPE;
    if (needs_L && (p->L <= 0 || p->L % p->C != 0)) return NATSL_ERR_SHAPE;
    if (!(p->eps > 0.f)) return NATSL_ERR_SHAPE;
    if (p->G < 0 || (p->G > 1 && p->d % p->G != 0)) return NATSL_ERR_SHAPE;
    if ((p->flags & NATSL_QK_NORM) && !(p->norm_eps >= 0.f)) return NATSL_ERR_SHAPE;
    return NATSL_OK;
}

// Grouped softmax heads / per-operation q, k normalisation (Section 4.3): what the forward supports.
bool grouped_or_normed(const natsl_params *p) { return p->G > 1 || (p->flags & NATSL_QK_NORM); }
HeadGroups head_groups(const natsl_params *p) {
    HeadGroups hg;
    hg.G = p->G > 1 ? p->G : 1;
    hg.norm_eps = (p->flags & NATSL_QK_NORM) ? p->norm_eps : -1.f;
    return hg;
}

Shape shape_of(const natsl_params *p) { return Shape{p->B, p->H, p->L, p->d, p->dtype == NATSL_BF16}; }

struct FwdWs {
    int32_t *status, *emit_flags, *sm_idx, *prefix, *lin_idx, *n_lin, *sm_len;
    size_t head_bytes;          // status page + emit_flags: cleared at the start of every call
    void *k_sm, *v_sm, *v16;
    void *kn16;                 // prefill in pieces with NATSL_QK_NORM: normalised fp16 keys of the whole cache
    void *o_la16;               // tensor-core path: the linear read-out as fp16 [B,L,H,d]
    float *W, *U, *P, *o_la;    // fp32 CUDA-core path only
    float *q_la, *k_la, *q_sm, *k_nsm;   // fp32 storage with NATSL_QK_NORM: normalised copies of q and k
    GdnTcWs tc;                 // tensor-core path only
    float *seg_incr, *seg_trans, *seg_start;   // segmented scan: [B*H, nseg, d, d] each
    size_t bytes;
};

bool use_tensor_cores(const natsl_params *p) {
    return p->dtype == NATSL_BF16 && !(p->flags & NATSL_FORCE_SIMT);
}

// Backward on tensor cores with d = 64: all chunk-level products in one fused kernel per chunk -- unless
// q and k are normalised, which that kernel does not know; the separate products then serve d = 64 too.
bool fused_chunk_path(const natsl_params *p) {
    return use_tensor_cores(p) && p->d == 64 && !grouped_or_normed(p);
}

// Segments of the forward scan (tensor-core path): the largest power of two that keeps the two
// runs per segment within ~one CTA per SM, divides the chunk count and leaves >= 8 chunks each.
int scan_segments(const natsl_params *p) {
    if (!use_tensor_cores(p) || (p->flags & NATSL_SINGLE_PASS_SCAN)) return 1;
    const int NC = p->L / kC, BH = p->B * p->H;
    int nseg = 1;
    while (2 * BH * (nseg * 2) <= 128 && NC % (nseg * 2) == 0 && NC / (nseg * 2) >= 8) nseg *= 2;
    // Once the scan is segmented (and so already pays its second run), one more doubling up to one CTA per
    // SM: the two runs shrink by half again, which outweighs what the softmax kernel loses beside them --
    // unless the call appends to a cache: the softmax kernel then also reads the earlier pieces' keys, is
    // the longer of the two and needs the multiprocessors (a long prompt in pieces was 14 % slower with it).
    if (!(p->flags & NATSL_APPEND_CACHE) && nseg >= 2 && BH * (nseg * 2) <= 128 && NC % (nseg * 2) == 0 &&
        NC / (nseg * 2) >= 8)
        nseg *= 2;
    return nseg;
}

FwdWs carve_fwd(const natsl_params *p, void *ws) {
    Carver c(ws);
    FwdWs f;
    const size_t B = p->B, H = p->H, L = p->L, d = p->d, NC = L / kC;
    const size_t esz = p->dtype == NATSL_BF16 ? 2 : 4;
    f.status = c.take<int32_t>(kStatusBytes / 4);
    // one counter per chunk, raised by the scan as the chunk's read-out is complete (tensor-core path)
    f.emit_flags = c.take<int32_t>(use_tensor_cores(p) ? B * H * NC : 0);
    f.head_bytes = c.off;
    f.sm_idx = c.take<int32_t>(B * H * L);
    f.prefix = c.take<int32_t>(B * H * (NC + 1));
    f.lin_idx = c.take<int32_t>(B * H * L);
    f.n_lin = c.take<int32_t>(B * H * NC);
    f.sm_len = c.take<int32_t>(B * H);
    f.k_sm = c.take<char>(B * H * L * d * esz);
    f.v_sm = c.take<char>(B * H * L * d * esz);
    if (use_tensor_cores(p)) {
        // fp16 V of the retained tokens; when the call appends to a cache, of the whole cache
        const size_t capv = (p->flags & NATSL_APPEND_CACHE) && p->sm_cap > 0 ? (size_t)p->sm_cap : L;
        f.v16 = c.take<char>(B * H * capv * d * 2);
        f.kn16 = c.take<char>((p->flags & NATSL_APPEND_CACHE) && (p->flags & NATSL_QK_NORM) ? B * H * capv * d * 2 : 0);
        f.tc.Qh = c.take<char>(B * H * L * d * 2);
        f.tc.Kh = c.take<char>(B * H * L * d * 2);
        f.tc.Wt = c.take<char>(B * H * L * d * 2);
        f.tc.Ut = c.take<float>(B * H * L * d);
        f.tc.Ph = c.take<char>(B * H * NC * kC * kC * 2);
        f.tc.Gd = c.take<float>(B * H * L * 2);
        f.W = f.U = f.P = nullptr;
        const size_t nseg = scan_segments(p), segf = nseg > 1 ? B * H * nseg * d * d : 0;
        f.seg_incr = c.take<float>(segf);
        f.seg_trans = c.take<float>(segf);
        f.seg_start = c.take<float>(segf);
        f.o_la16 = c.take<char>(B * L * H * d * 2);
        f.o_la = nullptr;
    } else {
        f.v16 = nullptr;
        f.kn16 = nullptr;
        f.o_la16 = nullptr;
        f.tc = GdnTcWs{};
        f.seg_incr = f.seg_trans = f.seg_start = nullptr;
        f.W = c.take<float>(B * L * H * d);
        f.U = c.take<float>(B * L * H * d);
        f.P = c.take<float>(B * H * NC * kC * kC);
        f.o_la = c.take<float>(B * L * H * d);
    }
    const size_t nrm = !use_tensor_cores(p) && (p->flags & NATSL_QK_NORM) ? B * L * H * d : 0;
    f.q_la = c.take<float>(nrm);
    f.k_la = c.take<float>(nrm);
    f.q_sm = c.take<float>(nrm);
    f.k_nsm = c.take<float>(nrm);
    f.bytes = c.off;
    return f;
}

struct BwdWs {
    int32_t *status, *emit_flags, *sm_idx, *prefix, *lin_idx, *n_lin, *sm_len;
    size_t head_bytes;                                       // status page + emit_flags: cleared per forward
    float *k_sm32, *v_sm32;                                  // [B,H,L,d] compacted, fp32
    float *q32, *k32, *v32;                                  // token-major fp32 copies
    float *qs32, *ks32;                                      // NATSL_QK_NORM, fp32 storage: RMS-normalised q, k
                                                             // (q32, k32 then hold the L2-normalised ones)
    float *W, *U, *Ut, *o_la, *o_nla, *do_la, *do_nla;       // token-major
    float *dUt, *dQg, *dW, *dKt, *dKb, *dVb, *X1p, *X2, *X3, *X4, *dq_sm, *dk_sm, *dv_sm;
    float *P, *Abar, *M, *N, *Mg, *Ms, *Ns;                  // [B,H,NC,64,64]
    float *S_c, *dS_c;                                       // [B,H,NC,d,d]
    float *Gcum, *lse, *Dsm, *dGrow, *kappa, *gS;            // [B,H,L] (gS: [B,H,NC,d/32])
    float *dk_x, *dv_x, *dmask;                              // block-level routing off the fused path: the
                                                             // softmax branch's dk, dv of every token
                                                             // (token-major), mask gradients per retained key [B,H,L]
    void *k_smb, *k16, *v16, *Qh, *dO16;                     // tensor-core softmax branch: 16-bit [B,H,L,d]
    void *dOla16, *dOlag16;                                  // tensor-core reverse scan: fp16 [B,H,L,d]
    void *o_la16;                                            // linear read-out as fp16 [B,L,H,d]
    GdnTcWs tc;                                              // tensor-core forward recomputation
    float *Tinv;                                             // (I + A)^-1 per chunk [B,H,NC,64,64]
    size_t bytes;
};

// Only what the selected path uses is carved (a buffer the path does not touch gets no bytes and a
// pointer nobody dereferences).  Paths: `fused` = tensor cores with d = 64 (reverse scan + one
// fused kernel per chunk), tensor cores with d = 128 (chunk-level products as batched tile GEMMs),
// fp32 CUDA cores.  Three pairs with disjoint lifetimes share their bytes on the tensor-core paths:
// o_la (dead once the combination's backward has run) / dUt (written by the reverse scan after it),
// o_nla / dq_sm likewise, and the fp16 o_la / the fp16 gradient copy dO16.
BwdWs carve_bwd(const natsl_params *p, void *ws) {
    Carver c(ws);
    BwdWs f;
    const size_t B = p->B, H = p->H, L = p->L, d = p->d, NC = L / kC;
    const size_t TM = B * L * H * d, CC = B * H * NC * kC * kC, ST = B * H * NC * d * d, BHL = B * H * L;
    const bool tcs = use_tensor_cores(p), fused = fused_chunk_path(p), general = !fused;
    const bool block = (p->flags & NATSL_BLOCK_ROUTING) != 0;
    auto tm = [&](bool need) { return c.take<float>(need ? TM : 0); };
    auto cc = [&](bool need) { return c.take<float>(need ? CC : 0); };
    f.status = c.take<int32_t>(kStatusBytes / 4);
    f.emit_flags = c.take<int32_t>(tcs ? B * H * NC : 0);    // per-chunk counters of the scan (forward part)
    f.head_bytes = c.off;
    f.sm_idx = c.take<int32_t>(BHL);
    f.prefix = c.take<int32_t>(B * H * (NC + 1));
    f.lin_idx = c.take<int32_t>(BHL);
    f.n_lin = c.take<int32_t>(B * H * NC);
    f.sm_len = c.take<int32_t>(B * H);
    f.k_sm32 = tm(!tcs); f.v_sm32 = tm(!tcs);
    f.q32 = tm(general); f.k32 = tm(general); f.v32 = tm(general);
    // (needed by the fp32 softmax kernels: all of them for fp32 storage, the own-block one of block-level routing)
    const bool normed = (p->flags & NATSL_QK_NORM) && (!tcs || (general && block));
    f.qs32 = tm(normed); f.ks32 = tm(normed);
    const size_t Gg = p->G > 1 ? (size_t)p->G : 1;           // softmax heads per linear head: lse, Dsm per softmax head
    f.W = tm(general); f.U = tm(general);
    f.Ut = tm(true);
    f.o_la = tm(true);
    f.o_nla = tm(true);
    f.do_la = tm(true);
    f.do_nla = tm(!tcs);
    f.dUt = tcs ? f.o_la : tm(true);
    f.dQg = tm(general); f.dW = tm(general); f.dKt = tm(general); f.dKb = tm(general); f.dVb = tm(general);
    // (the last four products' results: only the fp32 path stores them, the tensor-core path keeps them in
    // the accumulators of its assembly kernel; X3, X4 also serve the fused chunk kernel's block-routed call
    // as its side buffers)
    f.X1p = tm(general && !tcs); f.X2 = tm(general && !tcs);
    f.X3 = tm((general && !tcs) || (fused && block)); f.X4 = tm((general && !tcs) || (fused && block));
    f.dq_sm = tcs ? f.o_nla : tm(true);
    f.dk_sm = tm(true); f.dv_sm = tm(true);
    f.P = cc(!tcs); f.Abar = cc(!tcs);
    f.M = cc(general && !tcs); f.N = cc(general && !tcs);     // (tensor cores: M, N stay in gdn_tm_kernel's accumulators)
    f.Mg = cc(general); f.Ms = cc(general); f.Ns = cc(general);
    f.S_c = c.take<float>(ST);
    f.dS_c = c.take<float>(ST);
    f.Gcum = c.take<float>(BHL);
    f.lse = c.take<float>(BHL * Gg);
    f.Dsm = c.take<float>(BHL * Gg);
    f.dGrow = c.take<float>(BHL);
    f.kappa = c.take<float>(BHL);
    f.gS = c.take<float>(general ? B * H * NC * (d / 32) : 0);
    f.dk_x = tm(general && block); f.dv_x = tm(general && block);
    f.dmask = c.take<float>(general && block ? BHL * Gg : 0);
    const size_t h16 = tcs ? TM * 2 : 0;
    f.k_smb = c.take<char>(h16);
    f.k16 = c.take<char>(h16);
    f.v16 = c.take<char>(h16);
    f.Qh = c.take<char>(h16);
    f.dO16 = c.take<char>(h16);
    f.dOla16 = c.take<char>(h16);
    f.dOlag16 = c.take<char>(h16);
    f.o_la16 = f.dO16;
    f.tc = GdnTcWs{};
    if (tcs) {
        f.tc.Qh = f.Qh;                       // the same fp16 copy of q serves both branches
        f.tc.Kh = c.take<char>(h16);
        f.tc.Wt = c.take<char>(h16);
        f.tc.Ut = c.take<float>(TM);
        f.tc.Ph = c.take<char>(CC * 2);
        f.tc.Gd = c.take<float>(BHL * 2);
        f.Tinv = c.take<float>(CC);
    } else {
        f.Tinv = nullptr;
    }
    f.bytes = c.off;
    return f;
}

}  // namespace

namespace {

// The compaction and the gather of the retained K/V do not depend on the linear branch's prepare
// kernel (and that kernel does not depend on them), so the forward runs them beside it: on a
// library-owned stream per device, forked from the caller's stream with one event and joined back
// with another before the softmax kernel.  Stream and events are created on first use and kept;
// a mutex covers the enqueue of a call, since the two event objects are shared by all calls.
struct SideStream {
    cudaStream_t st = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    bool tried = false;
};
SideStream g_side[64];
std::mutex g_side_mu;

// Joins the side stream back into the caller's stream when a call leaves early after the fork,
// so that no library-owned stream is left with work the caller's stream does not wait for.
struct SideJoin {
    SideStream *side = nullptr;
    cudaStream_t st = nullptr;
    bool pending = false;
    void forked(SideStream *s, cudaStream_t caller) { side = s; st = caller; pending = true; }
    cudaError_t join() {
        if (!pending) return cudaSuccess;
        pending = false;
        cudaError_t e = cudaEventRecord(side->join, side->st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join, 0);
        return e;
    }
    ~SideJoin() { (void)join(); }
};


SideStream *side_stream_locked() {   // g_side_mu held; nullptr: run everything on the caller's stream
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    SideStream &s = g_side[dev];
    if (!s.tried) {
        s.tried = true;
        if (cudaStreamCreateWithFlags(&s.st, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess) {
            s.st = nullptr;
            (void)cudaGetLastError();
        }
    }
    return s.st ? &s : nullptr;
}

}  // namespace

// The forward as the backward needs it: the same kernels as natsl_hybrid_fwd's, which here also leave
// the chunkwise quantities the gradient kernels read (chunk-entry states, U~, (I + A)^-1, cumulative
// decays, log-sum-exp, raw branch outputs) in the backward workspace `f`.  natsl_hybrid_bwd runs it
// itself unless the caller did, through natsl_hybrid_fwd with NATSL_SAVE_FOR_BWD (then `out` and
// `state_out` are produced as well).
static int bwd_forward_part(const void *q, const void *k, const void *v, const float *g,
                            const float *beta, const uint8_t *route, void *out, float *state_out,
                            const natsl_params *p, const BwdWs &f, cudaStream_t st) {
    const Shape s = shape_of(p);
    Shape s32 = s;              // the same shapes with fp32 storage (the fp32 copies)
    s32.bf16 = false;
    const long long B = p->B, H = p->H, L = p->L, d = p->d;
    const bool block = (p->flags & NATSL_BLOCK_ROUTING) != 0;
    const uint8_t *block_route = block ? route : nullptr;
    const bool tensor_cores = use_tensor_cores(p);
    const bool fused_chunks = fused_chunk_path(p);          // chunk-level products in one kernel
    int32_t *flags = tensor_cores && !(p->flags & NATSL_SINGLE_STREAM) ? f.emit_flags : nullptr;
#define NATSL_TRY(call) do { if ((call) != cudaSuccess) return NATSL_ERR_CUDA; } while (0)
    NATSL_TRY(cudaMemsetAsync(f.status, 0, f.head_bytes, st));
    // compaction + gather beside the prepare kernel, on the library's side stream (as in the forward)
    std::unique_lock<std::mutex> side_lock;
    SideStream *side = nullptr;
    SideJoin side_join;
    if (fused_chunks && !(p->flags & NATSL_SINGLE_STREAM)) {
        side_lock = std::unique_lock<std::mutex>(g_side_mu);
        side = side_stream_locked();
        if (!side) side_lock.unlock();
    }
    cudaStream_t st0 = side ? side->st : st;
    if (side) {
        NATSL_TRY(cudaEventRecord(side->fork, st));
        NATSL_TRY(cudaStreamWaitEvent(st0, side->fork, 0));
        side_join.forked(side, st);
    }
    NATSL_TRY(launch_route_compact(route, f.sm_idx, f.prefix, f.lin_idx, f.n_lin, f.sm_len, nullptr,
                                   block ? f.status : nullptr, p->L, p->B, p->L, p->H, st0));
    const HeadGroups hg = head_groups(p);
    if (!fused_chunks) {     // (with NATSL_QK_NORM the copies of q, k are the normalised ones, made below)
        const bool qk = hg.norm_eps < 0.f;
        NATSL_TRY(launch_to_f32(qk ? q : nullptr, qk ? k : nullptr, v, f.q32, f.k32, f.v32,
                                (size_t)(B * L * H * d), s.bf16, st));
    }
    // fp32 storage with NATSL_QK_NORM: q32, k32 become the L2-normalised rows (everything of the linear
    // branch reads those), qs32, ks32 the slice-wise RMS-normalised ones (softmax branch)
    // (tensor cores: the kernels normalise inside; only the fp32 copies the separate chunk-level products
    // of the backward read are made here)
    const float *qs = f.q32, *ks = f.k32;
    if (hg.norm_eps >= 0.f) {
        const bool rms_copies = !tensor_cores || block;
        NATSL_TRY(launch_qk_norm_f32(q, k, s.bf16, f.q32, f.k32, rms_copies ? f.qs32 : nullptr,
                                     rms_copies ? f.ks32 : nullptr, (size_t)(B * L * H), p->d, hg.G,
                                     hg.norm_eps, st));
        if (!tensor_cores) { qs = f.qs32; ks = f.ks32; }
    }
    if (tensor_cores)
        NATSL_TRY(launch_gather_kv_tc(k, v, f.sm_idx, f.prefix, f.k_smb, nullptr, f.v16, f.k16, p->L,
                                      p->L, false, f.status, s, st0, hg));
    else
        NATSL_TRY(launch_gather_kv(ks, f.v32, f.sm_idx, f.prefix, f.k_sm32, f.v_sm32, p->L,
                                   f.status, s32, st));
    if (tensor_cores) {
        // the fused chunk kernel reads W^T, U^T as the forward keeps them: no fp32 copies for it
        const GdnTcExport ex{fused_chunks ? nullptr : f.W, fused_chunks ? nullptr : f.U, nullptr, f.Tinv,
                             f.Gcum, f.S_c, f.Ut};
        NATSL_TRY(launch_gdn_prepare_tc(q, k, v, g, beta, block ? nullptr : route, p->scale_la, f.tc, ex,
                                        f.status, s, st, hg.norm_eps));
        // (the side stream joins before the scan, so that the softmax kernel follows the scan directly
        // and can run beside it as its programmatic dependent, as in natsl_hybrid_fwd)
        NATSL_TRY(side_join.join());
        NATSL_TRY(launch_gdn_scan_tc(f.tc, p->scale_la, p->state_in, state_out, ScanOut{f.o_la16, f.o_la, flags},
                                     ex, ScanSegments{0, 1, 0, nullptr, nullptr, nullptr}, block_route,
                                     f.status, s, st));
    } else {
        NATSL_TRY(launch_gdn_prepare_simt(f.q32, f.k32, f.v32, g, beta, block ? nullptr : route, p->scale_la,
                                          f.W, f.U, f.P, f.Abar, f.Gcum, s32, st));
        NATSL_TRY(launch_gdn_scan_simt(f.q32, f.k32, g, f.W, f.U, f.P, p->scale_la, p->state_in, state_out,
                                       f.S_c, f.Ut, f.o_la, block_route, s32, st));
    }
    NATSL_TRY(side_join.join());
    if (tensor_cores)
        NATSL_TRY(launch_softmax_combine_tc(q, f.k_smb, f.v16, p->L, p->L, f.sm_idx, f.prefix, f.o_la16,
                                            flags, p->w, p->scale_sm, p->eps, out, f.o_nla, f.lse,
                                            BlockRouting{block_route, k, v}, false, f.status, s, st, hg));
    else
        NATSL_TRY(launch_softmax_combine_simt(qs, f.k_sm32, f.v_sm32, p->L, f.sm_idx, f.prefix,
                                              f.o_la, p->w, p->scale_sm, p->eps, out, f.o_nla,
                                              f.lse, BlockRouting{block_route, ks, f.v32}, s32, st, hg.G));
#undef NATSL_TRY
    return NATSL_OK;
}

extern "C" {

uint64_t natsl_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *natsl_stage_name(int op, int i) {
    static const char *fwd[] = {"route_compact+gather_kv", "gdn_prepare", "gdn_scan",
                                "softmax_combine"};
    if (op == NATSL_OP_FWD && i >= 0 && i < 4) return fwd[i];
    if (op == NATSL_OP_DECODE && i == 0) return "decode_step";
    return nullptr;
}

const char *natsl_strerror(int status) {
    switch (status) {
        case NATSL_OK: return "ok";
        case NATSL_ERR_NULL: return "a required pointer is NULL";
        case NATSL_ERR_SHAPE: return "unsupported shape (need B,H,L>0, L%64==0, d in {64,128}, C==64, eps>0)";
        case NATSL_ERR_DTYPE: return "dtype must be NATSL_F32 or NATSL_BF16";
        case NATSL_ERR_ALIGN: return "tensor base pointer not 16-byte aligned";
        case NATSL_ERR_WORKSPACE: return "workspace missing or too small";
        case NATSL_ERR_CUDA: return "CUDA launch or runtime error";
        case NATSL_ERR_CACHE_FULL: return "retained-KV cache full";
        case NATSL_ERR_UNSUPPORTED: return "request not implemented in this build";
        case NATSL_ERR_ROUTE: return "block-level routing: route changes inside a block";
        case NATSL_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case NATSL_ERR_TOO_LARGE: return "problem needs more scratch than the library's built-in array (NATSL_STATIC_WS_BYTES)";
        default: return "unknown natsl status";
    }
}

int natsl_workspace_size(const natsl_params *p, int op, size_t *bytes) {
    if (!bytes) return NATSL_ERR_NULL;
    int rc = check_params(p, op != NATSL_OP_DECODE);
    if (rc != NATSL_OK) return rc;
    switch (op) {
        case NATSL_OP_FWD: *bytes = carve_fwd(p, nullptr).bytes; return NATSL_OK;
        case NATSL_OP_BWD: *bytes = carve_bwd(p, nullptr).bytes; return NATSL_OK;
        case NATSL_OP_DECODE: *bytes = decode_workspace_bytes(p->B, p->H, p->d); return NATSL_OK;
        case NATSL_OP_COMPACT: *bytes = 0; return NATSL_OK;
        default: return NATSL_ERR_UNSUPPORTED;
    }
}

int natsl_route_compact(const uint8_t *route, int32_t *sm_idx, int32_t *sm_chunk_prefix,
                        int32_t *lin_idx, int32_t *n_lin, const natsl_params *p, void *, size_t,
                        void *stream) {
    int rc = check_params(p, true);
    if (rc != NATSL_OK) return rc;
    if (!route || !sm_idx || !sm_chunk_prefix || !lin_idx || !n_lin) return NATSL_ERR_NULL;
    cudaError_t e = launch_route_compact(route, sm_idx, sm_chunk_prefix, lin_idx, n_lin, nullptr,
                                         nullptr, nullptr, 0, p->B, p->L, p->H,
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NATSL_OK : NATSL_ERR_CUDA;
}

int natsl_score_layer(const void *x, const float *w_score, float *scores, uint8_t *route,
                      int32_t d_model, const natsl_params *p, void *stream) {
    int rc = check_params(p, true);
    if (rc != NATSL_OK) return rc;
    if (!x || !w_score || !route) return NATSL_ERR_NULL;
    // a row of X is read in 16-byte pieces
    const int per16 = p->dtype == NATSL_BF16 ? 8 : 4;
    // (the pooled rows of a CTA's two chunks and their scores live in shared memory)
    if (d_model <= 0 || d_model % per16 != 0 || ((size_t)d_model + 2 * (size_t)p->H) * 8 > 200 * 1024)
        return NATSL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(w_score)) return NATSL_ERR_ALIGN;
    cudaError_t e = launch_score_layer(x, w_score, scores, route, d_model, shape_of(p),
                                       static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NATSL_OK : NATSL_ERR_CUDA;
}

int natsl_hybrid_fwd(const void *q, const void *k, const void *v, const float *g,
                     const float *beta, const uint8_t *route, void *out, const natsl_params *p,
                     void *ws, size_t ws_bytes, void *stream) {
    int rc = check_params(p, true);
    if (rc != NATSL_OK) return rc;
    if (!q || !k || !v || !g || !beta || !route || !out) return NATSL_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(ws))
        return NATSL_ERR_ALIGN;
    const bool want_cache = p->k_sm || p->v_sm || p->sm_len;
    if (want_cache && !(p->k_sm && p->v_sm && p->sm_len && p->sm_cap > 0)) return NATSL_ERR_NULL;
    if (want_cache && (!aligned16(p->k_sm) || !aligned16(p->v_sm))) return NATSL_ERR_ALIGN;
    if ((p->o_la && !aligned16(p->o_la)) || (p->o_nla && !aligned16(p->o_nla))) return NATSL_ERR_ALIGN;
    const bool tensor_cores = use_tensor_cores(p);
    if (tensor_cores && !(p->scale_sm > 0.f)) return NATSL_ERR_SHAPE;   // (its kernel takes the maximum of raw logits)
    const bool block = (p->flags & NATSL_BLOCK_ROUTING) != 0;
    const bool append = (p->flags & NATSL_APPEND_CACHE) != 0;
    if (append && !tensor_cores) return NATSL_ERR_UNSUPPORTED;
    if (append && !want_cache) return NATSL_ERR_NULL;
    const HeadGroups hg = head_groups(p);
    if (grouped_or_normed(p)) {
        if (tensor_cores) {
            if (hg.G > 1 && !(hg.G == 2 && p->d == 128)) return NATSL_ERR_UNSUPPORTED;
            // (the saved forward is the backward's forward part: built where the backward is)
            if ((p->flags & NATSL_SAVE_FOR_BWD) && hg.G > 1 && p->d != 128) return NATSL_ERR_UNSUPPORTED;
        } else {
            if (p->dtype != NATSL_F32) return NATSL_ERR_UNSUPPORTED;
            if (hg.G > 1 && (hg.G > 4 || p->d / hg.G < 32)) return NATSL_ERR_UNSUPPORTED;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (p->flags & NATSL_SAVE_FOR_BWD) {
        // The forward of a training step: run in the backward's workspace, where it leaves what
        // natsl_hybrid_bwd (with NATSL_SAVED_FWD) would otherwise compute again.
        if (append || want_cache || p->o_la || p->o_nla || p->lse || p->stage_events) return NATSL_ERR_UNSUPPORTED;
        const BwdWs fb = carve_bwd(p, ws);
        if (!ws || ws_bytes < fb.bytes) return NATSL_ERR_WORKSPACE;
        return bwd_forward_part(q, k, v, g, beta, route, out, p->state_out, p, fb, st);
    }
    FwdWs f = carve_fwd(p, ws);
    if (!ws || ws_bytes < f.bytes) return NATSL_ERR_WORKSPACE;
    const Shape s = shape_of(p);
    const BlockRouting br{block ? route : nullptr, k, v};

#define NATSL_TRY(call) do { if ((call) != cudaSuccess) return NATSL_ERR_CUDA; } while (0)
    int stage = 0;
    auto mark = [&]() -> cudaError_t {
        if (p->stage_events && stage < p->n_stage_events)
            return cudaEventRecord(static_cast<cudaEvent_t>(p->stage_events[stage++]), st);
        return cudaSuccess;
    };
    NATSL_TRY(cudaMemsetAsync(f.status, 0, f.head_bytes, st));
    NATSL_TRY(mark());
    // Stage 0 (compaction, gather) beside stage 1 (prepare) on the side stream -- unless the caller
    // asks for one stream or for per-stage events, whose differences are only meaningful in sequence.
    std::unique_lock<std::mutex> side_lock;
    SideStream *side = nullptr;
    SideJoin side_join;
    if (tensor_cores && !(p->flags & NATSL_SINGLE_STREAM) && !p->stage_events) {
        side_lock = std::unique_lock<std::mutex>(g_side_mu);
        side = side_stream_locked();
        if (!side) side_lock.unlock();
    }
    cudaStream_t st0 = side ? side->st : st;
    if (side) {
        NATSL_TRY(cudaEventRecord(side->fork, st));
        NATSL_TRY(cudaStreamWaitEvent(st0, side->fork, 0));
        side_join.forked(side, st);
    }
    int32_t *sm_len = want_cache ? p->sm_len : f.sm_len;
    void *k_sm = want_cache ? p->k_sm : f.k_sm, *v_sm = want_cache ? p->v_sm : f.v_sm;
    const int32_t cap = want_cache ? p->sm_cap : p->L;
    const int32_t capv = append ? p->sm_cap : p->L;          // rows per head of the fp16 V copy
    NATSL_TRY(launch_route_compact(route, f.sm_idx, f.prefix, f.lin_idx, f.n_lin, sm_len,
                                   append ? sm_len : nullptr, block ? f.status : nullptr, cap, p->B,
                                   p->L, p->H, st0));
    // fp32 storage with NATSL_QK_NORM: normalised copies first (the tensor-core kernels normalise inside)
    const void *q_la = q, *k_la = k, *q_sm = q, *k_nsm = k;
    if (!tensor_cores && hg.norm_eps >= 0.f) {
        NATSL_TRY(launch_qk_norm_f32(q, k, false, f.q_la, f.k_la, f.q_sm, f.k_nsm,
                                     (size_t)p->B * p->L * p->H, p->d, hg.G, hg.norm_eps, st));
        q_la = f.q_la; k_la = f.k_la; q_sm = f.q_sm; k_nsm = f.k_nsm;
    }
    // A cache the call returns keeps the keys as given (the decode step normalises them as it reads them);
    // with the normalisation the softmax kernel then reads a normalised copy in the workspace instead.
    const bool raw_cache = want_cache && hg.norm_eps >= 0.f;
    void *k_norm = append ? f.kn16 : f.k_sm;     // (appending: normalised copies of the whole cache, capv rows per head)
    const void *k_soft = raw_cache ? k_norm : k_sm, *v_soft = raw_cache ? f.v_sm : v_sm;
    const int32_t cap_soft = raw_cache ? capv : cap;
    if (tensor_cores) {
        NATSL_TRY(launch_gather_kv_tc(k, v, f.sm_idx, f.prefix, k_sm, want_cache ? v_sm : nullptr,
                                      f.v16, raw_cache ? k_norm : nullptr, cap, capv, append, f.status, s, st0,
                                      hg, raw_cache));
    } else {
        if (raw_cache) NATSL_TRY(launch_gather_kv(k, v, f.sm_idx, f.prefix, k_sm, v_sm, cap, f.status, s, st));
        NATSL_TRY(launch_gather_kv(k_nsm, v, f.sm_idx, f.prefix, raw_cache ? f.k_sm : k_sm,
                                   raw_cache ? f.v_sm : v_sm, cap_soft, f.status, s, st));
    }
    NATSL_TRY(mark());
    if (tensor_cores) {
        // block-level routing: every token takes part in the delta rule of its own block
        const bool beside = !p->stage_events && !(p->flags & NATSL_SINGLE_STREAM);
        const int nseg = scan_segments(p);
        NATSL_TRY(launch_gdn_prepare_tc(q, k, v, g, beta, block ? nullptr : route, p->scale_la, f.tc,
                                        GdnTcExport{}, f.status, s, st, hg.norm_eps));
        NATSL_TRY(mark());
        // The side stream joins here, before the scan, so that nothing stands between the scan and
        // the softmax kernel in the stream: the softmax kernel is launched as a programmatic dependent
        // of the scan, starts once the scan's CTAs are all resident, runs its Q K^T / P V loop beside
        // it on the multiprocessors the scan leaves free, and picks up o_la chunk by chunk behind the
        // counters the scan raises.  Per-stage events and NATSL_SINGLE_STREAM switch this off
        // (stages in sequence).
        NATSL_TRY(side_join.join());
        int32_t *flags_scan = beside && !g_debug_withhold_flags.load(std::memory_order_relaxed) ? f.emit_flags : nullptr;
        const int32_t *flags_softmax = beside ? f.emit_flags : nullptr;
        const ScanOut so{f.o_la16, p->o_la, flags_scan};
        if (nseg > 1) {   // few (batch, head) pairs: segments in parallel, chained by their transitions
            ScanSegments sg{1, nseg, (int)(p->L / kC) / nseg, f.seg_incr, f.seg_trans, f.seg_start};
            NATSL_TRY(launch_gdn_scan_tc(f.tc, p->scale_la, nullptr, nullptr, so, GdnTcExport{}, sg,
                                         br.route, f.status, s, st));
            NATSL_TRY(launch_scan_combine(p->state_in, sg, s, st));
            sg.mode = 2;
            NATSL_TRY(launch_gdn_scan_tc(f.tc, p->scale_la, nullptr, p->state_out, so, GdnTcExport{}, sg,
                                         br.route, f.status, s, st));
        } else {
            NATSL_TRY(launch_gdn_scan_tc(f.tc, p->scale_la, p->state_in, p->state_out, so, GdnTcExport{},
                                         ScanSegments{0, 1, 0, nullptr, nullptr, nullptr}, br.route,
                                         f.status, s, st));
        }
        NATSL_TRY(mark());
        NATSL_TRY(launch_softmax_combine_tc(q, k_soft, f.v16, cap_soft, capv, f.sm_idx, f.prefix, f.o_la16,
                                            flags_softmax, p->w, p->scale_sm, p->eps, out, p->o_nla,
                                            p->lse, br, append, f.status, s, st, hg));
    } else {
        float *o_la = p->o_la ? p->o_la : f.o_la;
        NATSL_TRY(launch_gdn_prepare_simt(q_la, k_la, v, g, beta, block ? nullptr : route, p->scale_la, f.W,
                                          f.U, f.P, nullptr, nullptr, s, st));
        NATSL_TRY(mark());
        NATSL_TRY(launch_gdn_scan_simt(q_la, k_la, g, f.W, f.U, f.P, p->scale_la, p->state_in,
                                       p->state_out, nullptr, nullptr, o_la, br.route, s, st));
        NATSL_TRY(mark());
        // (an own-block tile of block-level routing reads the layer's keys: the softmax operation's copy)
        NATSL_TRY(launch_softmax_combine_simt(q_sm, k_soft, v_soft, cap_soft, f.sm_idx, f.prefix, o_la, p->w,
                                              p->scale_sm, p->eps, out, p->o_nla, p->lse,
                                              BlockRouting{br.route, k_nsm, v}, s, st, hg.G));
    }
    NATSL_TRY(mark());
#undef NATSL_TRY
    return NATSL_OK;
}

int natsl_hybrid_bwd(const void *q, const void *k, const void *v, const float *g,
                     const float *beta, const uint8_t *route, const void *dout, void *dq, void *dk,
                     void *dv, float *dg, float *dbeta, float *dw, const natsl_params *p, void *ws,
                     size_t ws_bytes, void *stream) {
    int rc = check_params(p, true);
    if (rc != NATSL_OK) return rc;
    if (!q || !k || !v || !g || !beta || !route || !dout || !dq || !dk || !dv || !dg || !dbeta)
        return NATSL_ERR_NULL;
    if (p->flags & NATSL_APPEND_CACHE) return NATSL_ERR_UNSUPPORTED;
    const HeadGroups hg = head_groups(p);
    if (grouped_or_normed(p)) {      // grouped heads, q/k normalisation: the paths with separate chunk-level products
        if (use_tensor_cores(p)) {      // softmax heads of 64 or 128 columns
            if (!((p->d == 128 && hg.G <= 2) || (p->d == 64 && hg.G == 1))) return NATSL_ERR_UNSUPPORTED;
        } else {
            if (p->dtype != NATSL_F32) return NATSL_ERR_UNSUPPORTED;
            if (hg.G > 1 && (hg.G > 4 || p->d / hg.G < 32)) return NATSL_ERR_UNSUPPORTED;
        }
    }
    if (use_tensor_cores(p) && !(p->scale_sm > 0.f)) return NATSL_ERR_SHAPE;
    const bool block = (p->flags & NATSL_BLOCK_ROUTING) != 0;
    if (p->dscore && !block) return NATSL_ERR_UNSUPPORTED;   // score gradients: one decision per block
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dout) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv) || !aligned16(ws))
        return NATSL_ERR_ALIGN;
    BwdWs f = carve_bwd(p, ws);
    if (!ws || ws_bytes < f.bytes) return NATSL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Shape s = shape_of(p);
    Shape s32 = s;              // the same shapes with fp32 storage (the fp32 copies)
    s32.bf16 = false;
    const long long B = p->B, H = p->H, L = p->L, d = p->d, NC = L / kC;
    auto TM = [&](const float *x) { return BMat{x, L * H * d, d, (long long)kC * H * d, (int)(H * d)}; };
    auto CC = [&](const float *x) { return BMat{x, H * NC * kC * kC, NC * kC * kC, (long long)kC * kC, kC}; };
    auto ST = [&](const float *x) { return BMat{x, H * NC * d * d, NC * d * d, d * d, (int)d}; };
    const int di = p->d;
    const uint8_t *block_route = block ? route : nullptr;
    const bool tensor_cores = use_tensor_cores(p);
    const bool fused_chunks = fused_chunk_path(p);          // chunk-level products in one kernel

    // ---- forward, keeping what the backward needs (unless the caller's forward already did) ----
    if (!(p->flags & NATSL_SAVED_FWD)) {
        rc = bwd_forward_part(q, k, v, g, beta, route, nullptr, nullptr, p, f, st);
        if (rc != NATSL_OK) return rc;
    }
#define NATSL_TRY(call) do { if ((call) != cudaSuccess) return NATSL_ERR_CUDA; } while (0)
    // From here on two more pairs of independent stages run side by side on the library's side
    // stream: the reverse scan of the linear branch beside the softmax branch's backward.
    std::unique_lock<std::mutex> side_lock;
    SideStream *side = nullptr;
    SideJoin side_join;
    // (tensor cores with separate chunk-level kernels: the whole linear branch -- reverse scan, the products
    // with the states, the middle of the chain -- runs on the side stream beside the softmax branch's
    // backward, and the two meet at the assembly)
    const bool side_general = tensor_cores && !fused_chunks;
    if ((fused_chunks || side_general) && !(p->flags & NATSL_SINGLE_STREAM)) {
        side_lock = std::unique_lock<std::mutex>(g_side_mu);
        side = side_stream_locked();
        if (!side) side_lock.unlock();
    }
    cudaStream_t st0 = side ? side->st : st;
    // ---- combination and softmax branch ----
    // Tensor cores: the fp16 gradient operands are scaled by a power of two taken from max |dout|,
    // so that a loss-scaled or a tiny dout stays inside fp16's range (grad_scale, common.cuh).
    if (tensor_cores) NATSL_TRY(launch_dout_amax(dout, (size_t)(B * L * H * d), s.bf16, f.status, st));
    const int32_t *gsc = tensor_cores ? f.status : nullptr;
    const bool general_block = block && !fused_chunks;   // block-level routing with separate chunk-level products
    NATSL_TRY(launch_combine_bwd(f.o_la, f.o_nla, dout, p->w, p->eps, f.do_la,
                                 tensor_cores ? nullptr : f.do_nla, dw, f.Dsm,
                                 tensor_cores ? f.dO16 : nullptr, tensor_cores ? f.dOla16 : nullptr,
                                 tensor_cores ? f.dOlag16 : nullptr, f.tc.Gd, p->scale_la, gsc, s, st, hg.G));
    // Dependencies from here on: the query-side softmax kernel, the key-side one and the reverse
    // scan need only what is already there; the chunk kernel needs the first and the third; the
    // scatter of the retained tokens' dk, dv needs the second.  With token-level routing the chunk
    // kernel therefore does not wait for the key-side kernel: side stream = reverse scan, key-side
    // kernel, scatter; caller's stream = query-side kernel, chunk kernel.  (Block-level routing:
    // the chunk kernel adds the scattered gradients and so waits for the side stream, but the
    // own-block kernel, which needs the query-side kernel only, still runs beside the key-side one.)
    const bool kv_aside = side != nullptr && fused_chunks;
    if (side) {
        NATSL_TRY(cudaEventRecord(side->fork, st));
        NATSL_TRY(cudaStreamWaitEvent(st0, side->fork, 0));
        side_join.forked(side, st);
    }
    // ---- linear branch: reverse scan (then chunk-parallel products) ----
    if (tensor_cores)
        NATSL_TRY(launch_gdn_rscan_tc(f.dOla16, f.dOlag16, f.tc, f.S_c, f.dUt, f.dS_c,
                                      fused_chunks ? nullptr : f.gS, p->dstate_out, p->dstate_in,
                                      block_route, f.status, s, st0));
    if (side && fused_chunks) NATSL_TRY(cudaEventRecord(side->join, st0));
    if (tensor_cores)   // (d = 64: the prepare kernel has left the fp16 copy of q in f.Qh, and the reverse
                        //  scan on the side stream reads it, so it is not written again)
        // (separate chunk-level kernels: the softmax branch writes its own fp16 copy of q -- raw, or RMS-
        //  normalised -- while the reverse scan beside it reads the linear operation's copy in f.Qh; the copy
        //  goes where the forward's softmax kernel had its gathered keys, which nothing reads any more)
        NATSL_TRY(launch_softmax_bwd_tc(q, fused_chunks ? f.Qh : f.k_smb, f.dO16, f.k16, f.v16, p->L, f.sm_idx, f.prefix, f.lse,
                                        f.Dsm, p->scale_sm, f.dq_sm, f.dk_sm, f.dv_sm,
                                        p->dscore ? (general_block ? f.dmask : f.dGrow) : nullptr, fused_chunks,
                                        f.status, s, st, kv_aside ? st0 : st, hg));
    else
        NATSL_TRY(launch_softmax_bwd(hg.norm_eps >= 0.f ? f.qs32 : f.q32, f.k_sm32, f.v_sm32, p->L, f.sm_idx,
                                     f.prefix, f.do_nla, f.lse, f.Dsm, p->scale_sm, f.dq_sm, f.dk_sm, f.dv_sm,
                                     s, st, p->dscore ? f.dmask : nullptr, hg.G));
    if (!tensor_cores)
        NATSL_TRY(launch_gdn_rscan(f.q32, f.k32, f.Gcum, f.W, f.P, f.do_la, f.S_c, p->scale_la, f.dUt,
                                   f.dS_c, f.gS, p->dstate_out, p->dstate_in, s, st, block_route));
    if (side && fused_chunks) NATSL_TRY(cudaStreamWaitEvent(st, side->join, 0));     // the reverse scan has finished
    // (with the normalisation the two operations' dq stay apart until its backward at the very end)
    const bool normed = hg.norm_eps >= 0.f;
    AssembleArgs a{f.q32, f.k32, f.v32, f.Gcum, beta, general_block ? nullptr : route, f.dQg, f.dKb, f.dVb, f.dKt, f.X1p, f.X2,
                   f.X3, f.X4, normed ? nullptr : f.dq_sm, f.dk_sm, f.dv_sm, f.gS, f.sm_idx, f.prefix, p->L,
                   p->scale_la, f.dGrow, f.kappa, dbeta, dg};
    if (fused_chunks && block) {
        // Every token has a softmax-branch dk, dv here: the retained tokens' from the compacted
        // gradients, the tokens of linear blocks' from their own block.  Both go to fp32
        // token-major buffers (each token is written by exactly one of the two), which the chunk
        // kernel adds to its own dk, dv.
        float *dk_x = f.X3, *dv_x = f.X4;
        NATSL_TRY(launch_gdn_finish(a, dk_x, dv_x, s32, kv_aside ? st0 : st, false));
        NATSL_TRY(launch_softmax_bwd_own_block(q, k, v, f.dO16, f.lse, f.Dsm, route, p->scale_sm,
                                               f.dq_sm, dk_x, dv_x, gsc, s, st));
        NATSL_TRY(side_join.join());      // the side stream's last kernels
        NATSL_TRY(launch_gdn_bwd_chunk(q, k, v, f.do_la, f.dUt, f.Ut, f.S_c, f.dS_c, f.Tinv, f.tc.Wt, f.tc.Ut,
                                       f.Gcum, beta, route, f.dq_sm, p->scale_la, dq, dk, dv, dg, dbeta,
                                       true, dk_x, dv_x, p->dscore ? f.kappa : nullptr, s, st));
        if (p->dscore)   // (dGrow, kappa: [B,H,L] scratch the fused path does not otherwise use)
            NATSL_TRY(launch_dscore(route, f.prefix, f.dGrow, f.kappa, nullptr, p->L, p->dscore, s, st));
        return NATSL_OK;
    }
    if (fused_chunks) {   // all chunk-level products and the assembly in one kernel per chunk
        NATSL_TRY(launch_gdn_bwd_chunk(q, k, v, f.do_la, f.dUt, f.Ut, f.S_c, f.dS_c, f.Tinv, f.tc.Wt, f.tc.Ut,
                                       f.Gcum, beta, route, f.dq_sm, p->scale_la, dq, dk, dv, dg, dbeta,
                                       false, nullptr, nullptr, nullptr, s, st));
        // scatter of the retained tokens' dk, dv (rows the chunk kernel does not write)
        NATSL_TRY(launch_gdn_finish(a, dk, dv, s, kv_aside ? st0 : st, false));
        NATSL_TRY(side_join.join());      // the side stream's last kernels
        return NATSL_OK;
    }
    // (the tile GEMMs run on tf32 tensor cores for bf16 storage -- unless the caller asked for fp32
    // arithmetic -- and as fp32 FMAs otherwise: launch_bgemm goes by the storage type it is told)
    const Shape sgemm = tensor_cores ? s : s32;
    // (block-level routing: beta~ = beta for every token, so the kernels below get no route)
    const uint8_t *route_bt = general_block ? nullptr : route;
    if (general_block) {
        // Every token has a softmax-branch dk, dv: the retained tokens' from the compacted gradients, the
        // tokens of linear blocks' from their own block (each token is written by exactly one of the
        // two); the assembly adds them to the linear branch's.
        // (With the normalisation the own-block kernel reads the softmax operation's copies of q and k, and
        // dk_x -- a gradient with respect to that copy -- stays apart from the linear branch's dk until the
        // normalisations' backward.)
        NATSL_TRY(launch_gdn_finish(a, f.dk_x, f.dv_x, s32, st, false));
        if (tensor_cores)      // softmax heads of 64 or 128 columns: warp-level tensor cores
            NATSL_TRY(launch_softmax_bwd_own_block(q, k, v, f.dO16, f.lse, f.Dsm, route, p->scale_sm, f.dq_sm,
                                                   f.dk_x, f.dv_x, gsc, s, st, hg.G, normed ? f.qs32 : nullptr,
                                                   normed ? f.ks32 : nullptr));
        else
            NATSL_TRY(launch_softmax_bwd_own_block_simt(normed ? f.qs32 : f.q32, normed ? f.ks32 : f.k32, f.v32,
                                                        f.do_nla, f.lse, f.Dsm, route, p->scale_sm, f.dq_sm, f.dk_x,
                                                        f.dv_x, gsc, s32, st, hg.G));
        a.dk_x = normed ? nullptr : f.dk_x;
        a.dv_x = f.dv_x;
        a.no_scatter = true;
    }
    cudaStream_t stl = side ? st0 : st;     // the linear branch's stream (behind the reverse scan)
    NATSL_TRY(launch_bgemm(false, true, 0, TM(f.do_la), ST(f.S_c), TM(f.dQg), kC, di, di, 1.f, false, sgemm, stl));
    NATSL_TRY(launch_bgemm(false, true, 0, TM(f.dUt), ST(f.S_c), TM(f.dW), kC, di, di, -1.f, false, sgemm, stl));
    NATSL_TRY(launch_bgemm(false, true, 0, TM(f.Ut), ST(f.dS_c), TM(f.dKt), kC, di, di, 1.f, false, sgemm, stl));
    if (tensor_cores) {   // [dKb | dVb] = (I + A)^-T [dW | dU~] with the inverse the forward already formed, M, N and
                          // their masked, scaled forms: one kernel per chunk
        NATSL_TRY(launch_gdn_tm(f.Tinv, f.dW, f.dUt, f.W, f.U, f.do_la, f.Ut, f.Gcum, beta, route_bt, p->scale_la,
                                f.dKb, f.dVb, f.Mg, f.Ms, f.Ns, s, stl));
        NATSL_TRY(side_join.join());      // the two branches meet at the assembly
    } else {
        NATSL_TRY(launch_bgemm(false, true, 1, TM(f.do_la), TM(f.Ut), CC(f.N), kC, kC, di, 1.f, false, sgemm, st));
        NATSL_TRY(launch_gdn_tsolve(f.Abar, beta, route_bt, f.dW, f.dUt, f.dKb, f.dVb, s, st));
        NATSL_TRY(launch_bgemm(false, true, 2, TM(f.dKb), TM(f.W), CC(f.M), kC, kC, di, -1.f, false, sgemm, st));
        NATSL_TRY(launch_bgemm(false, true, 2, TM(f.dVb), TM(f.U), CC(f.M), kC, kC, di, -1.f, true, sgemm, st));
        NATSL_TRY(launch_mask_scale(f.M, f.N, f.Gcum, beta, route_bt, p->scale_la, f.Mg, f.Ms, f.Ns, s, st));
    }
    // The last four products (X1 = Mg K, X2 = Ms^T K, X3 = Ns K, X4 = Ns^T Q) and the assembly: on tensor
    // cores one kernel per chunk that keeps the products in its accumulators; otherwise four tile GEMMs
    // and the row-local assembly.
    auto assemble = [&](void *dq_o, void *dk_o, void *dv_o, Shape so) -> cudaError_t {
        if (tensor_cores) return launch_gdn_xassemble(a, f.Mg, f.Ms, f.Ns, dq_o, dk_o, dv_o, so, st);
        cudaError_t e;
        if ((e = launch_bgemm(false, false, 0, CC(f.Mg), TM(f.k32), TM(f.X1p), kC, di, kC, 1.f, false, sgemm, st)) != cudaSuccess) return e;
        if ((e = launch_bgemm(true, false, 0, CC(f.Ms), TM(f.k32), TM(f.X2), kC, di, kC, 1.f, false, sgemm, st)) != cudaSuccess) return e;
        if ((e = launch_bgemm(false, false, 0, CC(f.Ns), TM(f.k32), TM(f.X3), kC, di, kC, 1.f, false, sgemm, st)) != cudaSuccess) return e;
        if ((e = launch_bgemm(true, false, 0, CC(f.Ns), TM(f.q32), TM(f.X4), kC, di, kC, 1.f, false, sgemm, st)) != cudaSuccess) return e;
        return launch_gdn_assemble(a, dq_o, dk_o, dv_o, so, st);
    };
    // With the normalisation the assembly's dq, dk are gradients with respect to the normalised rows; a
    // last kernel applies the two row-local Jacobians.  fp32 storage: in place.  bf16 storage: the
    // assembly writes fp32 (into buffers the chunk-level products are done with) and the last kernel
    // rounds once.
    if (!normed) {
        NATSL_TRY(assemble(dq, dk, dv, s));
    } else if (!s.bf16) {
        NATSL_TRY(assemble(dq, dk, dv, s));
        NATSL_TRY(launch_qk_norm_bwd_f32(q, k, false, route, (const float *)dq, f.dq_sm, (const float *)dk, nullptr,
                                         dq, dk, nullptr, (size_t)(B * L * H), p->d, hg.G, hg.norm_eps, st,
                                         general_block ? f.dk_x : nullptr));
    } else {
        float *dq32 = f.dW, *dk32 = f.W, *dv32 = f.U;
        NATSL_TRY(assemble(dq32, dk32, dv32, s32));
        NATSL_TRY(launch_qk_norm_bwd_f32(q, k, true, route, dq32, f.dq_sm, dk32, dv32, dq, dk, dv,
                                         (size_t)(B * L * H), p->d, hg.G, hg.norm_eps, st,
                                         general_block ? f.dk_x : nullptr));
    }
    if (p->dscore)   // softmax blocks: the mask gradients of their keys; linear blocks: the kappa of their tokens
        NATSL_TRY(launch_dscore(route, f.prefix, f.dmask, nullptr, f.kappa, p->L, p->dscore, s, st, hg.G));
#undef NATSL_TRY
    return NATSL_OK;
}

int natsl_decode_step(const void *q, const void *k, const void *v, const float *g,
                      const float *beta, const uint8_t *route, float *state, void *k_cache,
                      void *v_cache, int32_t *cache_len, int32_t cache_cap, void *out,
                      const natsl_params *p, void *ws, size_t ws_bytes, void *stream) {
    int rc = check_params(p, false);
    if (rc != NATSL_OK) return rc;
    if (!q || !k || !v || !g || !beta || !route || !state || !k_cache || !v_cache || !cache_len ||
        !out)
        return NATSL_ERR_NULL;
    if (cache_cap <= 0) return NATSL_ERR_SHAPE;
    const HeadGroups hg = head_groups(p);
    if (hg.G > 1 && (hg.G > 4 || p->d / hg.G < 32)) return NATSL_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(state) ||
        !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return NATSL_ERR_ALIGN;
    if (!ws || ws_bytes < decode_workspace_bytes(p->B, p->H, p->d)) return NATSL_ERR_WORKSPACE;
    cudaError_t e = launch_decode_step(q, k, v, g, beta, route, p->w, state, k_cache, v_cache,
                                       cache_len, cache_cap, out, p->scale_la, p->scale_sm, p->eps,
                                       ws, shape_of(p),
                                       static_cast<cudaStream_t>(stream), hg);
    return e == cudaSuccess ? NATSL_OK : NATSL_ERR_CUDA;
}

int natsl_decode_block_end(const uint8_t *route_block, const float *g_block, float *state,
                           float *state_start, int32_t *cache_len, int32_t block_len,
                           const natsl_params *p, void *ws, size_t ws_bytes, void *stream) {
    int rc = check_params(p, false);
    if (rc != NATSL_OK) return rc;
    if (!route_block || !g_block || !state || !state_start || !cache_len) return NATSL_ERR_NULL;
    if (block_len <= 0) return NATSL_ERR_SHAPE;
    if (!aligned16(state) || !aligned16(state_start) || !aligned16(ws)) return NATSL_ERR_ALIGN;
    if (!ws || ws_bytes < decode_workspace_bytes(p->B, p->H, p->d)) return NATSL_ERR_WORKSPACE;
    cudaError_t e = launch_decode_block_end(route_block, g_block, state, state_start, cache_len,
                                            block_len, ws, shape_of(p),
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NATSL_OK : NATSL_ERR_CUDA;
}

void natsl_debug_set_wait_limit(uint32_t kcycles, int withhold_scan_flags) {
    g_debug_wait_kcycles.store(kcycles > 0x7fffffffu ? 0x7fffffffu : kcycles, std::memory_order_relaxed);
    g_debug_withhold_flags.store(withhold_scan_flags ? 1 : 0, std::memory_order_relaxed);
}

int natsl_device_status(void *ws, void *stream) {
    if (!ws) return NATSL_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return NATSL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NATSL_ERR_CUDA;
    if (word != 0 && cudaMemsetAsync(ws, 0, sizeof(word), st) != cudaSuccess) return NATSL_ERR_CUDA;
    return word;
}

}  // extern "C"
