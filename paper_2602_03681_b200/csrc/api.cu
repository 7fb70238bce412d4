// C ABI of the library: argument validation, workspace carving and kernel sequencing.
// Nothing here allocates, synchronises (except natsl_device_status) or touches the CPU oracle.
#include <cstring>

#include "natsl_internal.h"

#include <atomic>

using namespace natsl;

namespace natsl {
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
    return NATSL_OK;
}

Shape shape_of(const natsl_params *p) { return Shape{p->B, p->H, p->L, p->d, p->dtype == NATSL_BF16}; }

struct FwdWs {
    int32_t *status, *sm_idx, *prefix, *lin_idx, *n_lin, *sm_len;
    void *k_sm, *v_sm;
    float *W, *U, *P, *o_la;
    size_t bytes;
};

FwdWs carve_fwd(const natsl_params *p, void *ws) {
    Carver c(ws);
    FwdWs f;
    const size_t B = p->B, H = p->H, L = p->L, d = p->d, NC = L / kC;
    const size_t esz = p->dtype == NATSL_BF16 ? 2 : 4;
    f.status = c.take<int32_t>(kStatusBytes / 4);
    f.sm_idx = c.take<int32_t>(B * H * L);
    f.prefix = c.take<int32_t>(B * H * (NC + 1));
    f.lin_idx = c.take<int32_t>(B * H * L);
    f.n_lin = c.take<int32_t>(B * H * NC);
    f.sm_len = c.take<int32_t>(B * H);
    f.k_sm = c.take<char>(B * H * L * d * esz);
    f.v_sm = c.take<char>(B * H * L * d * esz);
    f.W = c.take<float>(B * L * H * d);
    f.U = c.take<float>(B * L * H * d);
    f.P = c.take<float>(B * H * NC * kC * kC);
    f.o_la = c.take<float>(B * L * H * d);
    f.bytes = c.off;
    return f;
}

}  // namespace

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
        default: return "unknown natsl status";
    }
}

int natsl_workspace_size(const natsl_params *p, int op, size_t *bytes) {
    if (!bytes) return NATSL_ERR_NULL;
    int rc = check_params(p, op != NATSL_OP_DECODE);
    if (rc != NATSL_OK) return rc;
    switch (op) {
        case NATSL_OP_FWD: *bytes = carve_fwd(p, nullptr).bytes; return NATSL_OK;
        case NATSL_OP_DECODE: *bytes = kStatusBytes; return NATSL_OK;
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
                                         p->B, p->L, p->H, static_cast<cudaStream_t>(stream));
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
    FwdWs f = carve_fwd(p, ws);
    if (!ws || ws_bytes < f.bytes) return NATSL_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Shape s = shape_of(p);

#define NATSL_TRY(call) do { if ((call) != cudaSuccess) return NATSL_ERR_CUDA; } while (0)
    int stage = 0;
    auto mark = [&]() -> cudaError_t {
        if (p->stage_events && stage < p->n_stage_events)
            return cudaEventRecord(static_cast<cudaEvent_t>(p->stage_events[stage++]), st);
        return cudaSuccess;
    };
    NATSL_TRY(cudaMemsetAsync(f.status, 0, kStatusBytes, st));
    NATSL_TRY(mark());
    int32_t *sm_len = want_cache ? p->sm_len : f.sm_len;
    void *k_sm = want_cache ? p->k_sm : f.k_sm, *v_sm = want_cache ? p->v_sm : f.v_sm;
    const int32_t cap = want_cache ? p->sm_cap : p->L;
    NATSL_TRY(launch_route_compact(route, f.sm_idx, f.prefix, f.lin_idx, f.n_lin, sm_len, p->B, p->L,
                                   p->H, st));
    NATSL_TRY(launch_gather_kv(k, v, f.sm_idx, f.prefix, k_sm, v_sm, cap, f.status, s, st));
    NATSL_TRY(mark());
    float *o_la = p->o_la ? p->o_la : f.o_la;
    NATSL_TRY(launch_gdn_prepare_simt(q, k, v, g, beta, route, p->scale_la, f.W, f.U, f.P, s, st));
    NATSL_TRY(mark());
    NATSL_TRY(launch_gdn_scan_simt(q, k, g, f.W, f.U, f.P, p->scale_la, p->state_in, p->state_out,
                                   nullptr, o_la, s, st));
    NATSL_TRY(mark());
    NATSL_TRY(launch_softmax_combine_simt(q, k_sm, v_sm, cap, f.sm_idx, f.prefix, o_la, p->w,
                                          p->scale_sm, p->eps, out, p->o_nla, p->lse, s, st));
    NATSL_TRY(mark());
#undef NATSL_TRY
    return NATSL_OK;
}

int natsl_hybrid_bwd(const void *, const void *, const void *, const float *, const float *,
                     const uint8_t *, const void *, void *, void *, void *, float *, float *,
                     float *, const natsl_params *, void *, size_t, void *) {
    return NATSL_ERR_UNSUPPORTED;
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
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(state) ||
        !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return NATSL_ERR_ALIGN;
    if (!ws || ws_bytes < kStatusBytes) return NATSL_ERR_WORKSPACE;
    cudaError_t e = launch_decode_step(q, k, v, g, beta, route, p->w, state, k_cache, v_cache,
                                       cache_len, cache_cap, out, p->scale_la, p->scale_sm, p->eps,
                                       static_cast<int32_t *>(ws), shape_of(p),
                                       static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NATSL_OK : NATSL_ERR_CUDA;
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
