// Route compaction: the per-token routing mask becomes per-chunk index lists (Section 4.1,
// column masks M^nla / M^la), with warp ballots and a block prefix sum; and a gather of the
// retained tokens' K/V rows into the compacted cache layout [B,H,cap,d].  Two options: the
// prefix sums may start behind the entries a cache already holds (prefill in pieces), and the
// route may be checked to be one decision per chunk (block-level routing).
#include "common.cuh"
#include "natsl_internal.h"

namespace natsl {

namespace {

constexpr int kCompactThreads = 1024;
constexpr int kCompactTile = 1024;  // chunks scanned per pass (one per thread)

// One CTA per (batch, head).  A chunk of 64 tokens is one 64-bit ballot word.  32 warps, and the
// route bytes of two chunks per warp in flight at a time: the kernel is a chain of dependent
// global-memory round trips, so what counts is how few of them each warp makes.
__global__ void __launch_bounds__(kCompactThreads)
route_compact_kernel(const uint8_t *__restrict__ route, int32_t *__restrict__ sm_idx,
                     int32_t *__restrict__ sm_chunk_prefix, int32_t *__restrict__ lin_idx,
                     int32_t *__restrict__ n_lin, int32_t *sm_len, const int32_t *base_in,
                     int32_t *__restrict__ block_status, int cap, int L, int H) {
    __shared__ unsigned long long bits[kCompactTile];
    __shared__ int excl[kCompactTile];
    __shared__ int warp_tot[kCompactThreads / 32];
    __shared__ int tile_total;

    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kWarps = kCompactThreads / 32;
    const uint8_t *rt = route + (size_t)b * L * H + h;
    // Appending to a cache that already holds base0 retained tokens of earlier calls: the prefix
    // sums start there, the positions listed in sm_idx are still this call's own (index - base0).
    // (base_in may be the same array as sm_len: it is read here, written at the very end.)
    const int base0 = base_in ? base_in[bh] : 0;
    int base = base0;

    for (int tile0 = 0; tile0 < NC; tile0 += kCompactTile) {
        const int nt = min(kCompactTile, NC - tile0);
        for (int c = warp; c < nt; c += 2 * kWarps) {
            const int c2 = c + kWarps;
            const size_t l0 = (size_t)(tile0 + c) * kC, l2 = (size_t)(tile0 + c2) * kC;
            const bool two = c2 < nt;                      // warp-uniform
            const uint8_t a0 = rt[(l0 + lane) * H], a1 = rt[(l0 + 32 + lane) * H];
            const uint8_t b0 = two ? rt[(l2 + lane) * H] : (uint8_t)0, b1 = two ? rt[(l2 + 32 + lane) * H] : (uint8_t)0;
            const unsigned lo = __ballot_sync(0xffffffffu, a0 != 0), hi = __ballot_sync(0xffffffffu, a1 != 0);
            const unsigned lo2 = __ballot_sync(0xffffffffu, b0 != 0), hi2 = __ballot_sync(0xffffffffu, b1 != 0);
            if (lane == 0) {
                bits[c] = (unsigned long long)lo | ((unsigned long long)hi << 32);
                excl[c] = __popc(lo) + __popc(hi);
                if (two) {
                    bits[c2] = (unsigned long long)lo2 | ((unsigned long long)hi2 << 32);
                    excl[c2] = __popc(lo2) + __popc(hi2);
                }
            }
        }
        for (int c = nt + threadIdx.x; c < kCompactTile; c += kCompactThreads) excl[c] = 0;
        __syncthreads();
        // exclusive scan of the per-chunk counts: one entry per thread, warp scan, scan of the warp totals
        {
            const int mine = excl[threadIdx.x];
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += y;
            }
            if (lane == 31) warp_tot[warp] = incl;
            __syncthreads();
            if (warp == 0) {
                const int t = warp_tot[lane];
                int ti = t;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, ti, o);
                    if (lane >= o) ti += y;
                }
                warp_tot[lane] = ti - t;                   // exclusive offsets of the warps
                if (lane == 31) tile_total = ti;
            }
            __syncthreads();
            excl[threadIdx.x] = warp_tot[warp] + incl - mine;
        }
        __syncthreads();
        for (int c = warp; c < nt; c += kWarps) {
            const int cc = tile0 + c;
            const unsigned long long wbits = bits[c];
            const unsigned lo = (unsigned)wbits, hi = (unsigned)(wbits >> 32);
            const int pre = base + excl[c];
            // block-level routing: one decision per chunk, so a word is all zeros or all ones
            if (block_status && lane == 0 && wbits != 0ull && wbits != ~0ull)
                atomicMin(block_status, (int)NATSL_ERR_ROUTE);
            const unsigned lt = (1u << lane) - 1u;
            const int nlo = __popc(lo), nsm = nlo + __popc(hi);
            int32_t *sm = sm_idx + (size_t)bh * L + (pre - base0);
            int32_t *li = lin_idx + ((size_t)bh * NC + cc) * kC;
            if (lane == 0) {
                sm_chunk_prefix[(size_t)bh * (NC + 1) + cc] = pre;
                n_lin[(size_t)bh * NC + cc] = kC - nsm;
            }
            const int r_lo = __popc(lo & lt), r_hi = __popc(hi & lt);
            if ((lo >> lane) & 1u) sm[r_lo] = cc * kC + lane;
            else li[lane - r_lo] = lane;
            if ((hi >> lane) & 1u) sm[nlo + r_hi] = cc * kC + 32 + lane;
            else li[(32 - nlo) + lane - r_hi] = 32 + lane;
            const int nl = kC - nsm;
            if (lane >= nl) li[lane] = kC;
            if (lane + 32 >= nl) li[lane + 32] = kC;
        }
        __syncthreads();
        base += tile_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        sm_chunk_prefix[(size_t)bh * (NC + 1) + NC] = base;
        // The stored length never exceeds the rows the cache has (the gather stops there and
        // reports the overflow), so a later decode step cannot be led past the head's rows.
        if (sm_len) sm_len[bh] = cap > 0 ? min(base, cap) : base;
    }
}

// Copy the retained tokens' K and V rows into [B,H,cap,d].  grid = (row blocks, B*H).
template <typename T, int D>
__global__ void __launch_bounds__(256)
gather_kv_kernel(const T *__restrict__ k, const T *__restrict__ v, const int32_t *__restrict__ sm_idx,
                 const int32_t *__restrict__ sm_chunk_prefix, T *__restrict__ k_sm,
                 T *__restrict__ v_sm, int cap, int32_t *status, int L, int H) {
    constexpr int kVecPerRow = D * (int)sizeof(T) / 16;  // 16-byte pieces per row
    constexpr int kRows = 256 / kVecPerRow;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int n_sm = sm_chunk_prefix[(size_t)bh * (NC + 1) + NC];
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_sm > cap) atomicMin(status, NATSL_ERR_CACHE_FULL);
    const int n = min(n_sm, cap);
    const int row = blockIdx.x * kRows + threadIdx.x / kVecPerRow;
    const int piece = threadIdx.x % kVecPerRow;
    if (row >= n) return;
    const int tok = sm_idx[(size_t)bh * L + row];
    const size_t src = (((size_t)b * L + tok) * H + h) * D;
    const size_t dst = ((size_t)bh * cap + row) * D;
    reinterpret_cast<uint4 *>(k_sm + dst)[piece] = reinterpret_cast<const uint4 *>(k + src)[piece];
    reinterpret_cast<uint4 *>(v_sm + dst)[piece] = reinterpret_cast<const uint4 *>(v + src)[piece];
}

}  // namespace

cudaError_t launch_route_compact(const uint8_t *route, int32_t *sm_idx, int32_t *sm_chunk_prefix,
                                 int32_t *lin_idx, int32_t *n_lin, int32_t *sm_len,
                                 const int32_t *base_in, int32_t *block_status, int cap, int B, int L,
                                 int H, cudaStream_t st) {
    route_compact_kernel<<<B * H, kCompactThreads, 0, st>>>(route, sm_idx, sm_chunk_prefix, lin_idx, n_lin,
                                                            sm_len, base_in, block_status, cap, L, H);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t gather_impl(const void *k, const void *v, const int32_t *sm_idx,
                               const int32_t *pre, void *k_sm, void *v_sm, int cap,
                               int32_t *status, Shape s, cudaStream_t st) {
    constexpr int kRows = 256 / (D * (int)sizeof(T) / 16);
    const int max_rows = s.L < cap ? s.L : cap;
    dim3 grid((max_rows + kRows - 1) / kRows, s.B * s.H);
    gather_kv_kernel<T, D><<<grid, 256, 0, st>>>((const T *)k, (const T *)v, sm_idx, pre, (T *)k_sm,
                                                 (T *)v_sm, cap, status, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gather_kv(const void *k, const void *v, const int32_t *sm_idx,
                             const int32_t *sm_chunk_prefix, void *k_sm, void *v_sm, int32_t cap,
                             int32_t *status, Shape s, cudaStream_t st) {
    if (s.bf16) {
        if (s.d == 128) return gather_impl<__nv_bfloat16, 128>(k, v, sm_idx, sm_chunk_prefix, k_sm, v_sm, cap, status, s, st);
        return gather_impl<__nv_bfloat16, 64>(k, v, sm_idx, sm_chunk_prefix, k_sm, v_sm, cap, status, s, st);
    }
    if (s.d == 128) return gather_impl<float, 128>(k, v, sm_idx, sm_chunk_prefix, k_sm, v_sm, cap, status, s, st);
    return gather_impl<float, 64>(k, v, sm_idx, sm_chunk_prefix, k_sm, v_sm, cap, status, s, st);
}

}  // namespace natsl
