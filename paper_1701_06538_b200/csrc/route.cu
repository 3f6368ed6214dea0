// Routing: dispatch of token rows into contiguous per-expert segments (Section 3.1), the
// gate-weighted combine (Eq. 1) and their adjoints. All of it is HBM streaming: rows are moved
// with 16-byte vector accesses, every token row is read once and written k times (dispatch) or
// gathered k times and written once (combine).
#include "moe_internal.cuh"

namespace moe {

// ------------------------------------------------------------------------------------------
// Stable counting sort of the slots p = 0..R-1 by expert id, with no ordering race:
//   1. each chunk of CH consecutive slots builds a histogram              (dispatch_hist)
//   2. per expert, exclusive scan of the chunk histograms -> chunk bases,
//      totals -> counts                                                   (dispatch_scan_chunks)
//   3. exclusive scan of counts -> offsets                                (dispatch_scan_experts)
//   4. one warp per chunk walks its slots in order, 32 at a time; equal experts inside a group
//      of 32 are ranked with match_any, across groups with a shared-memory cursor per expert
//                                                                          (dispatch_rank)
// Integer atomics only (order-independent results); the permutation is unique and bit-exact.
// ------------------------------------------------------------------------------------------
constexpr int CH = 1024;  // slots per chunk

int64_t dispatch_ws_elems(int64_t R, int32_t n) { return cdiv(R, CH) * (int64_t)n + 64; }

__global__ void __launch_bounds__(256) dispatch_hist_kernel(const int32_t *__restrict__ topk_idx, int64_t R,
                                                            int32_t n, int32_t *__restrict__ chunk_hist) {
    extern __shared__ int32_t sh[];
    for (int e = threadIdx.x; e < n; e += blockDim.x) sh[e] = 0;
    __syncthreads();
    const int64_t p0 = (int64_t)blockIdx.x * CH;
    for (int i = threadIdx.x; i < CH; i += blockDim.x) {
        const int64_t p = p0 + i;
        if (p < R) {
            const int32_t e = topk_idx[p];
            if ((uint32_t)e < (uint32_t)n) atomicAdd(&sh[e], 1);
        }
    }
    __syncthreads();
    int32_t *out = chunk_hist + (int64_t)blockIdx.x * n;
    for (int e = threadIdx.x; e < n; e += blockDim.x) out[e] = sh[e];
}

// block = 32 experts x 32 chunk lanes; lane cl owns a contiguous run of chunks
__global__ void __launch_bounds__(1024) dispatch_scan_chunks_kernel(int32_t *__restrict__ chunk_hist,
                                                                    int32_t nchunks, int32_t n,
                                                                    int32_t *__restrict__ counts) {
    __shared__ int32_t part[32][33];
    const int el = threadIdx.x & 31, cl = threadIdx.x >> 5;
    const int32_t e = blockIdx.x * 32 + el;
    const int32_t per = (nchunks + 31) / 32;
    const int32_t c0 = cl * per, c1 = min(c0 + per, nchunks);
    int32_t sum = 0;
    if (e < n)
        for (int32_t c = c0; c < c1; ++c) sum += chunk_hist[(int64_t)c * n + e];
    part[cl][el] = sum;
    __syncthreads();
    if (cl == 0) {
        int32_t run = 0;
        for (int q = 0; q < 32; ++q) { int32_t v = part[q][el]; part[q][el] = run; run += v; }
        if (e < n) counts[e] = run;
    }
    __syncthreads();
    if (e < n) {
        int32_t run = part[cl][el];
        for (int32_t c = c0; c < c1; ++c) {
            const int64_t at = (int64_t)c * n + e;
            const int32_t v = chunk_hist[at];
            chunk_hist[at] = run;
            run += v;
        }
    }
}

__global__ void __launch_bounds__(1024) dispatch_scan_experts_kernel(const int32_t *__restrict__ counts, int32_t n,
                                                                     int32_t *__restrict__ offsets) {
    __shared__ int32_t warp_sum[32];
    __shared__ int32_t carry;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int32_t base = 0; base < n; base += 1024) {
        const int32_t e = base + threadIdx.x;
        const int32_t v = e < n ? counts[e] : 0;
        int32_t inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            int32_t o = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += o;
        }
        if (lane == 31) warp_sum[w] = inc;
        __syncthreads();
        if (w == 0) {
            int32_t s = warp_sum[lane], si = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                int32_t o = __shfl_up_sync(0xffffffffu, si, off);
                if (lane >= off) si += o;
            }
            warp_sum[lane] = si - s;  // exclusive
        }
        __syncthreads();
        const int32_t excl = carry + warp_sum[w] + inc - v;
        if (e < n) offsets[e] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) offsets[n] = carry;
}

__global__ void __launch_bounds__(32) dispatch_rank_kernel(const int32_t *__restrict__ topk_idx, int64_t R,
                                                           int32_t n, const int32_t *__restrict__ chunk_base,
                                                           const int32_t *__restrict__ offsets,
                                                           int32_t *__restrict__ perm,
                                                           int32_t *__restrict__ inv_perm) {
    extern __shared__ int32_t cursor[];  // next sorted row of each expert for this chunk
    const int lane = threadIdx.x;
    const int32_t *base = chunk_base + (int64_t)blockIdx.x * n;
    for (int e = lane; e < n; e += 32) cursor[e] = offsets[e] + base[e];
    __syncwarp();
    const int64_t p0 = (int64_t)blockIdx.x * CH;
    for (int i = 0; i < CH; i += 32) {
        const int64_t p = p0 + i + lane;
        const bool live = p < R;
        int32_t e = live ? topk_idx[p] : -1;
        MOE_BOUNDS_NOTE(!live || (uint32_t)e < (uint32_t)n);
        if ((uint32_t)e >= (uint32_t)n) e = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        const int leader = __ffs(peers) - 1;
        int32_t start = 0;
        if (e >= 0 && lane == leader) {
            start = cursor[e];
            cursor[e] = start + __popc(peers);
        }
        start = __shfl_sync(0xffffffffu, start, leader);
        if (e >= 0) {
            const int32_t r = start + rank;
            MOE_BOUNDS_NOTE((uint32_t)r < (uint32_t)R);
            perm[r] = (int32_t)p;
            inv_perm[p] = r;
        } else if (live) {
            inv_perm[p] = -1;  // expert id outside [0, n): the slot is dropped; the row movers skip negative rows
        }
        __syncwarp();
    }
}

int32_t launch_dispatch_index(const int32_t *topk_idx, int64_t R, int32_t n, int32_t *perm, int32_t *inv_perm,
                              int32_t *counts, int32_t *offsets, int32_t *scratch, cudaStream_t st) {
    const int32_t nchunks = (int32_t)cdiv(R, CH);
    if (nchunks == 0) {
        MOE_CUDA(cudaMemsetAsync(counts, 0, sizeof(int32_t) * n, st));
        MOE_CUDA(cudaMemsetAsync(offsets, 0, sizeof(int32_t) * (n + 1), st));
        return MOE_OK;
    }
    dispatch_hist_kernel<<<nchunks, 256, n * sizeof(int32_t), st>>>(topk_idx, R, n, scratch);
    MOE_LAUNCHED();
    dispatch_scan_chunks_kernel<<<(unsigned)cdiv(n, 32), 1024, 0, st>>>(scratch, nchunks, n, counts);
    MOE_LAUNCHED();
    dispatch_scan_experts_kernel<<<1, 1024, 0, st>>>(counts, n, offsets);
    MOE_LAUNCHED();
    dispatch_rank_kernel<<<nchunks, 32, n * sizeof(int32_t), st>>>(topk_idx, R, n, scratch, offsets, perm, inv_perm);
    MOE_LAUNCHED();
    return MOE_OK;
}

// The same for long inputs (one count per token), in tiles of 4096 counts: the tiles' sums first, then every tile
// scans its own counts behind the sum of the tiles before it. 16-byte accesses where the tile is whole.
constexpr int SCAN_TILE = 4096;
__device__ __forceinline__ int4 scan_tile_load(const int32_t *counts, int32_t n, int32_t i) {
    if (i + 4 <= n) return *reinterpret_cast<const int4 *>(counts + i);
    int4 v = make_int4(0, 0, 0, 0);
    if (i < n) v.x = counts[i];
    if (i + 1 < n) v.y = counts[i + 1];
    if (i + 2 < n) v.z = counts[i + 2];
    return v;
}
// sum over the block of one value per thread, returned to every thread (1024 threads)
__device__ __forceinline__ int32_t block_sum_1024(int32_t v, int32_t *sh /* [32] */) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();  // sh may still be read from an earlier call
    if (lane == 0) sh[w] = v;
    __syncthreads();
    int32_t t = sh[lane];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    return t;
}
__global__ void __launch_bounds__(1024) scan_tile_sums_kernel(const int32_t *__restrict__ counts, int32_t n,
                                                              int32_t *__restrict__ tile_sums) {
    __shared__ int32_t sh[32];
    const int4 v = scan_tile_load(counts, n, blockIdx.x * SCAN_TILE + threadIdx.x * 4);
    const int32_t total = block_sum_1024(v.x + v.y + v.z + v.w, sh);
    if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}
__global__ void __launch_bounds__(1024) scan_tiles_kernel(const int32_t *__restrict__ counts, int32_t n,
                                                          const int32_t *__restrict__ tile_sums,
                                                          int32_t *__restrict__ offsets) {
    __shared__ int32_t sh[32];
    __shared__ int32_t warp_excl[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int32_t before = 0;
    for (int32_t b = threadIdx.x; b < (int32_t)blockIdx.x; b += 1024) before += tile_sums[b];
    before = block_sum_1024(before, sh);
    const int32_t i = blockIdx.x * SCAN_TILE + threadIdx.x * 4;
    const int4 v = scan_tile_load(counts, n, i);
    const int32_t mine = v.x + v.y + v.z + v.w;
    int32_t inc = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        int32_t o = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += o;
    }
    if (lane == 31) warp_excl[w] = inc;
    __syncthreads();
    if (w == 0) {
        int32_t sv = warp_excl[lane], si = sv;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            int32_t o = __shfl_up_sync(0xffffffffu, si, off);
            if (lane >= off) si += o;
        }
        warp_excl[lane] = si - sv;
    }
    __syncthreads();
    const int32_t e0 = before + warp_excl[w] + inc - mine;
    const int4 out = make_int4(e0, e0 + v.x, e0 + v.x + v.y, e0 + v.x + v.y + v.z);
    // offsets has n + 1 entries: entry n is the grand total, written by whoever holds position n
    if (i + 4 <= n + 1 && (reinterpret_cast<uintptr_t>(offsets + i) & 15) == 0) {
        *reinterpret_cast<int4 *>(offsets + i) = out;
    } else {
        if (i <= n) offsets[i] = out.x;
        if (i + 1 <= n) offsets[i + 1] = out.y;
        if (i + 2 <= n) offsets[i + 2] = out.z;
        if (i + 3 <= n) offsets[i + 3] = out.w;
    }
}

// out[0..n] = exclusive prefix sums of counts[0..n-1]. Long inputs need tile_sums: cdiv(n + 1, 4096) ints of scratch.
int32_t launch_exclusive_scan(const int32_t *counts, int32_t n, int32_t *out, cudaStream_t st, int32_t *tile_sums) {
    if (n > 8192 && tile_sums) {
        const unsigned tiles = (unsigned)cdiv(n + 1, SCAN_TILE);  // position n (the total) falls into a tile as well
        scan_tile_sums_kernel<<<tiles, 1024, 0, st>>>(counts, n, tile_sums);
        MOE_LAUNCHED();
        scan_tiles_kernel<<<tiles, 1024, 0, st>>>(counts, n, tile_sums, out);
        MOE_LAUNCHED();
        return MOE_OK;
    }
    dispatch_scan_experts_kernel<<<1, 1024, 0, st>>>(counts, n, out);
    MOE_LAUNCHED();
    return MOE_OK;
}

// tile_prefix[e] = number of bm-row tiles of the segments before e (tile_prefix[n] = total)
__global__ void __launch_bounds__(1024) tile_prefix_kernel(const int32_t *__restrict__ offsets, int32_t n,
                                                           int32_t bm, int32_t *__restrict__ tile_prefix) {
    __shared__ int32_t warp_sum[32];
    __shared__ int32_t carry;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int32_t base = 0; base < n; base += 1024) {
        const int32_t e = base + threadIdx.x;
        const int32_t v = e < n ? (offsets[e + 1] - offsets[e] + bm - 1) / bm : 0;
        int32_t inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            int32_t o = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += o;
        }
        if (lane == 31) warp_sum[w] = inc;
        __syncthreads();
        if (w == 0) {
            int32_t s = warp_sum[lane], si = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                int32_t o = __shfl_up_sync(0xffffffffu, si, off);
                if (lane >= off) si += o;
            }
            warp_sum[lane] = si - s;
        }
        __syncthreads();
        const int32_t excl = carry + warp_sum[w] + inc - v;
        if (e < n) tile_prefix[e] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) tile_prefix[n] = carry;
}

int32_t launch_tile_prefix(const int32_t *offsets, int32_t n, int32_t bm, int32_t *tile_prefix, cudaStream_t st) {
    tile_prefix_kernel<<<1, 1024, 0, st>>>(offsets, n, bm, tile_prefix);
    MOE_LAUNCHED();
    return MOE_OK;
}

// ------------------------------------------------------------------------------------------
// Row movers. VEC = one 16-byte vector (8 bf16 or 4 float). One warp per token.
// ------------------------------------------------------------------------------------------
template <typename XT> struct Vec16 {
    static constexpr int N = 16 / sizeof(XT);
    uint4 raw;
    __device__ __forceinline__ float get(int i) const { return to_f32(reinterpret_cast<const XT *>(&raw)[i]); }
    __device__ __forceinline__ void set(int i, float v) { reinterpret_cast<XT *>(&raw)[i] = from_f32<XT>(v); }
};

// xs[inv_perm[t*k+s]] = x[t] for every slot s: x is read once, written k times
template <typename XT>
__global__ void __launch_bounds__(256) dispatch_rows_kernel(const XT *__restrict__ x, int64_t T, int32_t k,
                                                            int32_t d, const int32_t *__restrict__ inv_perm,
                                                            XT *__restrict__ xs) {
    constexpr int VN = 16 / sizeof(XT);
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nvec = d / VN;
    const int64_t R = T * k;  // a row index outside [0, R) (dropped slot, or a caller's bad inv_perm) is skipped, never followed
    for (int64_t t = warp; t < T; t += nwarps) {
        int32_t rows[MOE_MAX_K];
#pragma unroll
        for (int s = 0; s < MOE_MAX_K; ++s) {
            rows[s] = s < k ? inv_perm[t * k + s] : 0;
            MOE_BOUNDS_NOTE((uint32_t)rows[s] < (uint32_t)R);
        }
        const uint4 *src = reinterpret_cast<const uint4 *>(x + t * d);
        for (int v = lane; v < nvec; v += 32) {
            const uint4 val = src[v];
#pragma unroll
            for (int s = 0; s < MOE_MAX_K; ++s)
                if (s < k && (uint32_t)rows[s] < (uint32_t)R) reinterpret_cast<uint4 *>(xs + (int64_t)rows[s] * d)[v] = val;
        }
    }
}

int32_t launch_dispatch_rows(const void *x, int32_t act, int64_t T, int32_t k, int32_t d, const int32_t *inv_perm,
                             void *xs, cudaStream_t st) {
    if (T == 0) return MOE_OK;
    const unsigned grid = (unsigned)imin(cdiv(T, 8), 148 * 16);
    if (act == MOE_BF16)
        dispatch_rows_kernel<bf16><<<grid, 256, 0, st>>>((const bf16 *)x, T, k, d, inv_perm, (bf16 *)xs);
    else
        dispatch_rows_kernel<float><<<grid, 256, 0, st>>>((const float *)x, T, k, d, inv_perm, (float *)xs);
    MOE_LAUNCHED();
    return MOE_OK;
}

// The three kernels below gather or scatter the k rows of a token. KT is k rounded up to a power of two and VB
// the number of 16-byte vectors a lane handles per batch (KT * VB = 8): all loads of a batch are issued before
// any of them is used, so a lane keeps up to eight 16-byte loads in flight.
#define MOE_DISPATCH_KT(K_, CALL)          \
    do {                                   \
        if ((K_) <= 1) { CALL(1, 8); }     \
        else if ((K_) <= 2) { CALL(2, 4); }\
        else if ((K_) <= 4) { CALL(4, 2); }\
        else { CALL(8, 1); }               \
    } while (0)

// Dropout keep bit of column q of a token row: bit q % 8 of byte q / 8. A 16-byte vector holds VN = 8 (bf16) or 4
// (float) consecutive columns starting at a multiple of VN: its bits are one byte, or one half of a byte.
template <int VN> __device__ __forceinline__ uint32_t keep_bits_of(const uint8_t *row_bits, int v) {
    return VN == 8 ? (uint32_t)row_bits[v] : ((uint32_t)row_bits[v >> 1] >> ((v & 1) * 4)) & 0xFu;
}
// 1 / (1 + e^-y) with the hardware exponential and reciprocal (a few 1e-7 of relative error, far inside the tolerance of
// the float layer; the IEEE division and the full-range expf made the fused kernels arithmetic-bound)
__device__ __forceinline__ float logistic(float y) { return __fdividef(1.0f, 1.0f + __expf(-y)); }

// y[t] = sum_s gates[t,s] * ys[inv_perm[t*k+s]]   (Eq. 1), float sum in slot order.
// LAYER (Appendix C): out[t] = x[t] + keep[t] * sigmoid(y[t]) * keep_scale, y itself is not stored.
template <typename XT, int KT, int VB, bool LAYER>
__global__ void __launch_bounds__(256, LAYER ? 3 : 1) combine_kernel(const XT *__restrict__ ys, const float *__restrict__ gates,
                                                      const int32_t *__restrict__ inv_perm, int64_t T, int32_t k,
                                                      int32_t d, XT *__restrict__ y, const XT *__restrict__ xres,
                                                      const uint8_t *__restrict__ keep, float keep_scale) {
    constexpr int VN = 16 / sizeof(XT);
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nvec = d / VN;
    for (int64_t t = warp; t < T; t += nwarps) {
        const uint4 *rowp[KT];
        float g[KT];
#pragma unroll
        for (int s = 0; s < KT; ++s) {
            int32_t row = s < k ? inv_perm[t * k + s] : 0;
            const bool valid = (uint32_t)row < (uint32_t)(T * k);  // a dropped slot contributes nothing
            MOE_BOUNDS_NOTE(valid || s >= k);
            if (!valid) row = 0;
            rowp[s] = reinterpret_cast<const uint4 *>(ys + (int64_t)row * d);
            g[s] = (s < k && valid) ? gates[t * k + s] : 0.0f;
        }
        for (int v0 = lane; v0 < nvec; v0 += 32 * VB) {
            Vec16<XT> in[KT][VB], xr[VB];
            uint32_t kb[VB];
#pragma unroll
            for (int b = 0; b < VB; ++b) {
#pragma unroll
                for (int s = 0; s < KT; ++s)
                    if (s < k && v0 + 32 * b < nvec) in[s][b].raw = rowp[s][v0 + 32 * b];
                if (LAYER && v0 + 32 * b < nvec) {
                    xr[b].raw = reinterpret_cast<const uint4 *>(xres + t * d)[v0 + 32 * b];
                    kb[b] = keep_bits_of<VN>(keep + t * (d / 8), v0 + 32 * b);
                }
            }
#pragma unroll
            for (int b = 0; b < VB; ++b) {
                if (v0 + 32 * b >= nvec) break;
                float acc[VN];
#pragma unroll
                for (int i = 0; i < VN; ++i) acc[i] = 0.0f;
#pragma unroll
                for (int s = 0; s < KT; ++s)
                    if (s < k) {
#pragma unroll
                        for (int i = 0; i < VN; ++i) acc[i] = fmaf(g[s], in[s][b].get(i), acc[i]);
                    }
                if (LAYER) {
#pragma unroll
                    for (int i = 0; i < VN; ++i)
                        acc[i] = fmaf(((kb[b] >> i) & 1u) ? keep_scale : 0.0f, logistic(acc[i]), xr[b].get(i));  // a select, no branch: 0 * s + x = x
                }
                Vec16<XT> out;
#pragma unroll
                for (int i = 0; i < VN; ++i) out.set(i, acc[i]);
                reinterpret_cast<uint4 *>(y + t * d)[v0 + 32 * b] = out.raw;
            }
        }
    }
}

int32_t launch_combine(const void *ys, int32_t act, const float *gates, const int32_t *inv_perm, int64_t T,
                       int32_t k, int32_t d, void *y, cudaStream_t st, const void *xres, const uint8_t *keep,
                       float keep_scale) {
    if (T == 0) return MOE_OK;
    const unsigned grid = (unsigned)imin(cdiv(T, 8), 148 * 16);
#define MOE_CALL_L(KT, VB, L)                                                                                         \
    if (act == MOE_BF16)                                                                                              \
        combine_kernel<bf16, KT, VB, L><<<grid, 256, 0, st>>>((const bf16 *)ys, gates, inv_perm, T, k, d, (bf16 *)y,  \
                                                              (const bf16 *)xres, keep, keep_scale);                  \
    else                                                                                                              \
        combine_kernel<float, KT, VB, L><<<grid, 256, 0, st>>>((const float *)ys, gates, inv_perm, T, k, d, (float *)y, \
                                                               (const float *)xres, keep, keep_scale)
#define MOE_CALL(KT, VB)                     \
    if (keep) { MOE_CALL_L(KT, VB, true); }  \
    else { MOE_CALL_L(KT, VB, false); }
    MOE_DISPATCH_KT(k, MOE_CALL);
#undef MOE_CALL
#undef MOE_CALL_L
    MOE_LAUNCHED();
    return MOE_OK;
}

// dgates[t,s] = <dy[t], ys[row]>,  dys[row] = gates[t,s] * dy[t], with dy = dY, or (LAYER: adjoint of the sigmoid and
// the dropout of Appendix C) dy = dY * keep * keep_scale * s (1 - s), s = sigmoid(y), y recomputed from the ys rows
// this kernel gathers anyway (same order of operations as the forward, so the same y bit for bit).
template <typename XT, int KT, int VB, bool LAYER>
__global__ void __launch_bounds__(256, LAYER ? 3 : 1) combine_bwd_kernel(const XT *__restrict__ dY, const XT *__restrict__ ys,
                                                          const float *__restrict__ gates,
                                                          const int32_t *__restrict__ inv_perm, int64_t T,
                                                          int32_t k, int32_t d, float *__restrict__ dgates,
                                                          XT *__restrict__ dys, const uint8_t *__restrict__ keep,
                                                          float keep_scale) {
    constexpr int VN = 16 / sizeof(XT);
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nvec = d / VN;
    for (int64_t t = warp; t < T; t += nwarps) {
        int64_t rowo[KT];
        float g[KT], dot[KT];
        bool valid[KT];
#pragma unroll
        for (int s = 0; s < KT; ++s) {
            const int32_t row = s < k ? inv_perm[t * k + s] : -1;
            valid[s] = (uint32_t)row < (uint32_t)(T * k);  // a dropped slot: zero gate gradient, no row written
            MOE_BOUNDS_NOTE(valid[s] || s >= k);
            rowo[s] = (int64_t)(valid[s] ? row : 0) * d;
            g[s] = s < k ? gates[t * k + s] : 0.0f;
            dot[s] = 0.0f;
        }
        for (int v0 = lane; v0 < nvec; v0 += 32 * VB) {
            Vec16<XT> dy[VB], in[KT][VB];
            uint32_t kb[VB];
#pragma unroll
            for (int b = 0; b < VB; ++b) {
                if (v0 + 32 * b < nvec) {
                    dy[b].raw = reinterpret_cast<const uint4 *>(dY + t * d)[v0 + 32 * b];
                    if (LAYER) kb[b] = keep_bits_of<VN>(keep + t * (d / 8), v0 + 32 * b);
#pragma unroll
                    for (int s = 0; s < KT; ++s)
                        if (s < k) in[s][b].raw = reinterpret_cast<const uint4 *>(ys + rowo[s])[v0 + 32 * b];  // row 0 for a dropped slot
                }
            }
#pragma unroll
            for (int b = 0; b < VB; ++b) {
                if (v0 + 32 * b >= nvec) break;
                float dyv[VN];
#pragma unroll
                for (int i = 0; i < VN; ++i) dyv[i] = dy[b].get(i);
                if (LAYER) {
#pragma unroll
                    for (int i = 0; i < VN; ++i) {
                        float yv = 0.0f;
#pragma unroll
                        for (int s = 0; s < KT; ++s)
                            if (s < k) yv = fmaf(valid[s] ? g[s] : 0.0f, in[s][b].get(i), yv);
                        const float sg = logistic(yv);
                        dyv[i] = (((kb[b] >> i) & 1u) ? keep_scale : 0.0f) * (dyv[i] * (sg * (1.0f - sg)));
                    }
                }
#pragma unroll
                for (int s = 0; s < KT; ++s) {
                    if (s < k) {
                        Vec16<XT> out;
#pragma unroll
                        for (int i = 0; i < VN; ++i) {
                            dot[s] = fmaf(dyv[i], in[s][b].get(i), dot[s]);
                            out.set(i, g[s] * dyv[i]);
                        }
                        if (valid[s]) reinterpret_cast<uint4 *>(dys + rowo[s])[v0 + 32 * b] = out.raw;
                    }
                }
            }
        }
#pragma unroll
        for (int s = 0; s < KT; ++s) {
            if (s < k) {
                float v = dot[s];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (lane == 0) dgates[t * k + s] = valid[s] ? v : 0.0f;
            }
        }
    }
}

int32_t launch_combine_bwd(const void *dY, const void *ys, int32_t act, const float *gates,
                           const int32_t *inv_perm, int64_t T, int32_t k, int32_t d, float *dgates, void *dys,
                           cudaStream_t st, const uint8_t *keep, float keep_scale) {
    if (T == 0) return MOE_OK;
    const unsigned grid = (unsigned)imin(cdiv(T, 8), 148 * 16);
#define MOE_CALL_L(KT, VB, L)                                                                                            \
    if (act == MOE_BF16)                                                                                                 \
        combine_bwd_kernel<bf16, KT, VB, L><<<grid, 256, 0, st>>>((const bf16 *)dY, (const bf16 *)ys, gates, inv_perm, T, \
                                                                   k, d, dgates, (bf16 *)dys, keep, keep_scale);          \
    else                                                                                                                 \
        combine_bwd_kernel<float, KT, VB, L><<<grid, 256, 0, st>>>((const float *)dY, (const float *)ys, gates, inv_perm, \
                                                                    T, k, d, dgates, (float *)dys, keep, keep_scale)
#define MOE_CALL(KT, VB)                     \
    if (keep) { MOE_CALL_L(KT, VB, true); }  \
    else { MOE_CALL_L(KT, VB, false); }
    MOE_DISPATCH_KT(k, MOE_CALL);
#undef MOE_CALL
#undef MOE_CALL_L
    MOE_LAUNCHED();
    return MOE_OK;
}

// out[t] = sum_s dxs[inv_perm[t*k+s]] (+ add[t]) (+ add_act[t], a second addend in the act type: the gradient that
// reaches the layer input through the residual connection); float output, or rounded to the act type
template <typename XT, int KT, int VB>
__global__ void __launch_bounds__(256) dispatch_bwd_kernel(const XT *__restrict__ dxs,
                                                           const int32_t *__restrict__ inv_perm, int64_t T,
                                                           int32_t k, int32_t d, const float *add,
                                                           float *out_f32, XT *__restrict__ out_act,
                                                           const XT *__restrict__ add_act) {
    constexpr int VN = 16 / sizeof(XT);
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nvec = d / VN;
    for (int64_t t = warp; t < T; t += nwarps) {
        const uint4 *rowp[KT];
        bool valid[KT];
#pragma unroll
        for (int s = 0; s < KT; ++s) {
            const int32_t row = s < k ? inv_perm[t * k + s] : -1;
            valid[s] = (uint32_t)row < (uint32_t)(T * k);  // a dropped slot contributes nothing
            MOE_BOUNDS_NOTE(valid[s] || s >= k);
            rowp[s] = reinterpret_cast<const uint4 *>(dxs + (int64_t)(valid[s] ? row : 0) * d);
        }
        for (int v0 = lane; v0 < nvec; v0 += 32 * VB) {
            Vec16<XT> in[KT][VB], res[VB];
            float4 addv[VB][VN / 4];
#pragma unroll
            for (int b = 0; b < VB; ++b) {
                if (v0 + 32 * b < nvec) {
#pragma unroll
                    for (int s = 0; s < KT; ++s)
                        if (s < k) in[s][b].raw = valid[s] ? rowp[s][v0 + 32 * b] : make_uint4(0, 0, 0, 0);
                    if (add_act) res[b].raw = reinterpret_cast<const uint4 *>(add_act + t * d)[v0 + 32 * b];
                    if (add) {
#pragma unroll
                        for (int q = 0; q < VN / 4; ++q)
                            addv[b][q] = reinterpret_cast<const float4 *>(add + t * d + (int64_t)(v0 + 32 * b) * VN)[q];
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < VB; ++b) {
                if (v0 + 32 * b >= nvec) break;
                float acc[VN];
#pragma unroll
                for (int i = 0; i < VN; ++i) acc[i] = 0.0f;
#pragma unroll
                for (int s = 0; s < KT; ++s)
                    if (s < k) {
#pragma unroll
                        for (int i = 0; i < VN; ++i) acc[i] += in[s][b].get(i);
                    }
                if (add) {
#pragma unroll
                    for (int q = 0; q < VN / 4; ++q) {
                        acc[4 * q] += addv[b][q].x; acc[4 * q + 1] += addv[b][q].y;
                        acc[4 * q + 2] += addv[b][q].z; acc[4 * q + 3] += addv[b][q].w;
                    }
                }
                if (add_act) {
#pragma unroll
                    for (int i = 0; i < VN; ++i) acc[i] += res[b].get(i);
                }
                const int64_t at = t * d + (int64_t)(v0 + 32 * b) * VN;
                if (out_act) {
                    Vec16<XT> out;
#pragma unroll
                    for (int i = 0; i < VN; ++i) out.set(i, acc[i]);
                    *reinterpret_cast<uint4 *>(out_act + at) = out.raw;
                } else {
#pragma unroll
                    for (int q = 0; q < VN / 4; ++q)
                        reinterpret_cast<float4 *>(out_f32 + at)[q] =
                            make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
                }
            }
        }
    }
}

int32_t launch_dispatch_bwd(const void *dxs, int32_t act, const int32_t *inv_perm, int64_t T, int32_t k,
                            int32_t d, const float *add_f32, float *out_f32, void *out_act, cudaStream_t st,
                            const void *add_act) {
    if (T == 0) return MOE_OK;
    const unsigned grid = (unsigned)imin(cdiv(T, 8), 148 * 16);
#define MOE_CALL(KT, VB)                                                                                              \
    if (act == MOE_BF16)                                                                                              \
        dispatch_bwd_kernel<bf16, KT, VB><<<grid, 256, 0, st>>>((const bf16 *)dxs, inv_perm, T, k, d, add_f32, out_f32, \
                                                                 (bf16 *)out_act, (const bf16 *)add_act);              \
    else                                                                                                              \
        dispatch_bwd_kernel<float, KT, VB><<<grid, 256, 0, st>>>((const float *)dxs, inv_perm, T, k, d, add_f32,       \
                                                                  out_f32, (float *)out_act, (const float *)add_act)
    MOE_DISPATCH_KT(k, MOE_CALL);
#undef MOE_CALL
    MOE_LAUNCHED();
    return MOE_OK;
}

MOE_BOUNDS_READER(bounds_violations_route)

}  // namespace moe
