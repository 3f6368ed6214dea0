// Strictly balanced gating (Appendix F, Eq. 15-20): dense softmax gate, batchwise mask (the m = k T / n largest values
// of every expert's column over the batch, so that every expert receives exactly m examples), gates renormalised over
// the kept experts, threshold mask and L_batchwise. An example is kept by a variable number of experts, so the routing
// tables are by sorted row (expert-major, m rows per expert, token order inside an expert) plus a per-token list
// (CSR: tok_ptr, tok_rows) for the combine and its adjoint. Integer results (mask, tables) are unique: ties go to the
// lower token. Sums are taken in fixed orders; integer atomics only.
#include <math_constants.h>

#include "moe_internal.cuh"

namespace moe {

namespace {

// p = softmax(c) per row: exponentials and their sum in double (largest logit subtracted), one rounding to float.
__global__ void __launch_bounds__(256) bal_softmax_kernel(const float *__restrict__ c, int64_t T, int32_t n,
                                                          float *__restrict__ p) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const float *row = c + t * n;
    float mx = -CUDART_INF_F;
    for (int32_t j = lane; j < n; j += 32) mx = fmaxf(mx, row[j]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    double s = 0.0;
    for (int32_t j = lane; j < n; j += 32) s += exp((double)row[j] - (double)mx);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    for (int32_t j = lane; j < n; j += 32) p[t * n + j] = (float)(exp((double)row[j] - (double)mx) / s);
}

// out [cols, rows] = in [rows, cols]^T, 32 x 32 tiles
__global__ void __launch_bounds__(256) bal_transpose_kernel(const float *__restrict__ in, int64_t rows, int32_t cols,
                                                            float *__restrict__ out) {
    __shared__ float tile[32][33];
    const int64_t r0 = (int64_t)blockIdx.x * 32;
    const int32_t c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8)
        if (r0 + i < rows && c0 + tx < cols) tile[i][tx] = in[(r0 + i) * cols + c0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8)
        if (c0 + i < cols && r0 + tx < rows) out[(int64_t)(c0 + i) * rows + r0 + tx] = tile[tx][i];
}

// Batchwise mask of one expert (block = column i of p, given transposed: col [T]): the m largest values, equal values to
// the lower token. Radix select of the m-th largest key (the bit patterns of non-negative floats order like the
// values), then an order-preserving compaction: tok_of_row[i * m + q] = q-th kept token, and the expert's bit is set
// in the token's mask words.
__global__ void __launch_bounds__(1024) bal_select_kernel(const float *__restrict__ pT, int64_t T, int32_t n, int32_t m,
                                                          int32_t words, int32_t *__restrict__ tok_of_row,
                                                          uint32_t *__restrict__ mask_bits) {
    __shared__ int32_t hist[256];
    __shared__ int32_t warp_gt[32], warp_eq[32];
    __shared__ uint32_t s_prefix;
    __shared__ int32_t s_need, s_base_sel, s_base_eq;
    const int32_t i = blockIdx.x;
    const uint32_t *col = reinterpret_cast<const uint32_t *>(pT + (int64_t)i * T);
    const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
    if (tid == 0) { s_prefix = 0u; s_need = m; }
    uint32_t known = 0u;  // mask of the key bits fixed so far
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int64_t t = tid; t < T; t += 1024) {
            const uint32_t key = col[t];
            if ((key & known) == prefix) atomicAdd(&hist[(key >> shift) & 0xFFu], 1);
        }
        __syncthreads();
        if (tid == 0) {  // from the largest digit down: the digit that holds the need-th largest key
            int32_t need = s_need;
            int d = 255;
            for (; d > 0; --d) {
                if (hist[d] >= need) break;
                need -= hist[d];
            }
            s_need = need;
            s_prefix = prefix | ((uint32_t)d << shift);
        }
        known |= 0xFFu << shift;
        __syncthreads();
    }
    const uint32_t kth = s_prefix;    // the m-th largest key
    const int32_t take_eq = s_need;   // how many of the keys equal to it are kept (the first ones in token order)
    if (tid == 0) { s_base_sel = 0; s_base_eq = 0; }
    __syncthreads();
    for (int64_t t0 = 0; t0 < T; t0 += 1024) {
        const int64_t t = t0 + tid;
        const uint32_t key = t < T ? col[t] : 0u;
        const bool gt = t < T && key > kth, eq = t < T && key == kth;
        const uint32_t b_eq = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) warp_eq[wp] = __popc(b_eq);
        __syncthreads();
        int32_t eq_before = s_base_eq;
        for (int w = 0; w < wp; ++w) eq_before += warp_eq[w];
        const bool keep = gt || (eq && eq_before + __popc(b_eq & ((1u << lane) - 1u)) < take_eq);
        const uint32_t b_keep = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_gt[wp] = __popc(b_keep);
        __syncthreads();
        if (keep) {
            int32_t pos = s_base_sel;
            for (int w = 0; w < wp; ++w) pos += warp_gt[w];
            pos += __popc(b_keep & ((1u << lane) - 1u));
            if (pos < m) {  // always true: exactly m keys are kept
                tok_of_row[(int64_t)i * m + pos] = (int32_t)t;
                atomicOr(&mask_bits[t * words + (i >> 5)], 1u << (i & 31));
            }
        }
        __syncthreads();
        if (tid == 0) {
            int32_t a = 0, b = 0;
            for (int w = 0; w < 32; ++w) { a += warp_gt[w]; b += warp_eq[w]; }
            s_base_sel += a;
            s_base_eq += b;
        }
        __syncthreads();
    }
}

// Per token (one warp): den = sum of p over the kept experts, cnt = how many keep it, the token's part of L_batchwise
// (Eq. 20), and the per-expert counts of the threshold mask. Block partials of the loss go to loss_part.
__global__ void __launch_bounds__(256) bal_token_kernel(const float *__restrict__ p, const uint32_t *__restrict__ mask_bits,
                                                        const float *__restrict__ thr, int64_t T, int32_t n, int32_t words,
                                                        float *__restrict__ den, int32_t *__restrict__ cnt,
                                                        int32_t *__restrict__ thr_counts, double *__restrict__ loss_part) {
    extern __shared__ int32_t s_cnt[];  // [n] threshold-mask counts of this block
    __shared__ double s_loss[8];
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    for (int32_t j = threadIdx.x; j < n; j += blockDim.x) s_cnt[j] = 0;
    __syncthreads();
    const int64_t t = (int64_t)blockIdx.x * 8 + wp;
    double d = 0.0, l = 0.0;
    int32_t c = 0;
    if (t < T) {
        for (int32_t j = lane; j < n; j += 32) {
            const float pj = p[t * n + j];
            const bool mb = (mask_bits[t * words + (j >> 5)] >> (j & 31)) & 1u;
            const bool mt = pj > thr[j];
            if (mb) { d += (double)pj; ++c; }
            if (mt) atomicAdd(&s_cnt[j], 1);
            if (mt != mb) l += (mt ? 1.0 : -1.0) * ((double)pj - (double)thr[j]);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        d += __shfl_xor_sync(0xffffffffu, d, off);
        l += __shfl_xor_sync(0xffffffffu, l, off);
        c += __shfl_xor_sync(0xffffffffu, c, off);
    }
    if (lane == 0) {
        if (t < T) { den[t] = (float)d; cnt[t] = c; }
        s_loss[wp] = l;
    }
    __syncthreads();
    for (int32_t j = threadIdx.x; j < n; j += blockDim.x)
        if (s_cnt[j]) atomicAdd(&thr_counts[j], s_cnt[j]);
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += s_loss[w];
        loss_part[blockIdx.x] = s;
    }
}

__global__ void __launch_bounds__(256) bal_loss_final_kernel(const double *__restrict__ part, int64_t nparts,
                                                             float *__restrict__ loss) {
    __shared__ double sh[256];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < nparts; i += 256) s += part[i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[0] = (float)sh[0];
}

// rank of expert e among the experts that keep token t
__device__ __forceinline__ int32_t rank_in_token(const uint32_t *bits, int32_t e) {
    int32_t r = 0;
    for (int32_t w = 0; w < (e >> 5); ++w) r += __popc(bits[w]);
    return r + __popc(bits[e >> 5] & ((1u << (e & 31)) - 1u));
}

// Per sorted row: its place in its token's list (ascending expert); offsets[e] = e * m.
__global__ void __launch_bounds__(256) bal_fill_kernel(const int32_t *__restrict__ tok_of_row,
                                                       const uint32_t *__restrict__ mask_bits,
                                                       const int32_t *__restrict__ tok_ptr, int64_t R, int32_t n, int32_t m,
                                                       int32_t words, int32_t *__restrict__ tok_rows,
                                                       int32_t *__restrict__ offsets) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r <= n) offsets[r] = (int32_t)(r * m);
    if (r >= R) return;
    const int32_t t = tok_of_row[r], e = (int32_t)(r / m);
    tok_rows[tok_ptr[t] + rank_in_token(mask_bits + (int64_t)t * words, e)] = (int32_t)r;
}

template <typename XT> struct V16 {
    static constexpr int N = 16 / sizeof(XT);
    uint4 raw;
    __device__ __forceinline__ float get(int i) const { return to_f32(reinterpret_cast<const XT *>(&raw)[i]); }
    __device__ __forceinline__ void set(int i, float v) { reinterpret_cast<XT *>(&raw)[i] = from_f32<XT>(v); }
};

// xs[r] = x[tok_of_row[r]], one warp per row
template <typename XT>
__global__ void __launch_bounds__(256) bal_gather_kernel(const XT *__restrict__ x, const int32_t *__restrict__ tok_of_row,
                                                         int64_t R, int64_t T, int32_t d, XT *__restrict__ xs) {
    const int lane = threadIdx.x & 31;
    const int64_t r = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (r >= R) return;
    const int32_t t = tok_of_row[r];
    if ((uint32_t)t >= (uint32_t)T) return;
    const int nvec = d / V16<XT>::N;
    const uint4 *src = reinterpret_cast<const uint4 *>(x + (int64_t)t * d);
    uint4 *dst = reinterpret_cast<uint4 *>(xs + r * d);
    for (int v = lane; v < nvec; v += 32) dst[v] = src[v];
}

// y[t] = sum over the rows of token t (ascending expert) of p[t, e] / den[t] * ys[row]   (Eq. 1 with the gates of Eq. 16)
template <typename XT>
__global__ void __launch_bounds__(256) bal_combine_kernel(const XT *__restrict__ ys, const float *__restrict__ p,
                                                          const float *__restrict__ den, const int32_t *__restrict__ tok_ptr,
                                                          const int32_t *__restrict__ tok_rows, int64_t T, int64_t R,
                                                          int32_t n, int32_t m, int32_t d, XT *__restrict__ y) {
    constexpr int VN = V16<XT>::N;
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const int32_t j0 = tok_ptr[t], j1 = tok_ptr[t + 1];
    const float dn = den[t];
    const int nvec = d / VN;
    for (int v = lane; v < nvec; v += 32) {
        float acc[VN];
#pragma unroll
        for (int i = 0; i < VN; ++i) acc[i] = 0.0f;
        for (int32_t j = j0; j < j1; ++j) {
            const int32_t r = tok_rows[j];
            if ((uint32_t)r >= (uint32_t)R) continue;
            const float g = p[t * n + r / m] / dn;
            V16<XT> in;
            in.raw = reinterpret_cast<const uint4 *>(ys + (int64_t)r * d)[v];
#pragma unroll
            for (int i = 0; i < VN; ++i) acc[i] = fmaf(g, in.get(i), acc[i]);
        }
        V16<XT> out;
#pragma unroll
        for (int i = 0; i < VN; ++i) out.set(i, acc[i]);
        reinterpret_cast<uint4 *>(y + t * d)[v] = out.raw;
    }
}

// per row: dG_row[r] = <dY[t], ys[r]>, dys[r] = g * dY[t]
template <typename XT>
__global__ void __launch_bounds__(256) bal_combine_bwd_kernel(const XT *__restrict__ dY, const XT *__restrict__ ys,
                                                              const float *__restrict__ p, const float *__restrict__ den,
                                                              const int32_t *__restrict__ tok_of_row, int64_t R, int64_t T,
                                                              int32_t n, int32_t m, int32_t d, float *__restrict__ dG_row,
                                                              XT *__restrict__ dys) {
    constexpr int VN = V16<XT>::N;
    const int lane = threadIdx.x & 31;
    const int64_t r = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (r >= R) return;
    const int32_t t = tok_of_row[r];
    if ((uint32_t)t >= (uint32_t)T) return;
    const float g = p[(int64_t)t * n + r / m] / den[t];
    const int nvec = d / VN;
    float dot = 0.0f;
    for (int v = lane; v < nvec; v += 32) {
        V16<XT> a, b, o;
        a.raw = reinterpret_cast<const uint4 *>(dY + (int64_t)t * d)[v];
        b.raw = reinterpret_cast<const uint4 *>(ys + r * d)[v];
#pragma unroll
        for (int i = 0; i < VN; ++i) {
            dot = fmaf(a.get(i), b.get(i), dot);
            o.set(i, g * a.get(i));
        }
        reinterpret_cast<uint4 *>(dys + r * d)[v] = o.raw;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    if (lane == 0) dG_row[r] = dot;
}

// Logit gradients of one token (one warp): through Eq. 16 (mask constant), Eq. 20 scaled by w, and the softmax.
__global__ void __launch_bounds__(256) bal_gate_bwd_kernel(const float *__restrict__ p, const uint32_t *__restrict__ mask_bits,
                                                           const float *__restrict__ den, const float *__restrict__ thr,
                                                           const int32_t *__restrict__ tok_ptr,
                                                           const int32_t *__restrict__ tok_rows,
                                                           const float *__restrict__ dG_row, float w, int64_t T, int32_t n,
                                                           int32_t m, int32_t words, float *__restrict__ dc,
                                                           bf16 *__restrict__ dsplit) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const int32_t j0 = tok_ptr[t], j1 = tok_ptr[t + 1];
    const double dn = (double)den[t];
    double inner = 0.0;  // sum over the kept experts of G * dG
    for (int32_t j = j0 + lane; j < j1; j += 32) {
        const int32_t r = tok_rows[j];
        inner += (double)p[t * n + r / m] / dn * (double)dG_row[r];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) inner += __shfl_xor_sync(0xffffffffu, inner, off);
    const uint32_t *bits = mask_bits + t * words;
    double s2 = 0.0;
    for (int32_t j = lane; j < n; j += 32) {
        const double pj = (double)p[t * n + j];
        const bool mb = (bits[j >> 5] >> (j & 31)) & 1u;
        const bool mt = (float)pj > thr[j];
        double dp = (double)w * ((mt ? 1.0 : 0.0) - (mb ? 1.0 : 0.0));
        if (mb) dp += ((double)dG_row[tok_rows[j0 + rank_in_token(bits, j)]] - inner) / dn;
        s2 += dp * pj;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, off);
    for (int32_t j = lane; j < n; j += 32) {
        const double pj = (double)p[t * n + j];
        const bool mb = (bits[j >> 5] >> (j & 31)) & 1u;
        const bool mt = (float)pj > thr[j];
        double dp = (double)w * ((mt ? 1.0 : 0.0) - (mb ? 1.0 : 0.0));
        if (mb) dp += ((double)dG_row[tok_rows[j0 + rank_in_token(bits, j)]] - inner) / dn;
        const float v = (float)(pj * (dp - s2));
        if (dsplit) {  // three bf16 terms carry the 24 mantissa bits: [T, 3n] = (hi | mid | lo)
            const bf16 hi = __float2bfloat16_rn(v);
            const float r1 = v - __bfloat162float(hi);
            const bf16 mid = __float2bfloat16_rn(r1);
            bf16 *row = dsplit + t * 3 * n;
            row[j] = hi; row[n + j] = mid; row[2 * n + j] = __float2bfloat16_rn(r1 - __bfloat162float(mid));
        } else {
            dc[t * n + j] = v;
        }
    }
}

__global__ void bal_dthr_kernel(const int32_t *__restrict__ thr_counts, int32_t n, int32_t m, float w,
                                float *__restrict__ dthr) {
    const int32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < n) dthr[j] = -w * (float)(thr_counts[j] - m);
}

// dX[t] = sum over the rows of token t of dxs[row] + dX_gate[t], rounded to the act type
template <typename XT>
__global__ void __launch_bounds__(256) bal_dispatch_bwd_kernel(const XT *__restrict__ dxs, const int32_t *__restrict__ tok_ptr,
                                                               const int32_t *__restrict__ tok_rows,
                                                               const float *__restrict__ dX_gate, int64_t T, int64_t R,
                                                               int32_t d, XT *__restrict__ dX) {
    constexpr int VN = V16<XT>::N;
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const int32_t j0 = tok_ptr[t], j1 = tok_ptr[t + 1];
    const int nvec = d / VN;
    for (int v = lane; v < nvec; v += 32) {
        float acc[VN];
#pragma unroll
        for (int i = 0; i < VN; ++i) acc[i] = 0.0f;
        for (int32_t j = j0; j < j1; ++j) {
            const int32_t r = tok_rows[j];
            if ((uint32_t)r >= (uint32_t)R) continue;
            V16<XT> in;
            in.raw = reinterpret_cast<const uint4 *>(dxs + (int64_t)r * d)[v];
#pragma unroll
            for (int i = 0; i < VN; ++i) acc[i] += in.get(i);
        }
        V16<XT> out;
#pragma unroll
        for (int i = 0; i < VN; ++i) out.set(i, acc[i] + dX_gate[t * d + v * VN + i]);
        reinterpret_cast<uint4 *>(dX + t * d)[v] = out.raw;
    }
}

}  // namespace

int64_t balanced_ws_bytes(int64_t T, int32_t n) {
    // p^T, per-token counts, loss partials, tile sums of the scan over the tokens
    const int64_t a = (T * n * 4 + 255) & ~255ll, c = (T * 4 + 255) & ~255ll, e = (cdiv(T, 8) * 8 + 255) & ~255ll;
    const int64_t f = (cdiv(T + 1, 4096) * 4 + 255) & ~255ll;
    return a + c + e + f + 256;
}

int32_t launch_balanced_gate(const void *x, int32_t act, int64_t T, int32_t d, int32_t n, int32_t k, const float *Wg,
                             const float *thr, float *logits, float *probs, uint32_t *mask_bits, int32_t *tok_of_row,
                             int32_t *offsets, float *den, int32_t *tok_ptr, int32_t *tok_rows, float *loss,
                             int32_t *thr_counts, void *ws, cudaStream_t st) {
    const int64_t R = T * k;
    const int32_t m = (int32_t)(R / n), words = (n + 31) / 32;
    Carver cv(ws);
    float *pT = cv.take<float>(T * n);
    int32_t *cnt = cv.take<int32_t>(T);
    double *loss_part = cv.take<double>(cdiv(T, 8));
    int32_t *tile_sums = cv.take<int32_t>(cdiv(T + 1, 4096));
    MOE_CUDA(cudaMemsetAsync(mask_bits, 0, sizeof(uint32_t) * T * words, st));
    MOE_CUDA(cudaMemsetAsync(thr_counts, 0, sizeof(int32_t) * n, st));
    if (T == 0) {
        MOE_CUDA(cudaMemsetAsync(offsets, 0, sizeof(int32_t) * (n + 1), st));
        MOE_CUDA(cudaMemsetAsync(tok_ptr, 0, sizeof(int32_t), st));
        MOE_CUDA(cudaMemsetAsync(loss, 0, sizeof(float), st));
        return MOE_OK;
    }
    // logits by the fixed fma chain (one matrix: the projection kernel's second one is absent)
    MOE_TRY(launch_projection(x, act, T, d, n, Wg, nullptr, logits, nullptr, nullptr, 0, nullptr, 1, nullptr, st));
    bal_softmax_kernel<<<(unsigned)cdiv(T, 8), 256, 0, st>>>(logits, T, n, probs);
    MOE_LAUNCHED();
    bal_transpose_kernel<<<dim3((unsigned)cdiv(T, 32), (unsigned)cdiv(n, 32)), 256, 0, st>>>(probs, T, n, pT);
    MOE_LAUNCHED();
    bal_select_kernel<<<(unsigned)n, 1024, 0, st>>>(pT, T, n, m, words, tok_of_row, mask_bits);
    MOE_LAUNCHED();
    bal_token_kernel<<<(unsigned)cdiv(T, 8), 256, n * sizeof(int32_t), st>>>(probs, mask_bits, thr, T, n, words, den, cnt,
                                                                             thr_counts, loss_part);
    MOE_LAUNCHED();
    bal_loss_final_kernel<<<1, 256, 0, st>>>(loss_part, cdiv(T, 8), loss);
    MOE_LAUNCHED();
    MOE_TRY(launch_exclusive_scan(cnt, (int32_t)T, tok_ptr, st, tile_sums));
    bal_fill_kernel<<<(unsigned)cdiv(R > n ? R : n + 1, 256) + 1, 256, 0, st>>>(tok_of_row, mask_bits, tok_ptr, R, n, m, words,
                                                                                tok_rows, offsets);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_balanced_gather(const void *x, int32_t act, const int32_t *tok_of_row, int64_t R, int64_t T, int32_t d,
                               void *xs, cudaStream_t st) {
    if (R == 0) return MOE_OK;
    if (act == MOE_BF16) bal_gather_kernel<bf16><<<(unsigned)cdiv(R, 8), 256, 0, st>>>((const bf16 *)x, tok_of_row, R, T, d, (bf16 *)xs);
    else bal_gather_kernel<float><<<(unsigned)cdiv(R, 8), 256, 0, st>>>((const float *)x, tok_of_row, R, T, d, (float *)xs);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_balanced_combine(const void *ys, int32_t act, const float *p, const float *den, const int32_t *tok_ptr,
                                const int32_t *tok_rows, int64_t T, int64_t R, int32_t n, int32_t m, int32_t d, void *y,
                                cudaStream_t st) {
    if (T == 0) return MOE_OK;
    if (act == MOE_BF16)
        bal_combine_kernel<bf16><<<(unsigned)cdiv(T, 8), 256, 0, st>>>((const bf16 *)ys, p, den, tok_ptr, tok_rows, T, R, n, m, d, (bf16 *)y);
    else
        bal_combine_kernel<float><<<(unsigned)cdiv(T, 8), 256, 0, st>>>((const float *)ys, p, den, tok_ptr, tok_rows, T, R, n, m, d, (float *)y);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_balanced_combine_bwd(const void *dY, const void *ys, int32_t act, const float *p, const float *den,
                                    const int32_t *tok_of_row, int64_t R, int64_t T, int32_t n, int32_t m, int32_t d,
                                    float *dG_row, void *dys, cudaStream_t st) {
    if (R == 0) return MOE_OK;
    if (act == MOE_BF16)
        bal_combine_bwd_kernel<bf16><<<(unsigned)cdiv(R, 8), 256, 0, st>>>((const bf16 *)dY, (const bf16 *)ys, p, den, tok_of_row, R, T, n, m, d, dG_row, (bf16 *)dys);
    else
        bal_combine_bwd_kernel<float><<<(unsigned)cdiv(R, 8), 256, 0, st>>>((const float *)dY, (const float *)ys, p, den, tok_of_row, R, T, n, m, d, dG_row, (float *)dys);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_balanced_gate_bwd(const float *p, const uint32_t *mask_bits, const float *den, const float *thr,
                                 const int32_t *tok_ptr, const int32_t *tok_rows, const float *dG_row,
                                 const int32_t *thr_counts, float w, int64_t T, int32_t n, int32_t m, float *dc,
                                 void *dsplit, float *dthr, cudaStream_t st) {
    const int32_t words = (n + 31) / 32;
    if (T > 0) {
        bal_gate_bwd_kernel<<<(unsigned)cdiv(T, 8), 256, 0, st>>>(p, mask_bits, den, thr, tok_ptr, tok_rows, dG_row, w, T, n, m, words, dc,
                                                                  (bf16 *)dsplit);
        MOE_LAUNCHED();
    }
    bal_dthr_kernel<<<(unsigned)cdiv(n, 256), 256, 0, st>>>(thr_counts, n, T > 0 ? m : 0, w, dthr);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_balanced_dispatch_bwd(const void *dxs, int32_t act, const int32_t *tok_ptr, const int32_t *tok_rows,
                                     const float *dX_gate, int64_t T, int64_t R, int32_t d, void *dX, cudaStream_t st) {
    if (T == 0) return MOE_OK;
    if (act == MOE_BF16)
        bal_dispatch_bwd_kernel<bf16><<<(unsigned)cdiv(T, 8), 256, 0, st>>>((const bf16 *)dxs, tok_ptr, tok_rows, dX_gate, T, R, d, (bf16 *)dX);
    else
        bal_dispatch_bwd_kernel<float><<<(unsigned)cdiv(T, 8), 256, 0, st>>>((const float *)dxs, tok_ptr, tok_rows, dX_gate, T, R, d, (float *)dX);
    MOE_LAUNCHED();
    return MOE_OK;
}

}  // namespace moe
