// Noisy top-k gating (Section 2.1, Eq. 3-5): projection, noisy logits, KeepTopK, masked softmax.
#include <math_constants.h>

#include "moe_internal.cuh"

namespace moe {

// ------------------------------------------------------------------------------------------
// Projection  clean = x.W_g,  raw = x.W_noise   (the two products of Eq. 4)
//
// The routing must be reproducible bit for bit, so every output is ONE chain of fused
// multiply-adds over the input features in ascending order, starting from +0. A register-tiled
// SIMT kernel keeps that order by construction (each accumulator sees k = 0, 1, 2, ...); a
// tensor-core MMA would not. The kernel is therefore bound by the FP32 pipes, not by HBM.
//
// Tile 128 rows x BN virtual columns (the columns of [W_g | W_noise] side by side), BK = 16,
// 256 threads, 8 x (BN/16) accumulators per thread.
// ------------------------------------------------------------------------------------------
constexpr int PBM = 128;
constexpr int PBK = 16;

struct ProjArgs {
    const void *x;
    const float *W0, *W1;
    float *out0, *out1;
    const int32_t *offsets;      // grouped only
    const int32_t *perm;         // grouped only
    const int32_t *tile_prefix;  // grouped only
    const int32_t *row_count;    // optional (ungrouped): number of rows, read on the device
    int64_t M;
    int32_t d, n0, nseg, kdiv;
};

template <typename XT, int BN>
__global__ void __launch_bounds__(256) proj_kernel(ProjArgs a) {
    constexpr int TN = BN / 16;  // 8 or 4 columns per thread
    __shared__ __align__(16) float As[PBK][PBM];
    __shared__ __align__(16) float Bs[PBK][BN];
    __shared__ int32_t row_tok[PBM];  // source token of each tile row (-1: none)
    __shared__ int32_t row_out[PBM];  // output row of each tile row

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int32_t n0 = a.n0, d = a.d;
    const int32_t ncols = a.W1 ? 2 * n0 : n0;  // W1 == nullptr: one matrix only
    const int32_t j0 = blockIdx.y * BN;

    // which rows does this tile cover?
    const float *W0 = a.W0, *W1 = a.W1;
    int64_t r0, r_end;
    if (a.offsets == nullptr) {
        r0 = (int64_t)blockIdx.x * PBM;
        r_end = a.row_count ? (int64_t)*a.row_count : a.M;
        if (r0 >= r_end) return;
    } else {
        const int32_t b = blockIdx.x;
        if (b >= a.tile_prefix[a.nseg]) return;
        int lo = 0, hi = a.nseg;  // last e with tile_prefix[e] <= b
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (a.tile_prefix[mid] <= b) lo = mid; else hi = mid;
        }
        r0 = a.offsets[lo] + (int64_t)(b - a.tile_prefix[lo]) * PBM;
        r_end = a.offsets[lo + 1];
        W0 += (int64_t)lo * d * n0;
        if (W1) W1 += (int64_t)lo * d * n0;
    }
    if (tid < PBM) {
        int64_t r = r0 + tid;
        int32_t tok = -1, orow = -1;
        if (r < r_end) {
            if (a.perm) { orow = a.perm[r]; tok = orow / a.kdiv; }
            else { orow = (int32_t)r; tok = (int32_t)r; }
        }
        row_tok[tid] = tok;
        row_out[tid] = orow;
    }
    __syncthreads();

    float acc[8][TN];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.0f;

    // global -> register staging. A: thread loads 8 consecutive k of row (tid & 127).
    const int a_row = tid & 127, a_half = tid >> 7;
    const int32_t a_tok = row_tok[a_row];
    const XT *xrow = a_tok >= 0 ? reinterpret_cast<const XT *>(a.x) + (int64_t)a_tok * d : nullptr;
    float ra[8], rb[TN];

    auto load_tiles = [&](int k0) {
        const int kb = k0 + a_half * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) ra[i] = 0.0f;
        if (xrow) {
            if (kb + 8 <= d) {
                if constexpr (sizeof(XT) == 2) {
                    uint4 v = *reinterpret_cast<const uint4 *>(xrow + kb);
                    const bf16 *h = reinterpret_cast<const bf16 *>(&v);
#pragma unroll
                    for (int i = 0; i < 8; ++i) ra[i] = __bfloat162float(h[i]);
                } else {
                    float4 v0 = *reinterpret_cast<const float4 *>(xrow + kb);
                    float4 v1 = *reinterpret_cast<const float4 *>(xrow + kb + 4);
                    ra[0] = v0.x; ra[1] = v0.y; ra[2] = v0.z; ra[3] = v0.w;
                    ra[4] = v1.x; ra[5] = v1.y; ra[6] = v1.z; ra[7] = v1.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (kb + i < d) ra[i] = to_f32(xrow[kb + i]);
            }
        }
#pragma unroll
        for (int i = 0; i < TN; ++i) {
            const int e = tid + i * 256;
            const int kk = e / BN, j = j0 + (e % BN);
            float v = 0.0f;
            if (k0 + kk < d && j < ncols)
                v = j < n0 ? W0[(int64_t)(k0 + kk) * n0 + j] : W1[(int64_t)(k0 + kk) * n0 + (j - n0)];
            rb[i] = v;
        }
    };
    auto store_tiles = [&]() {
#pragma unroll
        for (int i = 0; i < 8; ++i) As[a_half * 8 + i][a_row] = ra[i];
#pragma unroll
        for (int i = 0; i < TN; ++i) {
            const int e = tid + i * 256;
            Bs[e / BN][e % BN] = rb[i];
        }
    };

    load_tiles(0);
    for (int k0 = 0; k0 < d; k0 += PBK) {
        store_tiles();
        __syncthreads();
        if (k0 + PBK < d) load_tiles(k0 + PBK);
#pragma unroll
        for (int kk = 0; kk < PBK; ++kk) {
            float av[8], bv[TN];
            *reinterpret_cast<float4 *>(&av[0]) = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
            *reinterpret_cast<float4 *>(&av[4]) = *reinterpret_cast<const float4 *>(&As[kk][64 + ty * 4]);
            *reinterpret_cast<float4 *>(&bv[0]) = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
            if constexpr (TN == 8)
                *reinterpret_cast<float4 *>(&bv[4]) = *reinterpret_cast<const float4 *>(&Bs[kk][64 + tx * 4]);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int lr = (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        const int32_t orow = row_out[lr];
        if (orow < 0) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int col = j0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
            if (col < n0) a.out0[(int64_t)orow * n0 + col] = acc[i][j];
            else if (col < ncols) a.out1[(int64_t)orow * n0 + (col - n0)] = acc[i][j];
        }
    }
}

int32_t launch_projection(const void *x, int32_t act, int64_t M, int32_t d, int32_t n0, const float *W0,
                          const float *W1, float *out0, float *out1, const int32_t *offsets, int32_t nseg,
                          const int32_t *perm, int32_t kdiv, int32_t *tile_prefix, cudaStream_t st,
                          const int32_t *row_count) {
    if (M == 0) return MOE_OK;
    ProjArgs a;
    a.x = x; a.W0 = W0; a.W1 = W1; a.out0 = out0; a.out1 = out1;
    a.offsets = offsets; a.perm = perm; a.tile_prefix = tile_prefix; a.row_count = row_count;
    a.M = M; a.d = d; a.n0 = n0; a.nseg = nseg; a.kdiv = kdiv;
    int64_t tiles_m = cdiv(M, PBM);
    if (offsets) {
        MOE_TRY(launch_tile_prefix(offsets, nseg, PBM, tile_prefix, st));
        tiles_m += nseg;
    }
    const int32_t ncols = W1 ? 2 * n0 : n0;
    const bool wide = ncols > 64;
    dim3 grid((unsigned)tiles_m, (unsigned)cdiv(ncols, wide ? 128 : 64));
    if (act == MOE_BF16) {
        if (wide) proj_kernel<bf16, 128><<<grid, 256, 0, st>>>(a);
        else proj_kernel<bf16, 64><<<grid, 256, 0, st>>>(a);
    } else {
        if (wide) proj_kernel<float, 128><<<grid, 256, 0, st>>>(a);
        else proj_kernel<float, 64><<<grid, 256, 0, st>>>(a);
    }
    MOE_LAUNCHED();
    return MOE_OK;
}

// ------------------------------------------------------------------------------------------
// Noisy logits H = clean + noise * softplus(raw) (Eq. 4), KeepTopK (Eq. 5) and the softmax over
// the kept entries (Eq. 3). One warp per row. Each lane keeps the k+1 best of its columns in a
// sorted register list (value descending, then index ascending); k+1 rounds of a warp arg-max
// over the list heads then produce the global order. Lowest index wins ties everywhere.
// softplus is evaluated in double and rounded once, H by one fused multiply-add.
// ------------------------------------------------------------------------------------------
template <int KL>  // length of the per-lane sorted lists, >= k + 1
__global__ void __launch_bounds__(256) gate_select_kernel(const float *__restrict__ clean,
                                                          const float *__restrict__ raw,
                                                          const float *__restrict__ noise, int64_t rows, int32_t n,
                                                          int32_t k, int32_t *__restrict__ idx,
                                                          float *__restrict__ gates, float *__restrict__ kth_vals,
                                                          int32_t *__restrict__ kth_idx,
                                                          const int32_t *__restrict__ row_list,
                                                          const int32_t *__restrict__ row_count,
                                                          const int2 *__restrict__ row_span,
                                                          const int2 *__restrict__ chain_list) {
    const int lane = threadIdx.x & 31;
    int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    // row_span (with a row list): {first chain entry, number of candidate columns} of a listed row whose other
    // columns are known to rank below k + 1, so only the candidates are looked at; {., -1}: every column
    int32_t cand_base = 0, cand_total = -1;
    if (row_list) {  // only the listed rows (their number is read on the device)
        if (row >= *row_count) return;
        if (row_span) { const int2 sp = row_span[row]; cand_base = sp.x; cand_total = sp.y; }
        row = row_list[row];
    } else if (row >= rows) {
        return;
    }
    float lv[KL];
    int32_t li[KL];
#pragma unroll
    for (int s = 0; s < KL; ++s) { lv[s] = -CUDART_INF_F; li[s] = INT32_MAX; }
    const float *c = clean + row * n, *r = raw + row * n, *e = noise + row * n;
    const int32_t visits = cand_total >= 0 ? cand_total : n;
    for (int32_t q = lane; q < visits; q += 32) {
        // a candidate's column is the code of its first chain entry (the clean one), modulo the group's block of 2n
        const int32_t j = cand_total >= 0 ? chain_list[cand_base + 2 * q].y % (2 * n) : q;
        const double rd = (double)r[j];
        const float sigma = (float)(fmax(rd, 0.0) + log1p(exp(-fabs(rd))));
        float v = fmaf(e[j], sigma, c[j]);
        if (!(v == v)) v = -CUDART_INF_F;  // a NaN logit ranks last: the selection stays total, indices stay in [0, n)
        int32_t id = j;
        bool shifting = false;
#pragma unroll
        for (int s = 0; s < KL; ++s) {
            if (shifting || v > lv[s] || li[s] == INT32_MAX) {  // an empty slot takes anything, -inf included
                float tv = lv[s]; int32_t ti = li[s];
                lv[s] = v; li[s] = id; v = tv; id = ti;
                shifting = true;
            }
        }
    }
    const int rounds = (k < n) ? k + 1 : k;
    float myv = -CUDART_INF_F;
    int32_t myi = -1;
    float v_k = -CUDART_INF_F, v_k1 = -CUDART_INF_F;
    int32_t i_k = -1, i_k1 = -1;
    for (int s = 0; s < rounds; ++s) {
        float hv = lv[0];
        int32_t hi = li[0];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, hv, off);
            int32_t oi = __shfl_xor_sync(0xffffffffu, hi, off);
            if (ov > hv || (ov == hv && oi < hi)) { hv = ov; hi = oi; }
        }
        if (li[0] == hi) {  // this lane held the winner: pop it
#pragma unroll
            for (int q = 0; q < KL - 1; ++q) { lv[q] = lv[q + 1]; li[q] = li[q + 1]; }
            lv[KL - 1] = -CUDART_INF_F;
            li[KL - 1] = INT32_MAX;
        }
        if (s < k && lane == s) { myv = hv; myi = hi; }
        if (s == k - 1) { v_k = hv; i_k = hi; }
        if (s == k) { v_k1 = hv; i_k1 = hi; }
    }
    // softmax over the k kept logits, denominator summed in slot order
    const float m = __shfl_sync(0xffffffffu, myv, 0);
    const float ex = lane < k ? expf(myv - m) : 0.0f;
    float den = 0.0f;
    for (int s = 0; s < k; ++s) den += __shfl_sync(0xffffffffu, ex, s);
    if (lane < k) {
        idx[row * k + lane] = myi;
        gates[row * k + lane] = ex / den;
    }
    if (lane == 0) {
        kth_vals[row * 2 + 0] = v_k;
        kth_vals[row * 2 + 1] = v_k1;
        kth_idx[row * 2 + 0] = i_k;
        kth_idx[row * 2 + 1] = i_k1;
    }
}

int32_t launch_gate_select(const float *clean, const float *raw, const float *noise, int64_t rows, int32_t n,
                           int32_t k, int32_t *idx, float *gates, float *kth_vals, int32_t *kth_idx,
                           cudaStream_t st, const int32_t *row_list, const int32_t *row_count, const void *row_span,
                           const void *chain_list) {
    if (rows == 0) return MOE_OK;
    const unsigned grid = (unsigned)cdiv(rows, 8);
#define MOE_SELECT(KL)                                                                                                 \
    gate_select_kernel<KL><<<grid, 256, 0, st>>>(clean, raw, noise, rows, n, k, idx, gates, kth_vals, kth_idx, row_list, \
                                                 row_count, (const int2 *)row_span, (const int2 *)chain_list)
    if (k <= 2) MOE_SELECT(3);
    else if (k <= 4) MOE_SELECT(5);
    else MOE_SELECT(MOE_MAX_K + 1);
#undef MOE_SELECT
    MOE_LAUNCHED();
    return MOE_OK;
}

// ------------------------------------------------------------------------------------------
// Tensor-core screening of the routing (bf16 activations). The projection x.[W_g|W_noise] is first
// done on the tensor cores with W split into three bf16 terms (~1e-7 of the fma-chain value). From
// those approximate logits each token's top-(k+2) is found together with a bound U on how far any
// approximate noisy logit can be from the value the fixed fma chain would give:
//     |H~_j - H_j| <= theta * |x|_2 * (|W_g[:,j]|_2 + |noise_j| * |W_noise[:,j]|_2) + rounding slack,
// theta covering the worst-case rounding of the chain (d * 2^-24) and of the tensor-core accumulation
// (modelled as one truncation of an fp32 accumulator per MMA step, doubled). If every gap between
// consecutive ranks 1..k+2 exceeds 2U, the order of the top k+1 under the chain values is provably the
// same, so the routing taken from the approximate logits IS the bit-exact routing. The other tokens
// (a few per cent) are listed and redone with the fma chain by the kernels above.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) split_gate_weights_kernel(const float *__restrict__ Wg,
                                                                 const float *__restrict__ Wn, int32_t d, int32_t n,
                                                                 bf16 *__restrict__ wsplit) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t n2 = 2 * n;
    if (i >= (int64_t)d * n2) return;
    const int32_t q = (int32_t)(i / n2), j = (int32_t)(i % n2);
    float v = j < n ? Wg[(int64_t)q * n + j] : Wn[(int64_t)q * n + (j - n)];
#pragma unroll
    for (int term = 0; term < 3; ++term) {  // wsplit[term][q][j]: hi, mid, lo
        const bf16 b = __float2bfloat16_rn(v);
        wsplit[((int64_t)term * d + q) * n2 + j] = b;
        v -= __bfloat162float(b);
    }
}

// one warp per column of [W_g | W_noise]; blockIdx.y = group (stacked [groups, d, n] matrices)
__global__ void __launch_bounds__(256) gate_col_norms_kernel(const float *__restrict__ Wg, const float *__restrict__ Wn,
                                                             int32_t d, int32_t n, float *__restrict__ wnorm) {
    const int lane = threadIdx.x & 31;
    const int32_t j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (j >= 2 * n) return;
    Wg += (int64_t)blockIdx.y * d * n; Wn += (int64_t)blockIdx.y * d * n; wnorm += (int64_t)blockIdx.y * 2 * n;
    const float *W = j < n ? Wg + j : Wn + (j - n);
    double s = 0.0;
    for (int32_t q = lane; q < d; q += 32) { const double v = W[(int64_t)q * n]; s += v * v; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) wnorm[j] = (float)(sqrt(s) * (1.0 + 1e-6));
}

// |x_t|_2 (slightly rounded up), one warp per row; bf16 rows are read 16 bytes per lane, four loads in flight
template <typename XT>
__global__ void __launch_bounds__(256) row_norms_kernel(const XT *__restrict__ x, int64_t T, int32_t d,
                                                        float *__restrict__ xnorm) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    float s = 0.0f;
    if constexpr (sizeof(XT) == 2) {
        if (d % 8 == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
            const uint4 *row = reinterpret_cast<const uint4 *>(x + t * d);
            const int32_t pieces = d / 8;
            for (int32_t q0 = lane; q0 < pieces; q0 += 128) {
                uint4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) v[i] = q0 + 32 * i < pieces ? row[q0 + 32 * i] : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const bf16 *h = reinterpret_cast<const bf16 *>(&v[i]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) { const float f = __bfloat162float(h[e]); s = fmaf(f, f, s); }
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            if (lane == 0) xnorm[t] = sqrtf(s) * (1.0f + 1e-5f);
            return;
        }
    }
    for (int32_t q = lane; q < d; q += 32) { const float v = to_f32(x[t * d + q]); s = fmaf(v, v, s); }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) xnorm[t] = sqrtf(s) * (1.0f + 1e-5f);
}

// Approximate noisy logit v of one column and a bound u on its distance from the fma chain's value; c, r = the
// tensor-core products, e = the noise, xn = theta |x|, wg / wn = the column norms of W_g / W_noise. Both screening
// kernels call this one function, written with the non-contracting intrinsics so that they get the same bits.
// The hardware exponential and logarithm are enough here: their error is an absolute 7.2e-7 at most on sigma (2.4e-7
// from __expf on [-inf, 0], 1.2e-7 from rounding 1 + y, 2^-21.41 from __logf on [1, 2]) and goes into u with a margin
// (2e-6 |noise|).
__device__ __forceinline__ void screen_eval(float c, float r, float e, float xn, float wg, float wn, float &v, float &u) {
    const float sigma = __fadd_rn(fmaxf(r, 0.0f), __logf(__fadd_rn(1.0f, __expf(-fabsf(r)))));
    v = __fmaf_rn(e, sigma, c);
    // |H~_j - H_j|: projection errors through c and through softplus(r) (slope <= 1) times |noise|, plus the error of
    // softplus (here approximate, there double rounded once) and of the final fma on both sides
    const float ae = fabsf(e);
    const float rounding = __fmul_rn(1.1920929e-7f, __fmaf_rn(16.0f * ae, sigma, 8.0f * fabsf(v)));
    u = __fmaf_rn(2.0e-6f, ae, __fmaf_rn(xn, __fmaf_rn(ae, wn, wg), rounding));
}

// The screen, one thread per token (sorted row): a warp stages 16 columns of its 32 rows at a time through shared memory
// (16-byte loads along the rows, 16-byte reads down the rows, both conflict free with a pitch of 20 words), copies
// them to clean / raw on the way, and every thread then walks its own row: a sorted list of the KL >= k + 2 largest
// approximate logits with their bounds, and the largest possible value of everything else. No shuffles, no arg-max
// rounds: a few dozen instructions per column. Certified rows get their routing here; the others are listed
// with `low`, the bound that decides which of their columns need an exact chain (gate_candidates_kernel).
// Grouped use (secondary gates of the hierarchical layer): cr rows are sorted by group; perm maps a sorted row to its
// output row (the slot t * k1 + s1), the token is output row / kdiv, group_of gives the slot's group, whose column
// norms are used. Flat use: perm = group_of = nullptr, kdiv = 1.
constexpr int SCREEN_CH = 16, SCREEN_PITCH = 20;
// four floats at p: one 16-byte access where the tensor allows it (V16), else four 4-byte ones (the secondary gates'
// part of noise / clean / raw starts T * a floats into the tensor, not always a multiple of four)
template <bool V16>
__device__ __forceinline__ float4 load4(const float *p) {
    if constexpr (V16) return *reinterpret_cast<const float4 *>(p);
    else return make_float4(p[0], p[1], p[2], p[3]);
}
template <bool V16>
__device__ __forceinline__ void store4(float *p, float4 v) {
    if constexpr (V16) *reinterpret_cast<float4 *>(p) = v;
    else { p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w; }
}
template <int KL, bool V16>
__global__ void __launch_bounds__(128) gate_screen_rows_kernel(const float *__restrict__ cr, const float *__restrict__ noise,
                                                               const float *__restrict__ xnorm,
                                                               const float *__restrict__ wnorm, float theta, int64_t T,
                                                               int32_t n, int32_t k, int32_t *__restrict__ idx,
                                                               float *__restrict__ gates, float *__restrict__ clean,
                                                               float *__restrict__ raw, float *__restrict__ kth_vals,
                                                               int32_t *__restrict__ kth_idx,
                                                               int32_t *__restrict__ unsafe_list,
                                                               float *__restrict__ unsafe_low,
                                                               int32_t *__restrict__ unsafe_count,
                                                               const int32_t *__restrict__ perm, int32_t kdiv,
                                                               const int32_t *__restrict__ group_of) {
    __shared__ __align__(16) float tile[4][3][32 * SCREEN_PITCH];
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const int64_t s0 = ((int64_t)blockIdx.x * 4 + wp) * 32;  // first sorted row of this warp
    if (s0 >= T) return;
    const int64_t srow = s0 + lane;
    const bool live = srow < T;
    const int64_t row = live ? (perm ? (int64_t)perm[srow] : srow) : 0;
    const float *wn = wnorm + (int64_t)(group_of && live ? group_of[row] : 0) * 2 * n;
    const float xn = live ? theta * xnorm[row / kdiv] : 0.0f;
    float lv[KL], lu[KL];
    int32_t li[KL];
#pragma unroll
    for (int s = 0; s < KL; ++s) { lv[s] = -CUDART_INF_F; li[s] = INT32_MAX; lu[s] = 0.0f; }
    float rest_hi = -CUDART_INF_F;  // largest possible chain value of anything that is not in the list
    auto insert = [&](int32_t j, float v, float u) {
        if (v > lv[KL - 1]) {
            // enters the list behind every entry that is at least as large (those have lower indices), the last
            // entry falls off
            rest_hi = fmaxf(rest_hi, lv[KL - 1] + lu[KL - 1]);
#pragma unroll
            for (int s = KL - 1; s >= 1; --s) {
                const bool stays = lv[s] >= v && s != KL - 1, here = lv[s - 1] >= v;
                if (!stays) {
                    lv[s] = here ? v : lv[s - 1];
                    lu[s] = here ? u : lu[s - 1];
                    li[s] = here ? j : li[s - 1];
                }
            }
            if (!(lv[0] >= v)) { lv[0] = v; lu[0] = u; li[0] = j; }
        } else {
            rest_hi = fmaxf(rest_hi, v + u);
        }
    };
    // four columns at a time: their values and bounds first (independent of each other, so the exponentials and
    // logarithms overlap), then the four list updates, which depend on one another
    auto consider4 = [&](int32_t j, const float4 &c4, const float4 &r4, const float4 &e4) {
        const float4 wg4 = *reinterpret_cast<const float4 *>(wn + j), wn4 = *reinterpret_cast<const float4 *>(wn + n + j);
        float v0, v1, v2, v3, u0, u1, u2, u3;
        screen_eval(c4.x, r4.x, e4.x, xn, wg4.x, wn4.x, v0, u0);
        screen_eval(c4.y, r4.y, e4.y, xn, wg4.y, wn4.y, v1, u1);
        screen_eval(c4.z, r4.z, e4.z, xn, wg4.z, wn4.z, v2, u2);
        screen_eval(c4.w, r4.w, e4.w, xn, wg4.w, wn4.w, v3, u3);
        insert(j, v0, u0);
        insert(j + 1, v1, u1);
        insert(j + 2, v2, u2);
        insert(j + 3, v3, u3);
    };
    // loads: instruction i covers the rows 8 i + lane / 4 of the warp, four columns per lane
    const int lr = lane >> 2, lq = (lane & 3) * 4;
    float *tc = tile[wp][0], *tr = tile[wp][1], *te = tile[wp][2];
    for (int32_t j0 = 0; j0 < n; j0 += SCREEN_CH) {
        float4 c4[4], r4[4], e4[4];
        int32_t orow[4];  // output rows fit 31 bits (they go into the int32 row lists)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t sr = s0 + 8 * i + lr;
            orow[i] = __shfl_sync(0xffffffffu, (int32_t)row, 8 * i + lr);
            c4[i] = r4[i] = e4[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (sr < T) {
                c4[i] = load4<V16>(cr + sr * 2 * n + j0 + lq);
                r4[i] = load4<V16>(cr + sr * 2 * n + n + j0 + lq);
                e4[i] = load4<V16>(noise + (int64_t)orow[i] * n + j0 + lq);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int at = (8 * i + lr) * SCREEN_PITCH + lq;
            *reinterpret_cast<float4 *>(tc + at) = c4[i];
            *reinterpret_cast<float4 *>(tr + at) = r4[i];
            *reinterpret_cast<float4 *>(te + at) = e4[i];
            if (s0 + 8 * i + lr < T) {
                store4<V16>(clean + (int64_t)orow[i] * n + j0 + lq, c4[i]);
                store4<V16>(raw + (int64_t)orow[i] * n + j0 + lq, r4[i]);
            }
        }
        __syncwarp();
#pragma unroll
        for (int q = 0; q < SCREEN_CH / 4; ++q) {
            const float4 cq = *reinterpret_cast<const float4 *>(tc + lane * SCREEN_PITCH + 4 * q);
            const float4 rq = *reinterpret_cast<const float4 *>(tr + lane * SCREEN_PITCH + 4 * q);
            const float4 eq = *reinterpret_cast<const float4 *>(te + lane * SCREEN_PITCH + 4 * q);
            consider4(j0 + 4 * q, cq, rq, eq);
        }
        __syncwarp();
    }
    // the first `rounds` entries are the ranked ones, whatever else is in the list is "rest" as well
    const int rounds = min(k + 2, n);
#pragma unroll
    for (int s = 0; s < KL; ++s)
        if (s >= rounds && li[s] != INT32_MAX) rest_hi = fmaxf(rest_hi, lv[s] + lu[s]);
    // ranks 1..k+1 are certain iff each one's lowest possible value beats the highest possible value of everything
    // ranked after it
    bool safe = true;
    float suffix = rest_hi;
#pragma unroll
    for (int s = KL - 1; s >= 0; --s) {
        if (s < rounds) {
            if (s <= k && !(lv[s] - lu[s] > suffix)) safe = false;
            suffix = fmaxf(suffix, lv[s] + lu[s]);
        }
    }
    // Not provably the chain's routing: only the columns that can still reach rank k+1 matter, those whose highest
    // possible value is at least `low`, a lower bound of the (k+1)-th largest chain value (the (k+1)-th largest lower end
    // among the ranked columns).
    float low = -CUDART_INF_F;
    if (!safe && k < rounds) {
#pragma unroll
        for (int s = 0; s < KL; ++s) {
            if (s < rounds) {
                const float ls = lv[s] - lu[s];
                int above = 0;
#pragma unroll
                for (int s2 = 0; s2 < KL; ++s2)
                    if (s2 < rounds && s2 != s) {
                        const float l2 = lv[s2] - lu[s2];
                        above += (l2 > ls || (l2 == ls && s2 < s)) ? 1 : 0;
                    }
                if (above == k) low = ls;
            }
        }
    }
    const bool listed = live && !safe;
    const uint32_t lb = __ballot_sync(0xffffffffu, listed);
    if (lb) {
        int32_t base = 0;
        if (lane == 0) base = atomicAdd(unsafe_count, __popc(lb));
        base = __shfl_sync(0xffffffffu, base, 0);
        if (listed) {
            const int32_t at = base + __popc(lb & ((1u << lane) - 1u));
            unsafe_list[at] = (int32_t)row;
            unsafe_low[at] = low;
        }
    }
    if (!live || !safe) return;
    float ex[KL], den = 0.0f;
#pragma unroll
    for (int s = 0; s < KL; ++s) {
        ex[s] = 0.0f;
        if (s < k) { ex[s] = expf(lv[s] - lv[0]); den += ex[s]; }
    }
#pragma unroll
    for (int s = 0; s < KL; ++s)
        if (s < k) {
            idx[row * k + s] = li[s];
            gates[row * k + s] = ex[s] / den;
        }
    float v_k = -CUDART_INF_F, v_k1 = -CUDART_INF_F;
    int32_t i_k = -1, i_k1 = -1;
#pragma unroll
    for (int s = 0; s < KL; ++s) {
        if (s == k - 1) { v_k = lv[s]; i_k = li[s]; }
        if (s == k && k < n) { v_k1 = lv[s]; i_k1 = li[s]; }
    }
    kth_vals[row * 2 + 0] = v_k;
    kth_vals[row * 2 + 1] = v_k1;
    kth_idx[row * 2 + 0] = i_k;
    kth_idx[row * 2 + 1] = i_k1;
}

// The rows the screen listed, one warp per row: the columns whose highest possible value reaches the row's `low` get
// their two fma chains redone (chain_list), the selection is then repeated on the patched row. Rows with more than
// SCREEN_MAX_CAND candidates (ties) take the full chain (full_list), or, where there is no whole-row fallback
// (full_list == nullptr), the chains of all their columns.
__global__ void __launch_bounds__(256) gate_candidates_kernel(const float *__restrict__ clean, const float *__restrict__ raw,
                                                              const float *__restrict__ noise,
                                                              const float *__restrict__ xnorm,
                                                              const float *__restrict__ wnorm, float theta, int32_t n,
                                                              const int32_t *__restrict__ unsafe_list,
                                                              const float *__restrict__ unsafe_low,
                                                              int32_t *__restrict__ unsafe_count,
                                                              int2 *__restrict__ chain_list,
                                                              int32_t *__restrict__ full_list, int32_t kdiv,
                                                              const int32_t *__restrict__ group_of, int32_t k,
                                                              int2 *__restrict__ unsafe_span) {
    // unsafe_span[i] = {first entry of the row's chains in chain_list, number of candidate columns}, or {0, -1}
    // where the repeated selection has to look at every column
    const int lane = threadIdx.x & 31;
    const int32_t total_rows = *unsafe_count;  // complete: the screen ran before this kernel
    const int32_t nwarps = gridDim.x * (blockDim.x >> 5);
    for (int32_t it = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); it < total_rows; it += nwarps) {
        const int64_t row = unsafe_list[it];
        const float low = unsafe_low[it];
        const int32_t group = group_of ? group_of[row] : 0;
        const float *wn = wnorm + (int64_t)group * 2 * n;
        const float xn = theta * xnorm[row / kdiv];
        const float *c = clean + row * n, *r = raw + row * n, *e = noise + row * n;
        auto candidate = [&](int32_t j) {
            if (j >= n) return false;
            float v, u;
            screen_eval(c[j], r[j], e[j], xn, wn[j], wn[n + j], v, u);
            return v + u >= low;
        };
        // one pass over the row: lane g keeps the ballot of the g-th group of 32 columns (rows wider than 1024
        // columns are evaluated again when their entries are written)
        int total = 0;
        uint32_t kept_word = 0u;
        for (int32_t j0 = 0; j0 < n; j0 += 32) {
            const uint32_t b = __ballot_sync(0xffffffffu, candidate(j0 + lane));
            if ((j0 >> 5) == lane) kept_word = b;
            total += __popc(b);
        }
        // (fewer than k + 1 candidates happens only with NaN logits, which are nobody's candidate)
        const bool few = total <= SCREEN_MAX_CAND && total >= min(k + 1, n);
        const int32_t wbase = group * 2 * n;  // this group's rows of the transposed weights
        int32_t base = 0;
        if (lane == 0) {
            if (few) base = atomicAdd(unsafe_count + 1, 2 * total);
            else if (full_list) full_list[atomicAdd(unsafe_count + 2, 1)] = (int32_t)row;
            else base = atomicAdd(unsafe_count + 1, 2 * n);
        }
        base = __shfl_sync(0xffffffffu, base, 0);
        if (lane == 0) unsafe_span[it] = few ? make_int2(base, total) : make_int2(0, -1);
        if (!few) {
            if (!full_list)
                for (int32_t j = lane; j < n; j += 32) {
                    chain_list[base + 2 * j] = make_int2((int32_t)row, wbase + j);
                    chain_list[base + 2 * j + 1] = make_int2((int32_t)row, wbase + n + j);
                }
            continue;
        }
        int pos = 0;
        for (int32_t j0 = 0; j0 < n; j0 += 32) {
            const int32_t j = j0 + lane;
            const uint32_t b = n <= 1024 ? __shfl_sync(0xffffffffu, kept_word, j0 >> 5)
                                         : __ballot_sync(0xffffffffu, candidate(j));
            const bool cand = (b >> lane) & 1u;
            if (cand) {
                const int at = base + 2 * (pos + __popc(b & ((1u << lane) - 1u)));
                chain_list[at] = make_int2((int32_t)row, wbase + j);
                chain_list[at + 1] = make_int2((int32_t)row, wbase + n + j);
            }
            pos += __popc(b);
        }
    }
}

// One fma chain per thread: entry (row, c) of chain_list recomputes clean[row, c] (c < n) or raw[row, c - n] exactly
// as the projection kernel does: fp32, from +0, ascending input feature. Wt [2n, d] holds the columns of
// [W_g | W_noise] as rows. The 32 chains of a warp read 32 different weight rows; a load instruction that touches 32
// lines costs the load/store unit 32 tag look-ups, which is what bounds this kernel, so the warp fetches the next 32
// features of its 32 rows cooperatively (eight lanes per 128-byte line, four lines per instruction), parks them in
// shared memory and every lane then reads its own row back. Loads for step s + 1 are in flight during the 32
// dependent fused multiply-adds of step s.
constexpr int CHAIN_PITCH = 144;  // bytes per staged row: 128 + 16, conflict-free both ways
template <typename XT>
__global__ void __launch_bounds__(128) gate_chain_kernel(const XT *__restrict__ x, int32_t d, int32_t n,
                                                         const float *__restrict__ Wt,
                                                         const int2 *__restrict__ chain_list,
                                                         const int32_t *__restrict__ chain_count,
                                                         float *__restrict__ clean, float *__restrict__ raw,
                                                         int32_t kdiv) {
    // entry {output row, row of Wt}: the token is output row / kdiv, the column code is Wt row mod 2n (grouped gates
    // keep one [2n, d] block of Wt per group)
    __shared__ __align__(16) uint8_t stage[4][2][32 * CHAIN_PITCH];
    const int32_t total = *chain_count;
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const int32_t steps = d / 32;  // d is a multiple of 64 on this path
    for (int32_t i0 = (blockIdx.x * 4 + wp) * 32; i0 < total; i0 += gridDim.x * 128) {  // warp-uniform
        const int32_t i = i0 + lane;
        const int2 en = chain_list[i < total ? i : total - 1];  // idle lanes shadow the last chain
        const XT *xr = x + (int64_t)(en.x / kdiv) * d;
        const float *wrow = Wt + (int64_t)en.y * d;
        // instruction u of a step loads 16 bytes of the row of lane 4 u + lane / 8, at byte (lane % 8) * 16
        const float *src[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const unsigned long long ptr = __shfl_sync(0xffffffffu, (unsigned long long)wrow, 4 * u + (lane >> 3));
            src[u] = reinterpret_cast<const float *>(ptr) + (lane & 7) * 4;
        }
        float4 wreg[8];
        uint4 xreg[4];
        auto fetch = [&](int32_t st) {
#pragma unroll
            for (int u = 0; u < 8; ++u) wreg[u] = *reinterpret_cast<const float4 *>(src[u] + st * 32);
            if constexpr (sizeof(XT) == 2) {
#pragma unroll
                for (int g = 0; g < 4; ++g) xreg[g] = *reinterpret_cast<const uint4 *>(xr + st * 32 + 8 * g);
            }
        };
        auto park = [&](int b) {
#pragma unroll
            for (int u = 0; u < 8; ++u)
                *reinterpret_cast<float4 *>(&stage[wp][b][(4 * u + (lane >> 3)) * CHAIN_PITCH + (lane & 7) * 16]) = wreg[u];
        };
        float acc = 0.0f;
        fetch(0);
        __syncwarp();  // the previous chains' last reads of the staging rows are done
        park(0);
        uint4 xcur[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) xcur[g] = xreg[g];
        __syncwarp();
        for (int32_t st = 0; st < steps; ++st) {
            if (st + 1 < steps) fetch(st + 1);
            const uint8_t *mine = &stage[wp][st & 1][lane * CHAIN_PITCH];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float4 wv = *reinterpret_cast<const float4 *>(mine + 16 * u);
                float x0, x1, x2, x3;
                if constexpr (sizeof(XT) == 2) {
                    const bf16 *hx = reinterpret_cast<const bf16 *>(&xcur[u >> 1]) + 4 * (u & 1);
                    x0 = __bfloat162float(hx[0]); x1 = __bfloat162float(hx[1]);
                    x2 = __bfloat162float(hx[2]); x3 = __bfloat162float(hx[3]);
                } else {
                    const int32_t q = st * 32 + 4 * u;
                    x0 = to_f32(xr[q]); x1 = to_f32(xr[q + 1]); x2 = to_f32(xr[q + 2]); x3 = to_f32(xr[q + 3]);
                }
                acc = fmaf(x0, wv.x, acc); acc = fmaf(x1, wv.y, acc);
                acc = fmaf(x2, wv.z, acc); acc = fmaf(x3, wv.w, acc);
            }
            if (st + 1 < steps) {
                park((st + 1) & 1);  // the other buffer: its readers finished a step ago (syncwarp below)
#pragma unroll
                for (int g = 0; g < 4; ++g) xcur[g] = xreg[g];
            }
            __syncwarp();
        }
        if (i < total) {
            const int32_t code = en.y % (2 * n);
            if (code >= n) raw[(int64_t)en.x * n + (code - n)] = acc;
            else clean[(int64_t)en.x * n + code] = acc;
        }
    }
}

// Wt[c, q] = [W_g | W_noise][q, c]
__global__ void __launch_bounds__(256) gate_transpose_weights_kernel(const float *__restrict__ Wg, const float *__restrict__ Wn,
                                                                     int32_t d, int32_t n, float *__restrict__ Wt) {
    __shared__ float tile[32][33];
    Wg += (int64_t)blockIdx.z * d * n; Wn += (int64_t)blockIdx.z * d * n; Wt += (int64_t)blockIdx.z * 2 * n * d;  // group
    const int q0 = blockIdx.x * 32, c0 = blockIdx.y * 32;  // 2n and d are multiples of 32 on this path
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + tx, q = q0 + i;
        tile[i][tx] = c < n ? Wg[(int64_t)q * n + c] : Wn[(int64_t)q * n + (c - n)];
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) Wt[(int64_t)(c0 + i) * d + q0 + tx] = tile[tx][i];
}

int32_t launch_gate_chains(const void *x, int32_t act, int32_t d, int32_t n, const float *Wt, const void *chain_list,
                           const int32_t *chain_count, float *clean, float *raw, cudaStream_t st, int32_t kdiv) {
    const unsigned grid = 148 * 16;
    if (act == MOE_BF16)
        gate_chain_kernel<bf16><<<grid, 128, 0, st>>>((const bf16 *)x, d, n, Wt, (const int2 *)chain_list, chain_count, clean,
                                                      raw, kdiv);
    else
        gate_chain_kernel<float><<<grid, 128, 0, st>>>((const float *)x, d, n, Wt, (const int2 *)chain_list, chain_count, clean,
                                                       raw, kdiv);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_gate_screen_prepare(const void *x, int32_t act, int64_t T, int32_t d, int32_t n, const float *Wg,
                                   const float *Wn, void *wsplit, float *wnorm, float *xnorm,
                                   int32_t *unsafe_count, float *wt, cudaStream_t st, int32_t groups, bool with_xnorm) {
    // groups > 1: Wg, Wn are stacks [groups, d, n]; wsplit [3][groups * d][2n], wnorm [groups][2n], wt [groups][2n][d]
    gate_transpose_weights_kernel<<<dim3((unsigned)(d / 32), (unsigned)(2 * n / 32), (unsigned)groups), 256, 0, st>>>(Wg, Wn, d, n,
                                                                                                                      wt);
    MOE_LAUNCHED();
    split_gate_weights_kernel<<<(unsigned)cdiv((int64_t)groups * d * 2 * n, 256), 256, 0, st>>>(Wg, Wn, groups * d, n,
                                                                                                  (bf16 *)wsplit);
    MOE_LAUNCHED();
    gate_col_norms_kernel<<<dim3((unsigned)cdiv(2 * n, 8), (unsigned)groups), 256, 0, st>>>(Wg, Wn, d, n, wnorm);
    MOE_LAUNCHED();
    if (with_xnorm) {
        if (act == MOE_BF16) row_norms_kernel<bf16><<<(unsigned)cdiv(T, 8), 256, 0, st>>>((const bf16 *)x, T, d, xnorm);
        else row_norms_kernel<float><<<(unsigned)cdiv(T, 8), 256, 0, st>>>((const float *)x, T, d, xnorm);
        MOE_LAUNCHED();
    }
    MOE_CUDA(cudaMemsetAsync(unsafe_count, 0, 4 * sizeof(int32_t), st));  // rows to re-select, chains, full-chain rows
    return MOE_OK;
}

int32_t launch_gate_screen(const float *cr, const float *noise, const float *xnorm, const float *wnorm, int32_t d,
                           int64_t T, int32_t n, int32_t k, int32_t *idx, float *gates, float *clean, float *raw,
                           float *kth_vals, int32_t *kth_idx, int32_t *unsafe_list, float *unsafe_low,
                           int32_t *unsafe_count, void *chain_list, int32_t *full_list, cudaStream_t st,
                           const int32_t *perm, int32_t kdiv, const int32_t *group_of, void *unsafe_span) {
    // worst-case rounding of the fma chain, plus two truncations of an fp32 accumulator per MMA step of the
    // three-term tensor-core product (3d/16 steps and the additions inside a step), plus the split residual
    const double u = ldexp(1.0, -24);
    const double chain = d * u / (1.0 - d * u);
    const double tc = 2.0 * (3.0 * d / 16.0 + 8.0) * ldexp(1.0, -23) + ldexp(1.0, -22);
    const float theta = (float)((chain + tc) * 1.01);
    if (T == 0) return MOE_OK;
    if (n % SCREEN_CH != 0) return MOE_ERR_INVALID_ARG;  // the screened path has 2n a multiple of 64
    const unsigned grid = (unsigned)cdiv(T, 128);
    const bool v16 = (((uintptr_t)noise | (uintptr_t)clean | (uintptr_t)raw | (uintptr_t)cr) & 15) == 0;
#define MOE_SCREEN_KL(KL)                                                                                              \
    do {                                                                                                               \
        if (v16)                                                                                                       \
            gate_screen_rows_kernel<KL, true><<<grid, 128, 0, st>>>(cr, noise, xnorm, wnorm, theta, T, n,                   \
                                                                    k, idx, gates, clean, raw, kth_vals, kth_idx,      \
                                                                    unsafe_list, unsafe_low, unsafe_count, perm, kdiv, \
                                                                    group_of);                                         \
        else                                                                                                           \
            gate_screen_rows_kernel<KL, false><<<grid, 128, 0, st>>>(cr, noise, xnorm, wnorm, theta, T,                     \
                                                                     n, k, idx, gates, clean, raw, kth_vals, kth_idx,  \
                                                                     unsafe_list, unsafe_low, unsafe_count, perm,      \
                                                                     kdiv, group_of);                                  \
    } while (0)
    if (k <= 2) MOE_SCREEN_KL(4);
    else if (k <= 4) MOE_SCREEN_KL(6);
    else MOE_SCREEN_KL(MOE_MAX_K + 2);
#undef MOE_SCREEN_KL
    MOE_LAUNCHED();
    gate_candidates_kernel<<<148 * 4, 256, 0, st>>>(clean, raw, noise, xnorm, wnorm, theta, n, unsafe_list, unsafe_low,
                                                    unsafe_count, (int2 *)chain_list, full_list, kdiv, group_of, k,
                                                    (int2 *)unsafe_span);
    MOE_LAUNCHED();
    return MOE_OK;
}

// Hierarchical gate (Eq. 12): flat expert id i*b + j and product gate, slots primary-major.
__global__ void hier_merge_kernel(int64_t total, int32_t k1, int32_t k2, int32_t b, const int32_t *idx_p,
                                  const float *g_p, const int32_t *idx_s, const float *g_s, int32_t *topk_idx,
                                  float *gates) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // over T*k1*k2
    if (i >= total) return;
    const int64_t p1 = i / k2;  // t*k1 + s1
    topk_idx[i] = idx_p[p1] * b + idx_s[i];
    gates[i] = g_p[p1] * g_s[i];
}

int32_t launch_hier_merge(int64_t T, int32_t k1, int32_t k2, int32_t b, const int32_t *idx_p, const float *g_p,
                          const int32_t *idx_s, const float *g_s, int32_t *topk_idx, float *gates,
                          cudaStream_t st) {
    const int64_t total = T * k1 * k2;
    if (total == 0) return MOE_OK;
    hier_merge_kernel<<<(unsigned)cdiv(total, 256), 256, 0, st>>>(total, k1, k2, b, idx_p, g_p, idx_s, g_s,
                                                                    topk_idx, gates);
    MOE_LAUNCHED();
    return MOE_OK;
}

MOE_BOUNDS_READER(bounds_violations_gate)

}  // namespace moe
