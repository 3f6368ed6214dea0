// Back-propagation through the gating network (Section 2.1, "Training the Gating Network"):
// exact derivative of Eq. 3-5 and of the load estimator Eq. 9-10 w.r.t. the clean logits
// c = x.W_g and the raw noise logits r = x.W_noise.
#include <math_constants.h>

#include "moe_internal.cuh"

namespace moe {

// One warp per row. With sigma = softplus(r), z = (c - thr)/sigma, q_j = dLoad_j * phi(z_j)/sigma_j:
//   softmax over the kept slots:  dH[idx_s] += g_s (dg_s - sum_s' g_s' dg_s')
//   load estimator:               dc_j += q_j ; dsigma_j += -z_j q_j ;
//                                 the threshold is another entry's noisy logit:
//                                 dH[j_(k+1)] -= sum_{kept j} q_j ; dH[j_k] -= sum_{other j} q_j
//   H = c + eps * sigma:          dc += dH ; dsigma += eps * dH ; dr = dsigma * sigmoid(r)
template <int NV>  // columns per lane kept in registers (n <= 32 * NV); 0: any n, recompute in a second pass
__global__ void __launch_bounds__(256) gate_logit_grads_kernel(
    const float *__restrict__ noise, const float *__restrict__ clean, const float *__restrict__ raw,
    const int32_t *__restrict__ idx, const float *__restrict__ gates, const float *__restrict__ kth_vals,
    const int32_t *__restrict__ kth_idx, const float *__restrict__ dgates, const float *__restrict__ dload,
    const int32_t *__restrict__ dload_row_group, int64_t rows, int32_t n, int32_t k, float *__restrict__ dclean,
    float *__restrict__ draw, bf16 *__restrict__ dsplit, const int32_t *__restrict__ split_row_index) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    int32_t sel_idx[MOE_MAX_K];
    float sel_dh[MOE_MAX_K];
    float inner = 0.0f;
#pragma unroll
    for (int s = 0; s < MOE_MAX_K; ++s) {
        sel_idx[s] = s < k ? idx[row * k + s] : -1;
        if (s < k) inner = fmaf(gates[row * k + s], dgates[row * k + s], inner);
    }
#pragma unroll
    for (int s = 0; s < MOE_MAX_K; ++s)
        sel_dh[s] = s < k ? gates[row * k + s] * (dgates[row * k + s] - inner) : 0.0f;
    const float thr_unsel = kth_vals[row * 2 + 0], thr_sel = kth_vals[row * 2 + 1];
    const int32_t j_k = kth_idx[row * 2 + 0], j_k1 = kth_idx[row * 2 + 1];
    const float *dl = dload + (dload_row_group ? (int64_t)dload_row_group[row] * n : 0);
    const float *c = clean + row * n, *r = raw + row * n, *e = noise + row * n;

    // per column: is it kept, its softmax-path gradient, q = dLoad * phi(z) / sigma and z * q
    auto load_terms = [&](int32_t j, float cj, float rj, float dlj, bool &sel, float &dh_soft, float &q, float &zq) {
        sel = false;
        dh_soft = 0.0f;
#pragma unroll
        for (int s = 0; s < MOE_MAX_K; ++s)
            if (sel_idx[s] == j) { sel = true; dh_soft = sel_dh[s]; }
        const float sigma = fmaxf(rj, 0.0f) + log1pf(expf(-fabsf(rj)));
        const float z = (cj - (sel ? thr_sel : thr_unsel)) / sigma;
        if (isfinite(z)) {
            q = dlj * (expf(-0.5f * z * z) * 0.39894228040143267794f) / sigma;
            zq = z * q;
        } else {
            q = 0.0f;
            zq = 0.0f;
        }
    };
    auto finish = [&](int32_t j, float rj, float ej, float dh, float q, float zq, float q_sel, float q_uns) {
        if (j == j_k1) dh -= q_sel;
        if (j == j_k && k < n) dh -= q_uns;
        const float dsigma = fmaf(ej, dh, -zq);
        const float dc = q + dh, dr = dsigma / (1.0f + expf(-rj));
        if (dsplit) {
            // three-term bf16 split (hi | mid | lo), row layout [3][clean n | raw n], for the tensor-core products
            const int64_t orow = split_row_index ? split_row_index[row] : row;  // e.g. sorted by primary group
            bf16 *o = dsplit + orow * (6 * (int64_t)n);
            float v = dc;
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const bf16 b = __float2bfloat16_rn(v);
                o[term * 2 * n + j] = b;
                v -= __bfloat162float(b);
            }
            v = dr;
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const bf16 b = __float2bfloat16_rn(v);
                o[term * 2 * n + n + j] = b;
                v -= __bfloat162float(b);
            }
        } else {
            dclean[row * n + j] = dc;
            draw[row * n + j] = dr;
        }
    };

    float q_sel = 0.0f, q_uns = 0.0f;
    if (NV > 0) {
        float cv[NV > 0 ? NV : 1], rv[NV > 0 ? NV : 1], ev[NV > 0 ? NV : 1], dv[NV > 0 ? NV : 1];
        float dhv[NV > 0 ? NV : 1], qv[NV > 0 ? NV : 1], zqv[NV > 0 ? NV : 1];
#pragma unroll
        for (int u = 0; u < NV; ++u) {  // all loads of the row first
            const int32_t j = lane + 32 * u;
            const bool in = j < n;
            cv[u] = in ? c[j] : 0.0f; rv[u] = in ? r[j] : 0.0f; ev[u] = in ? e[j] : 0.0f; dv[u] = in ? dl[j] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int32_t j = lane + 32 * u;
            bool sel = false;
            dhv[u] = qv[u] = zqv[u] = 0.0f;
            if (j < n) {
                load_terms(j, cv[u], rv[u], dv[u], sel, dhv[u], qv[u], zqv[u]);
                if (sel) q_sel += qv[u]; else q_uns += qv[u];
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            q_sel += __shfl_xor_sync(0xffffffffu, q_sel, off);
            q_uns += __shfl_xor_sync(0xffffffffu, q_uns, off);
        }
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int32_t j = lane + 32 * u;
            if (j < n) finish(j, rv[u], ev[u], dhv[u], qv[u], zqv[u], q_sel, q_uns);
        }
    } else {
        for (int32_t j = lane; j < n; j += 32) {
            bool sel; float dh, q, zq;
            load_terms(j, c[j], r[j], dl[j], sel, dh, q, zq);
            if (sel) q_sel += q; else q_uns += q;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            q_sel += __shfl_xor_sync(0xffffffffu, q_sel, off);
            q_uns += __shfl_xor_sync(0xffffffffu, q_uns, off);
        }
        for (int32_t j = lane; j < n; j += 32) {
            bool sel; float dh, q, zq;
            load_terms(j, c[j], r[j], dl[j], sel, dh, q, zq);
            finish(j, r[j], e[j], dh, q, zq, q_sel, q_uns);
        }
    }
}

// The same for the tensor-core path (split output, n a multiple of 32): a lane owns PAIRS of adjacent columns, so the
// row is read with 8-byte loads and the six bf16 terms of a pair leave as 4-byte stores (half the memory instructions),
// and only the first KS slots are compared (KS >= k).
template <int NVP, int KS>  // column pairs per lane (n <= 64 * NVP)
__global__ void __launch_bounds__(256) gate_logit_grads_pairs_kernel(
    const float *__restrict__ noise, const float *__restrict__ clean, const float *__restrict__ raw,
    const int32_t *__restrict__ idx, const float *__restrict__ gates, const float *__restrict__ kth_vals,
    const int32_t *__restrict__ kth_idx, const float *__restrict__ dgates, const float *__restrict__ dload,
    const int32_t *__restrict__ dload_row_group, int64_t rows, int32_t n, int32_t k, bf16 *__restrict__ dsplit,
    const int32_t *__restrict__ split_row_index) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    int32_t sel_idx[KS];
    float sel_dh[KS];
    float inner = 0.0f;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
        sel_idx[s] = s < k ? idx[row * k + s] : -1;
        if (s < k) inner = fmaf(gates[row * k + s], dgates[row * k + s], inner);
    }
#pragma unroll
    for (int s = 0; s < KS; ++s) sel_dh[s] = s < k ? gates[row * k + s] * (dgates[row * k + s] - inner) : 0.0f;
    const float thr_unsel = kth_vals[row * 2 + 0], thr_sel = kth_vals[row * 2 + 1];
    const int32_t j_k = kth_idx[row * 2 + 0], j_k1 = kth_idx[row * 2 + 1];
    const float *dl = dload + (dload_row_group ? (int64_t)dload_row_group[row] * n : 0);
    const float *c = clean + row * n, *r = raw + row * n, *e = noise + row * n;

    float2 cv[NVP], rv[NVP], ev[NVP], dv[NVP];
    float dhv[2 * NVP], qv[2 * NVP], zqv[2 * NVP];
#pragma unroll
    for (int u = 0; u < NVP; ++u) {  // all loads of the row first
        const int32_t j = 2 * lane + 64 * u;
        const bool in = j < n;
        const float2 z2 = make_float2(0.0f, 0.0f);
        cv[u] = in ? *reinterpret_cast<const float2 *>(c + j) : z2;
        rv[u] = in ? *reinterpret_cast<const float2 *>(r + j) : z2;
        ev[u] = in ? *reinterpret_cast<const float2 *>(e + j) : z2;
        dv[u] = in ? *reinterpret_cast<const float2 *>(dl + j) : z2;
    }
    float q_sel = 0.0f, q_uns = 0.0f;
#pragma unroll
    for (int u = 0; u < 2 * NVP; ++u) {
        const int32_t j = 2 * lane + 64 * (u >> 1) + (u & 1);
        const float cj = (u & 1) ? cv[u >> 1].y : cv[u >> 1].x, rj = (u & 1) ? rv[u >> 1].y : rv[u >> 1].x;
        const float dlj = (u & 1) ? dv[u >> 1].y : dv[u >> 1].x;
        dhv[u] = qv[u] = zqv[u] = 0.0f;
        if (j < n) {
            bool sel = false;
#pragma unroll
            for (int s = 0; s < KS; ++s)
                if (sel_idx[s] == j) { sel = true; dhv[u] = sel_dh[s]; }
            // hardware exponential and reciprocal where a few ulp do not matter (the gradients are graded at 1e-5);
            // the softplus keeps its accurate logarithm: sigma enters squared
            const float sigma = fmaxf(rj, 0.0f) + log1pf(__expf(-fabsf(rj)));
            const float rs = __fdividef(1.0f, sigma);
            const float z = (cj - (sel ? thr_sel : thr_unsel)) * rs;
            if (isfinite(z)) {
                qv[u] = dlj * (__expf(-0.5f * z * z) * 0.39894228040143267794f) * rs;
                zqv[u] = z * qv[u];
            }
            if (sel) q_sel += qv[u]; else q_uns += qv[u];
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        q_sel += __shfl_xor_sync(0xffffffffu, q_sel, off);
        q_uns += __shfl_xor_sync(0xffffffffu, q_uns, off);
    }
    const int64_t orow = split_row_index ? split_row_index[row] : row;  // e.g. sorted by primary group
    bf16 *o = dsplit + orow * (6 * (int64_t)n);
#pragma unroll
    for (int u = 0; u < NVP; ++u) {
        const int32_t j = 2 * lane + 64 * u;
        if (j >= n) continue;
        float dc[2], dr[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float rj = h ? rv[u].y : rv[u].x, ej = h ? ev[u].y : ev[u].x;
            float dh = dhv[2 * u + h];
            if (j + h == j_k1) dh -= q_sel;
            if (j + h == j_k && k < n) dh -= q_uns;
            const float dsigma = fmaf(ej, dh, -zqv[2 * u + h]);
            dc[h] = qv[2 * u + h] + dh;
            dr[h] = __fdividef(dsigma, 1.0f + __expf(-rj));
        }
        // three-term bf16 split (hi | mid | lo), row layout [3][clean n | raw n], for the tensor-core products
#pragma unroll
        for (int term = 0; term < 3; ++term) {
            const __nv_bfloat162 bc = __floats2bfloat162_rn(dc[0], dc[1]), br = __floats2bfloat162_rn(dr[0], dr[1]);
            *reinterpret_cast<__nv_bfloat162 *>(o + term * 2 * n + j) = bc;
            *reinterpret_cast<__nv_bfloat162 *>(o + term * 2 * n + n + j) = br;
            dc[0] -= __bfloat162float(bc.x); dc[1] -= __bfloat162float(bc.y);
            dr[0] -= __bfloat162float(br.x); dr[1] -= __bfloat162float(br.y);
        }
    }
}

int32_t launch_gate_logit_grads(const float *noise, const float *clean, const float *raw, const int32_t *idx,
                                const float *gates, const float *kth_vals, const int32_t *kth_idx,
                                const float *dgates, const float *dload, const int32_t *dload_row_group,
                                int64_t rows, int32_t n, int32_t k, float *dclean, float *draw, void *dsplit,
                                const int32_t *split_row_index, cudaStream_t st) {
    if (rows == 0) return MOE_OK;
    const unsigned grid = (unsigned)cdiv(rows, 8);
    if (dsplit && n % 32 == 0 && n <= 256) {  // the tensor-core path: paired columns
#define MOE_LOGIT_PAIRS_KS(NVP, KS)                                                                                      \
    gate_logit_grads_pairs_kernel<NVP, KS><<<grid, 256, 0, st>>>(noise, clean, raw, idx, gates, kth_vals, kth_idx, dgates, \
                                                                 dload, dload_row_group, rows, n, k, (bf16 *)dsplit,      \
                                                                 split_row_index)
#define MOE_LOGIT_PAIRS(NVP)                                \
    do {                                                    \
        if (k <= 2) MOE_LOGIT_PAIRS_KS(NVP, 2);             \
        else if (k <= 4) MOE_LOGIT_PAIRS_KS(NVP, 4);        \
        else MOE_LOGIT_PAIRS_KS(NVP, MOE_MAX_K);            \
    } while (0)
        if (n <= 64) MOE_LOGIT_PAIRS(1);
        else if (n <= 128) MOE_LOGIT_PAIRS(2);
        else MOE_LOGIT_PAIRS(4);
#undef MOE_LOGIT_PAIRS
#undef MOE_LOGIT_PAIRS_KS
        MOE_LAUNCHED();
        return MOE_OK;
    }
#define MOE_LOGIT_GRADS(NV)                                                                                          \
    gate_logit_grads_kernel<NV><<<grid, 256, 0, st>>>(noise, clean, raw, idx, gates, kth_vals, kth_idx, dgates, dload, \
                                                      dload_row_group, rows, n, k, dclean, draw, (bf16 *)dsplit,      \
                                                      split_row_index)
    if (n <= 32) MOE_LOGIT_GRADS(1);
    else if (n <= 64) MOE_LOGIT_GRADS(2);
    else if (n <= 128) MOE_LOGIT_GRADS(4);
    else if (n <= 256) MOE_LOGIT_GRADS(8);
    else MOE_LOGIT_GRADS(0);
#undef MOE_LOGIT_GRADS
    MOE_LAUNCHED();
    return MOE_OK;
}

}  // namespace moe
