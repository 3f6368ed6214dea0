// Balancing losses (Section 4 and Appendix A): Importance (Eq. 6), the smooth load estimator
// P(x, i) (Eq. 9), Load (Eq. 10), the two CV^2 losses (Eq. 7, 11) and their gradients.
// Batch sums are deterministic: per-chunk partial sums in float, then one ordered pass in double.
#include <math_constants.h>

#include "moe_internal.cuh"

namespace moe {

constexpr int LCHUNKS_MAX = 148 * 4;

static inline int32_t level_chunks(int64_t rows) { return (int32_t)imin(cdiv(rows, 32), LCHUNKS_MAX); }
int64_t losses_ws_floats(int64_t rows, int32_t n) { return 2 * (int64_t)level_chunks(rows) * n + 64; }

__device__ __forceinline__ float softplus_f(float r) { return fmaxf(r, 0.0f) + log1pf(expf(-fabsf(r))); }

// Thread (tl, cw): column lane cw in [0, CW), token lane tl in [0, 256/CW). A block owns a chunk of
// rows; for each of its columns a thread sums over its rows, the token lanes are then added in order.
__global__ void __launch_bounds__(256) level_sums_kernel(const int32_t *__restrict__ idx,
                                                         const float *__restrict__ gates,
                                                         const float *__restrict__ clean,
                                                         const float *__restrict__ raw,
                                                         const float *__restrict__ kth_vals, int64_t rows, int32_t n,
                                                         int32_t k, int32_t CW, float *__restrict__ part_imp,
                                                         float *__restrict__ part_load) {
    __shared__ float red_i[256], red_l[256];
    const int cw = threadIdx.x % CW, tl = threadIdx.x / CW, TL = 256 / CW;
    const int64_t per = (rows + gridDim.x - 1) / gridDim.x;
    const int64_t r0 = (int64_t)blockIdx.x * per, r1 = min(r0 + per, rows);
    for (int32_t jb = 0; jb < n; jb += CW) {
        const int32_t j = jb + cw;
        float s_imp = 0.0f, s_load = 0.0f;
        if (j < n) {
            for (int64_t t = r0 + tl; t < r1; t += TL) {
                bool sel = false;
                float g = 0.0f;
                for (int s = 0; s < k; ++s)
                    if (idx[t * k + s] == j) { sel = true; g = gates[t * k + s]; }
                const float thr = kth_vals[t * 2 + (sel ? 1 : 0)];  // kth_excluding(H, k, j)
                const float z = (clean[t * n + j] - thr) / softplus_f(raw[t * n + j]);
                s_load += 0.5f * erfcf(-z * 0.70710678118654752440f);  // Phi(z)
                s_imp += g;
            }
        }
        red_i[threadIdx.x] = s_imp;
        red_l[threadIdx.x] = s_load;
        __syncthreads();
        if (tl == 0 && j < n) {
            float a = 0.0f, b = 0.0f;
            for (int q = 0; q < TL; ++q) { a += red_i[q * CW + cw]; b += red_l[q * CW + cw]; }
            part_imp[(int64_t)blockIdx.x * n + j] = a;
            part_load[(int64_t)blockIdx.x * n + j] = b;
        }
        __syncthreads();
    }
}

// Same sums with one warp per row and the lanes across the columns (n <= 32 * NV): all loads of a row are
// issued first, a lane accumulates its columns over the rows of its warp, the block's 8 warps are then added
// in order through shared memory.
template <int NV>
__global__ void __launch_bounds__(256) level_sums_rows_kernel(const int32_t *__restrict__ idx,
                                                              const float *__restrict__ gates,
                                                              const float *__restrict__ clean,
                                                              const float *__restrict__ raw,
                                                              const float *__restrict__ kth_vals, int64_t rows,
                                                              int32_t n, int32_t k, float *__restrict__ part_imp,
                                                              float *__restrict__ part_load) {
    __shared__ float red[2][8][32 * NV];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t per = (rows + gridDim.x - 1) / gridDim.x;
    const int64_t r0 = (int64_t)blockIdx.x * per, r1 = min(r0 + per, rows);
    float s_imp[NV], s_load[NV];
#pragma unroll
    for (int u = 0; u < NV; ++u) s_imp[u] = s_load[u] = 0.0f;
    for (int64_t t = r0 + w; t < r1; t += 8) {
        float cv[NV], rv[NV];
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int32_t j = lane + 32 * u;
            cv[u] = j < n ? clean[t * n + j] : 0.0f;
            rv[u] = j < n ? raw[t * n + j] : 0.0f;
        }
        // the row's kept experts: bit u of `kept` = this lane's column lane + 32 u is one of them (its gate goes to
        // the Importance sum); an expert id outside [0, n) belongs to no lane
        uint32_t kept = 0u;
        for (int s = 0; s < k; ++s) {
            const int32_t e = idx[t * k + s];
            const float g = gates[t * k + s];
            if ((e & 31) == lane && (uint32_t)e < (uint32_t)n) {
#pragma unroll
                for (int u = 0; u < NV; ++u)
                    if ((e >> 5) == u) { kept |= 1u << u; s_imp[u] += g; }
            }
        }
        const float thr_unsel = kth_vals[t * 2 + 0], thr_sel = kth_vals[t * 2 + 1];
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int32_t j = lane + 32 * u;
            if (j < n) {
                // (the quotient may be off by two units in the last place: 1e-7 of z, far below what Load is held to)
                const float z = __fdividef(cv[u] - (((kept >> u) & 1u) ? thr_sel : thr_unsel), softplus_f(rv[u]));
                s_load[u] += 0.5f * erfcf(-z * 0.70710678118654752440f);  // Phi(z)
            }
        }
    }
#pragma unroll
    for (int u = 0; u < NV; ++u) { red[0][w][lane + 32 * u] = s_imp[u]; red[1][w][lane + 32 * u] = s_load[u]; }
    __syncthreads();
    for (int32_t j = threadIdx.x; j < n; j += 256) {
        float a = 0.0f, b = 0.0f;
#pragma unroll
        for (int q = 0; q < 8; ++q) { a += red[0][q][j]; b += red[1][q][j]; }
        part_imp[(int64_t)blockIdx.x * n + j] = a;
        part_load[(int64_t)blockIdx.x * n + j] = b;
    }
}

// Importance / Load = the blocks' partial sums added in double. A block takes 32 columns; its eight warps each add an
// eighth of the chunks (in ascending order, eight loads in flight), the eight sums are then added in warp order.
__global__ void __launch_bounds__(256) level_reduce_kernel(const float *__restrict__ part_imp,
                                                           const float *__restrict__ part_load, int32_t chunks,
                                                           int32_t n, float *__restrict__ importance,
                                                           float *__restrict__ load) {
    __shared__ double red[2][8][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int32_t j = blockIdx.x * 32 + lane;
    const int32_t per = (chunks + 7) / 8, c0 = w * per, c1 = min(c0 + per, chunks);
    double a = 0.0, b = 0.0;
    if (j < n) {
        int32_t c = c0;
        for (; c + 8 <= c1; c += 8) {
            float pa[8], pb[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                pa[q] = part_imp[(int64_t)(c + q) * n + j];
                pb[q] = part_load[(int64_t)(c + q) * n + j];
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) { a += (double)pa[q]; b += (double)pb[q]; }
        }
        for (; c < c1; ++c) {
            a += (double)part_imp[(int64_t)c * n + j];
            b += (double)part_load[(int64_t)c * n + j];
        }
    }
    red[0][w][lane] = a;
    red[1][w][lane] = b;
    __syncthreads();
    if (w == 0 && j < n) {
        a = 0.0; b = 0.0;
#pragma unroll
        for (int q = 0; q < 8; ++q) { a += red[0][q][lane]; b += red[1][q][lane]; }
        if (importance) importance[j] = (float)a;
        if (load) load[j] = (float)b;
    }
}

int32_t launch_level_sums(const int32_t *idx, const float *gates, const float *clean, const float *raw,
                          const float *kth_vals, int64_t rows, int32_t n, int32_t k, float *importance_out,
                          float *load_out, float *scratch, cudaStream_t st) {
    if (rows == 0) {
        if (importance_out) MOE_CUDA(cudaMemsetAsync(importance_out, 0, sizeof(float) * n, st));
        if (load_out) MOE_CUDA(cudaMemsetAsync(load_out, 0, sizeof(float) * n, st));
        return MOE_OK;
    }
    const int32_t chunks = level_chunks(rows);
    int32_t CW = 1;
    while (CW < n && CW < 256) CW <<= 1;
    float *part_imp = scratch, *part_load = scratch + (int64_t)chunks * n;
    if (n <= 32) level_sums_rows_kernel<1><<<chunks, 256, 0, st>>>(idx, gates, clean, raw, kth_vals, rows, n, k, part_imp, part_load);
    else if (n <= 64) level_sums_rows_kernel<2><<<chunks, 256, 0, st>>>(idx, gates, clean, raw, kth_vals, rows, n, k, part_imp, part_load);
    else if (n <= 128) level_sums_rows_kernel<4><<<chunks, 256, 0, st>>>(idx, gates, clean, raw, kth_vals, rows, n, k, part_imp, part_load);
    else if (n <= 256) level_sums_rows_kernel<8><<<chunks, 256, 0, st>>>(idx, gates, clean, raw, kth_vals, rows, n, k, part_imp, part_load);
    else level_sums_kernel<<<chunks, 256, 0, st>>>(idx, gates, clean, raw, kth_vals, rows, n, k, CW, part_imp, part_load);
    MOE_LAUNCHED();
    level_reduce_kernel<<<(unsigned)cdiv(n, 32), 256, 0, st>>>(part_imp, part_load, chunks, n, importance_out,
                                                                 load_out);
    MOE_LAUNCHED();
    return MOE_OK;
}

// ---- CV^2 = population variance / mean^2, and its gradient 2/(m mu^2) ((v_i - mu) - Var/mu) ----
struct Moments { double mu, var; };

__device__ Moments block_moments(const float *v, int32_t m, double *sh) {
    double s = 0.0;
    for (int32_t i = threadIdx.x; i < m; i += blockDim.x) s += (double)v[i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int off = blockDim.x / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    const double mu = sh[0] / m;
    __syncthreads();
    double q = 0.0;
    for (int32_t i = threadIdx.x; i < m; i += blockDim.x) { double dv = (double)v[i] - mu; q += dv * dv; }
    sh[threadIdx.x] = q;
    __syncthreads();
    for (int off = blockDim.x / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) sh[threadIdx.x] += sh[threadIdx.x + off];
        __syncthreads();
    }
    Moments r;
    r.mu = mu;
    r.var = sh[0] / m;
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(256) cv2_kernel(const float *importance, int32_t n_imp, const float *load,
                                                  int32_t n_load, float w_imp, float w_load, float *losses) {
    __shared__ double sh[256];
    Moments a = block_moments(importance, n_imp, sh);
    Moments b = block_moments(load, n_load, sh);
    if (threadIdx.x == 0) {
        losses[0] = (float)((double)w_imp * a.var / (a.mu * a.mu));
        losses[1] = (float)((double)w_load * b.var / (b.mu * b.mu));
    }
}

int32_t launch_cv2(const float *importance, int32_t n_imp, const float *load, int32_t n_load, float w_imp,
                   float w_load, float *losses, cudaStream_t st) {
    cv2_kernel<<<1, 256, 0, st>>>(importance, n_imp, load, n_load, w_imp, w_load, losses);
    MOE_LAUNCHED();
    return MOE_OK;
}

// out[i] = scale * dCV^2/dv_i
__global__ void __launch_bounds__(256) cv2_grad_kernel(const float *v, int32_t m, float scale, float *out) {
    __shared__ double sh[256];
    Moments a = block_moments(v, m, sh);
    const double c = 2.0 / ((double)m * a.mu * a.mu);
    for (int32_t i = threadIdx.x; i < m; i += blockDim.x)
        out[i] = (float)((double)scale * c * (((double)v[i] - a.mu) - a.var / a.mu));
}

// dgates[p] += dimp[topk_idx[p]]; an expert id outside [0, n) adds nothing
__global__ void add_gathered_kernel(float *dgates, const int32_t *topk_idx, const float *dimp, int64_t R, int32_t n) {
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= R) return;
    const int32_t e = topk_idx[p];
    MOE_BOUNDS_NOTE((uint32_t)e < (uint32_t)n);
    if ((uint32_t)e < (uint32_t)n) dgates[p] += dimp[e];
}

int32_t launch_cv2_grad(const float *v, int32_t m, float scale, float *out, cudaStream_t st) {
    cv2_grad_kernel<<<1, 256, 0, st>>>(v, m, scale, out);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_add_gathered(float *dgates, const int32_t *topk_idx, const float *dimp, int64_t R, int32_t n,
                            cudaStream_t st) {
    if (R == 0) return MOE_OK;
    add_gathered_kernel<<<(unsigned)cdiv(R, 256), 256, 0, st>>>(dgates, topk_idx, dimp, R, n);
    MOE_LAUNCHED();
    return MOE_OK;
}

int32_t launch_losses_bwd_flat(const float *importance, const float *load, int32_t n, const int32_t *topk_idx,
                               int64_t R, float w_imp, float w_load, float *dgates, float *dload, float *dimp_tmp,
                               cudaStream_t st) {
    cv2_grad_kernel<<<1, 256, 0, st>>>(importance, n, w_imp, dimp_tmp);
    MOE_LAUNCHED();
    cv2_grad_kernel<<<1, 256, 0, st>>>(load, n, w_load, dload);
    MOE_LAUNCHED();
    if (R > 0) {
        add_gathered_kernel<<<(unsigned)cdiv(R, 256), 256, 0, st>>>(dgates, topk_idx, dimp_tmp, R, n);
        MOE_LAUNCHED();
    }
    return MOE_OK;
}

MOE_BOUNDS_READER(bounds_violations_losses)

}  // namespace moe
