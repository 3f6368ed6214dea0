// Two-level hierarchical mixture of experts (Appendix B, Eq. 12-14): the pieces that differ from
// the flat layer. Rows of the secondary level are the slots p = t*k1 + s1 (token t, primary slot s1).
#include "moe_internal.cuh"

namespace moe {

// idx_p[t, s1] = group of primary slot s1; idx_s[p, s2] = expert inside that group
__global__ void hier_split_idx_kernel(const int32_t *__restrict__ topk_idx, int64_t total, int32_t k2, int32_t a,
                                      int32_t b, int32_t *__restrict__ idx_p, int32_t *__restrict__ idx_s) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // over T*k1*k2
    if (i >= total) return;
    int32_t id = topk_idx[i];
    MOE_BOUNDS_NOTE((uint32_t)id < (uint32_t)(a * b));
    if ((uint32_t)id >= (uint32_t)(a * b)) id = 0;  // a caller's bad id: the group index below stays inside its tables
    idx_s[i] = id % b;
    if (i % k2 == 0) idx_p[i / k2] = id / b;
}

int32_t launch_hier_split_idx(const int32_t *topk_idx, int64_t T, int32_t k1, int32_t k2, int32_t a, int32_t b,
                              int32_t *idx_p, int32_t *idx_s, cudaStream_t st) {
    const int64_t total = T * k1 * k2;
    if (total == 0) return MOE_OK;
    hier_split_idx_kernel<<<(unsigned)cdiv(total, 256), 256, 0, st>>>(topk_idx, total, k2, a, b, idx_p, idx_s);
    MOE_LAUNCHED();
    return MOE_OK;
}

// out[e] = sum over the sorted rows r of segment e of vals[perm[r]]   (Importance_H, Eq. 13)
__global__ void __launch_bounds__(256) segment_sum_kernel(const float *__restrict__ vals,
                                                          const int32_t *__restrict__ perm,
                                                          const int32_t *__restrict__ offsets, int32_t nseg,
                                                          float *__restrict__ out) {
    const int lane = threadIdx.x & 31;
    const int32_t e = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (e >= nseg) return;
    double s = 0.0;
    for (int32_t r = offsets[e] + lane; r < offsets[e + 1]; r += 32) s += (double)vals[perm[r]];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) out[e] = (float)s;
}

int32_t launch_segment_sum(const float *vals, const int32_t *perm, const int32_t *offsets, int32_t nseg, float *out,
                           cudaStream_t st) {
    segment_sum_kernel<<<(unsigned)cdiv(nseg, 8), 256, 0, st>>>(vals, perm, offsets, nseg, out);
    MOE_LAUNCHED();
    return MOE_OK;
}

// Load_i(X^(i))_j = sum over the slots of group i of P(x, j) for that group's secondary gate (Eq. 10
// inside Eq. 14). Tiles of GS_ROWS sorted rows (one group each) give partial column sums; an ordered
// pass adds the tiles of each group.
constexpr int GS_ROWS = 64;
int64_t grouped_sums_ws_floats(int64_t rows, int32_t nseg, int32_t n) { return (cdiv(rows, GS_ROWS) + nseg) * (int64_t)n + 64; }

__device__ __forceinline__ float softplus_g(float r) { return fmaxf(r, 0.0f) + log1pf(expf(-fabsf(r))); }

__global__ void __launch_bounds__(256) grouped_load_partial_kernel(
    const int32_t *__restrict__ idx_s, const float *__restrict__ clean, const float *__restrict__ raw,
    const float *__restrict__ kth_vals, const int32_t *__restrict__ perm, const int32_t *__restrict__ offsets,
    const int32_t *__restrict__ tile_prefix, int32_t nseg, int32_t n, int32_t k, int32_t CW, float *__restrict__ part) {
    __shared__ float red[256];
    const int32_t b = blockIdx.x;
    if (b >= tile_prefix[nseg]) return;
    int lo = 0, hi = nseg;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tile_prefix[mid] <= b) lo = mid; else hi = mid;
    }
    const int32_t r0 = offsets[lo] + (b - tile_prefix[lo]) * GS_ROWS;
    const int32_t r1 = min(r0 + GS_ROWS, offsets[lo + 1]);
    const int cw = threadIdx.x % CW, tl = threadIdx.x / CW, TL = 256 / CW;
    for (int32_t jb = 0; jb < n; jb += CW) {
        const int32_t j = jb + cw;
        float s = 0.0f;
        if (j < n) {
            for (int32_t r = r0 + tl; r < r1; r += TL) {
                const int64_t p = perm[r];
                bool sel = false;
                for (int q = 0; q < k; ++q) sel |= idx_s[p * k + q] == j;
                const float z = (clean[p * n + j] - kth_vals[p * 2 + (sel ? 1 : 0)]) / softplus_g(raw[p * n + j]);
                s += 0.5f * erfcf(-z * 0.70710678118654752440f);
            }
        }
        red[threadIdx.x] = s;
        __syncthreads();
        if (tl == 0 && j < n) {
            float a = 0.0f;
            for (int q = 0; q < TL; ++q) a += red[q * CW + cw];
            part[(int64_t)b * n + j] = a;
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) grouped_reduce_kernel(const float *__restrict__ part,
                                                             const int32_t *__restrict__ tile_prefix, int32_t n,
                                                             float *__restrict__ out) {
    const int32_t e = blockIdx.x;
    const int32_t j = blockIdx.y * 256 + threadIdx.x;
    if (j >= n) return;
    double s = 0.0;
    for (int32_t b = tile_prefix[e]; b < tile_prefix[e + 1]; ++b) s += (double)part[(int64_t)b * n + j];
    out[(int64_t)e * n + j] = (float)s;
}

int32_t launch_grouped_load(const int32_t *idx_s, const float *clean, const float *raw, const float *kth_vals,
                            const int32_t *perm, const int32_t *offsets, int32_t nseg, int64_t rows, int32_t n,
                            int32_t k, float *out, float *scratch, int32_t *tile_prefix, cudaStream_t st) {
    MOE_TRY(launch_tile_prefix(offsets, nseg, GS_ROWS, tile_prefix, st));
    int32_t CW = 1;
    while (CW < n && CW < 256) CW <<= 1;
    grouped_load_partial_kernel<<<(unsigned)(cdiv(rows, GS_ROWS) + nseg), 256, 0, st>>>(
        idx_s, clean, raw, kth_vals, perm, offsets, tile_prefix, nseg, n, k, CW, scratch);
    MOE_LAUNCHED();
    grouped_reduce_kernel<<<dim3((unsigned)nseg, (unsigned)cdiv(n, 256)), 256, 0, st>>>(scratch, tile_prefix, n, out);
    MOE_LAUNCHED();
    return MOE_OK;
}

// Load_H[i,j] = Load_primary[i] * Load_i[j] / |X^(i)|  (Eq. 14); a group nobody selected gets 0.
// load layout: [a*b] Load_H | [a] Load_primary | [a*b] Load_i | [a] |X^(i)|
__global__ void load_h_kernel(float *__restrict__ load, const int32_t *__restrict__ counts_p, int32_t a, int32_t b) {
    const int32_t i = blockIdx.x;
    const float *load_p = load + (int64_t)a * b, *load_s = load_p + a;
    float *cnt = load + 2 * (int64_t)a * b + a;
    const int32_t c = counts_p[i];
    for (int32_t j = threadIdx.x; j < b; j += blockDim.x)
        load[(int64_t)i * b + j] = c > 0 ? load_p[i] * load_s[(int64_t)i * b + j] / (float)c : 0.0f;
    if (threadIdx.x == 0) cnt[i] = (float)c;
}

int32_t launch_load_h(float *load, const int32_t *counts_p, int32_t a, int32_t b, cudaStream_t st) {
    load_h_kernel<<<a, 128, 0, st>>>(load, counts_p, a, b);
    MOE_LAUNCHED();
    return MOE_OK;
}

// dLoad_primary[i] = sum_j dLoad_H[i,j] Load_i[j] / |X^(i)| ; dLoad_i[j] = dLoad_H[i,j] Load_primary[i] / |X^(i)|
// dload layout: [a] | [a*b]
__global__ void __launch_bounds__(128) load_h_bwd_kernel(const float *__restrict__ load,
                                                         const float *__restrict__ dload_h, int32_t a, int32_t b,
                                                         float *__restrict__ dload) {
    __shared__ double red[128];
    const int32_t i = blockIdx.x;
    const float *load_p = load + (int64_t)a * b, *load_s = load_p + a, *cnt = load + 2 * (int64_t)a * b + a;
    const float c = cnt[i];
    double s = 0.0;
    for (int32_t j = threadIdx.x; j < b; j += blockDim.x) {
        const float g = dload_h[(int64_t)i * b + j];
        dload[a + (int64_t)i * b + j] = c > 0.0f ? g * load_p[i] / c : 0.0f;
        if (c > 0.0f) s += (double)g * (double)load_s[(int64_t)i * b + j] / (double)c;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int off = 64; off > 0; off >>= 1) {
        if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) dload[i] = (float)red[0];
}

int32_t launch_load_h_bwd(const float *load, const float *dload_h, int32_t a, int32_t b, float *dload,
                          cudaStream_t st) {
    load_h_bwd_kernel<<<a, 128, 0, st>>>(load, dload_h, a, b, dload);
    MOE_LAUNCHED();
    return MOE_OK;
}

// Product rule of Eq. 12: w = g_p * g_s  =>  dg_s = dw * g_p,  dg_p = sum_s2 dw * g_s
// gates / dgates layout: [T, k] product | [T, k1] primary | [T, k1, k2] secondary
__global__ void hier_gate_product_bwd_kernel(const float *__restrict__ gates, float *__restrict__ dgates, int64_t P1,
                                             int32_t k2, int64_t Tk) {
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // slot (t, s1)
    if (p >= P1) return;
    const float *g_p = gates + Tk, *g_s = g_p + P1;
    float *dg_p = dgates + Tk, *dg_s = dg_p + P1;
    float acc = 0.0f;
    for (int s2 = 0; s2 < k2; ++s2) {
        const float dw = dgates[p * k2 + s2];
        dg_s[p * k2 + s2] = dw * g_p[p];
        acc = fmaf(dw, g_s[p * k2 + s2], acc);
    }
    dg_p[p] = acc;
}

int32_t launch_hier_gate_product_bwd(const float *gates, float *dgates, int64_t T, int32_t k1, int32_t k2,
                                     cudaStream_t st) {
    const int64_t P1 = T * k1;
    if (P1 == 0) return MOE_OK;
    hier_gate_product_bwd_kernel<<<(unsigned)cdiv(P1, 256), 256, 0, st>>>(gates, dgates, P1, k2, T * k1 * k2);
    MOE_LAUNCHED();
    return MOE_OK;
}

// dX_gate[t] += sum_s1 dX_sec[t*k1 + s1]   (both float, [.., d])
__global__ void add_slot_rows_kernel(const float *__restrict__ dX_sec, int64_t total, int32_t k1, int32_t d,
                                     float *__restrict__ dX_gate) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // over T*d
    if (i >= total) return;
    const int64_t t = i / d, q = i % d;
    float acc = dX_gate[i];
    for (int s1 = 0; s1 < k1; ++s1) acc += dX_sec[(t * k1 + s1) * d + q];
    dX_gate[i] = acc;
}

int32_t launch_add_slot_rows(const float *dX_sec, int64_t T, int32_t k1, int32_t d, float *dX_gate, cudaStream_t st) {
    const int64_t total = T * d;
    if (total == 0) return MOE_OK;
    add_slot_rows_kernel<<<(unsigned)cdiv(total, 256), 256, 0, st>>>(dX_sec, total, k1, d, dX_gate);
    MOE_LAUNCHED();
    return MOE_OK;
}

MOE_BOUNDS_READER(bounds_violations_hier)

}  // namespace moe
