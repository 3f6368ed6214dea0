// Optimiser step on the expert parameters (Appendix D, "Training", the memory optimisations): Adam with beta1 = 0
// (no first-moment estimate) whose second-moment matrix is replaced by a factored approximation: for every expert
// weight matrix only the running row-wise and column-wise averages of the squared gradient are kept, and the matrix of
// estimators is taken to be their outer product divided by the mean of the row vector. Biases (vectors) keep a full
// second-moment estimate. All of it is HBM streaming: the gradient is read twice (averages, update), the parameters
// are read and written once. Sums are taken in fixed orders (no floating-point atomics): two runs agree bit for bit.
#include "moe_internal.cuh"

namespace moe {

namespace {

constexpr int RB = 32;  // rows per block of the averaging pass

template <typename XT> struct Vec {
    static constexpr int N = 16 / sizeof(XT);
    uint4 raw;
    __device__ __forceinline__ float get(int i) const { return to_f32(reinterpret_cast<const XT *>(&raw)[i]); }
    __device__ __forceinline__ void set(int i, float v) { reinterpret_cast<XT *>(&raw)[i] = from_f32<XT>(v); }
};

// Row block rb of expert e: row_avg[e, row] <- beta2 * row_avg + (1 - beta2) * mean_j g^2 for its RB rows (complete rows),
// and colpart[e, rb, j] = sum over its rows of g[row, j]^2. grid (row blocks, experts); 32..256 threads, one 16-byte
// column vector per thread and pass (narrow matrices get narrower blocks, so that no thread idles).
template <typename XT>
__global__ void __launch_bounds__(256) adam_averages_kernel(const XT *__restrict__ g, int32_t rows, int32_t cols,
                                                            float beta2, float *__restrict__ row_avg,
                                                            float *__restrict__ colpart) {
    constexpr int VN = Vec<XT>::N;
    __shared__ float warp_rows[8][RB];
    const int32_t e = blockIdx.y, rb = blockIdx.x, nrb = gridDim.x;
    const int32_t row0 = rb * RB;
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const XT *G = g + (int64_t)e * rows * cols;
    float *cp = colpart + ((int64_t)e * nrb + rb) * cols;
    float rowacc[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) rowacc[r] = 0.0f;
    const int nvec = cols / VN;
    for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
        float colacc[VN];
#pragma unroll
        for (int i = 0; i < VN; ++i) colacc[i] = 0.0f;
#pragma unroll
        for (int r0 = 0; r0 < RB; r0 += 8) {  // eight independent 16-byte loads in flight per thread
            Vec<XT> in[8];
#pragma unroll
            for (int r = 0; r < 8; ++r)
                in[r].raw = row0 + r0 + r < rows ? reinterpret_cast<const uint4 *>(G + (int64_t)(row0 + r0 + r) * cols)[v]
                                                 : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                float s = 0.0f;
#pragma unroll
                for (int i = 0; i < VN; ++i) {
                    const float x = in[r].get(i), q = x * x;
                    colacc[i] += q;
                    s += q;
                }
                rowacc[r0 + r] += s;
            }
        }
#pragma unroll
        for (int i = 0; i < VN; ++i) cp[v * VN + i] = colacc[i];
    }
    // row sums: lanes by butterfly, then the block's warps in order
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        float s = rowacc[r];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) warp_rows[wp][r] = s;
    }
    __syncthreads();
    if (threadIdx.x < RB && row0 + threadIdx.x < rows) {
        float s = 0.0f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += warp_rows[w][threadIdx.x];
        float *ra = row_avg + (int64_t)e * rows + row0 + threadIdx.x;
        *ra = beta2 * *ra + (1.0f - beta2) * (s / (float)cols);
    }
}

// col_avg[e, j] <- beta2 * col_avg + (1 - beta2) * (sum of the row blocks' partial sums, in order) / rows for the 256
// columns of block (x, e); block x = 0 also forms row_mean[e], the mean over the rows of the (already updated) row averages.
__global__ void __launch_bounds__(256) adam_columns_kernel(const float *__restrict__ colpart, int32_t nrb, int32_t rows,
                                                           int32_t cols, float beta2, float *__restrict__ col_avg,
                                                           const float *__restrict__ row_avg,
                                                           float *__restrict__ row_mean) {
    __shared__ double part[256];
    const int32_t e = blockIdx.y;
    const int32_t j = blockIdx.x * 256 + threadIdx.x;
    if (j < cols) {
        const float *src = colpart + (int64_t)e * nrb * cols + j;
        double s = 0.0;
        int32_t rb = 0;
        for (; rb + 4 <= nrb; rb += 4) {  // four loads in flight, added in order
            const float a0 = src[(int64_t)rb * cols], a1 = src[(int64_t)(rb + 1) * cols];
            const float a2 = src[(int64_t)(rb + 2) * cols], a3 = src[(int64_t)(rb + 3) * cols];
            s += (double)a0; s += (double)a1; s += (double)a2; s += (double)a3;
        }
        for (; rb < nrb; ++rb) s += (double)src[(int64_t)rb * cols];
        float *ca = col_avg + (int64_t)e * cols + j;
        *ca = beta2 * *ca + (1.0f - beta2) * (float)(s / (double)rows);
    }
    if (blockIdx.x != 0) return;
    double s = 0.0;
    for (int32_t r = threadIdx.x; r < rows; r += 256) s += (double)row_avg[(int64_t)e * rows + r];
    part[threadIdx.x] = s;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) part[threadIdx.x] += part[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) row_mean[e] = (float)(part[0] / (double)rows);
}

// W[e, i, j] -= lr * g / (sqrt(row_avg_i * col_avg_j / row_mean / correction) + eps). grid (blocks of UR rows, experts);
// the block walks its rows' 16-byte vectors as one flat index space, four independent vectors per thread in flight.
constexpr int UR = 16;
__device__ __forceinline__ float sqrt_fast(float x) { return x > 0.0f ? x * rsqrtf(x) : 0.0f; }  // ~2 ulp, no IEEE sqrt sequence

template <typename XT>
__global__ void __launch_bounds__(256) adam_update_kernel(XT *__restrict__ W, const XT *__restrict__ g, int32_t rows,
                                                          int32_t cols, const float *__restrict__ row_avg,
                                                          const float *__restrict__ col_avg,
                                                          const float *__restrict__ row_mean, float lr,
                                                          float inv_correction, float eps) {
    constexpr int VN = Vec<XT>::N;
    const int32_t e = blockIdx.y;
    const float rm = row_mean[e];
    const float scale = rm > 0.0f ? inv_correction / rm : 0.0f;  // v_hat = row_avg_i * col_avg_j * scale
    const int nvec = cols / VN;
    const float *ca = col_avg + (int64_t)e * cols;
    const int32_t r0 = blockIdx.x * UR, nr = min(UR, rows - r0);
    const int64_t base = ((int64_t)e * rows + r0) * cols;
    const int total = nr * nvec;
    for (int i0 = threadIdx.x; i0 < total; i0 += 4 * 256) {
        Vec<XT> w[4], gr[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = i0 + u * 256;
            if (idx < total) {
                w[u].raw = reinterpret_cast<const uint4 *>(W + base)[idx];
                gr[u].raw = reinterpret_cast<const uint4 *>(g + base)[idx];
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = i0 + u * 256;
            if (idx >= total) break;
            const int r = idx / nvec, v = idx - r * nvec;
            const float rs = row_avg[(int64_t)e * rows + r0 + r] * scale;
#pragma unroll
            for (int i = 0; i < VN; ++i)
                w[u].set(i, w[u].get(i) - __fdividef(lr * gr[u].get(i), sqrt_fast(rs * ca[v * VN + i]) + eps));
            reinterpret_cast<uint4 *>(W + base)[idx] = w[u].raw;
        }
    }
}

// vectors (biases): full second-moment estimate
template <typename XT>
__global__ void __launch_bounds__(256) adam_vector_kernel(XT *__restrict__ b, const XT *__restrict__ g, int64_t count,
                                                          float *__restrict__ v, float lr, float beta2,
                                                          float inv_correction, float eps) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const float gi = to_f32(g[i]);
    const float vi = beta2 * v[i] + (1.0f - beta2) * gi * gi;
    v[i] = vi;
    b[i] = from_f32<XT>(to_f32(b[i]) - lr * gi / (sqrtf(vi * inv_correction) + eps));  // tiny tensor: exact operations
}

template <typename XT>
int32_t adam_matrix(XT *W, const XT *g, int32_t n, int32_t rows, int32_t cols, float *row_avg, float *col_avg, float lr,
                    float beta2, float inv_correction, float eps, float *colpart, float *row_mean, cudaStream_t st) {
    const int32_t nrb = (int32_t)cdiv(rows, RB);
    const int nvec = cols / (int)(16 / sizeof(XT));
    const unsigned threads = (unsigned)imin(256, cdiv(nvec, 32) * 32);
    adam_averages_kernel<XT><<<dim3((unsigned)nrb, (unsigned)n), threads, 0, st>>>(g, rows, cols, beta2, row_avg, colpart);
    MOE_LAUNCHED();
    adam_columns_kernel<<<dim3((unsigned)cdiv(cols, 256), (unsigned)n), 256, 0, st>>>(colpart, nrb, rows, cols, beta2, col_avg, row_avg,
                                                                                     row_mean);
    MOE_LAUNCHED();
    adam_update_kernel<XT><<<dim3((unsigned)cdiv(rows, UR), (unsigned)n), 256, 0, st>>>(W, g, rows, cols, row_avg, col_avg,
                                                                                       row_mean, lr, inv_correction, eps);
    MOE_LAUNCHED();
    return MOE_OK;
}

}  // namespace

int64_t adam_ws_floats(int32_t n, int32_t d, int32_t h) {
    const int64_t a = (int64_t)n * cdiv(d, RB) * h, b = (int64_t)n * cdiv(h, RB) * d;
    return (a > b ? a : b) + n + 64;
}

int32_t launch_expert_adam(int32_t act, int32_t n, int32_t d, int32_t h, void *W1, void *b1, void *W2, void *b2,
                           const void *dW1, const void *db1, const void *dW2, const void *db2, float *state, float lr,
                           float beta2, float eps, int32_t step, float *ws, cudaStream_t st) {
    // state: r1 [n,d], c1 [n,h], r2 [n,h], c2 [n,d], vb1 [n,h], vb2 [n,d]
    float *r1 = state, *c1 = r1 + (int64_t)n * d, *r2 = c1 + (int64_t)n * h, *c2 = r2 + (int64_t)n * h;
    float *vb1 = c2 + (int64_t)n * d, *vb2 = vb1 + (int64_t)n * h;
    float *row_mean = ws, *colpart = ws + ((n + 63) & ~63);
    const float inv_correction = (float)(1.0 / (1.0 - pow((double)beta2, (double)step)));
    const unsigned gb1 = (unsigned)cdiv((int64_t)n * h, 256), gb2 = (unsigned)cdiv((int64_t)n * d, 256);
    if (act == MOE_BF16) {
        MOE_TRY(adam_matrix<bf16>((bf16 *)W1, (const bf16 *)dW1, n, d, h, r1, c1, lr, beta2, inv_correction, eps, colpart, row_mean, st));
        MOE_TRY(adam_matrix<bf16>((bf16 *)W2, (const bf16 *)dW2, n, h, d, r2, c2, lr, beta2, inv_correction, eps, colpart, row_mean, st));
        adam_vector_kernel<bf16><<<gb1, 256, 0, st>>>((bf16 *)b1, (const bf16 *)db1, (int64_t)n * h, vb1, lr, beta2, inv_correction, eps);
        MOE_LAUNCHED();
        adam_vector_kernel<bf16><<<gb2, 256, 0, st>>>((bf16 *)b2, (const bf16 *)db2, (int64_t)n * d, vb2, lr, beta2, inv_correction, eps);
        MOE_LAUNCHED();
    } else {
        MOE_TRY(adam_matrix<float>((float *)W1, (const float *)dW1, n, d, h, r1, c1, lr, beta2, inv_correction, eps, colpart, row_mean, st));
        MOE_TRY(adam_matrix<float>((float *)W2, (const float *)dW2, n, h, d, r2, c2, lr, beta2, inv_correction, eps, colpart, row_mean, st));
        adam_vector_kernel<float><<<gb1, 256, 0, st>>>((float *)b1, (const float *)db1, (int64_t)n * h, vb1, lr, beta2, inv_correction, eps);
        MOE_LAUNCHED();
        adam_vector_kernel<float><<<gb2, 256, 0, st>>>((float *)b2, (const float *)db2, (int64_t)n * d, vb2, lr, beta2, inv_correction, eps);
        MOE_LAUNCHED();
    }
    return MOE_OK;
}

}  // namespace moe
