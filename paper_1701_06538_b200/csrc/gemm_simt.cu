// Generic strided SIMT grouped GEMM in float accumulation. It serves the all-float32 layer
// (where the 1e-5 tolerance rules out tensor-core formats), shapes the tensor-core kernels do
// not take, and the two dense contractions of the gate backward. 64x64 tile, BK = 16, 4x4 per thread.
#include "moe_internal.cuh"

namespace moe {

constexpr int SBM = 64, SBN = 64, SBK = 16;

template <typename T> __device__ __forceinline__ float ld_as_f32(const void *p, int64_t i) {
    return to_f32(reinterpret_cast<const T *>(p)[i]);
}

template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256) simt_gemm_kernel(SimtGemm g, const int32_t *__restrict__ tile_prefix) {
    __shared__ float As[SBK][SBM + 1];
    __shared__ float Bs[SBK][SBN + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

    int64_t m0, m_end, kbeg, kend;
    int32_t e = 0;
    if (g.mode == 0) {
        if (g.offsets) {
            const int32_t b = blockIdx.x;
            if (b >= tile_prefix[g.nseg]) return;
            int lo = 0, hi = g.nseg;
            while (hi - lo > 1) {
                int mid = (lo + hi) >> 1;
                if (tile_prefix[mid] <= b) lo = mid; else hi = mid;
            }
            e = lo;
            m0 = g.offsets[e] + (int64_t)(b - tile_prefix[e]) * SBM;
            m_end = g.offsets[e + 1];
        } else {
            m0 = (int64_t)blockIdx.x * SBM;
            m_end = g.M;
        }
        kbeg = 0;
        kend = g.K;
    } else {
        e = blockIdx.z;
        m0 = (int64_t)blockIdx.x * SBM;
        m_end = g.M;
        kbeg = g.offsets ? g.offsets[e] : 0;
        kend = g.offsets ? g.offsets[e + 1] : g.K;
    }
    const int64_t n0 = (int64_t)blockIdx.y * SBN;
    const int64_t b_off = g.mode == 0 ? (int64_t)e * g.b_e : 0;
    const int64_t c_off = g.mode == 1 ? (int64_t)e * g.c_e : 0;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    const bool a_k_fast = g.sa_k == 1, b_j_fast = g.sb_j == 1;
    for (int64_t k0 = kbeg; k0 < kend; k0 += SBK) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int el = tid + q * 256;
            int i, kk;
            if (a_k_fast) { kk = el % SBK; i = el / SBK; } else { i = el % SBM; kk = el / SBM; }
            float v = 0.0f;
            if (m0 + i < m_end && k0 + kk < kend) {
                int64_t ri = m0 + i, rk = k0 + kk;
                if (g.a_row_index) {
                    if (g.mode == 0) ri = g.a_row_index[ri] / g.a_row_div;
                    else rk = g.a_row_index[rk] / g.a_row_div;
                }
                v = ld_as_f32<TA>(g.A, ri * g.sa_i + rk * g.sa_k);
            }
            As[kk][i] = v;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int el = tid + q * 256;
            int j, kk;
            if (b_j_fast) { j = el % SBN; kk = el / SBN; } else { kk = el % SBK; j = el / SBK; }
            float v = 0.0f;
            if (n0 + j < g.N && k0 + kk < kend) {
                int64_t rk = k0 + kk;
                if (g.mode == 1 && g.b_row_index) rk = g.b_row_index[rk];
                v = ld_as_f32<TB>(g.B, b_off + rk * g.sb_k + (n0 + j) * g.sb_j);
            }
            Bs[kk][j] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < SBK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t r = m0 + ty * 4 + i;
        if (r >= m_end) continue;
        const int64_t cr = (g.mode == 0 && g.c_row_index) ? g.c_row_index[r] : r;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t col = n0 + tx * 4 + j;
            if (col >= g.N) continue;
            float v = acc[i][j];
            if (g.bias) v += ld_as_f32<TC>(g.bias, (int64_t)e * g.N + col);
            if (g.relu) v = fmaxf(v, 0.0f);
            const int64_t at = c_off + cr * g.sc_i + col * g.sc_j;
            if (g.mask && !(ld_as_f32<TC>(g.mask, at) > 0.0f)) v = 0.0f;
            TC *C = reinterpret_cast<TC *>(g.C);
            if (g.accumulate) v += to_f32(C[at]);
            C[at] = from_f32<TC>(v);
        }
    }
}

int32_t launch_simt_gemm(const SimtGemm &g, int32_t *tile_prefix, cudaStream_t st) {
    dim3 grid;
    if (g.mode == 0) {
        if (g.M == 0) return MOE_OK;
        int64_t tiles = cdiv(g.M, SBM);
        if (g.offsets) {
            MOE_TRY(launch_tile_prefix(g.offsets, g.nseg, SBM, tile_prefix, st));
            tiles += g.nseg;
        }
        grid = dim3((unsigned)tiles, (unsigned)cdiv(g.N, SBN), 1);
    } else {
        grid = dim3((unsigned)cdiv(g.M, SBM), (unsigned)cdiv(g.N, SBN), (unsigned)(g.offsets ? g.nseg : 1));
    }
    if (grid.y > 65535 || grid.z > 65535) return MOE_ERR_UNSUPPORTED;
    if (g.ta == G_F32 && g.tb == G_F32 && g.tc == G_F32)
        simt_gemm_kernel<float, float, float><<<grid, 256, 0, st>>>(g, tile_prefix);
    else if (g.ta == G_BF16 && g.tb == G_BF16 && g.tc == G_BF16)
        simt_gemm_kernel<bf16, bf16, bf16><<<grid, 256, 0, st>>>(g, tile_prefix);
    else if (g.ta == G_BF16 && g.tb == G_F32 && g.tc == G_F32)
        simt_gemm_kernel<bf16, float, float><<<grid, 256, 0, st>>>(g, tile_prefix);
    else
        return MOE_ERR_UNSUPPORTED;
    MOE_LAUNCHED();
    return MOE_OK;
}

// ------------------------------------------------------------------------------------------
// Column sums per segment (bias gradients): partial sums over tiles of 128 rows, then an ordered
// pass over each segment's tiles. Deterministic.
// ------------------------------------------------------------------------------------------
constexpr int CS_ROWS = 128;
int64_t colsum_ws_floats(int64_t R, int32_t n, int32_t N) { return (cdiv(R, CS_ROWS) + n) * (int64_t)N + 64; }

// One block per 128-row tile and per slab of 32 * V columns (V = elements of a 16-byte vector): lane l owns V adjacent
// columns, warp w the tile's rows w, w + 8, ..., read with 16-byte loads, four rows in flight; the eight warps' sums are
// added in warp order.
template <typename XT>
__global__ void __launch_bounds__(256) colsum_partial_kernel(const XT *__restrict__ in,
                                                             const int32_t *__restrict__ offsets, int32_t nseg,
                                                             int32_t N, const int32_t *__restrict__ tile_prefix,
                                                             float *__restrict__ part) {
    constexpr int V = 16 / sizeof(XT);
    __shared__ float sh[8][32 * V];
    const int32_t b = blockIdx.x;
    if (b >= tile_prefix[nseg]) return;
    int lo = 0, hi = nseg;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (tile_prefix[mid] <= b) lo = mid; else hi = mid;
    }
    const int64_t r0 = offsets[lo] + (int64_t)(b - tile_prefix[lo]) * CS_ROWS;
    const int64_t r1 = min(r0 + (int64_t)CS_ROWS, (int64_t)offsets[lo + 1]);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int32_t j = (blockIdx.y * 32 + lane) * V;
    float s[V];
#pragma unroll
    for (int u = 0; u < V; ++u) s[u] = 0.0f;
    if (j + V <= N) {  // N is a multiple of V wherever rows are 16-byte aligned
        int64_t r = r0 + w;
        for (; r + 24 < r1; r += 32) {
            uint4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = *reinterpret_cast<const uint4 *>(in + (r + 8 * q) * N + j);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const XT *e = reinterpret_cast<const XT *>(&v[q]);
#pragma unroll
                for (int u = 0; u < V; ++u) s[u] += to_f32(e[u]);
            }
        }
        for (; r < r1; r += 8) {
            const uint4 v = *reinterpret_cast<const uint4 *>(in + r * N + j);
            const XT *e = reinterpret_cast<const XT *>(&v);
#pragma unroll
            for (int u = 0; u < V; ++u) s[u] += to_f32(e[u]);
        }
    }
#pragma unroll
    for (int u = 0; u < V; ++u) sh[w][lane * V + u] = s[u];
    __syncthreads();
    for (int c = threadIdx.x; c < 32 * V; c += 256) {
        const int32_t col = blockIdx.y * 32 * V + c;
        if (col < N) {
            float t = sh[0][c];
#pragma unroll
            for (int q = 1; q < 8; ++q) t += sh[q][c];
            part[(int64_t)b * N + col] = t;
        }
    }
}

// Sum of a segment's tile sums: a block takes 32 columns, its eight warps the tiles b0 + w, b0 + w + 8, ... (eight loads in
// flight: the largest expert of a skewed batch has hundreds of tiles), the eight sums are added in warp order.
template <typename XT>
__global__ void __launch_bounds__(256) colsum_final_kernel(const float *__restrict__ part, int32_t N,
                                                           const int32_t *__restrict__ tile_prefix,
                                                           XT *__restrict__ out) {
    __shared__ float sh[8][32];
    const int32_t e = blockIdx.x, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int32_t j = blockIdx.y * 32 + lane;
    const int32_t b1 = tile_prefix[e + 1];
    float s = 0.0f;
    if (j < N) {
        int32_t b = tile_prefix[e] + w;
        for (; b + 8 * 7 < b1; b += 64) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = part[(int64_t)(b + 8 * u) * N + j];
#pragma unroll
            for (int u = 0; u < 8; ++u) s += v[u];
        }
        for (; b < b1; b += 8) s += part[(int64_t)b * N + j];
    }
    sh[w][lane] = s;
    __syncthreads();
    if (w == 0 && j < N) {
        float t = sh[0][lane];
#pragma unroll
        for (int u = 1; u < 8; ++u) t += sh[u][lane];
        out[(int64_t)e * N + j] = from_f32<XT>(t);
    }
}

int32_t launch_segment_colsum(const void *in, int32_t act, const int32_t *offsets, int32_t nseg, int64_t R,
                              int32_t N, void *out, float *scratch, int32_t *tile_prefix, cudaStream_t st) {
    MOE_TRY(launch_tile_prefix(offsets, nseg, CS_ROWS, tile_prefix, st));
    const int vcols = act == MOE_BF16 ? 256 : 128;  // columns per block of the partial sums: 32 lanes x one 16-byte vector
    dim3 g1((unsigned)(cdiv(R, CS_ROWS) + nseg), (unsigned)cdiv(N, vcols));
    dim3 g2((unsigned)nseg, (unsigned)cdiv(N, 32));
    if (act == MOE_BF16) {
        colsum_partial_kernel<bf16><<<g1, 256, 0, st>>>((const bf16 *)in, offsets, nseg, N, tile_prefix, scratch);
        MOE_LAUNCHED();
        colsum_final_kernel<bf16><<<g2, 256, 0, st>>>(scratch, N, tile_prefix, (bf16 *)out);
    } else {
        colsum_partial_kernel<float><<<g1, 256, 0, st>>>((const float *)in, offsets, nseg, N, tile_prefix, scratch);
        MOE_LAUNCHED();
        colsum_final_kernel<float><<<g2, 256, 0, st>>>(scratch, N, tile_prefix, (float *)out);
    }
    MOE_LAUNCHED();
    return MOE_OK;
}

}  // namespace moe
