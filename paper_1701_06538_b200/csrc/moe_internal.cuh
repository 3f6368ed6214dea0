// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moe.h"

#define MOE_TRY(expr)                                \
    do {                                             \
        int32_t st_ = (expr);                        \
        if (st_ != MOE_OK) return st_;               \
    } while (0)

#define MOE_CUDA(expr)                               \
    do {                                             \
        if ((expr) != cudaSuccess) return MOE_ERR_CUDA; \
    } while (0)

#define MOE_LAUNCHED()                                           \
    do {                                                         \
        ::moe::count_launch();                                   \
        if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA; /* consumed: reported once */ \
    } while (0)

// Checking build (-DMOE_BOUNDS_CHECK, the stand-in for a memory checker): every place where a value read from memory
// becomes an index reports a value outside its range to a counter of the translation unit (never a trap; the access
// itself is skipped by the guards that are always compiled in). moe_debug_bounds_violations adds the counters up.
#ifdef MOE_BOUNDS_CHECK
static __device__ unsigned long long g_tu_bounds_violations = 0ull;
#define MOE_BOUNDS_NOTE(ok)                                                  \
    do {                                                                     \
        if (!(ok)) atomicAdd(&g_tu_bounds_violations, 1ull);                 \
    } while (0)
#define MOE_BOUNDS_READER(fn)                                                                                   \
    unsigned long long fn() {                                                                                   \
        unsigned long long v = 0;                                                                               \
        return cudaMemcpyFromSymbol(&v, g_tu_bounds_violations, sizeof(v)) == cudaSuccess ? v : ~0ull;          \
    }
#else
#define MOE_BOUNDS_NOTE(ok) do {} while (0)
#define MOE_BOUNDS_READER(fn) unsigned long long fn() { return 0ull; }
#endif

namespace moe {

void count_launch();  // diagnostics: kernels launched by this library so far (api.cu)
// per translation unit: out-of-range indices seen by the checking build (0 in the regular build)
unsigned long long bounds_violations_route();
unsigned long long bounds_violations_losses();
unsigned long long bounds_violations_hier();
unsigned long long bounds_violations_gate();
unsigned long long bounds_violations_ffn();

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

static inline size_t act_bytes(int32_t act) { return act == MOE_BF16 ? 2 : 4; }
static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int64_t imin(int64_t a, int64_t b) { return a < b ? a : b; }
static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31) == 0; }  // 32 bytes: the epilogues use 256-bit stores

// Carves 256-byte aligned pieces out of a workspace. With base == nullptr it only measures,
// so the size queries and the calls that use the workspace run the same code.
struct Carver {
    char *base;
    size_t off;
    explicit Carver(void *b) : base(static_cast<char *>(b)), off(0) {}
    template <typename T> T *take(int64_t count) {
        size_t bytes = (static_cast<size_t>(count < 0 ? 0 : count) * sizeof(T) + 255) & ~size_t(255);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += bytes;
        return p;
    }
    void *take_bytes(int64_t bytes) { return take<char>(bytes); }
};

// Every workspace begins with a 256-byte header; word 0 is the status word of bounded waits.
static const int64_t kWsHeader = 256;

// ----------------------------------------------------------------------------- gating (gate.cu)
// Projection clean = rows.W0, raw = rows.W1 with the fixed fused-multiply-add chain.
// Ungrouped: offsets == nullptr, rows are tokens 0..M-1, outputs [M, n0].
// Grouped (secondary gates): sorted row r belongs to segment e (offsets[e] <= r < offsets[e+1]),
// reads token perm[r] / kdiv, uses W0 + e*d*n0, and writes output row perm[r].
int32_t launch_projection(const void *x, int32_t act, int64_t M, int32_t d, int32_t n0, const float *W0,
                          const float *W1, float *out0, float *out1, const int32_t *offsets, int32_t nseg,
                          const int32_t *perm, int32_t kdiv, int32_t *tile_prefix, cudaStream_t st,
                          const int32_t *row_count = nullptr);
// Noisy logits, top-k, masked softmax for `rows` rows of n columns.
int32_t launch_gate_select(const float *clean, const float *raw, const float *noise, int64_t rows, int32_t n,
                           int32_t k, int32_t *idx, float *gates, float *kth_vals, int32_t *kth_idx,
                           cudaStream_t st, const int32_t *row_list = nullptr, const int32_t *row_count = nullptr,
                           const void *row_span = nullptr, const void *chain_list = nullptr);
// Tensor-core screening of the routing (see gate.cu): weights split / norms, then the screening select.
int32_t launch_gate_screen_prepare(const void *x, int32_t act, int64_t T, int32_t d, int32_t n, const float *Wg,
                                   const float *Wn, void *wsplit, float *wnorm, float *xnorm,
                                   int32_t *unsafe_count, float *wt /* [2n, d]: columns as rows */, cudaStream_t st,
                                   int32_t groups = 1, bool with_xnorm = true);
int32_t launch_gate_screen(const float *cr, const float *noise, const float *xnorm, const float *wnorm, int32_t d,
                           int64_t T, int32_t n, int32_t k, int32_t *idx, float *gates, float *clean, float *raw,
                           float *kth_vals, int32_t *kth_idx, int32_t *unsafe_list, float *unsafe_low,
                           int32_t *unsafe_count, void *chain_list, int32_t *full_list, cudaStream_t st,
                           const int32_t *perm, int32_t kdiv, const int32_t *group_of, void *unsafe_span);
// Rows the screen cannot certify: unsafe_list / unsafe_count[0] = rows whose selection is repeated (unsafe_low: the
// bound that picks their candidate columns); chain_list
// (int2 {row, column code}, unsafe_count[1] entries, at most 2 * SCREEN_MAX_CAND per row) = single fma chains to
// recompute; full_list / unsafe_count[2] = rows with more candidates than that, which take the whole projection.
constexpr int SCREEN_MAX_CAND = 16;
int32_t launch_gate_chains(const void *x, int32_t act, int32_t d, int32_t n, const float *Wt, const void *chain_list,
                           const int32_t *chain_count, float *clean, float *raw, cudaStream_t st,
                           int32_t kdiv = 1);  // Wt [2n, d] (per group); token = output row / kdiv
bool tc_gate_fwd_supported(int32_t act, int64_t T, int32_t d, int32_t n, int32_t flags);
// cr [T, 2n] (float) = x . [W_g | W_noise] from the three-term split wsplit [3, d, 2n]
int32_t launch_tc_gate_fwd(const void *x, int64_t T, int32_t d, int32_t n, const void *wsplit, float *cr,
                           int32_t *status, cudaStream_t st);
int32_t launch_hier_merge(int64_t T, int32_t k1, int32_t k2, int32_t b, const int32_t *idx_p, const float *g_p,
                          const int32_t *idx_s, const float *g_s, int32_t *topk_idx, float *gates,
                          cudaStream_t st);

// ----------------------------------------------------------------------------- routing (route.cu)
int64_t dispatch_ws_elems(int64_t R, int32_t n);  // int32 elements of scratch
int32_t launch_dispatch_index(const int32_t *topk_idx, int64_t R, int32_t n, int32_t *perm, int32_t *inv_perm,
                              int32_t *counts, int32_t *offsets, int32_t *scratch, cudaStream_t st);
int32_t launch_dispatch_rows(const void *x, int32_t act, int64_t T, int32_t k, int32_t d, const int32_t *inv_perm,
                             void *xs, cudaStream_t st);
// keep != nullptr: the layer epilogue of Appendix C (sigmoid, dropout through the packed keep bits [T, d/8] with the
// kept activations scaled by keep_scale = 1 / (1 - DropProb), residual xres added); see route.cu
int32_t launch_combine(const void *ys, int32_t act, const float *gates, const int32_t *inv_perm, int64_t T,
                       int32_t k, int32_t d, void *y, cudaStream_t st, const void *xres = nullptr,
                       const uint8_t *keep = nullptr, float keep_scale = 1.0f);
int32_t launch_combine_bwd(const void *dY, const void *ys, int32_t act, const float *gates,
                           const int32_t *inv_perm, int64_t T, int32_t k, int32_t d, float *dgates, void *dys,
                           cudaStream_t st, const uint8_t *keep = nullptr, float keep_scale = 1.0f);
// out_f32 = sum_s dxs[inv_perm[t*k+s]] (+ add_f32 if given); written as float or, if out_act
// is given instead, rounded to the act type.
int32_t launch_dispatch_bwd(const void *dxs, int32_t act, const int32_t *inv_perm, int64_t T, int32_t k,
                            int32_t d, const float *add_f32, float *out_f32, void *out_act, cudaStream_t st,
                            const void *add_act = nullptr);
// tile_prefix[e] = sum_{e' < e} ceil(count_e' / bm), e = 0..n
int32_t launch_tile_prefix(const int32_t *offsets, int32_t n, int32_t bm, int32_t *tile_prefix, cudaStream_t st);

// ----------------------------------------------------------------------------- losses (losses.cu)
int64_t losses_ws_floats(int64_t rows, int32_t n);
// Partial column sums over rows of the gate mass (importance) and of P(x, i) (load).
// flat / primary level: seg == nullptr. Secondary level: rows are slots p, grouped through
// perm/offsets (sorted row r -> slot perm[r]); sums are per segment: load_out [nseg, n].
int32_t launch_level_sums(const int32_t *idx, const float *gates, const float *clean, const float *raw,
                          const float *kth_vals, int64_t rows, int32_t n, int32_t k, float *importance_out,
                          float *load_out, float *scratch, cudaStream_t st);
int32_t launch_cv2(const float *importance, int32_t n_imp, const float *load, int32_t n_load, float w_imp,
                   float w_load, float *losses, cudaStream_t st);
int32_t launch_losses_bwd_flat(const float *importance, const float *load, int32_t n, const int32_t *topk_idx,
                               int64_t R, float w_imp, float w_load, float *dgates, float *dload, float *dimp_tmp,
                               cudaStream_t st);

// ----------------------------------------------------------------------------- hierarchical pieces (hier.cu)
int32_t launch_hier_split_idx(const int32_t *topk_idx, int64_t T, int32_t k1, int32_t k2, int32_t a, int32_t b,
                              int32_t *idx_p, int32_t *idx_s, cudaStream_t st);
int32_t launch_segment_sum(const float *vals, const int32_t *perm, const int32_t *offsets, int32_t nseg, float *out,
                           cudaStream_t st);
int64_t grouped_sums_ws_floats(int64_t rows, int32_t nseg, int32_t n);
int32_t launch_grouped_load(const int32_t *idx_s, const float *clean, const float *raw, const float *kth_vals,
                            const int32_t *perm, const int32_t *offsets, int32_t nseg, int64_t rows, int32_t n,
                            int32_t k, float *out, float *scratch, int32_t *tile_prefix, cudaStream_t st);
int32_t launch_load_h(float *load, const int32_t *counts_p, int32_t a, int32_t b, cudaStream_t st);
int32_t launch_load_h_bwd(const float *load, const float *dload_h, int32_t a, int32_t b, float *dload,
                          cudaStream_t st);
int32_t launch_hier_gate_product_bwd(const float *gates, float *dgates, int64_t T, int32_t k1, int32_t k2,
                                     cudaStream_t st);
int32_t launch_add_slot_rows(const float *dX_sec, int64_t T, int32_t k1, int32_t d, float *dX_gate, cudaStream_t st);
int32_t launch_cv2_grad(const float *v, int32_t m, float scale, float *out, cudaStream_t st);
int32_t launch_add_gathered(float *dgates, const int32_t *topk_idx, const float *dimp, int64_t R, int32_t n,
                            cudaStream_t st);

// ----------------------------------------------------------------------------- gate backward (gate_bwd.cu)
// dclean, draw [rows, n] from the saved gate tensors; dload_row_stride = 0 broadcasts dload [n].
int32_t launch_gate_logit_grads(const float *noise, const float *clean, const float *raw, const int32_t *idx,
                                const float *gates, const float *kth_vals, const int32_t *kth_idx,
                                const float *dgates, const float *dload, const int32_t *dload_row_group,
                                int64_t rows, int32_t n, int32_t k, float *dclean, float *draw, void *dsplit,
                                const int32_t *split_row_index, cudaStream_t st);

// ----------------------------------------------------------------------------- SIMT grouped GEMM (gemm_simt.cu)
enum GemmType { G_F32 = 0, G_BF16 = 1 };
struct SimtGemm {
    // C(i,j) = epilogue( sum_kk A(i,kk) * B(kk,j) ), element strides in elements.
    const void *A, *B;
    void *C;
    int32_t ta, tb, tc;  // GemmType of A, B, C
    int64_t sa_i, sa_k, sb_k, sb_j, sc_i, sc_j;
    // mode 0: output rows follow the segments (M_e = count_e, K fixed); A, C advance by rows,
    //         B by expert (b_e). mode 1: contraction over the segment rows (K_e = count_e);
    //         A, B advance by rows (their k index), C by expert (c_e).
    int32_t mode;
    const int32_t *offsets;  // nullptr: a single problem of M x N x K
    int32_t nseg;
    int64_t M, N, K;
    int64_t b_e, c_e;
    const void *bias;  // [nseg, N] of type tc, or nullptr
    int32_t relu;      // 1: max(.,0)
    const void *mask;  // mode 0: same shape/type as C; result multiplied by [mask > 0]
    int32_t accumulate;  // 1: C += (float C only)
    // optional row gathers through a permutation: mode 0: A row i reads row a_row_index[i] / a_row_div
    // and C row i is written at c_row_index[i]; mode 1: the contraction index r reads A row
    // a_row_index[r] / a_row_div and B row b_row_index[r].
    const int32_t *a_row_index;
    int32_t a_row_div;
    const int32_t *b_row_index;
    const int32_t *c_row_index;
};
int32_t launch_simt_gemm(const SimtGemm &g, int32_t *tile_prefix, cudaStream_t st);
// out[e, j] = sum over the rows of segment e of in[r, j]   (out, in of the act type)
int64_t colsum_ws_floats(int64_t R, int32_t n, int32_t N);
int32_t launch_segment_colsum(const void *in, int32_t act, const int32_t *offsets, int32_t nseg, int64_t R,
                              int32_t N, void *out, float *scratch, int32_t *tile_prefix, cudaStream_t st);

// ----------------------------------------------------------------------------- tensor-core experts (ffn_tc.cu)
bool tc_ffn_supported(const moe_config &c);
int64_t tc_ffn_ws_bytes(const moe_config &c);
// first_only: only hid = relu(xs.W1 + b1) (the recomputation of the hidden activations in the backward pass)
int32_t launch_tc_ffn(const moe_config &c, const void *xs, const int32_t *offsets, const void *W1, const void *b1,
                      const void *W2, const void *b2, void *hid, void *ys, void *ws, int32_t *status_word,
                      cudaStream_t st, bool first_only = false, uint32_t *relu_bits = nullptr);
// relu_bits [R, h / 32]: one bit per hidden activation (set where hid > 0), written by the first expert GEMM if given;
// the backward then masks dz with these bits instead of reading hid again as a mask (16 times less traffic)

// ----------------------------------------------------------------------------- strictly balanced gating (balanced.cu)
int32_t launch_exclusive_scan(const int32_t *counts, int32_t n, int32_t *out, cudaStream_t st,
                              int32_t *tile_sums = nullptr /* cdiv(n + 1, 4096) ints: long inputs in parallel */);  // route.cu
int64_t balanced_ws_bytes(int64_t T, int32_t n);
int32_t launch_balanced_gate(const void *x, int32_t act, int64_t T, int32_t d, int32_t n, int32_t k, const float *Wg,
                             const float *thr, float *logits, float *probs, uint32_t *mask_bits, int32_t *tok_of_row,
                             int32_t *offsets, float *den, int32_t *tok_ptr, int32_t *tok_rows, float *loss,
                             int32_t *thr_counts, void *ws, cudaStream_t st);
int32_t launch_balanced_gather(const void *x, int32_t act, const int32_t *tok_of_row, int64_t R, int64_t T, int32_t d,
                               void *xs, cudaStream_t st);
int32_t launch_balanced_combine(const void *ys, int32_t act, const float *p, const float *den, const int32_t *tok_ptr,
                                const int32_t *tok_rows, int64_t T, int64_t R, int32_t n, int32_t m, int32_t d, void *y,
                                cudaStream_t st);
int32_t launch_balanced_combine_bwd(const void *dY, const void *ys, int32_t act, const float *p, const float *den,
                                    const int32_t *tok_of_row, int64_t R, int64_t T, int32_t n, int32_t m, int32_t d,
                                    float *dG_row, void *dys, cudaStream_t st);
// dc [T, n] float, or (dsplit given) its three-term bf16 split [T, 3n] = (hi | mid | lo) for the tensor-core contractions
int32_t launch_balanced_gate_bwd(const float *p, const uint32_t *mask_bits, const float *den, const float *thr,
                                 const int32_t *tok_ptr, const int32_t *tok_rows, const float *dG_row,
                                 const int32_t *thr_counts, float w, int64_t T, int32_t n, int32_t m, float *dc,
                                 void *dsplit, float *dthr, cudaStream_t st);
int32_t launch_balanced_dispatch_bwd(const void *dxs, int32_t act, const int32_t *tok_ptr, const int32_t *tok_rows,
                                     const float *dX_gate, int64_t T, int64_t R, int32_t d, void *dX, cudaStream_t st);

int32_t launch_debug_wait(int32_t *status, unsigned long long limit_ns, cudaStream_t st);

// ----------------------------------------------------------------------------- optimiser step (optim.cu)
int64_t adam_ws_floats(int32_t n, int32_t d, int32_t h);
int32_t launch_expert_adam(int32_t act, int32_t n, int32_t d, int32_t h, void *W1, void *b1, void *W2, void *b2,
                           const void *dW1, const void *db1, const void *dW2, const void *db2, float *state, float lr,
                           float beta2, float eps, int32_t step, float *ws, cudaStream_t st);

bool tc_gate_bwd_supported(int32_t act, int32_t d, int32_t n);
int64_t tc_gate_bwd_partials(int64_t T, int32_t d, int32_t n);  // floats of partial-sum scratch
int32_t launch_tc_gate_bwd(const void *x, int64_t T, int32_t d, int32_t n, const float *Wg, const float *Wn,
                           const void *dsplit, void *wsplit, float *partials, float *dWg, float *dWn,
                           float *dX_gate, int32_t *status, cudaStream_t st, int32_t flags, int32_t ldw = 0);
// (ldw > 0: Wg / Wn, dWg / dWn are the left and right column halves of one [d, 2n] matrix with row stride ldw)
int32_t launch_tc_gate_fwd_grouped(const void *xs_p, int64_t P1, int32_t d, int32_t a, int32_t b, const void *wsplit_s,
                                   const int32_t *offsets_p, int32_t *tile_prefix, float *cr_s, int32_t *status,
                                   cudaStream_t st, int32_t flags);
bool tc_hier_gate_bwd_supported(int32_t act, int32_t d, int32_t a, int32_t b);
int32_t launch_tc_hier_secondary_bwd(const void *xs_p, const void *dsplit_s, void *wsplit_s, const float *Wg_s,
                                     const float *Wn_s, const int32_t *offsets_p, int32_t *tile_prefix, int32_t a,
                                     int64_t P1, int32_t d, int32_t b, float *partials, float *dWg_s, float *dWn_s,
                                     float *dX_sec, int32_t *status, cudaStream_t st);
int64_t tc_tile_ws_ints(int64_t R, int64_t nseg);  // int32s of a [nseg + 1] tile prefix followed by its tile table
int64_t tc_colsum_part_floats(int64_t R, int32_t nseg, int32_t N);  // scratch of the fused bias-gradient sums
int32_t launch_tc_ffn_bwd(const moe_config &c, const void *xs, const void *hid, const void *dys,
                          const int32_t *offsets, const void *W1, const void *W2, void *dxs, void *dW1, void *db1,
                          void *dW2, void *db2, void *dz, float *colsum, int32_t *tile_prefix, int32_t *status_word,
                          cudaStream_t st, const uint32_t *relu_bits = nullptr);

}  // namespace moe
