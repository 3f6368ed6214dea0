/*
 * moe.h -- C ABI of the B200 (sm_100a) hot path of the Sparsely-Gated Mixture-of-Experts layer
 * (Shazeer et al., 2017): noisy top-k gating, dispatch, one-hidden-layer ReLU experts,
 * gate-weighted combine, Importance / Load balancing losses, and their backward passes.
 *
 * Conventions, valid for every call unless a comment says otherwise
 * -----------------------------------------------------------------
 *  - Every pointer is a DEVICE pointer except `const moe_config*`, `moe_sizes*`,
 *    `moe_ctx_layout*` and pointers whose name starts with `host_`.
 *  - The caller owns every buffer (inputs, outputs, workspace, context). The library never
 *    allocates or frees device memory and never synchronises the host with the device (except
 *    moe_check_status and moe_debug_bounds_violations, which say so). It keeps no state between
 *    calls, with three small exceptions: a host-side launch counter (diagnostics), function
 *    attributes set on a kernel's first launch, and moe_dispatch_noalloc (see there: a fixed
 *    scratch array inside the library's device image and its cached address). All work is enqueued
 *    on `stream` (a cudaStream_t passed as void*; NULL is the default stream).
 *  - `ws` and `ctx` are bare pointers: a buffer that is too small cannot be detected by the call it
 *    is passed to. moe_query_sizes gives the sizes, moe_check_buffer_sizes checks one.
 *  - Tensors are row-major, contiguous, and start on a 32-byte boundary (256-byte for the
 *    workspace and the context). Outputs are overwritten, not accumulated into.
 *  - "act" tensors (x, xs, hid, ys, y, W1, b1, W2, b2 and their gradients) have the element
 *    type moe_config.act (float or bfloat16). Gating tensors (W_g, W_noise, noise, clean,
 *    raw_noise, gates, importance, load, losses and their gradients) are always float.
 *    Index tensors are int32.
 *  - Every function returns a moe_status; nothing is launched when it is not MOE_OK. Argument
 *    and shape errors are reported, never faulted on. Nothing is printed.
 *  - Notation: T tokens, d model width, h expert hidden width, n experts, k experts per token,
 *    R = T*k dispatched rows. A "slot" is p = t*k + s, the s-th kept expert of token t.
 *
 * Hierarchical layer (Appendix B; moe_config.a > 0): a groups with top-k1, b experts per group
 * with top-k2; n = a*b, k = k1*k2, flat expert id i*b + j, slot order primary-slot major.
 * Every gating tensor is then its primary part followed by its secondary part:
 *     Wg, Wnoise   : [d, a]  then [a, d, b]
 *     noise, clean, raw_noise : [T, a] then [T, k1, b]   (secondary indexed by PRIMARY SLOT)
 *     kth_vals, kth_idx       : [T, 2] then [T, k1, 2]
 *     gates        : [T, k] products, then [T, k1] primary gates, then [T, k1, k2] secondary gates
 *     topk_idx     : [T, k] flat expert ids (group = id / b, expert in group = id % b)
 *     importance   : [a*b]
 *     load         : [a*b] Load_H, then [a] primary Load, [a,b] per-group Load_i(X^(i)), [a] |X^(i)|
 *     dload        : [a] d/d(primary Load), then [a,b] d/d(per-group Load)
 * moe_query_sizes gives the element counts.
 *
 * Every call only enqueues work on the given stream: no host synchronisation, no allocation, no device-to-host read.
 * After one eager call per process and device (function attributes are set on first use) the calls may be recorded
 * in a CUDA graph by stream capture.
 */
#ifndef MOE_B200_H
#define MOE_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MOE_OK = 0,
    MOE_ERR_INVALID_ARG = 1, /* NULL pointer, misaligned pointer, inconsistent or non-positive size */
    MOE_ERR_UNSUPPORTED = 2, /* valid in the method but outside what this build implements          */
    MOE_ERR_WORKSPACE = 3,   /* the problem does not fit a fixed-size scratch (moe_dispatch_noalloc)  */
    MOE_ERR_CUDA = 4,        /* a CUDA runtime call or a launch failed                              */
    MOE_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (see moe_check_status)           */
} moe_status;

typedef enum { MOE_F32 = 0, MOE_BF16 = 1 } moe_dtype;

#define MOE_MAX_K 8          /* k, k1, k2 and k1*k2 are at most this                 */
#define MOE_MAX_EXPERTS 8192 /* n (flat) and a, b (hierarchical levels) are at most this */
#define MOE_MAX_FLAT_EXPERTS 12288 /* hierarchical: a*b beyond this is MOE_ERR_UNSUPPORTED (one int32 per expert in shared memory) */

typedef struct moe_config {
    int32_t T, d, h;            /* tokens, model width, expert hidden width                              */
    int32_t n, k;               /* experts, experts per token (hierarchical: n = a*b, k = k1*k2)         */
    int32_t a, k1, b, k2;       /* hierarchical levels; a = 0 selects the flat layer (k1, b, k2 ignored) */
    int32_t act;                /* moe_dtype of the "act" tensors                                        */
    float w_importance, w_load; /* scale factors of Eq. 7 and Eq. 11                                     */
    int32_t flags;              /* 0, or an OR of the MOE_FLAG_* switches below                          */
} moe_config;

/* Switches in moe_config.flags (0 = the library chooses by problem size):
 *   MOE_FLAG_GATE_SCREEN_OFF  every token's routing logits through the fixed fma chain (no tensor-core screen)
 *   MOE_FLAG_GATE_SCREEN_ON   screen the routing on the tensor cores whenever the shapes allow, however small
 *   MOE_FLAG_TC_ONE_CTA       one-CTA tensor-core GEMM kernels everywhere (no SM pairs), for A/B comparisons */
#define MOE_FLAG_GATE_SCREEN_OFF 1
#define MOE_FLAG_GATE_SCREEN_ON 2
#define MOE_FLAG_TC_ONE_CTA 4
/*   MOE_FLAG_RECOMPUTE_HID    the hidden activations of the experts are not kept between moe_forward and
 *                             moe_backward (Appendix D, memory optimisations): the context has no `hid`
 *                             (moe_ctx_layout.hid is then meaningless, the context R*h elements smaller), the
 *                             backward runs the first expert GEMM again (2*R*d*h extra flop) into its workspace */
#define MOE_FLAG_RECOMPUTE_HID 8

typedef struct moe_sizes {
    int64_t R;            /* T*k                                                                    */
    int64_t gate_cols;    /* gating columns per token: n (flat) or a + k1*b (hierarchical)          */
    int64_t logits_elems; /* elements of noise, clean, raw_noise: T*gate_cols                       */
    int64_t gates_elems;  /* elements of gates (and dgates): flat T*k, hierarchical T*(2k + k1)     */
    int64_t kth_elems;    /* elements of kth_vals, kth_idx: flat 2T, hierarchical 2T(1 + k1)        */
    int64_t wg_elems;     /* elements of Wg (and of Wnoise): flat d*n, hierarchical d*a + a*d*b     */
    int64_t load_elems;   /* elements of load: flat n, hierarchical 2ab + 2a                        */
    int64_t dload_elems;  /* elements of dload: flat n, hierarchical a + ab                         */
    int64_t ws_bytes;     /* workspace every stage call accepts (the largest any stage needs)       */
    int64_t ws_fwd_bytes; /* workspace of moe_forward                                               */
    int64_t ws_bwd_bytes; /* workspace of moe_backward                                              */
    int64_t ctx_bytes;    /* context written by moe_forward and read by moe_backward                */
    int64_t adam_state_elems; /* floats of optimiser state of moe_expert_adam_factored: n * (3d + 3h)   */
    int64_t ws_adam_bytes;    /* workspace of moe_expert_adam_factored                                  */
} moe_sizes;

/* Byte offsets, inside the context of moe_forward, of the tensors it saves (same layouts as
 * the stage calls). Lets a caller inspect intermediate results of the fused call. */
typedef struct moe_ctx_layout {
    int64_t topk_idx, gates, clean, raw_noise, kth_vals, kth_idx; /* moe_gate outputs     */
    int64_t xs, perm, inv_perm, counts, offsets;                  /* moe_dispatch outputs */
    int64_t hid, ys;                                              /* moe_expert_ffn outputs */
    int64_t importance, load, losses;                             /* moe_losses outputs   */
    int64_t relu_bits; /* bf16 layers on the tensor cores that keep hid: [R, h/32] uint32, bit set where hid > 0 (the
                          backward's ReLU mask, read instead of hid); absent otherwise */
} moe_ctx_layout;

/* Checks a configuration: positive sizes, 1 <= k <= min(n, MOE_MAX_K), n <= MOE_MAX_EXPERTS,
 * rows of x / hid a multiple of 16 bytes, hierarchical fields consistent (n = a*b, k = k1*k2). */
int32_t moe_validate(const moe_config *cfg);
int32_t moe_query_sizes(const moe_config *cfg, moe_sizes *host_out);
/* The two workspace sizes alone (bytes a forward / a backward call needs in `ws`), for callers that do not want
 * the whole moe_sizes record. Host pointers; either may be NULL. */
int32_t moe_workspace_bytes(const moe_config *cfg, size_t *host_fwd, size_t *host_bwd);
int32_t moe_query_ctx_layout(const moe_config *cfg, moe_ctx_layout *host_out);
const char *moe_status_string(int32_t status);

/* Diagnostics only: number of kernels this library has launched in this process so far
 * (a host-side counter; the one piece of process-wide state the library keeps). */
int64_t moe_debug_launch_count(void);

/* Is a buffer of `bytes` bytes large enough for its role with this configuration? MOE_OK, or MOE_ERR_WORKSPACE.
 * The calls themselves take `ws` / `ctx` as bare pointers and cannot see a short buffer: check here first. */
typedef enum {
    MOE_BUF_WS_STAGE = 0,    /* ws of any stage call (moe_sizes.ws_bytes)     */
    MOE_BUF_WS_FORWARD = 1,  /* ws of moe_forward / moe_layer_forward         */
    MOE_BUF_WS_BACKWARD = 2, /* ws of moe_backward / moe_layer_backward       */
    MOE_BUF_CONTEXT = 3,     /* ctx of the fused calls                        */
    MOE_BUF_WS_ADAM = 4      /* ws of moe_expert_adam_factored                */
} moe_buffer_role;
int32_t moe_check_buffer_sizes(const moe_config *cfg, int32_t which, size_t bytes);

/* Diagnostics: enqueues a one-thread kernel that waits, with the bounded-wait helper of the tensor-core kernels, for
 * limit_ns nanoseconds (at most 1e8) on a barrier nobody signals, gives up, and leaves MOE_ERR_TIMEOUT in the status
 * word of `ws` (read it with moe_check_status). Nothing else is outstanding in that kernel: it returns normally and the
 * context stays usable. Exists so that the expiry path can be tested without starving a real kernel. */
int32_t moe_debug_wait_timeout(void *ws, int64_t limit_ns, void *stream);

/* Diagnostics: in the checking build of the library (compiled with -DMOE_BOUNDS_CHECK) the number of values read
 * from memory that were about to be used as an index outside their range, over all kernels so far (such accesses are
 * skipped in every build; the checking build also counts them). Always 0 in the regular build; -1 on a CUDA error.
 * Synchronises the device. */
int64_t moe_debug_bounds_violations(void);

/* Synchronises `stream`, then reads the status word the kernels of the last call that used
 * `ws` left there. MOE_OK, or MOE_ERR_TIMEOUT if a bounded wait inside a tensor-core kernel
 * gave up (its outputs are then undefined; the context stays usable). */
int32_t moe_check_status(const void *ws, void *stream);

/* ------------------------------------------------------------------------------------------
 * Forward stages
 * ------------------------------------------------------------------------------------------ */

/* Noisy top-k gating (Section 2.1, Eq. 3-5):
 *   clean = x.W_g, raw_noise = x.W_noise, H = clean + noise * softplus(raw_noise),
 *   topk_idx = the k largest H of each token in descending order (lowest index wins ties),
 *   gates = softmax over those k values (all other gate values are exactly 0 and not stored),
 *   kth_vals/kth_idx[t] = value/index of the k-th and (k+1)-th largest H (the latter is
 *   (-inf, -1) when k = n); they are what Eq. 9's kth_excluding needs.
 * The logits that decide the routing are evaluated in single precision in one fixed order
 * (one fused-multiply-add chain per output over ascending input feature; softplus in double
 * rounded once; H by one fused multiply-add), so the routing is reproducible bit for bit.
 * For large bf16 batches the routing (of the flat gate and of both levels of the hierarchical one)
 * is first screened with a tensor-core product and an error bound; tokens whose order the bound
 * proves keep that result (indices identical to the chain's, clean / raw_noise / kth_vals within
 * 1e-7 of it). For every other token the columns that can still reach rank k+1 are re-evaluated
 * with the chain and the selection is repeated, so its indices are the chain's too; its other
 * columns keep the tensor-core values.
 * moe_config.flags: MOE_FLAG_GATE_SCREEN_OFF disables the screen, MOE_FLAG_GATE_SCREEN_ON uses it whenever the
 * shapes allow; by default it is used when the projection has at least 1e9 multiply-adds.
 * `noise` is an input: standard normal draws, or zeros for noiseless gating.
 * in : x [T,d] act, Wg/Wnoise [d,n], noise [T,n]
 * out: topk_idx [T,k], gates [T,k], clean [T,n], raw_noise [T,n], kth_vals [T,2], kth_idx [T,2] */
int32_t moe_gate(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise, const float *noise,
                 int32_t *topk_idx, float *gates, float *clean, float *raw_noise, float *kth_vals,
                 int32_t *kth_idx, void *ws, void *stream);

/* Dispatch (Section 3.1: each expert receives the batch of the examples that selected it):
 * stable counting sort of the slots by expert.
 * out: counts [n]; offsets [n+1] exclusive prefix sum, offsets[n] = R; perm [R] slot of sorted
 *      row r; inv_perm [R] sorted row of slot p; xs [R,d] act, xs[r] = x[perm[r] / k]. */
int32_t moe_dispatch(const moe_config *cfg, const void *x, const int32_t *topk_idx, void *xs, int32_t *perm,
                     int32_t *inv_perm, int32_t *counts, int32_t *offsets, void *ws, void *stream);

/* Dispatch without a workspace. (The paper has no counterpart: this entry point exists for the
 * integration, not for the method.) Same inputs, outputs and results as moe_dispatch, but it takes
 * no `ws`: its scratch is a fixed array of MOE_NOALLOC_SCRATCH_INTS int32 (4 MiB + 256 B) inside
 * the library's device image, held by every GPU that loads the library until the process exits.
 * It is meant for callers that cannot obtain device memory of their own at the point of the call
 * -- code running inside a host framework's memory plan or a real-time loop where cudaMalloc (a
 * device-wide synchronising call) is forbidden, or plug-ins handed fixed input/output buffers and
 * nothing else. The call itself allocates and frees nothing, on the device or through any library.
 *  - Limit: ceil(T*k / 1024) * n + 64 <= MOE_NOALLOC_SCRATCH_INTS, else MOE_ERR_WORKSPACE is
 *    returned and nothing is launched (e.g. T*k = 262144 rows with up to 4096 experts fit).
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and keeps it; make that first call before starting any stream capture. The kept
 *    address belongs to the device's primary context: after a cudaDeviceReset of that device it
 *    is stale and this entry point must not be called again in the process.
 *  - All calls in the process share the array, which keeps whatever the last call left there
 *    (the kernels overwrite every word before reading it, so nothing needs clearing). Two
 *    calls that overlap on the GPU -- different streams, or different host threads -- race on
 *    it: serialise them. */
#define MOE_NOALLOC_SCRATCH_INTS ((1 << 20) + 64)
int32_t moe_dispatch_noalloc(const moe_config *cfg, const void *x, const int32_t *topk_idx, void *xs,
                             int32_t *perm, int32_t *inv_perm, int32_t *counts, int32_t *offsets, void *stream);

/* Experts (Section 3.2, Appendix C): on the rows offsets[e] <= r < offsets[e+1],
 *   hid = relu(xs.W1[e] + b1[e]),  ys = hid.W2[e] + b2[e],
 * float accumulation, one rounding to the act type at hid and at ys.
 * in : xs [R,d], offsets [n+1], W1 [n,d,h], b1 [n,h], W2 [n,h,d], b2 [n,d]   out: hid [R,h], ys [R,d]
 * With MOE_FLAG_RECOMPUTE_HID `hid` may be NULL: the hidden activations then stay in the workspace. */
int32_t moe_expert_ffn(const moe_config *cfg, const void *xs, const int32_t *offsets, const void *W1,
                       const void *b1, const void *W2, const void *b2, void *hid, void *ys, void *ws,
                       void *stream);

/* The same two calls with the ReLU mask as bits (bf16 layers whose widths are multiples of 64; MOE_ERR_UNSUPPORTED
 * otherwise): moe_expert_ffn_bits also writes relu_bits [R, h/32] uint32 (bit j of word c of a row: hid[row, 32c+j] > 0),
 * and moe_expert_ffn_bwd_bits masks dz with those bits instead of reading hid a second time as a mask (R*h/8 bytes
 * instead of 2*R*h). Same results bit for bit. This is the path the fused calls take (moe_ctx_layout.relu_bits). */
int32_t moe_expert_ffn_bits(const moe_config *cfg, const void *xs, const int32_t *offsets, const void *W1,
                            const void *b1, const void *W2, const void *b2, void *hid, void *ys, uint32_t *relu_bits,
                            void *ws, void *stream);
int32_t moe_expert_ffn_bwd_bits(const moe_config *cfg, const void *xs, const void *hid, const uint32_t *relu_bits,
                                const void *dys, const int32_t *offsets, const void *W1, const void *W2, void *dxs,
                                void *dW1, void *db1, void *dW2, void *db2, void *ws, void *stream);

/* Combine (Eq. 1): y[t] = sum_s gates[t,s] * ys[inv_perm[t*k+s]], float sum in slot order.
 * `gates` is the [T,k] (product) gate tensor.   out: y [T,d] act */
int32_t moe_combine(const moe_config *cfg, const void *ys, const float *gates, const int32_t *inv_perm, void *y,
                    void *stream);

/* Balancing losses (Section 4, Appendix A; hierarchical: Appendix B, Eq. 13-14):
 *   importance = batch sum of the gate vectors (Eq. 6); load_i = sum_t Phi((clean_i - thr_i) /
 *   softplus(raw_noise_i)) with thr = (k+1)-th largest H for a kept expert, k-th otherwise (Eq. 9-10);
 *   losses = { w_importance * CV^2(importance), w_load * CV^2(load) } with the population variance.
 * out: importance [n], load [moe_sizes.load_elems], losses [2] */
int32_t moe_losses(const moe_config *cfg, const int32_t *topk_idx, const float *gates, const float *clean,
                   const float *raw_noise, const float *kth_vals, float *importance, float *load, float *losses,
                   void *ws, void *stream);

/* ------------------------------------------------------------------------------------------
 * Backward stages (Section 2.1, "Training the Gating Network": plain back-propagation)
 * ------------------------------------------------------------------------------------------ */

/* Adjoint of Eq. 1. in: dY [T,d] act, ys, gates [T,k], inv_perm
 * out: dgates [T,k] = <dY[t], ys[row]>,  dys [R,d] act = gates[t,s] * dY[t] */
int32_t moe_combine_bwd(const moe_config *cfg, const void *dY, const void *ys, const float *gates,
                        const int32_t *inv_perm, float *dgates, void *dys, void *stream);

/* Back-propagation through the experts (ReLU derivative 0 at 0):
 *   db2 = sum dys, dW2 = hid^T.dys, dz = (dys.W2^T) * [hid > 0] (rounded to act), db1 = sum dz,
 *   dW1 = xs^T.dz, dxs = dz.W1^T; experts with no rows get zero gradients.
 * out: dxs [R,d], dW1 [n,d,h], db1 [n,h], dW2 [n,h,d], db2 [n,d] (all act); dz lives in ws. */
int32_t moe_expert_ffn_bwd(const moe_config *cfg, const void *xs, const void *hid, const void *dys,
                           const int32_t *offsets, const void *W1, const void *W2, void *dxs, void *dW1,
                           void *db1, void *dW2, void *db2, void *ws, void *stream);

/* Adjoint of the dispatch copies: dX_expert[t] = sum_s dxs[inv_perm[t*k+s]].  out: [T,d] float */
int32_t moe_dispatch_bwd(const moe_config *cfg, const void *dxs, const int32_t *inv_perm, float *dX_expert,
                         void *stream);

/* Gradient of the two losses (upstream gradient 1) w.r.t. importance and load (Eq. 7, 11):
 *   dgates[t,s] += w_importance * dCV^2/dimportance[topk_idx[t,s]]   (in-out: the [T,k] product part)
 *   dload[i]     = w_load * dCV^2/dload[i]                          (out: [moe_sizes.dload_elems])   */
int32_t moe_losses_bwd(const moe_config *cfg, const float *importance, const float *load,
                       const int32_t *topk_idx, float *dgates, float *dload, void *ws, void *stream);

/* Back-propagation through the gating network: softmax over the kept slots, the normal-CDF
 * load estimator including its threshold (another expert's noisy logit), softplus, and the two
 * projections. dgates is d(loss)/d(gates) [T,k] product part (the other parts are scratch for
 * the hierarchical layer); dload [n] is d(loss)/d(load).
 * out: dWg, dWnoise (layout of Wg), dX_gate [T,d] float */
int32_t moe_gate_bwd(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise,
                     const float *noise, const float *clean, const float *raw_noise, const int32_t *topk_idx,
                     const float *gates, const float *kth_vals, const int32_t *kth_idx, float *dgates,
                     const float *dload, float *dWg, float *dWnoise, float *dX_gate,
                     void *ws, void *stream);

/* ------------------------------------------------------------------------------------------
 * Fused layer
 * ------------------------------------------------------------------------------------------ */

/* gate -> dispatch -> experts -> combine -> losses. Saves what the backward needs in `ctx`
 * (moe_sizes.ctx_bytes, layout from moe_query_ctx_layout).
 * out: y [T,d] act, losses [2], importance [n], load [n], counts [n] */
int32_t moe_forward(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise, const float *noise,
                    const void *W1, const void *b1, const void *W2, const void *b2, void *y, float *losses,
                    float *importance, float *load, int32_t *counts, void *ctx, void *ws, void *stream);

/* Backward of moe_forward for upstream dY plus both balancing losses with upstream gradient 1
 * (they are added to the model's loss, Section 4).
 * out: dX [T,d] act, dWg, dWnoise (float, layout of Wg), dW1, db1, dW2, db2 (act) */
int32_t moe_backward(const moe_config *cfg, const void *dY, const void *x, const float *Wg, const float *Wnoise,
                     const float *noise, const void *W1, const void *b1, const void *W2, const void *b2,
                     const void *ctx, void *dX, float *dWg, float *dWnoise, void *dW1, void *db1, void *dW2,
                     void *db2, void *ws, void *stream);

/* ------------------------------------------------------------------------------------------
 * Strictly balanced gating (Appendix F, Eq. 15-20), flat layers, training time: every expert receives exactly
 * m = k*T/n examples (k*T must be a multiple of n).
 *   probs  = Softmax(x.W_g)                                        (Eq. 15; logits by the fixed fma chain of moe_gate)
 *   mask   = for every expert the m largest probs of its column over the batch, equal values to the
 *            lower token                                           (Eq. 18, batchwise mask)
 *   G      = probs * mask / sum_j probs_j * mask_j                 (Eq. 16; an example nobody keeps gets G = 0, y = 0)
 *   loss   = sum (M_threshold - M_batchwise) * (probs - thresholds) with M_threshold = [probs > thresholds] (Eq. 19-20)
 * An example is kept by a variable number of experts, so the routing tables are by sorted row: rows are
 * expert-major (expert e owns rows e*m .. e*m+m-1, in token order), tok_of_row [R] is each row's token,
 * offsets [n+1] = e*m (for moe_expert_ffn / moe_expert_ffn_bwd, which run unchanged on these uniform segments),
 * and tok_ptr [T+1] / tok_rows [R] list every token's rows in ascending expert order. The gate of a row is
 * probs[token, expert] / den[token]. mask_bits [T, mask_words] uint32 holds the mask (bit e%32 of word e/32).
 * Routing by the threshold mask alone (inference without a batch) is not built; the mask enters the loss, and
 * thr_counts [n] = how many examples each expert's threshold would keep.
 * Sizes: moe_query_balanced_sizes. The backward treats the mask as a constant; L_batchwise enters scaled by
 * w_batchwise and reaches probs and the thresholds.
 * ------------------------------------------------------------------------------------------ */
typedef struct moe_balanced_sizes {
    int64_t m;          /* examples per expert: k*T/n                              */
    int64_t R;          /* sorted rows: n*m = k*T                                  */
    int64_t mask_words; /* uint32 words per token of mask_bits: ceil(n/32)         */
    int64_t ws_bytes;   /* workspace of moe_gate_balanced / moe_gate_balanced_bwd  */
} moe_balanced_sizes;
int32_t moe_query_balanced_sizes(const moe_config *cfg, moe_balanced_sizes *host_out);

/* in : x [T,d] act, Wg [d,n], thresholds [n]
 * out: logits, probs [T,n]; mask_bits [T,mask_words]; tok_of_row [R]; offsets [n+1]; den [T]; tok_ptr [T+1];
 *      tok_rows [R]; loss_batchwise [1]; thr_counts [n] */
int32_t moe_gate_balanced(const moe_config *cfg, const void *x, const float *Wg, const float *thresholds, float *logits,
                          float *probs, uint32_t *mask_bits, int32_t *tok_of_row, int32_t *offsets, float *den,
                          int32_t *tok_ptr, int32_t *tok_rows, float *loss_batchwise, int32_t *thr_counts, void *ws,
                          void *stream);
/* xs [R,d] act: xs[r] = x[tok_of_row[r]] */
int32_t moe_dispatch_balanced(const moe_config *cfg, const void *x, const int32_t *tok_of_row, void *xs, void *stream);
/* y[t] = sum over the rows of token t of G * ys[row], ascending expert (Eq. 1)   out: y [T,d] act */
int32_t moe_combine_balanced(const moe_config *cfg, const void *ys, const float *probs, const float *den,
                             const int32_t *tok_ptr, const int32_t *tok_rows, void *y, void *stream);
/* out: dG_row [R] = <dY[token], ys[row]>, dys [R,d] act = G * dY[token] */
int32_t moe_combine_balanced_bwd(const moe_config *cfg, const void *dY, const void *ys, const float *probs,
                                 const float *den, const int32_t *tok_of_row, float *dG_row, void *dys, void *stream);
/* out: dWg [d,n], dX_gate [T,d] float, dthresholds [n] */
int32_t moe_gate_balanced_bwd(const moe_config *cfg, const void *x, const float *Wg, const float *probs,
                              const uint32_t *mask_bits, const float *den, const float *thresholds,
                              const int32_t *tok_ptr, const int32_t *tok_rows, const float *dG_row,
                              const int32_t *thr_counts, float w_batchwise, float *dWg, float *dX_gate,
                              float *dthresholds, void *ws, void *stream);
/* dX [T,d] act = sum over the rows of token t of dxs[row] + dX_gate[t] */
int32_t moe_dispatch_balanced_bwd(const moe_config *cfg, const void *dxs, const int32_t *tok_ptr,
                                  const int32_t *tok_rows, const float *dX_gate, void *dX, void *stream);

/* ------------------------------------------------------------------------------------------
 * Optimiser step on the expert parameters (Appendix D, "Training": the memory optimisations): Adam with
 * beta1 = 0 (no first-moment estimate) and a factored second-moment estimate. For each expert weight matrix
 * only the running averages (decay beta2) of the row-wise and of the column-wise means of the squared
 * gradient are kept; the matrix of estimators is their outer product divided by the mean of the row vector.
 * Adam's bias correction 1 - beta2^step and its epsilon outside the square root are kept:
 *     W -= lr * g / (sqrt(row_i * col_j / mean(row) / (1 - beta2^step)) + eps)
 * The biases (vectors) keep a full second-moment estimate. Parameters are updated IN PLACE (one rounding to
 * the act type). `state` (moe_sizes.adam_state_elems floats, zero before the first step) holds, in this
 * order: row [n,d] and column [n,h] averages of W1, row [n,h] and column [n,d] averages of W2, second moments
 * of b1 [n,h] and b2 [n,d]. step >= 1 counts the calls. ws: moe_sizes.ws_adam_bytes.
 * ------------------------------------------------------------------------------------------ */
int32_t moe_expert_adam_factored(const moe_config *cfg, void *W1, void *b1, void *W2, void *b2, const void *dW1,
                                 const void *db1, const void *dW2, const void *db2, float *state, float lr,
                                 float beta2, float eps, int32_t step, void *ws, void *stream);

/* ------------------------------------------------------------------------------------------
 * The layer inside the paper's models (Appendix C, "Model Architecture" and "MoE Layer Architecture"):
 * the MoE output goes through a sigmoid, then dropout (each activation dropped with probability
 * drop_prob, the kept ones divided by 1 - drop_prob), then the layer's input is added (residual):
 *     out[t] = x[t] + keep[t] * sigmoid(y[t]) / (1 - drop_prob),   y[t] = sum_s gates[t,s] * ys[row(t,s)]  (Eq. 1)
 * fused into the combine kernels, so y makes no round trip through memory (it is never stored; the
 * backward recomputes it from the ys rows it gathers anyway).
 * keep_bits [T, d/8] uint8 is the dropout mask, an INPUT drawn by the caller like the gating noise:
 * bit (q % 8) of byte q / 8 of a token's row is 1 where column q is kept. Needs d % 8 == 0 and
 * 0 <= drop_prob < 1 (MOE_ERR_INVALID_ARG otherwise).
 * ------------------------------------------------------------------------------------------ */

/* Combine with the layer epilogue.   in: ys, gates [T,k], inv_perm, x [T,d] act   out: out [T,d] act */
int32_t moe_combine_layer(const moe_config *cfg, const void *ys, const float *gates, const int32_t *inv_perm,
                          const void *x, const uint8_t *keep_bits, float drop_prob, void *out, void *stream);

/* Its adjoint: dy = dOut * keep / (1 - drop_prob) * s (1 - s) with s = sigmoid(y), then as moe_combine_bwd:
 * dgates [T,k] = <dy[t], ys[row]>, dys [R,d] act = gates[t,s] * dy[t]. The gradient through the residual
 * connection is dOut itself: the caller adds it to dX (moe_layer_backward does). */
int32_t moe_combine_layer_bwd(const moe_config *cfg, const void *dOut, const void *ys, const float *gates,
                              const int32_t *inv_perm, const uint8_t *keep_bits, float drop_prob, float *dgates,
                              void *dys, void *stream);

/* moe_forward / moe_backward with the layer epilogue: `out` replaces y, dOut replaces dY, and dX also
 * receives dOut through the residual connection. Same context and workspaces as the plain calls. */
int32_t moe_layer_forward(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise,
                          const float *noise, const void *W1, const void *b1, const void *W2, const void *b2,
                          const uint8_t *keep_bits, float drop_prob, void *out, float *losses, float *importance,
                          float *load, int32_t *counts, void *ctx, void *ws, void *stream);
int32_t moe_layer_backward(const moe_config *cfg, const void *dOut, const void *x, const float *Wg,
                           const float *Wnoise, const float *noise, const void *W1, const void *b1, const void *W2,
                           const void *b2, const uint8_t *keep_bits, float drop_prob, const void *ctx, void *dX,
                           float *dWg, float *dWnoise, void *dW1, void *db1, void *dW2, void *db2, void *ws,
                           void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H */
