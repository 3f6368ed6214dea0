// The C ABI (include/moe.h): argument checks, workspace carving and the order of the launches.
#include <string.h>

#include "moe_internal.cuh"

#include <atomic>

using namespace moe;

static std::atomic<long long> g_launches{0};
void moe::count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

namespace {

struct Dims {
    int64_t T, d, h, n, k, R;
    bool hier;
    int64_t a, k1, b, k2;
    int64_t gate_cols, logits, gates, kth, wg, load, dload;
    int32_t act, flags;
    size_t esz;
};

int32_t check_config(const moe_config *c) {
    if (!c) return MOE_ERR_INVALID_ARG;
    if (c->T < 0 || c->d <= 0 || c->h <= 0 || c->n <= 0 || c->k <= 0) return MOE_ERR_INVALID_ARG;
    if (c->act != MOE_F32 && c->act != MOE_BF16) return MOE_ERR_INVALID_ARG;
    if (c->k > c->n || c->k > MOE_MAX_K) return MOE_ERR_INVALID_ARG;
    const size_t esz = act_bytes(c->act);
    if ((c->d * esz) % 16 != 0 || (c->h * esz) % 16 != 0) return MOE_ERR_INVALID_ARG;
    if ((int64_t)c->T * c->k >= (int64_t)1 << 31) return MOE_ERR_INVALID_ARG;
    if (c->a < 0) return MOE_ERR_INVALID_ARG;
    if (c->a > 0) {
        if (c->b <= 0 || c->k1 <= 0 || c->k2 <= 0) return MOE_ERR_INVALID_ARG;
        if (c->k1 > c->a || c->k2 > c->b) return MOE_ERR_INVALID_ARG;
        if ((int64_t)c->a * c->b != c->n || c->k1 * c->k2 != c->k) return MOE_ERR_INVALID_ARG;
        if (c->a > MOE_MAX_EXPERTS || c->b > MOE_MAX_EXPERTS) return MOE_ERR_INVALID_ARG;
        if ((int64_t)c->a * c->b > (int64_t)1 << 20) return MOE_ERR_INVALID_ARG;
        // the routing kernels keep one int32 per expert in (default-size) shared memory
        if ((int64_t)c->a * c->b > MOE_MAX_FLAT_EXPERTS) return MOE_ERR_UNSUPPORTED;
    } else if (c->n > MOE_MAX_EXPERTS) {
        return MOE_ERR_INVALID_ARG;
    }
    if (!(c->w_importance >= 0.0f) || !(c->w_load >= 0.0f)) return MOE_ERR_INVALID_ARG;
    if (c->flags & ~(MOE_FLAG_GATE_SCREEN_OFF | MOE_FLAG_GATE_SCREEN_ON | MOE_FLAG_TC_ONE_CTA | MOE_FLAG_RECOMPUTE_HID))
        return MOE_ERR_INVALID_ARG;
    if ((c->flags & MOE_FLAG_GATE_SCREEN_OFF) && (c->flags & MOE_FLAG_GATE_SCREEN_ON)) return MOE_ERR_INVALID_ARG;
    return MOE_OK;
}

Dims dims_of(const moe_config *c) {
    Dims D;
    D.T = c->T; D.d = c->d; D.h = c->h; D.n = c->n; D.k = c->k;
    D.R = D.T * D.k;
    D.hier = c->a > 0;
    D.a = c->a; D.k1 = c->k1; D.b = c->b; D.k2 = c->k2;
    D.act = c->act;
    D.flags = c->flags;
    D.esz = act_bytes(c->act);
    if (D.hier) {
        D.gate_cols = D.a + D.k1 * D.b;
        D.gates = D.T * (2 * D.k + D.k1);
        D.kth = 2 * D.T * (1 + D.k1);
        D.wg = D.d * D.a + D.a * D.d * D.b;
        D.load = 2 * D.a * D.b + 2 * D.a;
        D.dload = D.a + D.a * D.b;
    } else {
        D.gate_cols = D.n;
        D.gates = D.T * D.k;
        D.kth = 2 * D.T;
        D.wg = D.d * D.n;
        D.load = D.n;
        D.dload = D.n;
    }
    D.logits = D.T * D.gate_cols;
    return D;
}

bool bad_ptr(const void *p) { return p == nullptr || !aligned16(p); }
#define REQUIRE_PTRS(...)                                             \
    do {                                                              \
        const void *ps_[] = {__VA_ARGS__};                            \
        for (size_t i_ = 0; i_ < sizeof(ps_) / sizeof(ps_[0]); ++i_)  \
            if (bad_ptr(ps_[i_])) return MOE_ERR_INVALID_ARG;         \
    } while (0)

// arguments of the layer epilogue: packed keep bits [T, d/8] and the dropout probability
int32_t check_layer(const moe_config *c, const uint8_t *keep_bits, float drop_prob) {
    if (bad_ptr(keep_bits) || c->d % 8 != 0) return MOE_ERR_INVALID_ARG;
    if (!(drop_prob >= 0.0f) || !(drop_prob < 1.0f)) return MOE_ERR_INVALID_ARG;
    return MOE_OK;
}

cudaStream_t as_stream(void *s) { return static_cast<cudaStream_t>(s); }

int32_t *status_word(void *ws) { return static_cast<int32_t *>(ws); }

int32_t reset_status(void *ws, cudaStream_t st) {
    MOE_CUDA(cudaMemsetAsync(ws, 0, kWsHeader, st));
    return MOE_OK;
}

// ---------------------------------------------------------------------------- stage workspaces
struct GateWs {
    int32_t *idx_p, *idx_s, *perm_p, *inv_perm_p, *counts_p, *offsets_p, *scratch, *tile_prefix;
    // tensor-core routing screen (flat layer, or the primary level of the hierarchical one)
    bool screen;
    float *cr, *wnorm, *xnorm, *wt;
    void *wsplit;
    int32_t *unsafe_list, *unsafe_count, *full_list;
    float *unsafe_low, *unsafe_low_s;
    void *unsafe_span, *unsafe_span_s;  // int2 per listed row
    void *chain_list;
    // the same for the secondary gates of the hierarchical layer (rows = slots sorted by primary group)
    bool screen2;
    void *xs_p, *wsplit_s, *chain_list_s;
    float *cr_s, *wnorm_s, *wt_s;
    int32_t *unsafe_list_s, *unsafe_count_s;
    GateWs(Carver &cv, const Dims &D) {
        screen2 = false;
        xs_p = wsplit_s = chain_list_s = nullptr; cr_s = wnorm_s = wt_s = nullptr; unsafe_list_s = unsafe_count_s = nullptr; unsafe_low = unsafe_low_s = nullptr; unsafe_span = unsafe_span_s = nullptr;
        idx_p = idx_s = perm_p = inv_perm_p = counts_p = offsets_p = scratch = tile_prefix = nullptr;
        cr = wnorm = xnorm = wt = nullptr; wsplit = nullptr; unsafe_list = unsafe_count = full_list = nullptr; chain_list = nullptr;
        const int64_t n1 = D.hier ? D.a : D.n;  // width of the (first) gate
        screen = tc_gate_fwd_supported(D.act, D.T, (int32_t)D.d, (int32_t)n1, D.flags);
        if (screen) {
            cr = cv.take<float>(D.T * 2 * n1);
            wsplit = cv.take<bf16>(3 * D.d * 2 * n1);
            wnorm = cv.take<float>(2 * n1);
            wt = cv.take<float>(2 * n1 * D.d);
            xnorm = cv.take<float>(D.T);
            unsafe_list = cv.take<int32_t>(D.T);
            unsafe_low = cv.take<float>(D.T);
            unsafe_span = cv.take_bytes(D.T * 8);
            unsafe_count = cv.take<int32_t>(64);
            full_list = cv.take<int32_t>(D.T);
            chain_list = cv.take_bytes(D.T * 2 * SCREEN_MAX_CAND * 8);
        }
        if (!D.hier) return;
        idx_p = cv.take<int32_t>(D.T * D.k1);
        idx_s = cv.take<int32_t>(D.T * D.k);
        perm_p = cv.take<int32_t>(D.T * D.k1);
        inv_perm_p = cv.take<int32_t>(D.T * D.k1);
        counts_p = cv.take<int32_t>(D.a);
        offsets_p = cv.take<int32_t>(D.a + 1);
        scratch = cv.take<int32_t>(dispatch_ws_elems(D.T * D.k1, (int32_t)D.a));
        tile_prefix = cv.take<int32_t>(tc_tile_ws_ints(D.T * D.k1, D.a));  // prefix + tile table of the grouped product
        const int64_t P1 = D.T * D.k1;
        screen2 = tc_gate_fwd_supported(D.act, P1, (int32_t)D.d, (int32_t)D.b, D.flags);
        if (screen2) {
            if (!xnorm) xnorm = cv.take<float>(D.T);
            xs_p = cv.take_bytes(P1 * D.d * (int64_t)D.esz);
            cr_s = cv.take<float>(P1 * 2 * D.b);
            wsplit_s = cv.take<bf16>(3 * D.a * D.d * 2 * D.b);
            wnorm_s = cv.take<float>(D.a * 2 * D.b);
            wt_s = cv.take<float>(D.a * 2 * D.b * D.d);
            unsafe_list_s = cv.take<int32_t>(P1);
            unsafe_low_s = cv.take<float>(P1);
            unsafe_span_s = cv.take_bytes(P1 * 8);
            unsafe_count_s = cv.take<int32_t>(64);
            chain_list_s = cv.take_bytes(P1 * 2 * D.b * 8);  // worst case: every column of every slot
        }
    }
};

struct DispatchWs {
    int32_t *scratch;
    DispatchWs(Carver &cv, const Dims &D) { scratch = cv.take<int32_t>(dispatch_ws_elems(D.R, (int32_t)D.n)); }
};

struct FfnWs {
    int32_t *tile_prefix;
    void *tc;
    void *hid;  // MOE_FLAG_RECOMPUTE_HID: the hidden activations live here instead of in a buffer that is kept
    FfnWs(Carver &cv, const Dims &D, const moe_config *c) {
        tile_prefix = cv.take<int32_t>(D.n + 1);
        tc = tc_ffn_supported(*c) ? cv.take_bytes(tc_ffn_ws_bytes(*c)) : nullptr;
        hid = (D.flags & MOE_FLAG_RECOMPUTE_HID) ? cv.take_bytes(D.R * D.h * (int64_t)D.esz) : nullptr;
    }
};

// index tensors of the hierarchical levels, rebuilt from topk_idx where a stage needs them
struct HierIdxWs {
    int32_t *idx_p, *idx_s, *perm_p, *inv_perm_p, *counts_p, *offsets_p, *scratch, *tile_prefix;
    HierIdxWs(Carver &cv, const Dims &D) {
        idx_p = idx_s = perm_p = inv_perm_p = counts_p = offsets_p = scratch = tile_prefix = nullptr;
        if (!D.hier) return;
        idx_p = cv.take<int32_t>(D.T * D.k1);
        idx_s = cv.take<int32_t>(D.T * D.k);
        perm_p = cv.take<int32_t>(D.T * D.k1);
        inv_perm_p = cv.take<int32_t>(D.T * D.k1);
        counts_p = cv.take<int32_t>(D.a);
        offsets_p = cv.take<int32_t>(D.a + 1);
        scratch = cv.take<int32_t>(dispatch_ws_elems(D.T * D.k1, (int32_t)D.a));
        tile_prefix = cv.take<int32_t>(tc_tile_ws_ints(D.T * D.k1, D.a));  // prefix + tile table of the secondary-gate GEMMs
    }
    int32_t build(const Dims &D, const int32_t *topk_idx, cudaStream_t st) {
        MOE_TRY(launch_hier_split_idx(topk_idx, D.T, (int32_t)D.k1, (int32_t)D.k2, (int32_t)D.a, (int32_t)D.b, idx_p, idx_s, st));
        return launch_dispatch_index(idx_p, D.T * D.k1, (int32_t)D.a, perm_p, inv_perm_p, counts_p, offsets_p, scratch,
                                     st);
    }
};

struct LossesWs {
    float *scratch, *grouped;
    HierIdxWs H;
    int32_t *perm_e, *inv_perm_e, *counts_e, *offsets_e, *scratch_e;  // by flat expert, if the caller has none
    LossesWs(Carver &cv, const Dims &D) : H(cv, D) {
        scratch = cv.take<float>(losses_ws_floats(D.T, (int32_t)(D.hier ? D.a : D.n)));
        grouped = nullptr;
        perm_e = inv_perm_e = counts_e = offsets_e = scratch_e = nullptr;
        if (!D.hier) return;
        grouped = cv.take<float>(grouped_sums_ws_floats(D.T * D.k1, (int32_t)D.a, (int32_t)D.b));
        perm_e = cv.take<int32_t>(D.R);
        inv_perm_e = cv.take<int32_t>(D.R);
        counts_e = cv.take<int32_t>(D.n);
        offsets_e = cv.take<int32_t>(D.n + 1);
        scratch_e = cv.take<int32_t>(dispatch_ws_elems(D.R, (int32_t)D.n));
    }
};

struct FfnBwdWs {
    void *dz;
    int32_t *tile_prefix;
    float *colsum;
    FfnBwdWs(Carver &cv, const Dims &D) {
        dz = cv.take_bytes(D.R * D.h * (int64_t)D.esz);
        tile_prefix = cv.take<int32_t>(tc_tile_ws_ints(D.R, D.n));  // prefix + tile table of the row GEMMs
        int64_t cs = colsum_ws_floats(D.R, (int32_t)D.n, (int32_t)(D.h > D.d ? D.h : D.d));
        if (D.act == MOE_BF16) {  // the tensor-core path sums dz's columns per 32-row block in the GEMM epilogue
            const int64_t cs_tc = tc_colsum_part_floats(D.R, (int32_t)D.n, (int32_t)D.h);
            if (cs_tc > cs) cs = cs_tc;
        }
        colsum = cv.take<float>(cs);
    }
};

struct LossesBwdWs {
    float *dimp, *dload_h;
    LossesBwdWs(Carver &cv, const Dims &D) {
        dimp = cv.take<float>(D.n);
        dload_h = D.hier ? cv.take<float>(D.n) : nullptr;
    }
};

struct GateBwdWs {
    float *dclean, *draw, *partials, *dX_sec, *partials_s;
    void *dsplit, *wsplit, *dsplit_s, *wsplit_s, *xs_p;
    bool tc, tc_hier;
    HierIdxWs H;
    GateBwdWs(Carver &cv, const Dims &D) : H(cv, D) {
        dclean = draw = partials = dX_sec = partials_s = nullptr;
        dsplit = wsplit = dsplit_s = wsplit_s = xs_p = nullptr;
        if (D.hier) dX_sec = cv.take<float>(D.T * D.k1 * D.d);
        tc = !D.hier && tc_gate_bwd_supported(D.act, (int32_t)D.d, (int32_t)D.n);
        tc_hier = D.hier && tc_hier_gate_bwd_supported(D.act, (int32_t)D.d, (int32_t)D.a, (int32_t)D.b);
        if (tc_hier) {
            dsplit = cv.take<bf16>(D.T * 6 * D.a);
            wsplit = cv.take<bf16>(D.d * 6 * D.a);
            partials = cv.take<float>(tc_gate_bwd_partials(D.T, (int32_t)D.d, (int32_t)D.a));
            dsplit_s = cv.take<bf16>(D.T * D.k1 * 6 * D.b);
            wsplit_s = cv.take<bf16>(D.a * D.d * 6 * D.b);
            partials_s = cv.take<float>(3 * D.a * D.d * 2 * D.b);
            xs_p = cv.take<bf16>(D.T * D.k1 * D.d);
        } else if (tc) {
            dsplit = cv.take<bf16>(D.T * 6 * D.n);
            wsplit = cv.take<bf16>(D.d * 6 * D.n);
            partials = cv.take<float>(tc_gate_bwd_partials(D.T, (int32_t)D.d, (int32_t)D.n));
        } else {
            dclean = cv.take<float>(D.logits);
            draw = cv.take<float>(D.logits);
        }
    }
};

template <typename F> int64_t measure(F f) {
    Carver cv(nullptr);
    cv.take_bytes(kWsHeader);
    f(cv);
    return (int64_t)cv.off;
}

struct Ctx {
    int32_t *topk_idx, *kth_idx, *perm, *inv_perm, *counts, *offsets;
    float *gates, *clean, *raw_noise, *kth_vals, *importance, *load, *losses;
    void *xs, *hid, *ys;
    uint32_t *relu_bits;  // tensor-core layers that keep hid: one bit per hidden activation for the backward's ReLU mask
    moe_ctx_layout off;
    Ctx(void *base, const Dims &D, bool has_bits) {
        Carver cv(base);
        auto at = [&]() { return (int64_t)cv.off; };
        off.topk_idx = at(); topk_idx = cv.take<int32_t>(D.R);
        off.gates = at(); gates = cv.take<float>(D.gates);
        off.clean = at(); clean = cv.take<float>(D.logits);
        off.raw_noise = at(); raw_noise = cv.take<float>(D.logits);
        off.kth_vals = at(); kth_vals = cv.take<float>(D.kth);
        off.kth_idx = at(); kth_idx = cv.take<int32_t>(D.kth);
        off.xs = at(); xs = cv.take_bytes(D.R * D.d * (int64_t)D.esz);
        off.perm = at(); perm = cv.take<int32_t>(D.R);
        off.inv_perm = at(); inv_perm = cv.take<int32_t>(D.R);
        off.counts = at(); counts = cv.take<int32_t>(D.n);
        off.offsets = at(); offsets = cv.take<int32_t>(D.n + 1);
        off.hid = at(); hid = (D.flags & MOE_FLAG_RECOMPUTE_HID) ? nullptr : cv.take_bytes(D.R * D.h * (int64_t)D.esz);
        off.ys = at(); ys = cv.take_bytes(D.R * D.d * (int64_t)D.esz);
        off.importance = at(); importance = cv.take<float>(D.n);
        off.load = at(); load = cv.take<float>(D.load);
        off.losses = at(); losses = cv.take<float>(2);
        off.relu_bits = at();
        relu_bits = (has_bits && !(D.flags & MOE_FLAG_RECOMPUTE_HID)) ? cv.take<uint32_t>(D.R * (D.h / 32)) : nullptr;
        bytes = (int64_t)cv.off;
    }
    int64_t bytes;
};

struct BwdWs {
    float *dgates, *dload, *dX_gate;
    void *dys, *dxs;
    BwdWs(Carver &cv, const Dims &D) {
        dgates = cv.take<float>(D.gates);
        dload = cv.take<float>(D.dload);
        dX_gate = cv.take<float>(D.T * D.d);
        dys = cv.take_bytes(D.R * D.d * (int64_t)D.esz);
        dxs = cv.take_bytes(D.R * D.d * (int64_t)D.esz);
    }
};

// ---------------------------------------------------------------------------- stage bodies
// (pointers already checked; `cv` positioned after the workspace header)

int32_t do_gate(const moe_config *c, const Dims &D, const void *x, const float *Wg, const float *Wnoise,
                const float *noise, int32_t *topk_idx, float *gates, float *clean, float *raw_noise,
                float *kth_vals, int32_t *kth_idx, void *ws_base, Carver &cv, cudaStream_t st) {
    GateWs w(cv, D);
    // One gate over n1 columns with top-k1 (the flat gate, or the primary gate of the hierarchical layer).
    // With bf16 activations the routing is screened on the tensor cores and only the tokens whose order is
    // not provably that of the fixed fma chain are redone with the chain; otherwise the chain does all rows.
    auto first_gate = [&](int32_t n1, int32_t k1, int32_t *idx_out, float *gates_out) -> int32_t {
        if (w.screen) {
            MOE_TRY(launch_gate_screen_prepare(x, D.act, D.T, (int32_t)D.d, n1, Wg, Wnoise, w.wsplit, w.wnorm, w.xnorm,
                                               w.unsafe_count, w.wt, st));
            MOE_TRY(launch_tc_gate_fwd(x, D.T, (int32_t)D.d, n1, w.wsplit, w.cr, status_word(ws_base), st));
            MOE_TRY(launch_gate_screen(w.cr, noise, w.xnorm, w.wnorm, (int32_t)D.d, D.T, n1, k1, idx_out, gates_out,
                                       clean, raw_noise, kth_vals, kth_idx, w.unsafe_list, w.unsafe_low, w.unsafe_count,
                                       w.chain_list, w.full_list, st, nullptr, 1, nullptr, w.unsafe_span));
            // exact chains for the few columns that decide an uncertain row; whole rows only where there are many
            MOE_TRY(launch_gate_chains(x, D.act, (int32_t)D.d, n1, w.wt, w.chain_list, w.unsafe_count + 1, clean, raw_noise,
                                       st));
            MOE_TRY(launch_projection(x, D.act, D.T, (int32_t)D.d, n1, Wg, Wnoise, clean, raw_noise, nullptr, 0,
                                      w.full_list, 1, nullptr, st, w.unsafe_count + 2));
            return launch_gate_select(clean, raw_noise, noise, D.T, n1, k1, idx_out, gates_out, kth_vals, kth_idx, st,
                                      w.unsafe_list, w.unsafe_count, w.unsafe_span, w.chain_list);
        }
        MOE_TRY(launch_projection(x, D.act, D.T, (int32_t)D.d, n1, Wg, Wnoise, clean, raw_noise, nullptr, 0, nullptr, 1,
                                  nullptr, st));
        return launch_gate_select(clean, raw_noise, noise, D.T, n1, k1, idx_out, gates_out, kth_vals, kth_idx, st);
    };
    if (!D.hier) return first_gate((int32_t)D.n, (int32_t)D.k, topk_idx, gates);
    // primary gate over the a groups
    const int64_t P1 = D.T * D.k1;
    float *g_p = gates + D.T * D.k, *g_s = g_p + P1;
    MOE_TRY(first_gate((int32_t)D.a, (int32_t)D.k1, w.idx_p, g_p));
    // secondary gates: rows (t, s1) grouped by their group so each tile uses one group's matrices
    MOE_TRY(launch_dispatch_index(w.idx_p, P1, (int32_t)D.a, w.perm_p, w.inv_perm_p, w.counts_p, w.offsets_p,
                                  w.scratch, st));
    const int64_t lp = D.T * D.a;  // elements of the primary part of the logits tensors
    const float *Wg_s = Wg + D.d * D.a, *Wn_s = Wnoise + D.d * D.a;
    if (w.screen2) {
        // the routing screen on the grouped product: token rows gathered by group, one weight pair per group
        MOE_TRY(launch_dispatch_rows(x, D.act, D.T, (int32_t)D.k1, (int32_t)D.d, w.inv_perm_p, w.xs_p, st));
        MOE_TRY(launch_gate_screen_prepare(x, D.act, D.T, (int32_t)D.d, (int32_t)D.b, Wg_s, Wn_s, w.wsplit_s, w.wnorm_s,
                                           w.xnorm, w.unsafe_count_s, w.wt_s, st, (int32_t)D.a, !w.screen));
        MOE_TRY(launch_tc_gate_fwd_grouped(w.xs_p, P1, (int32_t)D.d, (int32_t)D.a, (int32_t)D.b, w.wsplit_s, w.offsets_p,
                                           w.tile_prefix, w.cr_s, status_word(ws_base), st, D.flags));
        MOE_TRY(launch_gate_screen(w.cr_s, noise + lp, w.xnorm, w.wnorm_s, (int32_t)D.d, P1, (int32_t)D.b, (int32_t)D.k2,
                                   w.idx_s, g_s, clean + lp, raw_noise + lp, kth_vals + 2 * D.T, kth_idx + 2 * D.T,
                                   w.unsafe_list_s, w.unsafe_low_s, w.unsafe_count_s, w.chain_list_s, nullptr, st, w.perm_p,
                                   (int32_t)D.k1, w.idx_p, w.unsafe_span_s));
        MOE_TRY(launch_gate_chains(x, D.act, (int32_t)D.d, (int32_t)D.b, w.wt_s, w.chain_list_s, w.unsafe_count_s + 1,
                                   clean + lp, raw_noise + lp, st, (int32_t)D.k1));
        MOE_TRY(launch_gate_select(clean + lp, raw_noise + lp, noise + lp, P1, (int32_t)D.b, (int32_t)D.k2, w.idx_s, g_s,
                                   kth_vals + 2 * D.T, kth_idx + 2 * D.T, st, w.unsafe_list_s, w.unsafe_count_s, w.unsafe_span_s,
                                   w.chain_list_s));
    } else {
        MOE_TRY(launch_projection(x, D.act, P1, (int32_t)D.d, (int32_t)D.b, Wg_s, Wn_s, clean + lp, raw_noise + lp,
                                  w.offsets_p, (int32_t)D.a, w.perm_p, (int32_t)D.k1, w.tile_prefix, st));
        MOE_TRY(launch_gate_select(clean + lp, raw_noise + lp, noise + lp, P1, (int32_t)D.b, (int32_t)D.k2, w.idx_s,
                                   g_s, kth_vals + 2 * D.T, kth_idx + 2 * D.T, st));
    }
    return launch_hier_merge(D.T, (int32_t)D.k1, (int32_t)D.k2, (int32_t)D.b, w.idx_p, g_p, w.idx_s, g_s, topk_idx,
                             gates, st);
}

int32_t do_dispatch(const Dims &D, const void *x, const int32_t *topk_idx, void *xs, int32_t *perm,
                    int32_t *inv_perm, int32_t *counts, int32_t *offsets, Carver &cv, cudaStream_t st) {
    DispatchWs w(cv, D);
    MOE_TRY(launch_dispatch_index(topk_idx, D.R, (int32_t)D.n, perm, inv_perm, counts, offsets, w.scratch, st));
    return launch_dispatch_rows(x, D.act, D.T, (int32_t)D.k, (int32_t)D.d, inv_perm, xs, st);
}

SimtGemm base_gemm(const Dims &D) {
    SimtGemm g;
    memset(&g, 0, sizeof(g));
    g.ta = g.tb = g.tc = D.act == MOE_BF16 ? G_BF16 : G_F32;
    g.a_row_div = 1;
    return g;
}

// hid == nullptr (only with MOE_FLAG_RECOMPUTE_HID): the hidden activations stay in the workspace.
// first_only: only hid = relu(xs.W1 + b1) is computed (ys is not touched).
int32_t do_expert_ffn(const moe_config *c, const Dims &D, const void *xs, const int32_t *offsets, const void *W1,
                      const void *b1, const void *W2, const void *b2, void *hid, void *ys, void *ws_base,
                      Carver &cv, cudaStream_t st, bool first_only = false, void **hid_used = nullptr,
                      uint32_t *relu_bits = nullptr) {
    FfnWs w(cv, D, c);
    if (!hid) hid = w.hid;
    if (!hid) return MOE_ERR_INVALID_ARG;
    if (hid_used) *hid_used = hid;
    if (w.tc)
        return launch_tc_ffn(*c, xs, offsets, W1, b1, W2, b2, hid, ys, w.tc, status_word(ws_base), st, first_only, relu_bits);
    SimtGemm g = base_gemm(D);  // hid = relu(xs.W1 + b1)
    g.A = xs; g.B = W1; g.C = hid; g.bias = b1; g.relu = 1;
    g.sa_i = D.d; g.sa_k = 1; g.sb_k = D.h; g.sb_j = 1; g.sc_i = D.h; g.sc_j = 1;
    g.mode = 0; g.offsets = offsets; g.nseg = (int32_t)D.n; g.M = D.R; g.N = D.h; g.K = D.d; g.b_e = D.d * D.h;
    MOE_TRY(launch_simt_gemm(g, w.tile_prefix, st));
    if (first_only) return MOE_OK;
    g = base_gemm(D);  // ys = hid.W2 + b2
    g.A = hid; g.B = W2; g.C = ys; g.bias = b2;
    g.sa_i = D.h; g.sa_k = 1; g.sb_k = D.d; g.sb_j = 1; g.sc_i = D.d; g.sc_j = 1;
    g.mode = 0; g.offsets = offsets; g.nseg = (int32_t)D.n; g.M = D.R; g.N = D.d; g.K = D.h; g.b_e = D.h * D.d;
    return launch_simt_gemm(g, w.tile_prefix, st);
}

int32_t do_losses(const moe_config *c, const Dims &D, const int32_t *topk_idx, const float *gates,
                  const float *clean, const float *raw_noise, const float *kth_vals, float *importance, float *load,
                  float *losses, const int32_t *perm, const int32_t *offsets, Carver &cv, cudaStream_t st) {
    LossesWs w(cv, D);
    if (!D.hier) {
        MOE_TRY(launch_level_sums(topk_idx, gates, clean, raw_noise, kth_vals, D.T, (int32_t)D.n, (int32_t)D.k,
                                  importance, load, w.scratch, st));
        return launch_cv2(importance, (int32_t)D.n, load, (int32_t)D.n, c->w_importance, c->w_load, losses, st);
    }
    // Eq. 13: Importance_H = batch sum of the product gates per expert (ordered sum over each expert's rows)
    if (!perm) {
        MOE_TRY(launch_dispatch_index(topk_idx, D.R, (int32_t)D.n, w.perm_e, w.inv_perm_e, w.counts_e, w.offsets_e,
                                      w.scratch_e, st));
        perm = w.perm_e;
        offsets = w.offsets_e;
    }
    MOE_TRY(launch_segment_sum(gates, perm, offsets, (int32_t)D.n, importance, st));
    // Eq. 14: Load_primary, the per-group Load_i over X^(i), |X^(i)|
    MOE_TRY(w.H.build(D, topk_idx, st));
    const int64_t ab = D.a * D.b, lp = D.T * D.a;
    float *load_p = load + ab, *load_s = load_p + D.a;
    MOE_TRY(launch_level_sums(w.H.idx_p, gates + D.T * D.k, clean, raw_noise, kth_vals, D.T, (int32_t)D.a,
                              (int32_t)D.k1, nullptr, load_p, w.scratch, st));
    MOE_TRY(launch_grouped_load(w.H.idx_s, clean + lp, raw_noise + lp, kth_vals + 2 * D.T, w.H.perm_p, w.H.offsets_p,
                                (int32_t)D.a, D.T * D.k1, (int32_t)D.b, (int32_t)D.k2, load_s, w.grouped,
                                w.H.tile_prefix, st));
    MOE_TRY(launch_load_h(load, w.H.counts_p, (int32_t)D.a, (int32_t)D.b, st));
    return launch_cv2(importance, (int32_t)ab, load, (int32_t)ab, c->w_importance, c->w_load, losses, st);
}

int32_t do_expert_ffn_bwd(const moe_config *c, const Dims &D, const void *xs, const void *hid, const void *dys,
                          const int32_t *offsets, const void *W1, const void *W2, void *dxs, void *dW1, void *db1,
                          void *dW2, void *db2, void *ws_base, Carver &cv, cudaStream_t st,
                          const uint32_t *relu_bits = nullptr) {
    FfnBwdWs w(cv, D);
    const int32_t n = (int32_t)D.n;
    if (tc_ffn_supported(*c))
        return launch_tc_ffn_bwd(*c, xs, hid, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, w.dz, w.colsum,
                                 w.tile_prefix, status_word(ws_base), st, relu_bits);
    MOE_TRY(launch_segment_colsum(dys, D.act, offsets, n, D.R, (int32_t)D.d, db2, w.colsum, w.tile_prefix, st));
    SimtGemm g = base_gemm(D);  // dW2[e] = hid_e^T . dys_e
    g.A = hid; g.B = dys; g.C = dW2;
    g.sa_i = 1; g.sa_k = D.h; g.sb_k = D.d; g.sb_j = 1; g.sc_i = D.d; g.sc_j = 1;
    g.mode = 1; g.offsets = offsets; g.nseg = n; g.M = D.h; g.N = D.d; g.c_e = D.h * D.d;
    MOE_TRY(launch_simt_gemm(g, w.tile_prefix, st));
    g = base_gemm(D);  // dz = (dys . W2[e]^T) * [hid > 0]
    g.A = dys; g.B = W2; g.C = w.dz; g.mask = hid;
    g.sa_i = D.d; g.sa_k = 1; g.sb_k = 1; g.sb_j = D.d; g.sc_i = D.h; g.sc_j = 1;
    g.mode = 0; g.offsets = offsets; g.nseg = n; g.M = D.R; g.N = D.h; g.K = D.d; g.b_e = D.h * D.d;
    MOE_TRY(launch_simt_gemm(g, w.tile_prefix, st));
    MOE_TRY(launch_segment_colsum(w.dz, D.act, offsets, n, D.R, (int32_t)D.h, db1, w.colsum, w.tile_prefix, st));
    g = base_gemm(D);  // dW1[e] = xs_e^T . dz_e
    g.A = xs; g.B = w.dz; g.C = dW1;
    g.sa_i = 1; g.sa_k = D.d; g.sb_k = D.h; g.sb_j = 1; g.sc_i = D.h; g.sc_j = 1;
    g.mode = 1; g.offsets = offsets; g.nseg = n; g.M = D.d; g.N = D.h; g.c_e = D.d * D.h;
    MOE_TRY(launch_simt_gemm(g, w.tile_prefix, st));
    g = base_gemm(D);  // dxs = dz . W1[e]^T
    g.A = w.dz; g.B = W1; g.C = dxs;
    g.sa_i = D.h; g.sa_k = 1; g.sb_k = 1; g.sb_j = D.h; g.sc_i = D.d; g.sc_j = 1;
    g.mode = 0; g.offsets = offsets; g.nseg = n; g.M = D.R; g.N = D.d; g.K = D.h; g.b_e = D.d * D.h;
    return launch_simt_gemm(g, w.tile_prefix, st);
}

int32_t do_losses_bwd(const moe_config *c, const Dims &D, const float *importance, const float *load,
                      const int32_t *topk_idx, float *dgates, float *dload, Carver &cv, cudaStream_t st) {
    LossesBwdWs w(cv, D);
    if (!D.hier)
        return launch_losses_bwd_flat(importance, load, (int32_t)D.n, topk_idx, D.R, c->w_importance, c->w_load,
                                      dgates, dload, w.dimp, st);
    MOE_TRY(launch_cv2_grad(importance, (int32_t)D.n, c->w_importance, w.dimp, st));
    MOE_TRY(launch_add_gathered(dgates, topk_idx, w.dimp, D.R, (int32_t)D.n, st));
    MOE_TRY(launch_cv2_grad(load, (int32_t)D.n, c->w_load, w.dload_h, st));  // load[0 : a*b] is Load_H
    return launch_load_h_bwd(load, w.dload_h, (int32_t)D.a, (int32_t)D.b, dload, st);
}

// dW = x^T . dlogit [d, n];  dX (+)= dlogit . W^T [T, d]
int32_t gate_weight_grads(const Dims &D, const void *x, const float *dlogit, const float *W, int64_t n,
                          float *dW, float *dX, bool accumulate, cudaStream_t st) {
    SimtGemm g;
    memset(&g, 0, sizeof(g));
    g.a_row_div = 1;
    g.ta = D.act == MOE_BF16 ? G_BF16 : G_F32; g.tb = G_F32; g.tc = G_F32;
    g.A = x; g.B = dlogit; g.C = dW;
    g.sa_i = 1; g.sa_k = D.d; g.sb_k = n; g.sb_j = 1; g.sc_i = n; g.sc_j = 1;
    g.mode = 1; g.offsets = nullptr; g.nseg = 1; g.M = D.d; g.N = n; g.K = D.T;
    MOE_TRY(launch_simt_gemm(g, nullptr, st));
    memset(&g, 0, sizeof(g));
    g.a_row_div = 1;
    g.ta = g.tb = g.tc = G_F32;
    g.A = dlogit; g.B = W; g.C = dX; g.accumulate = accumulate ? 1 : 0;
    g.sa_i = n; g.sa_k = 1; g.sb_k = 1; g.sb_j = n; g.sc_i = D.d; g.sc_j = 1;
    g.mode = 0; g.offsets = nullptr; g.nseg = 1; g.M = D.T; g.N = D.d; g.K = n;
    return launch_simt_gemm(g, nullptr, st);
}

int32_t do_gate_bwd(const moe_config *c, const Dims &D, const void *x, const float *Wg, const float *Wnoise,
                    const float *noise, const float *clean, const float *raw_noise, const int32_t *topk_idx,
                    const float *gates, const float *kth_vals, const int32_t *kth_idx, float *dgates,
                    const float *dload, float *dWg, float *dWnoise, float *dX_gate, void *ws_base, Carver &cv,
                    cudaStream_t st) {
    GateBwdWs w(cv, D);
    if (D.hier) {
        const int64_t P1 = D.T * D.k1, lp = D.T * D.a, wp = D.d * D.a;
        const float *g_p = gates + D.T * D.k, *g_s = g_p + P1;
        float *dg_p = dgates + D.T * D.k, *dg_s = dg_p + P1;
        float *dc_p = w.dclean, *dr_p = w.draw, *dc_s = w.dclean + lp, *dr_s = w.draw + lp;
        MOE_TRY(w.H.build(D, topk_idx, st));
        MOE_TRY(launch_hier_gate_product_bwd(gates, dgates, D.T, (int32_t)D.k1, (int32_t)D.k2, st));
        if (w.tc_hier) {
            // both levels on the tensor cores: split logit gradients (the secondary ones written in the
            // order sorted by primary group), grouped products, then the slots' rows are added per token
            MOE_TRY(launch_gate_logit_grads(noise, clean, raw_noise, w.H.idx_p, g_p, kth_vals, kth_idx, dg_p, dload,
                                            nullptr, D.T, (int32_t)D.a, (int32_t)D.k1, nullptr, nullptr, w.dsplit,
                                            nullptr, st));
            MOE_TRY(launch_tc_gate_bwd(x, D.T, (int32_t)D.d, (int32_t)D.a, Wg, Wnoise, w.dsplit, w.wsplit, w.partials,
                                       dWg, dWnoise, dX_gate, status_word(ws_base), st, D.flags));
            MOE_TRY(launch_gate_logit_grads(noise + lp, clean + lp, raw_noise + lp, w.H.idx_s, g_s, kth_vals + 2 * D.T,
                                            kth_idx + 2 * D.T, dg_s, dload + D.a, w.H.idx_p, P1, (int32_t)D.b,
                                            (int32_t)D.k2, nullptr, nullptr, w.dsplit_s, w.H.inv_perm_p, st));
            MOE_TRY(launch_dispatch_rows(x, D.act, D.T, (int32_t)D.k1, (int32_t)D.d, w.H.inv_perm_p, w.xs_p, st));
            MOE_TRY(launch_tc_hier_secondary_bwd(w.xs_p, w.dsplit_s, w.wsplit_s, Wg + wp, Wnoise + wp, w.H.offsets_p,
                                                 w.H.tile_prefix, (int32_t)D.a, P1, (int32_t)D.d, (int32_t)D.b,
                                                 w.partials_s, dWg + wp, dWnoise + wp, w.dX_sec, status_word(ws_base),
                                                 st));
            return launch_dispatch_bwd(w.dX_sec, MOE_F32, w.H.inv_perm_p, D.T, (int32_t)D.k1, (int32_t)D.d, dX_gate,
                                       dX_gate, nullptr, st);
        }
        // primary gate (Eq. 12: G_primary), rows = tokens
        MOE_TRY(launch_gate_logit_grads(noise, clean, raw_noise, w.H.idx_p, g_p, kth_vals, kth_idx, dg_p, dload,
                                        nullptr, D.T, (int32_t)D.a, (int32_t)D.k1, dc_p, dr_p, nullptr, nullptr, st));
        MOE_TRY(gate_weight_grads(D, x, dc_p, Wg, D.a, dWg, dX_gate, false, st));
        MOE_TRY(gate_weight_grads(D, x, dr_p, Wnoise, D.a, dWnoise, dX_gate, true, st));
        // secondary gates G_i, rows = slots (t, s1); dLoad_i of the row's group
        MOE_TRY(launch_gate_logit_grads(noise + lp, clean + lp, raw_noise + lp, w.H.idx_s, g_s, kth_vals + 2 * D.T,
                                        kth_idx + 2 * D.T, dg_s, dload + D.a, w.H.idx_p, P1, (int32_t)D.b,
                                        (int32_t)D.k2, dc_s, dr_s, nullptr, nullptr, st));
        for (int part = 0; part < 2; ++part) {
            const float *dl = part == 0 ? dc_s : dr_s;
            const float *W = (part == 0 ? Wg : Wnoise) + wp;
            float *dW = (part == 0 ? dWg : dWnoise) + wp;
            SimtGemm g;  // dW_s[i] = sum over the slots of group i of x[token]^T . dlogit[slot]
            memset(&g, 0, sizeof(g));
            g.ta = D.act == MOE_BF16 ? G_BF16 : G_F32; g.tb = G_F32; g.tc = G_F32;
            g.A = x; g.B = dl; g.C = dW;
            g.sa_i = 1; g.sa_k = D.d; g.sb_k = D.b; g.sb_j = 1; g.sc_i = D.b; g.sc_j = 1;
            g.mode = 1; g.offsets = w.H.offsets_p; g.nseg = (int32_t)D.a; g.M = D.d; g.N = D.b; g.c_e = D.d * D.b;
            g.a_row_index = w.H.perm_p; g.a_row_div = (int32_t)D.k1; g.b_row_index = w.H.perm_p;
            MOE_TRY(launch_simt_gemm(g, w.H.tile_prefix, st));
            memset(&g, 0, sizeof(g));  // dX_sec[slot] (+)= dlogit[slot] . W_s[group]^T
            g.ta = g.tb = g.tc = G_F32;
            g.A = dl; g.B = W; g.C = w.dX_sec; g.accumulate = part;
            g.sa_i = D.b; g.sa_k = 1; g.sb_k = 1; g.sb_j = D.b; g.sc_i = D.d; g.sc_j = 1;
            g.mode = 0; g.offsets = w.H.offsets_p; g.nseg = (int32_t)D.a; g.M = P1; g.N = D.d; g.K = D.b;
            g.b_e = D.d * D.b;
            g.a_row_index = w.H.perm_p; g.a_row_div = 1; g.c_row_index = w.H.perm_p;
            MOE_TRY(launch_simt_gemm(g, w.H.tile_prefix, st));
        }
        return launch_add_slot_rows(w.dX_sec, D.T, (int32_t)D.k1, (int32_t)D.d, dX_gate, st);
    }
    MOE_TRY(launch_gate_logit_grads(noise, clean, raw_noise, topk_idx, gates, kth_vals, kth_idx, dgates, dload,
                                    nullptr, D.T, (int32_t)D.n, (int32_t)D.k, w.dclean, w.draw, w.dsplit, nullptr,
                                    st));
    if (w.tc)
        return launch_tc_gate_bwd(x, D.T, (int32_t)D.d, (int32_t)D.n, Wg, Wnoise, w.dsplit, w.wsplit, w.partials, dWg,
                                  dWnoise, dX_gate, status_word(ws_base), st, D.flags);
    MOE_TRY(gate_weight_grads(D, x, w.dclean, Wg, D.n, dWg, dX_gate, false, st));
    return gate_weight_grads(D, x, w.draw, Wnoise, D.n, dWnoise, dX_gate, true, st);
}

}  // namespace

// ============================================================================ exported
extern "C" {

const char *moe_status_string(int32_t s) {
    switch (s) {
        case MOE_OK: return "ok";
        case MOE_ERR_INVALID_ARG: return "invalid argument";
        case MOE_ERR_UNSUPPORTED: return "unsupported configuration";
        case MOE_ERR_WORKSPACE: return "workspace too small";
        case MOE_ERR_CUDA: return "CUDA error";
        case MOE_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

int64_t moe_debug_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

int32_t moe_validate(const moe_config *cfg) { return check_config(cfg); }

int32_t moe_workspace_bytes(const moe_config *cfg, size_t *host_fwd, size_t *host_bwd) {
    moe_sizes s;
    MOE_TRY(moe_query_sizes(cfg, &s));
    if (host_fwd) *host_fwd = (size_t)s.ws_fwd_bytes;
    if (host_bwd) *host_bwd = (size_t)s.ws_bwd_bytes;
    return MOE_OK;
}

int32_t moe_query_sizes(const moe_config *cfg, moe_sizes *out) {
    MOE_TRY(check_config(cfg));
    if (!out) return MOE_ERR_INVALID_ARG;
    const Dims D = dims_of(cfg);
    out->R = D.R; out->gate_cols = D.gate_cols; out->logits_elems = D.logits; out->gates_elems = D.gates;
    out->kth_elems = D.kth; out->wg_elems = D.wg; out->load_elems = D.load; out->dload_elems = D.dload;
    const int64_t s_gate = measure([&](Carver &cv) { GateWs w(cv, D); (void)w; });
    const int64_t s_disp = measure([&](Carver &cv) { DispatchWs w(cv, D); (void)w; });
    const int64_t s_ffn = measure([&](Carver &cv) { FfnWs w(cv, D, cfg); (void)w; });
    const int64_t s_loss = measure([&](Carver &cv) { LossesWs w(cv, D); (void)w; });
    const int64_t s_fbwd = measure([&](Carver &cv) { FfnBwdWs w(cv, D); (void)w; });
    const int64_t s_lbwd = measure([&](Carver &cv) { LossesBwdWs w(cv, D); (void)w; });
    const int64_t s_gbwd = measure([&](Carver &cv) { GateBwdWs w(cv, D); (void)w; });
    int64_t fwd = s_gate;
    if (s_disp > fwd) fwd = s_disp;
    if (s_ffn > fwd) fwd = s_ffn;
    if (s_loss > fwd) fwd = s_loss;
    int64_t stage_bwd = s_fbwd;
    if (s_lbwd > stage_bwd) stage_bwd = s_lbwd;
    if (s_gbwd > stage_bwd) stage_bwd = s_gbwd;
    const int64_t s_fbwd_recompute = measure([&](Carver &cv) { FfnBwdWs w(cv, D); FfnWs f(cv, D, cfg); (void)w; (void)f; });
    if ((D.flags & MOE_FLAG_RECOMPUTE_HID) && s_fbwd_recompute > stage_bwd) stage_bwd = s_fbwd_recompute;
    out->adam_state_elems = D.n * (3 * D.d + 3 * D.h);
    out->ws_adam_bytes = kWsHeader + ((adam_ws_floats((int32_t)D.n, (int32_t)D.d, (int32_t)D.h) * 4 + 255) & ~(int64_t)255);
    out->ws_bytes = fwd > stage_bwd ? fwd : stage_bwd;
    out->ws_fwd_bytes = fwd;
    out->ws_bwd_bytes = measure([&](Carver &cv) { BwdWs w(cv, D); (void)w; }) + stage_bwd;
    Ctx ctx(nullptr, D, tc_ffn_supported(*cfg));
    out->ctx_bytes = ctx.bytes;
    return MOE_OK;
}

int32_t moe_query_ctx_layout(const moe_config *cfg, moe_ctx_layout *out) {
    MOE_TRY(check_config(cfg));
    if (!out) return MOE_ERR_INVALID_ARG;
    Ctx ctx(nullptr, dims_of(cfg), tc_ffn_supported(*cfg));
    *out = ctx.off;
    return MOE_OK;
}

int64_t moe_debug_bounds_violations(void) {
    const unsigned long long parts[] = {bounds_violations_route(), bounds_violations_losses(), bounds_violations_hier(),
                                        bounds_violations_gate(), bounds_violations_ffn()};
    unsigned long long sum = 0;
    for (unsigned long long v : parts) {
        if (v == ~0ull) return -1;
        sum += v;
    }
    return (int64_t)sum;
}

int32_t moe_debug_wait_timeout(void *ws, int64_t limit_ns, void *stream) {
    if (bad_ptr(ws) || limit_ns < 0 || limit_ns > 100000000) return MOE_ERR_INVALID_ARG;  // at most 0.1 s
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return launch_debug_wait(status_word(ws), (unsigned long long)limit_ns, as_stream(stream));
}

int32_t moe_check_buffer_sizes(const moe_config *cfg, int32_t which, size_t bytes) {
    moe_sizes s;
    MOE_TRY(moe_query_sizes(cfg, &s));
    int64_t need;
    switch (which) {
        case MOE_BUF_WS_STAGE: need = s.ws_bytes; break;
        case MOE_BUF_WS_FORWARD: need = s.ws_fwd_bytes; break;
        case MOE_BUF_WS_BACKWARD: need = s.ws_bwd_bytes; break;
        case MOE_BUF_CONTEXT: need = s.ctx_bytes; break;
        case MOE_BUF_WS_ADAM: need = s.ws_adam_bytes; break;
        default: return MOE_ERR_INVALID_ARG;
    }
    return (int64_t)bytes >= need ? MOE_OK : MOE_ERR_WORKSPACE;
}

int32_t moe_check_status(const void *ws, void *stream) {
    if (!ws) return MOE_ERR_INVALID_ARG;
    MOE_CUDA(cudaStreamSynchronize(as_stream(stream)));
    int32_t word = 0;
    MOE_CUDA(cudaMemcpy(&word, ws, sizeof(word), cudaMemcpyDeviceToHost));
    return word == 0 ? MOE_OK : MOE_ERR_TIMEOUT;
}

int32_t moe_gate(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise, const float *noise,
                 int32_t *topk_idx, float *gates, float *clean, float *raw_noise, float *kth_vals,
                 int32_t *kth_idx, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(x, Wg, Wnoise, noise, topk_idx, gates, clean, raw_noise, kth_vals, kth_idx, ws);
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return do_gate(cfg, D, x, Wg, Wnoise, noise, topk_idx, gates, clean, raw_noise, kth_vals, kth_idx, ws, cv,
                   as_stream(stream));
}

int32_t moe_dispatch(const moe_config *cfg, const void *x, const int32_t *topk_idx, void *xs, int32_t *perm,
                     int32_t *inv_perm, int32_t *counts, int32_t *offsets, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(x, topk_idx, xs, perm, inv_perm, counts, offsets, ws);
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    return do_dispatch(D, x, topk_idx, xs, perm, inv_perm, counts, offsets, cv, as_stream(stream));
}

int32_t moe_expert_ffn(const moe_config *cfg, const void *xs, const int32_t *offsets, const void *W1,
                       const void *b1, const void *W2, const void *b2, void *hid, void *ys, void *ws,
                       void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(xs, offsets, W1, b1, W2, b2, ys, ws);
    if (hid ? !aligned16(hid) : !(cfg->flags & MOE_FLAG_RECOMPUTE_HID)) return MOE_ERR_INVALID_ARG;
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return do_expert_ffn(cfg, D, xs, offsets, W1, b1, W2, b2, hid, ys, ws, cv, as_stream(stream));
}

int32_t moe_expert_ffn_bits(const moe_config *cfg, const void *xs, const int32_t *offsets, const void *W1,
                            const void *b1, const void *W2, const void *b2, void *hid, void *ys, uint32_t *relu_bits,
                            void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(xs, offsets, W1, b1, W2, b2, hid, ys, relu_bits, ws);
    if (!tc_ffn_supported(*cfg)) return MOE_ERR_UNSUPPORTED;
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return do_expert_ffn(cfg, D, xs, offsets, W1, b1, W2, b2, hid, ys, ws, cv, as_stream(stream), false, nullptr, relu_bits);
}

int32_t moe_expert_ffn_bwd_bits(const moe_config *cfg, const void *xs, const void *hid, const uint32_t *relu_bits,
                                const void *dys, const int32_t *offsets, const void *W1, const void *W2, void *dxs,
                                void *dW1, void *db1, void *dW2, void *db2, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(xs, hid, relu_bits, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws);
    if (!tc_ffn_supported(*cfg)) return MOE_ERR_UNSUPPORTED;
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return do_expert_ffn_bwd(cfg, D, xs, hid, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws, cv, as_stream(stream),
                             relu_bits);
}

int32_t moe_combine(const moe_config *cfg, const void *ys, const float *gates, const int32_t *inv_perm, void *y,
                    void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(ys, gates, inv_perm, y);
    return launch_combine(ys, cfg->act, gates, inv_perm, cfg->T, cfg->k, cfg->d, y, as_stream(stream));
}

int32_t moe_losses(const moe_config *cfg, const int32_t *topk_idx, const float *gates, const float *clean,
                   const float *raw_noise, const float *kth_vals, float *importance, float *load, float *losses,
                   void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(topk_idx, gates, clean, raw_noise, kth_vals, importance, load, losses, ws);
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    return do_losses(cfg, D, topk_idx, gates, clean, raw_noise, kth_vals, importance, load, losses, nullptr, nullptr, cv,
                     as_stream(stream));
}

int32_t moe_combine_bwd(const moe_config *cfg, const void *dY, const void *ys, const float *gates,
                        const int32_t *inv_perm, float *dgates, void *dys, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(dY, ys, gates, inv_perm, dgates, dys);
    return launch_combine_bwd(dY, ys, cfg->act, gates, inv_perm, cfg->T, cfg->k, cfg->d, dgates, dys,
                              as_stream(stream));
}

int32_t moe_expert_ffn_bwd(const moe_config *cfg, const void *xs, const void *hid, const void *dys,
                           const int32_t *offsets, const void *W1, const void *W2, void *dxs, void *dW1,
                           void *db1, void *dW2, void *db2, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(xs, hid, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws);
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return do_expert_ffn_bwd(cfg, D, xs, hid, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws, cv,
                             as_stream(stream));
}

int32_t moe_dispatch_bwd(const moe_config *cfg, const void *dxs, const int32_t *inv_perm, float *dX_expert,
                         void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(dxs, inv_perm, dX_expert);
    return launch_dispatch_bwd(dxs, cfg->act, inv_perm, cfg->T, cfg->k, cfg->d, nullptr, dX_expert, nullptr,
                               as_stream(stream));
}

int32_t moe_losses_bwd(const moe_config *cfg, const float *importance, const float *load,
                       const int32_t *topk_idx, float *dgates, float *dload, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(importance, load, topk_idx, dgates, dload, ws);
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    return do_losses_bwd(cfg, D, importance, load, topk_idx, dgates, dload, cv, as_stream(stream));
}

int32_t moe_gate_bwd(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise,
                     const float *noise, const float *clean, const float *raw_noise, const int32_t *topk_idx,
                     const float *gates, const float *kth_vals, const int32_t *kth_idx, float *dgates,
                     const float *dload, float *dWg, float *dWnoise, float *dX_gate, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(x, Wg, Wnoise, noise, clean, raw_noise, topk_idx, gates, kth_vals, kth_idx, dgates, dload, dWg,
                 dWnoise, dX_gate, ws);
    const Dims D = dims_of(cfg);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    MOE_TRY(reset_status(ws, as_stream(stream)));
    return do_gate_bwd(cfg, D, x, Wg, Wnoise, noise, clean, raw_noise, topk_idx, gates, kth_vals, kth_idx, dgates,
                       dload, dWg, dWnoise, dX_gate, ws, cv, as_stream(stream));
}

// keep_bits != nullptr: the output is that of the layer epilogue (sigmoid, dropout, residual) instead of Eq. 1 alone
static int32_t forward_impl(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise,
                            const float *noise, const void *W1, const void *b1, const void *W2, const void *b2,
                            const uint8_t *keep_bits, float drop_prob, void *y, float *losses, float *importance,
                            float *load, int32_t *counts, void *ctx, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(x, Wg, Wnoise, noise, W1, b1, W2, b2, y, losses, importance, load, counts, ctx, ws);
    if (keep_bits) MOE_TRY(check_layer(cfg, keep_bits, drop_prob));
    const Dims D = dims_of(cfg);
    cudaStream_t st = as_stream(stream);
    Ctx C(ctx, D, tc_ffn_supported(*cfg));
    MOE_TRY(reset_status(ws, st));
    auto fresh = [&]() { Carver cv(ws); cv.take_bytes(kWsHeader); return cv; };
    { Carver cv = fresh();
      MOE_TRY(do_gate(cfg, D, x, Wg, Wnoise, noise, C.topk_idx, C.gates, C.clean, C.raw_noise, C.kth_vals,
                      C.kth_idx, ws, cv, st)); }
    { Carver cv = fresh();
      MOE_TRY(do_dispatch(D, x, C.topk_idx, C.xs, C.perm, C.inv_perm, C.counts, C.offsets, cv, st)); }
    { Carver cv = fresh();
      MOE_TRY(do_expert_ffn(cfg, D, C.xs, C.offsets, W1, b1, W2, b2, C.hid, C.ys, ws, cv, st, false, nullptr,
                            C.relu_bits)); }  // C.hid null: stays in ws
    MOE_TRY(launch_combine(C.ys, D.act, C.gates, C.inv_perm, D.T, (int32_t)D.k, (int32_t)D.d, y, st,
                           keep_bits ? x : nullptr, keep_bits, keep_bits ? 1.0f / (1.0f - drop_prob) : 1.0f));
    { Carver cv = fresh();
      MOE_TRY(do_losses(cfg, D, C.topk_idx, C.gates, C.clean, C.raw_noise, C.kth_vals, C.importance, C.load,
                        C.losses, C.perm, C.offsets, cv, st)); }
    MOE_CUDA(cudaMemcpyAsync(losses, C.losses, 2 * sizeof(float), cudaMemcpyDeviceToDevice, st));
    MOE_CUDA(cudaMemcpyAsync(importance, C.importance, D.n * sizeof(float), cudaMemcpyDeviceToDevice, st));
    MOE_CUDA(cudaMemcpyAsync(load, C.load, D.load * sizeof(float), cudaMemcpyDeviceToDevice, st));
    MOE_CUDA(cudaMemcpyAsync(counts, C.counts, D.n * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return MOE_OK;
}

int32_t moe_forward(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise, const float *noise,
                    const void *W1, const void *b1, const void *W2, const void *b2, void *y, float *losses,
                    float *importance, float *load, int32_t *counts, void *ctx, void *ws, void *stream) {
    return forward_impl(cfg, x, Wg, Wnoise, noise, W1, b1, W2, b2, nullptr, 0.0f, y, losses, importance, load, counts,
                        ctx, ws, stream);
}

int32_t moe_layer_forward(const moe_config *cfg, const void *x, const float *Wg, const float *Wnoise,
                          const float *noise, const void *W1, const void *b1, const void *W2, const void *b2,
                          const uint8_t *keep_bits, float drop_prob, void *out, float *losses, float *importance,
                          float *load, int32_t *counts, void *ctx, void *ws, void *stream) {
    if (!keep_bits) return MOE_ERR_INVALID_ARG;
    return forward_impl(cfg, x, Wg, Wnoise, noise, W1, b1, W2, b2, keep_bits, drop_prob, out, losses, importance, load,
                        counts, ctx, ws, stream);
}

static int32_t backward_impl(const moe_config *cfg, const void *dY, const void *x, const float *Wg,
                             const float *Wnoise, const float *noise, const void *W1, const void *b1, const void *W2,
                             const void *b2, const uint8_t *keep_bits, float drop_prob, const void *ctx, void *dX,
                             float *dWg, float *dWnoise, void *dW1, void *db1, void *dW2, void *db2, void *ws,
                             void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(dY, x, Wg, Wnoise, noise, W1, b1, W2, b2, ctx, dX, dWg, dWnoise, dW1, db1, dW2, db2, ws);
    if (keep_bits) MOE_TRY(check_layer(cfg, keep_bits, drop_prob));
    const Dims D = dims_of(cfg);
    cudaStream_t st = as_stream(stream);
    Ctx C(const_cast<void *>(ctx), D, tc_ffn_supported(*cfg));
    MOE_TRY(reset_status(ws, st));
    Carver base(ws);
    base.take_bytes(kWsHeader);
    BwdWs B(base, D);
    auto fresh = [&]() { return base; };  // stage scratch starts after the tensors that live across stages
    MOE_TRY(launch_combine_bwd(dY, C.ys, D.act, C.gates, C.inv_perm, D.T, (int32_t)D.k, (int32_t)D.d, B.dgates,
                               B.dys, st, keep_bits, keep_bits ? 1.0f / (1.0f - drop_prob) : 1.0f));
    { Carver cv = fresh();
      const void *hid = C.hid;
      if (!hid) {  // MOE_FLAG_RECOMPUTE_HID: the forward kept no hidden activations; the first GEMM is run again
          FfnBwdWs skip(cv, D);  // the expert backward's own scratch comes first, the recomputed tensor behind it
          (void)skip;
          void *again = nullptr;
          MOE_TRY(do_expert_ffn(cfg, D, C.xs, C.offsets, W1, b1, W2, b2, nullptr, nullptr, ws, cv, st, true, &again));
          hid = again;
          cv = fresh();
      }
      MOE_TRY(do_expert_ffn_bwd(cfg, D, C.xs, hid, B.dys, C.offsets, W1, W2, B.dxs, dW1, db1, dW2, db2, ws, cv,
                                st, C.relu_bits)); }
    { Carver cv = fresh();
      MOE_TRY(do_losses_bwd(cfg, D, C.importance, C.load, C.topk_idx, B.dgates, B.dload, cv, st)); }
    { Carver cv = fresh();
      MOE_TRY(do_gate_bwd(cfg, D, x, Wg, Wnoise, noise, C.clean, C.raw_noise, C.topk_idx, C.gates, C.kth_vals,
                          C.kth_idx, B.dgates, B.dload, dWg, dWnoise, B.dX_gate, ws, cv, st)); }
    // dX = expert path + gating path (+ the upstream gradient itself through the residual connection)
    return launch_dispatch_bwd(B.dxs, D.act, C.inv_perm, D.T, (int32_t)D.k, (int32_t)D.d, B.dX_gate, nullptr, dX,
                               st, keep_bits ? dY : nullptr);
}

int32_t moe_backward(const moe_config *cfg, const void *dY, const void *x, const float *Wg, const float *Wnoise,
                     const float *noise, const void *W1, const void *b1, const void *W2, const void *b2,
                     const void *ctx, void *dX, float *dWg, float *dWnoise, void *dW1, void *db1, void *dW2,
                     void *db2, void *ws, void *stream) {
    return backward_impl(cfg, dY, x, Wg, Wnoise, noise, W1, b1, W2, b2, nullptr, 0.0f, ctx, dX, dWg, dWnoise, dW1, db1,
                         dW2, db2, ws, stream);
}

int32_t moe_layer_backward(const moe_config *cfg, const void *dOut, const void *x, const float *Wg,
                           const float *Wnoise, const float *noise, const void *W1, const void *b1, const void *W2,
                           const void *b2, const uint8_t *keep_bits, float drop_prob, const void *ctx, void *dX,
                           float *dWg, float *dWnoise, void *dW1, void *db1, void *dW2, void *db2, void *ws,
                           void *stream) {
    if (!keep_bits) return MOE_ERR_INVALID_ARG;
    return backward_impl(cfg, dOut, x, Wg, Wnoise, noise, W1, b1, W2, b2, keep_bits, drop_prob, ctx, dX, dWg, dWnoise,
                         dW1, db1, dW2, db2, ws, stream);
}

int32_t moe_expert_adam_factored(const moe_config *cfg, void *W1, void *b1, void *W2, void *b2, const void *dW1,
                                 const void *db1, const void *dW2, const void *db2, float *state, float lr,
                                 float beta2, float eps, int32_t step, void *ws, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(W1, b1, W2, b2, dW1, db1, dW2, db2, state, ws);
    if (!(lr >= 0.0f) || !(beta2 >= 0.0f) || !(beta2 < 1.0f) || !(eps >= 0.0f) || step < 1) return MOE_ERR_INVALID_ARG;
    return launch_expert_adam(cfg->act, cfg->n, cfg->d, cfg->h, W1, b1, W2, b2, dW1, db1, dW2, db2, state, lr, beta2, eps,
                              step, reinterpret_cast<float *>(static_cast<char *>(ws) + kWsHeader), as_stream(stream));
}

// ---------------------------------------------------------------------------- strictly balanced gating (Appendix F)
static int32_t check_balanced(const moe_config *c) {
    MOE_TRY(check_config(c));
    if (c->a > 0) return MOE_ERR_UNSUPPORTED;                       // flat layers only
    if (c->T > 0 && ((int64_t)c->T * c->k) % c->n != 0) return MOE_ERR_INVALID_ARG;  // m = k T / n must be whole
    return MOE_OK;
}

int32_t moe_query_balanced_sizes(const moe_config *cfg, moe_balanced_sizes *out) {
    MOE_TRY(check_balanced(cfg));
    if (!out) return MOE_ERR_INVALID_ARG;
    out->m = (int64_t)cfg->T * cfg->k / cfg->n;
    out->R = (int64_t)cfg->T * cfg->k;
    out->mask_words = (cfg->n + 31) / 32;
    const int64_t fwd = balanced_ws_bytes(cfg->T, cfg->n);
    const int64_t bwd = measure([&](Carver &cv) {   // the larger of the two ways moe_gate_balanced_bwd carves
        cv.take<bf16>((int64_t)cfg->T * 3 * cfg->n); cv.take<bf16>((int64_t)cfg->d * 3 * cfg->n);
        cv.take<float>(tc_gate_bwd_partials(cfg->T, cfg->d, cfg->n / 2 > 0 ? cfg->n / 2 : 1));
        cv.take<float>((int64_t)cfg->T * cfg->n);
    });
    out->ws_bytes = kWsHeader + (fwd > bwd ? fwd : bwd);
    return MOE_OK;
}

int32_t moe_gate_balanced(const moe_config *cfg, const void *x, const float *Wg, const float *thresholds, float *logits,
                          float *probs, uint32_t *mask_bits, int32_t *tok_of_row, int32_t *offsets, float *den,
                          int32_t *tok_ptr, int32_t *tok_rows, float *loss_batchwise, int32_t *thr_counts, void *ws,
                          void *stream) {
    MOE_TRY(check_balanced(cfg));
    REQUIRE_PTRS(x, Wg, thresholds, logits, probs, mask_bits, tok_of_row, offsets, den, tok_ptr, tok_rows, loss_batchwise,
                 thr_counts, ws);
    return launch_balanced_gate(x, cfg->act, cfg->T, cfg->d, cfg->n, cfg->k, Wg, thresholds, logits, probs, mask_bits,
                                tok_of_row, offsets, den, tok_ptr, tok_rows, loss_batchwise, thr_counts,
                                static_cast<char *>(ws) + kWsHeader, as_stream(stream));
}

int32_t moe_dispatch_balanced(const moe_config *cfg, const void *x, const int32_t *tok_of_row, void *xs, void *stream) {
    MOE_TRY(check_balanced(cfg));
    REQUIRE_PTRS(x, tok_of_row, xs);
    return launch_balanced_gather(x, cfg->act, tok_of_row, (int64_t)cfg->T * cfg->k, cfg->T, cfg->d, xs, as_stream(stream));
}

int32_t moe_combine_balanced(const moe_config *cfg, const void *ys, const float *probs, const float *den,
                             const int32_t *tok_ptr, const int32_t *tok_rows, void *y, void *stream) {
    MOE_TRY(check_balanced(cfg));
    REQUIRE_PTRS(ys, probs, den, tok_ptr, tok_rows, y);
    const int64_t R = (int64_t)cfg->T * cfg->k;
    return launch_balanced_combine(ys, cfg->act, probs, den, tok_ptr, tok_rows, cfg->T, R, cfg->n, (int32_t)(R / cfg->n),
                                   cfg->d, y, as_stream(stream));
}

int32_t moe_combine_balanced_bwd(const moe_config *cfg, const void *dY, const void *ys, const float *probs,
                                 const float *den, const int32_t *tok_of_row, float *dG_row, void *dys, void *stream) {
    MOE_TRY(check_balanced(cfg));
    REQUIRE_PTRS(dY, ys, probs, den, tok_of_row, dG_row, dys);
    const int64_t R = (int64_t)cfg->T * cfg->k;
    return launch_balanced_combine_bwd(dY, ys, cfg->act, probs, den, tok_of_row, R, cfg->T, cfg->n, (int32_t)(R / cfg->n),
                                       cfg->d, dG_row, dys, as_stream(stream));
}

int32_t moe_gate_balanced_bwd(const moe_config *cfg, const void *x, const float *Wg, const float *probs,
                              const uint32_t *mask_bits, const float *den, const float *thresholds,
                              const int32_t *tok_ptr, const int32_t *tok_rows, const float *dG_row,
                              const int32_t *thr_counts, float w_batchwise, float *dWg, float *dX_gate,
                              float *dthresholds, void *ws, void *stream) {
    MOE_TRY(check_balanced(cfg));
    REQUIRE_PTRS(x, Wg, probs, mask_bits, den, thresholds, tok_ptr, tok_rows, dG_row, thr_counts, dWg, dX_gate, dthresholds,
                 ws);
    const Dims D = dims_of(cfg);
    cudaStream_t st = as_stream(stream);
    Carver cv(ws);
    cv.take_bytes(kWsHeader);
    // the two contractions on the tensor cores (three-term bf16 splits, as in moe_gate_bwd) when the shapes allow: the
    // n logit columns are handled as the two column halves of one [d, n] matrix
    const int32_t half = (int32_t)(D.n / 2);
    const bool tc = D.n % 2 == 0 && D.T > 0 && tc_gate_bwd_supported(D.act, (int32_t)D.d, half);
    if (tc) {
        void *dsplit = cv.take<bf16>(D.T * 3 * D.n);
        void *wsplit = cv.take<bf16>(D.d * 3 * D.n);
        float *partials = cv.take<float>(tc_gate_bwd_partials(D.T, (int32_t)D.d, half));
        MOE_TRY(reset_status(ws, st));
        MOE_TRY(launch_balanced_gate_bwd(probs, mask_bits, den, thresholds, tok_ptr, tok_rows, dG_row, thr_counts,
                                         w_batchwise, D.T, (int32_t)D.n, (int32_t)(D.R / D.n), nullptr, dsplit, dthresholds,
                                         st));
        return launch_tc_gate_bwd(x, D.T, (int32_t)D.d, half, Wg, Wg + half, dsplit, wsplit, partials, dWg, dWg + half, dX_gate,
                                  status_word(ws), st, D.flags, (int32_t)D.n);
    }
    float *dc = cv.take<float>(D.T * D.n);
    MOE_TRY(launch_balanced_gate_bwd(probs, mask_bits, den, thresholds, tok_ptr, tok_rows, dG_row, thr_counts, w_batchwise,
                                     D.T, (int32_t)D.n, (int32_t)(D.R / D.n), dc, nullptr, dthresholds, st));
    if (D.T == 0) {
        MOE_CUDA(cudaMemsetAsync(dWg, 0, sizeof(float) * D.d * D.n, st));
        return MOE_OK;
    }
    return gate_weight_grads(D, x, dc, Wg, D.n, dWg, dX_gate, false, st);
}

int32_t moe_dispatch_balanced_bwd(const moe_config *cfg, const void *dxs, const int32_t *tok_ptr,
                                  const int32_t *tok_rows, const float *dX_gate, void *dX, void *stream) {
    MOE_TRY(check_balanced(cfg));
    REQUIRE_PTRS(dxs, tok_ptr, tok_rows, dX_gate, dX);
    return launch_balanced_dispatch_bwd(dxs, cfg->act, tok_ptr, tok_rows, dX_gate, cfg->T, (int64_t)cfg->T * cfg->k, cfg->d,
                                        dX, as_stream(stream));
}

int32_t moe_combine_layer(const moe_config *cfg, const void *ys, const float *gates, const int32_t *inv_perm,
                          const void *x, const uint8_t *keep_bits, float drop_prob, void *out, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(ys, gates, inv_perm, x, out);
    MOE_TRY(check_layer(cfg, keep_bits, drop_prob));
    return launch_combine(ys, cfg->act, gates, inv_perm, cfg->T, cfg->k, cfg->d, out, as_stream(stream), x, keep_bits,
                          1.0f / (1.0f - drop_prob));
}

int32_t moe_combine_layer_bwd(const moe_config *cfg, const void *dOut, const void *ys, const float *gates,
                              const int32_t *inv_perm, const uint8_t *keep_bits, float drop_prob, float *dgates,
                              void *dys, void *stream) {
    MOE_TRY(check_config(cfg));
    REQUIRE_PTRS(dOut, ys, gates, inv_perm, dgates, dys);
    MOE_TRY(check_layer(cfg, keep_bits, drop_prob));
    return launch_combine_bwd(dOut, ys, cfg->act, gates, inv_perm, cfg->T, cfg->k, cfg->d, dgates, dys,
                              as_stream(stream), keep_bits, 1.0f / (1.0f - drop_prob));
}

}  // extern "C"
