"""Parity at the full benchmark sizes, in the launch configuration bench.py times (fused calls).

The oracle cannot run the expert GEMMs of these batches in reasonable time, so:
  - everything integer (routing, order statistics, dispatch permutation, counts) and every gating
    tensor (gates, Importance, Load, losses) is compared IN FULL: the oracle's gate and loss code
    handles the whole batch;
  - expert-side outputs are compared on samples the oracle computes one by one: y and dX of sampled
    tokens (each token's experts are evaluated on that token alone, which is exact because the
    experts act row by row), the complete weight / bias gradients of two small experts (every row
    of those experts is evaluated), and, for the LARGEST expert (the longest contraction the weight-gradient
    GEMMs see), the gradients of a sample of its hidden units spread over every 256-wide tile: the expert
    restricted to those units is itself a one-hidden-layer expert whose hid, dW1[:, J], db1[J], dW2[J, :]
    and db2 are exactly the full expert's slices, so the oracle evaluates that smaller network on all rows;
  - the gate backward is compared in full through its stage call, fed with the oracle's gate state
    (flat and hierarchical).
"""
import numpy as np
import pytest
import torch

import bench
from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import TOL_BF16, TOL_F32, assert_close, cat_parts, f32, host
from test_gpu_hier import gate_tensors

pytestmark = pytest.mark.gpu

N_TOKENS = 48
MAX_FLIP_RATE = 2e-5   # share of ReLU decisions that may differ (pre-activation within rounding of zero)
UNITS_PER_TILE = 16    # hidden units of the largest expert sampled in every 256-wide tile
DROP = 0.1             # DropProb of the layer epilogue check


def slice_gate(G, rows):
    from types import SimpleNamespace as NS
    return NS(**{k: getattr(G, k)[rows] for k in ("idx", "gates", "clean", "raw", "sigma", "H", "kth_val", "kth_idx")})


@pytest.mark.parametrize("name", ["c3", "c4", "c5"])
def test_full_size_fused(name):
    w = synth.CONFIGS[name]
    cfg, S, D, hostI = bench.build_device_state(w, keep_host_experts=False)
    B.moe_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], D["y"],
                  D["losses"], D["importance"], D["load"], D["counts"], D["ctx"], D["ws"])
    B.moe_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], D["ctx"],
                   D["dX"], D["dWg"], D["dWnoise"], D["dW1"], D["db1"], D["dW2"], D["db2"], D["ws"])
    assert B.moe_check_status(D["ws"]) == 0
    V = B.ctx_views(cfg, D["ctx"])
    x, dY = hostI["x"], hostI["dY"]
    Wg, Wn, noise = hostI["Wg"], hostI["Wnoise"], hostI["noise"]
    hier = w.hier
    # ---------------- gating, in full
    if hier is None:
        G = O.gate(x, Wg, Wn, noise, w.k, "bf16")
        LS = O.losses(G.idx, G.gates, G.clean, G.raw, G.kth_val, w.w_importance, w.w_load, "bf16")
        want_gates, want_kidx = G.gates.reshape(-1), G.kth_idx.reshape(-1)
    else:
        G = O.gate_h(x, Wg[0], Wn[0], noise[0], Wg[1], Wn[1], noise[1], w.k1, w.k2, "bf16")
        LS = O.losses_h(G, w.a, w.b, w.w_importance, w.w_load, "bf16")
        GT = gate_tensors(G)
        want_gates, want_kidx = GT["gates"], GT["kth_idx"]
    Dp = O.dispatch(np.zeros((w.T, 1), np.float32), G.idx, w.n)
    assert (host(V["topk_idx"]) == G.idx).all(), "routing must be bit-exact"
    assert (host(V["kth_idx"]).reshape(-1) == want_kidx).all()
    assert (host(D["counts"]) == Dp.counts).all() and (host(V["offsets"]) == Dp.offsets).all()
    assert (host(V["perm"]) == Dp.perm).all() and (host(V["inv_perm"]) == Dp.inv_perm).all()
    assert_close(host(V["gates"]), want_gates, TOL_F32, "gates")
    assert_close(host(D["importance"]), LS.importance, TOL_F32, "importance")
    assert_close(host(D["load"])[:w.n], LS.load, TOL_F32, "load")
    assert_close(host(D["losses"]), LS.losses, TOL_F32, "losses")
    xs_rows = host(V["xs"][torch.from_numpy(np.arange(0, S.R, max(1, S.R // 97))).cuda()])
    assert (xs_rows == x[Dp.perm[np.arange(0, S.R, max(1, S.R // 97))] // w.k]).all()

    # ---------------- sampled tokens: y and dX
    g = np.random.default_rng(7)
    first_of_big, last_of_small = Dp.perm[Dp.offsets[np.argmax(Dp.counts)]] // w.k, Dp.perm[-1] // w.k
    toks = np.unique(np.concatenate([g.choice(w.T, N_TOKENS, replace=False), [0, w.T - 1, first_of_big, last_of_small]]))
    experts = np.unique(G.idx[toks])
    local = {int(e): i for i, e in enumerate(experts)}
    Wl = [synth.make_expert(w, int(e)) for e in experts]
    W1, b1, W2, b2 = (np.stack([p[i] for p in Wl]) for i in range(4))
    idx_l = np.vectorize(local.get)(G.idx[toks]).astype(np.int32)
    Ds = O.dispatch(x[toks], idx_l, len(experts))
    hid, ys = O.expert_ffn(Ds.xs, Ds.offsets, W1, b1, W2, b2, "bf16")
    y = O.combine(ys, G.gates[toks], Ds.inv_perm, "bf16")
    assert_close(host(D["y"])[toks], y, TOL_BF16, "y (sampled tokens)")
    # the layer epilogue (sigmoid, dropout, residual) at this size, through its stage calls on the saved context:
    # the oracle evaluates the sampled tokens from scratch
    keep_bits = synth.make_keep_bits(w, DROP)
    keep = O.unpack_keep(keep_bits[toks], w.d)
    out_d = torch.empty_like(D["y"])
    kb_d = torch.from_numpy(keep_bits).cuda()
    B.moe_combine_layer(cfg, V["ys"], V["gates"][:w.T * w.k], V["inv_perm"], D["x"], kb_d, DROP, out_d)
    want_out = O.combine_layer(ys, G.gates[toks], Ds.inv_perm, x[toks], keep, DROP, "bf16")
    assert_close(host(out_d)[toks], want_out, TOL_BF16, "layer output (sampled tokens)")
    got_out = host(out_d)[toks]
    assert (got_out[~keep] == np.asarray(x[toks], np.float32)[~keep]).all(), "a dropped activation leaves the residual alone"
    dg, dys = O.combine_bwd(dY[toks], ys, G.gates[toks], Ds.inv_perm, "bf16")
    E = O.expert_ffn_bwd(Ds.xs, hid, dys, Ds.offsets, W1, W2, "bf16")
    dX_exp = O.dispatch_bwd(E.dxs, Ds.inv_perm, len(toks), w.k, "bf16")
    if hier is None:
        dg2, dload = O.losses_bwd(LS.importance, LS.load, G.idx[toks], dg, w.w_importance, w.w_load, "bf16")
        dc, dr = O.gate_logit_grads(noise[toks], G.clean[toks], G.raw[toks], G.idx[toks], G.gates[toks],
                                    G.kth_val[toks], G.kth_idx[toks], dg2, dload, "bf16")
        dXg = dc @ Wg.astype(np.float64).T + dr @ Wn.astype(np.float64).T
    else:
        from types import SimpleNamespace as NS
        Gs = NS(idx=G.idx[toks], gates=G.gates[toks], primary=slice_gate(G.primary, toks),
                secondary=slice_gate(G.secondary, toks))
        GB = O.gate_h_bwd(x[toks], Wg[0], Wn[0], noise[0][toks], Wg[1], Wn[1], noise[1][toks], Gs, LS, dg,
                          w.w_importance, w.w_load, "bf16")
        dXg = np.asarray(GB.dX_gate, np.float64)
    dX = O.store(np.asarray(dX_exp, np.float64) + dXg, "bf16", expert_side=True)
    got_hid = host(V["hid"][torch.from_numpy(Dp.inv_perm.reshape(w.T, w.k)[toks].reshape(-1).astype(np.int64)).cuda()])
    want_hid = np.asarray(hid)[Ds.inv_perm]
    assert_close(got_hid, want_hid, TOL_BF16, "hid (sampled rows)")
    flips = (got_hid > 0) != (want_hid > 0)   # ReLU decisions within rounding of 0: rare, and their tokens set aside
    assert flips.sum() <= max(2, MAX_FLIP_RATE * flips.size), int(flips.sum())
    clean_rows = ~flips.reshape(len(toks), -1).any(axis=1)
    assert_close(host(D["dX"])[toks][clean_rows], dX[clean_rows], TOL_BF16, "dX (sampled tokens)")

    # ---------------- experts: two small ones and an empty one in full, the largest one on sampled hidden units
    order = np.argsort(Dp.counts, kind="stable")
    small = [int(e) for e in order if Dp.counts[e] > 0][:2]
    largest = int(np.argmax(Dp.counts))
    gu = np.random.default_rng(9)
    units_big = np.unique(np.concatenate([np.concatenate([[c0, c0 + 255], c0 + gu.choice(256, UNITS_PER_TILE - 2, False)])
                                          for c0 in range(0, w.h, 256)]))
    for e, units in [(e, None) for e in small + [int(e) for e in order if Dp.counts[e] == 0][:1]] + [(largest, units_big)]:
        got = {k2: host(D[k2][e]) for k2 in ("dW1", "db1", "dW2", "db2")}
        if Dp.counts[e] == 0:
            assert all(np.abs(v).max() == 0 for v in got.values()), "an expert without rows has zero gradients"
            continue
        slots = Dp.perm[Dp.offsets[e]:Dp.offsets[e + 1]]
        t_e, s_e = slots // w.k, slots % w.k
        W1e, b1e, W2e, b2e = synth.make_expert(w, e)
        if units is None:
            units = np.arange(w.h)
        W1e, b1e, W2e = W1e[:, units], b1e[units], W2e[units, :]   # the expert restricted to these hidden units
        offs = np.array([0, len(slots)], np.int32)
        hid_e, _ = O.expert_ffn(x[t_e], offs, W1e[None], b1e[None], W2e[None], b2e[None], "bf16")
        dys_e = O.store(np.asarray(G.gates, np.float64)[t_e, s_e][:, None] * dY[t_e].astype(np.float64), "bf16", True)
        Ee = O.expert_ffn_bwd(x[t_e], hid_e, dys_e, offs, W1e[None], W2e[None], "bf16")
        got_hid_e = host(V["hid"][int(Dp.offsets[e]):int(Dp.offsets[e + 1])])[:, units]
        assert_close(got_hid_e, hid_e, TOL_BF16, f"hid[{e}]")
        flips_e = (got_hid_e > 0) != (np.asarray(hid_e) > 0)
        assert flips_e.sum() <= max(2, MAX_FLIP_RATE * flips_e.size), (e, int(flips_e.sum()))
        keep_cols = ~flips_e.any(axis=0)
        assert_close(got["dW2"][units, :], Ee.dW2[0], TOL_BF16, f"dW2[{e}]")
        assert_close(got["db2"], Ee.db2[0], TOL_BF16, f"db2[{e}]")
        assert_close(got["dW1"][:, units][:, keep_cols], Ee.dW1[0][:, keep_cols], TOL_BF16, f"dW1[{e}]")
        assert_close(got["db1"][units][keep_cols], Ee.db1[0][keep_cols], TOL_BF16, f"db1[{e}]")

    # ---------------- gate backward in full, through its stage call, fed with the oracle's gate state
    gd = np.random.default_rng(8)
    dgates = gd.standard_normal((w.T, w.k)).astype(np.float32)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    dWg, dWn, dXg_d = f32(S.wg_elems), f32(S.wg_elems), f32(w.T, w.d)
    if hier is None:
        dload = (gd.standard_normal(w.n) * 1e-3).astype(np.float32)
        GBf = O.gate_bwd(x, Wg, Wn, noise, G.clean, G.raw, G.idx, G.gates, G.kth_val, G.kth_idx, dgates, dload, "bf16")
        B.moe_gate_bwd(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], dev(G.clean), dev(G.raw), dev(G.idx),
                       dev(G.gates), dev(G.kth_val), dev(G.kth_idx), dev(dgates), dev(dload), dWg, dWn, dXg_d, D["ws"])
        want_dWg, want_dWn, want_dXg = GBf.dWg, GBf.dWnoise, GBf.dX_gate
    else:
        # both levels: the upstream gradients of the stage call are the oracle's own (product-gate gradient with the
        # Importance term added, d/dLoad of both levels from Eq. 14), so the gate backward is compared alone
        a_, b_ = w.a, w.b
        dI = w.w_importance * O.cv_squared_grad(LS.importance)
        dLH = (w.w_load * O.cv_squared_grad(LS.load)).reshape(a_, b_)
        safe = np.where(LS.cnt > 0, LS.cnt, 1.0)
        live = (LS.cnt > 0)[:, None]
        dload = np.concatenate([np.where(live, dLH * LS.load_s / safe[:, None], 0).sum(1),
                                np.where(live, dLH * LS.load_p[:, None] / safe[:, None], 0).reshape(-1)]).astype(np.float32)
        GBh = O.gate_h_bwd(x, Wg[0], Wn[0], noise[0], Wg[1], Wn[1], noise[1], G, LS, dgates, w.w_importance, w.w_load,
                           "bf16")
        dg = torch.zeros(S.gates_elems, device="cuda")
        dg[:w.T * w.k] = dev((dgates.astype(np.float64) + dI[G.idx]).astype(np.float32)).reshape(-1)
        B.moe_gate_bwd(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], dev(GT["clean"]), dev(GT["raw"]),
                       dev(GT["topk_idx"]), dev(GT["gates"]), dev(GT["kth_vals"]), dev(GT["kth_idx"]), dg, dev(dload),
                       dWg, dWn, dXg_d, D["ws"])
        want_dWg, want_dWn = cat_parts((GBh.dWg_p, GBh.dWg_s)), cat_parts((GBh.dWn_p, GBh.dWn_s))
        want_dXg = GBh.dX_gate
    assert B.moe_check_status(D["ws"]) == 0
    assert_close(host(dWg), want_dWg, TOL_F32, "dWg (full)")
    assert_close(host(dWn), want_dWn, TOL_F32, "dWnoise (full)")
    # The uneven-load workloads route a constant feature through W_g[0, :] with offsets up to ~4 while
    # sum_j dclean_j ~ 0: that column of dX_gate is a cancelling sum, and fp32 accumulation (any order)
    # leaves ~1e-5 of the result there; the mean error stays at the 1e-7 level.
    assert_close(host(dXg_d), want_dXg, dict(max=5e-5, mean=1e-6), "dX_gate (full)")


REPEATS = {"c3": 40, "c4": 20, "c5": 60}


@pytest.mark.parametrize("name", ["c3", "c4", "c5"])
def test_full_size_repeated_steps_agree_bit_for_bit(name):
    """Tiles are handed to the SM pairs at run time, so which pair computes a tile changes from run to run; the
    result must not. Every output of the fused step and the saved context is compared byte for byte with the first
    run. The forward between two backward passes overwrites the workspace, so a piece of a backward tensor that a
    run fails to write shows up as different bytes instead of hiding behind the previous run's identical values."""
    w = synth.CONFIGS[name]
    cfg, S, D, _ = bench.build_device_state(w, keep_host_experts=False)
    outs = ("y", "losses", "importance", "load", "counts", "dX", "dWg", "dWnoise", "dW1", "db1", "dW2", "db2")

    def step():
        B.moe_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], D["y"],
                      D["losses"], D["importance"], D["load"], D["counts"], D["ctx"], D["ws"])
        B.moe_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"],
                       D["ctx"], D["dX"], D["dWg"], D["dWnoise"], D["dW1"], D["db1"], D["dW2"], D["db2"], D["ws"])
        torch.cuda.synchronize()
        assert B.moe_check_status(D["ws"]) == 0

    step()
    first = {k: D[k].clone() for k in outs}
    first_ctx = D["ctx"].clone()
    for it in range(REPEATS[name]):
        step()
        differing = [k for k in outs if not torch.equal(first[k].view(torch.uint8), D[k].view(torch.uint8))]
        if not torch.equal(first_ctx.view(torch.uint8), D["ctx"].view(torch.uint8)):
            differing.append("ctx")
        assert not differing, f"run {it + 1} differs from the first in {differing}"


def test_full_size_balanced_gate():
    """Strictly balanced gating at the bench's widest workload: logits, batchwise masks, row tables and per-token lists
    bit for bit against the oracle (its gate handles the whole batch), probabilities, denominators and L_batchwise at the
    gating tolerance, every expert with exactly m rows."""
    w = synth.CONFIGS["c5"]
    x, Wg = synth.make_x(w), synth.make_gate(w)[0]
    logits, p = O.softmax_gate(x, Wg, "bf16")
    m = w.T * w.k // w.n
    srt = -np.sort(-np.asarray(p, np.float64), axis=0)
    thr = (srt[m - 1] * (1 + 0.05 * np.random.default_rng(5).standard_normal(w.n))).astype(np.float32)
    mask = O.batchwise_mask(p, m)
    G_want, den = O.masked_gate(p, mask, "bf16")
    Dw = O.dispatch_balanced(x, mask)
    loss = O.batchwise_loss(p, mask, thr)
    cfg = B.make_config(w.T, w.d, w.h, w.n, w.k, w.act, w.w_importance, w.w_load)
    S = B.moe_query_balanced_sizes(cfg)
    assert S.m == m
    e = lambda *s_, dt=torch.float32: torch.empty(*s_, dtype=dt, device="cuda")
    out = dict(logits=e(w.T, w.n), probs=e(w.T, w.n), mask_bits=e(w.T, S.mask_words, dt=torch.int32),
               tok_of_row=e(S.R, dt=torch.int32), offsets=e(w.n + 1, dt=torch.int32), den=e(w.T),
               tok_ptr=e(w.T + 1, dt=torch.int32), tok_rows=e(S.R, dt=torch.int32), loss=e(1),
               thr_counts=e(w.n, dt=torch.int32), ws=B.empty_bytes(S.ws_bytes))
    B.moe_gate_balanced(cfg, torch.from_numpy(x).to(torch.bfloat16).cuda(), torch.from_numpy(Wg).cuda(),
                        torch.from_numpy(thr).cuda(), out["logits"], out["probs"], out["mask_bits"], out["tok_of_row"],
                        out["offsets"], out["den"], out["tok_ptr"], out["tok_rows"], out["loss"], out["thr_counts"], out["ws"])
    assert (host(out["logits"]) == np.asarray(logits)).all(), "logits by the fixed fma chain"
    assert_close(host(out["probs"]), p, TOL_F32, "probs")
    bits = np.packbits(mask, axis=1, bitorder="little")
    assert (host(out["mask_bits"]).view(np.uint8).reshape(w.T, -1)[:, :bits.shape[1]] == bits).all(), "batchwise mask"
    assert (host(out["offsets"]) == np.arange(w.n + 1) * m).all(), "every expert gets exactly m rows"
    assert (host(out["tok_of_row"]) == Dw.tok_of_row).all()
    ptr = np.zeros(w.T + 1, np.int64)
    np.add.at(ptr, Dw.tok_of_row.astype(np.int64) + 1, 1)
    assert (host(out["tok_ptr"]) == np.cumsum(ptr)).all()
    assert (host(out["tok_rows"]) == np.lexsort((Dw.expert_of_row, Dw.tok_of_row))).all()
    assert_close(host(out["den"]), den, TOL_F32, "den")
    assert (host(out["thr_counts"]) == O.threshold_mask(p, thr).sum(axis=0)).all()
    assert_close(host(out["loss"]), loss, TOL_F32, "L_batchwise")


def test_full_size_factored_adam():
    """The optimiser step on all 128 experts of the widest workload (2.1 GB of weights and as much of gradients); the
    oracle steps three of them: the first, one in the middle, the last."""
    w = synth.CONFIGS["c5"]
    cfg = B.make_config(w.T, w.d, w.h, w.n, w.k, w.act, w.w_importance, w.w_load)
    S = B.moe_query_sizes(cfg)
    gen = torch.Generator(device="cuda").manual_seed(11)
    bf = torch.bfloat16
    rnd = lambda *s_, scale=1.0: (torch.randn(*s_, device="cuda", generator=gen) * scale).to(bf)
    W1, b1, W2, b2 = rnd(w.n, w.d, w.h, scale=0.03), rnd(w.n, w.h, scale=0.1), rnd(w.n, w.h, w.d, scale=0.02), rnd(w.n, w.d, scale=0.1)
    # gradients with a row structure so that the factored estimate matters
    g1 = (torch.randn(w.n, w.d, w.h, device="cuda", generator=gen) * (1 + 3 * torch.rand(w.n, w.d, 1, device="cuda", generator=gen))).to(bf)
    g2 = (torch.randn(w.n, w.h, w.d, device="cuda", generator=gen) * (1 + 3 * torch.rand(w.n, w.h, 1, device="cuda", generator=gen))).to(bf)
    gb1, gb2 = rnd(w.n, w.h), rnd(w.n, w.d)
    state = torch.rand(S.adam_state_elems, device="cuda", generator=gen) + 0.5   # a running state, not the first step
    picks = [0, w.n // 2, w.n - 1]
    f = lambda t: t.float().cpu().numpy()
    before = {e_: [f(a[e_]) for a in (W1, b1, W2, b2, g1, gb1, g2, gb2)] for e_ in picks}
    st0 = f(state)
    sizes = [("r1", w.d), ("c1", w.h), ("r2", w.h), ("c2", w.d), ("vb1", w.h), ("vb2", w.d)]
    parts, at = {}, 0
    for name, width in sizes:
        parts[name] = st0[at:at + w.n * width].reshape(w.n, width)
        at += w.n * width
    lr, beta2, eps, step = 1e-2, 0.99, 1e-8, 7
    B.moe_expert_adam_factored(cfg, W1, b1, W2, b2, g1, gb1, g2, gb2, state, lr, beta2, eps, step, B.empty_bytes(S.ws_adam_bytes))
    torch.cuda.synchronize()
    st1, at, got_parts = f(state), 0, {}
    for name, width in sizes:
        got_parts[name] = st1[at:at + w.n * width].reshape(w.n, width)
        at += w.n * width
    for e_ in picks:
        a = before[e_]
        one = {k_: v_[e_:e_ + 1] for k_, v_ in parts.items()}
        want = O.expert_adam_factored(a[0][None], a[1][None], a[2][None], a[3][None], a[4][None], a[5][None], a[6][None],
                                      a[7][None], one, lr, beta2, eps, step, "bf16")
        for name, got, exp in zip(("W1", "b1", "W2", "b2"), (W1, b1, W2, b2), want[:4]):
            assert_close(f(got[e_]), exp[0], TOL_BF16, f"{name} of expert {e_}")
        for name, _ in sizes:
            assert_close(got_parts[name][e_], np.asarray(want[4][name])[0], TOL_F32, f"state {name} of expert {e_}")
