"""Stage-by-stage parity of the CUDA library against the CPU oracle, through the C ABI.

Each stage gets the ORACLE's upstream tensors as inputs, so one kernel is tested at a time:
indices and permutations bit-exact, fp32 gating tensors within 1e-5, expert-side tensors within
1e-5 (fp32 layer) or 2e-2 max / 1e-2 mean (bf16 layer), in the rms-floored relative metric of
helpers.rel_err.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import (SCREEN_OFF, SCREEN_ON, TOL_F32, act_empty, assert_close, cfg_of, dev, dev_act, device_inputs, f32, host, i32,
                     oracle_run, prec_of, screened, small_workload, tol_act)

pytestmark = pytest.mark.gpu

FLAT = [
    small_workload("ragged-f32", T=333, d=36, h=52, n=7, k=3),
    small_workload("k1-f32", T=130, d=16, h=24, n=5, k=1, seed=2),
    small_workload("k-eq-n-f32", T=65, d=8, h=8, n=4, k=4, seed=3),
    small_workload("many-experts-f32", T=257, d=32, h=16, n=300, k=4, seed=4),   # most experts empty
    small_workload("wide-n-bf16", T=1200, d=128, h=192, n=70, k=2, act="bf16", seed=5),
    small_workload("k8-bf16", T=515, d=64, h=64, n=33, k=8, act="bf16", seed=6),
    small_workload("one-expert-f32", T=100, d=12, h=20, n=1, k=1, seed=7),
    small_workload("long-segments-bf16", T=3000, d=128, h=320, n=5, k=2, act="bf16", seed=8),  # 256-row tile pairs
    small_workload("screened-gate-bf16", T=4096, d=128, h=64, n=32, k=4, act="bf16", seed=9),  # tensor-core routing screen
    # routing screen + tensor-core gate backward with a token count that is no multiple of any tile or row range
    small_workload("screened-ragged-bf16", T=4100, d=128, h=64, n=32, k=2, act="bf16", seed=12),
    # SM-pair kernels with a heavily skewed load: one very long segment, short ones, (nearly) empty ones
    small_workload("skewed-long-bf16", T=4096, d=192, h=256, n=6, k=1, act="bf16", seed=11, skew="zipf", gamma=3.0),
    # SM-pair kernels with a deep model width and a hidden width that is no multiple of the 256-column tile
    small_workload("deep-d-bf16", T=2048, d=2048, h=192, n=4, k=2, act="bf16", seed=14),
    # a single expert: one long segment, every tile but the last is full
    small_workload("one-expert-bf16", T=5000, d=64, h=128, n=1, k=1, act="bf16", seed=15),
    # the largest expert count the ABI admits, the largest k: generic (any-n) paths of the gating, loss and routing kernels
    small_workload("max-experts-bf16", T=600, d=64, h=64, n=8192, k=8, act="bf16", seed=13),
    synth.CONFIGS["c1"],
]


@pytest.fixture(scope="module", params=FLAT, ids=lambda w: w.name)
def case(request):
    w = request.param
    I = synth.make_all(w)
    F, Bk = oracle_run(w, I)
    # small test shapes would otherwise stay below the automatic threshold of the routing screen
    return w, I, F, Bk, device_inputs(w, I), cfg_of(w, SCREEN_ON)


def ws_for(cfg):
    S = B.moe_query_sizes(cfg)
    return B.empty_bytes(S.ws_bytes), S


def test_gate(case):
    w, I, F, _, D, cfg = case
    ws, S = ws_for(cfg)
    idx, gates = i32(w.T, w.k), f32(w.T, w.k)
    clean, raw = f32(w.T, w.n), f32(w.T, w.n)
    kv, ki = f32(w.T, 2), i32(w.T, 2)
    B.moe_gate(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], idx, gates, clean, raw, kv, ki, ws)
    assert B.moe_check_status(ws) == 0
    assert (host(idx) == F.G.idx).all(), "routing must be bit-exact"
    assert (host(ki) == F.G.kth_idx).all()
    if screened(w):  # logits of provably-routed tokens come from the tensor-core product: 1e-5, not bit-exact
        assert_close(host(clean), F.G.clean, TOL_F32, "clean")
        assert_close(host(raw), F.G.raw, TOL_F32, "raw")
        assert_close(host(kv), F.G.kth_val, TOL_F32, "kth_vals")
    else:
        assert (host(clean) == F.G.clean).all(), "clean logits must be bit-exact (fixed fma chain)"
        assert (host(raw) == F.G.raw).all()
        assert (host(kv) == F.G.kth_val).all()
    assert_close(host(gates), F.G.gates, TOL_F32, "gates")
    assert np.abs(host(gates).sum(axis=1) - 1).max() < 1e-6


def test_gate_with_ties_prefers_lowest_index():
    w = small_workload("ties", T=64, d=8, h=8, n=40, k=3)
    cfg = cfg_of(w)
    ws, _ = ws_for(cfg)
    x = torch.zeros(w.T, w.d, device="cuda")          # all logits equal: 0 + noise * ln 2
    Wz = torch.zeros(w.d, w.n, device="cuda")
    noise = torch.zeros(w.T, w.n, device="cuda")
    noise[:, 7] = 1.0
    noise[:, 35] = 1.0                                  # two-way tie at the top, 38-way tie below
    idx, gates, clean, raw = i32(w.T, w.k), f32(w.T, w.k), f32(w.T, w.n), f32(w.T, w.n)
    kv, ki = f32(w.T, 2), i32(w.T, 2)
    B.moe_gate(cfg, x, Wz, Wz, noise, idx, gates, clean, raw, kv, ki, ws)
    assert (host(idx) == np.array([7, 35, 0])).all()
    assert (host(ki) == np.array([0, 1])).all()
    G = O.gate(host(x), host(Wz), host(Wz), host(noise), w.k, "f32")
    assert (G.idx == host(idx)).all() and (G.kth_idx == host(ki)).all()


def test_gate_screen_sends_ties_and_near_ties_to_the_exact_chain():
    """Pairs of experts with identical weights and identical noise have exactly equal noisy logits: the screen
    cannot certify their order, the fma-chain pass must, and the lowest index must win as in the oracle."""
    w = small_workload("screen-ties", T=2048, d=64, h=64, n=64, k=4, act="bf16", seed=10)
    I = synth.make_all(w)
    for name in ("Wg", "Wnoise", "noise"):
        I[name][:, 1::2] = I[name][:, 0::2]
    I["Wg"][:, 2] = I["Wg"][:, 0] * np.float32(1 + 2 ** -20)  # and a near-tie far below any provable gap
    G = O.gate(I["x"], I["Wg"], I["Wnoise"], I["noise"], w.k, "bf16")
    cfg = cfg_of(w, SCREEN_ON)
    ws, S = ws_for(cfg)
    D = device_inputs(w, I)
    idx, gates, clean, raw = i32(w.T, w.k), f32(w.T, w.k), f32(w.T, w.n), f32(w.T, w.n)
    kv, ki = f32(w.T, 2), i32(w.T, 2)
    B.moe_gate(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], idx, gates, clean, raw, kv, ki, ws)
    assert B.moe_check_status(ws) == 0
    assert (host(idx) == G.idx).all() and (host(ki) == G.kth_idx).all()
    top = G.idx[:, 0]
    assert ((top % 2 == 0) | (top == 3)).all()  # the even (lower) twin wins every exact tie (columns 2/3 differ)
    assert_close(host(gates), G.gates, TOL_F32, "gates")
    assert_close(host(clean), G.clean, TOL_F32, "clean")


def test_screened_routing_equals_pure_chain_routing_on_many_batches():
    """The screen must never change the routing: with MOE_FLAG_GATE_SCREEN_OFF every token goes through the fma
    chain; both runs must give identical indices on fresh batches of a wide, skewed gate (c5's shape)."""
    from dataclasses import replace
    base = replace(synth.CONFIGS["c5"], T=16384)
    for seed in range(6):
        w = replace(base, seed=synth.BASE_SEED + 500 + seed, name=f"c5-seed{seed}")
        x, (Wg, Wn, noise) = dev_act(synth.make_x(w), w), [dev(a) for a in synth.make_gate(w)]
        out = []
        for flags in (SCREEN_ON, SCREEN_OFF):
            cfg = cfg_of(w, flags)
            ws, S = ws_for(cfg)
            idx, gates, clean, raw = i32(w.T, w.k), f32(w.T, w.k), f32(w.T, w.n), f32(w.T, w.n)
            kv, ki = f32(w.T, 2), i32(w.T, 2)
            B.moe_gate(cfg, x, Wg, Wn, noise, idx, gates, clean, raw, kv, ki, ws)
            assert B.moe_check_status(ws) == 0
            out.append((idx, ki, gates, clean))
        assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1]), seed
        assert_close(host(out[0][2]), host(out[1][2]), TOL_F32, "gates")
        assert_close(host(out[0][3]), host(out[1][3]), TOL_F32, "clean")


def test_screened_routing_equals_pure_chain_routing_on_badly_scaled_inputs():
    """The same property where the screen's error model is stressed: features and weight rows spanning six orders of
    magnitude, heavy-tailed activations, large noise, cancelling logits (so the intervals are wide against the gaps)."""
    from dataclasses import replace
    base = replace(synth.CONFIGS["c5"], T=8192, skew="none")
    for seed in range(4):
        w = replace(base, seed=synth.BASE_SEED + 600 + seed, name=f"c5-rough{seed}")
        rng = np.random.default_rng(900 + seed)
        x = synth.make_x(w).astype(np.float32)
        Wg, Wn, noise = [np.array(a, np.float32) for a in synth.make_gate(w)]
        scale = (10.0 ** rng.uniform(-3, 3, size=w.d)).astype(np.float32)
        x = x * scale * (1.0 + 5.0 * (rng.random(x.shape) < 0.01))          # per-feature scales, 1 % outliers
        Wg = Wg / scale[:, None]; Wn = Wn / scale[:, None]                    # logits stay O(1): sums of huge and tiny terms
        if seed & 1:
            Wg[:, 1::2] = Wg[:, 0::2] * (1.0 + 1e-7)                          # near-duplicate experts
        noise = noise * 4.0
        xd, Wgd, Wnd, nd = dev_act(x, w), dev(Wg), dev(Wn), dev(noise)
        out = []
        for flags in (SCREEN_ON, SCREEN_OFF):
            cfg = cfg_of(w, flags)
            ws, S = ws_for(cfg)
            idx, gates, clean, raw = i32(w.T, w.k), f32(w.T, w.k), f32(w.T, w.n), f32(w.T, w.n)
            kv, ki = f32(w.T, 2), i32(w.T, 2)
            B.moe_gate(cfg, xd, Wgd, Wnd, nd, idx, gates, clean, raw, kv, ki, ws)
            assert B.moe_check_status(ws) == 0
            out.append((idx, ki))
        assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1]), seed


def test_dispatch(case):
    w, I, F, _, D, cfg = case
    ws, S = ws_for(cfg)
    xs, perm, inv = act_empty(w, S.R, w.d), i32(S.R), i32(S.R)
    counts, offsets = i32(w.n), i32(w.n + 1)
    B.moe_dispatch(cfg, D["x"], dev(F.G.idx), xs, perm, inv, counts, offsets, ws)
    assert (host(counts) == F.D.counts).all() and (host(offsets) == F.D.offsets).all()
    assert (host(perm) == F.D.perm).all() and (host(inv) == F.D.inv_perm).all()
    assert (host(xs) == np.asarray(F.D.xs, np.float32)).all(), "dispatched rows are exact copies"


def test_expert_ffn(case):
    w, I, F, _, D, cfg = case
    ws, S = ws_for(cfg)
    hid, ys = act_empty(w, S.R, w.h), act_empty(w, S.R, w.d)
    B.moe_expert_ffn(cfg, dev_act(F.D.xs, w), dev(F.D.offsets), D["W1"], D["b1"], D["W2"], D["b2"], hid, ys, ws)
    assert B.moe_check_status(ws) == 0
    assert_close(host(hid), F.hid, tol_act(w), "hid")
    assert_close(host(ys), F.ys, tol_act(w), "ys")


def test_combine(case):
    w, I, F, _, D, cfg = case
    y = act_empty(w, w.T, w.d)
    B.moe_combine(cfg, dev_act(F.ys, w), dev(F.G.gates), dev(F.D.inv_perm), y)
    assert_close(host(y), F.y, tol_act(w), "y")


def test_losses(case):
    w, I, F, _, D, cfg = case
    ws, S = ws_for(cfg)
    imp, load, L = f32(w.n), f32(S.load_elems), f32(2)
    B.moe_losses(cfg, dev(F.G.idx), dev(F.G.gates), dev(F.G.clean), dev(F.G.raw), dev(F.G.kth_val), imp, load, L, ws)
    assert_close(host(imp), F.LS.importance, TOL_F32, "importance")
    assert_close(host(load), F.LS.load, TOL_F32, "load")
    assert_close(host(L), F.LS.losses, TOL_F32, "losses")


def test_combine_bwd(case):
    w, I, F, Bk, D, cfg = case
    S = B.moe_query_sizes(cfg)
    dg, dys = f32(w.T, w.k), act_empty(w, S.R, w.d)
    B.moe_combine_bwd(cfg, D["dY"], dev_act(F.ys, w), dev(F.G.gates), dev(F.D.inv_perm), dg, dys)
    assert_close(host(dg), Bk.dgates, tol_act(w) if w.act == "bf16" else TOL_F32, "dgates")
    assert_close(host(dys), Bk.dys, tol_act(w), "dys")


def test_expert_ffn_bwd(case):
    w, I, F, Bk, D, cfg = case
    ws, S = ws_for(cfg)
    dxs = act_empty(w, S.R, w.d)
    dW1, db1 = act_empty(w, w.n, w.d, w.h), act_empty(w, w.n, w.h)
    dW2, db2 = act_empty(w, w.n, w.h, w.d), act_empty(w, w.n, w.d)
    B.moe_expert_ffn_bwd(cfg, dev_act(F.D.xs, w), dev_act(F.hid, w), dev_act(Bk.dys, w), dev(F.D.offsets), D["W1"],
                         D["W2"], dxs, dW1, db1, dW2, db2, ws)
    assert B.moe_check_status(ws) == 0
    tol = tol_act(w)
    for name, got, want in (("dxs", dxs, Bk.dxs), ("dW1", dW1, Bk.dW1), ("db1", db1, Bk.db1), ("dW2", dW2, Bk.dW2),
                            ("db2", db2, Bk.db2)):
        assert_close(host(got), want, tol, name)
    empty = np.nonzero(F.D.counts == 0)[0]
    if empty.size:
        assert float(host(dW1)[empty].__abs__().max()) == 0.0 and float(host(db2)[empty].__abs__().max()) == 0.0


def test_dispatch_bwd(case):
    w, I, F, Bk, D, cfg = case
    out = f32(w.T, w.d)
    B.moe_dispatch_bwd(cfg, dev_act(Bk.dxs, w), dev(F.D.inv_perm), out)
    assert_close(host(out), Bk.dX_expert, TOL_F32, "dX_expert")


def test_losses_bwd_and_gate_bwd(case):
    w, I, F, Bk, D, cfg = case
    ws, S = ws_for(cfg)
    prec = prec_of(w)
    dg_want, dload_want = O.losses_bwd(F.LS.importance, F.LS.load, F.G.idx, Bk.dgates, w.w_importance, w.w_load, prec)
    dg, dload = dev(np.asarray(Bk.dgates, np.float32)), f32(S.dload_elems)
    B.moe_losses_bwd(cfg, dev(F.LS.importance), dev(F.LS.load), dev(F.G.idx), dg, dload, ws)
    assert_close(host(dg), dg_want, TOL_F32, "dgates+importance")
    assert_close(host(dload), dload_want, TOL_F32, "dload")
    GB = O.gate_bwd(I["x"], I["Wg"], I["Wnoise"], I["noise"], F.G.clean, F.G.raw, F.G.idx, F.G.gates, F.G.kth_val,
                    F.G.kth_idx, dg_want, dload_want, prec)
    dWg, dWn, dXg = f32(w.d, w.n), f32(w.d, w.n), f32(w.T, w.d)
    B.moe_gate_bwd(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], dev(F.G.clean), dev(F.G.raw), dev(F.G.idx),
                   dev(F.G.gates), dev(F.G.kth_val), dev(F.G.kth_idx), dev(dg_want), dev(dload_want), dWg, dWn, dXg,
                   ws)
    assert_close(host(dWg), GB.dWg, TOL_F32, "dWg")
    assert_close(host(dWn), GB.dWnoise, TOL_F32, "dWnoise")
    assert_close(host(dXg), GB.dX_gate, TOL_F32, "dX_gate")


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_expert_stages_with_no_rows_give_zero_gradients(act):
    """T = 0: every segment is empty; the weight and bias gradients must come out as exact zeros (both GEMM paths)."""
    w = small_workload("no-rows", T=0, d=64, h=128, n=8, k=2, act=act)
    cfg = cfg_of(w)
    ws, S = ws_for(cfg)
    I = synth.make_all(dataclasses.replace(w, T=4))
    offsets = torch.zeros(w.n + 1, dtype=torch.int32, device="cuda")
    one = lambda *shape: torch.full(shape, 7.0, dtype=torch.bfloat16 if act == "bf16" else torch.float32, device="cuda")
    dW1, db1, dW2, db2 = one(w.n, w.d, w.h), one(w.n, w.h), one(w.n, w.h, w.d), one(w.n, w.d)
    rows_d, rows_h = act_empty(w, 1, w.d), act_empty(w, 1, w.h)
    B.moe_expert_ffn(cfg, rows_d, offsets, dev_act(I["W1"], w), dev_act(I["b1"], w), dev_act(I["W2"], w),
                     dev_act(I["b2"], w), rows_h, act_empty(w, 1, w.d), ws)
    B.moe_expert_ffn_bwd(cfg, rows_d, rows_h, act_empty(w, 1, w.d), offsets, dev_act(I["W1"], w), dev_act(I["W2"], w),
                         act_empty(w, 1, w.d), dW1, db1, dW2, db2, ws)
    assert B.moe_check_status(ws) == 0
    for name, g in (("dW1", dW1), ("db1", db1), ("dW2", dW2), ("db2", db2)):
        assert float(g.float().abs().max()) == 0.0, name


def test_empty_batch():
    w = small_workload("empty", T=0, d=16, h=16, n=4, k=2)
    cfg = cfg_of(w)
    ws, S = ws_for(cfg)
    counts, offsets = i32(w.n), i32(w.n + 1)
    B.moe_dispatch(cfg, act_empty(w, 1, w.d), i32(1), act_empty(w, 1, w.d), i32(1), i32(1), counts, offsets, ws)
    torch.cuda.synchronize()
    assert host(counts).sum() == 0 and host(offsets).sum() == 0


def test_non_finite_inputs_never_leave_the_index_range():
    """A token full of NaN (and one with an infinite feature) gives NaN logits: the selection must still return k
    distinct experts in [0, n), so that nothing downstream follows a bad index; the whole layer then runs without a
    fault and the other tokens' routing is the oracle's."""
    for flags, T in ((SCREEN_ON, 1024), (SCREEN_OFF, 300)):
        w = small_workload("nan-token", T=T, d=64, h=64, n=32, k=2, act="bf16", seed=21)
        I = synth.make_all(w)
        I["x"][5, :] = np.nan
        I["x"][9, 3] = np.inf
        cfg = cfg_of(w, flags)
        S = B.moe_query_sizes(cfg)
        D = device_inputs(w, I)
        ctx, ws = B.empty_bytes(S.ctx_bytes), B.empty_bytes(max(S.ws_fwd_bytes, S.ws_bwd_bytes))
        ctx.fill_(0xFF)  # stale context: any index taken from it would be far out of range
        y, losses, imp, load, counts = act_empty(w, w.T, w.d), f32(2), f32(w.n), f32(S.load_elems), i32(w.n)
        B.moe_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], y, losses, imp,
                      load, counts, ctx, ws)
        dX, dWg, dWn = act_empty(w, w.T, w.d), f32(S.wg_elems), f32(S.wg_elems)
        dW1, db1 = act_empty(w, w.n, w.d, w.h), act_empty(w, w.n, w.h)
        dW2, db2 = act_empty(w, w.n, w.h, w.d), act_empty(w, w.n, w.d)
        B.moe_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], ctx,
                       dX, dWg, dWn, dW1, db1, dW2, db2, ws)
        assert B.moe_check_status(ws) == 0
        V = B.ctx_views(cfg, ctx)
        idx = host(V["topk_idx"])
        assert idx.min() >= 0 and idx.max() < w.n
        assert (idx[:, 0] != idx[:, 1]).all()
        inv = host(V["inv_perm"])
        assert inv.min() >= 0 and inv.max() < S.R and int(host(counts).sum()) == S.R
        good = np.ones(w.T, bool)
        good[[5, 9]] = False
        I2 = dict(I, x=np.where(np.isfinite(I["x"]), I["x"], 0.0).astype(np.float32))
        G = O.gate(I2["x"], I["Wg"], I["Wnoise"], I["noise"], w.k, "bf16")
        assert (idx[good] == G.idx[good]).all()
        assert np.isfinite(host(y)[good]).all()


def test_dispatch_drops_expert_ids_outside_the_range():
    """moe_dispatch with caller-made indices: ids outside [0, n) are dropped (inv_perm -1), the row movers skip them."""
    w = small_workload("bad-ids", T=200, d=32, h=16, n=6, k=2, act="f32", seed=22)
    cfg = cfg_of(w)
    ws, S = ws_for(cfg)
    rng = np.random.default_rng(3)
    idx = rng.integers(0, w.n, size=(w.T, w.k)).astype(np.int32)
    idx[7, 1] = w.n + 3
    idx[11, 0] = -2
    idx[100, 1] = 2 ** 31 - 1
    x = dev_act(synth.make_x(w), w)
    xs, perm, inv = act_empty(w, S.R, w.d), i32(S.R), i32(S.R)
    xs.fill_(-7.0)
    counts, offsets = i32(w.n), i32(w.n + 1)
    B.moe_dispatch(cfg, x, dev(idx), xs, perm, inv, counts, offsets, ws)
    inv_h = host(inv).reshape(w.T, w.k)
    assert inv_h[7, 1] == -1 and inv_h[11, 0] == -1 and inv_h[100, 1] == -1
    assert int(host(counts).sum()) == S.R - 3 and (np.sort(inv_h[inv_h >= 0]) == np.arange(S.R - 3)).all()
    gates = dev(np.full((w.T, w.k), 0.5, np.float32))
    y = act_empty(w, w.T, w.d)
    B.moe_combine(cfg, xs, gates, inv, y)                      # dropped slots contribute nothing
    xh = host(x)
    want = xh.copy()
    want[[7, 11, 100]] *= 0.5
    assert np.allclose(host(y), want, rtol=1e-6, atol=1e-6)
    dg, dys = f32(w.T, w.k), act_empty(w, S.R, w.d)
    B.moe_combine_bwd(cfg, x, xs, gates, inv, dg, dys)
    assert host(dg)[7, 1] == 0 and host(dg)[11, 0] == 0
    out = f32(w.T, w.d)
    B.moe_dispatch_bwd(cfg, xs, inv, out)
    torch.cuda.synchronize()
    assert np.isfinite(host(out)).all()


def test_non_finite_rows_of_one_expert_do_not_reach_the_others_weight_gradients():
    """The weight-gradient GEMMs contract over ragged row ranges; the rows behind a segment's end belong to the next
    expert and are cleared in both operands, so Inf there cannot turn into 0 x Inf = NaN in this expert's sums."""
    for T, n, d, h in ((3000, 5, 128, 256), (700, 9, 64, 64)):   # SM-pair kernels / one-CTA kernels
        w = small_workload("inf-rows", T=T, d=d, h=h, n=n, k=2, act="bf16", seed=23)
        I = synth.make_all(w)
        F, Bk = oracle_run(w, I)
        cfg = cfg_of(w)
        ws, S = ws_for(cfg)
        bad = 2
        o0, o1 = int(F.D.offsets[bad]), int(F.D.offsets[bad + 1])
        assert o1 - o0 > 0 and o0 % 64 != 0
        dys = np.asarray(Bk.dys, np.float32).copy()
        dys[o0:o1] = np.inf
        hid = np.asarray(F.hid, np.float32).copy()
        hid[o0:o1] = np.inf
        dxs = act_empty(w, S.R, w.d)
        dW1, db1 = act_empty(w, w.n, w.d, w.h), act_empty(w, w.n, w.h)
        dW2, db2 = act_empty(w, w.n, w.h, w.d), act_empty(w, w.n, w.d)
        D = device_inputs(w, I)
        B.moe_expert_ffn_bwd(cfg, dev_act(F.D.xs, w), dev_act(hid, w), dev_act(dys, w), dev(F.D.offsets), D["W1"],
                             D["W2"], dxs, dW1, db1, dW2, db2, ws)
        assert B.moe_check_status(ws) == 0
        others = [e for e in range(w.n) if e != bad]
        for name, got, want in (("dW1", dW1, Bk.dW1), ("dW2", dW2, Bk.dW2), ("db1", db1, Bk.db1), ("db2", db2, Bk.db2)):
            assert_close(host(got)[others], np.asarray(want)[others], tol_act(w), name)


def test_expert_stages_with_the_relu_mask_as_bits(case):
    """moe_expert_ffn_bits / moe_expert_ffn_bwd_bits: the mask bits are exactly [hid > 0], and the backward that reads
    them gives bit for bit what the backward that reads hid gives."""
    w, I, F, Bk, D, cfg = case
    if not (w.act == "bf16" and w.d % 64 == 0 and w.h % 64 == 0):
        with pytest.raises(B.MoeError):
            B.moe_expert_ffn_bits(cfg, dev_act(F.D.xs, w), dev(F.D.offsets), D["W1"], D["b1"], D["W2"], D["b2"],
                                  act_empty(w, 1, 1), act_empty(w, 1, 1), i32(8), B.empty_bytes(1024))
        return
    ws, S = ws_for(cfg)
    hid, ys = act_empty(w, S.R, w.h), act_empty(w, S.R, w.d)
    bits = torch.full((S.R, w.h // 32), -1, dtype=torch.int32, device="cuda")
    xs, offs = dev_act(F.D.xs, w), dev(F.D.offsets)
    B.moe_expert_ffn_bits(cfg, xs, offs, D["W1"], D["b1"], D["W2"], D["b2"], hid, ys, bits, ws)
    assert B.moe_check_status(ws) == 0
    want = np.packbits(host(hid) > 0, axis=1, bitorder="little").view(np.uint32)
    assert (host(bits).view(np.uint32) == want).all()
    dys = dev_act(Bk.dys, w)
    a = [act_empty(w, S.R, w.d), act_empty(w, w.n, w.d, w.h), act_empty(w, w.n, w.h), act_empty(w, w.n, w.h, w.d), act_empty(w, w.n, w.d)]
    b = [torch.empty_like(t) for t in a]
    B.moe_expert_ffn_bwd(cfg, xs, hid, dys, offs, D["W1"], D["W2"], *a, ws)
    B.moe_expert_ffn_bwd_bits(cfg, xs, hid, bits, dys, offs, D["W1"], D["W2"], *b, ws)
    assert B.moe_check_status(ws) == 0
    for name, p, q in zip(("dxs", "dW1", "db1", "dW2", "db2"), a, b):
        assert torch.equal(p, q), name
