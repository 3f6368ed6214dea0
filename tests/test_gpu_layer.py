"""The layer as it sits in the paper's models (Appendix C): sigmoid on the MoE output, dropout, residual connection,
fused into the combine kernels. Stage-wise and end-to-end parity against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import (TOL_F32, act_empty, assert_close, assert_expert_backward_close, cat_parts, cfg_of, dev, dev_act,
                     device_inputs, f32, host, i32, oracle_run, prec_of, small_workload, tol_act)

pytestmark = pytest.mark.gpu

DROP = 0.3
CASES = [
    small_workload("layer-f32", T=333, d=40, h=52, n=7, k=3, seed=51),
    small_workload("layer-bf16", T=1500, d=128, h=256, n=24, k=4, act="bf16", seed=52),
    small_workload("layer-k1-bf16", T=600, d=64, h=64, n=5, k=1, act="bf16", seed=53),
    small_workload("layer-k8-f32", T=130, d=24, h=16, n=12, k=8, seed=54),
    small_workload("layer-hier-bf16", T=1000, d=64, h=128, n=64, k=4, a=8, k1=2, b=8, k2=2, act="bf16", seed=55),
    synth.CONFIGS["c2"],
]


@pytest.fixture(scope="module", params=CASES, ids=lambda w: w.name)
def case(request):
    w = request.param
    I = synth.make_all(w)
    bits = synth.make_keep_bits(w, DROP)
    keep = O.unpack_keep(bits, w.d)
    prec = prec_of(w)
    F = O.forward(I["x"], I["Wg"], I["Wnoise"], I["noise"], I["W1"], I["b1"], I["W2"], I["b2"], w.k, w.w_importance,
                  w.w_load, prec, hier=w.hier, layer=(keep, DROP))
    Bk = O.backward(I["dY"], I["x"], I["Wg"], I["Wnoise"], I["noise"], I["W1"], I["b1"], I["W2"], I["b2"], F,
                    w.w_importance, w.w_load, prec, hier=w.hier, layer=(keep, DROP))
    return w, I, bits, keep, F, Bk


def test_keep_rate(case):
    w, I, bits, keep, F, Bk = case
    assert abs(keep.mean() - (1 - DROP)) < 0.02


def test_combine_layer_stages(case):
    w, I, bits, keep, F, Bk = case
    cfg = cfg_of(w)
    S = B.moe_query_sizes(cfg)
    gates = dev(np.asarray(F.G.gates, np.float32))
    ys, inv, x, kb = dev_act(F.ys, w), dev(F.D.inv_perm), dev_act(I["x"], w), dev(bits)
    out = act_empty(w, w.T, w.d)
    B.moe_combine_layer(cfg, ys, gates, inv, x, kb, DROP, out)
    assert_close(host(out), F.y, tol_act(w), "out")
    dropped = ~keep
    assert (host(out)[dropped] == np.asarray(I["x"], np.float32)[dropped]).all(), "a dropped activation leaves the residual alone"
    dg, dys = f32(w.T, w.k), act_empty(w, S.R, w.d)
    B.moe_combine_layer_bwd(cfg, dev_act(I["dY"], w), ys, gates, inv, kb, DROP, dg, dys)
    assert_close(host(dg), Bk.dgates, tol_act(w) if w.act == "bf16" else TOL_F32, "dgates")
    assert_close(host(dys), Bk.dys, tol_act(w), "dys")


def test_layer_fused(case):
    w, I, bits, keep, F, Bk = case
    cfg = cfg_of(w)
    S = B.moe_query_sizes(cfg)
    D = device_inputs(w, I)
    kb = dev(bits)
    ctx, ws = B.empty_bytes(S.ctx_bytes), B.empty_bytes(max(S.ws_fwd_bytes, S.ws_bwd_bytes))
    out, losses, imp, load, counts = act_empty(w, w.T, w.d), f32(2), f32(w.n), f32(S.load_elems), i32(w.n)
    B.moe_layer_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], kb, DROP, out,
                        losses, imp, load, counts, ctx, ws)
    assert B.moe_check_status(ws) == 0
    G = dict(dX=act_empty(w, w.T, w.d), dWg=f32(S.wg_elems), dWnoise=f32(S.wg_elems), dW1=act_empty(w, w.n, w.d, w.h),
             db1=act_empty(w, w.n, w.h), dW2=act_empty(w, w.n, w.h, w.d), db2=act_empty(w, w.n, w.d))
    B.moe_layer_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], kb,
                         DROP, ctx, G["dX"], G["dWg"], G["dWnoise"], G["dW1"], G["db1"], G["dW2"], G["db2"], ws)
    assert B.moe_check_status(ws) == 0
    V = B.ctx_views(cfg, ctx)
    assert (host(V["topk_idx"]) == F.G.idx).all() and (host(V["perm"]) == F.D.perm).all()
    tol = tol_act(w)
    assert_close(host(out), F.y, tol, "out")
    assert_close(host(losses), F.LS.losses, TOL_F32, "losses")
    hid = host(V["hid"])
    assert_close(hid, F.hid, tol, "hid")
    assert_expert_backward_close(w, F, Bk, G, hid, tol)
    assert_close(host(G["dWg"]), cat_parts(Bk.dWg), tol, "dWg")
    assert_close(host(G["dWnoise"]), cat_parts(Bk.dWnoise), tol, "dWnoise")


def test_layer_arguments_are_checked():
    w = small_workload("layer-args", T=16, d=36, h=16, n=4, k=2, seed=56)   # d is no multiple of 8
    cfg = cfg_of(w)
    t = lambda *s: torch.zeros(*s, device="cuda")
    with pytest.raises(B.MoeError):
        B.moe_combine_layer(cfg, t(32, 36), t(16, 2), i32(32), t(16, 36), torch.zeros(16, 5, dtype=torch.uint8, device="cuda"),
                            0.1, t(16, 36))
    w = small_workload("layer-args", T=16, d=40, h=16, n=4, k=2, seed=56)
    cfg = cfg_of(w)
    for bad in (1.0, -0.1, float("nan")):
        with pytest.raises(B.MoeError):
            B.moe_combine_layer(cfg, t(32, 40), t(16, 2), i32(32), t(16, 40),
                                torch.zeros(16, 5, dtype=torch.uint8, device="cuda"), bad, t(16, 40))
