"""End-to-end parity of moe_forward / moe_backward against the CPU oracle on identical seeded inputs."""
import numpy as np
import pytest
import torch

from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import (SCREEN_ON, TOL_F32, act_empty, assert_close, assert_expert_backward_close, cat_parts, cfg_of,
                     device_inputs, f32, host, i32, oracle_run, screened, small_workload, tol_act)

pytestmark = pytest.mark.gpu

CASES = [
    small_workload("fused-ragged-f32", T=333, d=36, h=52, n=7, k=3, seed=11),
    small_workload("fused-bf16", T=1500, d=128, h=256, n=24, k=4, act="bf16", seed=12),
    small_workload("fused-empty-experts-bf16", T=200, d=64, h=128, n=150, k=2, act="bf16", seed=13),
    synth.CONFIGS["c1"],
    synth.CONFIGS["c2"],
]


def run_fused(w, I, flags=0):
    cfg = cfg_of(w, flags)
    S = B.moe_query_sizes(cfg)
    D = device_inputs(w, I)
    ctx = B.empty_bytes(S.ctx_bytes)
    ws = B.empty_bytes(max(S.ws_fwd_bytes, S.ws_bwd_bytes))
    ws.fill_(0xFF)  # the library must not rely on a zeroed workspace
    y, losses, imp, load, counts = act_empty(w, w.T, w.d), f32(2), f32(w.n), f32(S.load_elems), i32(w.n)
    B.moe_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], y, losses, imp,
                  load, counts, ctx, ws)
    assert B.moe_check_status(ws) == 0
    dX = act_empty(w, w.T, w.d)
    dWg, dWn = f32(S.wg_elems), f32(S.wg_elems)
    dW1, db1 = act_empty(w, w.n, w.d, w.h), act_empty(w, w.n, w.h)
    dW2, db2 = act_empty(w, w.n, w.h, w.d), act_empty(w, w.n, w.d)
    B.moe_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], ctx,
                   dX, dWg, dWn, dW1, db1, dW2, db2, ws)
    assert B.moe_check_status(ws) == 0
    V = B.ctx_views(cfg, ctx)
    return dict(y=y, losses=losses, importance=imp, load=load, counts=counts, dX=dX, dWg=dWg, dWnoise=dWn, dW1=dW1,
                db1=db1, dW2=dW2, db2=db2, ctx=V)


_ORACLE = {}


def oracle_cached(w):
    if w.name not in _ORACLE:
        I = synth.make_all(w)
        _ORACLE[w.name] = (I,) + tuple(oracle_run(w, I))
    return _ORACLE[w.name]


# flags 0: the kernels the library picks by itself (what bench.py runs); SCREEN_ON: the routing screen forced on
# for these small shapes (it only applies to bf16 layers whose widths are multiples of 64)
@pytest.mark.parametrize("flags", [0, SCREEN_ON], ids=["default", "screen-on"])
@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_fused_forward_backward(w, flags):
    if flags and not screened(w, flags):
        pytest.skip("the routing screen does not apply to this shape")
    I, F, Bk = oracle_cached(w)
    G = run_fused(w, I, flags)
    V = G["ctx"]
    # routing: bit-exact
    assert (host(V["topk_idx"]) == F.G.idx).all()
    assert (host(V["perm"]) == F.D.perm).all() and (host(V["inv_perm"]) == F.D.inv_perm).all()
    assert (host(G["counts"]) == F.D.counts).all() and (host(V["offsets"]) == F.D.offsets).all()
    assert (host(V["kth_idx"]) == F.G.kth_idx).all()
    # gating floats
    assert_close(host(V["gates"]), cat_parts(F.G.gates), TOL_F32, "gates")
    assert_close(host(G["importance"]), F.LS.importance, TOL_F32, "importance")
    assert_close(host(G["load"]), F.LS.load, TOL_F32, "load")
    assert_close(host(G["losses"]), F.LS.losses, TOL_F32, "losses")
    # expert side
    tol = tol_act(w)
    hid = host(V["hid"])
    assert_close(hid, F.hid, tol, "hid")
    assert_close(host(V["ys"]), F.ys, tol, "ys")
    assert_close(host(G["y"]), F.y, tol, "y")
    # ReLU decisions within rounding of zero may differ: bounded in number and size, their dependants set aside
    assert_expert_backward_close(w, F, Bk, G, hid, tol)
    # gate gradients inherit the expert-side error through dgates
    assert_close(host(G["dWg"]), cat_parts(Bk.dWg), tol, "dWg")
    assert_close(host(G["dWnoise"]), cat_parts(Bk.dWnoise), tol, "dWnoise")


def test_fused_is_deterministic():
    w = small_workload("det-bf16", T=700, d=64, h=128, n=16, k=2, act="bf16", seed=14)
    I = synth.make_all(w)
    a, b = run_fused(w, I), run_fused(w, I)
    for name in ("y", "losses", "importance", "load", "dX", "dWg", "dWnoise", "dW1", "db1", "dW2", "db2"):
        assert torch.equal(a[name], b[name]), name


def test_two_runs_give_bitwise_identical_results():
    """Nothing in the path depends on timing: the tile order is static, sums are taken in fixed orders, the lists of
    uncertain tokens are only worked through element by element. Two runs on the same inputs must agree bit for bit."""
    w = synth.CONFIGS["c3"].scaled(8192)
    I = synth.make_all(w)
    a, b = run_fused(w, I), run_fused(w, I)
    for name in ("y", "losses", "importance", "load", "counts", "dX", "dWg", "dWnoise", "dW1", "db1", "dW2", "db2"):
        assert torch.equal(a[name], b[name]), name
    for name in ("topk_idx", "gates", "clean", "raw_noise", "hid", "ys"):
        assert torch.equal(a["ctx"][name], b["ctx"][name]), name


def test_the_fused_calls_can_be_captured_in_a_cuda_graph():
    """moe_forward + moe_backward only enqueue work on the caller's stream (no synchronisation, no allocation), so a
    stream capture records them; replaying the graph must reproduce the eager results bit for bit."""
    w = synth.CONFIGS["c2"]
    I = synth.make_all(w)
    cfg = cfg_of(w)
    S = B.moe_query_sizes(cfg)
    D = device_inputs(w, I)
    ctx, ws = B.empty_bytes(S.ctx_bytes), B.empty_bytes(max(S.ws_fwd_bytes, S.ws_bwd_bytes))
    out = dict(y=act_empty(w, w.T, w.d), losses=f32(2), imp=f32(w.n), load=f32(S.load_elems), counts=i32(w.n),
               dX=act_empty(w, w.T, w.d), dWg=f32(S.wg_elems), dWn=f32(S.wg_elems), dW1=act_empty(w, w.n, w.d, w.h),
               db1=act_empty(w, w.n, w.h), dW2=act_empty(w, w.n, w.h, w.d), db2=act_empty(w, w.n, w.d))

    def step():
        B.moe_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], out["y"],
                      out["losses"], out["imp"], out["load"], out["counts"], ctx, ws)
        B.moe_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], ctx,
                       out["dX"], out["dWg"], out["dWn"], out["dW1"], out["db1"], out["dW2"], out["db2"], ws)

    step()  # eager: also the first-call set-up (function attributes, driver entry points)
    torch.cuda.synchronize()
    eager = {k: v.clone() for k, v in out.items()}
    for v in out.values():
        v.zero_()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for v in out.values():
        v.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert B.moe_check_status(ws) == 0
    for k in out:
        assert torch.equal(out[k], eager[k]), k
