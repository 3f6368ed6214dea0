"""Hierarchical mixture of experts (Appendix B): stage-wise and fused parity against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import (SCREEN_OFF, SCREEN_ON, TOL_F32, act_empty, assert_close, assert_expert_backward_close, cat_parts, cfg_of, dev,
                     dev_act, device_inputs, f32, host, i32, oracle_run, prec_of, screened, small_workload, tol_act)

pytestmark = pytest.mark.gpu

HIER = [
    small_workload("hier-f32", T=300, d=32, h=24, n=30, k=4, a=5, k1=2, b=6, k2=2, seed=31),
    small_workload("hier-k1-eq-a-f32", T=150, d=16, h=16, n=12, k=3, a=1, k1=1, b=12, k2=3, seed=32),
    small_workload("hier-bf16", T=1000, d=64, h=128, n=64, k=4, a=8, k1=2, b=8, k2=2, act="bf16", seed=33),
    small_workload("hier-wide-bf16", T=777, d=128, h=64, n=96, k=6, a=3, k1=2, b=32, k2=3, act="bf16", seed=34),
    # both gating levels wide enough for the tensor-core gate backward (2a and 2b multiples of 64)
    small_workload("hier-tc-bf16", T=2100, d=64, h=64, n=1024, k=4, a=32, k1=2, b=32, k2=2, act="bf16", seed=35),
    # few tokens over many groups: some groups get no token at all (|X^(i)| = 0: zero Load_H row, zero gradients)
    small_workload("hier-empty-groups-f32", T=40, d=32, h=16, n=128, k=4, a=32, k1=2, b=4, k2=2, seed=38),
    small_workload("hier-empty-groups-bf16", T=48, d=64, h=64, n=1024, k=4, a=32, k1=2, b=32, k2=2, act="bf16", seed=39),
    # primary gate wide enough for the routing screen, secondary gates too narrow for it
    small_workload("hier-primary-screen-bf16", T=1024, d=64, h=64, n=256, k=4, a=32, k1=2, b=8, k2=2, act="bf16", seed=37),
]


def gate_tensors(G):
    """Oracle gate state in the ABI's layouts (primary part then secondary part)."""
    P, S = G.primary, G.secondary
    return dict(topk_idx=G.idx, gates=cat_parts((G.gates, P.gates, S.gates)), clean=cat_parts((P.clean, S.clean)),
                raw=cat_parts((P.raw, S.raw)), kth_vals=cat_parts((P.kth_val, S.kth_val)),
                kth_idx=np.concatenate([P.kth_idx.reshape(-1), S.kth_idx.reshape(-1)]).astype(np.int32))


@pytest.fixture(scope="module", params=HIER, ids=lambda w: w.name)
def case(request):
    w = request.param
    I = synth.make_all(w)
    F, Bk = oracle_run(w, I)
    return w, I, F, Bk, device_inputs(w, I), cfg_of(w, SCREEN_ON)


def test_the_empty_group_cases_do_have_empty_groups(case):
    w, I, F, _, D, cfg = case
    if "empty-groups" in w.name:
        assert (np.asarray(F.LS.cnt) == 0).any()


def test_hier_gate(case):
    w, I, F, _, D, cfg = case
    S = B.moe_query_sizes(cfg)
    ws = B.empty_bytes(S.ws_bytes)
    idx, gates = i32(w.T, w.k), f32(S.gates_elems)
    clean, raw = f32(S.logits_elems), f32(S.logits_elems)
    kv, ki = f32(S.kth_elems), i32(S.kth_elems)
    B.moe_gate(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], idx, gates, clean, raw, kv, ki, ws)
    want = gate_tensors(F.G)
    assert (host(idx) == want["topk_idx"]).all(), "hierarchical routing must be bit-exact"
    assert (host(ki) == want["kth_idx"]).all()
    if screened(w):  # primary logits of provably-routed tokens come from the tensor-core product
        for name, got in (("clean", clean), ("raw", raw), ("kth_vals", kv)):
            assert_close(host(got), want[name], TOL_F32, name)
    else:
        assert (host(clean) == want["clean"]).all() and (host(raw) == want["raw"]).all()
        assert (host(kv) == want["kth_vals"]).all()
    assert_close(host(gates), want["gates"], TOL_F32, "gates")


def test_hier_losses_and_backward_stages(case):
    w, I, F, Bk, D, cfg = case
    S = B.moe_query_sizes(cfg)
    ws = B.empty_bytes(S.ws_bytes)
    G = gate_tensors(F.G)
    imp, load, L = f32(w.n), f32(S.load_elems), f32(2)
    B.moe_losses(cfg, dev(G["topk_idx"]), dev(G["gates"]), dev(G["clean"]), dev(G["raw"]), dev(G["kth_vals"]), imp,
                 load, L, ws)
    ab = w.a * w.b
    LS = F.LS
    want_load = np.concatenate([np.asarray(LS.load, np.float64), LS.load_p, LS.load_s.reshape(-1), LS.cnt])
    assert_close(host(imp), LS.importance, TOL_F32, "importance_H")
    assert_close(host(load)[:ab], want_load[:ab], TOL_F32, "load_H")
    assert_close(host(load)[ab:], want_load[ab:], TOL_F32, "load levels")
    assert_close(host(L), LS.losses, TOL_F32, "losses")
    # losses backward + gate backward, fed with the oracle's upstream gradients
    prec = prec_of(w)
    dI = w.w_importance * O.cv_squared_grad(LS.importance)
    dLH = (w.w_load * O.cv_squared_grad(LS.load)).reshape(w.a, w.b)
    safe = np.where(LS.cnt > 0, LS.cnt, 1.0)
    live = (LS.cnt > 0)[:, None]
    want_dload = np.concatenate([np.where(live, dLH * LS.load_s / safe[:, None], 0).sum(1),
                                 np.where(live, dLH * LS.load_p[:, None] / safe[:, None], 0).reshape(-1)])
    dg = torch.zeros(S.gates_elems, device="cuda")
    dg[:w.T * w.k] = dev(np.asarray(Bk.dgates, np.float32)).reshape(-1)
    dload = f32(S.dload_elems)
    B.moe_losses_bwd(cfg, imp, load, dev(G["topk_idx"]), dg, dload, ws)
    assert_close(host(dg)[:w.T * w.k], (np.asarray(Bk.dgates, np.float64) + dI[F.G.idx]).reshape(-1), TOL_F32, "dgates")
    assert_close(host(dload), want_dload, TOL_F32, "dload")
    GB = O.gate_h_bwd(I["x"], I["Wg"][0], I["Wnoise"][0], I["noise"][0], I["Wg"][1], I["Wnoise"][1], I["noise"][1], F.G,
                      LS, Bk.dgates, w.w_importance, w.w_load, prec)
    dWg, dWn, dXg = f32(S.wg_elems), f32(S.wg_elems), f32(w.T, w.d)
    B.moe_gate_bwd(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], dev(G["clean"]), dev(G["raw"]), dev(G["topk_idx"]),
                   dev(G["gates"]), dev(G["kth_vals"]), dev(G["kth_idx"]), dg, dload, dWg, dWn, dXg, ws)
    tol = TOL_F32
    assert_close(host(dWg), cat_parts((GB.dWg_p, GB.dWg_s)), tol, "dWg")
    assert_close(host(dWn), cat_parts((GB.dWn_p, GB.dWn_s)), tol, "dWnoise")
    assert_close(host(dXg), GB.dX_gate, tol, "dX_gate")


@pytest.mark.parametrize("flags", [0, SCREEN_ON], ids=["default", "screen-on"])
def test_hier_fused(case, flags):
    from test_gpu_fused import run_fused
    w, I, F, Bk, D, cfg = case
    if flags and not screened(w, flags):
        pytest.skip("the routing screen does not apply to this shape")
    G = run_fused(w, I, flags)
    V = G["ctx"]
    want = gate_tensors(F.G)
    assert (host(V["topk_idx"]) == F.G.idx).all()
    assert (host(V["perm"]) == F.D.perm).all() and (host(G["counts"]) == F.D.counts).all()
    assert_close(host(V["gates"]), want["gates"], TOL_F32, "gates")
    assert_close(host(G["importance"]), F.LS.importance, TOL_F32, "importance")
    assert_close(host(G["load"])[:w.n], F.LS.load, TOL_F32, "load")
    assert_close(host(G["losses"]), F.LS.losses, TOL_F32, "losses")
    tol = tol_act(w)
    assert_close(host(G["y"]), F.y, tol_act(w), "y")
    hid = host(V["hid"])
    assert_close(hid, F.hid, tol_act(w), "hid")
    assert_expert_backward_close(w, F, Bk, G, hid, tol)
    assert_close(host(G["dWg"]), cat_parts(Bk.dWg), tol, "dWg")
    assert_close(host(G["dWnoise"]), cat_parts(Bk.dWnoise), tol, "dWnoise")


def test_hier_secondary_ties_take_every_column_through_the_chain():
    """Identical secondary gate columns and zero secondary noise: every expert of a group ties, far more candidates
    than the screen resolves column by column, so each such slot gets the chains of all its columns; the oracle's
    lowest-index rule must come out."""
    w = small_workload("hier-sec-ties", T=600, d=64, h=64, n=3 * 32, k=4, a=3, k1=2, b=32, k2=2, act="bf16", seed=36)
    I = synth.make_all(w)
    Wg_p, Wg_s = I["Wg"]
    Wn_p, Wn_s = I["Wnoise"]
    n_p, n_s = I["noise"]
    Wg_s[:] = Wg_s[:, :, :1]          # all columns of a group equal
    Wn_s[:] = Wn_s[:, :, :1]
    n_s[:] = 0.0
    assert screened(w)
    F, _ = oracle_run(w, I, backward=False)
    D, cfg = device_inputs(w, I), cfg_of(w, SCREEN_ON)
    S = B.moe_query_sizes(cfg)
    ws = B.empty_bytes(S.ws_bytes)
    idx, gates = i32(w.T, w.k), f32(S.gates_elems)
    clean, raw = f32(S.logits_elems), f32(S.logits_elems)
    kv, ki = f32(S.kth_elems), i32(S.kth_elems)
    B.moe_gate(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], idx, gates, clean, raw, kv, ki, ws)
    assert B.moe_check_status(ws) == 0
    want = gate_tensors(F.G)
    sec = host(idx).reshape(w.T, w.k1, w.k2) % w.b
    assert (sec[..., 0] == 0).all() and (sec[..., 1] == 1).all()   # lowest indices win the ties
    assert (host(idx) == want["topk_idx"]).all()
    assert (host(ki) == want["kth_idx"]).all()
    assert_close(host(gates), want["gates"], TOL_F32, "gates")


def test_hier_screened_routing_equals_pure_chain_routing():
    """Both gating levels screened on the tensor cores against every slot through the fma chain (c4's shape, 8192 tokens):
    the flat expert ids and both levels' k-th / (k+1)-th indices must be identical."""
    from dataclasses import replace
    for seed in range(3):
        w = replace(synth.CONFIGS["c4"], T=8192, seed=synth.BASE_SEED + 700 + seed, name=f"c4-seed{seed}")
        x = dev_act(synth.make_x(w), w)
        Wg, Wn, noise = [dev(cat_parts(a)) for a in synth.make_gate(w)]
        out = []
        for flags in (SCREEN_ON, SCREEN_OFF):
            cfg = cfg_of(w, flags)
            S = B.moe_query_sizes(cfg)
            ws = B.empty_bytes(S.ws_bytes)
            idx, gates = i32(w.T, w.k), f32(S.gates_elems)
            clean, raw = f32(S.logits_elems), f32(S.logits_elems)
            kv, ki = f32(S.kth_elems), i32(S.kth_elems)
            B.moe_gate(cfg, x, Wg, Wn, noise, idx, gates, clean, raw, kv, ki, ws)
            assert B.moe_check_status(ws) == 0
            out.append((idx, ki, gates))
        assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1]), seed
        assert_close(host(out[0][2]), host(out[1][2]), TOL_F32, "gates")
