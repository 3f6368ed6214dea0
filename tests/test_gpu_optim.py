"""Memory mode and optimiser step of the paper's large models (Appendix D, "Training"): hidden activations recomputed
in the backward pass, and Adam with beta1 = 0 and a factored second-moment estimate on the expert parameters."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import (TOL_F32, act_empty, assert_close, cfg_of, dev, dev_act, device_inputs, f32, host, i32, oracle_run,
                     prec_of, small_workload, tol_act)
from test_gpu_fused import run_fused

pytestmark = pytest.mark.gpu

RECOMPUTE = B.MOE_FLAG_RECOMPUTE_HID


@pytest.mark.parametrize("w", [
    small_workload("recompute-f32", T=333, d=36, h=52, n=7, k=3, seed=61),
    small_workload("recompute-bf16", T=1500, d=128, h=256, n=24, k=4, act="bf16", seed=62),
    small_workload("recompute-hier-bf16", T=1000, d=64, h=128, n=64, k=4, a=8, k1=2, b=8, k2=2, act="bf16", seed=63),
    synth.CONFIGS["c2"],
], ids=lambda w: w.name)
def test_recomputing_the_hidden_activations_changes_nothing_but_the_memory(w):
    """With MOE_FLAG_RECOMPUTE_HID the context is R*h elements smaller and every result is bit-identical: the
    backward runs the same first GEMM again on the same inputs."""
    I = synth.make_all(w)
    a, b = run_fused(w, I), run_fused(w, I, RECOMPUTE)
    for name in ("y", "losses", "importance", "load", "counts", "dX", "dWg", "dWnoise", "dW1", "db1", "dW2", "db2"):
        assert torch.equal(a[name], b[name]), name
    assert "hid" in a["ctx"] and "hid" not in b["ctx"]
    esz = 2 if w.act == "bf16" else 4
    S0, S1 = B.moe_query_sizes(cfg_of(w)), B.moe_query_sizes(cfg_of(w, RECOMPUTE))
    assert S0.ctx_bytes - S1.ctx_bytes >= w.R * w.h * esz
    assert S1.ws_bwd_bytes >= S0.ws_bwd_bytes


def test_expert_ffn_stage_without_a_hidden_buffer():
    w = small_workload("ffn-nohid-bf16", T=900, d=128, h=192, n=9, k=2, act="bf16", seed=64)
    I = synth.make_all(w)
    F, _ = oracle_run(w, I, backward=False)
    cfg = cfg_of(w, RECOMPUTE)
    S = B.moe_query_sizes(cfg)
    ws = B.empty_bytes(S.ws_bytes)
    D = device_inputs(w, I)
    ys = act_empty(w, S.R, w.d)
    B.moe_expert_ffn(cfg, dev_act(F.D.xs, w), dev(F.D.offsets), D["W1"], D["b1"], D["W2"], D["b2"], None, ys, ws)
    assert B.moe_check_status(ws) == 0
    assert_close(host(ys), F.ys, tol_act(w), "ys")
    with pytest.raises(B.MoeError):   # without the flag a missing buffer is an argument error
        B.moe_expert_ffn(cfg_of(w), dev_act(F.D.xs, w), dev(F.D.offsets), D["W1"], D["b1"], D["W2"], D["b2"], None, ys, ws)


ADAM = [
    small_workload("adam-f32", T=64, d=36, h=52, n=5, k=2, seed=65),
    small_workload("adam-bf16", T=64, d=128, h=320, n=6, k=2, act="bf16", seed=66),
    small_workload("adam-tall-bf16", T=64, d=1024, h=64, n=3, k=2, act="bf16", seed=67),
]


@pytest.mark.parametrize("w", ADAM, ids=lambda w: w.name)
def test_factored_adam_steps(w):
    """Three optimiser steps with fresh gradients: parameters and state against the oracle after every step."""
    g = np.random.default_rng(w.seed)
    prec = prec_of(w)
    W1, b1, W2, b2 = synth.make_experts(w)
    b1 = synth.storage_grid((0.1 * g.standard_normal(b1.shape)).astype(np.float32), w.act)
    b2 = synth.storage_grid((0.1 * g.standard_normal(b2.shape)).astype(np.float32), w.act)
    cfg = cfg_of(w)
    S = B.moe_query_sizes(cfg)
    assert S.adam_state_elems == w.n * (3 * w.d + 3 * w.h)
    ws = B.empty_bytes(S.ws_adam_bytes)
    dW1_, db1_, dW2_, db2_ = (dev_act(a, w) for a in (W1, b1, W2, b2))
    state_d = torch.zeros(S.adam_state_elems, device="cuda")
    state = dict(r1=np.zeros((w.n, w.d)), c1=np.zeros((w.n, w.h)), r2=np.zeros((w.n, w.h)), c2=np.zeros((w.n, w.d)),
                 vb1=np.zeros((w.n, w.h)), vb2=np.zeros((w.n, w.d)))
    lr, beta2, eps = 1e-2, 0.99, 1e-8
    P = [W1, b1, W2, b2]
    P_d = [dW1_, db1_, dW2_, db2_]
    for step in (1, 2, 3):
        # gradients with a row / column structure (so that the factored estimate matters) and one all-zero expert
        grads = []
        for a in P:
            gr = g.standard_normal(a.shape).astype(np.float32) * (1 + 3 * g.random(a.shape[:2] + (1,) * (a.ndim - 2))).astype(np.float32)
            gr[0] = 0
            grads.append(synth.storage_grid(gr.astype(np.float32), w.act))
        G_d = [dev_act(a, w) for a in grads]
        want = O.expert_adam_factored(P[0], P[1], P[2], P[3], grads[0], grads[1], grads[2], grads[3], state, lr, beta2, eps,
                                      step, prec)
        B.moe_expert_adam_factored(cfg, P_d[0], P_d[1], P_d[2], P_d[3], G_d[0], G_d[1], G_d[2], G_d[3], state_d, lr, beta2,
                                   eps, step, ws)
        torch.cuda.synchronize()
        for name, got, exp in zip(("W1", "b1", "W2", "b2"), P_d, want[:4]):
            assert_close(host(got), exp, tol_act(w), f"{name} after step {step}")
        got_state = host(state_d)
        flat_want = np.concatenate([np.asarray(want[4][k_], np.float64).reshape(-1) for k_ in ("r1", "c1", "r2", "c2", "vb1", "vb2")])
        assert_close(got_state, flat_want, TOL_F32, f"state after step {step}")
        # continue from the ORACLE's parameters and state on both sides, so that every step is compared on equal inputs
        P = [np.asarray(a, np.float32) for a in want[:4]]
        state = want[4]
        for dst, src in zip(P_d, P):
            dst.copy_(dev_act(src, w))
        state_d.copy_(dev(flat_want.astype(np.float32)))
    assert (host(P_d[0])[0] == np.asarray(W1[0], np.float32)).all(), "an expert whose gradient is zero does not move"
