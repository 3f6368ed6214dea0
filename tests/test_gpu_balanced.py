"""Strictly balanced gating (Appendix F, Eq. 15-20): the CUDA path against the CPU oracle, stage by stage and composed
into a forward + backward step. Masks, row tables and per-token lists are compared bit for bit."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

from helpers import (TOL_F32, act_empty, assert_close, assert_expert_backward_close, cfg_of, dev, dev_act, f32, host, i32,
                     prec_of, small_workload, tol_act)

pytestmark = pytest.mark.gpu

CASES = [
    small_workload("bal-f32", T=96, d=24, h=20, n=8, k=2, seed=81),
    small_workload("bal-odd-n-f32", T=210, d=16, h=12, n=35, k=5, seed=82),        # n no multiple of 32, m = 30
    small_workload("bal-bf16", T=2048, d=128, h=256, n=64, k=4, act="bf16", seed=83),
    small_workload("bal-wide-bf16", T=3072, d=64, h=64, n=192, k=2, act="bf16", seed=84),   # six mask words per token
    synth.CONFIGS["c3"].scaled(8192),                                              # the many-expert shape, m = 128
    # more than 8192 tokens: the per-token row pointers come from the tiled scan (a whole number of 4096-token tiles, so
    # the total falls into a tile of its own; and a token count that is no multiple of four)
    small_workload("bal-long-bf16", T=12288, d=64, h=64, n=32, k=2, act="bf16", seed=88),
    small_workload("bal-long-odd-f32", T=9002, d=16, h=8, n=2, k=1, seed=89),
]
W_BATCHWISE = 0.5


def thresholds_for(w, p):
    """Per-expert thresholds near (not at) the batchwise cut, so that the two masks differ in a few per cent of the entries."""
    m = w.T * w.k // w.n
    srt = -np.sort(-np.asarray(p, np.float64), axis=0)
    g = np.random.default_rng(w.seed)
    return (srt[m - 1] * (1 + 0.05 * g.standard_normal(w.n))).astype(np.float32)


def packed(mask):
    bits = np.packbits(mask, axis=1, bitorder="little")
    words = (mask.shape[1] + 31) // 32
    out = np.zeros((mask.shape[0], words * 4), np.uint8)
    out[:, :bits.shape[1]] = bits
    return out.view(np.uint32)


def tok_lists(D, T):
    """Per-token row lists (ascending expert) from the oracle's row tables."""
    order = np.lexsort((D.expert_of_row, D.tok_of_row))
    ptr = np.zeros(T + 1, np.int32)
    np.add.at(ptr, D.tok_of_row.astype(np.int64) + 1, 1)
    return np.cumsum(ptr).astype(np.int32), order.astype(np.int32)


@pytest.fixture(scope="module", params=CASES, ids=lambda w: w.name)
def case(request):
    w = request.param
    I = synth.make_all(w)
    Wg = I["Wg"]
    prec = prec_of(w)
    _, p = O.softmax_gate(I["x"], Wg, prec)
    thr = thresholds_for(w, p)
    F = O.forward_balanced(I["x"], Wg, thr, I["W1"], I["b1"], I["W2"], I["b2"], w.k, prec)
    Bk = O.backward_balanced(I["dY"], I["x"], Wg, thr, I["W1"], I["b1"], I["W2"], I["b2"], F, W_BATCHWISE, prec)
    return w, I, thr, F, Bk


def run_gate(w, I, thr):
    cfg = cfg_of(w)
    S = B.moe_query_balanced_sizes(cfg)
    out = dict(logits=f32(w.T, w.n), probs=f32(w.T, w.n),
               mask_bits=torch.empty(w.T, S.mask_words, dtype=torch.int32, device="cuda"), tok_of_row=i32(S.R),
               offsets=i32(w.n + 1), den=f32(w.T), tok_ptr=i32(w.T + 1), tok_rows=i32(S.R), loss=f32(1), thr_counts=i32(w.n),
               ws=B.empty_bytes(S.ws_bytes))
    for v in out.values():
        v.fill_(-1 if v.dtype != torch.uint8 else 255)
    B.moe_gate_balanced(cfg, dev_act(I["x"], w), dev(I["Wg"]), dev(thr), out["logits"], out["probs"], out["mask_bits"],
                        out["tok_of_row"], out["offsets"], out["den"], out["tok_ptr"], out["tok_rows"], out["loss"],
                        out["thr_counts"], out["ws"])
    return cfg, S, out


def test_balanced_gate(case):
    w, I, thr, F, Bk = case
    cfg, S, G = run_gate(w, I, thr)
    assert S.m == F.m and S.R == w.T * w.k
    assert (host(G["logits"]) == np.asarray(F.logits)).all(), "logits by the fixed fma chain"
    assert_close(host(G["probs"]), F.p, TOL_F32, "probs")
    assert (host(G["mask_bits"]).view(np.uint32) == packed(F.mask)).all(), "batchwise mask must be bit-exact"
    assert (host(G["tok_of_row"]) == F.D.tok_of_row).all() and (host(G["offsets"]) == F.D.offsets).all()
    ptr, rows = tok_lists(F.D, w.T)
    assert (host(G["tok_ptr"]) == ptr).all() and (host(G["tok_rows"]) == rows).all()
    assert_close(host(G["den"]), F.den, TOL_F32, "den")
    assert (host(G["thr_counts"]) == F.mask_thr.sum(axis=0)).all()
    assert 0.0 < (F.mask_thr != F.mask).mean() < 0.2
    assert_close(host(G["loss"]), F.loss, TOL_F32, "L_batchwise")


def test_balanced_ties_go_to_the_lower_token():
    """Every token appears twice (identical rows): each expert's column holds pairs of equal values, and where the cut
    falls between the two copies the earlier one must be kept, as in the oracle."""
    w = small_workload("bal-ties", T=240, d=32, h=16, n=16, k=3, act="bf16", seed=85)   # m = 45 is odd: every cut splits a pair
    I = synth.make_all(w)
    I["x"][1::2] = I["x"][0::2]
    thr = np.full(w.n, 1.0 / w.n, np.float32)
    F = O.forward_balanced(I["x"], I["Wg"], thr, I["W1"], I["b1"], I["W2"], I["b2"], w.k, "bf16")
    split = (F.mask[0::2] != F.mask[1::2])
    assert split.any() and (F.mask[0::2][split]).all()      # where the copies differ, the lower token has it
    cfg, S, G = run_gate(w, I, thr)
    assert (host(G["mask_bits"]).view(np.uint32) == packed(F.mask)).all()
    assert (host(G["tok_of_row"]) == F.D.tok_of_row).all()


def test_balanced_forward_backward(case):
    """gate -> dispatch -> experts (the unchanged grouped GEMMs on uniform segments) -> combine, and back."""
    w, I, thr, F, Bk = case
    cfg, S, G = run_gate(w, I, thr)
    x, dY = dev_act(I["x"], w), dev_act(I["dY"], w)
    W1, b1, W2, b2 = (dev_act(I[k_], w) for k_ in ("W1", "b1", "W2", "b2"))
    Sz = B.moe_query_sizes(cfg)
    ws = B.empty_bytes(Sz.ws_bytes)
    xs, hid, ys, y = act_empty(w, S.R, w.d), act_empty(w, S.R, w.h), act_empty(w, S.R, w.d), act_empty(w, w.T, w.d)
    B.moe_dispatch_balanced(cfg, x, G["tok_of_row"], xs)
    assert (host(xs) == np.asarray(F.D.xs, np.float32)).all()
    B.moe_expert_ffn(cfg, xs, G["offsets"], W1, b1, W2, b2, hid, ys, ws)
    B.moe_combine_balanced(cfg, ys, G["probs"], G["den"], G["tok_ptr"], G["tok_rows"], y)
    assert B.moe_check_status(ws) == 0
    tol = tol_act(w)
    assert_close(host(hid), F.hid, tol, "hid")
    assert_close(host(y), F.y, tol, "y")
    unkept = ~F.mask.any(axis=1)
    assert (host(y)[unkept] == 0).all()
    # backward
    dG_row, dys, dxs = f32(S.R), act_empty(w, S.R, w.d), act_empty(w, S.R, w.d)
    out = dict(dW1=act_empty(w, w.n, w.d, w.h), db1=act_empty(w, w.n, w.h), dW2=act_empty(w, w.n, w.h, w.d),
               db2=act_empty(w, w.n, w.d), dX=act_empty(w, w.T, w.d))
    B.moe_combine_balanced_bwd(cfg, dY, ys, G["probs"], G["den"], G["tok_of_row"], dG_row, dys)
    assert_close(host(dG_row), Bk.dG_row, tol if w.act == "bf16" else TOL_F32, "dG_row")
    assert_close(host(dys), Bk.dys, tol, "dys")
    B.moe_expert_ffn_bwd(cfg, xs, hid, dys, G["offsets"], W1, W2, dxs, out["dW1"], out["db1"], out["dW2"], out["db2"], ws)
    dWg, dXg, dthr = f32(w.d, w.n), f32(w.T, w.d), f32(w.n)
    B.moe_gate_balanced_bwd(cfg, x, dev(I["Wg"]), G["probs"], G["mask_bits"], G["den"], dev(thr), G["tok_ptr"], G["tok_rows"],
                            dG_row, G["thr_counts"], W_BATCHWISE, dWg, dXg, dthr, G["ws"])
    B.moe_dispatch_balanced_bwd(cfg, dxs, G["tok_ptr"], G["tok_rows"], dXg, out["dX"])
    assert B.moe_check_status(ws) == 0
    assert (host(dthr) == np.asarray(Bk.dthr, np.float32)).all(), "threshold gradients are exact (counts)"
    assert_close(host(dWg), Bk.dWg, tol, "dWg")
    assert_close(host(dXg), Bk.dX_gate, tol, "dX_gate")
    # the expert-side comparison of the flat layer, with the row tables of this gate (token of a row instead of slot / k)
    from types import SimpleNamespace as NS
    Fk = NS(hid=F.hid, D=NS(offsets=F.D.offsets, perm=F.D.tok_of_row.astype(np.int64)))
    w1 = NS(n=w.n, d=w.d, h=w.h, T=w.T, k=1)
    assert_expert_backward_close(w1, Fk, Bk, out, host(hid), tol)


def test_balanced_gate_backward_alone(case):
    """The gate's backward fed with the oracle's forward state and row gradients: fp32 path at 1e-5."""
    w, I, thr, F, Bk = case
    cfg = cfg_of(w)
    S = B.moe_query_balanced_sizes(cfg)
    ptr, rows = tok_lists(F.D, w.T)
    dWg, dXg, dthr = f32(w.d, w.n), f32(w.T, w.d), f32(w.n)
    B.moe_gate_balanced_bwd(cfg, dev_act(I["x"], w), dev(I["Wg"]), dev(np.asarray(F.p, np.float32)),
                            torch.from_numpy(packed(F.mask).view(np.int32)).cuda(), dev(np.asarray(F.den, np.float32)), dev(thr),
                            dev(ptr), dev(rows), dev(np.asarray(Bk.dG_row, np.float32)),
                            dev(F.mask_thr.sum(axis=0).astype(np.int32)), W_BATCHWISE, dWg, dXg, dthr, B.empty_bytes(S.ws_bytes))
    assert_close(host(dWg), Bk.dWg, TOL_F32, "dWg")
    assert_close(host(dXg), Bk.dX_gate, TOL_F32, "dX_gate")
    assert (host(dthr) == np.asarray(Bk.dthr, np.float32)).all()


def test_balanced_arguments_are_checked():
    w = small_workload("bal-args", T=100, d=16, h=16, n=8, k=3, seed=86)   # k T = 300 is no multiple of n = 8
    with pytest.raises(B.MoeError):
        B.moe_query_balanced_sizes(cfg_of(w))
    w = small_workload("bal-hier", T=64, d=16, h=16, n=16, k=4, a=4, k1=2, b=4, k2=2, seed=87)
    with pytest.raises(B.MoeError):
        B.moe_query_balanced_sizes(cfg_of(w))
