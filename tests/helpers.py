"""Shared test plumbing: workloads -> oracle results and device tensors, and the error metric."""
from __future__ import annotations

import numpy as np
import torch

from oracle import moe_oracle as O
from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

TOL_F32 = dict(max=1e-5, mean=1e-5)    # fp32 gating path and the all-fp32 layer
TOL_BF16 = dict(max=2e-2, mean=1e-2)   # bf16 expert outputs and gradients


def rel_err(got, want):
    """Per tensor: e_i = |got_i - want_i| / (|want_i| + rms(want)); returns (max e, mean e).
    The rms floor keeps near-zero elements produced by cancellation from dominating."""
    got = np.asarray(got, np.float64).reshape(-1)
    want = np.asarray(want, np.float64).reshape(-1)
    assert got.shape == want.shape, (got.shape, want.shape)
    if want.size == 0:
        return 0.0, 0.0
    assert np.isfinite(got).all(), "non-finite values in the result"
    rms = float(np.sqrt(np.mean(want * want)))
    e = np.abs(got - want) / (np.abs(want) + rms + 1e-300)
    return float(e.max()), float(e.mean())


def assert_close(got, want, tol, what=""):
    mx, mean = rel_err(got, want)
    assert mx <= tol["max"] and mean <= tol["mean"], f"{what}: max rel {mx:.3e}, mean rel {mean:.3e} (tol {tol})"
    return mx, mean


def prec_of(w):
    return "bf16" if w.act == "bf16" else "f32"


def tol_act(w):
    return TOL_BF16 if w.act == "bf16" else TOL_F32


SCREEN_ON, SCREEN_OFF = B.MOE_FLAG_GATE_SCREEN_ON, B.MOE_FLAG_GATE_SCREEN_OFF


def cfg_of(w, flags=0):
    """flags = 0 is what a user (and bench.py) gets: the library chooses its kernels by problem size."""
    return B.make_config(w.T, w.d, w.h, w.n, w.k, w.act, w.w_importance, w.w_load, w.a, w.k1, w.b, w.k2, flags)


def screened(w, flags=SCREEN_ON):
    """True where moe_gate screens the routing on the tensor cores: bf16, widths that are multiples of 64, and
    either forced (MOE_FLAG_GATE_SCREEN_ON) or a projection of at least 1e9 multiply-adds."""
    if flags & SCREEN_OFF:
        return False

    def level(rows, width):
        ok = w.act == "bf16" and rows >= 256 and w.d % 64 == 0 and (2 * width) % 64 == 0
        return ok and (bool(flags & SCREEN_ON) or float(rows) * w.d * 2.0 * width >= 1.0e9)

    first = level(w.T, w.a if w.a else w.n)
    # the secondary gates of the hierarchical layer are screened on their own (rows = T * k1 slots, width b)
    second = bool(w.a) and level(w.T * w.k1, w.b)
    return first or second


def cat_parts(parts):
    """Hierarchical gating tensors are (primary, secondary) pairs: flatten and concatenate."""
    if isinstance(parts, (tuple, list)):
        return np.concatenate([np.asarray(p, np.float32).reshape(-1) for p in parts])
    return np.asarray(parts, np.float32).reshape(-1)


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def dev_act(a, w):
    return dev(np.asarray(a, np.float32), torch.bfloat16 if w.act == "bf16" else torch.float32)


def host(t):
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def device_inputs(w, I):
    """Device copies of a workload's inputs, in the layouts of the ABI."""
    return dict(x=dev_act(I["x"], w), Wg=dev(cat_parts(I["Wg"])), Wnoise=dev(cat_parts(I["Wnoise"])),
                noise=dev(cat_parts(I["noise"])), W1=dev_act(I["W1"], w), b1=dev_act(I["b1"], w),
                W2=dev_act(I["W2"], w), b2=dev_act(I["b2"], w), dY=dev_act(I["dY"], w))


def oracle_run(w, I, backward=True):
    prec = prec_of(w)
    F = O.forward(I["x"], I["Wg"], I["Wnoise"], I["noise"], I["W1"], I["b1"], I["W2"], I["b2"], w.k,
                  w.w_importance, w.w_load, prec, hier=w.hier)
    Bk = None
    if backward:
        Bk = O.backward(I["dY"], I["x"], I["Wg"], I["Wnoise"], I["noise"], I["W1"], I["b1"], I["W2"], I["b2"], F,
                        w.w_importance, w.w_load, prec, hier=w.hier)
    return F, Bk


def f32(*shape):
    return torch.empty(*shape, dtype=torch.float32, device="cuda")


def i32(*shape):
    return torch.empty(*shape, dtype=torch.int32, device="cuda")


def act_empty(w, *shape):
    return torch.empty(*shape, dtype=torch.bfloat16 if w.act == "bf16" else torch.float32, device="cuda")


def small_workload(name, T, d, h, n, k, act="f32", seed=1, **kw):
    return synth.Workload(name, T=T, d=d, h=h, n=n, k=k, act=act, seed=synth.BASE_SEED + 1000 + seed,
                          bias_std=kw.pop("bias_std", 0.3), **kw)


def assert_expert_backward_close(w, F, Bk, G, hid, tol, max_flip_rate=2e-5):
    """Expert-side gradients of a fused run (dict G) against the oracle's backward Bk, aware of ReLU flips.

    The ReLU derivative is a yes/no decision on a rounded number: where the pre-activation is within
    rounding of 0 the two sides may legitimately decide differently. Those (row, hidden unit) pairs must
    be rare and tiny; what they feed (column j of dW1/db1 of that expert, the token's dX) is set aside,
    everything else must meet the tolerance. Returns the number of flips."""
    want_hid = np.asarray(F.hid)
    flip_r, flip_j = np.nonzero((hid > 0) != (want_hid > 0))
    assert flip_r.size <= max(2, max_flip_rate * hid.size), f"{flip_r.size} ReLU decisions differ"
    if flip_r.size:
        rms_hid = float(np.sqrt(np.mean(want_hid.astype(np.float64) ** 2)))
        assert np.abs(hid[flip_r, flip_j]).max() <= 1e-2 * rms_hid
        assert np.abs(want_hid[flip_r, flip_j]).max() <= 1e-2 * rms_hid
    flip_e = np.searchsorted(F.D.offsets[1:], flip_r, side="right")
    flip_tok = F.D.perm[flip_r] // w.k
    keep = {"dW1": np.ones((w.n, w.d, w.h), bool), "db1": np.ones((w.n, w.h), bool),
            "dX": np.ones((w.T, w.d), bool)}
    keep["dW1"][flip_e, :, flip_j] = False
    keep["db1"][flip_e, flip_j] = False
    keep["dX"][flip_tok] = False
    for name in ("dW1", "db1", "dW2", "db2", "dX"):
        got, want = host(G[name]), np.asarray(getattr(Bk, name))
        if name in keep and flip_r.size:
            got, want = got[keep[name]], want[keep[name]]
        assert_close(got, want, tol, name)
    return int(flip_r.size)
