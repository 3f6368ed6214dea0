"""Plain CPU statement of the Sparsely-Gated Mixture-of-Experts layer.

TEST INFRASTRUCTURE -- slow on purpose, written to be checked against the paper
by eye. Only tests, the smoke check and the benchmark's CPU-baseline leg may use
it. It shares nothing with the CUDA library.

Every function cites the equation it follows. Arithmetic is float64 except where
a rounding decides an integer: the gate logits H(x) of Eq. 4 (they decide the
routing of Eq. 5) are evaluated in single precision in one fixed order, see
`project` / `noisy_logits` and `chain.c`.

Precision modes (`prec`):
  "f64"  everything in float64, nothing rounded: used by the finite-difference
         and closed-form pins.
  "f32"  gate logits in the fixed single-precision order; every tensor the
         layer materialises is rounded once to float32.
  "bf16" as "f32" for the gating tensors; expert-side tensors (hid, ys, y and
         the backward tensors dys, dz, dxs, weight/bias gradients, dX) are
         rounded once to bfloat16, round-to-nearest-even.
Reductions over the batch (Importance, Load, bias and weight gradients) are
accumulated in float64 and rounded once.

Pins (tests/test_oracle_*.py): exactly-k / sum-to-one invariants and brute-force
top-k; k = n with zero noise equals the dense softmax mixture of Eq. 2 into
Eq. 1; one expert equals a textbook two-layer MLP; dispatch/combine round trip;
CV^2 closed forms; P(x, i) against Monte-Carlo on its definition, against a
delete-and-sort kth_excluding, and against the zero-initialisation closed form;
hierarchical reductions to the flat layer; every backward against central finite
differences of the forward in float64; the single-precision chain against an
exact rational emulation; the layer epilogue (sigmoid, dropout, residual) against its
closed forms and finite differences; strictly balanced gating against brute-force column
sorts, its counting invariants and finite differences; the factored optimiser step against full Adam
on rank-one squared gradients and its textbook limits. The table of trained-model balance metrics in the
paper's Appendix A cannot be reproduced without the trained model: for those
printed values parity is unpinned; the metric definitions themselves are pinned
by the CV^2 closed forms.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from types import SimpleNamespace

import numpy as np
from scipy.special import ndtr  # Phi, the standard normal CDF of Eq. 9

f32 = np.float32
f64 = np.float64
_HERE = os.path.dirname(os.path.abspath(__file__))
_CHAIN = None


# --------------------------------------------------------------------------------------
# the single-precision chain (compiled C, because numpy has no fused multiply-add)
# --------------------------------------------------------------------------------------
def build_chain_library(force: bool = False) -> str:
    """Compile chain.c next to its source (gcc); returns the path of the library."""
    src = os.path.join(_HERE, "chain.c")
    out = os.path.join(_HERE, "liboracle_chain.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        tmp = out + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-mfma", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, src, "-lm"])
        os.replace(tmp, out)
    return out


def _chain():
    global _CHAIN
    if _CHAIN is None:
        lib = ctypes.CDLL(build_chain_library())
        i64, fp = ctypes.c_int64, ctypes.POINTER(ctypes.c_float)
        lib.oracle_proj_chain_f32.argtypes = [i64, i64, i64, fp, i64, fp, fp]
        lib.oracle_proj_chain_f32.restype = None
        lib.oracle_fma_f32.argtypes = [i64, fp, fp, fp, fp]
        lib.oracle_fma_f32.restype = None
        _CHAIN = lib
    return _CHAIN


def _fp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


# --------------------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------------------
def round_bf16(a):
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=f32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(f32).reshape(a.shape)


def store(a, prec, expert_side=False):
    """Round once to the type in which the layer materialises this tensor."""
    if prec == "f64":
        return np.asarray(a, dtype=f64)
    a32 = np.asarray(a, dtype=f64).astype(f32)
    if prec == "bf16" and expert_side:
        return round_bf16(a32)
    return a32


# --------------------------------------------------------------------------------------
# gating: Eq. 3, 4, 5
# --------------------------------------------------------------------------------------
def project(x, W, prec):
    """(x . W) of Eq. 2 / Eq. 4. In the rounded modes: one fused-multiply-add chain per
    output over the input features in ascending order, single precision, from +0."""
    if prec == "f64":
        return np.asarray(x, f64) @ np.asarray(W, f64)
    x = np.ascontiguousarray(x, dtype=f32)
    W = np.ascontiguousarray(W, dtype=f32)
    T, d = x.shape
    n = W.shape[1]
    out = np.empty((T, n), f32)
    if T:
        _chain().oracle_proj_chain_f32(T, d, n, _fp(x), d, _fp(W), _fp(out))
    return out


def softplus(r, prec):
    """Softplus of Eq. 4, log(1 + e^r), in its overflow-free form, evaluated in float64."""
    r64 = np.asarray(r, f64)
    s = np.maximum(r64, 0.0) + np.log1p(np.exp(-np.abs(r64)))
    return s if prec == "f64" else s.astype(f32)


def noisy_logits(clean, noise, sigma, prec):
    """H(x) = x.W_g + StandardNormal() * Softplus(x.W_noise)   (Eq. 4).
    Rounded modes: a single fused multiply-add, i.e. one rounding."""
    if prec == "f64":
        return np.asarray(clean, f64) + np.asarray(noise, f64) * np.asarray(sigma, f64)
    a = np.ascontiguousarray(noise, dtype=f32)
    b = np.ascontiguousarray(sigma, dtype=f32)
    c = np.ascontiguousarray(clean, dtype=f32)
    out = np.empty_like(c)
    if c.size:
        _chain().oracle_fma_f32(c.size, _fp(a), _fp(b), _fp(c), _fp(out))
    return out


def keep_top_k(H, k):
    """KeepTopK (Eq. 5): the k largest entries of each row, the lowest index winning ties,
    reported in descending order. Also returns the k-th and (k+1)-th largest (value and
    index), which Eq. 9 needs; the (k+1)-th is (-inf, -1) when k = n."""
    T, n = H.shape
    assert 1 <= k <= n
    order = np.argsort(-H, axis=1, kind="stable")  # descending H; equal H keep index order
    rows = np.arange(T)
    idx = order[:, :k].astype(np.int32)
    kth_idx = np.full((T, 2), -1, np.int32)
    kth_val = np.full((T, 2), -np.inf, H.dtype)
    kth_idx[:, 0] = order[:, k - 1]
    kth_val[:, 0] = H[rows, order[:, k - 1]]
    if k < n:
        kth_idx[:, 1] = order[:, k]
        kth_val[:, 1] = H[rows, order[:, k]]
    return idx, kth_val, kth_idx


def softmax_of_kept(H, idx, prec):
    """Softmax over the kept entries (Eq. 3); the -inf entries give gate 0 and are not stored."""
    Hk = np.take_along_axis(H, idx.astype(np.int64), axis=1).astype(f64)
    e = np.exp(Hk - Hk[:, :1])  # slot 0 holds the row maximum
    den = e[:, 0].copy()
    for s in range(1, idx.shape[1]):
        den = den + e[:, s]
    return store(e / den[:, None], prec)


def gate(x, Wg, Wnoise, noise, k, prec):
    """Noisy top-k gating G(x) = Softmax(KeepTopK(H(x), k))   (Eq. 3-5).

    Returns idx [T,k] (expert of each kept slot, descending H), gates [T,k], the clean
    logits x.W_g [T,n], the raw noise logits x.W_noise [T,n], sigma, H and the k-th /
    (k+1)-th order statistics of H."""
    clean = project(x, Wg, prec)
    raw = project(x, Wnoise, prec)
    sigma = softplus(raw, prec)
    H = noisy_logits(clean, noise, sigma, prec)
    idx, kth_val, kth_idx = keep_top_k(H, k)
    gates = softmax_of_kept(H, idx, prec)
    return SimpleNamespace(idx=idx, gates=gates, clean=clean, raw=raw, sigma=sigma, H=H,
                           kth_val=kth_val, kth_idx=kth_idx)


# --------------------------------------------------------------------------------------
# routing: each expert receives the batch of the examples that selected it (Section 3.1)
# --------------------------------------------------------------------------------------
def dispatch(x, idx, n):
    """Stable counting sort of the slots p = t*k + s by expert.

    counts[e] rows go to expert e; offsets is the exclusive prefix sum (offsets[n] = T*k);
    perm[r] = slot held by sorted row r; inv_perm[p] = sorted row of slot p; xs[r] is a
    copy of the token row x[perm[r] // k]."""
    T, k = idx.shape
    flat = idx.reshape(-1).astype(np.int64)
    counts = np.bincount(flat, minlength=n).astype(np.int32)
    offsets = np.zeros(n + 1, np.int32)
    offsets[1:] = np.cumsum(counts)
    perm = np.argsort(flat, kind="stable").astype(np.int32)
    inv_perm = np.empty(T * k, np.int32)
    inv_perm[perm] = np.arange(T * k, dtype=np.int32)
    xs = np.asarray(x)[perm // k]
    return SimpleNamespace(xs=xs, perm=perm, inv_perm=inv_perm, counts=counts, offsets=offsets)


def expert_ffn(xs, offsets, W1, b1, W2, b2, prec):
    """Each expert is a feed-forward network with one ReLU hidden layer (Section 3.2,
    Appendix C): hid = relu(xs.W1_e + b1_e), ys = hid.W2_e + b2_e on the expert's rows."""
    R = xs.shape[0]
    n, d, h = W1.shape
    out_t = f64 if prec == "f64" else f32
    hid = np.zeros((R, h), out_t)
    ys = np.zeros((R, W2.shape[2]), out_t)
    for e in range(n):
        o0, o1 = int(offsets[e]), int(offsets[e + 1])
        if o0 == o1:
            continue
        z = np.asarray(xs[o0:o1], f64) @ np.asarray(W1[e], f64) + np.asarray(b1[e], f64)
        hid[o0:o1] = store(np.maximum(z, 0.0), prec, expert_side=True)
        ys[o0:o1] = store(np.asarray(hid[o0:o1], f64) @ np.asarray(W2[e], f64)
                          + np.asarray(b2[e], f64), prec, expert_side=True)
    return hid, ys


def combine(ys, gates, inv_perm, prec):
    """y = sum_i G(x)_i E_i(x) over the k experts with a non-zero gate (Eq. 1)."""
    T, k = gates.shape
    rows = inv_perm.reshape(T, k).astype(np.int64)
    y = np.zeros((T, ys.shape[1]), f64)
    for s in range(k):
        y = y + np.asarray(gates[:, s], f64)[:, None] * np.asarray(ys[rows[:, s]], f64)
    return store(y, prec, expert_side=True)


def unpack_keep(keep_bits, d):
    """Dropout keep mask [T, d] (bool) from its packed form: bit (q % 8) of byte q // 8 of a row is column q."""
    bits = np.unpackbits(np.asarray(keep_bits, np.uint8), axis=1, bitorder="little")
    return bits[:, :d].astype(bool)


def combine_layer(ys, gates, inv_perm, x, keep, drop_prob, prec):
    """The MoE layer as it sits in the paper's models (Appendix C, model and MoE layer architecture): the MoE output
    y of Eq. 1 goes through a sigmoid, then dropout (each activation dropped with probability DropProb, the kept
    ones divided by 1 - DropProb), then the layer's input is added (residual connection):
        out = x + keep * sigmoid(y) / (1 - DropProb).
    `keep` [T, d] is the 0/1 dropout mask, an input (drawn by the caller, like the gating noise). Only `out` is
    materialised (one rounding); y stays in working precision."""
    T, k = gates.shape
    rows = inv_perm.reshape(T, k).astype(np.int64)
    y = np.zeros((T, ys.shape[1]), f64)
    for s in range(k):
        y = y + np.asarray(gates[:, s], f64)[:, None] * np.asarray(ys[rows[:, s]], f64)
    sig = 1.0 / (1.0 + np.exp(-y))
    out = np.asarray(x, f64) + np.asarray(keep, f64) * sig / (1.0 - drop_prob)
    return store(out, prec, expert_side=True)


def combine_layer_bwd(dOut, ys, gates, inv_perm, keep, drop_prob, prec):
    """Adjoint of combine_layer. Through the residual connection dOut reaches the layer input unchanged (the
    caller adds it to dX); through dropout and the sigmoid dy = dOut * keep / (1 - DropProb) * s (1 - s) with
    s = sigmoid(y), and from there on as in combine_bwd."""
    T, k = gates.shape
    rows = inv_perm.reshape(T, k).astype(np.int64)
    y = np.zeros((T, ys.shape[1]), f64)
    for s in range(k):
        y = y + np.asarray(gates[:, s], f64)[:, None] * np.asarray(ys[rows[:, s]], f64)
    sig = 1.0 / (1.0 + np.exp(-y))
    dy = np.asarray(dOut, f64) * np.asarray(keep, f64) / (1.0 - drop_prob) * sig * (1.0 - sig)
    dgates = np.zeros((T, k), f64)
    dys = np.zeros(ys.shape, f64)
    for s in range(k):
        dgates[:, s] = (dy * np.asarray(ys[rows[:, s]], f64)).sum(axis=1)
        dys[rows[:, s]] = np.asarray(gates[:, s], f64)[:, None] * dy
    return store(dgates, prec), store(dys, prec, expert_side=True)


# --------------------------------------------------------------------------------------
# balancing losses: Eq. 6, 7 and Eq. 8-11
# --------------------------------------------------------------------------------------
def cv_squared(v):
    """Square of the coefficient of variation (Eq. 7, 11): population variance / mean^2."""
    v = np.asarray(v, f64).reshape(-1)
    mu = v.mean()
    return float(((v - mu) ** 2).mean() / (mu * mu))


def importance_of(idx, gates, n):
    """Importance(X) = sum over the batch of G(x)   (Eq. 6)."""
    imp = np.zeros(n, f64)
    np.add.at(imp, idx.reshape(-1).astype(np.int64), np.asarray(gates, f64).reshape(-1))
    return imp


def selected_mask(idx, n):
    T = idx.shape[0]
    sel = np.zeros((T, n), bool)
    sel[np.arange(T)[:, None], idx.astype(np.int64)] = True
    return sel


def load_probability(clean, sigma, idx, kth_val):
    """P(x, i) = Phi((x.W_g)_i - kth_excluding(H(x), k, i)) / Softplus((x.W_noise)_i))  (Eq. 9).

    kth_excluding(H, k, i) is the k-th largest entry of H once entry i is removed: removing
    a selected entry promotes the (k+1)-th largest, removing any other leaves the k-th."""
    sel = selected_mask(idx, clean.shape[1])
    thr = np.where(sel, np.asarray(kth_val[:, 1:2], f64), np.asarray(kth_val[:, 0:1], f64))
    with np.errstate(invalid="ignore"):
        z = (np.asarray(clean, f64) - thr) / np.asarray(sigma, f64)
    return ndtr(z), z, sel


def losses(idx, gates, clean, raw, kth_val, w_importance, w_load, prec):
    """Importance (Eq. 6), Load (Eq. 10) and the two scaled CV^2 losses (Eq. 7, Eq. 11)."""
    n = clean.shape[1]
    imp = importance_of(idx, gates, n)
    P, _, _ = load_probability(clean, softplus(raw, prec), idx, kth_val)
    load = P.sum(axis=0)
    L = np.array([w_importance * cv_squared(imp), w_load * cv_squared(load)], f64)
    return SimpleNamespace(importance=store(imp, prec), load=store(load, prec), losses=store(L, prec))


def cv_squared_grad(v):
    """d CV^2(v) / d v_i = 2 / (m mu^2) * ((v_i - mu) - Var(v) / mu)."""
    v = np.asarray(v, f64).reshape(-1)
    m = v.size
    mu = v.mean()
    var = ((v - mu) ** 2).mean()
    return 2.0 / (m * mu * mu) * ((v - mu) - var / mu)


# --------------------------------------------------------------------------------------
# backward (Section 2.1, "Training the Gating Network": plain back-propagation; the
# formulas are the exact derivatives of the forward above)
# --------------------------------------------------------------------------------------
def combine_bwd(dY, ys, gates, inv_perm, prec):
    """Adjoint of Eq. 1: dgates[t,s] = <dY[t], ys[row]>, dys[row] = gates[t,s] dY[t]."""
    T, k = gates.shape
    rows = inv_perm.reshape(T, k).astype(np.int64)
    dY64 = np.asarray(dY, f64)
    dgates = np.zeros((T, k), f64)
    dys = np.zeros(ys.shape, f64)
    for s in range(k):
        dgates[:, s] = (dY64 * np.asarray(ys[rows[:, s]], f64)).sum(axis=1)
        dys[rows[:, s]] = np.asarray(gates[:, s], f64)[:, None] * dY64
    return store(dgates, prec), store(dys, prec, expert_side=True)


def expert_ffn_bwd(xs, hid, dys, offsets, W1, W2, prec):
    """Back-propagation through one-hidden-layer ReLU experts (derivative 0 at 0)."""
    n, d, h = W1.shape
    out_t = f64 if prec == "f64" else f32
    dxs = np.zeros(xs.shape, out_t)
    dz_all = np.zeros(hid.shape, out_t)
    dW1 = np.zeros(W1.shape, out_t)
    dW2 = np.zeros(W2.shape, out_t)
    db1 = np.zeros((n, h), out_t)
    db2 = np.zeros((n, W2.shape[2]), out_t)
    for e in range(n):
        o0, o1 = int(offsets[e]), int(offsets[e + 1])
        if o0 == o1:
            continue
        dy = np.asarray(dys[o0:o1], f64)
        hd = np.asarray(hid[o0:o1], f64)
        db2[e] = store(dy.sum(axis=0), prec, True)
        dW2[e] = store(hd.T @ dy, prec, True)
        dhid = dy @ np.asarray(W2[e], f64).T
        dz = store(dhid * (hd > 0.0), prec, True)
        dz_all[o0:o1] = dz
        dz64 = np.asarray(dz, f64)
        db1[e] = store(dz64.sum(axis=0), prec, True)
        dW1[e] = store(np.asarray(xs[o0:o1], f64).T @ dz64, prec, True)
        dxs[o0:o1] = store(dz64 @ np.asarray(W1[e], f64).T, prec, True)
    return SimpleNamespace(dxs=dxs, dW1=dW1, db1=db1, dW2=dW2, db2=db2, dz=dz_all)


def dispatch_bwd(dxs, inv_perm, T, k, prec):
    """Adjoint of the row copies: dX_expert[t] = sum_s dxs[inv_perm[t*k+s]]."""
    rows = inv_perm.reshape(T, k).astype(np.int64)
    dX = np.zeros((T, dxs.shape[1]), f64)
    for s in range(k):
        dX = dX + np.asarray(dxs[rows[:, s]], f64)
    return store(dX, prec)


def losses_bwd(importance, load, idx, dgates, w_importance, w_load, prec):
    """Adds d L_importance / d gates to dgates and returns d L_load / d Load  (Eq. 7, 11)."""
    dI = w_importance * cv_squared_grad(importance)
    dload = w_load * cv_squared_grad(load)
    out = np.asarray(dgates, f64) + dI[idx.astype(np.int64)]
    return store(out, prec), store(dload, prec)


def gate_logit_grads(noise, clean, raw, idx, gates, kth_val, kth_idx, dgates, dload, prec):
    """Gradients of the main path and of L_load w.r.t. the clean logits c = x.W_g and the raw
    noise logits r = x.W_noise. dload is d L / d Load [n] (or [T,n] per-row weights)."""
    T, n = clean.shape
    k = idx.shape[1]
    rows = np.arange(T)
    idx64 = idx.astype(np.int64)
    g = np.asarray(gates, f64)
    dg = np.asarray(dgates, f64)
    eps = np.asarray(noise, f64)
    sigma = np.asarray(softplus(raw, prec), f64)
    # softmax over the kept slots (Eq. 3)
    dH = np.zeros((T, n), f64)
    inner = (g * dg).sum(axis=1)
    dH[rows[:, None], idx64] = g * (dg - inner[:, None])
    # load estimator (Eq. 9, 10): dP -> z -> (c, thr, sigma)
    P, z, sel = load_probability(clean, sigma, idx, kth_val)
    finite = np.isfinite(z)
    zf = np.where(finite, z, 0.0)
    phi = np.where(finite, np.exp(-0.5 * zf * zf) / math.sqrt(2.0 * math.pi), 0.0)
    dP = np.broadcast_to(np.asarray(dload, f64), (T, n))
    q = dP * phi / sigma
    dc = q.copy()
    dsigma = -zf * q
    if k < n:  # the threshold is another entry's noisy logit: it receives -q
        np.add.at(dH, (rows, kth_idx[:, 1].astype(np.int64)), -(q * sel).sum(axis=1))
        np.add.at(dH, (rows, kth_idx[:, 0].astype(np.int64)), -(q * ~sel).sum(axis=1))
    # H = c + eps * softplus(r)   (Eq. 4)
    dc = dc + dH
    dsigma = dsigma + eps * dH
    r64 = np.asarray(raw, f64)
    dr = dsigma / (1.0 + np.exp(-r64))
    return dc, dr


def gate_bwd(x, Wg, Wnoise, noise, clean, raw, idx, gates, kth_val, kth_idx, dgates, dload, prec):
    """Back-propagation through the gating network to W_g, W_noise and the layer input."""
    dc, dr = gate_logit_grads(noise, clean, raw, idx, gates, kth_val, kth_idx, dgates, dload, prec)
    x64 = np.asarray(x, f64)
    dWg = x64.T @ dc
    dWn = x64.T @ dr
    dXg = dc @ np.asarray(Wg, f64).T + dr @ np.asarray(Wnoise, f64).T
    return SimpleNamespace(dWg=store(dWg, prec), dWnoise=store(dWn, prec), dX_gate=store(dXg, prec),
                           dclean=dc, draw=dr)


# --------------------------------------------------------------------------------------
# hierarchical mixture of experts (Appendix B, Eq. 12-14)
# --------------------------------------------------------------------------------------
def gate_h(x, Wg_p, Wn_p, noise_p, Wg_s, Wn_s, noise_s, k1, k2, prec):
    """Primary gate over a groups, then for each kept group its own secondary gate over b
    experts. Flat expert id i*b + j, gate G_primary(x)_i * G_i(x)_j   (Eq. 12). Slots are
    ordered primary slot major, secondary slot minor; noise_s is [T, k1, b], indexed by
    primary slot."""
    T = x.shape[0]
    a, d, b = Wg_s.shape
    P = gate(x, Wg_p, Wn_p, noise_p, k1, prec)
    lt = f64 if prec == "f64" else f32
    S = SimpleNamespace(idx=np.zeros((T, k1, k2), np.int32), gates=np.zeros((T, k1, k2), lt),
                        clean=np.zeros((T, k1, b), lt), raw=np.zeros((T, k1, b), lt),
                        sigma=np.zeros((T, k1, b), lt), H=np.zeros((T, k1, b), lt),
                        kth_val=np.zeros((T, k1, 2), lt), kth_idx=np.zeros((T, k1, 2), np.int32))
    for s1 in range(k1):
        for i in range(a):
            rows = np.nonzero(P.idx[:, s1] == i)[0]
            if rows.size == 0:
                continue
            G = gate(np.asarray(x)[rows], Wg_s[i], Wn_s[i], np.asarray(noise_s)[rows, s1], k2, prec)
            for name in ("idx", "gates", "clean", "raw", "sigma", "H", "kth_val", "kth_idx"):
                getattr(S, name)[rows, s1] = getattr(G, name)
    idx = (P.idx[:, :, None].astype(np.int64) * b + S.idx).reshape(T, k1 * k2).astype(np.int32)
    w = store(np.asarray(P.gates, f64)[:, :, None] * np.asarray(S.gates, f64), prec).reshape(T, k1 * k2)
    return SimpleNamespace(idx=idx, gates=w, primary=P, secondary=S)


def losses_h(G, a, b, w_importance, w_load, prec):
    """Importance_H (Eq. 13) and Load_H = Load_primary_i * Load_i(X^(i))_j / |X^(i)| (Eq. 14),
    CV^2 of each taken over all a*b entries. A group no example selected has Load_H = 0."""
    P, S = G.primary, G.secondary
    T, k1 = P.idx.shape
    imp = importance_of(G.idx, G.gates, a * b)
    Pp, _, _ = load_probability(P.clean, P.sigma, P.idx, P.kth_val)
    load_p = Pp.sum(axis=0)
    load_s = np.zeros((a, b), f64)
    cnt = np.zeros(a, f64)
    for s1 in range(k1):
        Ps, _, _ = load_probability(S.clean[:, s1], S.sigma[:, s1], S.idx[:, s1], S.kth_val[:, s1])
        np.add.at(load_s, P.idx[:, s1].astype(np.int64), Ps)
        np.add.at(cnt, P.idx[:, s1].astype(np.int64), 1.0)
    safe = np.where(cnt > 0, cnt, 1.0)
    load_h = np.where(cnt[:, None] > 0, load_p[:, None] * load_s / safe[:, None], 0.0)
    L = np.array([w_importance * cv_squared(imp), w_load * cv_squared(load_h)], f64)
    return SimpleNamespace(importance=store(imp, prec), load=store(load_h.reshape(-1), prec),
                           losses=store(L, prec), load_p=load_p, load_s=load_s, cnt=cnt)


def gate_h_bwd(x, Wg_p, Wn_p, noise_p, Wg_s, Wn_s, noise_s, G, LS, dgates, w_importance, w_load, prec):
    """Back-propagation through both gating levels, including both balancing losses.
    dgates [T, k1*k2] is the main-path gradient w.r.t. the product gates."""
    P, S = G.primary, G.secondary
    T, k1 = P.idx.shape
    k2 = S.idx.shape[2]
    a, d, b = Wg_s.shape
    dI = w_importance * cv_squared_grad(LS.importance)
    dLH = (w_load * cv_squared_grad(LS.load)).reshape(a, b)
    dw = (np.asarray(dgates, f64) + dI[G.idx.astype(np.int64)]).reshape(T, k1, k2)
    gp = np.asarray(P.gates, f64)
    gs = np.asarray(S.gates, f64)
    dgs = dw * gp[:, :, None]
    dgp = (dw * gs).sum(axis=2)
    safe = np.where(LS.cnt > 0, LS.cnt, 1.0)
    live = (LS.cnt > 0)[:, None]
    dload_p = np.where(live, dLH * LS.load_s / safe[:, None], 0.0).sum(axis=1)
    dload_s = np.where(live, dLH * LS.load_p[:, None] / safe[:, None], 0.0)  # [a, b]
    out = gate_bwd(x, Wg_p, Wn_p, noise_p, P.clean, P.raw, P.idx, P.gates, P.kth_val, P.kth_idx,
                   dgp, dload_p, prec)
    dXg = np.asarray(out.dX_gate, f64).copy()
    dWg_s = np.zeros(Wg_s.shape, f64)
    dWn_s = np.zeros(Wn_s.shape, f64)
    x64 = np.asarray(x, f64)
    for s1 in range(k1):
        grp = P.idx[:, s1].astype(np.int64)
        dc, dr = gate_logit_grads(np.asarray(noise_s)[:, s1], S.clean[:, s1], S.raw[:, s1], S.idx[:, s1],
                                  S.gates[:, s1], S.kth_val[:, s1], S.kth_idx[:, s1], dgs[:, s1],
                                  dload_s[grp], prec)
        for i in range(a):
            rows = np.nonzero(grp == i)[0]
            if rows.size == 0:
                continue
            dWg_s[i] += x64[rows].T @ dc[rows]
            dWn_s[i] += x64[rows].T @ dr[rows]
            dXg[rows] += dc[rows] @ np.asarray(Wg_s[i], f64).T + dr[rows] @ np.asarray(Wn_s[i], f64).T
    return SimpleNamespace(dWg_p=out.dWg, dWn_p=out.dWnoise, dWg_s=store(dWg_s, prec),
                           dWn_s=store(dWn_s, prec), dX_gate=store(dXg, prec))


# --------------------------------------------------------------------------------------
# strictly balanced gating (Appendix F, Eq. 15-20)
# --------------------------------------------------------------------------------------
def softmax_gate(x, Wg, prec):
    """G_sigma(x) = Softmax(x . W_g)   (Eq. 15). The logits come from `project` (the fixed single-precision chain in
    the rounded modes, because the masks below are integer decisions taken on these numbers); the exponentials and
    their sum are taken in float64, largest logit subtracted first, and the quotient is rounded once."""
    c = project(x, Wg, prec)
    c64 = np.asarray(c, f64)
    e = np.exp(c64 - c64.max(axis=1, keepdims=True))
    den = np.zeros(c64.shape[0], f64)
    for i in range(c64.shape[1]):  # ascending expert
        den = den + e[:, i]
    p = e / den[:, None]
    return c, (p if prec == "f64" else p.astype(f32))


def batchwise_mask(p, m):
    """M_batchwise(X, m)   (Eq. 18): for every expert (column) the m largest values over the batch are kept, so that
    every expert receives exactly m examples; equal values go to the lower token index."""
    T, n = p.shape
    assert 0 <= m <= T
    mask = np.zeros((T, n), bool)
    for i in range(n):
        order = np.argsort(-np.asarray(p[:, i]), kind="stable")  # descending value, equal values keep token order
        mask[order[:m], i] = True
    return mask


def threshold_mask(p, thr):
    """M_threshold(x, T)_i = 1 if x_i > T_i   (Eq. 19), the mask used when no batch is available (inference)."""
    return np.asarray(p) > np.asarray(thr)[None, :]


def masked_gate(p, mask, prec):
    """G(x)_i = G_sigma(x)_i M_i / sum_j G_sigma(x)_j M_j   (Eq. 16); an example no expert keeps has G(x) = 0.
    The denominator is summed in ascending expert order."""
    p64 = np.asarray(p, f64)
    den = np.zeros(p64.shape[0], f64)
    for i in range(p64.shape[1]):
        den = den + np.where(mask[:, i], p64[:, i], 0.0)
    safe = np.where(den > 0, den, 1.0)
    G = np.where(mask, p64 / safe[:, None], 0.0)
    return store(G, prec), store(den, prec)


def batchwise_loss(p, mask_b, thr):
    """L_batchwise(X, T, m) = sum_j sum_i (M_threshold(x_j, T)_i - M_batchwise(X, m)_{j,i}) (X_{j,i} - T_i)   (Eq. 20):
    zero exactly when the two masks agree, positive otherwise."""
    p64, t64 = np.asarray(p, f64), np.asarray(thr, f64)[None, :]
    diff = threshold_mask(p, thr).astype(f64) - np.asarray(mask_b, f64)
    return float((diff * (p64 - t64)).sum())


def dispatch_balanced(x, mask):
    """Each expert receives the examples its mask column keeps, in token order: sorted row r belongs to expert
    r // m when every column keeps m. Returns the token of each row, the expert of each row, offsets and xs."""
    T, n = mask.shape
    tok, exp = [], []
    offsets = np.zeros(n + 1, np.int32)
    for i in range(n):
        rows = np.nonzero(mask[:, i])[0]
        tok.append(rows)
        exp.append(np.full(rows.size, i))
        offsets[i + 1] = offsets[i] + rows.size
    tok = np.concatenate(tok).astype(np.int32) if n else np.zeros(0, np.int32)
    exp = np.concatenate(exp).astype(np.int32) if n else np.zeros(0, np.int32)
    return SimpleNamespace(tok_of_row=tok, expert_of_row=exp, offsets=offsets, xs=np.asarray(x)[tok])


def combine_balanced(ys, G, tok_of_row, expert_of_row, T, prec):
    """y = sum_i G(x)_i E_i(x)   (Eq. 1) over however many experts keep the example, in ascending expert order."""
    y = np.zeros((T, ys.shape[1]), f64)
    G64 = np.asarray(G, f64)
    for r in range(len(tok_of_row)):  # rows are sorted by expert, so every token adds its experts in ascending order
        t, e = int(tok_of_row[r]), int(expert_of_row[r])
        y[t] += G64[t, e] * np.asarray(ys[r], f64)
    return store(y, prec, expert_side=True)


def combine_balanced_bwd(dY, ys, G, tok_of_row, expert_of_row, prec):
    """Adjoint of combine_balanced: dG of each row's (token, expert) pair and dys."""
    dY64, G64 = np.asarray(dY, f64), np.asarray(G, f64)
    t, e = tok_of_row.astype(np.int64), expert_of_row.astype(np.int64)
    dG_row = (dY64[t] * np.asarray(ys, f64)).sum(axis=1)
    dys = G64[t, e][:, None] * dY64[t]
    return store(dG_row, prec), store(dys, prec, expert_side=True)


def gate_balanced_bwd(x, Wg, p, mask_b, thr, dG_row, tok_of_row, expert_of_row, w_batchwise, prec):
    """Back-propagation through Eq. 16 (the mask is a constant), Eq. 20 scaled by w_batchwise, and the softmax of
    Eq. 15, to W_g, the layer input and the thresholds."""
    T, n = p.shape
    p64 = np.asarray(p, f64)
    dG = np.zeros((T, n), f64)
    dG[tok_of_row.astype(np.int64), expert_of_row.astype(np.int64)] = np.asarray(dG_row, f64)
    den = np.where(mask_b, p64, 0.0).sum(axis=1)
    safe = np.where(den > 0, den, 1.0)
    G = np.where(mask_b, p64 / safe[:, None], 0.0)
    inner = (G * dG).sum(axis=1)
    dp = np.where(mask_b, (dG - inner[:, None]) / safe[:, None], 0.0)
    diff = threshold_mask(p, thr).astype(f64) - np.asarray(mask_b, f64)
    dp = dp + w_batchwise * diff                     # d L_batchwise / d X_{j,i}
    dthr = -w_batchwise * diff.sum(axis=0)           # d L_batchwise / d T_i
    dc = p64 * (dp - (dp * p64).sum(axis=1, keepdims=True))
    x64 = np.asarray(x, f64)
    return SimpleNamespace(dWg=store(x64.T @ dc, prec), dX_gate=store(dc @ np.asarray(Wg, f64).T, prec),
                           dthr=store(dthr, prec), dlogits=dc)


def forward_balanced(x, Wg, thr, W1, b1, W2, b2, k, prec):
    """The layer with strictly balanced gating at training time: every expert gets m = k |X| / n examples."""
    T, n = x.shape[0], W1.shape[0]
    assert (k * T) % n == 0
    m = k * T // n
    c, p = softmax_gate(x, Wg, prec)
    mask = batchwise_mask(p, m)
    G, den = masked_gate(p, mask, prec)
    D = dispatch_balanced(x, mask)
    hid, ys = expert_ffn(D.xs, D.offsets, W1, b1, W2, b2, prec)
    y = combine_balanced(ys, G, D.tok_of_row, D.expert_of_row, T, prec)
    loss = batchwise_loss(p, mask, thr)
    return SimpleNamespace(y=y, logits=c, p=p, mask=mask, G=G, den=den, D=D, hid=hid, ys=ys, m=m,
                           loss=store(np.array([loss]), prec), mask_thr=threshold_mask(p, thr))


def backward_balanced(dY, x, Wg, thr, W1, b1, W2, b2, F, w_batchwise, prec):
    T = x.shape[0]
    dG_row, dys = combine_balanced_bwd(dY, F.ys, F.G, F.D.tok_of_row, F.D.expert_of_row, prec)
    E = expert_ffn_bwd(F.D.xs, F.hid, dys, F.D.offsets, W1, W2, prec)
    dX_exp = np.zeros((T, x.shape[1]), f64)
    np.add.at(dX_exp, F.D.tok_of_row.astype(np.int64), np.asarray(E.dxs, f64))
    GB = gate_balanced_bwd(x, Wg, F.p, F.mask, thr, dG_row, F.D.tok_of_row, F.D.expert_of_row, w_batchwise, prec)
    dX = store(dX_exp + np.asarray(GB.dX_gate, f64), prec, expert_side=True)
    return SimpleNamespace(dX=dX, dWg=GB.dWg, dthr=GB.dthr, dW1=E.dW1, db1=E.db1, dW2=E.dW2, db2=E.db2, dG_row=dG_row,
                           dys=dys, dxs=E.dxs, dX_gate=GB.dX_gate, dX_expert=store(dX_exp, prec))


# --------------------------------------------------------------------------------------
# optimiser step on the expert parameters (Appendix D, "Training": the memory optimisations)
# --------------------------------------------------------------------------------------
def adam_factored_step(W, g, row_avg, col_avg, lr, beta2, eps, step):
    """One step of Adam with beta1 = 0 (no first-moment estimate: the gradient itself is used) whose second-moment
    matrix is kept only through its row-wise and column-wise averages: those two vectors are the running averages
    (decay beta2) of the row / column means of g*g, and the matrix of estimators is taken to be their outer product
    divided by the mean of either one. Adam's bias correction 1 - beta2^step and its epsilon outside the square root
    are kept. W, g [rows, cols]; returns (W', row_avg', col_avg')."""
    g = np.asarray(g, f64)
    sq = g * g
    row_avg = beta2 * np.asarray(row_avg, f64) + (1.0 - beta2) * sq.mean(axis=1)
    col_avg = beta2 * np.asarray(col_avg, f64) + (1.0 - beta2) * sq.mean(axis=0)
    mean = row_avg.mean()
    v = np.outer(row_avg, col_avg) / mean if mean > 0 else np.zeros_like(sq)
    v_hat = v / (1.0 - beta2 ** step)
    W = np.asarray(W, f64) - lr * g / (np.sqrt(v_hat) + eps)
    return W, row_avg, col_avg


def adam_vector_step(b, g, v, lr, beta2, eps, step):
    """The same optimiser on a vector of parameters (the expert biases): a vector has no rows and columns to
    average over, so its second-moment estimate is kept in full (plain Adam with beta1 = 0)."""
    g = np.asarray(g, f64)
    v = beta2 * np.asarray(v, f64) + (1.0 - beta2) * g * g
    b = np.asarray(b, f64) - lr * g / (np.sqrt(v / (1.0 - beta2 ** step)) + eps)
    return b, v


def expert_adam_factored(W1, b1, W2, b2, dW1, db1, dW2, db2, state, lr, beta2, eps, step, prec):
    """adam_factored_step on every expert's two weight matrices and adam_vector_step on its biases.
    state = dict(r1 [n,d], c1 [n,h], r2 [n,h], c2 [n,d], vb1 [n,h], vb2 [n,d]) (float), updated in place on a copy.
    The parameters are rounded once to the layer's storage type, the state to float32."""
    n = W1.shape[0]
    out = {k_: np.array(v_, f64) for k_, v_ in state.items()}
    nW1, nb1, nW2, nb2 = (np.zeros(a.shape, f64) for a in (W1, b1, W2, b2))
    for e in range(n):
        nW1[e], out["r1"][e], out["c1"][e] = adam_factored_step(W1[e], dW1[e], out["r1"][e], out["c1"][e], lr, beta2, eps, step)
        nW2[e], out["r2"][e], out["c2"][e] = adam_factored_step(W2[e], dW2[e], out["r2"][e], out["c2"][e], lr, beta2, eps, step)
        nb1[e], out["vb1"][e] = adam_vector_step(b1[e], db1[e], out["vb1"][e], lr, beta2, eps, step)
        nb2[e], out["vb2"][e] = adam_vector_step(b2[e], db2[e], out["vb2"][e], lr, beta2, eps, step)
    out = {k_: store(v_, prec) for k_, v_ in out.items()}
    return (store(nW1, prec, True), store(nb1, prec, True), store(nW2, prec, True), store(nb2, prec, True), out)


# --------------------------------------------------------------------------------------
# the whole layer
# --------------------------------------------------------------------------------------
def forward(x, Wg, Wnoise, noise, W1, b1, W2, b2, k, w_importance, w_load, prec, hier=None, layer=None):
    """Forward of the layer with both balancing losses.

    Flat: Wg, Wnoise [d,n], noise [T,n]. Hierarchical (hier=(a, k1, b, k2)): Wg, Wnoise and
    noise are pairs (primary, secondary) and k is ignored. layer=(keep [T,d], drop_prob): the output is
    that of combine_layer (sigmoid, dropout, residual) instead of the plain mixture of Eq. 1."""
    n = W1.shape[0]
    if hier is None:
        G = gate(x, Wg, Wnoise, noise, k, prec)
        LS = losses(G.idx, G.gates, G.clean, G.raw, G.kth_val, w_importance, w_load, prec)
    else:
        a, k1, b, k2 = hier
        G = gate_h(x, Wg[0], Wnoise[0], noise[0], Wg[1], Wnoise[1], noise[1], k1, k2, prec)
        LS = losses_h(G, a, b, w_importance, w_load, prec)
    D = dispatch(x, G.idx, n)
    hid, ys = expert_ffn(D.xs, D.offsets, W1, b1, W2, b2, prec)
    if layer is None:
        y = combine(ys, G.gates, D.inv_perm, prec)
    else:
        y = combine_layer(ys, G.gates, D.inv_perm, x, layer[0], layer[1], prec)
    return SimpleNamespace(y=y, G=G, D=D, LS=LS, hid=hid, ys=ys)


def backward(dY, x, Wg, Wnoise, noise, W1, b1, W2, b2, F, w_importance, w_load, prec, hier=None, layer=None):
    """Backward of the layer; both balancing losses enter with upstream gradient 1
    (they are added to the model's loss, Section 4). With layer=(keep, drop_prob) dY is the gradient of
    combine_layer's output and also reaches dX directly through the residual connection."""
    T, k = F.G.idx.shape
    if layer is None:
        dgates, dys = combine_bwd(dY, F.ys, F.G.gates, F.D.inv_perm, prec)
    else:
        dgates, dys = combine_layer_bwd(dY, F.ys, F.G.gates, F.D.inv_perm, layer[0], layer[1], prec)
    E = expert_ffn_bwd(F.D.xs, F.hid, dys, F.D.offsets, W1, W2, prec)
    dX_exp = dispatch_bwd(E.dxs, F.D.inv_perm, T, k, prec)
    if hier is None:
        dg2, dload = losses_bwd(F.LS.importance, F.LS.load, F.G.idx, dgates, w_importance, w_load, prec)
        GB = gate_bwd(x, Wg, Wnoise, noise, F.G.clean, F.G.raw, F.G.idx, F.G.gates, F.G.kth_val,
                      F.G.kth_idx, dg2, dload, prec)
        dWg, dWn = GB.dWg, GB.dWnoise
    else:
        GB = gate_h_bwd(x, Wg[0], Wnoise[0], noise[0], Wg[1], Wnoise[1], noise[1], F.G, F.LS, dgates,
                        w_importance, w_load, prec)
        dWg, dWn = (GB.dWg_p, GB.dWg_s), (GB.dWn_p, GB.dWn_s)
    dX_sum = np.asarray(dX_exp, f64) + np.asarray(GB.dX_gate, f64)
    if layer is not None:
        dX_sum = dX_sum + np.asarray(dY, f64)  # residual connection
    dX = store(dX_sum, prec, expert_side=True)
    return SimpleNamespace(dX=dX, dWg=dWg, dWnoise=dWn, dW1=E.dW1, db1=E.db1, dW2=E.dW2, db2=E.db2,
                           dgates=dgates, dys=dys, dxs=E.dxs, dz=E.dz, dX_expert=dX_exp, dX_gate=GB.dX_gate)
