"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

The paper prints no worked numeric example of the layer, so each pin is a closed form, an
invariant, a special case that reduces to a textbook routine, a brute force on tiny
inputs, a Monte-Carlo run of a definition, or a finite difference.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O

f64 = np.float64


def rng(seed):
    return np.random.default_rng(seed)


def tiny(seed, T=6, d=5, n=7, h=4, bias=True):
    g = rng(seed)
    p = dict(x=g.standard_normal((T, d)), Wg=g.standard_normal((d, n)) * 0.7,
             Wnoise=g.standard_normal((d, n)) * 0.5, noise=g.standard_normal((T, n)),
             W1=g.standard_normal((n, d, h)) * 0.6, b1=g.standard_normal((n, h)) * (0.3 if bias else 0),
             W2=g.standard_normal((n, h, d)) * 0.6, b2=g.standard_normal((n, d)) * (0.3 if bias else 0))
    return p


# ---------------------------------------------------------------- single-precision chain
def round_to_f32(fr: Fraction) -> Fraction:
    """Round an exact rational to the nearest float32 (ties to even); normal range only."""
    if fr == 0:
        return Fraction(0)
    s = -1 if fr < 0 else 1
    m = abs(fr)
    e = m.numerator.bit_length() - m.denominator.bit_length()
    if Fraction(2) ** e > m:
        e -= 1
    assert Fraction(2) ** e <= m < Fraction(2) ** (e + 1) and -126 <= e <= 127
    quantum = Fraction(2) ** (e - 23)
    q = m / quantum
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return s * lo * quantum


def exact_chain(xrow, wcol, order):
    acc = Fraction(0)
    for q in order:
        acc = round_to_f32(Fraction(float(xrow[q])) * Fraction(float(wcol[q])) + acc)
    return float(acc)


def test_chain_is_ascending_fma_chain_exact_rational():
    g = rng(1)
    T, d, n = 3, 37, 5
    x = g.standard_normal((T, d)).astype(np.float32)
    W = (g.standard_normal((d, n)) / 6).astype(np.float32)
    got = O.project(x, W, "f32")
    n_order_sensitive = 0
    for t in range(T):
        for j in range(n):
            asc = exact_chain(x[t], W[:, j], range(d))
            assert float(got[t, j]) == asc  # bit-exact
            n_order_sensitive += asc != exact_chain(x[t], W[:, j], range(d - 1, -1, -1))
    assert n_order_sensitive > 0  # the inputs do tell the two orders apart


def test_chain_is_fused_not_two_roundings():
    # x*w = 1 - 2^-24 + 2^-48 exactly; product rounded alone gives 1, fused keeps the tail
    x = np.array([[1 + 2.0 ** -12, 1.0]], np.float32)
    W = np.array([[1 - 2.0 ** -12], [-1.0]], np.float32)
    got = float(O.project(x, W, "f32")[0, 0])
    assert got == exact_chain(x[0], W[:, 0], range(2)) and got != 0.0
    one = O.noisy_logits(np.array([-1.0], np.float32), x[0, :1], W[:1, 0], "f32")
    assert float(one[0]) == -(2.0 ** -24)


def test_chain_close_to_float64_matmul():
    g = rng(2)
    x = g.standard_normal((50, 64)).astype(np.float32)
    W = (g.standard_normal((64, 9)) / 8).astype(np.float32)
    assert np.allclose(O.project(x, W, "f32"), x.astype(f64) @ W.astype(f64), rtol=0, atol=2e-6)


def test_softplus_closed_values():
    r = np.array([0.0, 1.0, -1.0, 30.0, -30.0])
    want = [math.log(2.0), math.log1p(math.e), math.log1p(1 / math.e), 30 + math.log1p(math.exp(-30)),
            math.log1p(math.exp(-30))]
    assert np.allclose(O.softplus(r, "f64"), want, rtol=1e-15)
    assert O.softplus(np.array([1000.0]), "f64")[0] == 1000.0  # no overflow


# ---------------------------------------------------------------- top-k, gates (Eq. 3-5)
def test_keep_top_k_brute_force_with_ties():
    g = rng(3)
    for trial in range(40):
        T, n = 5, int(g.integers(1, 9))
        k = int(g.integers(1, n + 1))
        H = g.integers(-2, 3, size=(T, n)).astype(np.float32)  # many ties
        if trial % 4 == 0:
            H[H == 0] = -0.0  # -0 and +0 tie
        idx, kv, ki = O.keep_top_k(H, k)
        for t in range(T):
            ranked = sorted(range(n), key=lambda j: (-float(H[t, j]), j))  # lowest index wins ties
            assert list(idx[t]) == ranked[:k]
            assert ki[t, 0] == ranked[k - 1] and kv[t, 0] == H[t, ranked[k - 1]]
            if k < n:
                assert ki[t, 1] == ranked[k] and kv[t, 1] == H[t, ranked[k]]
            else:
                assert ki[t, 1] == -1 and kv[t, 1] == -np.inf


@pytest.mark.parametrize("prec", ["f64", "f32"])
def test_gate_invariants(prec):
    p = tiny(4, T=64, n=11)
    G = O.gate(p["x"], p["Wg"], p["Wnoise"], p["noise"], 3, prec)
    assert G.idx.shape == (64, 3)
    assert all(len(set(row)) == 3 for row in G.idx.tolist())  # exactly k distinct experts
    assert (G.gates > 0).all()
    assert np.allclose(G.gates.sum(axis=1), 1.0, atol=1e-6)
    # the dense gate vector has exactly k non-zeros and they are the k largest H
    Hk = np.take_along_axis(G.H, G.idx.astype(np.int64), 1)
    assert (np.diff(Hk, axis=1) <= 0).all()
    kept_min = np.where(O.selected_mask(G.idx, 11), G.H, np.inf).min(axis=1)
    others_max = np.where(O.selected_mask(G.idx, 11), -np.inf, G.H).max(axis=1)
    assert (others_max <= kept_min).all()


def test_gate_matches_literal_masked_softmax():
    """Eq. 3 written literally: set non-top-k entries to -inf, softmax over all n."""
    p = tiny(5, T=20, n=9)
    G = O.gate(p["x"], p["Wg"], p["Wnoise"], p["noise"], 4, "f64")
    c, r = p["x"] @ p["Wg"], p["x"] @ p["Wnoise"]
    H = c + p["noise"] * np.log1p(np.exp(r))
    for t in range(20):
        kept = np.argsort(-H[t])[:4]
        v = np.full(9, -np.inf)
        v[kept] = H[t, kept]
        dense = np.exp(v - v.max()) / np.exp(v - v.max()).sum()
        mine = np.zeros(9)
        mine[G.idx[t]] = G.gates[t]
        assert np.allclose(mine, dense, rtol=1e-12, atol=0)


def test_k_equals_one_gate_is_one_and_output_is_argmax_expert():
    p = tiny(6)
    F = O.forward(p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"], p["W2"], p["b2"], 1, 0.1, 0.1, "f64")
    assert (F.G.gates == 1.0).all()
    for t in range(p["x"].shape[0]):
        e = int(np.argmax(F.G.H[t]))
        want = np.maximum(p["x"][t] @ p["W1"][e] + p["b1"][e], 0) @ p["W2"][e] + p["b2"][e]
        assert np.allclose(F.y[t], want, rtol=1e-12)
    B = O.backward(rng(0).standard_normal(F.y.shape), p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"],
                   p["W2"], p["b2"], F, 0.0, 0.0, "f64")
    assert np.abs(B.dWg).max() == 0 and np.abs(B.dWnoise).max() == 0  # no gate gradient when k = 1


# ---------------------------------------------------------------- whole forward, Eq. 2 into Eq. 1
def test_k_equals_n_zero_noise_is_dense_softmax_mixture():
    p = tiny(7, T=9, n=6)
    n = 6
    zero = np.zeros_like(p["noise"])
    F = O.forward(p["x"], p["Wg"], p["Wnoise"], zero, p["W1"], p["b1"], p["W2"], p["b2"], n, 0.1, 0.1, "f64")
    for t in range(9):
        logits = [sum(p["x"][t, q] * p["Wg"][q, i] for q in range(5)) for i in range(n)]
        m = max(logits)
        den = sum(math.exp(v - m) for v in logits)
        y = np.zeros(5)
        for i in range(n):
            hid = np.maximum(p["x"][t] @ p["W1"][i] + p["b1"][i], 0)
            y += math.exp(logits[i] - m) / den * (hid @ p["W2"][i] + p["b2"][i])
        assert np.allclose(F.y[t], y, rtol=1e-12)
    assert np.allclose(F.LS.load, 9.0)  # k = n: every expert is certain to be selected


def test_single_expert_is_textbook_mlp():
    g = rng(8)
    xs = g.standard_normal((17, 6))
    W1, b1 = g.standard_normal((1, 6, 10)), g.standard_normal((1, 10))
    W2, b2 = g.standard_normal((1, 10, 6)), g.standard_normal((1, 6))
    hid, ys = O.expert_ffn(xs, np.array([0, 17]), W1, b1, W2, b2, "f64")
    tx = torch.from_numpy(xs)
    th = torch.relu(torch.nn.functional.linear(tx, torch.from_numpy(W1[0]).T.contiguous(), torch.from_numpy(b1[0])))
    ty = torch.nn.functional.linear(th, torch.from_numpy(W2[0]).T.contiguous(), torch.from_numpy(b2[0]))
    assert np.allclose(hid, th.numpy(), rtol=1e-13) and np.allclose(ys, ty.numpy(), rtol=1e-13)


def test_bf16_rounding_points():
    v = np.array([1.0, 1.00390625, 1.001953125, 1.005859375, -3.1415927, 65504.0], np.float32)
    want = torch.from_numpy(v).bfloat16().float().numpy()  # library round-to-nearest-even
    assert (O.round_bf16(v) == want).all()
    assert O.round_bf16(np.array([1.001953125], np.float32))[0] == 1.0  # tie -> even
    assert O.round_bf16(np.array([1.005859375], np.float32))[0] == np.float32(1.0078125)  # tie -> even (up)
    g = rng(9)
    xs = O.round_bf16(g.standard_normal((8, 16)).astype(np.float32))
    W1 = O.round_bf16(g.standard_normal((1, 16, 8)).astype(np.float32) / 4)
    W2 = O.round_bf16(g.standard_normal((1, 8, 16)).astype(np.float32) / 3)
    hid, ys = O.expert_ffn(xs, np.array([0, 8]), W1, np.zeros((1, 8)), W2, np.zeros((1, 16)), "bf16")
    assert (O.round_bf16(hid) == hid).all() and (O.round_bf16(ys) == ys).all()
    exact = np.maximum(xs.astype(f64) @ W1[0].astype(f64), 0)
    assert np.abs(hid - exact).max() <= np.abs(exact).max() * 2.0 ** -8


def test_bf16_rounding_points_of_the_backward():
    """In "bf16" mode every expert-side tensor the backward materialises (dys, dz, dxs, dW1, db1, dW2, db2, dX) is
    rounded once to bfloat16: each must be representable (checked with the library's rounding, not the oracle's) and
    within one bf16 unit of the float64-mode value computed from the same rounded inputs; the gating-side tensors
    (dgates, dWg, dWnoise) stay float32. A forgotten rounding would leave non-representable values behind."""
    def representable(a):
        a = np.asarray(a, np.float32)
        return (torch.from_numpy(np.ascontiguousarray(a)).bfloat16().float().numpy() == a).all()

    g = rng(31)
    T, d, n, k, h = 48, 16, 4, 2, 24
    x = O.round_bf16(g.standard_normal((T, d)).astype(np.float32))
    dY = O.round_bf16(g.standard_normal((T, d)).astype(np.float32))
    Wg, Wn = (g.standard_normal((d, n)).astype(np.float32) / 4 for _ in range(2))
    noise = g.standard_normal((T, n)).astype(np.float32)
    W1 = O.round_bf16(g.standard_normal((n, d, h)).astype(np.float32) / 4)
    W2 = O.round_bf16(g.standard_normal((n, h, d)).astype(np.float32) / 5)
    b1 = O.round_bf16(g.standard_normal((n, h)).astype(np.float32) / 3)
    b2 = O.round_bf16(g.standard_normal((n, d)).astype(np.float32) / 3)
    F = O.forward(x, Wg, Wn, noise, W1, b1, W2, b2, k, 0.1, 0.1, "bf16")
    Bk = O.backward(dY, x, Wg, Wn, noise, W1, b1, W2, b2, F, 0.1, 0.1, "bf16")
    for name in ("dys", "dz", "dxs", "dW1", "db1", "dW2", "db2", "dX"):
        assert representable(getattr(Bk, name)), name
    for name in ("dgates", "dWg", "dWnoise"):   # fp32 gating path: not squeezed into bf16
        assert not representable(getattr(Bk, name)), name
    # one rounding each: against float64 evaluations of the single steps on the same (rounded) inputs
    ulp = 2.0 ** -8  # half-ulp relative error of round-to-nearest is 2^-9; one unit leaves room for the rms floor below

    def one_rounding(got, exact, name):
        got, exact = np.asarray(got, f64), np.asarray(exact, f64)
        assert np.abs(got - exact).max() <= ulp * np.abs(exact).max(), name
        assert (np.abs(got - exact) <= ulp * np.abs(exact) + 1e-30).all(), name

    rows = F.D.inv_perm.reshape(T, k)
    for s_ in range(k):
        one_rounding(Bk.dys[rows[:, s_]], np.asarray(F.G.gates, f64)[:, s_, None] * dY.astype(f64), "dys")
    E64 = O.expert_ffn_bwd(F.D.xs, F.hid, Bk.dys, F.D.offsets, W1, W2, "f64")
    one_rounding(Bk.dz, E64.dz, "dz")
    one_rounding(Bk.dW2, E64.dW2, "dW2")
    one_rounding(Bk.db2, E64.db2, "db2")
    for e in range(n):   # the steps behind dz take the ROUNDED dz as their input
        o0, o1 = int(F.D.offsets[e]), int(F.D.offsets[e + 1])
        dz = np.asarray(Bk.dz[o0:o1], f64)
        one_rounding(Bk.db1[e], dz.sum(axis=0), "db1")
        one_rounding(Bk.dW1[e], np.asarray(F.D.xs[o0:o1], f64).T @ dz, "dW1")
        one_rounding(Bk.dxs[o0:o1], dz @ W1[e].astype(f64).T, "dxs")
    one_rounding(Bk.dX, np.asarray(Bk.dX_expert, f64) + np.asarray(Bk.dX_gate, f64), "dX")


# ---------------------------------------------------------------- dispatch / combine
def test_dispatch_is_stable_counting_sort_and_round_trips():
    g = rng(10)
    T, k, n, d = 40, 3, 6, 4
    idx = np.stack([g.permutation(n)[:k] for _ in range(T)]).astype(np.int32)
    x = g.standard_normal((T, d))
    D = O.dispatch(x, idx, n + 1)  # expert n receives nothing
    assert D.counts.sum() == T * k and D.counts[n] == 0 and D.offsets[-1] == T * k
    assert (np.diff(D.offsets) == D.counts).all()
    assert (D.perm[D.inv_perm] == np.arange(T * k)).all()
    flat = idx.reshape(-1)
    for e in range(n + 1):
        seg = D.perm[D.offsets[e]:D.offsets[e + 1]]
        assert (flat[seg] == e).all() and (np.diff(seg) > 0).all()  # stable: slots ascending inside a segment
    assert (D.xs == x[D.perm // k]).all()
    gates = g.random((T, k))
    gates /= gates.sum(axis=1, keepdims=True)
    assert np.allclose(O.combine(D.xs, gates, D.inv_perm, "f64"), x, rtol=1e-13)  # sum of gates = 1


# ---------------------------------------------------------------- CV^2, Importance (Eq. 6, 7)
def test_cv_squared_closed_forms():
    assert O.cv_squared(np.full(9, 3.5)) == 0.0
    for n in (2, 5, 16):
        one_hot = np.zeros(n)
        one_hot[1] = 4.2
        assert math.isclose(O.cv_squared(one_hot), n - 1, rel_tol=1e-13)  # sample variance would give n
    assert math.isclose(O.cv_squared([1.0, 3.0]), 0.25, rel_tol=1e-15)
    v = rng(11).random(7) + 0.5
    num = np.array([(O.cv_squared(v + 1e-6 * np.eye(7)[i]) - O.cv_squared(v - 1e-6 * np.eye(7)[i])) / 2e-6
                    for i in range(7)])
    assert np.allclose(O.cv_squared_grad(v), num, rtol=1e-6, atol=1e-9)


def test_importance_sums_to_batch_size():
    p = tiny(12, T=50, n=8)
    G = O.gate(p["x"], p["Wg"], p["Wnoise"], p["noise"], 2, "f64")
    LS = O.losses(G.idx, G.gates, G.clean, G.raw, G.kth_val, 0.1, 0.1, "f64")
    assert math.isclose(LS.importance.sum(), 50.0, rel_tol=1e-13)
    dense = np.zeros((50, 8))
    for t in range(50):
        dense[t, G.idx[t]] = G.gates[t]
    assert np.allclose(LS.importance, dense.sum(axis=0), rtol=1e-13)
    assert math.isclose(LS.losses[0], 0.1 * dense.sum(0).var() / dense.sum(0).mean() ** 2, rel_tol=1e-12)


# ---------------------------------------------------------------- Load estimator (Eq. 8-10)
def test_load_probability_against_delete_and_sort():
    p = tiny(13, T=30, n=9)
    for k in (1, 3, 8, 9):
        G = O.gate(p["x"], p["Wg"], p["Wnoise"], p["noise"], k, "f64")
        P, _, _ = O.load_probability(G.clean, G.sigma, G.idx, G.kth_val)
        for t in range(30):
            for i in range(9):
                rest = sorted(np.delete(G.H[t], i), reverse=True)
                thr = rest[k - 1] if k - 1 < len(rest) else -np.inf  # kth_excluding(H, k, i)
                z = (G.clean[t, i] - thr) / G.sigma[t, i]
                want = 0.5 * math.erfc(-z / math.sqrt(2.0)) if np.isfinite(z) else 1.0
                assert math.isclose(P[t, i], want, rel_tol=1e-12, abs_tol=1e-300)


def test_load_probability_is_the_resampling_probability_monte_carlo():
    """Definition above Eq. 8: redraw the noise of entry i only; P = Pr(G(x)_i != 0)."""
    p = tiny(14, T=2, n=6)
    k = 2
    G = O.gate(p["x"], p["Wg"], p["Wnoise"], p["noise"], k, "f64")
    P, _, _ = O.load_probability(G.clean, G.sigma, G.idx, G.kth_val)
    g = rng(15)
    N = 200_000
    for t in range(2):
        for i in range(6):
            Hi = G.clean[t, i] + g.standard_normal(N) * G.sigma[t, i]
            others = np.delete(G.H[t], i)
            kth_other = np.sort(others)[::-1][k - 1]
            freq = (Hi > kth_other).mean()
            assert abs(freq - P[t, i]) < 4.5 * math.sqrt(max(P[t, i] * (1 - P[t, i]), 1e-4) / N)


def test_load_zero_initialisation_closed_form():
    """W_g = W_noise = 0 (Appendix A): no signal, noise std ln 2, routing = top-k of the noise."""
    g = rng(16)
    T, d, n, k = 25, 4, 8, 3
    x, eps = g.standard_normal((T, d)), g.standard_normal((T, n))
    G = O.gate(x, np.zeros((d, n)), np.zeros((d, n)), eps, k, "f64")
    assert (G.clean == 0).all() and np.allclose(G.sigma, math.log(2.0), rtol=1e-15)
    assert (G.idx == np.argsort(-eps, axis=1)[:, :k]).all()
    P, _, _ = O.load_probability(G.clean, G.sigma, G.idx, G.kth_val)
    srt = -np.sort(-eps, axis=1)
    for t in range(T):
        for i in range(n):
            thr_eps = srt[t, k] if i in G.idx[t] else srt[t, k - 1]
            assert math.isclose(P[t, i], 0.5 * math.erfc(thr_eps / math.sqrt(2.0)), rel_tol=1e-12)


def test_load_probability_half_at_threshold():
    clean = np.array([[0.3, 0.9, -0.2]])
    sigma = np.array([[0.5, 2.0, 1.0]])
    idx = np.array([[1]], np.int32)
    kth_val = np.array([[0.3, 0.9]])  # unselected compare against 0.3 = clean[0]; selected against 0.9 = clean[1]
    P, _, _ = O.load_probability(clean, sigma, idx, kth_val)
    assert P[0, 0] == 0.5 and P[0, 1] == 0.5 and P[0, 2] < 0.5


# ---------------------------------------------------------------- hierarchical (Eq. 12-14)
def tiny_h(seed, T=8, d=5, a=3, b=4, h=3):
    g = rng(seed)
    n = a * b
    return dict(x=g.standard_normal((T, d)),
                Wg=(g.standard_normal((d, a)) * 0.7, g.standard_normal((a, d, b)) * 0.7),
                Wnoise=(g.standard_normal((d, a)) * 0.5, g.standard_normal((a, d, b)) * 0.5),
                W1=g.standard_normal((n, d, h)) * 0.6, b1=g.standard_normal((n, h)) * 0.3,
                W2=g.standard_normal((n, h, d)) * 0.6, b2=g.standard_normal((n, d)) * 0.3), g


def test_hierarchical_invariants_and_literal_double_sum():
    p, g = tiny_h(17)
    T, a, b, k1, k2 = 8, 3, 4, 2, 2
    noise = (g.standard_normal((T, a)), g.standard_normal((T, k1, b)))
    F = O.forward(p["x"], p["Wg"], p["Wnoise"], noise, p["W1"], p["b1"], p["W2"], p["b2"], None, 0.1, 0.1, "f64",
                  hier=(a, k1, b, k2))
    assert np.allclose(F.G.gates.sum(axis=1), 1.0, rtol=1e-13)
    assert math.isclose(F.LS.importance.sum(), T, rel_tol=1e-13)
    # Eq. 12 literally: dense primary gate times dense secondary gate of each kept group
    for t in range(T):
        y = np.zeros(5)
        Gp = np.zeros(a)
        Gp[F.G.primary.idx[t]] = F.G.primary.gates[t]
        for s1, i in enumerate(F.G.primary.idx[t]):
            Gi = np.zeros(b)
            Gi[F.G.secondary.idx[t, s1]] = F.G.secondary.gates[t, s1]
            for j in range(b):
                e = i * b + j
                E = np.maximum(p["x"][t] @ p["W1"][e] + p["b1"][e], 0) @ p["W2"][e] + p["b2"][e]
                y += Gp[i] * Gi[j] * E
        assert np.allclose(F.y[t], y, rtol=1e-12)
    # Eq. 14 literally
    LS = F.LS
    for i in range(a):
        Xi = [t for t in range(T) if i in F.G.primary.idx[t]]
        assert LS.cnt[i] == len(Xi)
        for j in range(b):
            want = 0.0 if not Xi else LS.load_p[i] * LS.load_s[i, j] / len(Xi)
            assert math.isclose(LS.load[i * b + j], want, rel_tol=1e-12, abs_tol=1e-15)


def test_hierarchical_with_one_group_is_the_flat_layer():
    g = rng(18)
    T, d, b, h, k = 10, 5, 7, 3, 3
    x = g.standard_normal((T, d))
    Wg_s, Wn_s = g.standard_normal((1, d, b)), g.standard_normal((1, d, b)) * 0.5
    eps = g.standard_normal((T, b))
    W1, b1 = g.standard_normal((b, d, h)), g.standard_normal((b, h))
    W2, b2 = g.standard_normal((b, h, d)), g.standard_normal((b, d))
    flat = O.forward(x, Wg_s[0], Wn_s[0], eps, W1, b1, W2, b2, k, 0.1, 0.2, "f64")
    hier = O.forward(x, (g.standard_normal((d, 1)), Wg_s), (g.standard_normal((d, 1)), Wn_s),
                     (g.standard_normal((T, 1)), eps[:, None, :]), W1, b1, W2, b2, None, 0.1, 0.2, "f64",
                     hier=(1, 1, b, k))
    assert (flat.G.idx == hier.G.idx).all()
    assert np.allclose(flat.y, hier.y, rtol=1e-13)
    assert np.allclose(flat.LS.importance, hier.LS.importance, rtol=1e-13)
    assert np.allclose(flat.LS.load, hier.LS.load, rtol=1e-13)  # Load_primary = |X| when k1 = a
    assert np.allclose(flat.LS.losses, hier.LS.losses, rtol=1e-12)


# ---------------------------------------------------------------- backward against finite differences
def scalar_loss(p, noise, dY, k, wi, wl, hier):
    F = O.forward(p["x"], p["Wg"], p["Wnoise"], noise, p["W1"], p["b1"], p["W2"], p["b2"], k, wi, wl, "f64", hier=hier)
    return float((F.y * dY).sum() + F.LS.losses.sum()), F


def fd_check(p, noise, dY, k, wi, wl, hier, names, seed, per_tensor=12, step=1e-6):
    base, F = scalar_loss(p, noise, dY, k, wi, wl, hier)
    B = O.backward(dY, p["x"], p["Wg"], p["Wnoise"], noise, p["W1"], p["b1"], p["W2"], p["b2"], F, wi, wl, "f64",
                   hier=hier)
    g = rng(seed)
    worst = 0.0
    for name, grad, arr in names(p, B):
        flat = arr.reshape(-1)
        scale = max(np.abs(grad).max(), 1e-3)
        for pos in g.choice(flat.size, size=min(per_tensor, flat.size), replace=False):
            old = flat[pos]
            flat[pos] = old + step
            up, Fu = scalar_loss(p, noise, dY, k, wi, wl, hier)
            flat[pos] = old - step
            dn, Fd = scalar_loss(p, noise, dY, k, wi, wl, hier)
            flat[pos] = old
            assert (Fu.G.idx == F.G.idx).all() and (Fd.G.idx == F.G.idx).all()  # no routing switch in the stencil
            num = (up - dn) / (2 * step)
            err = abs(num - grad.reshape(-1)[pos]) / scale
            worst = max(worst, err)
            assert err < 2e-6, (name, pos, num, grad.reshape(-1)[pos])
    return B, worst


def flat_names(p, B):
    return [("x", B.dX, p["x"]), ("Wg", B.dWg, p["Wg"]), ("Wnoise", B.dWnoise, p["Wnoise"]),
            ("W1", B.dW1, p["W1"]), ("b1", B.db1, p["b1"]), ("W2", B.dW2, p["W2"]), ("b2", B.db2, p["b2"])]


@pytest.mark.parametrize("k,wi,wl", [(3, 0.1, 0.1), (2, 0.0, 1.0), (2, 1.0, 0.0), (7, 0.3, 0.3), (1, 0.5, 0.5)])
def test_backward_flat_matches_finite_differences(k, wi, wl):
    p = tiny(20 + k)
    dY = rng(21).standard_normal(p["x"].shape)
    B, _ = fd_check(p, p["noise"], dY, k, wi, wl, None, flat_names, seed=22)
    # softmax path alone sends no net gradient into a token's kept logits
    if wl == 0.0:
        F = scalar_loss(p, p["noise"], dY, k, wi, wl, None)[1]
        dg2, dload = O.losses_bwd(F.LS.importance, F.LS.load, F.G.idx, B.dgates, wi, wl, "f64")
        dc, dr = O.gate_logit_grads(p["noise"], F.G.clean, F.G.raw, F.G.idx, F.G.gates, F.G.kth_val, F.G.kth_idx,
                                    dg2, dload, "f64")
        assert np.abs(dc.sum(axis=1)).max() < 1e-12


def test_backward_hierarchical_matches_finite_differences():
    p, g = tiny_h(23)
    T, a, b, k1, k2 = 8, 3, 4, 2, 2
    noise = (g.standard_normal((T, a)), g.standard_normal((T, k1, b)))
    dY = g.standard_normal(p["x"].shape)

    def names(p, B):
        return [("x", B.dX, p["x"]), ("Wg_p", B.dWg[0], p["Wg"][0]), ("Wg_s", B.dWg[1], p["Wg"][1]),
                ("Wn_p", B.dWnoise[0], p["Wnoise"][0]), ("Wn_s", B.dWnoise[1], p["Wnoise"][1]),
                ("W1", B.dW1, p["W1"]), ("b1", B.db1, p["b1"]), ("W2", B.dW2, p["W2"]), ("b2", B.db2, p["b2"])]

    fd_check(p, noise, dY, None, 0.4, 0.6, (a, k1, b, k2), names, seed=24)


def test_expert_without_rows_has_zero_gradient():
    p = tiny(25, T=4, n=9)
    dY = rng(26).standard_normal(p["x"].shape)
    _, F = scalar_loss(p, p["noise"], dY, 2, 0.1, 0.1, None)
    B = O.backward(dY, p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"], p["W2"], p["b2"], F, 0.1, 0.1, "f64")
    empty = np.nonzero(F.D.counts == 0)[0]
    assert empty.size > 0
    assert np.abs(B.dW1[empty]).max() == 0 and np.abs(B.dW2[empty]).max() == 0
    assert np.abs(B.db1[empty]).max() == 0 and np.abs(B.db2[empty]).max() == 0


def test_rounded_modes_stay_close_to_float64():
    p = tiny(27, T=32, n=8, d=16, h=12)
    p32 = {k: v.astype(np.float32) for k, v in p.items()}
    dY = rng(28).standard_normal(p["x"].shape).astype(np.float32)
    out = {}
    for prec, q in (("f64", {k: v.astype(f64) for k, v in p32.items()}), ("f32", p32)):
        F = O.forward(q["x"], q["Wg"], q["Wnoise"], q["noise"], q["W1"], q["b1"], q["W2"], q["b2"], 2, 0.1, 0.1, prec)
        B = O.backward(dY.astype(q["x"].dtype), q["x"], q["Wg"], q["Wnoise"], q["noise"], q["W1"], q["b1"], q["W2"],
                       q["b2"], F, 0.1, 0.1, prec)
        out[prec] = (F, B)
    assert (out["f64"][0].G.idx == out["f32"][0].G.idx).all()
    for name in ("dX", "dWg", "dWnoise", "dW1", "dW2"):
        ref = getattr(out["f64"][1], name)
        assert np.abs(getattr(out["f32"][1], name) - ref).max() <= 1e-5 * (np.abs(ref).max() + 1)


# ---------------------------------------------------------------- layer epilogue: sigmoid, dropout, residual (Appendix C)
def test_layer_epilogue_closed_forms():
    g = rng(40)
    T, k, d = 9, 2, 16
    ys = g.standard_normal((T * k, d))
    gates = g.random((T, k)); gates /= gates.sum(axis=1, keepdims=True)
    inv = g.permutation(T * k).astype(np.int32)
    x = g.standard_normal((T, d))
    y = np.asarray(O.combine(ys, gates, inv, "f64"))
    ones = np.ones((T, d), bool)
    # no dropout: out - x is the logistic function of the mixture; textbook values of the logistic function
    out = O.combine_layer(ys, gates, inv, x, ones, 0.0, "f64")
    assert np.allclose(out - x, 1.0 / (1.0 + np.exp(-y)), rtol=1e-14)
    assert np.allclose(out - x + (O.combine_layer(-ys, gates, inv, x, ones, 0.0, "f64") - x), 1.0, rtol=1e-13)  # s(y)+s(-y)=1
    zero = O.combine_layer(np.zeros_like(ys), gates, inv, x, ones, 0.0, "f64")
    assert np.allclose(zero - x, 0.5, rtol=1e-15)
    # everything dropped: the residual alone; everything kept with DropProb 1/2: twice the sigmoid
    assert (O.combine_layer(ys, gates, inv, x, ~ones, 0.3, "f64") == x).all()
    assert np.allclose(O.combine_layer(ys, gates, inv, x, ones, 0.5, "f64") - x, 2.0 * (out - x), rtol=1e-14)
    # dropout is unbiased: averaging over a mask and its complement, each scaled for DropProb 1/2, gives back the sigmoid
    keep = g.random((T, d)) < 0.5
    a = O.combine_layer(ys, gates, inv, x, keep, 0.5, "f64") - x
    b = O.combine_layer(ys, gates, inv, x, ~keep, 0.5, "f64") - x
    assert np.allclose(0.5 * (a + b), out - x, rtol=1e-13)
    # the packed mask format
    bits = np.packbits(keep, axis=1, bitorder="little")
    assert (O.unpack_keep(bits, d) == keep).all()
    assert O.unpack_keep(np.array([[0b00000101]], np.uint8), 8).tolist() == [[True, False, True] + [False] * 5]


def test_layer_epilogue_backward_matches_finite_differences():
    p = tiny(41)
    T, d = p["x"].shape
    g = rng(42)
    keep = g.random((T, d)) < 0.7
    layer = (keep, 0.3)
    dOut = g.standard_normal((T, d))
    k, wi, wl = 3, 0.1, 0.2

    def loss():
        F = O.forward(p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"], p["W2"], p["b2"], k, wi, wl, "f64",
                      layer=layer)
        return float((F.y * dOut).sum() + F.LS.losses.sum()), F

    base, F = loss()
    Bk = O.backward(dOut, p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"], p["W2"], p["b2"], F, wi, wl, "f64",
                    layer=layer)
    step = 1e-6
    for name, grad, arr in flat_names(p, Bk):
        flat = arr.reshape(-1)
        scale = max(np.abs(grad).max(), 1e-3)
        for pos in g.choice(flat.size, size=min(10, flat.size), replace=False):
            old = flat[pos]
            flat[pos] = old + step
            up, Fu = loss()
            flat[pos] = old - step
            dn, Fd = loss()
            flat[pos] = old
            assert (Fu.G.idx == F.G.idx).all() and (Fd.G.idx == F.G.idx).all()
            assert abs((up - dn) / (2 * step) - grad.reshape(-1)[pos]) / scale < 2e-6, (name, pos)
    # dropped activations pass no gradient into the experts: with everything dropped only the residual and the
    # balancing losses are left
    none = (np.zeros((T, d), bool), 0.3)
    F0 = O.forward(p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"], p["W2"], p["b2"], k, wi, wl, "f64", layer=none)
    B0 = O.backward(dOut, p["x"], p["Wg"], p["Wnoise"], p["noise"], p["W1"], p["b1"], p["W2"], p["b2"], F0, wi, wl, "f64",
                    layer=none)
    assert np.abs(B0.dW1).max() == 0 and np.abs(B0.dW2).max() == 0 and np.abs(B0.dys).max() == 0


# ---------------------------------------------------------------- factored second-moment Adam, beta1 = 0 (Appendix D)
def full_adam_beta1_zero(W, g, v, lr, beta2, eps, step):
    """Textbook Adam (Kingma & Ba) with beta1 = 0 and the complete second-moment matrix."""
    v = beta2 * v + (1 - beta2) * g * g
    return W - lr * g / (np.sqrt(v / (1 - beta2 ** step)) + eps), v


def test_factored_adam_is_full_adam_when_the_squared_gradient_has_rank_one():
    g_ = rng(60)
    rows, cols = 7, 5
    a, b = g_.standard_normal(rows), g_.standard_normal(cols)
    G = np.outer(a, b)            # G*G = (a*a)(b*b)^T: its row and column averages determine it completely
    W = g_.standard_normal((rows, cols))
    r, c, v = np.zeros(rows), np.zeros(cols), np.zeros((rows, cols))
    for step in (1, 2, 3):
        Wf, r, c = O.adam_factored_step(W, G, r, c, 1e-2, 0.9, 1e-8, step)
        Wa, v = full_adam_beta1_zero(W, G, v, 1e-2, 0.9, 1e-8, step)
        assert np.allclose(Wf, Wa, rtol=1e-12, atol=1e-14)
        assert np.allclose(np.outer(r, c) / r.mean(), v, rtol=1e-12)
        assert math.isclose(r.mean(), c.mean(), rel_tol=1e-13)   # "the mean of either one"
        W = Wf
        G = G * 1.5               # still rank one, and proportional: the running averages stay rank-one consistent


def test_factored_adam_textbook_limits():
    g_ = rng(61)
    W = g_.standard_normal((4, 6))
    # constant-magnitude gradient: v = g^2 everywhere, every entry moves by lr * sign(g) (up to eps), at every step
    G = 0.3 * np.sign(g_.standard_normal((4, 6)))
    r, c = np.zeros(4), np.zeros(6)
    Wn = W
    for step in (1, 2, 3, 4):
        Wn, r, c = O.adam_factored_step(Wn, G, r, c, 1e-3, 0.999, 0.0, step)
        assert np.allclose(W - Wn, step * 1e-3 * np.sign(G), rtol=1e-10)
    # bias correction: after t identical steps the corrected estimate is exactly the squared gradient's averages
    assert np.allclose(r / (1 - 0.999 ** 4), 0.09, rtol=1e-12) and np.allclose(c / (1 - 0.999 ** 4), 0.09, rtol=1e-12)
    # a zero gradient leaves the parameters alone (0 / (0 + eps))
    W0, _, _ = O.adam_factored_step(W, np.zeros_like(W), np.zeros(4), np.zeros(6), 1e-3, 0.999, 1e-8, 1)
    assert (W0 == W).all()
    # the approximation keeps the row and column averages of the true second-moment matrix exactly
    G = g_.standard_normal((4, 6))
    _, r, c = O.adam_factored_step(W, G, np.zeros(4), np.zeros(6), 1e-3, 0.0, 1e-8, 1)   # beta2 = 0: averages of G*G
    V = np.outer(r, c) / r.mean()
    assert np.allclose(V.mean(axis=1), (G * G).mean(axis=1), rtol=1e-12)
    assert np.allclose(V.mean(axis=0), (G * G).mean(axis=0), rtol=1e-12)
    # vectors: plain Adam with beta1 = 0
    b, gb = g_.standard_normal(5), g_.standard_normal(5)
    bn, vb = O.adam_vector_step(b, gb, np.zeros(5), 1e-2, 0.9, 1e-8, 1)
    ba, va = full_adam_beta1_zero(b, gb, np.zeros(5), 1e-2, 0.9, 1e-8, 1)
    assert np.allclose(bn, ba, rtol=1e-14) and np.allclose(vb, va, rtol=1e-14)


# ---------------------------------------------------------------- strictly balanced gating (Appendix F, Eq. 15-20)
def balanced_tiny(seed, T=12, d=5, n=6, h=4):
    g = rng(seed)
    return dict(x=g.standard_normal((T, d)), Wg=g.standard_normal((d, n)) * 0.8, W1=g.standard_normal((n, d, h)) * 0.6,
                b1=g.standard_normal((n, h)) * 0.3, W2=g.standard_normal((n, h, d)) * 0.6, b2=g.standard_normal((n, d)) * 0.3)


def test_balanced_gating_invariants_and_brute_force():
    p_ = balanced_tiny(70)
    k = 2
    T, n = p_["x"].shape[0], p_["Wg"].shape[1]
    m = k * T // n
    thr = np.full(n, 0.2)
    F = O.forward_balanced(p_["x"], p_["Wg"], thr, p_["W1"], p_["b1"], p_["W2"], p_["b2"], k, "f64")
    # Eq. 15 is the textbook softmax
    z = p_["x"] @ p_["Wg"]
    assert np.allclose(F.p, np.exp(z) / np.exp(z).sum(axis=1, keepdims=True), rtol=1e-13)
    # every expert receives exactly m examples, on average k per example
    assert (F.mask.sum(axis=0) == m).all() and F.mask.sum() == k * T
    assert (np.diff(F.D.offsets) == m).all()
    # the mask by brute force: per column, pair (value, -token) sorted descending, first m
    for i in range(n):
        best = sorted(range(T), key=lambda t: (-F.p[t, i], t))[:m]
        assert sorted(best) == list(np.nonzero(F.mask[:, i])[0])
    # kept gates renormalise to one; an example nobody keeps has a zero gate vector and a zero output
    kept = F.mask.any(axis=1)
    assert np.allclose(F.G.sum(axis=1)[kept], 1.0, rtol=1e-13) and (F.G[~F.mask] == 0).all()
    assert (F.G.sum(axis=1)[~kept] == 0).all() and (np.asarray(F.y)[~kept] == 0).all()
    # the output is the literal double sum of Eq. 1 with these gates
    want = np.zeros_like(p_["x"])
    for t in range(T):
        for i in range(n):
            if F.mask[t, i]:
                hidden = np.maximum(p_["x"][t] @ p_["W1"][i] + p_["b1"][i], 0)
                want[t] += F.G[t, i] * (hidden @ p_["W2"][i] + p_["b2"][i])
    assert np.allclose(F.y, want, rtol=1e-12, atol=1e-14)


def test_balanced_ties_go_to_the_lower_token():
    p = np.array([[0.5, 0.1], [0.5, 0.3], [0.5, 0.3], [0.2, 0.3]])
    mask = O.batchwise_mask(p, 2)
    assert mask[:, 0].tolist() == [True, True, False, False]      # three-way tie at 0.5: tokens 0 and 1
    assert mask[:, 1].tolist() == [False, True, True, False]      # three-way tie at 0.3: tokens 1 and 2


def test_threshold_mask_and_batchwise_loss():
    p_ = balanced_tiny(71)
    k = 2
    T, n = p_["x"].shape[0], p_["Wg"].shape[1]
    m = k * T // n
    _, p = O.softmax_gate(p_["x"], p_["Wg"], "f64")
    mask = O.batchwise_mask(p, m)
    # thresholds between each column's m-th and (m+1)-th largest value reproduce the batchwise mask: the loss is zero
    srt = -np.sort(-p, axis=0)
    thr = 0.5 * (srt[m - 1] + srt[m])
    assert (O.threshold_mask(p, thr) == mask).all()
    assert O.batchwise_loss(p, mask, thr) == 0.0
    # any other thresholds give a positive loss: every disagreeing entry contributes |X - T|
    for shift in (-0.05, 0.07):
        thr2 = thr + shift
        dis = O.threshold_mask(p, thr2) != mask
        assert dis.any()
        assert math.isclose(O.batchwise_loss(p, mask, thr2), np.abs(p - thr2[None, :])[dis].sum(), rel_tol=1e-12)
    # Eq. 19 is a strict inequality
    assert not O.threshold_mask(np.array([[0.25]]), np.array([0.25]))[0, 0]


def test_balanced_backward_matches_finite_differences():
    p_ = balanced_tiny(72)
    k, wb = 2, 0.7
    T, n = p_["x"].shape[0], p_["Wg"].shape[1]
    g = rng(73)
    dY = g.standard_normal(p_["x"].shape)
    thr = np.full(n, 1.0 / n) + 0.02 * g.standard_normal(n)
    p_["thr"] = thr

    def loss():
        F = O.forward_balanced(p_["x"], p_["Wg"], p_["thr"], p_["W1"], p_["b1"], p_["W2"], p_["b2"], k, "f64")
        return float((F.y * dY).sum() + wb * F.loss[0]), F

    base, F = loss()
    Bk = O.backward_balanced(dY, p_["x"], p_["Wg"], p_["thr"], p_["W1"], p_["b1"], p_["W2"], p_["b2"], F, wb, "f64")
    step = 1e-6
    for name, grad in (("x", Bk.dX), ("Wg", Bk.dWg), ("thr", Bk.dthr), ("W1", Bk.dW1), ("b1", Bk.db1), ("W2", Bk.dW2),
                       ("b2", Bk.db2)):
        flat = p_[name].reshape(-1)
        scale = max(np.abs(grad).max(), 1e-3)
        for pos in g.choice(flat.size, size=min(10, flat.size), replace=False):
            old = flat[pos]
            flat[pos] = old + step
            up, Fu = loss()
            flat[pos] = old - step
            dn, Fd = loss()
            flat[pos] = old
            same = (Fu.mask == F.mask).all() and (Fd.mask == F.mask).all() and (Fu.mask_thr == F.mask_thr).all() and \
                (Fd.mask_thr == F.mask_thr).all()
            assert same, "a mask switched inside the stencil: pick another seed"
            assert abs((up - dn) / (2 * step) - np.asarray(grad).reshape(-1)[pos]) / scale < 2e-6, (name, pos)
