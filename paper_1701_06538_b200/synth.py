"""Seeded synthetic inputs for the Mixture-of-Experts layer.

This module only draws numbers: it holds none of the layer's arithmetic and is the one
piece the CPU oracle's callers and the CUDA library's callers both use. Every tensor comes
from its own counter-based stream (numpy's Philox, key = (seed, tensor id, block)), so any
expert's weights can be drawn alone, in any order, on any machine.

The workloads stand in for the paper's language-modelling and translation batches
(Appendix C-E): the shapes are those of its models (d_model 512 or 1024, hidden layer of
1024 to 8192 units, 4 experts per token, up to 4096 experts hierarchically), the batch is
all time steps of a training batch flattened into T rows, values are standard normal with
fan-in scaled weights.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 0x17010653

# tensor ids of the streams
_X, _WG, _WN, _NOISE, _W1, _W2, _DY, _BETA, _WG_S, _WN_S, _NOISE_S, _B1, _B2, _KEEP = range(1, 15)


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    d: int
    h: int
    n: int
    k: int
    a: int = 0  # hierarchical when a > 0: a groups (top k1) of b experts (top k2); n = a*b, k = k1*k2
    k1: int = 0
    b: int = 0
    k2: int = 0
    act: str = "bf16"  # storage type of activations and expert weights: "f32" or "bf16"
    w_importance: float = 0.1
    w_load: float = 0.1
    seed: int = BASE_SEED
    skew: str = "none"  # "none" | "normal" | "zipf": per-expert logit offsets through a constant feature
    gamma: float = 0.0  # scale of those offsets
    bias_std: float = 0.0  # expert biases are zero in the paper-shaped workloads

    @property
    def R(self) -> int:
        return self.T * self.k

    @property
    def hier(self):
        return (self.a, self.k1, self.b, self.k2) if self.a > 0 else None

    def scaled(self, T: int) -> "Workload":
        return replace(self, T=T, name=f"{self.name}-T{T}")


# The five workloads. gamma of c3 / c5 was found once by bisection on the realised expert
# counts (c3: max/min count about 4; c5: log-log slope of count against rank about -1.1).
CONFIGS = {
    "c1": Workload("c1-tiny-f32", T=256, d=64, h=128, n=8, k=2, act="f32", seed=BASE_SEED + 0),
    "c2": Workload("c2-lm-flat-32", T=8192, d=512, h=1024, n=32, k=4, seed=BASE_SEED + 1),
    "c3": Workload("c3-flat-256-uneven", T=32768, d=512, h=1024, n=256, k=4, seed=BASE_SEED + 2,
                   skew="normal", gamma=0.205),
    "c4": Workload("c4-hier-64x64", T=65536, d=512, h=1024, n=4096, k=4, a=64, k1=2, b=64, k2=2,
                   seed=BASE_SEED + 3),
    "c5": Workload("c5-wide-zipf-128", T=131072, d=1024, h=4096, n=128, k=2, seed=BASE_SEED + 4,
                   skew="zipf", gamma=0.79),
}


def _rng(w: Workload, tensor: int, block: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[w.seed, (tensor << 32) | block]))


def _normal(w, tensor, shape, std=1.0, block=0):
    out = _rng(w, tensor, block).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out


def storage_grid(a: np.ndarray, act: str) -> np.ndarray:
    """Snap float32 values to the values representable in the storage type (no-op for f32)."""
    if act == "f32":
        return a
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).bfloat16().float().numpy()


def make_x(w: Workload) -> np.ndarray:
    x = _normal(w, _X, (w.T, w.d))
    if w.skew != "none":
        x[:, 0] = 1.0  # constant feature: the gate of Eq. 4 has no bias term of its own
    return storage_grid(x, w.act)


def make_dY(w: Workload) -> np.ndarray:
    return storage_grid(_normal(w, _DY, (w.T, w.d)), w.act)


def make_keep_bits(w: Workload, drop_prob: float) -> np.ndarray:
    """Dropout keep mask of the layer epilogue, packed: [T, d/8] uint8, bit (q % 8) of byte q // 8 is column q;
    a column is kept with probability 1 - drop_prob."""
    keep = _rng(w, _KEEP).random((w.T, w.d), dtype=np.float32) >= np.float32(drop_prob)
    return np.packbits(keep, axis=1, bitorder="little")


def expert_offsets(w: Workload) -> np.ndarray:
    """Per-expert logit offsets beta_i placed in row 0 of W_g (zero when skew is "none")."""
    n_gate = w.a if w.a > 0 else w.n
    if w.skew == "normal":
        return (w.gamma * _normal(w, _BETA, (n_gate,))).astype(np.float32)
    if w.skew == "zipf":
        return (-w.gamma * 1.1 * np.log(np.arange(1, n_gate + 1))).astype(np.float32)
    return np.zeros(n_gate, np.float32)


def make_gate(w: Workload):
    """Gate weights and noise. Flat: (Wg [d,n], Wnoise [d,n], noise [T,n]).
    Hierarchical: each is a pair (primary over a groups, secondary [a,d,b] / [T,k1,b])."""
    std = 1.0 / np.sqrt(w.d)
    n_gate = w.a if w.a > 0 else w.n
    Wg = _normal(w, _WG, (w.d, n_gate), std)
    Wn = _normal(w, _WN, (w.d, n_gate), std)
    if w.skew != "none":
        Wg[0, :] = expert_offsets(w)
    noise = _normal(w, _NOISE, (w.T, n_gate))
    if w.a == 0:
        return Wg, Wn, noise
    Wg_s = _normal(w, _WG_S, (w.a, w.d, w.b), std)
    Wn_s = _normal(w, _WN_S, (w.a, w.d, w.b), std)
    noise_s = _normal(w, _NOISE_S, (w.T, w.k1, w.b))
    return (Wg, Wg_s), (Wn, Wn_s), (noise, noise_s)


def make_expert(w: Workload, e: int):
    """Weights of expert e alone: W1 [d,h], b1 [h], W2 [h,d], b2 [d]."""
    W1 = storage_grid(_normal(w, _W1, (w.d, w.h), 1.0 / np.sqrt(w.d), block=e), w.act)
    W2 = storage_grid(_normal(w, _W2, (w.h, w.d), 1.0 / np.sqrt(w.h), block=e), w.act)
    if w.bias_std > 0:
        b1 = storage_grid(_normal(w, _B1, (w.h,), w.bias_std, block=e), w.act)
        b2 = storage_grid(_normal(w, _B2, (w.d,), w.bias_std, block=e), w.act)
    else:
        b1 = np.zeros(w.h, np.float32)
        b2 = np.zeros(w.d, np.float32)
    return W1, b1, W2, b2


def make_experts(w: Workload):
    """All expert weights stacked: W1 [n,d,h], b1 [n,h], W2 [n,h,d], b2 [n,d] (float32 host arrays)."""
    W1 = np.empty((w.n, w.d, w.h), np.float32)
    W2 = np.empty((w.n, w.h, w.d), np.float32)
    b1 = np.empty((w.n, w.h), np.float32)
    b2 = np.empty((w.n, w.d), np.float32)
    for e in range(w.n):
        W1[e], b1[e], W2[e], b2[e] = make_expert(w, e)
    return W1, b1, W2, b2


def make_all(w: Workload) -> dict:
    Wg, Wn, noise = make_gate(w)
    W1, b1, W2, b2 = make_experts(w)
    return dict(x=make_x(w), Wg=Wg, Wnoise=Wn, noise=noise, W1=W1, b1=b1, W2=W2, b2=b2, dY=make_dY(w))
