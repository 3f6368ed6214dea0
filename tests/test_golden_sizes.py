"""The sizes the library reports against the figures the paper prints (Appendix C, Table 7).

Rows of that table differ only by their MoE layer, so the differences of its two size columns are the layer's expert
and gating parameters and the gating network's multiply-adds: they pin the shapes the input generator draws and the
element counts the C library computes (moe_query_sizes: wg_elems, gate_cols) for flat and hierarchical layers."""
import os

import numpy as np

from paper_1701_06538_b200 import binding as B
from paper_1701_06538_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "appendix_c_table7_model_sizes.txt")


def rows():
    out = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, n, a, b, k, ops, params = line.split()
        out.append(dict(name=name, n=int(n), a=int(a), b=int(b), k=int(k), ops=float(ops), params=float(params)))
    return out


def layer_sizes(r, d=512, h=1024):
    """(parameters, forward multiply-adds per token) of the MoE layer of one table row, from the product's own code."""
    hier = r["a"] > 0
    cfg = B.make_config(T=16, d=d, h=h, n=r["n"], k=r["k"], act="f32", a=r["a"], k1=2 if hier else 0, b=r["b"],
                        k2=2 if hier else 0)
    assert B.moe_validate(cfg) == 0
    S = B.moe_query_sizes(cfg)
    w = synth.Workload(r["name"], T=16, d=d, h=h, n=r["n"], k=r["k"], a=r["a"], k1=2 if hier else 0, b=r["b"],
                       k2=2 if hier else 0)
    W1, b1, W2, b2 = synth.make_expert(w, 0)
    per_expert = W1.size + W2.size            # the paper's count has no biases (they are zero in these workloads)
    assert (W1.shape, W2.shape) == ((d, h), (h, d)) and not b1.any() and not b2.any()
    params = r["n"] * per_expert + 2 * S.wg_elems           # W_g and W_noise
    macs = r["k"] * per_expert + 2 * d * S.gate_cols         # k experts + both gate projections
    return params, macs


def test_expert_size_is_the_papers_one_million():
    params, macs = layer_sizes(rows()[0])
    assert (params - 2 * 512 * 4) // 4 == 512 * 1024 + 1024 * 512 == 1048576


def test_table7_differences_between_models():
    R = rows()
    base = R[0]
    p0, m0 = layer_sizes(base)
    for r in R[1:]:
        p, m = layer_sizes(r)
        # two printed values, each rounded to 0.1 million
        assert abs((p - p0) / 1e6 - (r["params"] - base["params"])) <= 0.1 + 1e-9, r["name"]
        assert abs((m - m0) / 1e6 - (r["ops"] - base["ops"])) <= 0.1 + 1e-9, r["name"]


def test_moe4_layer_is_half_of_the_eight_million_ops_budget():
    # Appendix C: with four active experts the MoE layer accounts for about 4 of the 8 million multiply-adds per step
    _, macs = layer_sizes(rows()[0])
    assert abs(macs / 1e6 - 4.2) < 0.01
