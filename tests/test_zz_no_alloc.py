"""moe_dispatch_noalloc against moe_dispatch, through the C ABI.

Some callers of this library cannot hand it a workspace: they run where device allocation is
forbidden (inside another framework's fixed memory plan, or in a latency-critical loop where
cudaMalloc would stall the whole device) and only own their input and output buffers. For them
the library carries a fixed scratch array of its own. This file checks that the entry point using
that array gives exactly the results of the ordinary one, on two calls in a row (the array is
shared and keeps the previous call's contents), and that it refuses sizes the array cannot hold.
It is collected last so that a failure here cannot hide the other tests' results.
"""
import numpy as np
import pytest
import torch

from paper_1701_06538_b200 import binding as B

pytestmark = pytest.mark.gpu


def routing(T, n, k, seed):
    g = np.random.default_rng(seed)
    idx = np.stack([g.permutation(n)[:k] for _ in range(T)]).astype(np.int32)
    return torch.from_numpy(idx).cuda()


def run_both(T, d, n, k, act, seed):
    cfg = B.make_config(T=T, d=d, h=d, n=n, k=k, act=act)
    S = B.moe_query_sizes(cfg)
    adt = torch.bfloat16 if act == "bf16" else torch.float32
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = torch.randn(T, d, device="cuda", generator=g).to(adt)
    idx = routing(T, n, k, seed)
    outs = []
    for fn in ("ws", "noalloc"):
        xs = torch.zeros(S.R, d, dtype=adt, device="cuda")
        perm, inv = (torch.full((S.R,), -1, dtype=torch.int32, device="cuda") for _ in range(2))
        counts = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        offsets = torch.full((n + 1,), -1, dtype=torch.int32, device="cuda")
        if fn == "ws":
            B.moe_dispatch(cfg, x, idx, xs, perm, inv, counts, offsets, B.empty_bytes(S.ws_bytes))
        else:
            B.moe_dispatch_noalloc(cfg, x, idx, xs, perm, inv, counts, offsets)
        torch.cuda.synchronize()
        outs.append((xs, perm, inv, counts, offsets))
    for a, b in zip(*outs):
        assert torch.equal(a, b)  # integer and copy work: bit-exact
    return outs[1]


def test_noalloc_matches_workspace_variant_twice_in_a_row():
    # first call: many experts, ragged tail; second call: different shape and type, reusing the
    # same fixed scratch while it still holds the first call's histograms
    xs, perm, inv, counts, offsets = run_both(T=3000, d=64, n=300, k=4, act="bf16", seed=1)
    assert int(counts.sum()) == 3000 * 4 and int(offsets[-1]) == 3000 * 4
    assert torch.equal(perm[inv.long()].cpu(), torch.arange(3000 * 4, dtype=torch.int32))
    run_both(T=1111, d=36, n=7, k=3, act="f32", seed=2)
    run_both(T=3000, d=64, n=300, k=4, act="bf16", seed=3)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    cfg = B.make_config(T=1 << 20, d=64, h=64, n=4096, k=2, act="bf16")  # needs 2048 * 4096 + 64 ints
    t = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MoeError) as err:
        B.moe_dispatch_noalloc(cfg, t, t, t, t, t, t, t)
    assert err.value.status == 3  # MOE_ERR_WORKSPACE: nothing was launched
    assert B.lib().moe_status_string(3) == b"workspace too small"
