"""ctypes binding of the C ABI declared in include/moe.h.

Argument marshalling only: every function here has the name and the argument order of its
C counterpart, takes torch CUDA tensors (device memory) where the C function takes device
pointers, enqueues on torch's current stream and raises `MoeError` on a non-zero status.
There is no fallback: if the shared library has not been built, importing it fails loudly.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmoe_b200.so")

MOE_F32, MOE_BF16 = 0, 1
MOE_FLAG_GATE_SCREEN_OFF, MOE_FLAG_GATE_SCREEN_ON, MOE_FLAG_TC_ONE_CTA, MOE_FLAG_RECOMPUTE_HID = 1, 2, 4, 8
STATUS_NAMES = {0: "MOE_OK", 1: "MOE_ERR_INVALID_ARG", 2: "MOE_ERR_UNSUPPORTED", 3: "MOE_ERR_WORKSPACE",
                4: "MOE_ERR_CUDA", 5: "MOE_ERR_TIMEOUT"}

EXPORTS = ["moe_debug_launch_count", "moe_validate", "moe_query_sizes", "moe_workspace_bytes", "moe_query_ctx_layout", "moe_status_string", "moe_check_status",
           "moe_gate", "moe_dispatch", "moe_dispatch_noalloc", "moe_expert_ffn", "moe_combine", "moe_losses", "moe_combine_bwd",
           "moe_expert_ffn_bwd", "moe_dispatch_bwd", "moe_losses_bwd", "moe_gate_bwd", "moe_forward",
           "moe_backward", "moe_combine_layer", "moe_combine_layer_bwd", "moe_layer_forward", "moe_layer_backward",
           "moe_expert_adam_factored", "moe_check_buffer_sizes", "moe_debug_wait_timeout", "moe_debug_bounds_violations",
           "moe_expert_ffn_bits", "moe_expert_ffn_bwd_bits", "moe_query_balanced_sizes", "moe_gate_balanced", "moe_dispatch_balanced", "moe_combine_balanced",
           "moe_combine_balanced_bwd", "moe_gate_balanced_bwd", "moe_dispatch_balanced_bwd"]


class MoeError(RuntimeError):
    def __init__(self, fn, status):
        super().__init__(f"{fn} returned {STATUS_NAMES.get(status, status)}")
        self.status = status


class moe_config(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int32) for name in ("T", "d", "h", "n", "k", "a", "k1", "b", "k2", "act")] + \
               [("w_importance", ctypes.c_float), ("w_load", ctypes.c_float), ("flags", ctypes.c_int32)]


class moe_sizes(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int64) for name in
                ("R", "gate_cols", "logits_elems", "gates_elems", "kth_elems", "wg_elems", "load_elems",
                 "dload_elems", "ws_bytes", "ws_fwd_bytes", "ws_bwd_bytes", "ctx_bytes", "adam_state_elems",
                 "ws_adam_bytes")]


class moe_ctx_layout(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int64) for name in
                ("topk_idx", "gates", "clean", "raw_noise", "kth_vals", "kth_idx", "xs", "perm", "inv_perm",
                 "counts", "offsets", "hid", "ys", "importance", "load", "losses", "relu_bits")]


class moe_balanced_sizes(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int64) for name in ("m", "R", "mask_words", "ws_bytes")]


_lib = None


def lib():
    """The loaded shared library. Raises if it was not built (python -m paper_1701_06538_b200.build)."""
    global _lib
    if _lib is None:
        path = os.environ.get("MOE_B200_LIB", LIB_PATH)  # e.g. the checking build (libmoe_b200_check.so), for the test that runs it
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_1701_06538_b200.build`; "
                              "there is no fallback path")
        L = ctypes.CDLL(path)
        for name in EXPORTS:
            getattr(L, name).restype = ctypes.c_int32
        L.moe_status_string.restype = ctypes.c_char_p
        L.moe_debug_launch_count.restype = ctypes.c_int64
        L.moe_debug_bounds_violations.restype = ctypes.c_int64
        _lib = L
    return _lib


def make_config(T, d, h, n, k, act, w_importance=0.1, w_load=0.1, a=0, k1=0, b=0, k2=0, flags=0) -> moe_config:
    act_id = {"f32": MOE_F32, "bf16": MOE_BF16}.get(act, act)
    return moe_config(T, d, h, n, k, a, k1, b, k2, act_id, w_importance, w_load, flags)


def act_dtype(cfg: moe_config):
    return torch.bfloat16 if cfg.act == MOE_BF16 else torch.float32


def _p(t):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _call(name, cfg, *tensors, stream=True):
    # device tensors become pointers; a Python float is a `float` argument passed by value
    args = [ctypes.byref(cfg)] + [ctypes.c_float(t) if isinstance(t, float) else
                                  ctypes.c_int32(t) if isinstance(t, int) else _p(t) for t in tensors]
    if stream:
        args.append(_stream())
    status = getattr(lib(), name)(*args)
    if status != 0:
        raise MoeError(name, status)


def moe_debug_launch_count() -> int:
    return int(lib().moe_debug_launch_count())


def moe_validate(cfg) -> int:
    return lib().moe_validate(ctypes.byref(cfg))


def moe_workspace_bytes(cfg):
    """(forward, backward) workspace bytes."""
    f, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    status = lib().moe_workspace_bytes(ctypes.byref(cfg), ctypes.byref(f), ctypes.byref(b))
    if status:
        raise MoeError("moe_workspace_bytes", status)
    return f.value, b.value


def moe_query_sizes(cfg) -> moe_sizes:
    out = moe_sizes()
    status = lib().moe_query_sizes(ctypes.byref(cfg), ctypes.byref(out))
    if status != 0:
        raise MoeError("moe_query_sizes", status)
    return out


def moe_query_ctx_layout(cfg) -> moe_ctx_layout:
    out = moe_ctx_layout()
    status = lib().moe_query_ctx_layout(ctypes.byref(cfg), ctypes.byref(out))
    if status != 0:
        raise MoeError("moe_query_ctx_layout", status)
    return out


def moe_check_buffer_sizes(cfg, which, nbytes) -> int:
    return lib().moe_check_buffer_sizes(ctypes.byref(cfg), ctypes.c_int32(which), ctypes.c_size_t(nbytes))


def moe_debug_wait_timeout(ws, limit_ns):
    status = lib().moe_debug_wait_timeout(_p(ws), ctypes.c_int64(limit_ns), _stream())
    if status:
        raise MoeError("moe_debug_wait_timeout", status)


def moe_debug_bounds_violations() -> int:
    return int(lib().moe_debug_bounds_violations())


def moe_check_status(ws) -> int:
    return lib().moe_check_status(_p(ws), _stream())


def moe_gate(cfg, x, Wg, Wnoise, noise, topk_idx, gates, clean, raw_noise, kth_vals, kth_idx, ws):
    _call("moe_gate", cfg, x, Wg, Wnoise, noise, topk_idx, gates, clean, raw_noise, kth_vals, kth_idx, ws)


def moe_dispatch(cfg, x, topk_idx, xs, perm, inv_perm, counts, offsets, ws):
    _call("moe_dispatch", cfg, x, topk_idx, xs, perm, inv_perm, counts, offsets, ws)


def moe_dispatch_noalloc(cfg, x, topk_idx, xs, perm, inv_perm, counts, offsets):
    """moe_dispatch for callers that cannot provide a workspace: the scratch is a fixed array inside
    the library (see include/moe.h for the size limit and the sharing rules)."""
    _call("moe_dispatch_noalloc", cfg, x, topk_idx, xs, perm, inv_perm, counts, offsets)


def moe_expert_ffn(cfg, xs, offsets, W1, b1, W2, b2, hid, ys, ws):
    _call("moe_expert_ffn", cfg, xs, offsets, W1, b1, W2, b2, hid, ys, ws)


def moe_expert_ffn_bits(cfg, xs, offsets, W1, b1, W2, b2, hid, ys, relu_bits, ws):
    _call("moe_expert_ffn_bits", cfg, xs, offsets, W1, b1, W2, b2, hid, ys, relu_bits, ws)


def moe_expert_ffn_bwd_bits(cfg, xs, hid, relu_bits, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws):
    _call("moe_expert_ffn_bwd_bits", cfg, xs, hid, relu_bits, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws)


def moe_combine(cfg, ys, gates, inv_perm, y):
    _call("moe_combine", cfg, ys, gates, inv_perm, y)


def moe_losses(cfg, topk_idx, gates, clean, raw_noise, kth_vals, importance, load, losses, ws):
    _call("moe_losses", cfg, topk_idx, gates, clean, raw_noise, kth_vals, importance, load, losses, ws)


def moe_combine_bwd(cfg, dY, ys, gates, inv_perm, dgates, dys):
    _call("moe_combine_bwd", cfg, dY, ys, gates, inv_perm, dgates, dys)


def moe_expert_ffn_bwd(cfg, xs, hid, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws):
    _call("moe_expert_ffn_bwd", cfg, xs, hid, dys, offsets, W1, W2, dxs, dW1, db1, dW2, db2, ws)


def moe_dispatch_bwd(cfg, dxs, inv_perm, dX_expert):
    _call("moe_dispatch_bwd", cfg, dxs, inv_perm, dX_expert)


def moe_losses_bwd(cfg, importance, load, topk_idx, dgates, dload, ws):
    _call("moe_losses_bwd", cfg, importance, load, topk_idx, dgates, dload, ws)


def moe_gate_bwd(cfg, x, Wg, Wnoise, noise, clean, raw_noise, topk_idx, gates, kth_vals, kth_idx, dgates, dload,
                 dWg, dWnoise, dX_gate, ws):
    _call("moe_gate_bwd", cfg, x, Wg, Wnoise, noise, clean, raw_noise, topk_idx, gates, kth_vals, kth_idx, dgates,
          dload, dWg, dWnoise, dX_gate, ws)


def moe_forward(cfg, x, Wg, Wnoise, noise, W1, b1, W2, b2, y, losses, importance, load, counts, ctx, ws):
    _call("moe_forward", cfg, x, Wg, Wnoise, noise, W1, b1, W2, b2, y, losses, importance, load, counts, ctx, ws)


def moe_backward(cfg, dY, x, Wg, Wnoise, noise, W1, b1, W2, b2, ctx, dX, dWg, dWnoise, dW1, db1, dW2, db2, ws):
    _call("moe_backward", cfg, dY, x, Wg, Wnoise, noise, W1, b1, W2, b2, ctx, dX, dWg, dWnoise, dW1, db1, dW2, db2,
          ws)


def moe_query_balanced_sizes(cfg) -> moe_balanced_sizes:
    out = moe_balanced_sizes()
    status = lib().moe_query_balanced_sizes(ctypes.byref(cfg), ctypes.byref(out))
    if status != 0:
        raise MoeError("moe_query_balanced_sizes", status)
    return out


def moe_gate_balanced(cfg, x, Wg, thresholds, logits, probs, mask_bits, tok_of_row, offsets, den, tok_ptr, tok_rows,
                      loss_batchwise, thr_counts, ws):
    _call("moe_gate_balanced", cfg, x, Wg, thresholds, logits, probs, mask_bits, tok_of_row, offsets, den, tok_ptr,
          tok_rows, loss_batchwise, thr_counts, ws)


def moe_dispatch_balanced(cfg, x, tok_of_row, xs):
    _call("moe_dispatch_balanced", cfg, x, tok_of_row, xs)


def moe_combine_balanced(cfg, ys, probs, den, tok_ptr, tok_rows, y):
    _call("moe_combine_balanced", cfg, ys, probs, den, tok_ptr, tok_rows, y)


def moe_combine_balanced_bwd(cfg, dY, ys, probs, den, tok_of_row, dG_row, dys):
    _call("moe_combine_balanced_bwd", cfg, dY, ys, probs, den, tok_of_row, dG_row, dys)


def moe_gate_balanced_bwd(cfg, x, Wg, probs, mask_bits, den, thresholds, tok_ptr, tok_rows, dG_row, thr_counts, w_batchwise,
                          dWg, dX_gate, dthresholds, ws):
    _call("moe_gate_balanced_bwd", cfg, x, Wg, probs, mask_bits, den, thresholds, tok_ptr, tok_rows, dG_row, thr_counts,
          float(w_batchwise), dWg, dX_gate, dthresholds, ws)


def moe_dispatch_balanced_bwd(cfg, dxs, tok_ptr, tok_rows, dX_gate, dX):
    _call("moe_dispatch_balanced_bwd", cfg, dxs, tok_ptr, tok_rows, dX_gate, dX)


def moe_expert_adam_factored(cfg, W1, b1, W2, b2, dW1, db1, dW2, db2, state, lr, beta2, eps, step, ws):
    _call("moe_expert_adam_factored", cfg, W1, b1, W2, b2, dW1, db1, dW2, db2, state, float(lr), float(beta2), float(eps),
          int(step), ws)


def moe_combine_layer(cfg, ys, gates, inv_perm, x, keep_bits, drop_prob, out):
    _call("moe_combine_layer", cfg, ys, gates, inv_perm, x, keep_bits, float(drop_prob), out)


def moe_combine_layer_bwd(cfg, dOut, ys, gates, inv_perm, keep_bits, drop_prob, dgates, dys):
    _call("moe_combine_layer_bwd", cfg, dOut, ys, gates, inv_perm, keep_bits, float(drop_prob), dgates, dys)


def moe_layer_forward(cfg, x, Wg, Wnoise, noise, W1, b1, W2, b2, keep_bits, drop_prob, out, losses, importance, load,
                      counts, ctx, ws):
    _call("moe_layer_forward", cfg, x, Wg, Wnoise, noise, W1, b1, W2, b2, keep_bits, float(drop_prob), out, losses,
          importance, load, counts, ctx, ws)


def moe_layer_backward(cfg, dOut, x, Wg, Wnoise, noise, W1, b1, W2, b2, keep_bits, drop_prob, ctx, dX, dWg, dWnoise,
                       dW1, db1, dW2, db2, ws):
    _call("moe_layer_backward", cfg, dOut, x, Wg, Wnoise, noise, W1, b1, W2, b2, keep_bits, float(drop_prob), ctx, dX,
          dWg, dWnoise, dW1, db1, dW2, db2, ws)


# ----------------------------------------------------------------------------------------------
# Buffer helpers (allocation only; torch is the allocator, nothing is computed here)
# ----------------------------------------------------------------------------------------------
def empty_bytes(nbytes, device="cuda"):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def ctx_views(cfg, ctx):
    """Typed views of the tensors moe_forward saved in `ctx` (no copies)."""
    L, S = moe_query_ctx_layout(cfg), moe_query_sizes(cfg)
    T, d, h, n, k, R = cfg.T, cfg.d, cfg.h, cfg.n, cfg.k, S.R
    adt = act_dtype(cfg)
    esz = 2 if cfg.act == MOE_BF16 else 4

    def view(off, count, dtype, shape):
        size = torch.empty((), dtype=dtype).element_size()
        return ctx[off:off + count * size].view(dtype).view(*shape)

    views = dict(topk_idx=view(L.topk_idx, R, torch.int32, (T, k)),
                gates=view(L.gates, S.gates_elems, torch.float32, (-1,)),
                clean=view(L.clean, S.logits_elems, torch.float32, (-1,)),
                raw_noise=view(L.raw_noise, S.logits_elems, torch.float32, (-1,)),
                kth_vals=view(L.kth_vals, S.kth_elems, torch.float32, (-1, 2)),
                kth_idx=view(L.kth_idx, S.kth_elems, torch.int32, (-1, 2)),
                xs=view(L.xs, R * d, adt, (R, d)), perm=view(L.perm, R, torch.int32, (R,)),
                inv_perm=view(L.inv_perm, R, torch.int32, (R,)), counts=view(L.counts, n, torch.int32, (n,)),
                offsets=view(L.offsets, n + 1, torch.int32, (n + 1,)),
                ys=view(L.ys, R * d, adt, (R, d)), importance=view(L.importance, n, torch.float32, (n,)),
                load=view(L.load, S.load_elems, torch.float32, (-1,)), losses=view(L.losses, 2, torch.float32, (2,)))
    if not cfg.flags & MOE_FLAG_RECOMPUTE_HID:  # with the flag the context keeps no hidden activations
        views["hid"] = view(L.hid, R * h, adt, (R, h))
        if L.relu_bits + R * (h // 32) * 4 <= S.ctx_bytes and h % 32 == 0 and L.relu_bits > L.losses:
            views["relu_bits"] = view(L.relu_bits, R * (h // 32), torch.int32, (R, h // 32))
    return views
