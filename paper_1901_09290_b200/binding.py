"""Thin ctypes binding of the C ABI in ``include/pt.h``: same names, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; their ``data_ptr()`` is what the
library sees. Every computation happens inside the library's CUDA kernels; if the shared
library is missing or a call fails, this module raises -- there is no CPU path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import (POINTER, c_int64, Structure, byref, c_char_p, c_double, c_float, c_int32, c_size_t, c_uint8, c_uint64,
                    c_void_p)
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpt_b200.so")

PT_OK = 0
PT_CONV_FWD, PT_CONV_DGRAD, PT_CONV_WGRAD = 0, 1, 2
STATUS_NAMES = ["PT_OK", "PT_ERR_INVALID_ARG", "PT_ERR_UNSUPPORTED", "PT_ERR_WORKSPACE", "PT_ERR_CUDA",
                "PT_ERR_TIMEOUT", "PT_ERR_ARCH"]


class PtError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        detail = ""
        if name == "PT_ERR_CUDA":
            detail = ": " + (lib().pt_last_cuda_error() or b"").decode()
        super().__init__(f"{what} failed: {name}{detail}")


class pt_conv_desc(Structure):
    _fields_ = [(n, c_int32) for n in ("N", "H", "W", "C", "K", "R", "S", "stride", "pad",
                                       "ldx", "ldy", "ldw", "out_f32", "algo")]


class pt_layer(Structure):
    _fields_ = [("w", c_void_p), ("g", c_void_p), ("v", c_void_p), ("w_bf16", c_void_p),
                ("K", c_int32), ("C", c_int32), ("RS", c_int32), ("ldw", c_int32),
                ("reg_in", c_uint8), ("reg_out", c_uint8),
                ("sumsq_out", c_void_p), ("sumsq_in", c_void_p), ("zero_out", c_void_p), ("zero_in", c_void_p)]


class pt_sgd_hparams(Structure):
    _fields_ = [("lambda_", c_float), ("lr", c_float), ("momentum", c_float), ("weight_decay", c_float)]


class pt_bn_desc(Structure):
    _fields_ = [("N", c_int32), ("H", c_int32), ("W", c_int32), ("C", c_int32), ("ld", c_int32),
                ("eps", c_float), ("momentum", c_float), ("relu", c_int32)]


class pt_pool_desc(Structure):
    _fields_ = [(n, c_int32) for n in ("N", "H", "W", "C", "ld", "R", "stride", "pad")]


class pt_layer_shape(Structure):
    _fields_ = [(n, c_int32) for n in ("H", "W", "C", "K", "R", "S", "stride", "pad")]


class pt_space(Structure):
    _fields_ = [("size", c_int32), ("fixed", c_uint8)]


class pt_layer_link(Structure):
    _fields_ = [("in_space", c_int32), ("out_space", c_int32), ("bn", c_void_p * 4)]


class pt_graph(Structure):
    _fields_ = [("spaces", POINTER(pt_space)), ("n_spaces", c_int32),
                ("layers", POINTER(pt_layer)), ("links", POINTER(pt_layer_link)), ("n_layers", c_int32)]


EXPORTS = {
    "pt_create": (c_int32, [POINTER(c_void_p), c_int32]),
    "pt_destroy": (c_int32, [c_void_p]),
    "pt_status_string": (c_char_p, [c_int32]),
    "pt_last_cuda_error": (c_char_p, []),
    "pt_poll_device_status": (c_int32, [c_void_p, c_void_p]),
    "pt_launch_count": (c_uint64, [c_void_p]),
    "pt_test_set_wait_limit": (c_int32, [c_void_p, ctypes.c_uint32]),
    "pt_test_skip_next_arrive": (c_int32, [c_void_p, c_int32]),
    "pt_set_wgrad_cta_limit": (c_int32, [c_void_p, c_int32]),
    "pt_conv_wgrad_ctas": (c_int32, [c_void_p, POINTER(pt_conv_desc), POINTER(c_int32)]),
    "pt_conv_workspace_bytes": (c_size_t, [c_void_p, POINTER(pt_conv_desc), c_int32]),
    "pt_conv_fwd": (c_int32, [c_void_p, POINTER(pt_conv_desc), c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "pt_conv_fwd_stats_bytes": (c_size_t, [c_void_p, POINTER(pt_conv_desc)]),
    "pt_conv_fwd_stats": (c_int32, [c_void_p, POINTER(pt_conv_desc), c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, POINTER(c_int32),
                                    c_void_p, c_size_t, c_void_p]),
    "pt_bn_relu_fwd_stats": (c_int32, [c_void_p, POINTER(pt_bn_desc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                       c_void_p, c_void_p, c_void_p, c_int32, c_void_p]),
    "pt_maxpool_fwd": (c_int32, [c_void_p, POINTER(pt_pool_desc), c_void_p, c_void_p, c_void_p, c_void_p]),
    "pt_maxpool_bwd": (c_int32, [c_void_p, POINTER(pt_pool_desc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "pt_conv_dgrad": (c_int32, [c_void_p, POINTER(pt_conv_desc), c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "pt_conv_wgrad": (c_int32, [c_void_p, POINTER(pt_conv_desc), c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "pt_group_lasso_workspace_bytes": (c_size_t, [c_void_p, POINTER(pt_layer), c_int32]),
    "pt_group_lasso_sgd_step": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, POINTER(pt_sgd_hparams), c_void_p,
                                          c_void_p, c_size_t, c_void_p]),
    "pt_group_lasso_norms": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, c_void_p, c_void_p, c_size_t, c_void_p]),
    "pt_group_lasso_sgd_apply": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, POINTER(pt_sgd_hparams), c_void_p, c_size_t, c_void_p]),
    "pt_group_lasso_sgd_apply_layers": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, c_int32, c_int32, POINTER(pt_sgd_hparams), c_void_p,
                                                  c_size_t, c_void_p]),
    "pt_find_zero_groups": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, c_float, c_int32, c_void_p, c_size_t, c_void_p]),
    "pt_find_zero_groups_carried": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, c_float, c_int32, c_void_p, c_size_t, c_void_p]),
    "pt_group_lasso_sgd_step_carried": (c_int32, [c_void_p, POINTER(pt_layer), c_int32, POINTER(pt_sgd_hparams), c_int32, c_void_p,
                                                  c_void_p, c_size_t, c_void_p]),
    "pt_find_zero_groups_noalloc": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p]),
    "pt_bn_workspace_bytes": (c_size_t, [c_void_p, POINTER(pt_bn_desc)]),
    "pt_bn_relu_fwd": (c_int32, [c_void_p, POINTER(pt_bn_desc)] + [c_void_p] * 9 + [c_void_p, c_size_t, c_void_p]),
    "pt_bn_relu_bwd": (c_int32, [c_void_p, POINTER(pt_bn_desc)] + [c_void_p] * 10 + [c_void_p, c_size_t, c_void_p]),
    "pt_training_memory_bytes": (c_size_t, [POINTER(pt_layer_shape), c_int32, c_int32]),
    "pt_update_mini_batch": (c_int32, [POINTER(pt_layer_shape), c_int32, c_size_t, c_int32, c_float, c_int32, POINTER(c_int32), POINTER(c_float)]),
    "pt_cross_entropy_workspace_bytes": (c_size_t, [c_int32]),
    "pt_cross_entropy": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_size_t, c_void_p]),
    "pt_set_coeff": (c_int32, [c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_void_p]),
    "pt_dense_channel_list": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p]),
    "pt_channel_gather": (c_int32, [c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p]),
    "pt_channel_scatter_add": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_void_p, c_void_p, c_int32, c_int32, c_int64,
                                         c_int32, c_void_p]),
    "pt_reconfigure_plan": (c_int32, [c_void_p, POINTER(pt_graph), c_void_p, POINTER(c_int32), c_void_p]),
    "pt_reconfigure": (c_int32, [c_void_p, POINTER(pt_graph), c_void_p, POINTER(pt_graph), c_void_p]),
}

_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library. Raises if it has not been built (run ``python -m paper_1901_09290_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"CUDA library not built: {LIB_PATH} is missing (python -m paper_1901_09290_b200.build)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(L, name)          # AttributeError if a declared symbol is not exported
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, what: str):
    if status != PT_OK:
        raise PtError(status, what)


class Context:
    """Owns a pt_ctx for one device."""

    def __init__(self, device: int = 0):
        self.handle = c_void_p()
        _check(lib().pt_create(byref(self.handle), device), "pt_create")
        self.device = device

    def close(self):
        if self.handle:
            lib().pt_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def launch_count(self) -> int:
        return int(lib().pt_launch_count(self.handle))

    def set_wgrad_cta_limit(self, max_ctas: int):
        _check(lib().pt_set_wgrad_cta_limit(self.handle, int(max_ctas)), "pt_set_wgrad_cta_limit")

    def poll(self, stream=None):
        _check(lib().pt_poll_device_status(self.handle, _stream(stream)), "pt_poll_device_status")


def make_conv_desc(N, H, W, C, K, R, S, stride, pad, ldx=None, ldy=None, ldw=None, out_f32=0, algo=0) -> pt_conv_desc:
    p8 = lambda c: (c + 7) // 8 * 8
    return pt_conv_desc(N, H, W, C, K, R, S, stride, pad, ldx or p8(C), ldy or p8(K), ldw or p8(C), out_f32, algo)


def pt_test_set_wait_limit(ctx: Context, milliseconds: int):
    _check(lib().pt_test_set_wait_limit(ctx.handle, milliseconds), "pt_test_set_wait_limit")


def pt_test_skip_next_arrive(ctx: Context, which: int):
    _check(lib().pt_test_skip_next_arrive(ctx.handle, which), "pt_test_skip_next_arrive")


def pt_set_wgrad_cta_limit(ctx: Context, max_ctas: int):
    ctx.set_wgrad_cta_limit(max_ctas)


def pt_conv_workspace_bytes(ctx: Context, d: pt_conv_desc, which: int) -> int:
    return int(lib().pt_conv_workspace_bytes(ctx.handle, byref(d), which))


def _ws(ws):
    return (None, 0) if ws is None else (ws.data_ptr(), ws.numel() * ws.element_size())


def pt_conv_fwd(ctx, d, x, w, y, ws=None, stream=None):
    p, n = _ws(ws)
    _check(lib().pt_conv_fwd(ctx.handle, byref(d), _ptr(x), _ptr(w), _ptr(y), p, n, _stream(stream)), "pt_conv_fwd")


def pt_conv_fwd_stats_bytes(ctx, d) -> int:
    return int(lib().pt_conv_fwd_stats_bytes(ctx.handle, byref(d)))


def pt_conv_fwd_stats(ctx, d, x, w, y, stats, ws=None, stream=None) -> int:
    """Returns the number of rows of partial sums the launch left in `stats`."""
    p, n = _ws(ws)
    parts = c_int32(0)
    _check(lib().pt_conv_fwd_stats(ctx.handle, byref(d), _ptr(x), _ptr(w), _ptr(y), _ptr(stats), stats.numel() * stats.element_size(),
                                   byref(parts), p, n, _stream(stream)), "pt_conv_fwd_stats")
    return int(parts.value)


def pt_bn_relu_fwd_stats(ctx, d, x, residual, gamma, beta, running_mean, running_var, save_mean, save_invstd, y, stats, n_parts,
                         stream=None):
    _check(lib().pt_bn_relu_fwd_stats(ctx.handle, byref(d), _ptr(x), _ptr(residual), _ptr(gamma), _ptr(beta), _ptr(running_mean),
                                      _ptr(running_var), _ptr(save_mean), _ptr(save_invstd), _ptr(y), _ptr(stats), n_parts,
                                      _stream(stream)), "pt_bn_relu_fwd_stats")


def pt_conv_dgrad(ctx, d, dy, w, dx, ws=None, stream=None):
    p, n = _ws(ws)
    _check(lib().pt_conv_dgrad(ctx.handle, byref(d), _ptr(dy), _ptr(w), _ptr(dx), p, n, _stream(stream)), "pt_conv_dgrad")


def pt_conv_wgrad(ctx, d, x, dy, dw, ws=None, stream=None):
    p, n = _ws(ws)
    _check(lib().pt_conv_wgrad(ctx.handle, byref(d), _ptr(x), _ptr(dy), _ptr(dw), p, n, _stream(stream)), "pt_conv_wgrad")


def make_layer(w, g, v, w_bf16, K, C, RS, ldw, reg_in, reg_out, sumsq_out, sumsq_in, zero_out, zero_in) -> pt_layer:
    return pt_layer(_ptr(w), _ptr(g), _ptr(v), _ptr(w_bf16), K, C, RS, ldw, int(bool(reg_in)), int(bool(reg_out)),
                    _ptr(sumsq_out), _ptr(sumsq_in), _ptr(zero_out), _ptr(zero_in))


def layer_array(layers: Sequence[pt_layer]):
    return (pt_layer * len(layers))(*layers)


def pt_group_lasso_workspace_bytes(ctx, layers) -> int:
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    return int(lib().pt_group_lasso_workspace_bytes(ctx.handle, arr, len(arr)))


def pt_group_lasso_sgd_step(ctx, layers, lam, lr, momentum, weight_decay=0.0, reg_sum_out=None, ws=None, stream=None):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    hp = pt_sgd_hparams(lam, lr, momentum, weight_decay)
    p, n = _ws(ws)
    _check(lib().pt_group_lasso_sgd_step(ctx.handle, arr, len(arr), byref(hp), _ptr(reg_sum_out), p, n, _stream(stream)),
           "pt_group_lasso_sgd_step")


def pt_group_lasso_sgd_step_carried(ctx, layers, lam, lr, momentum, weight_decay=0.0, reg_sum_next=None, ws=None, stream=None,
                                    with_maxima=False):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    hp = pt_sgd_hparams(lam, lr, momentum, weight_decay)
    p, n = _ws(ws)
    _check(lib().pt_group_lasso_sgd_step_carried(ctx.handle, arr, len(arr), byref(hp), int(bool(with_maxima)), _ptr(reg_sum_next), p, n,
                                                 _stream(stream)),
           "pt_group_lasso_sgd_step_carried")


def pt_find_zero_groups_carried(ctx, layers, threshold=1e-4, zero_in_place=False, ws=None, stream=None):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    p, n = _ws(ws)
    _check(lib().pt_find_zero_groups_carried(ctx.handle, arr, len(arr), threshold, int(bool(zero_in_place)), p, n, _stream(stream)),
           "pt_find_zero_groups_carried")


def pt_group_lasso_norms(ctx, layers, reg_sum_out=None, ws=None, stream=None):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    p, n = _ws(ws)
    _check(lib().pt_group_lasso_norms(ctx.handle, arr, len(arr), _ptr(reg_sum_out), p, n, _stream(stream)), "pt_group_lasso_norms")


def pt_group_lasso_sgd_apply(ctx, layers, lam, lr, momentum, weight_decay=0.0, ws=None, stream=None):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    hp = pt_sgd_hparams(lam, lr, momentum, weight_decay)
    p, n = _ws(ws)
    _check(lib().pt_group_lasso_sgd_apply(ctx.handle, arr, len(arr), byref(hp), p, n, _stream(stream)), "pt_group_lasso_sgd_apply")


def pt_group_lasso_sgd_apply_layers(ctx, layers, first, count, lam, lr, momentum, weight_decay=0.0, ws=None, stream=None):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    hp = pt_sgd_hparams(lam, lr, momentum, weight_decay)
    p, n = _ws(ws)
    _check(lib().pt_group_lasso_sgd_apply_layers(ctx.handle, arr, len(arr), first, count, byref(hp), p, n, _stream(stream)),
           "pt_group_lasso_sgd_apply_layers")


def pt_find_zero_groups(ctx, layers, threshold=1e-4, zero_in_place=False, ws=None, stream=None):
    arr = layers if not isinstance(layers, (list, tuple)) else layer_array(layers)
    p, n = _ws(ws)
    _check(lib().pt_find_zero_groups(ctx.handle, arr, len(arr), threshold, int(bool(zero_in_place)), p, n, _stream(stream)),
           "pt_find_zero_groups")


def pt_find_zero_groups_noalloc(w, K, C, RS, threshold, zero_out, zero_in, stream=None):
    """Detection of one weight tensor with the library's static scratch: for callers that cannot allocate a workspace."""
    _check(lib().pt_find_zero_groups_noalloc(_ptr(w), K, C, RS, threshold, _ptr(zero_out), _ptr(zero_in), _stream(stream)),
           "pt_find_zero_groups_noalloc")


def make_bn_desc(N, H, W, C, ld=None, eps=1e-5, momentum=0.1, relu=True) -> pt_bn_desc:
    return pt_bn_desc(N, H, W, C, ld or (C + 7) // 8 * 8, eps, momentum, int(bool(relu)))


def pt_bn_workspace_bytes(ctx, d: pt_bn_desc) -> int:
    return int(lib().pt_bn_workspace_bytes(ctx.handle, byref(d)))


def pt_bn_relu_fwd(ctx, d, x, residual, gamma, beta, running_mean, running_var, save_mean, save_invstd, y, ws, stream=None):
    p, n = _ws(ws)
    _check(lib().pt_bn_relu_fwd(ctx.handle, byref(d), _ptr(x), _ptr(residual), _ptr(gamma), _ptr(beta), _ptr(running_mean),
                                _ptr(running_var), _ptr(save_mean), _ptr(save_invstd), _ptr(y), p, n, _stream(stream)),
           "pt_bn_relu_fwd")


def pt_bn_relu_bwd(ctx, d, x, y, dy, gamma, save_mean, save_invstd, dx, dresidual, dgamma, dbeta, ws, stream=None):
    p, n = _ws(ws)
    _check(lib().pt_bn_relu_bwd(ctx.handle, byref(d), _ptr(x), _ptr(y), _ptr(dy), _ptr(gamma), _ptr(save_mean), _ptr(save_invstd),
                                _ptr(dx), _ptr(dresidual), _ptr(dgamma), _ptr(dbeta), p, n, _stream(stream)), "pt_bn_relu_bwd")


def make_pool_desc(N, H, W, C, ld=None, R=3, stride=2, pad=1) -> pt_pool_desc:
    return pt_pool_desc(N, H, W, C, ld or (C + 7) // 8 * 8, R, stride, pad)


def pt_maxpool_fwd(ctx, d, x, y, stream=None, index=None):
    _check(lib().pt_maxpool_fwd(ctx.handle, byref(d), _ptr(x), _ptr(y), _ptr(index), _stream(stream)), "pt_maxpool_fwd")


def pt_maxpool_bwd(ctx, d, x, dy, dx, stream=None, index=None):
    _check(lib().pt_maxpool_bwd(ctx.handle, byref(d), _ptr(x), _ptr(dy), _ptr(index), _ptr(dx), _stream(stream)), "pt_maxpool_bwd")


def shape_array(shapes) -> "ctypes.Array":
    """shapes: iterable of (H, W, C, K, R, S, stride, pad)."""
    shapes = list(shapes)
    return (pt_layer_shape * len(shapes))(*[pt_layer_shape(*[int(v) for v in t]) for t in shapes])


def pt_training_memory_bytes(shapes, batch: int) -> int:
    arr = shape_array(shapes)
    return int(lib().pt_training_memory_bytes(arr, len(arr), batch))


def pt_update_mini_batch(shapes, capacity_bytes: int, cur_batch: int, cur_lr: float, granularity: int = 32):
    arr = shape_array(shapes)
    nb, nl = c_int32(), c_float()
    _check(lib().pt_update_mini_batch(arr, len(arr), capacity_bytes, cur_batch, cur_lr, granularity, byref(nb), byref(nl)),
           "pt_update_mini_batch")
    return nb.value, nl.value


def pt_cross_entropy_workspace_bytes(n: int) -> int:
    return int(lib().pt_cross_entropy_workspace_bytes(n))


def pt_cross_entropy(ctx, logits, labels, n, classes, ld, loss_out, ws, stream=None):
    p, nb = _ws(ws)
    _check(lib().pt_cross_entropy(ctx.handle, _ptr(logits), _ptr(labels), n, classes, ld, _ptr(loss_out), p, nb, _stream(stream)),
           "pt_cross_entropy")


def pt_conv_wgrad_ctas(ctx, d):
    """(CTAs of the weight-gradient launch at the current limit, whether they wait for one another)."""
    w = c_int32(0)
    n = int(lib().pt_conv_wgrad_ctas(ctx.handle, byref(d), byref(w)))
    return n, bool(w.value)


def pt_set_coeff(ctx, loss, reg_sum, ratio, lambda_out, stream=None):
    _check(lib().pt_set_coeff(ctx.handle, _ptr(loss), _ptr(reg_sum), ratio, _ptr(lambda_out), _stream(stream)), "pt_set_coeff")


def pt_dense_channel_list(ctx, zero_flags, n, idx, count, stream=None):
    _check(lib().pt_dense_channel_list(ctx.handle, _ptr(zero_flags), n, _ptr(idx), _ptr(count), _stream(stream)), "pt_dense_channel_list")


def pt_channel_gather(ctx, src, ld_src, c_src, idx, n_sel, dst, ld_dst, npix, stream=None):
    _check(lib().pt_channel_gather(ctx.handle, _ptr(src), ld_src, c_src, _ptr(idx), n_sel, _ptr(dst), ld_dst, npix, _stream(stream)),
           "pt_channel_gather")


def pt_channel_scatter_add(ctx, branch, ld_branch, idx, n_sel, node_in, node_out, ld_node, c_node, npix, relu, stream=None):
    _check(lib().pt_channel_scatter_add(ctx.handle, _ptr(branch), ld_branch, _ptr(idx), n_sel, _ptr(node_in),
                                        _ptr(node_out), ld_node, c_node, npix, 1 if relu else 0, _stream(stream)), "pt_channel_scatter_add")


class GraphHandle:
    """Keeps the ctypes arrays of a pt_graph alive."""

    def __init__(self, sizes: Sequence[int], fixed: Sequence[bool], layers: Sequence[pt_layer],
                 links: Sequence[tuple], bn: Optional[Sequence[Optional[Sequence]]] = None):
        self.spaces = (pt_space * len(sizes))(*[pt_space(int(s), int(bool(f))) for s, f in zip(sizes, fixed)])
        self.layers = layer_array(layers)
        lk = []
        for i, (isp, osp) in enumerate(links):
            ptrs = (c_void_p * 4)()
            if bn is not None and bn[i] is not None:
                for b in range(4):
                    ptrs[b] = _ptr(bn[i][b])
            lk.append(pt_layer_link(isp, osp, ptrs))
        self.links = (pt_layer_link * len(lk))(*lk)
        self.graph = pt_graph(self.spaces, len(sizes), self.layers, self.links, len(lk))


def pt_reconfigure_plan(ctx, graph: GraphHandle, new2old, stream=None) -> List[int]:
    n = graph.graph.n_spaces
    sizes = (c_int32 * n)()
    _check(lib().pt_reconfigure_plan(ctx.handle, byref(graph.graph), _ptr(new2old), sizes, _stream(stream)),
           "pt_reconfigure_plan")
    return list(sizes)


def pt_reconfigure(ctx, old: GraphHandle, new2old, new: GraphHandle, stream=None):
    _check(lib().pt_reconfigure(ctx.handle, byref(old.graph), _ptr(new2old), byref(new.graph), _stream(stream)),
           "pt_reconfigure")
