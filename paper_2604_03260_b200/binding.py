"""ctypes binding of libfocus_b200.so: same names as the C ABI (include/focus.h), argument
marshalling only.  torch supplies device memory and the current stream; every step of the path
runs inside the library's CUDA kernels.  There is no CPU fallback: loading fails loudly when the
library has not been built (``python -m paper_2604_03260_b200.build``)."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfocus_b200.so")

FOCUS_LAYOUT_ORIGINAL = 0
FOCUS_LAYOUT_CLASS_SORTED = 1
FOCUS_LAYOUT_AUTO = 2
FOCUS_LAYOUT_SORTED_LOCAL = 3
FOCUS_LAYOUT_GROUP_MAJOR = 4
FOCUS_MAX_CLASSES = 64


class focus_shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("n", C.c_int32), ("D", C.c_int32),
                ("K", C.c_int32), ("topk", C.c_int32), ("window", C.c_int32), ("scale", C.c_float),
                ("softcap", C.c_float)]


class focus_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_n", C.c_int64)]


class focus_tiles_layout(C.Structure):
    _fields_ = [("layout", C.c_int32), ("nqt", C.c_int32), ("nkt", C.c_int32), ("nkw", C.c_int32),
                ("total_bytes", C.c_size_t), ("counters", C.c_size_t),
                ("orq", C.c_size_t), ("andq", C.c_size_t), ("ork", C.c_size_t), ("andk", C.c_size_t),
                ("gbits", C.c_size_t), ("live", C.c_size_t), ("live_cnt", C.c_size_t),
                ("kany", C.c_size_t), ("kall", C.c_size_t),
                ("nqp", C.c_int32), ("nkp", C.c_int32),
                ("ncls_q", C.c_size_t), ("ncls_k", C.c_size_t), ("cls_q", C.c_size_t), ("cls_k", C.c_size_t),
                ("cnt_q", C.c_size_t), ("cnt_k", C.c_size_t),
                ("seg_q", C.c_size_t), ("seg_k", C.c_size_t), ("perm_q", C.c_size_t), ("perm_k", C.c_size_t),
                ("qrange", C.c_size_t), ("order", C.c_size_t), ("gbits_s", C.c_size_t), ("qs", C.c_size_t), ("ks", C.c_size_t),
                ("vs", C.c_size_t), ("scratch", C.c_size_t), ("o_sorted", C.c_size_t), ("o_local", C.c_size_t),
                ("lse_local", C.c_size_t)]


class FocusError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"focus status {status}: {message}")
        self.status = status


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_03260_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
        SP = C.POINTER(focus_shape)
        L.focus_version.restype = C.c_int
        L.focus_status_string.restype = C.c_char_p
        L.focus_status_string.argtypes = [C.c_int]
        L.focus_last_error.restype = C.c_char_p
        L.focus_assign.restype = C.c_int
        L.focus_assign.argtypes = [SP, focus_tensor, i32, vp, vp, vp, f32, vp]
        L.focus_assign_hidden.restype = C.c_int
        L.focus_assign_hidden.argtypes = [SP, vp, C.c_int64, C.c_int64, i32, i32, vp, vp, vp, vp, vp, vp, vp, f32, vp]
        L.focus_tiles_layout_of.restype = C.c_int
        L.focus_tiles_layout_of.argtypes = [SP, i32, C.POINTER(focus_tiles_layout)]
        L.focus_tiles_workspace_bytes.restype = sz
        L.focus_tiles_workspace_bytes.argtypes = [SP, i32]
        L.focus_build_tiles.restype = C.c_int
        L.focus_build_tiles.argtypes = [SP, vp, vp, i32, vp, sz, vp]
        L.focus_attn_fwd.restype = C.c_int
        L.focus_attn_fwd.argtypes = [SP, focus_tensor, focus_tensor, focus_tensor, vp, vp, vp, i32, focus_tensor, vp,
                                     vp, vp]
        L.focus_decode_workspace_bytes.restype = sz
        L.focus_decode_workspace_bytes.argtypes = [SP]
        L.focus_decode_step.restype = C.c_int
        L.focus_decode_step.argtypes = [SP, focus_tensor, focus_tensor, focus_tensor, vp, vp, focus_tensor, vp, vp, sz, vp]
        L.focus_router_scores.restype = C.c_int
        L.focus_router_scores.argtypes = [SP, vp, C.c_int64, C.c_int64, i32, i32, vp, vp, vp, vp, vp]
        L.focus_soft_ld.restype = i32
        L.focus_soft_ld.argtypes = [i32]
        L.focus_sinkhorn_workspace_bytes.restype = sz
        L.focus_sinkhorn_workspace_bytes.argtypes = [SP, i32]
        L.focus_sinkhorn.restype = C.c_int
        L.focus_sinkhorn.argtypes = [SP, vp, f32, i32, vp, sz, vp, vp]
        L.focus_sinkhorn_bwd_workspace_bytes.restype = sz
        L.focus_sinkhorn_bwd_workspace_bytes.argtypes = [SP, i32]
        L.focus_sinkhorn_bwd.restype = C.c_int
        L.focus_sinkhorn_bwd.argtypes = [SP, vp, f32, i32, vp, sz, vp, vp, vp]
        L.focus_gate_attn_fwd.restype = C.c_int
        L.focus_gate_attn_fwd.argtypes = [SP, focus_tensor, focus_tensor, focus_tensor, vp, f32, focus_tensor, vp, vp, vp]
        L.focus_count_kept.restype = C.c_int
        L.focus_count_kept.argtypes = [SP, vp, vp, vp, vp]
        L.focus_count_kept_noalloc.restype = C.c_int
        L.focus_count_kept_noalloc.argtypes = [SP, vp, vp, vp, vp]
        L.focus_selftest_umma.restype = C.c_int
        L.focus_selftest_umma.argtypes = [i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.focus_selftest_umma_pair.restype = C.c_int
        L.focus_selftest_umma_pair.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
        L.focus_selftest_mma_rate.restype = C.c_int
        L.focus_selftest_mma_rate.argtypes = [i32, i32, i32, i32, i32, vp, vp]
        L.focus_selftest_stalled_wait.restype = C.c_int
        L.focus_selftest_stalled_wait.argtypes = [SP, focus_tensor, focus_tensor, focus_tensor, focus_tensor, vp, C.c_uint64, vp, vp]
        _lib = L
    return _lib


def _check(rc):
    if rc != 0:
        raise FocusError(rc, lib().focus_last_error().decode())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _p(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def make_shape(Hq, Hkv, n, D, K, topk, window, scale=0.0, softcap=0.0, batch=1) -> focus_shape:
    return focus_shape(batch, Hq, Hkv, n, D, K, topk, window, scale, softcap)


def shape_of(wl) -> focus_shape:
    """focus_shape of an inputs.Workload"""
    return make_shape(wl.Hq, wl.Hkv, wl.n, wl.D, wl.K, wl.topk, wl.window, wl.scale, wl.softcap)


def tensor_arg(t: torch.Tensor) -> focus_tensor:
    """[H, n, D] or [batch, H, n, D] bf16 CUDA tensor with D contiguous"""
    assert t.is_cuda and t.dtype == torch.bfloat16 and t.stride(-1) == 1
    if t.dim() == 3:
        return focus_tensor(t.data_ptr(), t.stride(0) * t.shape[0], t.stride(0), t.stride(1))
    assert t.dim() == 4
    return focus_tensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def focus_version() -> int:
    return lib().focus_version()


def focus_assign(shape, x, H, centroids, masks_out, near_ties=None, near_tie_eps=1e-5, stream=None):
    _check(lib().focus_assign(C.byref(shape), tensor_arg(x), H, _p(centroids), _p(masks_out), _p(near_ties),
                              near_tie_eps, _stream(stream)))


def focus_assign_hidden(shape, h, Wg, Cg, bias, folded, mq_out, mk_out, near_ties=None, near_tie_eps=1e-5, stream=None):
    """h bf16 [batch, n, d_model] (or [n, d_model]); Wg fp32 [d_model, d_g]; Cg fp32 [K, d_g]; folded fp32 [K, d_model] scratch"""
    assert h.is_cuda and h.dtype == torch.bfloat16 and h.stride(-1) == 1
    sb, sn = (h.stride(0), h.stride(1)) if h.dim() == 3 else (h.stride(0) * h.shape[0], h.stride(0))
    _check(lib().focus_assign_hidden(C.byref(shape), _p(h), sb, sn, h.shape[-1], Wg.shape[1], _p(Wg), _p(Cg), _p(bias),
                                     _p(folded), _p(mq_out), _p(mk_out), _p(near_ties), near_tie_eps, _stream(stream)))


def focus_tiles_layout_of(shape, layout) -> focus_tiles_layout:
    out = focus_tiles_layout()
    _check(lib().focus_tiles_layout_of(C.byref(shape), layout, C.byref(out)))
    return out


def focus_tiles_workspace_bytes(shape, layout) -> int:
    return int(lib().focus_tiles_workspace_bytes(C.byref(shape), layout))


def focus_build_tiles(shape, mq, mk, layout, ws, stream=None):
    _check(lib().focus_build_tiles(C.byref(shape), _p(mq), _p(mk), layout, _p(ws), ws.numel() * ws.element_size(),
                                   _stream(stream)))


def focus_attn_fwd(shape, q, k, v, mq, mk, tiles_ws, layout, o, lse, dev_status=None, stream=None):
    _check(lib().focus_attn_fwd(C.byref(shape), tensor_arg(q), tensor_arg(k), tensor_arg(v), _p(mq), _p(mk),
                                _p(tiles_ws), layout, tensor_arg(o), _p(lse), _p(dev_status), _stream(stream)))


def focus_decode_workspace_bytes(shape) -> int:
    return int(lib().focus_decode_workspace_bytes(C.byref(shape)))


def focus_decode_step(shape, q, k, v, mq_new, mk, o, lse, ws, stream=None):
    """q, o bf16 [Hq, D] (or [batch, Hq, D]); k, v bf16 caches [Hkv, n, D]; mq_new int32 [batch*Hq]; mk int32 [batch*Hkv, n]"""
    def vec_arg(t):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.stride(-1) == 1
        if t.dim() == 2:
            return focus_tensor(t.data_ptr(), t.stride(0) * t.shape[0], t.stride(0), t.shape[-1])
        return focus_tensor(t.data_ptr(), t.stride(0), t.stride(1), t.shape[-1])
    _check(lib().focus_decode_step(C.byref(shape), vec_arg(q), tensor_arg(k), tensor_arg(v), _p(mq_new), _p(mk), vec_arg(o),
                                   _p(lse), _p(ws), ws.numel() * ws.element_size(), _stream(stream)))


def focus_soft_ld(K) -> int:
    return int(lib().focus_soft_ld(K))


def focus_router_scores(shape, h, Wg, Cg, folded, scores_out, stream=None):
    """h bf16 [batch, n, d_model] (or [n, d_model]); scores_out fp32 [batch, n, focus_soft_ld(K)]"""
    assert h.is_cuda and h.dtype == torch.bfloat16 and h.stride(-1) == 1
    sb, sn = (h.stride(0), h.stride(1)) if h.dim() == 3 else (h.stride(0) * h.shape[0], h.stride(0))
    _check(lib().focus_router_scores(C.byref(shape), _p(h), sb, sn, h.shape[-1], Wg.shape[1], _p(Wg), _p(Cg), _p(folded),
                                     _p(scores_out), _stream(stream)))


def focus_sinkhorn_workspace_bytes(shape, iters) -> int:
    return int(lib().focus_sinkhorn_workspace_bytes(C.byref(shape), iters))


def focus_sinkhorn(shape, scores, tau, iters, ws, g_out, stream=None):
    """scores, g_out fp32 [batch, n, focus_soft_ld(K)] (may be the same tensor); ws uint8 scratch"""
    _check(lib().focus_sinkhorn(C.byref(shape), _p(scores), tau, iters, _p(ws), ws.numel() * ws.element_size(), _p(g_out),
                                _stream(stream)))


def focus_sinkhorn_bwd_workspace_bytes(shape, iters) -> int:
    return int(lib().focus_sinkhorn_bwd_workspace_bytes(C.byref(shape), iters))


def focus_sinkhorn_bwd(shape, scores, tau, iters, ws, dg, dscores_out, stream=None):
    """scores, dg, dscores_out fp32 [batch, n, focus_soft_ld(K)] (dscores_out may be dg); ws uint8 scratch"""
    _check(lib().focus_sinkhorn_bwd(C.byref(shape), _p(scores), tau, iters, _p(ws), ws.numel() * ws.element_size(), _p(dg),
                                    _p(dscores_out), _stream(stream)))


def focus_gate_attn_fwd(shape, q, k, v, g, lam, o, lse, dev_status=None, stream=None):
    """training-time gated forward; g fp32 [batch, n, focus_soft_ld(K)]"""
    _check(lib().focus_gate_attn_fwd(C.byref(shape), tensor_arg(q), tensor_arg(k), tensor_arg(v), _p(g), lam, tensor_arg(o),
                                     _p(lse), _p(dev_status), _stream(stream)))


def focus_count_kept(shape, mq, tiles_ws, counts_out, stream=None):
    _check(lib().focus_count_kept(C.byref(shape), _p(mq), _p(tiles_ws), _p(counts_out), _stream(stream)))


def focus_count_kept_noalloc(shape, mq, mk, counts_out, stream=None):
    """focus_count_kept for callers that may not allocate: the group bitmaps go to an array built into the
    library (at most 1 MiB: batch*Hkv*ceil(n/128)*K*16 bytes), no workspace argument."""
    _check(lib().focus_count_kept_noalloc(C.byref(shape), _p(mq), _p(mk), _p(counts_out), _stream(stream)))


def focus_selftest_umma(D, a, b, p, v, s_out, o_out, dev_status, stream=None):
    _check(lib().focus_selftest_umma(D, _p(a), _p(b), _p(p), _p(v), _p(s_out), _p(o_out), _p(dev_status),
                                     _stream(stream)))


def focus_selftest_umma_pair(a, b, p, v, s_out, o_out, dev_status, stream=None):
    _check(lib().focus_selftest_umma_pair(_p(a), _p(b), _p(p), _p(v), _p(s_out), _p(o_out), _p(dev_status), _stream(stream)))


def focus_selftest_mma_rate(pair, N, ts, pattern, rounds, result, stream=None):
    """result: int64 device tensor of 3 words (cycles, nanoseconds, fault flag)"""
    _check(lib().focus_selftest_mma_rate(pair, N, ts, pattern, rounds, _p(result), _stream(stream)))


def focus_selftest_stalled_wait(shape, q, k, v, o, lse, wait_limit_ns, dev_status, stream=None):
    _check(lib().focus_selftest_stalled_wait(C.byref(shape), tensor_arg(q), tensor_arg(k), tensor_arg(v), tensor_arg(o), _p(lse),
                                             wait_limit_ns, _p(dev_status), _stream(stream)))


def alloc_workspace(shape, layout, device="cuda") -> torch.Tensor:
    """uint8 device buffer of focus_tiles_workspace_bytes (torch allocations are 256-byte aligned)"""
    nbytes = focus_tiles_workspace_bytes(shape, layout)
    if nbytes == 0:
        raise FocusError(-1, lib().focus_last_error().decode())
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def ws_view(ws: torch.Tensor, offset: int, count: int, dtype) -> torch.Tensor:
    """typed view of `count` elements at byte `offset` of a workspace"""
    size = torch.empty((), dtype=dtype).element_size()
    return ws[offset:offset + count * size].view(dtype)
