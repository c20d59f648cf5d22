"""ctypes binding over libswimba.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/swimba.h).  Tensors are
torch CUDA tensors used purely as device memory; every step of the path runs inside the library's
kernels.  There is no fallback: if the library is missing, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libswimba.so")

OK = 0
ERR_NULL_ARG = -1
ERR_BAD_CONFIG = -2
ERR_UNSUPPORTED_SHAPE = -3
ERR_MISALIGNED = -4
ERR_WORKSPACE_TOO_SMALL = -5
ERR_CUDA = -6
ERR_DEVICE_TIMEOUT = -7
ERR_DEVICE_BOUNDS = -8
DTYPE_FP32 = 0
DTYPE_BF16 = 1
FLAG_CHECK_INDICES = 1

EXPORTS = [
    "swimba_create", "swimba_workspace_bytes", "swimba_ssd_segments", "swimba_forward", "swimba_route_mix", "swimba_ssd",
    "swimba_packed_workspace_bytes", "swimba_packed_segments", "swimba_forward_packed",
    "swimba_shard_workspace_bytes", "swimba_shard_summary", "swimba_shard_finish",
    "swimba_backward_workspace_bytes", "swimba_backward_weights",
    "swimba_route_project_slots", "swimba_ssd_slots_workspace_bytes", "swimba_ssd_slots",
    "swimba_block_workspace_bytes", "swimba_block_forward",
    "swimba_decode_workspace_bytes", "swimba_decode_step", "swimba_host_workspace_bytes",
    "swimba_forward_host", "swimba_route_mix_static", "swimba_profile", "swimba_profile_read",
    "swimba_selftest_wait", "swimba_last_launch_count", "swimba_status", "swimba_last_error",
    "swimba_destroy",
]


class SwimbaError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"swimba error {code}: {msg}")
        self.code = code


class swimba_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "d_model", "n_heads", "head_dim", "d_state", "n_groups", "n_experts", "top_k", "chunk",
        "dtype", "flags")]


class swimba_weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("W_router", "W_expert", "A", "dt_bias", "D")]


class swimba_block_weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("W_in", "conv_w", "conv_b", "norm_w", "W_out")] + \
               [("d_conv", ctypes.c_int32), ("eps", ctypes.c_float)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libswimba.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2603_06938_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.swimba_create.argtypes = [ctypes.POINTER(swimba_config), ctypes.POINTER(vp)]
        L.swimba_create.restype = ctypes.c_int
        L.swimba_workspace_bytes.argtypes = [vp, i32, i32]
        L.swimba_workspace_bytes.restype = sz
        L.swimba_ssd_segments.argtypes = [vp, i32, i32]
        L.swimba_ssd_segments.restype = i32
        L.swimba_decode_workspace_bytes.argtypes = [vp, i32]
        L.swimba_decode_workspace_bytes.restype = sz
        L.swimba_host_workspace_bytes.argtypes = [vp, i32, i32]
        L.swimba_host_workspace_bytes.restype = sz
        L.swimba_forward.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp, i32, i32,
                                     vp, vp, vp, vp, vp, sz, vp]
        L.swimba_forward.restype = ctypes.c_int
        L.swimba_packed_workspace_bytes.argtypes = [vp, ctypes.POINTER(i32), i32]
        L.swimba_packed_workspace_bytes.restype = sz
        L.swimba_packed_segments.argtypes = [vp, ctypes.POINTER(i32), i32]
        L.swimba_packed_segments.restype = i32
        L.swimba_forward_packed.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp,
                                            ctypes.POINTER(i32), i32, vp, vp, vp, vp, vp, sz, vp]
        L.swimba_forward_packed.restype = ctypes.c_int
        L.swimba_backward_workspace_bytes.argtypes = [vp, i32, i32]
        L.swimba_backward_workspace_bytes.restype = sz
        L.swimba_backward_weights.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp, vp, i32, i32,
                                              vp, vp, vp, vp, sz, vp]
        L.swimba_backward_weights.restype = ctypes.c_int
        L.swimba_shard_workspace_bytes.argtypes = [vp, i32, i32]
        L.swimba_shard_workspace_bytes.restype = sz
        L.swimba_shard_summary.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, i32, i32, vp, vp,
                                           vp, vp, vp, sz, vp]
        L.swimba_shard_summary.restype = ctypes.c_int
        L.swimba_shard_finish.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp, i32, i32, i32,
                                          i32, vp, vp, vp, sz, vp]
        L.swimba_shard_finish.restype = ctypes.c_int
        L.swimba_route_mix.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, i64, vp, vp, vp, vp,
                                       sz, vp]
        L.swimba_route_mix.restype = ctypes.c_int
        L.swimba_ssd.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp, i32, i32, vp,
                                 vp, vp, sz, vp]
        L.swimba_ssd.restype = ctypes.c_int
        L.swimba_route_project_slots.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, i64, vp, vp, vp,
                                                 vp, sz, vp]
        L.swimba_route_project_slots.restype = ctypes.c_int
        L.swimba_ssd_slots_workspace_bytes.argtypes = [vp, i32, i32]
        L.swimba_ssd_slots_workspace_bytes.restype = sz
        L.swimba_ssd_slots.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp, i32, i32, vp,
                                       vp, vp, sz, vp]
        L.swimba_ssd_slots.restype = ctypes.c_int
        L.swimba_block_workspace_bytes.argtypes = [vp, i32, i32]
        L.swimba_block_workspace_bytes.restype = sz
        L.swimba_block_forward.argtypes = [vp, ctypes.POINTER(swimba_weights), ctypes.POINTER(swimba_block_weights),
                                           vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.swimba_block_forward.restype = ctypes.c_int
        L.swimba_decode_step.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, vp, i32,
                                         vp, vp, vp, vp, sz, vp]
        L.swimba_decode_step.restype = ctypes.c_int
        L.swimba_forward_host.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, vp, vp, i32, i32,
                                          vp, vp, vp, vp, vp, sz, vp]
        L.swimba_forward_host.restype = ctypes.c_int
        L.swimba_route_mix_static.argtypes = [vp, ctypes.POINTER(swimba_weights), vp, i64, vp, vp, vp,
                                              vp]
        L.swimba_route_mix_static.restype = ctypes.c_int
        L.swimba_profile.argtypes = [vp, ctypes.c_int]
        L.swimba_profile.restype = ctypes.c_int
        L.swimba_profile_read.argtypes = [vp, vp, vp, i32]
        L.swimba_profile_read.restype = ctypes.c_int
        L.swimba_selftest_wait.argtypes = [vp, i64, vp, vp]
        L.swimba_selftest_wait.restype = ctypes.c_int
        L.swimba_last_launch_count.argtypes = [vp]
        L.swimba_last_launch_count.restype = ctypes.c_int
        L.swimba_status.argtypes = [vp]
        L.swimba_status.restype = ctypes.c_int
        L.swimba_last_error.argtypes = [vp]
        L.swimba_last_error.restype = ctypes.c_char_p
        L.swimba_destroy.argtypes = [vp]
        L.swimba_destroy.restype = None
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


class Handle:
    """Owns one swimba_handle*; `cfg` mirrors the C configuration."""

    def __init__(self, ptr: ctypes.c_void_p, cfg: swimba_config):
        self.ptr = ptr
        self.cfg = cfg

    def _raise(self, code: int):
        msg = lib().swimba_last_error(self.ptr)
        raise SwimbaError(code, msg.decode() if msg else "")


def swimba_create(d_model: int, n_heads: int, head_dim: int, d_state: int, n_groups: int,
                  n_experts: int, top_k: int, chunk: int, dtype: int, flags: int = 0) -> Handle:
    cfg = swimba_config(d_model, n_heads, head_dim, d_state, n_groups, n_experts, top_k, chunk,
                        dtype, flags)
    out = ctypes.c_void_p()
    rc = lib().swimba_create(ctypes.byref(cfg), ctypes.byref(out))
    if rc != OK:
        raise SwimbaError(rc, "swimba_create rejected the configuration")
    return Handle(out, cfg)


def swimba_destroy(h: Handle) -> None:
    if h.ptr:
        lib().swimba_destroy(h.ptr)
        h.ptr = None


def make_weights(W_router, W_expert, A, dt_bias, D) -> swimba_weights:
    w = swimba_weights()
    w.W_router = W_router.data_ptr() if W_router is not None else None
    w.W_expert = W_expert.data_ptr() if W_expert is not None else None
    w.A = A.data_ptr() if A is not None else None
    w.dt_bias = dt_bias.data_ptr() if dt_bias is not None else None
    w.D = D.data_ptr() if D is not None else None
    w._keep = (W_router, W_expert, A, dt_bias, D)   # keep the tensors alive
    return w


def swimba_workspace_bytes(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_workspace_bytes(h.ptr, B, L))


def swimba_ssd_segments(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_ssd_segments(h.ptr, B, L))


def swimba_decode_workspace_bytes(h: Handle, B: int) -> int:
    return int(lib().swimba_decode_workspace_bytes(h.ptr, B))


def swimba_host_workspace_bytes(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_host_workspace_bytes(h.ptr, B, L))


def _ws(workspace: Optional[torch.Tensor]):
    if workspace is None:
        return None, 0
    return ctypes.c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size()


def swimba_forward(h: Handle, w: swimba_weights, u, x, dt, h0, B: int, L: int, y, h_final,
                   topk_idx, topk_w, workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_forward(h.ptr, ctypes.byref(w), _ptr(u), _ptr(x), _ptr(dt), _ptr(h0), B, L,
                              _ptr(y), _ptr(h_final), _ptr(topk_idx), _ptr(topk_w), wp, wb,
                              _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_backward_workspace_bytes(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_backward_workspace_bytes(h.ptr, B, L))


def swimba_backward_weights(h: Handle, w: swimba_weights, u, x, dt, h0, dy, B: int, L: int, dW_router,
                            dW_expert, topk_idx, workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_backward_weights(h.ptr, ctypes.byref(w), _ptr(u), _ptr(x), _ptr(dt), _ptr(h0), _ptr(dy),
                                       B, L, _ptr(dW_router), _ptr(dW_expert), _ptr(topk_idx), wp, wb,
                                       _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_shard_workspace_bytes(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_shard_workspace_bytes(h.ptr, B, L))


def swimba_shard_summary(h: Handle, w: swimba_weights, u, x, dt, B: int, L: int, summary_state,
                         summary_decay, topk_idx, topk_w, workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_shard_summary(h.ptr, ctypes.byref(w), _ptr(u), _ptr(x), _ptr(dt), B, L,
                                    _ptr(summary_state), _ptr(summary_decay), _ptr(topk_idx), _ptr(topk_w),
                                    wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_shard_finish(h: Handle, w: swimba_weights, x, h0, all_state, all_decay, rank: int, n_ranks: int,
                        B: int, L: int, y, h_end, workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_shard_finish(h.ptr, ctypes.byref(w), _ptr(x), _ptr(h0), _ptr(all_state),
                                   _ptr(all_decay), rank, n_ranks, B, L, _ptr(y), _ptr(h_end), wp, wb,
                                   _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def _offsets(cu_seqlens):
    """Host offsets (a sequence of ints) as a C array of nseq + 1 int32."""
    n = len(cu_seqlens)
    return (ctypes.c_int32 * n)(*[int(v) for v in cu_seqlens]), n - 1


def swimba_packed_workspace_bytes(h: Handle, cu_seqlens) -> int:
    arr, nseq = _offsets(cu_seqlens)
    return int(lib().swimba_packed_workspace_bytes(h.ptr, arr, nseq))


def swimba_packed_segments(h: Handle, cu_seqlens) -> int:
    arr, nseq = _offsets(cu_seqlens)
    return int(lib().swimba_packed_segments(h.ptr, arr, nseq))


def swimba_forward_packed(h: Handle, w: swimba_weights, u, x, dt, h0, cu_seqlens, y, h_final,
                          topk_idx, topk_w, workspace, stream=None, check: bool = True) -> int:
    arr, nseq = _offsets(cu_seqlens)
    wp, wb = _ws(workspace)
    rc = lib().swimba_forward_packed(h.ptr, ctypes.byref(w), _ptr(u), _ptr(x), _ptr(dt), _ptr(h0), arr,
                                     nseq, _ptr(y), _ptr(h_final), _ptr(topk_idx), _ptr(topk_w), wp, wb,
                                     _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_route_mix(h: Handle, w: swimba_weights, u, T: int, BC, topk_idx, topk_w, workspace,
                     stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_route_mix(h.ptr, ctypes.byref(w), _ptr(u), T, _ptr(BC), _ptr(topk_idx),
                                _ptr(topk_w), wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_route_mix_static(h: Handle, w: swimba_weights, u, T: int, BC, topk_idx, topk_w,
                            stream=None, check: bool = True) -> int:
    """swimba_route_mix without a workspace argument: for callers that cannot allocate device
    memory, the stage's scratch is a fixed array inside the library (8 MiB per GPU, shared by all
    calls on that GPU, so overlapping calls must be serialised; larger T is rejected)."""
    rc = lib().swimba_route_mix_static(h.ptr, ctypes.byref(w), _ptr(u), T, _ptr(BC),
                                       _ptr(topk_idx), _ptr(topk_w), _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_route_project_slots(h: Handle, w: swimba_weights, u, T: int, BC_slots, topk_idx, topk_w,
                               workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_route_project_slots(h.ptr, ctypes.byref(w), _ptr(u), T, _ptr(BC_slots),
                                          _ptr(topk_idx), _ptr(topk_w), wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_ssd_slots_workspace_bytes(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_ssd_slots_workspace_bytes(h.ptr, B, L))


def swimba_ssd_slots(h: Handle, w: swimba_weights, x_slots, BC_slots, dt, h0, B: int, L: int, y,
                     h_final, workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_ssd_slots(h.ptr, ctypes.byref(w), _ptr(x_slots), _ptr(BC_slots), _ptr(dt),
                                _ptr(h0), B, L, _ptr(y), _ptr(h_final), wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def make_block_weights(W_in, conv_w, conv_b, norm_w, W_out, d_conv: int, eps: float = 1e-5) -> swimba_block_weights:
    bw = swimba_block_weights()
    bw.W_in, bw.conv_w, bw.norm_w, bw.W_out = W_in.data_ptr(), conv_w.data_ptr(), norm_w.data_ptr(), W_out.data_ptr()
    bw.conv_b = conv_b.data_ptr() if conv_b is not None else None
    bw.d_conv, bw.eps = d_conv, eps
    bw._keep = (W_in, conv_w, conv_b, norm_w, W_out)
    return bw


def swimba_block_workspace_bytes(h: Handle, B: int, L: int) -> int:
    return int(lib().swimba_block_workspace_bytes(h.ptr, B, L))


def swimba_block_forward(h: Handle, w: swimba_weights, bw: swimba_block_weights, u, conv_state_in, h0,
                         B: int, L: int, out, conv_state_out, h_final, topk_idx, topk_w, workspace,
                         stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_block_forward(h.ptr, ctypes.byref(w), ctypes.byref(bw), _ptr(u), _ptr(conv_state_in),
                                    _ptr(h0), B, L, _ptr(out), _ptr(conv_state_out), _ptr(h_final),
                                    _ptr(topk_idx), _ptr(topk_w), wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_ssd(h: Handle, w: swimba_weights, x, BC, dt, h0, B: int, L: int, y, h_final, workspace,
               stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_ssd(h.ptr, ctypes.byref(w), _ptr(x), _ptr(BC), _ptr(dt), _ptr(h0), B, L,
                          _ptr(y), _ptr(h_final), wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_decode_step(h: Handle, w: swimba_weights, u, x, dt, state, B: int, y, topk_idx, topk_w,
                       workspace, stream=None, check: bool = True) -> int:
    wp, wb = _ws(workspace)
    rc = lib().swimba_decode_step(h.ptr, ctypes.byref(w), _ptr(u), _ptr(x), _ptr(dt), _ptr(state),
                                  B, _ptr(y), _ptr(topk_idx), _ptr(topk_w), wp, wb,
                                  _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


def swimba_forward_host(h: Handle, w: swimba_weights, u_host, x_host, dt_host, B: int, L: int,
                        y_host, h_final_host, topk_idx_host, topk_w_host, workspace, stream=None,
                        check: bool = True) -> int:
    """Host tensors (ideally pinned) in and out; the caller synchronises the stream."""
    wp, wb = _ws(workspace)
    rc = lib().swimba_forward_host(h.ptr, ctypes.byref(w), _ptr(u_host), _ptr(x_host),
                                   _ptr(dt_host), B, L, _ptr(y_host), _ptr(h_final_host),
                                   _ptr(topk_idx_host), _ptr(topk_w_host), wp, wb, _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc


KERNEL_NAMES = {1: "router_topk", 4: "expert_gemm",
                5: "mix_slots", 6: "project_mix_simt", 7: "ssd_sequential", 8: "decode_update",
                9: "ssd_tiles", 10: "segment_scan", 11: "ssd_scalars", 12: "slot_streams",
                13: "slot_sum", 14: "project_small", 15: "conv_silu", 16: "gated_rmsnorm",
                17: "dt_columns", 18: "ssd_adjoint", 19: "router_softmax", 20: "dpi_dg", 21: "dw_router",
                22: "dw_expert", 23: "adjoint_pack", 24: "ssd_state"}


def swimba_profile(h: Handle, enable: bool) -> None:
    rc = lib().swimba_profile(h.ptr, 1 if enable else 0)
    if rc != OK:
        h._raise(rc)


def swimba_profile_read(h: Handle):
    """[(kernel name, milliseconds)] of the kernels the most recent call launched."""
    ids = (ctypes.c_int32 * 64)()
    ms = (ctypes.c_float * 64)()
    n = lib().swimba_profile_read(h.ptr, ctypes.cast(ids, ctypes.c_void_p),
                                  ctypes.cast(ms, ctypes.c_void_p), 64)
    if n < 0:
        h._raise(n)
    return [(KERNEL_NAMES.get(ids[i], str(ids[i])), float(ms[i])) for i in range(n)]


def swimba_selftest_wait(h: Handle, limit_cycles: int, stream=None, check: bool = True):
    """Runs the bounded-wait self-test; returns (rc, [first gave up, second gave up, cycles])."""
    res = (ctypes.c_int64 * 3)()
    rc = lib().swimba_selftest_wait(h.ptr, limit_cycles, ctypes.cast(res, ctypes.c_void_p),
                                    _stream(stream))
    if check and rc != OK:
        h._raise(rc)
    return rc, [int(v) for v in res]


def swimba_last_launch_count(h: Handle) -> int:
    return int(lib().swimba_last_launch_count(h.ptr))


def swimba_status(h: Handle) -> int:
    return int(lib().swimba_status(h.ptr))


def swimba_last_error(h: Handle) -> str:
    msg = lib().swimba_last_error(h.ptr)
    return msg.decode() if msg else ""
