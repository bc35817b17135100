"""ctypes binding of libcat_loss.so: argument marshalling only.

Each function has the name and the arguments of its C entry point (include/cat_loss.h).
torch is used for device memory and streams; every step of the path runs in the library's
own kernels.  There is no fallback: if the library is missing or a call fails, this raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

CAT_BF16, CAT_F32 = 0, 1
CAT_WEIGHT_CONFIDENCE, CAT_WEIGHT_FIXED_DECAY = 0, 1
CAT_OK = 0


class cat_shape(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int64), ("d", ctypes.c_int64), ("V", ctypes.c_int64), ("K", ctypes.c_int32),
                ("in_dtype", ctypes.c_int32), ("dW_dtype", ctypes.c_int32), ("slab_mib", ctypes.c_int32),
                ("ldH", ctypes.c_int64), ("ldW", ctypes.c_int64), ("weight_mode", ctypes.c_int32),
                ("decay_gamma", ctypes.c_float)]


class cat_stats(ctypes.Structure):
    _fields_ = [("n_valid", ctypes.c_int64), ("n_bad_labels", ctypes.c_int64), ("sum_weight", ctypes.c_float),
                ("est_accept_len", ctypes.c_float), ("device_status", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class cat_kd_desc(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int64), ("d_t", ctypes.c_int64), ("ldHt", ctypes.c_int64), ("ldWt", ctypes.c_int64),
                ("beta", ctypes.c_float), ("conf_source", ctypes.c_int32)]


CAT_CONF_TARGET, CAT_CONF_DRAFT = 0, 1


class CatError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed: {code} ({cat_status_string(code)})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building first if the sources are newer) the shared library; raises if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = ctypes.CDLL(path)
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        L.cat_status_string.restype = ctypes.c_char_p
        L.cat_status_string.argtypes = [ctypes.c_int]
        L.cat_loss_workspace_bytes.restype = sz
        L.cat_loss_workspace_bytes.argtypes = [ctypes.POINTER(cat_shape), ctypes.c_int]
        L.cat_loss_launch_count.restype = ctypes.c_int
        L.cat_loss_launch_count.argtypes = [ctypes.POINTER(cat_shape), ctypes.c_int]
        L.cat_loss_fwd.restype = ctypes.c_int
        L.cat_loss_fwd.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 10 + [vp, sz, vp]
        L.cat_loss_fwd_static.restype = ctypes.c_int
        L.cat_loss_fwd_static.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 10 + [vp]
        L.cat_loss_fwd_bwd.restype = ctypes.c_int
        L.cat_loss_fwd_bwd.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 13 + [ctypes.c_int, vp, sz, vp]
        L.cat_loss_bwd.restype = ctypes.c_int
        L.cat_loss_bwd.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 9 + [ctypes.c_int, vp, sz, vp]
        L.cat_accept_len.restype = ctypes.c_int
        L.cat_accept_len.argtypes = [ctypes.POINTER(cat_shape), vp, vp, vp, vp]
        L.cat_conf_fwd.restype = ctypes.c_int
        L.cat_conf_fwd.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 6 + [vp, sz, vp]
        L.cat_conf_window.restype = ctypes.c_int
        L.cat_conf_window.argtypes = [vp, ctypes.c_int64, vp, ctypes.c_int64, ctypes.c_int32, vp, vp]
        L.cat_loss_fwd_bwd_events.restype = ctypes.c_int
        L.cat_loss_fwd_bwd_events.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 13 + [ctypes.c_int, vp, sz, vp, vp, ctypes.c_int]
        L.cat_loss_fused_slabs.restype = ctypes.c_int
        L.cat_loss_fused_slabs.argtypes = [ctypes.POINTER(cat_shape), vp, ctypes.c_int]
        L.cat_loss_bwd_events.restype = ctypes.c_int
        L.cat_loss_bwd_events.argtypes = [ctypes.POINTER(cat_shape)] + [vp] * 9 + [ctypes.c_int, vp, sz, vp, vp, ctypes.c_int]
        L.cat_loss_bwd_slabs.restype = ctypes.c_int
        L.cat_loss_bwd_slabs.argtypes = [ctypes.POINTER(cat_shape), vp, ctypes.c_int]
        L.cat_count_valid.restype = ctypes.c_int
        L.cat_count_valid.argtypes = [ctypes.POINTER(cat_shape), vp, vp, vp, vp]
        L.cat_kd_workspace_bytes.restype = sz
        L.cat_kd_workspace_bytes.argtypes = [ctypes.POINTER(cat_shape), ctypes.POINTER(cat_kd_desc), vp]
        L.cat_kd_loss_fwd_bwd.restype = ctypes.c_int
        L.cat_kd_loss_fwd_bwd.argtypes = [ctypes.POINTER(cat_shape), ctypes.POINTER(cat_kd_desc)] + [vp] * 16 + [ctypes.c_int, vp, sz, vp]
        L.cat_die_map.restype = ctypes.c_int
        L.cat_die_map.argtypes = [vp, ctypes.c_int, vp, vp]
        L.cat_selftest_wait_timeout.restype = ctypes.c_int
        L.cat_selftest_wait_timeout.argtypes = [ctypes.c_int, ctypes.c_uint64, ctypes.c_uint64, vp, vp, vp]
        _lib = L
    return _lib


def cat_status_string(code: int) -> str:
    return lib().cat_status_string(int(code)).decode()


def make_shape(T, d, V, K, in_dtype, dW_dtype=CAT_F32, ldH=None, ldW=None, slab_mib=0,
               weight_mode=CAT_WEIGHT_CONFIDENCE, decay_gamma=0.0) -> cat_shape:
    return cat_shape(T, d, V, K, in_dtype, dW_dtype, slab_mib, d if ldH is None else ldH, d if ldW is None else ldW,
                     weight_mode, decay_gamma)


def cat_loss_workspace_bytes(shape: cat_shape, which: int) -> int:
    return int(lib().cat_loss_workspace_bytes(ctypes.byref(shape), int(which)))


def cat_loss_launch_count(shape: cat_shape, which: int) -> int:
    return int(lib().cat_loss_launch_count(ctypes.byref(shape), int(which)))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def cat_loss_fwd(shape, H, W, labels, valid, conf_ext, loss, lse, conf, weight, stats, workspace) -> None:
    """All tensor arguments are CUDA tensors (or None where the C API allows NULL); outputs are written in place."""
    rc = lib().cat_loss_fwd(ctypes.byref(shape), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid), _ptr(conf_ext),
                            _ptr(loss), _ptr(lse), _ptr(conf), _ptr(weight), _ptr(stats),
                            _ptr(workspace), workspace.numel() * workspace.element_size() if workspace is not None else 0,
                            _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_loss_fwd")


CAT_STATIC_SCRATCH_BYTES = 32 << 20


def cat_loss_fwd_static(shape, H, W, labels, valid, conf_ext, loss, lse, conf, weight, stats) -> None:
    """Forward pass that takes no workspace: its scratch is an array built into the library
    (CAT_STATIC_SCRATCH_BYTES per GPU).  For callers that are not allowed to allocate device
    memory.  Calls share that array, so do not let two of them overlap on the GPU."""
    rc = lib().cat_loss_fwd_static(ctypes.byref(shape), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid), _ptr(conf_ext),
                                   _ptr(loss), _ptr(lse), _ptr(conf), _ptr(weight), _ptr(stats), _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_loss_fwd_static")


def cat_loss_bwd(shape, H, W, labels, valid, lse, weight, grad_loss, dH, dW, accumulate_dW, workspace) -> None:
    rc = lib().cat_loss_bwd(ctypes.byref(shape), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid), _ptr(lse), _ptr(weight),
                            _ptr(grad_loss), _ptr(dH), _ptr(dW), int(bool(accumulate_dW)),
                            _ptr(workspace), workspace.numel() * workspace.element_size() if workspace is not None else 0,
                            _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_loss_bwd")


def cat_loss_fwd_bwd(shape, H, W, labels, valid, conf_ext, grad_loss, loss, lse, conf, weight, stats, dH, dW,
                     accumulate_dW, workspace) -> None:
    rc = lib().cat_loss_fwd_bwd(ctypes.byref(shape), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid), _ptr(conf_ext),
                                _ptr(grad_loss), _ptr(loss), _ptr(lse), _ptr(conf), _ptr(weight), _ptr(stats),
                                _ptr(dH), _ptr(dW), int(bool(accumulate_dW)), _ptr(workspace),
                                workspace.numel() * workspace.element_size() if workspace is not None else 0, _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_loss_fwd_bwd")


def cat_accept_len(shape, conf, weight, accept_len) -> None:
    rc = lib().cat_accept_len(ctypes.byref(shape), _ptr(conf), _ptr(weight), _ptr(accept_len), _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_accept_len")


def cat_conf_fwd(shape, Ht, Wt, labels, valid, conf_seq, lse_seq, workspace) -> None:
    rc = lib().cat_conf_fwd(ctypes.byref(shape), _ptr(Ht), _ptr(Wt), _ptr(labels), _ptr(valid), _ptr(conf_seq),
                            _ptr(lse_seq), _ptr(workspace),
                            workspace.numel() * workspace.element_size() if workspace is not None else 0, _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_conf_fwd")


def cat_conf_window(conf_seq, L, block_start, n_blocks, K, conf_ext) -> None:
    rc = lib().cat_conf_window(_ptr(conf_seq), int(L), _ptr(block_start), int(n_blocks), int(K), _ptr(conf_ext), _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_conf_window")


def cat_loss_fused_slabs(shape) -> list:
    """First row of every row slab of cat_loss_fwd_bwd, plus T at the end."""
    n = int(lib().cat_loss_fused_slabs(ctypes.byref(shape), None, 0))
    if n <= 0:
        raise ValueError("invalid shape for cat_loss_fwd_bwd slabs")
    arr = (ctypes.c_int64 * n)()
    lib().cat_loss_fused_slabs(ctypes.byref(shape), arr, n)
    return list(arr) + [int(shape.T)]


def _event_array(events):
    for e in events:          # torch creates the CUDA event lazily, on first record
        if getattr(e, "cuda_event", 0) == 0:
            e.record()
    return (ctypes.c_void_p * len(events))(*[ctypes.c_void_p(e.cuda_event) for e in events])


def cat_loss_fwd_bwd_events(shape, H, W, labels, valid, conf_ext, grad_loss, loss, lse, conf, weight, stats, dH, dW,
                            accumulate_dW, workspace, events) -> None:
    """cat_loss_fwd_bwd that records `events` (torch.cuda.Event with enable_timing=True, 6 per row slab + 3)
    between its stages."""
    arr = _event_array(events)
    rc = lib().cat_loss_fwd_bwd_events(ctypes.byref(shape), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid), _ptr(conf_ext),
                                       _ptr(grad_loss), _ptr(loss), _ptr(lse), _ptr(conf), _ptr(weight), _ptr(stats),
                                       _ptr(dH), _ptr(dW), int(bool(accumulate_dW)), _ptr(workspace),
                                       workspace.numel() * workspace.element_size() if workspace is not None else 0, _stream(),
                                       arr, len(events))
    if rc != CAT_OK:
        raise CatError(rc, "cat_loss_fwd_bwd_events")


def cat_loss_bwd_slabs(shape) -> list:
    """First vocabulary row of every slab of cat_loss_bwd, plus V at the end."""
    n = int(lib().cat_loss_bwd_slabs(ctypes.byref(shape), None, 0))
    if n <= 0:
        raise ValueError("invalid shape for cat_loss_bwd")
    arr = (ctypes.c_int64 * n)()
    lib().cat_loss_bwd_slabs(ctypes.byref(shape), arr, n)
    return list(arr) + [int(shape.V)]


def cat_loss_bwd_events(shape, H, W, labels, valid, lse, weight, grad_loss, dH, dW, accumulate_dW, workspace, events) -> None:
    """`events`: list of torch.cuda.Event, one per vocabulary slab; event i is recorded once rows
    [slabs[i], slabs[i+1]) of dW are final."""
    arr = _event_array(events)
    rc = lib().cat_loss_bwd_events(ctypes.byref(shape), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid), _ptr(lse), _ptr(weight),
                                   _ptr(grad_loss), _ptr(dH), _ptr(dW), int(bool(accumulate_dW)), _ptr(workspace),
                                   workspace.numel() * workspace.element_size() if workspace is not None else 0, _stream(),
                                   arr, len(events))
    if rc != CAT_OK:
        raise CatError(rc, "cat_loss_bwd_events")


def cat_count_valid(shape, labels, valid, n_valid) -> None:
    rc = lib().cat_count_valid(ctypes.byref(shape), _ptr(labels), _ptr(valid), _ptr(n_valid), _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_count_valid")


def make_kd_desc(L, d_t, beta, conf_source=CAT_CONF_TARGET, ldHt=None, ldWt=None) -> cat_kd_desc:
    return cat_kd_desc(L, d_t, d_t if ldHt is None else ldHt, d_t if ldWt is None else ldWt, beta, conf_source)


def _host_i64(t):
    """Host pointer of a contiguous int64 CPU tensor (block starts are read on the host)."""
    if t.device.type != "cpu" or t.dtype != torch.int64 or not t.is_contiguous():
        raise TypeError("block_start must be a contiguous int64 CPU tensor")
    return ctypes.c_void_p(t.data_ptr())


def cat_kd_workspace_bytes(shape, desc, block_start_host) -> int:
    return int(lib().cat_kd_workspace_bytes(ctypes.byref(shape), ctypes.byref(desc), _host_i64(block_start_host)))


def cat_kd_loss_fwd_bwd(shape, desc, H, W, labels, valid, Ht, Wt, block_start_host, conf_ext, grad_loss, loss, lse, conf,
                        weight, stats, dH, dW, accumulate_dW, workspace) -> None:
    rc = lib().cat_kd_loss_fwd_bwd(ctypes.byref(shape), ctypes.byref(desc), _ptr(H), _ptr(W), _ptr(labels), _ptr(valid),
                                   _ptr(Ht), _ptr(Wt), _host_i64(block_start_host), _ptr(conf_ext), _ptr(grad_loss),
                                   _ptr(loss), _ptr(lse), _ptr(conf), _ptr(weight), _ptr(stats), _ptr(dH), _ptr(dW),
                                   int(bool(accumulate_dW)), _ptr(workspace),
                                   workspace.numel() * workspace.element_size() if workspace is not None else 0, _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_kd_loss_fwd_bwd")


def cat_die_map():
    """(worker_of_tpc list, TPCs on the die of SM 0) as measured on the current device, or ([], 0) when the
    measurement could not be used.  Waits for the current stream."""
    arr = (ctypes.c_int32 * 128)()
    n0 = ctypes.c_int32(0)
    n = lib().cat_die_map(arr, 128, ctypes.byref(n0), _stream())
    if n < 0:
        raise CatError(n, "cat_die_map")
    return list(arr[:n]), int(n0.value)


def cat_selftest_wait_timeout(role: int, short_ns: int, long_ns: int, status, elapsed_ns) -> None:
    """Runs the kernels' time-out path on purpose (a bounded wait that nothing satisfies);
    `status` int32[1] and `elapsed_ns` int64[12] are CUDA tensors written by the kernel."""
    rc = lib().cat_selftest_wait_timeout(int(role), int(short_ns), int(long_ns), _ptr(status), _ptr(elapsed_ns), _stream())
    if rc != CAT_OK:
        raise CatError(rc, "cat_selftest_wait_timeout")


def read_stats(stats_tensor: torch.Tensor) -> cat_stats:
    """Copy a 32-byte device cat_stats (a uint8[32] tensor) to the host."""
    raw = bytes(stats_tensor.cpu().numpy().tobytes())
    return cat_stats.from_buffer_copy(raw)
