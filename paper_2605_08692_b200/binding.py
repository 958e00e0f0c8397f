"""ctypes binding of libaaac_b200.so.  Argument marshalling only.

Functions mirror the C entry points (see include/aaac.h for the meaning, layout and ownership
of every argument).  Tensors must live on the current CUDA device; work is enqueued on
``torch.cuda.current_stream()`` and is not synchronised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

INT4, NVFP4 = 0, 1
INIT_QUANTILE, INIT_GRID, INIT_USER = 0, 1, 2
DEV_NONFINITE = 1
DEV_TIMEOUT = 2          # a bounded wait between the blocks of the fit-rounds kernel ran out: results are not valid
DEV_SCRATCH = 4          # the quantile start ran out of scratch: pass a larger workspace (workspace_bytes_full)
ERR_TIMEOUT = 10

_LIB_PATH = os.environ.get("AAAC_B200_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libaaac_b200.so")
_lib = None

EXPORTS = ["aaac_status_string", "aaac_workspace_bytes", "aaac_act_stats", "aaac_fit_layer", "aaac_pack",
           "aaac_dequant", "aaac_act_stats_noalloc", "aaac_host_workspace_bytes", "aaac_quantize_layer_host", "aaac_timing_begin",
           "aaac_timing_end", "aaac_fit_layer_sel", "aaac_pack_sel", "aaac_dequant_sel", "aaac_prescale_columns",
           "aaac_quantize_layer_host_async", "aaac_launch_count", "aaac_debug_fit_wait", "aaac_fit_layers", "aaac_workspace_bytes_full", "aaac_debug_quantile_cap",
           "aaac_quantize_layers"]


class AaacError(RuntimeError):
    pass


class LayerDesc(C.Structure):
    """aaac_layer of include/aaac.h."""
    _fields_ = [("W", C.c_void_p), ("N", C.c_int64), ("K", C.c_int64), ("ldw", C.c_int64), ("I", C.c_void_p),
                ("X", C.c_void_p), ("T", C.c_int64), ("ldx", C.c_int64), ("T01", C.c_void_p), ("scales", C.c_void_p),
                ("tensor_scale", C.c_void_p), ("err_trace", C.c_void_p), ("ws", C.c_void_p), ("ws_bytes", C.c_size_t)]


def lib():
    """Loads the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise AaacError(f"{_LIB_PATH} is missing: build it with `python -m paper_2605_08692_b200.build`")
        L = C.CDLL(_LIB_PATH)
        L.aaac_status_string.restype = C.c_char_p
        L.aaac_status_string.argtypes = [C.c_int]
        L.aaac_workspace_bytes.restype = C.c_size_t
        L.aaac_workspace_bytes.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64]
        L.aaac_workspace_bytes_full.restype = C.c_size_t
        L.aaac_workspace_bytes_full.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64]
        L.aaac_host_workspace_bytes.restype = C.c_size_t
        L.aaac_host_workspace_bytes.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64]
        vp, i64, ci = C.c_void_p, C.c_int64, C.c_int
        L.aaac_act_stats.argtypes = [vp, i64, i64, i64, vp, ci, vp, vp, C.c_size_t, vp]
        L.aaac_act_stats_noalloc.argtypes = [vp, i64, i64, i64, vp, ci, vp, vp]
        L.aaac_act_stats_noalloc.restype = ci
        L.aaac_fit_layer.argtypes = [vp, i64, i64, i64, ci, ci, vp, vp, i64, i64, ci, ci, ci, vp, vp, vp, vp, vp, vp,
                                     C.c_size_t, vp]
        L.aaac_pack.argtypes = [vp, i64, i64, i64, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        L.aaac_dequant.argtypes = [vp, vp, vp, vp, i64, i64, ci, ci, vp, i64, vp]
        L.aaac_fit_layer_sel.argtypes = [vp, i64, i64, i64, ci, ci, ci, vp, vp, i64, i64, ci, ci, ci, vp, vp, vp, vp,
                                         vp, vp, C.c_size_t, vp]
        L.aaac_pack_sel.argtypes = [vp, i64, i64, i64, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                    C.c_size_t, vp]
        L.aaac_dequant_sel.argtypes = [vp, vp, vp, vp, vp, i64, i64, ci, ci, ci, vp, i64, vp]
        L.aaac_prescale_columns.argtypes = [vp, i64, i64, i64, vp, vp, i64, vp, vp, vp, vp]
        L.aaac_prescale_columns.restype = ci
        L.aaac_quantize_layer_host.argtypes = [vp, i64, i64, ci, ci, vp, i64, ci, ci, vp, vp, vp, vp, vp, vp, vp,
                                               C.c_size_t, vp]
        L.aaac_quantize_layer_host_async.argtypes = [vp, i64, i64, ci, ci, vp, i64, ci, ci, vp, vp, vp, vp, vp, vp, vp,
                                                     vp, C.c_size_t, vp]
        L.aaac_quantize_layer_host_async.restype = ci
        L.aaac_fit_layers.argtypes = [C.POINTER(LayerDesc), ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.aaac_fit_layers.restype = ci
        L.aaac_quantize_layers.argtypes = [C.POINTER(LayerDesc), C.POINTER(LayerOut), ci, ci, ci, ci, ci, ci, ci, vp, vp]
        L.aaac_quantize_layers.restype = ci
        L.aaac_debug_quantile_cap.argtypes = [C.c_size_t]
        L.aaac_debug_quantile_cap.restype = ci
        L.aaac_debug_fit_wait.argtypes = [ci, C.c_uint]
        L.aaac_debug_fit_wait.restype = ci
        L.aaac_launch_count.restype = C.c_ulonglong
        L.aaac_launch_count.argtypes = []
        L.aaac_timing_begin.argtypes = [ci]
        L.aaac_timing_end.argtypes = [vp, ci]
        for f in ("aaac_act_stats", "aaac_fit_layer", "aaac_pack", "aaac_dequant", "aaac_quantize_layer_host",
                  "aaac_fit_layer_sel", "aaac_pack_sel", "aaac_dequant_sel",
                  "aaac_timing_begin", "aaac_timing_end"):
            getattr(L, f).restype = C.c_int
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise AaacError(f"aaac status {rc}: {lib().aaac_status_string(rc).decode()}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def group_of(mode: int) -> int:
    return 128 if mode == INT4 else 16


def workspace_bytes(mode: int, N: int, K: int, T: int = 0) -> int:
    return int(lib().aaac_workspace_bytes(mode, N, K, T))


def workspace_bytes_full(mode: int, N: int, K: int, T: int = 0) -> int:
    """The workspace size with which the quantile start can never run out of scratch."""
    return int(lib().aaac_workspace_bytes_full(mode, N, K, T))


def alloc_workspace(mode: int, N: int, K: int, T: int = 0, device="cuda", full: bool = False) -> torch.Tensor:
    nbytes = workspace_bytes_full(mode, N, K, T) if full else workspace_bytes(mode, N, K, T)
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def act_stats(X: torch.Tensor, I: torch.Tensor, ws: torch.Tensor, accumulate: bool = False, dev_status=None):
    T, K = X.shape
    _check(lib().aaac_act_stats(_ptr(X), T, K, X.stride(0), _ptr(I), int(accumulate), _ptr(dev_status), _ptr(ws),
                                ws.numel(), _stream()))


def act_stats_noalloc(X: torch.Tensor, I: torch.Tensor, accumulate: bool = False, dev_status=None):
    """aaac_act_stats without a workspace: for callers that may not allocate device memory.
    K <= 32768; calls on one GPU share the library's built-in scratch and must not overlap."""
    T, K = X.shape
    _check(lib().aaac_act_stats_noalloc(_ptr(X), T, K, X.stride(0), _ptr(I), int(accumulate), _ptr(dev_status),
                                        _stream()))


def fit_layer(W, mode, *, I=None, X=None, n_outer, init, T01, scales, tensor_scale, ws, err_trace=None,
              dev_status=None, n_inner=1, group=None, sel_group=None):
    N, K = W.shape
    T, ldx = (X.shape[0], X.stride(0)) if X is not None else (0, 0)
    if sel_group is not None:
        _check(lib().aaac_fit_layer_sel(_ptr(W), N, K, W.stride(0), mode, group or group_of(mode), sel_group, _ptr(I),
                                        _ptr(X), T, ldx, n_outer, n_inner, init, _ptr(T01), _ptr(scales),
                                        _ptr(tensor_scale), _ptr(err_trace), _ptr(dev_status), _ptr(ws), ws.numel(),
                                        _stream()))
        return
    _check(lib().aaac_fit_layer(_ptr(W), N, K, W.stride(0), mode, group or group_of(mode), _ptr(I), _ptr(X), T, ldx,
                                n_outer, n_inner, init, _ptr(T01), _ptr(scales), _ptr(tensor_scale), _ptr(err_trace),
                                _ptr(dev_status), _ptr(ws), ws.numel(), _stream()))


def fit_layers(layers, mode, *, n_outer, init, n_inner=1, group=None, sel_group=None, dev_status=None):
    """aaac_fit_layers: `layers` is a list of dicts with the keyword arguments of fit_layer that belong
    to one layer (W, I or X, T01, scales, tensor_scale, ws, optionally err_trace)."""
    g = group or group_of(mode)
    arr = _layer_descs(layers)
    _check(lib().aaac_fit_layers(arr, len(layers), mode, g, sel_group or g, n_outer, n_inner, init, _ptr(dev_status),
                                 _stream()))


class LayerOut(C.Structure):
    """aaac_layer_out of include/aaac.h."""
    _fields_ = [("T01_bf16", C.c_void_p), ("codes", C.c_void_p), ("sigma_bits", C.c_void_p), ("err_out", C.c_void_p),
                ("stats", C.c_void_p), ("What", C.c_void_p), ("ldo", C.c_int64)]


def _layer_descs(layers):
    arr = (LayerDesc * len(layers))()
    for d, a in zip(arr, layers):
        W, X = a["W"], a.get("X")
        d.W, d.N, d.K, d.ldw = W.data_ptr(), W.shape[0], W.shape[1], W.stride(0)
        d.I = a["I"].data_ptr() if a.get("I") is not None else None
        d.X = X.data_ptr() if X is not None else None
        d.T, d.ldx = (X.shape[0], X.stride(0)) if X is not None else (0, 0)
        d.T01, d.scales, d.tensor_scale = a["T01"].data_ptr(), a["scales"].data_ptr(), a["tensor_scale"].data_ptr()
        d.err_trace = a["err_trace"].data_ptr() if a.get("err_trace") is not None else None
        d.ws, d.ws_bytes = a["ws"].data_ptr(), a["ws"].numel()
    return arr


def quantize_layers(layers, mode, *, n_outer, init, n_inner=1, group=None, sel_group=None, dev_status=None):
    """aaac_quantize_layers: the dicts of fit_layers plus the outputs of the pack pass (T01_bf16, codes,
    optionally sigma_bits, err_out, stats) and optionally What for the reconstruction."""
    g = group or group_of(mode)
    arr = _layer_descs(layers)
    outs = (LayerOut * len(layers))()
    for o, a in zip(outs, layers):
        o.T01_bf16, o.codes = a["T01_bf16"].data_ptr(), a["codes"].data_ptr()
        for name in ("sigma_bits", "err_out", "stats"):
            setattr(o, name, a[name].data_ptr() if a.get(name) is not None else None)
        What = a.get("What")
        o.What, o.ldo = (What.data_ptr(), What.stride(0)) if What is not None else (None, 0)
    _check(lib().aaac_quantize_layers(arr, outs, len(layers), mode, g, sel_group or g, n_outer, n_inner, init,
                                      _ptr(dev_status), _stream()))


def pack(W, mode, *, I, T01, T01_bf16, scales, tensor_scale, codes, ws, err_out=None, stats=None, group=None,
         sel_group=None, sigma_bits=None):
    N, K = W.shape
    if sel_group is not None:
        _check(lib().aaac_pack_sel(_ptr(W), N, K, W.stride(0), mode, group or group_of(mode), sel_group, _ptr(I),
                                   _ptr(T01), _ptr(T01_bf16), _ptr(scales), _ptr(tensor_scale), _ptr(codes),
                                   _ptr(sigma_bits), _ptr(err_out), _ptr(stats), _ptr(ws), ws.numel(), _stream()))
        return
    _check(lib().aaac_pack(_ptr(W), N, K, W.stride(0), mode, group or group_of(mode), _ptr(I), _ptr(T01),
                           _ptr(T01_bf16), _ptr(scales), _ptr(tensor_scale), _ptr(codes), _ptr(err_out), _ptr(stats),
                           _ptr(ws), ws.numel(), _stream()))


def dequant(codes, scales, tensor_scale, T01_bf16, mode, What, group=None, sel_group=None, sigma_bits=None):
    N, K = What.shape
    if sel_group is not None:
        _check(lib().aaac_dequant_sel(_ptr(codes), _ptr(scales), _ptr(sigma_bits), _ptr(tensor_scale), _ptr(T01_bf16),
                                      N, K, mode, group or group_of(mode), sel_group, _ptr(What), What.stride(0),
                                      _stream()))
        return
    _check(lib().aaac_dequant(_ptr(codes), _ptr(scales), _ptr(tensor_scale), _ptr(T01_bf16), N, K, mode,
                              group or group_of(mode), _ptr(What), What.stride(0), _stream()))


def prescale_columns(W, a, W_out, I=None, I_out=None, dev_status=None):
    """W_out = bf16(W * a) per input channel (in place if W_out is W); I_out = I / a^2."""
    N, K = W.shape
    _check(lib().aaac_prescale_columns(_ptr(W), N, K, W.stride(0), _ptr(a), _ptr(W_out), W_out.stride(0), _ptr(I),
                                       _ptr(I_out), _ptr(dev_status), _stream()))


def host_workspace_bytes(mode, N, K, T) -> int:
    return int(lib().aaac_host_workspace_bytes(mode, N, K, T))


def quantize_layer_host(W_host, X_host, mode, *, n_outer, init, T01_host, T01_bf16_host, scales_host,
                        tensor_scale_host, codes_host, err_out_host, ws):
    """Host tensors in and out (pinned for asynchronous copies); ws is device scratch."""
    N, K = W_host.shape
    T = X_host.shape[0]
    _check(lib().aaac_quantize_layer_host(_ptr(W_host), N, K, mode, group_of(mode), _ptr(X_host), T, n_outer, init,
                                          _ptr(T01_host), _ptr(T01_bf16_host), _ptr(scales_host),
                                          _ptr(tensor_scale_host), _ptr(codes_host), _ptr(err_out_host), _ptr(ws),
                                          ws.numel(), _stream()))


def quantize_layer_host_async(W_host, X_host, mode, *, n_outer, init, T01_host, T01_bf16_host, scales_host,
                              tensor_scale_host, codes_host, err_out_host, status_host, ws):
    """As quantize_layer_host, but only enqueued on the current stream: synchronise it before
    reading the host tensors; status_host (pinned int32[1]) then holds the device status bits."""
    N, K = W_host.shape
    T = X_host.shape[0]
    _check(lib().aaac_quantize_layer_host_async(_ptr(W_host), N, K, mode, group_of(mode), _ptr(X_host), T, n_outer,
                                                init, _ptr(T01_host), _ptr(T01_bf16_host), _ptr(scales_host),
                                                _ptr(tensor_scale_host), _ptr(codes_host), _ptr(err_out_host),
                                                _ptr(status_host), _ptr(ws), ws.numel(), _stream()))


def debug_fit_wait(extra_arrivals: int = 0, spin_limit: int = 0):
    """Test hook: make the fit rounds' bounded wait run out (extra_arrivals > 0) after spin_limit
    polls; (0, 0) restores normal operation."""
    _check(lib().aaac_debug_fit_wait(extra_arrivals, spin_limit))


def debug_quantile_cap(entries: int = 0):
    """Test hook: cap the quantile start's candidate list at `entries` (0 restores the normal size)."""
    _check(lib().aaac_debug_quantile_cap(entries))


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(lib().aaac_launch_count())


def timing_begin(max_launches: int):
    _check(lib().aaac_timing_begin(max_launches))


def timing_end(capacity: int):
    buf = (C.c_float * capacity)()
    n = lib().aaac_timing_end(buf, capacity)
    if n < 0:
        raise AaacError("aaac_timing_end failed")
    return [buf[i] for i in range(n)]


# ---- convenience for tests and the benchmark: allocate outputs, run the whole path ----

def quantize_layer(W, mode, *, I=None, X=None, n_outer, init, ws=None, want_trace=False, T01_init=None, n_inner=1,
                   sel_group=None):
    """Runs aaac_fit_layer then aaac_pack on device tensors and returns a dict of device tensors."""
    N, K = W.shape
    g = group_of(mode)
    dev = W.device
    if ws is None:
        ws = alloc_workspace(mode, N, K, 0 if X is None else X.shape[0], dev)
    T01 = torch.zeros(2, 16, dtype=torch.float32, device=dev)
    if T01_init is not None:
        T01.copy_(T01_init)
    scales = torch.empty(N, K // g, dtype=torch.uint16 if mode == INT4 else torch.uint8, device=dev)
    ts = torch.ones(1, dtype=torch.float32, device=dev)
    trace = torch.zeros(max(n_outer, 1), dtype=torch.float64, device=dev) if want_trace else None
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if I is None:
        I = torch.empty(K, dtype=torch.float32, device=dev)
        act_stats(X, I, ws, dev_status=status)
    fit_layer(W, mode, I=I, n_outer=n_outer, init=init, T01=T01, scales=scales, tensor_scale=ts, ws=ws,
              err_trace=trace, dev_status=status, n_inner=n_inner, sel_group=sel_group)
    T01_fit = T01.clone()
    scales_pos = scales.clone()
    Tb = torch.empty(2, 16, dtype=torch.uint16, device=dev)
    codes = torch.empty(N, K // 2, dtype=torch.uint8, device=dev)
    err = torch.zeros(2, dtype=torch.float64, device=dev)
    stats = torch.zeros(4, dtype=torch.int64, device=dev)
    sigma_bits = None
    if sel_group is not None and sel_group != g:
        sigma_bits = torch.empty(N, K // (8 * sel_group), dtype=torch.uint8, device=dev)
    pack(W, mode, I=I, T01=T01, T01_bf16=Tb, scales=scales, tensor_scale=ts, codes=codes, ws=ws, err_out=err,
         stats=stats, sel_group=sel_group, sigma_bits=sigma_bits)
    return dict(I=I, T01=T01_fit, T01_bf16=Tb, scales=scales, scales_pos=scales_pos, tensor_scale=ts, codes=codes,
                err=err, stats=stats, trace=trace, status=status, sigma_bits=sigma_bits)
