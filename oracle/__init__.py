"""CPU oracle for the AAAC per-layer procedure -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrappers around ``aaac_oracle.c`` (plain C, double precision, the paper's
Algorithm 1 step by step) plus ``fit_layer``, which strings the steps together in the
paper's order.  Only the test suite, the smoke check and the benchmark's CPU-baseline
leg may import this package; the CUDA library and its Python binding never do, and this
package imports nothing from them.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
# AAAC_ORACLE_SRC names another copy of the source (the mutation tests plant one mistake in a
# copy and check that a pin fails); its library is built beside it.
_SRC = os.environ.get("AAAC_ORACLE_SRC") or os.path.join(_DIR, "aaac_oracle.c")
_LIB = (os.path.splitext(_SRC)[0] + ".so") if os.environ.get("AAAC_ORACLE_SRC") else os.path.join(_DIR, "libaaac_oracle.so")
_lib = None

INT4, NVFP4 = 0, 1
M = 16


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_objective.restype = C.c_double
        _lib.oracle_output_error.restype = C.c_double
        _lib.oracle_e4m3_to_f32.restype = C.c_float
        _lib.oracle_e4m3_to_f32.argtypes = [C.c_uint8]
        _lib.oracle_e4m3_encode.restype = C.c_uint8
        _lib.oracle_e4m3_encode.argtypes = [C.c_float]
        _lib.oracle_max_threads.restype = C.c_int
        _lib.oracle_output_error_sel.restype = C.c_double
    return _lib


def set_threads(n: int) -> None:
    lib().oracle_set_threads(C.c_int(n))


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16
    return a


def act_stats(X: np.ndarray) -> np.ndarray:
    """Eq. 7: I_k = sum_t X[t,k]^2.  X: bf16 bits [T x K]."""
    X = _u16(X)
    T, K = X.shape
    I = np.empty(K, dtype=np.float32)
    lib().oracle_act_stats(_p(X), C.c_int64(T), C.c_int64(K), C.c_int64(K), _p(I))
    return I


def scales(W: np.ndarray, mode: int, g: int):
    """Alg. 1 line 1.  Returns (scales, tensor_scale): bf16 bits [N x K/g] (INT4) or E4M3
    bytes (NVFP4) and a float32[1] tensor scale (1.0 for INT4)."""
    W = _u16(W)
    N, K = W.shape
    s = np.empty((N, K // g), dtype=np.uint16 if mode == INT4 else np.uint8)
    ts = np.ones(1, dtype=np.float32)
    rc = lib().oracle_scales(_p(W), C.c_int64(N), C.c_int64(K), C.c_int64(K), C.c_int(mode), C.c_int(g),
                             _p(s), _p(ts))
    if rc:
        raise ValueError(f"oracle_scales failed: {rc}")
    return s, ts


def normalise(W, mode, g, s, ts) -> np.ndarray:
    """Eq. 2: w~ = fl32(w * fl32(1/s)) as float32 [N x K]."""
    W = _u16(W)
    N, K = W.shape
    wt = np.empty((N, K), dtype=np.float32)
    lib().oracle_normalise(_p(W), C.c_int64(N), C.c_int64(K), C.c_int64(K), C.c_int(mode), C.c_int(g),
                           _p(np.ascontiguousarray(s)), _p(ts), _p(wt))
    return wt


def init_quantile(wt: np.ndarray) -> np.ndarray:
    """Eq. 9-10.  Returns float64[2,16]."""
    wt = np.ascontiguousarray(wt, dtype=np.float32)
    T = np.empty((2, M), dtype=np.float64)
    lib().oracle_init_quantile(_p(wt), C.c_int64(wt.size), _p(T))
    return T


def init_grid(mode: int) -> np.ndarray:
    T = np.empty((2, M), dtype=np.float64)
    lib().oracle_init_grid(C.c_int(mode), _p(T))
    return T


def fit_round(wt, I, g, T01, want_sigma=False):
    """One outer iteration (n_inner = 1).  Returns (new tables, objective E of the assignment
    step under the *input* tables[, sigma])."""
    wt = np.ascontiguousarray(wt, dtype=np.float32)
    I = np.ascontiguousarray(I, dtype=np.float32)
    N, K = wt.shape
    T = np.array(T01, dtype=np.float64).reshape(2, M).copy()
    E = C.c_double(0.0)
    sig = np.empty((N, K // g), dtype=np.uint8) if want_sigma else None
    rc = lib().oracle_fit_round(_p(wt), _p(I), C.c_int64(N), C.c_int64(K), C.c_int(g), _p(T), C.byref(E), _p(sig))
    if rc:
        raise ValueError(f"oracle_fit_round failed: {rc}")
    return (T, E.value, sig) if want_sigma else (T, E.value)


def assign(wt, I, g, T01):
    """Assignment step alone (Alg. 1 lines 7-11).  Returns (sigma uint8 [N x K/g], objective)."""
    wt = np.ascontiguousarray(wt, dtype=np.float32)
    I = np.ascontiguousarray(I, dtype=np.float32)
    N, K = wt.shape
    T = np.ascontiguousarray(T01, dtype=np.float64).reshape(2, M)
    sig = np.empty((N, K // g), dtype=np.uint8)
    E = C.c_double(0.0)
    rc = lib().oracle_assign(_p(wt), _p(I), C.c_int64(N), C.c_int64(K), C.c_int(g), _p(T), _p(sig), C.byref(E))
    if rc:
        raise ValueError(f"oracle_assign failed: {rc}")
    return sig, E.value


def inner_update(wt, I, g, sigma, T01) -> np.ndarray:
    """One inner k-means iteration with sigma frozen (Alg. 1 lines 15-20), unsorted result."""
    wt = np.ascontiguousarray(wt, dtype=np.float32)
    I = np.ascontiguousarray(I, dtype=np.float32)
    N, K = wt.shape
    T = np.array(T01, dtype=np.float64).reshape(2, M).copy()
    sig = np.ascontiguousarray(sigma, dtype=np.uint8)
    assert sig.shape == (N, K // g)
    rc = lib().oracle_inner_update(_p(wt), _p(I), _p(sig), C.c_int64(N), C.c_int64(K), C.c_int(g), _p(T))
    if rc:
        raise ValueError(f"oracle_inner_update failed: {rc}")
    return T


def sort_tables(T01) -> np.ndarray:
    T = np.array(T01, dtype=np.float64).reshape(2, M).copy()
    lib().oracle_sort_tables(_p(T))
    return T


def outer_iteration(wt, I, g, T01, n_inner):
    """One pass of Alg. 1's outer loop in the paper's order: assignment step, then n_inner inner
    iterations of each table with the selection frozen, then the sort.  Returns (new tables,
    objective of the assignment step, sigma)."""
    sig, E = assign(wt, I, g, T01)
    T = np.array(T01, dtype=np.float64).reshape(2, M).copy()
    for _ in range(n_inner):
        T = inner_update(wt, I, g, sig, T)
    return sort_tables(T), E, sig


def objective(wt, I, g, T01) -> float:
    wt = np.ascontiguousarray(wt, dtype=np.float32)
    I = np.ascontiguousarray(I, dtype=np.float32)
    N, K = wt.shape
    T = np.ascontiguousarray(T01, dtype=np.float64)
    return float(lib().oracle_objective(_p(wt), _p(I), C.c_int64(N), C.c_int64(K), C.c_int(g), _p(T)))


def round_tables(T01):
    """Alg. 1 line 17.  Returns (float32[2,16], bf16 bits uint16[2,16])."""
    T = np.ascontiguousarray(T01, dtype=np.float64)
    Tf = np.empty((2, M), dtype=np.float32)
    Tb = np.empty((2, M), dtype=np.uint16)
    lib().oracle_round_tables(_p(T), _p(Tf), _p(Tb))
    return Tf, Tb


def pack(wt, I, g, Tb):
    """Alg. 1 lines 18-19.  Returns (codes uint8 [N x K/2], sigma uint8 [N x K/g], E_final, ties[2])."""
    wt = np.ascontiguousarray(wt, dtype=np.float32)
    I = np.ascontiguousarray(I, dtype=np.float32)
    N, K = wt.shape
    codes = np.zeros((N, K // 2), dtype=np.uint8)
    sig = np.empty((N, K // g), dtype=np.uint8)
    E = C.c_double(0.0)
    ties = np.zeros(2, dtype=np.uint64)
    rc = lib().oracle_pack(_p(wt), _p(I), C.c_int64(N), C.c_int64(K), C.c_int(g), _p(_u16(Tb)), _p(codes), _p(sig),
                           C.byref(E), _p(ties))
    if rc:
        raise ValueError(f"oracle_pack failed: {rc}")
    return codes, sig, E.value, ties


def apply_sigma(s, sig, mode):
    """Alg. 1 line 20: returns a copy of the scales with sigma in the sign bit."""
    out = np.ascontiguousarray(s).copy()
    lib().oracle_apply_sigma(_p(out), _p(np.ascontiguousarray(sig)), C.c_int64(out.size), C.c_int(mode))
    return out


def dequant(codes, s, ts, Tb, mode, g) -> np.ndarray:
    """Eq. 5.  Returns bf16 bits [N x K]."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape[0], codes.shape[1] * 2
    out = np.empty((N, K), dtype=np.uint16)
    lib().oracle_dequant(_p(codes), _p(np.ascontiguousarray(s)), _p(ts), _p(_u16(Tb)), C.c_int64(N), C.c_int64(K),
                         C.c_int(mode), C.c_int(g), _p(out), C.c_int64(K))
    return out


def output_error(W, codes, s, ts, Tb, I, mode, g) -> float:
    W = _u16(W)
    N, K = W.shape
    return float(lib().oracle_output_error(_p(W), C.c_int64(K), _p(np.ascontiguousarray(codes)),
                                           _p(np.ascontiguousarray(s)), _p(ts), _p(_u16(Tb)),
                                           _p(np.ascontiguousarray(I, dtype=np.float32)),
                                           C.c_int64(N), C.c_int64(K), C.c_int(mode), C.c_int(g)))


def prescale(W, a, I=None):
    """Per-input-channel scaling before the fit (Sec. 4, combining with AWQ): returns
    (bf16 bits of w * a_k, I_k / a_k^2 or None)."""
    W = _u16(W)
    N, K = W.shape
    a = np.ascontiguousarray(a, dtype=np.float32)
    Wo = np.empty_like(W)
    Io = None if I is None else np.empty(K, dtype=np.float32)
    Ii = None if I is None else np.ascontiguousarray(I, dtype=np.float32)
    lib().oracle_prescale(_p(W), C.c_int64(N), C.c_int64(K), C.c_int64(K), _p(a), _p(Wo), C.c_int64(K), _p(Ii), _p(Io))
    return Wo, Io


def pack_sigma_bits(sigma) -> np.ndarray:
    """Alg. 1 line 20 for S < g: sigma [N x K/S] -> bits uint8 [N x K/(8 S)], group j of a row in bit
    j % 8 of byte j // 8."""
    sig = np.ascontiguousarray(sigma, dtype=np.uint8)
    N, GS = sig.shape
    bits = np.empty((N, GS // 8), dtype=np.uint8)
    rc = lib().oracle_pack_sigma_bits(_p(sig), C.c_int64(N), C.c_int64(GS), _p(bits))
    if rc:
        raise ValueError(f"oracle_pack_sigma_bits failed: {rc}")
    return bits


def dequant_sel(codes, s, ts, Tb, sigma_bits, S, mode, g) -> np.ndarray:
    """Eq. 5 with separately stored selection bits (selection group S, scale group g)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape[0], codes.shape[1] * 2
    out = np.empty((N, K), dtype=np.uint16)
    lib().oracle_dequant_sel(_p(codes), _p(np.ascontiguousarray(s)), _p(ts), _p(_u16(Tb)),
                             _p(np.ascontiguousarray(sigma_bits, dtype=np.uint8)), C.c_int(S), C.c_int64(N),
                             C.c_int64(K), C.c_int(mode), C.c_int(g), _p(out), C.c_int64(K))
    return out


def output_error_sel(W, codes, s, ts, Tb, sigma_bits, S, I, mode, g) -> float:
    W = _u16(W)
    N, K = W.shape
    return float(lib().oracle_output_error_sel(_p(W), C.c_int64(K), _p(np.ascontiguousarray(codes)),
                                               _p(np.ascontiguousarray(s)), _p(ts), _p(_u16(Tb)),
                                               _p(np.ascontiguousarray(sigma_bits, dtype=np.uint8)), C.c_int(S),
                                               _p(np.ascontiguousarray(I, dtype=np.float32)),
                                               C.c_int64(N), C.c_int64(K), C.c_int(mode), C.c_int(g)))


def fit_layer(W, mode, g, rounds, *, I=None, X=None, init="quantile", T_init=None, n_inner=1, S=None):
    """Algorithm 1 for one layer (rounds = n_outer).  S = selection group size (default g); with
    S < g the scales keep a clear sign bit and the selection bits come back as sigma_bits.

    Returns a dict: I, scales (sign bit = sigma), tensor_scale, T (float64 tables after the
    last round), T_f32, T_bf16, codes, sigma, trace (objective of each round's assignment
    step), E_final (objective under the BF16 tables), ties, wt.
    """
    if I is None:
        I = act_stats(X)
    s, ts = scales(W, mode, g)
    wt = normalise(W, mode, g, s, ts)
    if init == "quantile":
        T = init_quantile(wt)
    elif init == "grid":
        T = init_grid(mode)
    else:
        T = np.array(T_init, dtype=np.float64).reshape(2, M)
    T_start = T.copy()
    trace = []
    for _ in range(rounds):
        if n_inner == 1:
            T, E = fit_round(wt, I, S or g, T)
        else:
            T, E, _ = outer_iteration(wt, I, S or g, T, n_inner)
        trace.append(E)
    Tf, Tb = round_tables(T)
    codes, sig, E_final, ties = pack(wt, I, S or g, Tb)
    if S is not None and S != g:
        return dict(I=I, scales=s, scales_unsigned=s, sigma_bits=pack_sigma_bits(sig), tensor_scale=ts, T=T,
                    T_init=T_start, T_f32=Tf, T_bf16=Tb, codes=codes, sigma=sig, trace=np.array(trace),
                    E_final=E_final, ties=ties, wt=wt)
    s_signed = apply_sigma(s, sig, mode)
    return dict(I=I, scales=s_signed, scales_unsigned=s, tensor_scale=ts, T=T, T_init=T_start, T_f32=Tf, T_bf16=Tb,
                codes=codes, sigma=sig, trace=np.array(trace), E_final=E_final, ties=ties, wt=wt)
