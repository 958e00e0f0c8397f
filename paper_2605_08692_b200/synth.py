"""Seeded synthetic layers and calibration activations.

This module only *creates inputs*: weight matrices W [N x K] and calibration
activations X [T x K] as bf16 bit patterns (numpy uint16).  It contains none of
the quantisation method's arithmetic, so the CPU oracle's tests and the CUDA
path's tests may both draw their inputs from it.

Random numbers come from a counter-based generator: element ``i`` of stream
``name`` under ``seed`` is ``splitmix64(seed ^ (fnv1a(name) * GOLD) + i)``.
Any element can therefore be regenerated on its own, and the result does not
depend on chunking.  Normals are Box-Muller in float64, rounded to bf16 with
round-to-nearest-even.

The shapes and value distributions stand in for the Llama / Qwen layers and the
C4 calibration activations the paper quantises (Sec. 4.1 "Models", "AAAC
configurations"); the real checkpoints and data are not used anywhere.
"""
from __future__ import annotations

import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def fnv1a64(name: str) -> int:
    h = 0xCBF29CE484222325
    for b in name.encode():
        h = ((h ^ b) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + _GOLD
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def raw_u64(seed: int, name: str, start: int, n: int) -> np.ndarray:
    """n consecutive 64-bit draws of stream ``name`` starting at counter ``start``."""
    base = (seed ^ ((fnv1a64(name) * 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
    with np.errstate(over="ignore"):
        ctr = np.arange(start, start + n, dtype=np.uint64) + np.uint64(base)
    return _splitmix64(ctr)


def uniform(seed: int, name: str, n: int, start: int = 0) -> np.ndarray:
    """float64 uniforms in (0, 1)."""
    u = raw_u64(seed, name, start, n)
    return ((u >> np.uint64(11)).astype(np.float64) + 0.5) * (2.0 ** -53)


def normal(seed: int, name: str, n: int, start: int = 0) -> np.ndarray:
    """float64 standard normals; element i uses counters 2i and 2i+1."""
    u = uniform(seed, name, 2 * n, 2 * start)
    return np.sqrt(-2.0 * np.log(u[0::2])) * np.cos(2.0 * np.pi * u[1::2])


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _pick_columns(seed: int, name: str, K: int, count: int) -> np.ndarray:
    """``count`` distinct columns: the positions of the smallest uniforms."""
    if count <= 0:
        return np.zeros(0, dtype=np.int64)
    return np.sort(np.argsort(uniform(seed, name, K), kind="stable")[:count])


def weights(N: int, K: int, seed: int, name: str, *, dist: str = "normal", std: float = 0.02,
            outlier_frac: float = 0.0, outlier_count: int | None = None,
            outlier_mult: float = 10.0) -> np.ndarray:
    """W [N x K] as bf16 bits.  ``dist``: 'normal' or 'student5' (Student-t, 5 d.o.f.).
    A set of input channels (columns) is multiplied by ``outlier_mult``."""
    count = outlier_count if outlier_count is not None else int(round(outlier_frac * K))
    cols = _pick_columns(seed, name + "/outlier_cols", K, count)
    colmul = np.ones(K, dtype=np.float64)
    colmul[cols] = outlier_mult
    out = np.empty((N, K), dtype=np.uint16)
    rows_per = max(1, _CHUNK // K)
    for r0 in range(0, N, rows_per):
        r1 = min(N, r0 + rows_per)
        n = (r1 - r0) * K
        z = normal(seed, name, n, r0 * K)
        if dist == "student5":
            chi = np.zeros(n)
            for j in range(5):
                g = normal(seed, f"{name}/chi{j}", n, r0 * K)
                chi += g * g
            z = z / np.sqrt(chi / 5.0)
        elif dist != "normal":
            raise ValueError(dist)
        w = (z * std).reshape(r1 - r0, K) * colmul[None, :]
        out[r0:r1] = f32_to_bf16_bits(w.astype(np.float32))
    return out


def channel_scales(K: int, seed: int, name: str, *, kind: str = "lognormal",
                   massive_frac: float = 0.0, massive_mult: float = 30.0) -> np.ndarray:
    """Per-input-channel standard deviations c_k of the activations."""
    if kind == "loguniform":            # c = 10^u, u ~ U[-1, 1]
        c = 10.0 ** (2.0 * uniform(seed, name + "/cscale", K) - 1.0)
    elif kind == "lognormal":           # c = exp(z)
        c = np.exp(normal(seed, name + "/cscale", K))
    elif kind == "ones":
        c = np.ones(K)
    else:
        raise ValueError(kind)
    cols = _pick_columns(seed, name + "/massive_cols", K, int(round(massive_frac * K)))
    c[cols] *= massive_mult
    return c


def activations(T: int, K: int, seed: int, name: str, *, kind: str = "lognormal",
                massive_frac: float = 0.0, massive_mult: float = 30.0) -> np.ndarray:
    """X [T x K] as bf16 bits: x[t,k] = c_k * z, z ~ N(0,1)."""
    c = channel_scales(K, seed, name, kind=kind, massive_frac=massive_frac, massive_mult=massive_mult)
    out = np.empty((T, K), dtype=np.uint16)
    rows_per = max(1, _CHUNK // K)
    for r0 in range(0, T, rows_per):
        r1 = min(T, r0 + rows_per)
        z = normal(seed, name, (r1 - r0) * K, r0 * K).reshape(r1 - r0, K)
        out[r0:r1] = f32_to_bf16_bits((z * c[None, :]).astype(np.float32))
    return out


# ---------------------------------------------------------------------------
# The benchmark configurations (shapes and distributions only).
# ---------------------------------------------------------------------------

INT4, NVFP4 = 0, 1
INIT_QUANTILE, INIT_GRID, INIT_USER = 0, 1, 2


def config1(seed: int = 0):
    """512x512 linear, N(0, 0.02) with 4 outlier input channels x10; X 256x512 with
    log-uniform channel scales; INT4 g=128, grid init, 10 rounds."""
    W = weights(512, 512, seed, "cfg1/W", outlier_count=4)
    X = activations(256, 512, seed, "cfg1/X", kind="loguniform")
    return dict(name="cfg1", W=W, X=X, mode=INT4, group=128, init=INIT_GRID, rounds=10)


LLAMA8B_LINEARS = {"q_proj": (4096, 4096), "gate_proj": (14336, 4096), "down_proj": (4096, 14336)}


def config2_layer(which: str, seed: int = 0, *, rows: int | None = None, tokens: int = 4096):
    """One Llama-3-8B-shaped linear: Gaussian weights with 1% outlier columns x10,
    X with log-normal channel scales and 0.5% massive channels x30; NVFP4 g=16,
    quantile init, 20 rounds.  ``rows`` truncates N (for CPU-sized parity cases)."""
    N, K = LLAMA8B_LINEARS[which]
    if rows is not None:
        N = rows
    W = weights(N, K, seed, f"cfg2/{which}/W", outlier_frac=0.01)
    X = activations(tokens, K, seed, f"cfg2/{which}/X", kind="lognormal", massive_frac=0.005)
    return dict(name=f"cfg2/{which}", W=W, X=X, mode=NVFP4, group=16, init=INIT_QUANTILE, rounds=20)


def scaled_layer(N: int, K: int, T: int, seed: int, name: str, *, mode: int, dist: str = "normal",
                 outlier_frac: float = 0.0, init: int = INIT_QUANTILE, rounds: int = 20):
    """Generic stand-in used for the stack-shaped configurations (3, 4, 5) at any size."""
    W = weights(N, K, seed, name + "/W", dist=dist, outlier_frac=outlier_frac)
    X = activations(T, K, seed, name + "/X", kind="lognormal", massive_frac=0.005)
    return dict(name=name, W=W, X=X, mode=mode, group=128 if mode == INT4 else 16, init=init, rounds=rounds)
