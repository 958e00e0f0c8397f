"""Pins for the oracle's per-input-channel scaling step (the hook that lets AWQ's channel
scaling run before the fit, Section 4 "Combining AAAC with AWQ")."""
import ml_dtypes
import numpy as np

import oracle
from paper_2605_08692_b200 import synth

INT4, NVFP4 = oracle.INT4, oracle.NVFP4


def _case(N=16, K=256, T=64, seed=21):
    W = synth.weights(N, K, seed, "pre/W", outlier_frac=0.02)
    X = synth.activations(T, K, seed, "pre/X", kind="lognormal", massive_frac=0.01)
    return W, X


def test_unit_multipliers_change_nothing():
    W, X = _case()
    I = oracle.act_stats(X)
    Wo, Io = oracle.prescale(W, np.ones(W.shape[1], np.float32), I)
    assert np.array_equal(Wo, W) and np.array_equal(Io, I)


def test_scaled_weights_round_like_ml_dtypes():
    W, X = _case()
    rng = np.random.default_rng(1)
    a = np.exp(rng.normal(size=W.shape[1])).astype(np.float32)
    Wo, _ = oracle.prescale(W, a)
    want = (W.view(ml_dtypes.bfloat16).astype(np.float32) * a[None, :]).astype(ml_dtypes.bfloat16).view(np.uint16)
    assert np.array_equal(Wo, want)


def test_importance_is_that_of_the_inversely_scaled_activations():
    """For multipliers that are powers of two X / a is exact in BF16, so I' must equal Eq. 7 on the
    scaled activations bit for bit; for general a it agrees to FP32 rounding."""
    W, X = _case()
    I = oracle.act_stats(X)
    rng = np.random.default_rng(2)
    a = (2.0 ** rng.integers(-3, 4, size=W.shape[1])).astype(np.float32)
    _, Io = oracle.prescale(W, a, I)
    Xs = (X.view(ml_dtypes.bfloat16).astype(np.float32) / a[None, :]).astype(ml_dtypes.bfloat16).view(np.uint16)
    assert np.array_equal(Io, oracle.act_stats(Xs))
    a2 = np.exp(rng.normal(size=W.shape[1])).astype(np.float32)
    _, Io2 = oracle.prescale(W, a2, I)
    xs = X.view(ml_dtypes.bfloat16).astype(np.float64) / a2[None, :].astype(np.float64)
    assert np.allclose(Io2, (xs * xs).sum(axis=0), rtol=1e-6)


def test_layer_output_is_preserved_by_the_exchange():
    """(x / a) (w a) = x w: with power-of-two multipliers the scaled layer computes the same outputs."""
    W, X = _case()
    rng = np.random.default_rng(3)
    a = (2.0 ** rng.integers(-2, 3, size=W.shape[1])).astype(np.float32)
    Wo, _ = oracle.prescale(W, a)
    w = W.view(ml_dtypes.bfloat16).astype(np.float64)
    ws = Wo.view(ml_dtypes.bfloat16).astype(np.float64)
    x = X.view(ml_dtypes.bfloat16).astype(np.float64)
    assert np.array_equal(x @ w.T, (x / a[None, :]) @ ws.T)


def test_uniform_power_of_two_scaling_commutes_with_the_fit():
    """One multiplier for every channel rescales W and the scales together: normalised weights,
    tables and codes are unchanged, the importance (hence the objective) is divided by a^2."""
    W, X = _case(N=24, K=512)
    I = oracle.act_stats(X)
    a = np.full(W.shape[1], 4.0, np.float32)
    Wo, Io = oracle.prescale(W, a, I)
    assert np.array_equal(Io, I / np.float32(16.0))
    for mode, g in ((INT4, 128), (NVFP4, 16)):
        r0 = oracle.fit_layer(W, mode, g, 4, I=I)
        r1 = oracle.fit_layer(Wo, mode, g, 4, I=Io)
        assert np.array_equal(r0["wt"], r1["wt"])
        assert np.array_equal(r0["T"], r1["T"]) and np.array_equal(r0["codes"], r1["codes"])
        assert np.allclose(r1["trace"] * 16.0, r0["trace"], rtol=1e-14)
