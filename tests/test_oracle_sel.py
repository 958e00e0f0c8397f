"""Pins for the oracle with a selection group S smaller than the scale group g (the paper's
INT4 variant g = 128, S = 16, selection bits stored apart at 1/S bit per weight)."""
import os

import numpy as np
import pytest

import oracle
from paper_2605_08692_b200 import synth

INT4 = oracle.INT4
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _case(N=16, K=512, seed=9, name="sel"):
    W = synth.weights(N, K, seed, name + "/W", outlier_frac=0.02)
    X = synth.activations(64, K, seed, name + "/X", kind="lognormal", massive_frac=0.01)
    return W, X


def test_selection_overhead_is_one_over_S_bits_per_weight():
    """Section 3.1: S < g costs 1/S bit per weight; the paper quotes 0.0625 bpw for S = 16."""
    consts = dict((k.strip(), v.strip()) for k, v in
                  (l.split("=") for l in open(os.path.join(GOLDEN, "paper_constants.txt"))
                   if l.strip() and not l.startswith("#")))
    W, X = _case()
    r = oracle.fit_layer(W, INT4, 128, 2, X=X, S=16)
    bpw = r["sigma_bits"].size * 8 / W.size
    assert bpw == 1 / 16 == float(consts["selection_bpw_S16"])
    assert np.all(r["scales"] >> 15 == 0)                     # sign bits stay clear


def test_sigma_bit_order_matches_numpy_packbits():
    rng = np.random.default_rng(0)
    sig = rng.integers(0, 2, size=(5, 48), dtype=np.uint8)
    bits = oracle.pack_sigma_bits(sig)
    assert np.array_equal(bits, np.packbits(sig, axis=1, bitorder="little"))
    assert np.array_equal(np.unpackbits(bits, axis=1, bitorder="little"), sig)


def test_S_equal_g_is_the_sign_bit_path():
    W, X = _case()
    a = oracle.fit_layer(W, INT4, 128, 3, X=X)
    b = oracle.fit_layer(W, INT4, 128, 3, X=X, S=128)
    for k in ("T", "codes", "scales", "trace"):
        assert np.array_equal(a[k], b[k])


def test_finer_selection_never_raises_the_objective_under_fixed_tables():
    """For fixed tables the best choice per 16 weights is at least as good as one choice per 128:
    min over a finer partition."""
    W, X = _case(N=24)
    I = oracle.act_stats(X)
    s, ts = oracle.scales(W, INT4, 128)
    wt = oracle.normalise(W, INT4, 128, s, ts)
    T = oracle.init_quantile(wt)
    prev = None
    for S in (128, 64, 32, 16, 8):
        E = oracle.objective(wt, I, S, T)
        if prev is not None:
            assert E <= prev * (1 + 1e-14)
        prev = E
    # and the per-16 selection equals the brute-force choice group by group
    sig, E16 = oracle.assign(wt, I, 16, T)
    x = wt.astype(np.float64).reshape(wt.shape[0], -1, 16)
    w = I.astype(np.float64).reshape(-1, 16)
    e = [((np.abs(x[..., None] - T[r]).min(axis=-1)) ** 2 * w).sum(axis=-1) for r in range(2)]
    assert np.array_equal(sig, (e[1] < e[0]).astype(np.uint8))
    assert np.isclose(E16, np.minimum(e[0], e[1]).sum(), rtol=1e-13)


def test_dequant_with_separate_bits_is_table_times_scale():
    W, X = _case()
    g, S = 128, 16
    r = oracle.fit_layer(W, INT4, g, 2, X=X, S=S)
    What = oracle.dequant_sel(r["codes"], r["scales"], r["tensor_scale"], r["T_bf16"], r["sigma_bits"], S, INT4, g)
    N, K = W.shape
    codes = np.stack([r["codes"] & 15, r["codes"] >> 4], axis=-1).reshape(N, K)
    sig = np.repeat(np.unpackbits(r["sigma_bits"], axis=1, bitorder="little"), S, axis=1)
    Tf = synth.bf16_bits_to_f32(r["T_bf16"]).reshape(2, 16)
    sc = np.repeat(synth.bf16_bits_to_f32(r["scales"]), g, axis=1)
    want = synth.f32_to_bf16_bits((Tf[sig, codes] * sc).astype(np.float32))
    assert np.array_equal(What, want)
    # the reported weight-unit error is that of these dequantised weights (before the BF16 rounding)
    I = r["I"].astype(np.float64)
    d = synth.bf16_bits_to_f32(W).astype(np.float64) - Tf[sig, codes].astype(np.float64) * sc.astype(np.float64)
    E = oracle.output_error_sel(W, r["codes"], r["scales"], r["tensor_scale"], r["T_bf16"], r["sigma_bits"], S, I, INT4, g)
    assert np.isclose(E, np.sum(I * d * d), rtol=1e-12)
    # S = g through the same routine equals the sign-bit dequant
    a = oracle.fit_layer(W, INT4, g, 2, X=X)
    bits = oracle.pack_sigma_bits(np.repeat(a["sigma"], 8, axis=1))          # 8 identical bits per scale group
    Wa = oracle.dequant_sel(a["codes"], a["scales_unsigned"], a["tensor_scale"], a["T_bf16"], bits, 16, INT4, g)
    assert np.array_equal(Wa, oracle.dequant(a["codes"], a["scales"], a["tensor_scale"], a["T_bf16"], INT4, g))


def test_S16_fits_better_than_S128_and_is_monotone():
    """The paper's reason for S = 16 at g = 128: finer selection lowers the error."""
    W, X = _case(N=32, K=1024)
    a = oracle.fit_layer(W, INT4, 128, 6, X=X, S=128)
    b = oracle.fit_layer(W, INT4, 128, 6, X=X, S=16)
    assert np.all(b["trace"][1:] <= b["trace"][:-1] * (1 + 1e-12))
    assert b["E_final"] < a["E_final"]
