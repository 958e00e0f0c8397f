"""Pins for the CPU oracle: each test checks it against something other than itself --
facts the paper prints, closed forms, invariants of the procedure, independent library
routines (numpy, scikit-learn, ml_dtypes) and brute force on tiny inputs."""
import itertools
import os

import ml_dtypes
import numpy as np
import pytest

import oracle
from paper_2605_08692_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
INT4, NVFP4 = oracle.INT4, oracle.NVFP4


def _consts():
    out = {}
    for line in open(os.path.join(GOLDEN, "paper_constants.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split("=")
            out[k.strip()] = v.strip()
    return out


def _small(mode, N=24, K=256, T=64, seed=3, name="pin"):
    W = synth.weights(N, K, seed, name + "/W", outlier_frac=0.02)
    X = synth.activations(T, K, seed, name + "/X", kind="lognormal", massive_frac=0.01)
    g = 128 if mode == INT4 else 16
    return W, X, g


# ------------------------------------------------------------------ formats

def test_bf16_rounding_matches_ml_dtypes():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    want = x.astype(ml_dtypes.bfloat16).view(np.uint16)
    got = synth.f32_to_bf16_bits(x)
    assert np.array_equal(want, got)
    # the oracle's own rounding, through round_tables
    t = np.sort(x[:32].astype(np.float64)).reshape(2, 16)
    t.sort(axis=1)
    Tf, Tb = oracle.round_tables(t)
    assert np.array_equal(Tb, t.astype(np.float32).astype(ml_dtypes.bfloat16).view(np.uint16))


def test_e4m3_codec_matches_ml_dtypes():
    L = oracle.lib()
    codes = np.arange(0x7F, dtype=np.uint8)
    want = codes.view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    got = np.array([L.oracle_e4m3_to_f32(int(c)) for c in codes], dtype=np.float32)
    assert np.array_equal(want, got)
    assert got[0x7E] == 448.0 and got[1] == 2.0 ** -9
    rng = np.random.default_rng(1)
    xs = np.concatenate([np.exp(rng.uniform(np.log(1e-4), np.log(600), 4000)),
                         0.5 * (got[:-1] + got[1:]),            # exact half-way points
                         got, [0.0, 1e-9, 448.0, 460.0, 1e6]]).astype(np.float32)
    for x in xs:
        enc = int(L.oracle_e4m3_encode(float(x)))
        ref = np.float32(min(float(x), 464.0)).astype(ml_dtypes.float8_e4m3fn)   # saturate; 464 -> 448 (RNE)
        if float(x) > 464.0:
            ref = np.float32(448.0).astype(ml_dtypes.float8_e4m3fn)
        assert enc == int(ref.view(np.uint8)), (x, enc, ref)


def test_paper_constants():
    c = _consts()
    M = int(c["table_entries"])
    assert M == oracle.M
    # Storage: 2 tables x 16 BF16 entries = 64 bytes; ~224 layers -> about 14 KB
    W, X, g = _small(INT4)
    r = oracle.fit_layer(W, INT4, g, 2, X=X, init="grid")
    assert r["T_bf16"].dtype == np.uint16 and r["T_bf16"].nbytes == int(c["table_bytes_per_layer"])
    assert round(int(c["layers_7b"]) * r["T_bf16"].nbytes / 1024) == int(c["table_kib_7b"])
    assert 1.0 / 16 == float(c["selection_bpw_S16"])
    # NVFP4 grid = signed E2M1 values
    mags = [float(v) for v in c["e2m1_magnitudes"].split()]
    grid = oracle.init_grid(NVFP4)[0]
    assert sorted(set(np.abs(grid))) == mags and len(grid) == 16
    assert np.array_equal(grid, -grid[::-1])
    assert np.array_equal(oracle.init_grid(INT4)[0], np.arange(-8, 8))
    # Eq. 10 delta
    assert abs(float(c["delta"]) - 1.0 / (2 * (M - 1))) < 1e-16


def test_grid_start_second_table_is_the_first_moved_up_half_a_step():
    """The grid start's T1 against values written by hand from what the words fix (golden file):
    INT4's uniform grid moved up half a step is -7.5 .. 7.5; on the E2M1 grid every entry of T1 is
    the midpoint of two neighbours of T0 and the last step repeats half the last spacing."""
    c = _consts()
    t1_int4 = np.array([float(v) for v in c["grid_t1_int4"].split()])
    t0_nv = np.array([float(v) for v in c["grid_t0_nvfp4"].split()])
    t1_nv = np.array([float(v) for v in c["grid_t1_nvfp4"].split()])
    assert len(t1_int4) == len(t0_nv) == len(t1_nv) == 16
    g_int4, g_nv = oracle.init_grid(INT4), oracle.init_grid(NVFP4)
    assert np.array_equal(g_int4[1], t1_int4)
    assert np.array_equal(g_nv[0], t0_nv) and np.array_equal(g_nv[1], t1_nv)
    # closed form, independent of the stored numbers: a uniform grid shifted by half its step
    assert np.array_equal(g_int4[1], g_int4[0] + 0.5)
    # every T1 entry but the last lies strictly between two neighbours of T0 (or on a doubled
    # zero), at equal distance from both
    for T0, T1 in ((g_int4[0], g_int4[1]), (g_nv[0], g_nv[1])):
        assert np.array_equal(T1[:-1] - T0[:-1], T0[1:] - T1[:-1])
        assert T1[-1] - T0[-1] == (T0[-1] - T0[-2]) / 2
        assert np.all(np.diff(T1) >= 0)


def _bf16_direct(v):
    """double -> BF16 in one round-to-nearest-even step (normal range), in exact arithmetic:
    v = q * 2^(e-8) with |q| in [128, 256); rint is exact and rounds half to even."""
    v = np.asarray(v, dtype=np.float64)
    m, e = np.frexp(v)                                     # v = m 2^e, |m| in [0.5, 1)
    quantum = np.ldexp(1.0, e - 8)
    r = np.rint(v / quantum) * quantum                     # exact: a multiple of the quantum
    return (r.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def test_double_rounding_of_tables_equals_direct_rounding_on_the_seeded_layers():
    """Alg. 1 rounds the tables to BF16; the chain here is double -> FP32 -> BF16.  It can differ
    from double -> BF16 only next to a BF16 half-way point: counted over fitted tables, expected 0."""
    differ = total = 0
    for mode in (INT4, NVFP4):
        for seed in range(4):
            W, X, g = _small(mode, N=32, K=256, seed=seed, name=f"pin/dr{seed}")
            for init in ("grid", "quantile"):
                r = oracle.fit_layer(W, mode, g, 6, X=X, init=init)
                direct = _bf16_direct(r["T"])
                differ += int(np.sum(direct != r["T_bf16"]))
                total += direct.size
    assert total == 2 * 4 * 2 * 32 and differ == 0
    # and a constructed value that the two chains do round differently: just above a BF16 half-way
    # point, by less than half an FP32 step, so the FP32 rounding lands on the half-way point
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    T = np.sort(np.concatenate([[v], np.arange(2, 33, dtype=np.float64)])).reshape(2, 16)
    Tf, Tb = oracle.round_tables(T)
    assert Tf[0, 0] == np.float32(1.0 + 2.0 ** -8)
    assert Tb[0, 0] == 0x3F80                               # ties-to-even of the FP32 value: 1.0
    assert _bf16_direct([v])[0] == 0x3F81
    x = np.random.default_rng(5).standard_normal(4000) * 3
    assert np.array_equal(_bf16_direct(x.astype(np.float32)), synth.f32_to_bf16_bits(x.astype(np.float32)))


# ------------------------------------------------------------------ Eq. 7

def test_act_stats_is_column_sum_of_squares():
    X = synth.activations(300, 96, 5, "pin/actX", kind="loguniform")
    I = oracle.act_stats(X)
    x = synth.bf16_bits_to_f32(X).astype(np.float64)
    want = np.einsum("tk,tk->k", x, x)
    assert I.dtype == np.float32
    assert np.allclose(I, want, rtol=1e-7, atol=0)
    # a single token: exactly x^2
    I1 = oracle.act_stats(X[:1])
    assert np.array_equal(I1, (x[0] ** 2).astype(np.float32))


# ------------------------------------------------------------------ scales, Eq. 2

def test_int4_scales_absmax_over_7_and_range():
    W, X, g = _small(INT4)
    W[3, 128:256] = 0                                   # an all-zero group
    s, ts = oracle.scales(W, INT4, g)
    w = synth.bf16_bits_to_f32(W).reshape(W.shape[0], -1, g)
    a = np.abs(w).max(axis=2)
    want = (a / np.float32(7.0)).astype(np.float32).astype(ml_dtypes.bfloat16)
    want = np.where(a == 0, ml_dtypes.bfloat16(1.0), want)
    assert np.array_equal(s, want.view(np.uint16))
    assert np.all(s >> 15 == 0) and ts[0] == 1.0
    wt = oracle.normalise(W, INT4, g, s, ts)
    sf = synth.bf16_bits_to_f32(s)
    r = (np.float32(1.0) / sf).astype(np.float32)
    assert np.array_equal(wt.reshape(w.shape), (w * r[:, :, None]).astype(np.float32))
    assert np.abs(wt).max() < 8.0 and np.abs(wt).max() > 6.9
    assert np.all(wt[3, 128:256] == 0)


def test_nvfp4_scales_e4m3_and_range():
    W, X, g = _small(NVFP4)
    W[2, 32:48] = 0
    W[5, 0:16] = synth.f32_to_bf16_bits(np.full(16, 1e-9, np.float32))   # far below the tensor scale
    s, ts = oracle.scales(W, NVFP4, g)
    w = synth.bf16_bits_to_f32(W).reshape(W.shape[0], -1, g)
    A = np.abs(w).max()
    assert ts[0] == np.float32(A) / np.float32(2688.0)
    a = np.abs(w).max(axis=2)
    x = (a / (np.float32(6.0) * ts[0])).astype(np.float32)
    want = x.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    normal = want >= 2
    assert np.array_equal(s[normal], want[normal])
    assert s.min() >= 1 and s.max() <= 0x7E and s.max() == 0x7E     # the absmax group saturates at 448
    assert s[2, 2] == 1 and s[5, 0] == 1
    wt = oracle.normalise(W, NVFP4, g, s, ts)
    assert np.abs(wt).max() < 8.0


def test_nonfinite_weights_are_rejected():
    W, X, g = _small(INT4)
    W[0, 0] = 0x7F80
    with pytest.raises(ValueError):
        oracle.scales(W, INT4, g)


# ------------------------------------------------------------------ Eq. 9-10

@pytest.mark.parametrize("n", [31, 1000, 4097])
def test_quantile_init_matches_numpy(n):
    rng = np.random.default_rng(n)
    wt = (rng.standard_normal(n) * 2.5).astype(np.float32)
    T = oracle.init_quantile(wt)
    q0 = np.arange(16) / 15.0
    d = 1.0 / 30.0
    q1 = d + (1 - d) * np.arange(16) / 15.0
    want0 = np.quantile(wt.astype(np.float64), q0, method="linear")
    want1 = np.quantile(wt.astype(np.float64), q1, method="linear")
    assert np.allclose(T[0], want0, rtol=3e-7, atol=1e-9)
    assert np.allclose(T[1], want1, rtol=3e-7, atol=1e-9)
    assert T[0, 0] == wt.min() and T[0, 15] == wt.max() and T[1, 15] == wt.max()
    assert np.isclose(T[1, 0], np.quantile(wt.astype(np.float64), 1 / 30.0), rtol=3e-7)
    assert np.all(np.diff(T, axis=1) >= 0)


# ------------------------------------------------------------------ Eq. 4, 6, 8: brute force

@pytest.mark.parametrize("S", [1, 2, 3])
def test_selection_and_codes_are_brute_force_optimal(S):
    rng = np.random.default_rng(10 + S)
    N, K = 6, 4 * S
    wt = rng.uniform(-7, 7, (N, K)).astype(np.float32)
    I = rng.uniform(0.1, 5.0, K).astype(np.float32)
    T = np.sort(rng.uniform(-7, 7, (2, 16)), axis=1)
    Tf, Tb = oracle.round_tables(T)
    Tv = synth.bf16_bits_to_f32(Tb).astype(np.float64)
    codes, sig, E, ties = oracle.pack(wt, I, S, Tb) if K % 2 == 0 else (None,) * 4
    nib = np.stack([codes & 15, codes >> 4], axis=2).reshape(N, K)
    total = 0.0
    for n in range(N):
        for j in range(K // S):
            x = wt[n, j * S:(j + 1) * S].astype(np.float64)
            w = I[j * S:(j + 1) * S].astype(np.float64)
            best = (np.inf, None, None)
            for r in range(2):
                for cv in itertools.product(range(16), repeat=S):
                    e = float(np.sum(w * (x - Tv[r, list(cv)]) ** 2))
                    if e < best[0]:
                        best = (e, r, cv)
            got_e = float(np.sum(w * (x - Tv[sig[n, j], nib[n, j * S:(j + 1) * S]]) ** 2))
            assert got_e <= best[0] * (1 + 1e-12) + 1e-300
            assert sig[n, j] == best[1]
            assert np.array_equal(Tv[best[1], list(best[2])], Tv[sig[n, j], nib[n, j * S:(j + 1) * S]])
            total += best[0]
    assert np.isclose(E, total, rtol=1e-12)


# ------------------------------------------------------------------ Lloyd properties

@pytest.mark.parametrize("mode,init", [(INT4, "grid"), (INT4, "quantile"), (NVFP4, "quantile"), (NVFP4, "grid")])
def test_objective_is_monotone_non_increasing(mode, init):
    W, X, g = _small(mode, N=32, K=512)
    r = oracle.fit_layer(W, mode, g, 12, X=X, init=init)
    tr = r["trace"]
    assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-12))
    assert tr[-1] < tr[0]
    # the objective after the last update is no worse than the last assignment's
    assert oracle.objective(r["wt"], r["I"], g, r["T"]) <= tr[-1] * (1 + 1e-12)
    assert np.all(np.diff(r["T"], axis=1) >= 0)


def _lloyd_step_numpy(x, w, T):
    """Independent 1-D weighted Lloyd step: cells from midpoints (searchsorted), weighted means."""
    mids = 0.5 * (T[1:] + T[:-1])
    idx = np.searchsorted(mids, x, side="left")         # x == mid -> lower cell
    num = np.bincount(idx, weights=w * x, minlength=16)
    den = np.bincount(idx, weights=w, minlength=16)
    out = T.copy()
    out[den > 0] = num[den > 0] / den[den > 0]
    return np.sort(out)


def test_identical_tables_reduce_to_single_codebook_weighted_kmeans():
    from sklearn.cluster import KMeans
    W, X, g = _small(INT4, N=16, K=256)
    I = oracle.act_stats(X)
    s, ts = oracle.scales(W, INT4, g)
    wt = oracle.normalise(W, INT4, g, s, ts)
    T0 = np.linspace(-6.5, 6.5, 16)
    T = np.stack([T0, T0])
    x = wt.astype(np.float64).ravel()
    w = np.tile(I.astype(np.float64), wt.shape[0])
    ref = T0.copy()
    for it in range(5):
        Tn, E, sig = oracle.fit_round(wt, I, g, T, want_sigma=True)
        assert np.all(sig == 0)                           # every group ties -> table 0
        assert np.array_equal(Tn[1], T[1])                # table 1 never receives a weight
        ref_next = _lloyd_step_numpy(x, w, ref)
        assert np.allclose(Tn[0], ref_next, rtol=1e-12, atol=1e-12)
        if it == 0:
            km = KMeans(n_clusters=16, init=T0.reshape(-1, 1), n_init=1, max_iter=1, algorithm="lloyd", tol=0)
            km.fit(x.reshape(-1, 1), sample_weight=w)
            assert np.allclose(np.sort(km.cluster_centers_.ravel()), Tn[0], rtol=1e-6, atol=1e-6)
            # and E is the weighted inertia under the *input* table
            d = np.abs(x[:, None] - T0[None, :]).min(axis=1)
            assert np.isclose(E, np.sum(w * d * d), rtol=1e-12)
        ref = ref_next
        T = np.stack([Tn[0], T[1]])                       # keep table 1 = old table 0? no: keep both equal
        T = np.stack([Tn[0], Tn[0]])


def test_importance_metamorphic():
    W, X, g = _small(NVFP4, N=16, K=256)
    I = oracle.act_stats(X)
    s, ts = oracle.scales(W, NVFP4, g)
    wt = oracle.normalise(W, NVFP4, g, s, ts)
    T = oracle.init_quantile(wt)
    Ta, Ea, siga = oracle.fit_round(wt, I, g, T, want_sigma=True)
    # scaling I by a power of two changes neither sigma nor the tables, and scales E
    Tb_, Eb, sigb = oracle.fit_round(wt, I * np.float32(4.0), g, T, want_sigma=True)
    assert np.array_equal(siga, sigb) and np.array_equal(Ta, Tb_) and Eb == 4.0 * Ea
    # uniform I: unweighted k-means centroids
    ones = np.ones_like(I)
    Tu, Eu, sigu = oracle.fit_round(wt, ones, g, T, want_sigma=True)
    x = wt.astype(np.float64)
    for r in range(2):
        sel = np.repeat(sigu == r, g, axis=1)
        xs = x[sel]
        idx = np.abs(xs[:, None] - T[r][None, :]).argmin(axis=1)
        want = T[r].copy()
        for i in range(16):
            if np.any(idx == i):
                want[i] = xs[idx == i].mean()
        assert np.allclose(np.sort(want), Tu[r], rtol=1e-12, atol=1e-13)
    # a zero-importance column: changing its weights changes nothing in other groups or the tables
    I0 = I.copy()
    I0[5] = 0.0
    wt2 = wt.copy()
    wt2[:, 5] = -wt2[:, 5] * 0.5
    T1, E1, s1 = oracle.fit_round(wt, I0, g, T, want_sigma=True)
    T2, E2, s2 = oracle.fit_round(wt2, I0, g, T, want_sigma=True)
    assert np.array_equal(s1, s2) and np.array_equal(T1, T2) and E1 == E2


def test_empty_cell_keeps_previous_value():
    W, X, g = _small(INT4, N=8, K=128)
    I = oracle.act_stats(X)
    s, ts = oracle.scales(W, INT4, g)
    wt = oracle.normalise(W, INT4, g, s, ts)
    T = oracle.init_grid(INT4)
    T[0, 15] = 40.0                                        # nothing is nearest to 40
    T[1, 0] = -40.0
    Tn, E = oracle.fit_round(wt, I, g, T)
    assert Tn[0, 15] == 40.0 and Tn[1, 0] == -40.0


# ------------------------------------------------------------------ fixed grid => round to nearest

def _rtn_e2m1(x):
    """Textbook round-to-nearest onto the signed E2M1 values (ties toward the smaller magnitude index)."""
    mags = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    a = np.abs(x)
    k = np.abs(a[..., None] - mags).argmin(axis=-1)
    return np.sign(x) * mags[k]


def test_zero_rounds_fixed_grid_is_round_to_nearest():
    for mode in (INT4, NVFP4):
        W, X, g = _small(mode, N=16, K=256)
        I = oracle.act_stats(X)
        s, ts = oracle.scales(W, mode, g)
        wt = oracle.normalise(W, mode, g, s, ts)
        grid = oracle.init_grid(mode)[0]
        T = np.stack([grid, grid])                        # both tables = the format's grid
        Tf, Tb = oracle.round_tables(T)
        codes, sig, E, ties = oracle.pack(wt, I, g, Tb)
        nib = np.stack([codes & 15, codes >> 4], axis=2).reshape(wt.shape)
        rec = grid[nib]
        x = wt.astype(np.float64)
        if mode == INT4:
            want = np.clip(np.round(x), -8, 7)            # round half to even
            frac_tie = np.abs(x - np.floor(x) - 0.5) < 1e-12
            assert np.array_equal(rec[~frac_tie], want[~frac_tie])
            assert np.all(np.abs(rec - x) <= 0.5 + 1e-12)
        else:
            want = _rtn_e2m1(x)
            d_want = np.abs(want - x)
            assert np.allclose(np.abs(rec - x), d_want, rtol=0, atol=1e-12)
        assert np.all(sig == 0)
        assert ties[0] == sig.size                        # identical tables: every group ties


def _bf16_table(vals):
    return synth.f32_to_bf16_bits(np.asarray(vals, dtype=np.float32))


def test_pack_counts_weights_half_way_between_two_entries():
    """ties[1] on hand-built tables: only the weights at exactly 0.5 sit half-way between two
    different entries (0 and 1) of the table their group selects."""
    far = np.arange(100, 114, dtype=np.float64)            # 14 entries nothing comes near
    T_a = np.concatenate([[0.0, 1.0], far])                # 0.5 is its midpoint
    T_b = np.concatenate([[0.0, 2.0], far])                # 0.5 is nearer to 0; its midpoint is 1
    g, K, N = 16, 64, 3
    rng = np.random.default_rng(11)
    wt = np.full((N, K), 0.25, dtype=np.float32)
    half = rng.random((N, K)) < 0.3
    wt[half] = 0.5
    I = rng.uniform(0.5, 2.0, K).astype(np.float32)
    # identical tables: every group ties in selection, table 0 is used, the half-way weights count
    codes, sig, E, ties = oracle.pack(wt, I, g, _bf16_table(np.stack([T_a, T_a])))
    assert int(ties[0]) == sig.size and np.all(sig == 0)
    assert int(ties[1]) == int(half.sum())
    nib = np.stack([codes & 15, codes >> 4], axis=2).reshape(wt.shape)
    assert np.all(nib == 0)                                # 0.25 is nearest to 0; the tie at 0.5 goes to the smaller entry
    # table 1 = T_a wins exactly in the groups that hold a weight equal to 1 (error 0 against 1
    # under T_b); elsewhere the errors are equal and table 0 = T_b stays, under which 0.5 is no tie
    wt2 = wt.copy()
    ones = np.zeros((N, K // g), dtype=bool)
    ones[0, 1] = ones[2, 0] = ones[2, 3] = True
    for n, j in zip(*np.nonzero(ones)):
        wt2[n, j * g + 5] = 1.0
        half[n, j * g + 5] = False
    codes, sig, E, ties = oracle.pack(wt2, I, g, _bf16_table(np.stack([T_b, T_a])))
    assert np.array_equal(sig.astype(bool), ones)
    want = sum(int(half[n, j * g:(j + 1) * g].sum()) for n, j in zip(*np.nonzero(ones)))
    assert want > 0 and int(ties[1]) == want
    assert int(ties[0]) == int((~ones).sum())
    # a duplicated entry is not "two different entries": a weight on it does not count
    T_d = np.concatenate([[0.0, 1.0, 1.0], far[:-1]])
    wt3 = np.full((1, g), 1.0, dtype=np.float32)
    codes, sig, E, ties = oracle.pack(wt3, I[:g], g, _bf16_table(np.stack([T_d, T_d])))
    assert int(ties[1]) == 0 and np.all((codes & 15) == 1) and np.all((codes >> 4) == 1)


# ------------------------------------------------------------------ sign bit, dequant

@pytest.mark.parametrize("mode", [INT4, NVFP4])
def test_sign_bit_round_trip_and_dequant(mode):
    W, X, g = _small(mode, N=16, K=256)
    r = oracle.fit_layer(W, mode, g, 4, X=X, init="quantile")
    s, sig = r["scales"], r["sigma"]
    top = 15 if mode == INT4 else 7
    assert np.array_equal(s >> top, sig)
    mag = s & ((1 << top) - 1)
    assert np.array_equal(mag, r["scales_unsigned"]) and np.all(mag > 0)
    assert 0 < sig.mean() < 1
    What = oracle.dequant(r["codes"], s, r["tensor_scale"], r["T_bf16"], mode, g)
    # independent numpy restatement of Eq. 5
    Tv = synth.bf16_bits_to_f32(r["T_bf16"])
    nib = np.stack([r["codes"] & 15, r["codes"] >> 4], axis=2).reshape(W.shape)
    if mode == INT4:
        sv = synth.bf16_bits_to_f32(mag)
    else:
        sv = (mag.view(ml_dtypes.float8_e4m3fn).astype(np.float32) * r["tensor_scale"][0]).astype(np.float32)
    sel = np.repeat(sig, g, axis=1)
    want = (Tv[sel, nib] * np.repeat(sv, g, axis=1)).astype(np.float32)
    assert np.array_equal(What, synth.f32_to_bf16_bits(want))
    # the codes are nearest-entry indices under the chosen table: |w~ - T[c]| is minimal
    x = r["wt"].astype(np.float64)
    dist = np.abs(x - Tv[sel, nib].astype(np.float64))
    best = np.abs(x[..., None] - Tv.astype(np.float64)[sel]).min(axis=-1)
    assert np.array_equal(dist, best)
    # quantisation improved on the fixed grid: E_final below the RTN objective
    grid = oracle.init_grid(mode)[0]
    E_rtn = oracle.objective(r["wt"], r["I"], g, np.stack([grid, grid]))
    assert r["E_final"] < E_rtn
    # weight-domain error agrees with a direct evaluation
    Eo = oracle.output_error(W, r["codes"], s, r["tensor_scale"], r["T_bf16"], r["I"], mode, g)
    w = synth.bf16_bits_to_f32(W).astype(np.float64)
    direct = np.sum(r["I"].astype(np.float64)[None, :] * (w - Tv[sel, nib].astype(np.float64) * np.repeat(sv, g, axis=1).astype(np.float64)) ** 2)
    assert np.isclose(Eo, direct, rtol=1e-12)


def test_thread_count_does_not_change_results():
    W, X, g = _small(NVFP4, N=33, K=256)
    oracle.set_threads(1)
    a = oracle.fit_layer(W, NVFP4, g, 3, X=X)
    oracle.set_threads(4)
    b = oracle.fit_layer(W, NVFP4, g, 3, X=X)
    oracle.set_threads(oracle.max_threads())
    assert np.array_equal(a["T"], b["T"]) and np.array_equal(a["trace"], b["trace"])
    assert np.array_equal(a["codes"], b["codes"])


def test_config1_golden_regression():
    """The stored values were written by tests/golden/make_golden.py, which calls only the oracle."""
    import json
    gold = json.load(open(os.path.join(GOLDEN, "cfg1_oracle.json")))
    c = synth.config1()
    r = oracle.fit_layer(c["W"], c["mode"], c["group"], c["rounds"], X=c["X"], init="grid")
    assert np.allclose(r["T"].ravel(), gold["T"], rtol=1e-13)
    assert np.allclose(r["trace"], gold["trace"], rtol=1e-13)
    assert [int(v) for v in r["T_bf16"].ravel()] == gold["T_bf16"]
    assert int(r["sigma"].sum()) == gold["sigma_ones"] and int(r["ties"][0]) == 0
    import zlib
    assert zlib.crc32(r["codes"].tobytes()) == gold["codes_crc32"]
