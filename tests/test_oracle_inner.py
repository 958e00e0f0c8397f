"""Pins for the oracle's inner k-means refinement (Algorithm 1's table update step with
n_inner > 1): each is fixed by the mathematics or by an independent numpy / scikit-learn
routine, not by the oracle itself."""
import numpy as np
import pytest

import oracle
from paper_2605_08692_b200 import synth

INT4, NVFP4 = oracle.INT4, oracle.NVFP4


def _case(mode, N=24, K=256, T=64, seed=5, name="inner"):
    W = synth.weights(N, K, seed, name + "/W", outlier_frac=0.02)
    X = synth.activations(T, K, seed, name + "/X", kind="lognormal", massive_frac=0.01)
    g = 128 if mode == INT4 else 16
    I = oracle.act_stats(X)
    s, ts = oracle.scales(W, mode, g)
    wt = oracle.normalise(W, mode, g, s, ts)
    return W, X, I, wt, g


def _frozen_objective(wt, I, g, sig, T):
    """sum over weights of I (x - nearest entry of T_sigma)^2, brute force in numpy."""
    x = wt.astype(np.float64)
    w = np.broadcast_to(I.astype(np.float64), x.shape)
    sel = np.repeat(sig.astype(bool), g, axis=1)
    E = 0.0
    for r in range(2):
        m = sel == bool(r)
        d = np.abs(x[m][:, None] - T[r][None, :]).min(axis=1)
        E += np.sum(w[m] * d * d)
    return E


@pytest.mark.parametrize("mode", [INT4, NVFP4])
def test_fused_round_equals_assign_then_one_inner_update_then_sort(mode):
    """With n_inner = 1 the cells of the update are the nearest-entry indices of the assignment
    step, so the one-pass round and the three separate steps give the same tables."""
    _, _, I, wt, g = _case(mode)
    T = oracle.init_quantile(wt)
    for _ in range(3):
        Tf, Ef, sf = oracle.fit_round(wt, I, g, T, want_sigma=True)
        Tc, Ec, sc = oracle.outer_iteration(wt, I, g, T, 1)
        assert np.array_equal(sf, sc)
        assert Ef == Ec
        assert np.allclose(Tf, Tc, rtol=1e-14, atol=0)
        T = Tf


@pytest.mark.parametrize("mode", [INT4, NVFP4])
def test_inner_update_is_a_weighted_lloyd_step_per_table(mode):
    """Brute force: every entry becomes the weighted mean of the weights (of its table's groups)
    whose nearest entry it is; an entry nothing is nearest to keeps its value."""
    _, _, I, wt, g = _case(mode, N=12, K=256)
    T = oracle.init_quantile(wt)
    T[0, 15] = 50.0                                      # never nearest
    sig, _ = oracle.assign(wt, I, g, T)
    assert 0 < sig.mean() < 1
    Tn = oracle.inner_update(wt, I, g, sig, T)
    x = wt.astype(np.float64)
    w = np.broadcast_to(I.astype(np.float64), x.shape)
    sel = np.repeat(sig.astype(bool), g, axis=1)
    for r in range(2):
        m = sel == bool(r)
        xs, ws = x[m], w[m]
        idx = np.abs(xs[:, None] - T[r][None, :]).argmin(axis=1)
        for i in range(16):
            k = idx == i
            if ws[k].sum() > 0:
                assert np.isclose(Tn[r, i], np.sum(ws[k] * xs[k]) / ws[k].sum(), rtol=1e-12, atol=1e-14)
            else:
                assert Tn[r, i] == T[r, i]
    assert Tn[0, 15] == 50.0


def test_inner_iterations_match_sklearn_weighted_kmeans():
    """All groups on table 0 (sigma forced to 0): n inner iterations are n Lloyd iterations of
    one weighted 1-D k-means, which scikit-learn runs from the same start."""
    from sklearn.cluster import KMeans
    _, _, I, wt, g = _case(INT4, N=16, K=256)
    sig = np.zeros((16, 256 // g), dtype=np.uint8)
    T0 = np.linspace(-6.5, 6.5, 16)
    T = np.stack([T0, T0 + 0.25])
    n = 4
    Tn = T.copy()
    for _ in range(n):
        Tn = oracle.inner_update(wt, I, g, sig, Tn)
    assert np.array_equal(Tn[1], T[1])                   # table 1 has no weights: untouched
    x = wt.astype(np.float64).ravel()
    w = np.tile(I.astype(np.float64), wt.shape[0])
    km = KMeans(n_clusters=16, init=T0.reshape(-1, 1), n_init=1, max_iter=n, algorithm="lloyd", tol=0)
    km.fit(x.reshape(-1, 1), sample_weight=w)
    assert np.allclose(np.sort(km.cluster_centers_.ravel()), np.sort(Tn[0]), rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("mode", [INT4, NVFP4])
def test_inner_iterations_never_raise_the_frozen_objective_and_keep_order(mode):
    """Lloyd: with the selection frozen each inner iteration lowers (or keeps) the weighted error;
    1-D centroid updates keep an ascending table ascending, so the final sort moves nothing
    unless entries coincide."""
    _, _, I, wt, g = _case(mode, N=32, K=512)
    T = oracle.init_quantile(wt)
    sig, E = oracle.assign(wt, I, g, T)
    prev = _frozen_objective(wt, I, g, sig, T)
    assert np.isclose(prev, E, rtol=1e-12)               # assignment objective = frozen objective at the start
    for _ in range(6):
        T = oracle.inner_update(wt, I, g, sig, T)
        cur = _frozen_objective(wt, I, g, sig, T)
        assert cur <= prev * (1 + 1e-12)
        assert np.all(np.diff(T, axis=1) >= 0)
        prev = cur
    assert np.array_equal(oracle.sort_tables(T), T)


@pytest.mark.parametrize("mode,n_inner", [(INT4, 3), (NVFP4, 10)])
def test_outer_objective_is_monotone_with_inner_refinement(mode, n_inner):
    W, X, I, wt, g = _case(mode, N=32, K=512)
    r = oracle.fit_layer(W, mode, g, 5, X=X, init="quantile", n_inner=n_inner)
    tr = r["trace"]
    assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-12)) and tr[-1] < tr[0]
    assert oracle.objective(wt, I, g, r["T"]) <= tr[-1] * (1 + 1e-12)
    # more inner iterations refine further within the same outer budget's first step
    r1 = oracle.fit_layer(W, mode, g, 1, X=X, init="quantile", n_inner=1)
    rn = oracle.fit_layer(W, mode, g, 1, X=X, init="quantile", n_inner=n_inner)
    assert oracle.objective(wt, I, g, rn["T"]) <= oracle.objective(wt, I, g, r1["T"]) * (1 + 1e-9)


def test_unsorted_table_ties_go_to_the_smaller_entry():
    """Between inner iterations a table may be out of index order (an entry that coincided with
    its neighbour keeps its value while the neighbour moves past it); cells depend on the entries'
    values only, so relabelling the table does not change the updated set of values."""
    _, _, I, wt, g = _case(INT4, N=8, K=256)
    T = oracle.init_grid(INT4)
    sig, _ = oracle.assign(wt, I, g, T)
    perm = np.array([3, 0, 1, 2, 7, 6, 5, 4, 8, 9, 10, 11, 15, 14, 13, 12])
    Tp = T.copy()
    Tp[0] = T[0][perm]
    a = oracle.inner_update(wt, I, g, sig, T)
    b = oracle.inner_update(wt, I, g, sig, Tp)
    assert np.array_equal(a[0][perm], b[0]) and np.array_equal(a[1], b[1])
    # an exact midpoint goes to the smaller entry whatever its index: one weight at 0.5 between
    # entries 0 and 1, everything else far away
    x = np.full((1, 128), 0.5, dtype=np.float32)
    I1 = np.ones(128, dtype=np.float32)
    s0 = np.zeros((1, 1), dtype=np.uint8)
    for Tt in (np.array([0.0, 1.0] + [100.0 + i for i in range(14)]), np.array([1.0, 0.0] + [100.0 + i for i in range(14)])):
        out = oracle.inner_update(x, I1, 128, s0, np.stack([Tt, Tt]))
        assert sorted(out[0][:2]) == [0.5, 1.0]          # the entry at 0 moved to 0.5, the entry at 1 stayed
