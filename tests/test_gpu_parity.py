"""Parity of the CUDA library (called through its C ABI) against the CPU oracle, element by
element on the same seeded inputs.  Bars: bit-exact for scales, start tables, packed codes,
selection bits and dequantised weights; 1e-6 relative for importances; 1e-5 relative for the
fitted tables (|dT| <= 1e-5 * max(|T|, 1e-3 * range)); 1e-4 relative for the weighted error."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08692_b200 import binding, build, synth

pytestmark = pytest.mark.gpu
INT4, NVFP4 = 0, 1
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def dev_bf16(a):
    return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)


def host(t):
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.uint16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def table_close(got, want, rel=1e-5):
    got = np.asarray(got, dtype=np.float64).reshape(2, 16)
    want = np.asarray(want, dtype=np.float64).reshape(2, 16)
    rng = want.max() - want.min()
    tol = rel * np.maximum(np.abs(want), 1e-3 * rng)
    return np.all(np.abs(got - want) <= tol), float(np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-3 * rng)))


def layer(mode, N, K, T=64, seed=11, name="par", dist="normal"):
    W = synth.weights(N, K, seed, f"{name}/W", outlier_frac=0.01, dist=dist)
    X = synth.activations(T, K, seed, f"{name}/X", kind="lognormal", massive_frac=0.005)
    return W, X


# ------------------------------------------------------------------ a1 act_stats

@pytest.mark.parametrize("T,K", [(1, 8), (7, 256), (300, 520), (1024, 4096), (333, 14336)])
def test_act_stats(T, K):
    X = synth.activations(T, K, 2, f"act/{T}x{K}", kind="loguniform", massive_frac=0.01)
    want = oracle.act_stats(X)
    Xd = dev_bf16(X)
    I = torch.empty(K, dtype=torch.float32, device=DEV)
    ws = binding.alloc_workspace(NVFP4, 1, K)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.act_stats(Xd, I, ws, dev_status=st)
    got = host(I)
    assert np.allclose(got, want, rtol=1e-6, atol=0)
    assert np.mean(got == want) > 0.999          # double accumulation: bit-equal but for rounding order
    assert int(st.item()) == 0
    # streaming in two chunks with accumulate = 1
    if T >= 2:
        h = T // 2
        binding.act_stats(Xd[:h], I, ws)
        binding.act_stats(Xd[h:], I, ws, accumulate=True)
        assert np.allclose(host(I), want, rtol=1e-6, atol=0)


def test_act_stats_strided_and_nonfinite():
    X = synth.activations(40, 512, 2, "act/strided", kind="loguniform")
    Xd = dev_bf16(X)
    I = torch.empty(256, dtype=torch.float32, device=DEV)
    ws = binding.alloc_workspace(NVFP4, 1, 512)
    binding.act_stats(Xd[:, 256:], I, ws)         # ldx = 512, K = 256
    assert np.allclose(host(I), oracle.act_stats(np.ascontiguousarray(X[:, 256:])), rtol=1e-6)
    X[3, 300] = 0x7F80                           # +inf
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.act_stats(dev_bf16(X)[:, 256:], I, ws, dev_status=st)
    assert int(st.item()) & binding.DEV_NONFINITE


# ------------------------------------------------------------------ a2 scales, a3 init

def run_fit(W, mode, I, rounds, init, want_trace=True, T01_init=None, n_inner=1):
    Wd = dev_bf16(W)
    Id = torch.from_numpy(np.ascontiguousarray(I)).to(DEV)
    t0 = None if T01_init is None else torch.from_numpy(np.asarray(T01_init, dtype=np.float32)).to(DEV)
    return binding.quantize_layer(Wd, mode, I=Id, n_outer=rounds, init=init, want_trace=want_trace, T01_init=t0,
                                  n_inner=n_inner)


@pytest.mark.parametrize("mode", [INT4, NVFP4])
@pytest.mark.parametrize("N,K", [(1, 128), (5, 384), (33, 512), (64, 1280)])
def test_scales_and_start_tables_bit_exact(mode, N, K):
    g = 128 if mode == INT4 else 16
    W, X = layer(mode, N, K, name=f"sc{mode}/{N}x{K}")
    W[0, 0:g] = 0                                                           # all-zero group
    if K >= 2 * g:
        W[N - 1, g:2 * g] = synth.f32_to_bf16_bits(np.full(g, 3e-12, np.float32))   # far below the tensor scale
    I = oracle.act_stats(X)
    s, ts = oracle.scales(W, mode, g)
    wt = oracle.normalise(W, mode, g, s, ts)
    for init, Tw in ((binding.INIT_QUANTILE, oracle.init_quantile(wt)), (binding.INIT_GRID, oracle.init_grid(mode))):
        r = run_fit(W, mode, I, 0, init)
        assert np.array_equal(host(r["scales_pos"]), s)
        assert host(r["tensor_scale"])[0] == ts[0]
        assert np.array_equal(host(r["T01"]), Tw.astype(np.float32)), (init, host(r["T01"]), Tw)
        assert int(r["status"].item()) == 0


@pytest.mark.parametrize("mode", [INT4, NVFP4])
@pytest.mark.parametrize("kind", ["constant", "three_values", "two_spikes_large"])
def test_quantile_start_tables_on_degenerate_value_sets(mode, kind):
    """Order statistics when (nearly) all normalised weights coincide: every requested rank falls
    into one or two histogram bins, whose lists are far longer than what the selection keeps in
    registers, all keys share all (or all but a few) bits, and neighbouring ranks have equal keys."""
    g = 128 if mode == INT4 else 16
    rng = np.random.default_rng(7)
    if kind == "constant":
        N, K = 64, 1280
        vals = np.full((N, K), 0.5, np.float32)
    elif kind == "three_values":
        N, K = 96, 1024
        vals = rng.choice(np.array([-0.25, 0.125, 0.5], np.float32), size=(N, K))
    else:
        N, K = 257, 4096                              # ~1 M values on a handful of distinct w~
        vals = rng.choice(np.array([-1.0, 1.0, 0.0], np.float32), size=(N, K), p=[0.495, 0.495, 0.01])
    W = synth.f32_to_bf16_bits(vals)
    I = np.ones(K, np.float32)
    s, ts = oracle.scales(W, mode, g)
    wt = oracle.normalise(W, mode, g, s, ts)
    want = oracle.init_quantile(wt).astype(np.float32)
    r = run_fit(W, mode, I, 0, binding.INIT_QUANTILE)
    assert np.array_equal(host(r["T01"]), want), (host(r["T01"]), want)
    # and a round from there stays on the oracle's path (many duplicate entries, empty cells)
    o = oracle.fit_layer(W, mode, g, 2, I=I)
    r2 = run_fit(W, mode, I, 2, binding.INIT_QUANTILE)
    assert table_close(host(r2["T01"]), o["T"])[0]


def test_quantile_start_when_a_bin_does_not_fit_the_candidate_list():
    """The candidate list of the quantile start is bounded.  A bin whose weights do not fit is
    still answered exactly when they all share one value (constant and sparse layers); when they
    do not, AAAC_DEV_SCRATCH is set (and the host-buffer call returns AAAC_ERR_WORKSPACE), and a
    workspace of the full size never falls short."""
    # (a) the default capacity on a layer whose weights take three values (each bin far over capacity)
    rng = np.random.default_rng(5)
    N, K = 512, 4096
    vals = rng.choice(np.array([-1.0, 0.0, 1.0], np.float32), size=(N, K), p=[0.3, 0.4, 0.3])
    vals[:, ::16] = 1.0                                     # every group's largest magnitude: one scale for all
    W = synth.f32_to_bf16_bits(vals)
    I = np.ones(K, np.float32)
    for mode in (INT4, NVFP4):
        g = 128 if mode == INT4 else 16
        s, ts = oracle.scales(W, mode, g)
        want = oracle.init_quantile(oracle.normalise(W, mode, g, s, ts)).astype(np.float32)
        assert binding.workspace_bytes(mode, N, K) < W.nbytes * 4      # bounded: the full list alone would be 4 N K bytes
        r = run_fit(W, mode, I, 0, binding.INIT_QUANTILE)
        assert int(r["status"].item()) == 0
        assert np.array_equal(host(r["T01"]), want), (host(r["T01"]), want)
    # (b) a forced small capacity on an ordinary layer: several values per bin cannot be resolved
    W2, X2 = layer(NVFP4, 300, 768, name="qcap")
    I2 = oracle.act_stats(X2)
    ref = run_fit(W2, NVFP4, I2, 2, binding.INIT_QUANTILE)
    try:
        binding.debug_quantile_cap(1000)
        bad = run_fit(W2, NVFP4, I2, 2, binding.INIT_QUANTILE)
        torch.cuda.synchronize()
        assert int(bad["status"].item()) & binding.DEV_SCRATCH
    finally:
        binding.debug_quantile_cap(0)
    # (c) the full-size workspace and the default one give the same start tables and fit
    Wd = dev_bf16(W2)
    Id = torch.from_numpy(I2).to(DEV)
    full = binding.quantize_layer(Wd, NVFP4, I=Id, n_outer=2, init=binding.INIT_QUANTILE,
                                  ws=binding.alloc_workspace(NVFP4, 300, 768, full=True))
    assert int(full["status"].item()) == 0
    assert torch.equal(full["T01"], ref["T01"]) and torch.equal(full["codes"], ref["codes"])


def test_user_tables_and_nonfinite_weights():
    W, X = layer(INT4, 16, 256, name="user")
    I = oracle.act_stats(X)
    T0 = np.linspace(-7, 7, 32, dtype=np.float32).reshape(2, 16)
    r = run_fit(W, INT4, I, 0, binding.INIT_USER, T01_init=T0)
    assert np.array_equal(host(r["T01"]), T0)
    W[2, 5] = 0x7FC0                              # NaN
    r = run_fit(W, INT4, I, 0, binding.INIT_GRID)
    assert int(r["status"].item()) & binding.DEV_NONFINITE
    W2, _ = layer(NVFP4, 16, 256, name="user2")
    W2[1, 7] = 0xFF80                             # -inf
    r = run_fit(W2, NVFP4, I, 0, binding.INIT_GRID)
    assert int(r["status"].item()) & binding.DEV_NONFINITE


# ------------------------------------------------------------------ a4-a6 fit rounds

def check_fit(W, X, mode, rounds, init_name, rel_T=1e-5, rel_E=1e-4, n_inner=1):
    g = 128 if mode == INT4 else 16
    o = oracle.fit_layer(W, mode, g, rounds, X=X, init=init_name, n_inner=n_inner)
    init = dict(quantile=binding.INIT_QUANTILE, grid=binding.INIT_GRID)[init_name]
    r = run_fit(W, mode, o["I"], rounds, init, n_inner=n_inner)
    ok, worst = table_close(host(r["T01"]), o["T"], rel_T)
    assert ok, f"tables differ: worst {worst:.3e}"
    if rounds:
        tr = host(r["trace"])[:rounds]
        assert np.allclose(tr, o["trace"], rtol=rel_E, atol=0), (tr, o["trace"])
        assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-6))
    return o, r, worst


def check_pack(W, mode, o, r):
    """GPU pack on the oracle's tables / scales / I must reproduce the oracle's bits."""
    g = 128 if mode == INT4 else 16
    N, K = W.shape
    Wd = dev_bf16(W)
    Id = torch.from_numpy(o["I"]).to(DEV)
    T01 = torch.from_numpy(o["T_f32"]).to(DEV)
    sc = torch.from_numpy(o["scales_unsigned"].view(np.int16) if mode == INT4 else o["scales_unsigned"]).to(DEV)
    if mode == INT4:
        sc = sc.view(torch.uint16)
    ts = torch.from_numpy(o["tensor_scale"]).to(DEV)
    Tb = torch.empty(2, 16, dtype=torch.uint16, device=DEV)
    codes = torch.empty(N, K // 2, dtype=torch.uint8, device=DEV)
    err = torch.zeros(2, dtype=torch.float64, device=DEV)
    stats = torch.zeros(4, dtype=torch.int64, device=DEV)
    ws = binding.alloc_workspace(mode, N, K)
    binding.pack(Wd, mode, I=Id, T01=T01, T01_bf16=Tb, scales=sc, tensor_scale=ts, codes=codes, ws=ws, err_out=err,
                 stats=stats)
    assert np.array_equal(host(Tb), o["T_bf16"])
    assert np.array_equal(host(sc), o["scales"]), "scales / selection bits differ"
    assert np.array_equal(host(codes), o["codes"]), "packed codes differ"
    st = host(stats)
    assert st[0] == o["ties"][0] and st[1] == o["ties"][1]
    e = host(err)
    assert np.isclose(e[0], o["E_final"], rtol=1e-4)
    Eo = oracle.output_error(W, o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"], o["I"], mode, g)
    assert np.isclose(e[1], Eo, rtol=1e-4)
    # dequant, bit-exact
    What = torch.empty(N, K, dtype=torch.bfloat16, device=DEV)
    binding.dequant(codes, sc, ts, Tb, mode, What)
    assert np.array_equal(host(What), oracle.dequant(o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"], mode, g))
    return st


def check_end_to_end_bits(r, o, label, sel=False):
    """End to end: the library's own fit must give the oracle's BF16 tables -- the entries that
    land on the other side of a BF16 rounding boundary are counted, printed and required to be
    none on the seeded inputs -- and from equal tables the same packed bits follow."""
    got, want = host(r["T01_bf16"]), o["T_bf16"]
    differ = int(np.sum(got != want))
    print(f"{label}: BF16 table entries that differ from the oracle's: {differ} of {want.size}")
    assert differ == 0, f"{label}: {differ} BF16 table entries straddle a rounding boundary: {got} vs {want}"
    assert np.array_equal(host(r["codes"]), o["codes"]), f"{label}: packed codes differ end to end"
    if sel:
        assert np.array_equal(host(r["sigma_bits"]), o["sigma_bits"]), f"{label}: selection bits differ end to end"
        assert np.array_equal(host(r["scales"]), o["scales_unsigned"])
    else:
        assert np.array_equal(host(r["scales"]), o["scales"]), f"{label}: scales / selection bits differ end to end"


@pytest.mark.parametrize("mode,init", [(INT4, "grid"), (INT4, "quantile"), (NVFP4, "quantile"), (NVFP4, "grid")])
@pytest.mark.parametrize("N,K", [(3, 256), (70, 640), (257, 1024)])
def test_fit_and_pack_small(mode, init, N, K):
    W, X = layer(mode, N, K, name=f"fit{mode}{init}/{N}x{K}")
    o, r, worst = check_fit(W, X, mode, 6, init)
    check_pack(W, mode, o, r)
    check_end_to_end_bits(r, o, f"small {mode} {init} {N}x{K}")


def test_config1_end_to_end():
    c = synth.config1()
    o, r, worst = check_fit(c["W"], c["X"], c["mode"], c["rounds"], "grid")
    st = check_pack(c["W"], c["mode"], o, r)
    assert st[0] == 0                              # no exact selection ties on the seeded config
    assert np.array_equal(host(r["T01_bf16"]), o["T_bf16"])
    assert np.array_equal(host(r["codes"]), o["codes"]) and np.array_equal(host(r["scales"]), o["scales"])
    # importance from X inside aaac_fit_layer
    Wd, Xd = dev_bf16(c["W"]), dev_bf16(c["X"])
    r2 = binding.quantize_layer(Wd, c["mode"], X=Xd, n_outer=c["rounds"], init=binding.INIT_GRID, want_trace=True)
    assert np.array_equal(host(r2["T01"]), host(r["T01"]))


def test_student_t_weights_nvfp4():
    W, X = layer(NVFP4, 96, 1792, name="qwen", dist="student5")
    o, r, worst = check_fit(W, X, NVFP4, 8, "quantile")
    check_pack(W, NVFP4, o, r)


def test_degenerate_identical_tables_and_empty_cells():
    W, X = layer(INT4, 24, 256, name="degen")
    I = oracle.act_stats(X)
    g = 128
    T0 = np.linspace(-6.5, 6.5, 16)
    T = np.stack([T0, T0]).astype(np.float32)
    # one round from identical tables: every group ties exactly, table 1 never receives a weight
    o = oracle.fit_layer(W, INT4, g, 1, I=I, init="user", T_init=T)
    r = run_fit(W, INT4, I, 1, binding.INIT_USER, T01_init=T)
    ok, worst = table_close(host(r["T01"]), o["T"])
    assert ok, worst
    assert np.array_equal(host(r["T01"])[1], T[1])
    # zero rounds: pack with identical tables, every group an exact tie -> sigma = 0 everywhere
    o0 = oracle.fit_layer(W, INT4, g, 0, I=I, init="user", T_init=T)
    r0 = run_fit(W, INT4, I, 0, binding.INIT_USER, T01_init=T)
    st = check_pack(W, INT4, o0, r0)
    assert st[0] == W.size // g
    assert np.all(host(r0["scales"]) >> 15 == 0)
    # and three rounds stay on the oracle's trajectory
    o = oracle.fit_layer(W, INT4, g, 3, I=I, init="user", T_init=T)
    r = run_fit(W, INT4, I, 3, binding.INIT_USER, T01_init=T)
    assert table_close(host(r["T01"]), o["T"])[0]
    check_pack(W, INT4, o, r)
    # an entry nothing is nearest to keeps its value
    T2 = oracle.init_grid(INT4).astype(np.float32)
    T2[0, 15] = 40.0
    T2[1, 0] = -40.0
    o2 = oracle.fit_layer(W, INT4, g, 2, I=I, init="user", T_init=T2)
    r2 = run_fit(W, INT4, I, 2, binding.INIT_USER, T01_init=T2)
    assert host(r2["T01"])[0, 15] == 40.0 and host(r2["T01"])[1, 0] == -40.0
    assert table_close(host(r2["T01"]), o2["T"])[0]


def test_runs_are_bitwise_reproducible():
    W, X = layer(NVFP4, 200, 768, name="repro")
    I = oracle.act_stats(X)
    a = run_fit(W, NVFP4, I, 5, binding.INIT_QUANTILE)
    b = run_fit(W, NVFP4, I, 5, binding.INIT_QUANTILE)
    for k in ("T01", "codes", "scales", "trace", "err"):
        assert torch.equal(a[k], b[k]), k


def test_host_buffer_entry_point_matches_device_path():
    W, X = layer(NVFP4, 64, 512, T=128, name="hostpath")
    N, K = W.shape
    Wh = torch.from_numpy(W.view(np.int16)).pin_memory()
    Xh = torch.from_numpy(X.view(np.int16)).pin_memory()
    T01 = torch.empty(2, 16, dtype=torch.float32).pin_memory()
    Tb = torch.empty(2, 16, dtype=torch.int16).pin_memory()
    sc = torch.empty(N, K // 16, dtype=torch.uint8).pin_memory()
    ts = torch.empty(1, dtype=torch.float32).pin_memory()
    codes = torch.empty(N, K // 2, dtype=torch.uint8).pin_memory()
    err = torch.empty(2, dtype=torch.float64).pin_memory()
    ws = torch.empty(binding.host_workspace_bytes(NVFP4, N, K, X.shape[0]), dtype=torch.uint8, device=DEV)
    binding.quantize_layer_host(Wh, Xh, NVFP4, n_outer=4, init=binding.INIT_QUANTILE, T01_host=T01, T01_bf16_host=Tb,
                                scales_host=sc, tensor_scale_host=ts, codes_host=codes, err_out_host=err, ws=ws)
    r = binding.quantize_layer(dev_bf16(W), NVFP4, X=dev_bf16(X), n_outer=4, init=binding.INIT_QUANTILE)
    torch.cuda.synchronize()
    assert np.array_equal(T01.numpy(), host(r["T01"]))
    assert np.array_equal(codes.numpy(), host(r["codes"]))
    assert np.array_equal(sc.numpy(), host(r["scales"]))
    assert np.array_equal(err.numpy(), host(r["err"]))
    o = oracle.fit_layer(W, NVFP4, 16, 4, X=X)
    assert table_close(T01.numpy(), o["T"])[0]
    # the call that only enqueues: two layers on two streams, then one synchronisation
    outs = []
    for k in range(2):
        st_ = torch.cuda.Stream()
        bufs = dict(T01=torch.empty(2, 16, dtype=torch.float32).pin_memory(), Tb=torch.empty(2, 16, dtype=torch.int16).pin_memory(),
                    sc=torch.empty(N, K // 16, dtype=torch.uint8).pin_memory(), ts=torch.empty(1, dtype=torch.float32).pin_memory(),
                    codes=torch.empty(N, K // 2, dtype=torch.uint8).pin_memory(), err=torch.empty(2, dtype=torch.float64).pin_memory(),
                    status=torch.ones(1, dtype=torch.int32).pin_memory(),
                    ws=torch.empty(binding.host_workspace_bytes(NVFP4, N, K, X.shape[0]), dtype=torch.uint8, device=DEV))
        with torch.cuda.stream(st_):
            binding.quantize_layer_host_async(Wh, Xh, NVFP4, n_outer=4, init=binding.INIT_QUANTILE, T01_host=bufs["T01"],
                                              T01_bf16_host=bufs["Tb"], scales_host=bufs["sc"], tensor_scale_host=bufs["ts"],
                                              codes_host=bufs["codes"], err_out_host=bufs["err"], status_host=bufs["status"],
                                              ws=bufs["ws"])
        outs.append(bufs)
    torch.cuda.synchronize()
    for bufs in outs:
        assert int(bufs["status"].item()) == 0
        assert np.array_equal(bufs["codes"].numpy(), codes.numpy()) and np.array_equal(bufs["T01"].numpy(), T01.numpy())


def test_fit_wait_runs_out_and_is_reported():
    """The blocks of the fit-rounds kernel wait for each other's sums once per pass, with a poll
    limit.  Made to run out (the totals are asked to show one more block than exists; a thousand
    polls), every block gives up within a fraction of a millisecond, the kernel returns, the device
    status word carries AAAC_DEV_TIMEOUT, the host-buffer call returns AAAC_ERR_TIMEOUT -- and the
    next ordinary call on the same workspace is bit for bit what it was before."""
    W, X = layer(NVFP4, 300, 768, T=128, name="timeout")
    N, K = W.shape
    Wd, Xd = dev_bf16(W), dev_bf16(X)
    ws = binding.alloc_workspace(NVFP4, N, K, X.shape[0])
    good = binding.quantize_layer(Wd, NVFP4, X=Xd, n_outer=3, init=binding.INIT_QUANTILE, ws=ws, want_trace=True)
    torch.cuda.synchronize()
    assert int(good["status"].item()) == 0
    try:
        binding.debug_fit_wait(1, 1000)
        bad = binding.quantize_layer(Wd, NVFP4, X=Xd, n_outer=3, init=binding.INIT_QUANTILE, ws=ws, want_trace=True)
        torch.cuda.synchronize()
        assert int(bad["status"].item()) & binding.DEV_TIMEOUT
        # the host-buffer entry point turns the status bit into an error code
        Wh = torch.from_numpy(W.view(np.int16)).pin_memory()
        Xh = torch.from_numpy(X.view(np.int16)).pin_memory()
        hws = torch.empty(binding.host_workspace_bytes(NVFP4, N, K, X.shape[0]), dtype=torch.uint8, device=DEV)
        with pytest.raises(binding.AaacError, match="status 10"):
            binding.quantize_layer_host(Wh, Xh, NVFP4, n_outer=2, init=binding.INIT_QUANTILE,
                                        T01_host=torch.empty(2, 16, dtype=torch.float32).pin_memory(),
                                        T01_bf16_host=torch.empty(2, 16, dtype=torch.int16).pin_memory(),
                                        scales_host=torch.empty(N, K // 16, dtype=torch.uint8).pin_memory(),
                                        tensor_scale_host=torch.empty(1, dtype=torch.float32).pin_memory(),
                                        codes_host=torch.empty(N, K // 2, dtype=torch.uint8).pin_memory(),
                                        err_out_host=torch.empty(2, dtype=torch.float64).pin_memory(), ws=hws)
    finally:
        binding.debug_fit_wait(0, 0)
    again = binding.quantize_layer(Wd, NVFP4, X=Xd, n_outer=3, init=binding.INIT_QUANTILE, ws=ws, want_trace=True)
    torch.cuda.synchronize()
    assert int(again["status"].item()) == 0
    for k in ("T01", "codes", "scales", "trace", "err"):
        assert torch.equal(again[k], good[k]), k


# ------------------------------------------------------------------ several layers in one call

def run_fit_batch(cases, mode, rounds, init, n_inner=1, sel_group=None):
    """aaac_fit_layers on a list of (W, I) cases; returns per layer the fitted tables, scales, trace."""
    g = 128 if mode == INT4 else 16
    descs, keep = [], []
    for W, I in cases:
        N, K = W.shape
        d = dict(W=dev_bf16(W), I=torch.from_numpy(np.ascontiguousarray(I)).to(DEV),
                 T01=torch.zeros(2, 16, dtype=torch.float32, device=DEV),
                 scales=torch.empty(N, K // g, dtype=torch.uint16 if mode == INT4 else torch.uint8, device=DEV),
                 tensor_scale=torch.ones(1, dtype=torch.float32, device=DEV),
                 err_trace=torch.zeros(max(rounds, 1), dtype=torch.float64, device=DEV),
                 ws=binding.alloc_workspace(mode, N, K))
        descs.append(d)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.fit_layers(descs, mode, n_outer=rounds, init=init, n_inner=n_inner, sel_group=sel_group, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return descs


@pytest.mark.parametrize("mode", [INT4, NVFP4])
def test_fit_layers_batch_matches_oracle_per_layer(mode):
    """Several layers of different shapes (ragged rows and columns, a one-row layer) fitted in one
    call: every layer against the oracle, like a layer fitted alone; twice for reproducibility."""
    g = 128 if mode == INT4 else 16
    shapes = [(257, 1024), (3, 256), (70, 640), (1, 128), (300, 768)]
    cases, oracles = [], []
    for i, (N, K) in enumerate(shapes):
        W, X = layer(mode, N, K, name=f"batch{mode}/{i}")
        o = oracle.fit_layer(W, mode, g, 6, X=X, init="quantile")
        cases.append((W, o["I"]))
        oracles.append(o)
    a = run_fit_batch(cases, mode, 6, binding.INIT_QUANTILE)
    b = run_fit_batch(cases, mode, 6, binding.INIT_QUANTILE)
    for i, (d, d2, o) in enumerate(zip(a, b, oracles)):
        ok, worst = table_close(host(d["T01"]), o["T"])
        assert ok, f"layer {i}: tables differ: worst {worst:.3e}"
        tr = host(d["err_trace"])[:6]
        assert np.allclose(tr, o["trace"], rtol=1e-4, atol=0)
        assert np.array_equal(host(d["scales"]), o["scales_unsigned"])
        assert torch.equal(d["T01"], d2["T01"]) and torch.equal(d["err_trace"], d2["err_trace"])
        # and the pack pass from these tables gives the oracle's bits
        W = cases[i][0]
        r = dict(T01_bf16=None)
        Tb = torch.empty(2, 16, dtype=torch.uint16, device=DEV)
        codes = torch.empty(W.shape[0], W.shape[1] // 2, dtype=torch.uint8, device=DEV)
        binding.pack(d["W"], mode, I=d["I"], T01=d["T01"], T01_bf16=Tb, scales=d["scales"], tensor_scale=d["tensor_scale"],
                     codes=codes, ws=d["ws"])
        assert np.array_equal(host(Tb), o["T_bf16"]), f"layer {i}: BF16 tables differ"
        assert np.array_equal(host(codes), o["codes"]) and np.array_equal(host(d["scales"]), o["scales"])


def test_fit_layers_more_layers_than_one_launch_takes_and_inner_refinement():
    """Eleven layers (more than one launch holds) and a batch with n_inner > 1 (run layer by layer)."""
    rng = np.random.default_rng(3)
    cases, oracles = [], []
    for i in range(11):
        N, K = int(rng.integers(1, 90)), 256 * int(rng.integers(1, 4))
        W, X = layer(NVFP4, N, K, name=f"batch11/{i}")
        o = oracle.fit_layer(W, NVFP4, 16, 3, X=X, init="grid")
        cases.append((W, o["I"]))
        oracles.append(o)
    for d, o in zip(run_fit_batch(cases, NVFP4, 3, binding.INIT_GRID), oracles):
        assert table_close(host(d["T01"]), o["T"])[0]
    cases, oracles = [], []
    for i, (N, K) in enumerate([(70, 640), (130, 512)]):
        W, X = layer(INT4, N, K, name=f"batchinner/{i}")
        o = oracle.fit_layer(W, INT4, 128, 2, X=X, init="quantile", n_inner=3, S=16)
        cases.append((W, o["I"]))
        oracles.append(o)
    for d, o in zip(run_fit_batch(cases, INT4, 2, binding.INIT_QUANTILE, n_inner=3, sel_group=16), oracles):
        assert table_close(host(d["T01"]), o["T"])[0]
        assert np.allclose(host(d["err_trace"])[:2], o["trace"], rtol=1e-4)


def carved_importance(d):
    """The importances of a layer as aaac_act_stats gives them for the X the batch call was given
    (the batch call keeps its own copy inside the layer's workspace)."""
    I = torch.empty(d["X"].shape[1], dtype=torch.float32, device=DEV)
    binding.act_stats(d["X"], I, binding.alloc_workspace(NVFP4, 8, d["X"].shape[1], d["X"].shape[0]))
    torch.cuda.synchronize()
    return I


def run_quantize_batch(cases, mode, rounds, init, sel_group=None, what_pad=0):
    """aaac_quantize_layers on a list of (W, X) cases, importances from X inside the call."""
    g = 128 if mode == INT4 else 16
    descs = []
    for W, X in cases:
        N, K = W.shape
        d = dict(W=dev_bf16(W), X=dev_bf16(X),
                 T01=torch.zeros(2, 16, dtype=torch.float32, device=DEV),
                 scales=torch.empty(N, K // g, dtype=torch.uint16 if mode == INT4 else torch.uint8, device=DEV),
                 tensor_scale=torch.ones(1, dtype=torch.float32, device=DEV),
                 err_trace=torch.zeros(max(rounds, 1), dtype=torch.float64, device=DEV),
                 ws=binding.alloc_workspace(mode, N, K, X.shape[0]),
                 T01_bf16=torch.empty(2, 16, dtype=torch.uint16, device=DEV),
                 codes=torch.empty(N, K // 2, dtype=torch.uint8, device=DEV),
                 err_out=torch.zeros(2, dtype=torch.float64, device=DEV),
                 stats=torch.zeros(4, dtype=torch.int64, device=DEV),
                 What_full=torch.full((N, K + what_pad), 7.0, dtype=torch.bfloat16, device=DEV))
        d["What"] = d["What_full"][:, :K]
        if sel_group is not None:
            d["sigma_bits"] = torch.zeros(N, K // (8 * sel_group), dtype=torch.uint8, device=DEV)
        descs.append(d)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.quantize_layers(descs, mode, n_outer=rounds, init=init, sel_group=sel_group, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return descs


@pytest.mark.parametrize("mode,sel", [(NVFP4, None), (INT4, None), (INT4, 16)])
def test_quantize_layers_whole_path_matches_oracle_per_layer(mode, sel):
    """The whole path for several layers in one call (importances from X, scales, start, rounds, pack,
    reconstruction), more layers than there are side streams: every output of every layer against the oracle."""
    g = 128 if mode == INT4 else 16
    shapes = [(257, 1024), (3, 256), (70, 640), (1, 128), (300, 768), (40, 512), (64, 256), (9, 384), (129, 256)]
    cases, oracles = [], []
    for i, (N, K) in enumerate(shapes):
        W, X = layer(mode, N, K, name=f"qbatch{mode}{sel}/{i}")
        kw = dict(S=sel) if sel else {}
        oracles.append(oracle.fit_layer(W, mode, g, 5, X=X, init="quantile", **kw))
        cases.append((W, X))
    a = run_quantize_batch(cases, mode, 5, binding.INIT_QUANTILE, sel_group=sel, what_pad=8)
    b = run_quantize_batch(cases, mode, 5, binding.INIT_QUANTILE, sel_group=sel)
    for i, (d, d2, o) in enumerate(zip(a, b, oracles)):
        label = f"quantize_layers mode {mode} S {sel} layer {i}"
        ok, worst = table_close(host(d["T01"]), o["T"])
        assert ok, f"{label}: tables differ: worst {worst:.3e}"
        assert np.allclose(host(d["err_trace"])[:5], o["trace"], rtol=1e-4, atol=0)
        check_end_to_end_bits(d, o, label, sel=bool(sel))
        assert np.isclose(host(d["err_out"])[0], o["E_final"], rtol=1e-4)
        st = host(d["stats"])
        assert st[0] == o["ties"][0] and st[1] == o["ties"][1]
        if sel:
            want = oracle.dequant_sel(o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"], o["sigma_bits"], sel, mode, g)
        else:
            want = oracle.dequant(o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"], mode, g)
        assert np.array_equal(host(d["What"].contiguous()), want), f"{label}: reconstruction differs"
        for k in ("T01", "T01_bf16", "codes", "scales", "err_out"):
            assert torch.equal(d[k], d2[k]), f"{label}: {k} differs between two calls"
        assert torch.equal(d["What"], d2["What"])
        assert bool((d["What_full"][:, o["codes"].shape[1] * 2:] == 7.0).all()), f"{label}: wrote past a row of What"


def test_quantize_layers_share_the_importances_of_a_common_input():
    """Layers of a batch that read the same activations (q, k and v of a decoder layer): the importances
    are computed once -- two kernels fewer per further layer -- and every layer still matches the oracle."""
    K = 512
    X = synth.activations(96, K, 11, "shared/X", kind="lognormal", massive_frac=0.005)
    Ws = [synth.weights(N, K, 11, f"shared/W{i}", outlier_frac=0.01) for i, N in enumerate((70, 33, 129))]
    Xd = dev_bf16(X)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def descs(shared):
        out = []
        for W in Ws:
            N = W.shape[0]
            out.append(dict(W=dev_bf16(W), X=Xd if shared else Xd.clone(),
                            T01=torch.zeros(2, 16, dtype=torch.float32, device=DEV),
                            scales=torch.empty(N, K // 16, dtype=torch.uint8, device=DEV),
                            tensor_scale=torch.ones(1, dtype=torch.float32, device=DEV),
                            ws=binding.alloc_workspace(NVFP4, N, K, X.shape[0]),
                            T01_bf16=torch.empty(2, 16, dtype=torch.uint16, device=DEV),
                            codes=torch.empty(N, K // 2, dtype=torch.uint8, device=DEV),
                            err_out=torch.zeros(2, dtype=torch.float64, device=DEV)))
        return out

    counts = {}
    for shared in (False, True):
        d = descs(shared)
        n0 = binding.launch_count()
        binding.quantize_layers(d, NVFP4, n_outer=4, init=binding.INIT_QUANTILE, dev_status=status)
        torch.cuda.synchronize()
        counts[shared] = binding.launch_count() - n0
        assert int(status.item()) == 0
        for i, (W, r) in enumerate(zip(Ws, d)):
            o = oracle.fit_layer(W, NVFP4, 16, 4, X=X, init="quantile")
            assert table_close(host(r["T01"]), o["T"])[0]
            check_end_to_end_bits(r, o, f"shared input {shared} layer {i}")
            assert np.isclose(host(r["err_out"])[0], o["E_final"], rtol=1e-4)
    assert counts[False] - counts[True] == 2 * (len(Ws) - 1), counts


def test_quantize_layers_rejects_a_bad_output_before_enqueuing_anything():
    W, X = layer(NVFP4, 16, 256, name="qbatchbad")
    good = dict(W=dev_bf16(W), I=torch.ones(256, device=DEV), T01=torch.zeros(2, 16, device=DEV),
                scales=torch.empty(16, 16, dtype=torch.uint8, device=DEV), tensor_scale=torch.ones(1, device=DEV),
                ws=binding.alloc_workspace(NVFP4, 16, 256), T01_bf16=torch.empty(2, 16, dtype=torch.uint16, device=DEV),
                codes=torch.empty(16, 128, dtype=torch.uint8, device=DEV))
    bad = dict(good, What=torch.empty(16, 260, dtype=torch.bfloat16, device=DEV)[:, :256])      # row stride not a multiple of 8
    before = binding.launch_count()
    with pytest.raises(binding.AaacError, match="status"):
        binding.quantize_layers([good, bad], NVFP4, n_outer=2, init=binding.INIT_GRID)
    assert binding.launch_count() == before


def test_fit_refuses_a_layer_of_two_to_the_32_elements():
    """The fit kernels index a layer with 32 bits: N * ldw = 2^32 is refused on the host, before the
    workspace is looked at and before anything is enqueued (the buffers here are never touched)."""
    small = torch.zeros(4096, dtype=torch.bfloat16, device=DEV)
    d = dict(W=small.as_strided((1, 4096), (4096, 1)), I=torch.ones(4096, device=DEV), T01=torch.zeros(2, 16, device=DEV),
             scales=torch.empty(256, dtype=torch.uint8, device=DEV), tensor_scale=torch.ones(1, device=DEV),
             ws=torch.empty(1 << 20, dtype=torch.uint8, device=DEV))
    arr = binding._layer_descs([d])
    arr[0].N = 1 << 20                                   # 2^20 rows of 4096: exactly 2^32 elements
    before = binding.launch_count()
    rc = binding.lib().aaac_fit_layers(arr, 1, NVFP4, 16, 16, 2, 1, binding.INIT_GRID, None, None)
    assert rc == 9, rc
    arr[0].N = (1 << 20) - 1                             # one row less: now it is the workspace that is too small
    rc = binding.lib().aaac_fit_layers(arr, 1, NVFP4, 16, 16, 2, 1, binding.INIT_GRID, None, None)
    assert rc == 5, rc
    # the pack pass has the same limit
    codes = torch.empty(4096, dtype=torch.uint8, device=DEV)
    Tb = torch.empty(2, 16, dtype=torch.uint16, device=DEV)
    args = lambda N: (d["W"].data_ptr(), N, 4096, 4096, NVFP4, 16, d["I"].data_ptr(), d["T01"].data_ptr(), Tb.data_ptr(),
                      d["scales"].data_ptr(), d["tensor_scale"].data_ptr(), codes.data_ptr(), None, None, d["ws"].data_ptr(),
                      d["ws"].numel(), None)
    assert binding.lib().aaac_pack(*args(1 << 20)) == 9
    assert binding.lib().aaac_pack(*args((1 << 20) - 1)) == 5
    assert binding.launch_count() == before


def test_fit_layers_rejects_a_bad_layer_before_enqueuing_anything():
    W, X = layer(NVFP4, 16, 256, name="batchbad")
    good = dict(W=dev_bf16(W), I=torch.ones(256, device=DEV), T01=torch.zeros(2, 16, device=DEV),
                scales=torch.empty(16, 16, dtype=torch.uint8, device=DEV), tensor_scale=torch.ones(1, device=DEV),
                ws=binding.alloc_workspace(NVFP4, 16, 256))
    bad = dict(good, ws=torch.empty(64, dtype=torch.uint8, device=DEV))       # workspace too small
    before = binding.launch_count()
    with pytest.raises(binding.AaacError, match="status 5"):
        binding.fit_layers([good, bad], NVFP4, n_outer=2, init=binding.INIT_GRID)
    assert binding.launch_count() == before


def test_config2_layers_in_one_batch_full_size():
    """The benchmark's step as the benchmark makes it -- its three layers through aaac_quantize_layers in one
    call, importances from X, scales, quantile start, the 20 rounds of all three in one launch, pack and
    reconstruction -- with every output of every layer against the whole-layer oracle."""
    names = ("q_proj", "gate_proj", "down_proj")
    cases, oracles = [], []
    for which in names:
        c = synth.config2_layer(which)
        oracles.append(oracle.fit_layer(c["W"], NVFP4, 16, c["rounds"], X=c["X"], init="quantile"))
        cases.append((c["W"], c["X"]))
    for which, d, o in zip(names, run_quantize_batch(cases, NVFP4, 20, binding.INIT_QUANTILE), oracles):
        assert np.allclose(host(carved_importance(d)), o["I"], rtol=1e-6, atol=0), f"{which}: importances differ"
        ok, worst = table_close(host(d["T01"]), o["T"])
        assert ok, f"{which}: tables differ: worst {worst:.3e}"
        tr = host(d["err_trace"])[:20]
        assert np.allclose(tr, o["trace"], rtol=1e-4, atol=0) and np.all(tr[1:] <= tr[:-1] * (1 + 1e-6))
        differ = int(np.sum(host(d["T01_bf16"]) != o["T_bf16"]))
        print(f"batched {which}: worst table deviation {worst:.2e}, BF16 entries that differ {differ}")
        assert differ == 0
        assert np.array_equal(host(d["codes"]), o["codes"]) and np.array_equal(host(d["scales"]), o["scales"])
        assert np.isclose(host(d["err_out"])[0], o["E_final"], rtol=1e-4)
        want = oracle.dequant(o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"], NVFP4, 16)
        assert np.array_equal(host(d["What"].contiguous()), want), f"{which}: reconstruction differs"


# ------------------------------------------------------------------ inner refinement (n_inner > 1)

@pytest.mark.parametrize("mode,init", [(INT4, "grid"), (INT4, "quantile"), (NVFP4, "quantile")])
@pytest.mark.parametrize("N,K,n_outer,n_inner", [(3, 256, 2, 2), (70, 640, 3, 4), (257, 1024, 3, 10)])
def test_inner_refinement_small(mode, init, N, K, n_outer, n_inner):
    """Algorithm 1 with n_inner > 1: ragged rows and columns, several items per block."""
    W, X = layer(mode, N, K, name=f"inner{mode}{init}/{N}x{K}")
    o, r, worst = check_fit(W, X, mode, n_outer, init, n_inner=n_inner)
    check_pack(W, mode, o, r)
    assert np.all(host(r["scales_pos"]) == o["scales_unsigned"])      # the fit leaves the scales' sign bits clear


def test_inner_refinement_paper_budgets_full_size():
    """The paper's default budget (n_outer, n_inner) = (3, 10) on the q_proj-sized layer of the
    benchmark configuration, whole layer against the oracle, and n_inner = 1 through the same
    entry point still equal to the single-pass rounds."""
    c = synth.config2_layer("q_proj")
    W, X = c["W"], c["X"]
    o, r, worst = check_fit(W, X, NVFP4, 3, "quantile", n_inner=10)
    check_pack(W, NVFP4, o, r)
    print(f"(3,10): worst table deviation {worst:.2e}")
    a = run_fit(W, NVFP4, o["I"], 3, binding.INIT_QUANTILE, n_inner=10)
    assert torch.equal(a["T01"], r["T01"]) and torch.equal(a["codes"], r["codes"])   # reproducible


def test_inner_refinement_degenerate_tables():
    """Identical tables: every group ties (table 0), table 1 receives nothing in any inner
    iteration and keeps its entries; entries of table 0 that coincide stay put."""
    W, X = layer(INT4, 24, 256, name="innerdegen")
    I = oracle.act_stats(X)
    T0 = np.linspace(-6.5, 6.5, 16)
    T0[7] = T0[6]                                        # a duplicate entry: its cell is empty
    T = np.stack([T0, T0]).astype(np.float32)
    o = oracle.fit_layer(W, INT4, 128, 2, I=I, init="user", T_init=T, n_inner=5)
    r = run_fit(W, INT4, I, 2, binding.INIT_USER, T01_init=T, n_inner=5)
    ok, worst = table_close(host(r["T01"]), o["T"])
    assert ok, worst
    assert np.allclose(host(r["trace"])[:2], o["trace"], rtol=1e-4)


# ------------------------------------------------------------------ selection group S < g (INT4 g = 128, S = 16)

def check_sel16(W, X, rounds, init_name, n_inner=1):
    """INT4 with one scale per 128 weights and one codebook choice per 16: fit against the oracle,
    then the pack pass on the oracle's tables bit for bit (codes, separate selection bits, untouched
    scales), then the dequantised weights."""
    g, S = 128, 16
    N, K = W.shape
    o = oracle.fit_layer(W, INT4, g, rounds, X=X, init=init_name, n_inner=n_inner, S=S)
    init = dict(quantile=binding.INIT_QUANTILE, grid=binding.INIT_GRID)[init_name]
    Wd = dev_bf16(W)
    Id = torch.from_numpy(o["I"]).to(DEV)
    r = binding.quantize_layer(Wd, INT4, I=Id, n_outer=rounds, init=init, want_trace=True, n_inner=n_inner, sel_group=S)
    assert int(r["status"].item()) == 0
    ok, worst = table_close(host(r["T01"]), o["T"])
    assert ok, f"tables differ: worst {worst:.3e}"
    if rounds:
        tr = host(r["trace"])[:rounds]
        assert np.allclose(tr, o["trace"], rtol=1e-4, atol=0)
        assert np.all(tr[1:] <= tr[:-1] * (1 + 1e-6))
    # pack on the oracle's tables
    T01 = torch.from_numpy(o["T_f32"]).to(DEV)
    sc = torch.from_numpy(o["scales_unsigned"].view(np.int16)).to(DEV).view(torch.uint16)
    ts = torch.from_numpy(o["tensor_scale"]).to(DEV)
    Tb = torch.empty(2, 16, dtype=torch.uint16, device=DEV)
    codes = torch.empty(N, K // 2, dtype=torch.uint8, device=DEV)
    bits = torch.zeros(N, K // (8 * S), dtype=torch.uint8, device=DEV)
    err = torch.zeros(2, dtype=torch.float64, device=DEV)
    stats = torch.zeros(4, dtype=torch.int64, device=DEV)
    ws = binding.alloc_workspace(INT4, N, K)
    binding.pack(Wd, INT4, I=Id, T01=T01, T01_bf16=Tb, scales=sc, tensor_scale=ts, codes=codes, ws=ws, err_out=err,
                 stats=stats, sel_group=S, sigma_bits=bits)
    assert np.array_equal(host(Tb), o["T_bf16"])
    assert np.array_equal(host(sc), o["scales_unsigned"]), "scales must keep a clear sign bit"
    assert np.array_equal(host(bits), o["sigma_bits"]), "selection bits differ"
    assert np.array_equal(host(codes), o["codes"]), "packed codes differ"
    st = host(stats)
    assert st[0] == o["ties"][0] and st[1] == o["ties"][1]
    e = host(err)
    assert np.isclose(e[0], o["E_final"], rtol=1e-4)
    Eo = oracle.output_error_sel(W, o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"], o["sigma_bits"], S, o["I"], INT4, g)
    assert np.isclose(e[1], Eo, rtol=1e-4)
    What = torch.empty(N, K, dtype=torch.bfloat16, device=DEV)
    binding.dequant(codes, sc, ts, Tb, INT4, What, sel_group=S, sigma_bits=bits)
    assert np.array_equal(host(What), oracle.dequant_sel(o["codes"], o["scales"], o["tensor_scale"], o["T_bf16"],
                                                         o["sigma_bits"], S, INT4, g))
    check_end_to_end_bits(r, o, f"S=16 {N}x{K} {init_name}", sel=True)
    return o, r


@pytest.mark.parametrize("init", ["grid", "quantile"])
@pytest.mark.parametrize("N,K", [(3, 256), (70, 640), (257, 1024), (64, 128)])
def test_selection_group_16_small(init, N, K):
    W, X = layer(INT4, N, K, name=f"sel16{init}/{N}x{K}")
    check_sel16(W, X, 5, init)


def test_selection_group_16_with_inner_refinement():
    W, X = layer(INT4, 130, 896, name="sel16inner")
    check_sel16(W, X, 3, "quantile", n_inner=4)


def test_selection_group_16_full_size_and_beats_128():
    """Llama-8B-shaped k_proj at full size; and the paper's reason for S = 16: a lower error than
    one choice per 128 weights on the same layer."""
    c = synth.scaled_layer(1024, 4096, 512, 0, "stack/llama8b/k_proj", mode=INT4)
    o, r = check_sel16(c["W"], c["X"], 20, "quantile")
    r128 = run_fit(c["W"], INT4, o["I"], 20, binding.INIT_QUANTILE)
    assert host(r["err"])[0] < host(r128["err"])[0]


def test_selection_group_argument_checks():
    W, X = layer(NVFP4, 16, 256, name="selargs")
    Wd = dev_bf16(W)
    I = torch.ones(256, device=DEV)
    with pytest.raises(binding.AaacError):
        binding.quantize_layer(Wd, NVFP4, I=I, n_outer=1, init=binding.INIT_GRID, sel_group=8)
    with pytest.raises(binding.AaacError):
        binding.quantize_layer(Wd, INT4, I=I, n_outer=1, init=binding.INIT_GRID, sel_group=32)
    a = binding.quantize_layer(Wd, NVFP4, I=I, n_outer=2, init=binding.INIT_GRID, sel_group=16)
    b = binding.quantize_layer(Wd, NVFP4, I=I, n_outer=2, init=binding.INIT_GRID)
    assert torch.equal(a["codes"], b["codes"]) and torch.equal(a["scales"], b["scales"]) and a["sigma_bits"] is None


# ------------------------------------------------------------------ channel scaling before the fit

@pytest.mark.parametrize("N,K", [(1, 8), (7, 264), (130, 1024), (4096, 4096)])
def test_prescale_columns_bit_exact(N, K):
    W = synth.weights(N, K, 4, f"pre/{N}x{K}/W", outlier_frac=0.02)
    X = synth.activations(32, K, 4, f"pre/{N}x{K}/X", kind="lognormal")
    I = oracle.act_stats(X)
    rng = np.random.default_rng(N * 1000 + K)
    a = np.exp(rng.normal(size=K)).astype(np.float32)
    Wo, Io = oracle.prescale(W, a, I)
    Wd = dev_bf16(W)
    ad = torch.from_numpy(a).to(DEV)
    Id = torch.from_numpy(I).to(DEV)
    out = torch.empty_like(Wd)
    Iout = torch.empty_like(Id)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.prescale_columns(Wd, ad, out, Id, Iout, dev_status=st)
    assert np.array_equal(host(out), Wo)
    assert np.array_equal(host(Iout), Io)
    assert int(st.item()) == 0
    # in place, without the importance
    binding.prescale_columns(Wd, ad, Wd)
    assert np.array_equal(host(Wd), Wo)
    # a multiplier that is not positive and finite is reported
    ad[K // 2] = 0.0
    binding.prescale_columns(out, ad, out, dev_status=st)
    assert int(st.item()) & binding.DEV_NONFINITE


def test_prescaled_layer_goes_through_the_fit_like_any_other():
    """Scale, then fit and pack: the same as the oracle run on the oracle's scaled layer."""
    W, X = layer(NVFP4, 96, 768, name="prefit")
    I = oracle.act_stats(X)
    a = np.ones(768, np.float32)
    a[np.argsort(I)[-16:]] = 1.75
    Wo, Io = oracle.prescale(W, a, I)
    Wd, ad, Id = dev_bf16(W), torch.from_numpy(a).to(DEV), torch.from_numpy(I).to(DEV)
    binding.prescale_columns(Wd, ad, Wd, Id, Id)
    o = oracle.fit_layer(Wo, NVFP4, 16, 5, I=Io)
    r = binding.quantize_layer(Wd, NVFP4, I=Id, n_outer=5, init=binding.INIT_QUANTILE, want_trace=True)
    assert table_close(host(r["T01"]), o["T"])[0]
    check_pack(Wo, NVFP4, o, r)


# ------------------------------------------------------------------ full benchmark sizes

@pytest.mark.parametrize("which", ["q_proj", "gate_proj", "down_proj"])
def test_config2_full_size(which):
    """Llama-3-8B-shaped linears, NVFP4, quantile init, 20 rounds -- the launch configuration
    the benchmark times -- against the oracle over the whole layer."""
    c = synth.config2_layer(which)
    W, X = c["W"], c["X"]
    o, r, worst = check_fit(W, X, NVFP4, c["rounds"], "quantile")
    st = check_pack(W, NVFP4, o, r)
    assert st[0] == 0
    print(f"{which}: worst table deviation {worst:.2e}, selection ties {st[0]}, half-way weights {st[1]}, "
          f"double re-evaluations {st[2]}")
    check_end_to_end_bits(r, o, f"cfg2 {which}")
    assert np.isclose(host(r["err"])[0], o["E_final"], rtol=1e-4)


# ------------------------------------------------------------------ other model shapes at full size

@pytest.mark.parametrize("name,N,K,mode,dist", [
    ("llama8b/k_proj", 1024, 4096, INT4, "normal"),          # configuration 3 shapes, INT4 g128
    ("llama8b/down_proj", 4096, 14336, INT4, "normal"),
    ("qwen7b/k_proj", 512, 3584, NVFP4, "student5"),         # configuration 4 shapes, NVFP4 g16, Student-t weights
    ("qwen7b/q_proj", 3584, 3584, NVFP4, "student5"),
    ("llama8b/gate_proj", 14336, 4096, INT4, "normal"),      # the widest / tallest linears of both stacks
    ("qwen7b/gate_proj", 18944, 3584, NVFP4, "student5"),
    ("qwen7b/down_proj", 3584, 18944, NVFP4, "student5"),
])
def test_stack_shaped_layers_full_size(name, N, K, mode, dist):
    """Single linears of the decoder-stack configurations, whole layer against the oracle,
    quantile init, 20 rounds."""
    c = synth.scaled_layer(N, K, 512, 0, f"stack/{name}", mode=mode, dist=dist)
    o, r, worst = check_fit(c["W"], c["X"], mode, 20, "quantile")
    st = check_pack(c["W"], mode, o, r)
    print(f"{name}: worst table deviation {worst:.2e}, selection ties {st[0]}, half-way weights {st[1]}, "
          f"double re-evaluations {st[2]}")
    assert st[0] == 0
    check_end_to_end_bits(r, o, name)


@pytest.mark.parametrize("name,N,K,mode", [
    ("gate_proj", 28672, 8192, NVFP4),
    ("down_proj", 8192, 28672, INT4),
])
def test_config5_whole_layer(name, N, K, mode):
    """The 70B-shaped largest layers, 30 rounds, whole layer against the oracle: fitted tables
    and objective trace, then the pack pass and the dequantised weights bit for bit, then the
    library's own end-to-end output.  This is the size at which the lane-private FP32 sums of the
    fit are longest."""
    rounds = 30
    c = synth.scaled_layer(N, K, 256, 0, f"cfg5/{name}", mode=mode, outlier_frac=0.005, rounds=rounds)
    W, X = c["W"], c["X"]
    o, r, worst = check_fit(W, X, mode, rounds, "quantile")
    assert int(r["status"].item()) == 0
    st = check_pack(W, mode, o, r)
    print(f"cfg5 {name}: worst table deviation {worst:.2e}, selection ties {st[0]}, half-way weights {st[1]}, "
          f"double re-evaluations {st[2]}")
    assert st[0] == 0
    check_end_to_end_bits(r, o, f"cfg5 {name}")
    assert np.isclose(host(r["err"])[0], o["E_final"], rtol=1e-4)
