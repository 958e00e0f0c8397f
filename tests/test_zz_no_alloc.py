"""aaac_act_stats_noalloc -- the entry point for callers that cannot allocate device memory
(a plugin that only receives its tensors, an engine whose pool is fixed at start-up) -- must
give what aaac_act_stats gives.  Called through the C ABI twice in a row, the second time on
a narrower, shorter input so that partials left behind by the first call would show up if they
were ever read.  Collected last on purpose: a failure here cannot hide the other tests."""
import numpy as np
import pytest
import torch

from paper_2605_08692_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def test_noalloc_matches_workspace_entry_point_twice():
    build.build()
    for call, (T, K) in enumerate([(1500, 4096), (37, 520)]):
        X = _dev(synth.activations(T, K, 4, f"noalloc/{call}", kind="loguniform", massive_frac=0.01))
        want = torch.empty(K, dtype=torch.float32, device="cuda")
        ws = binding.alloc_workspace(binding.NVFP4, 1, K)
        binding.act_stats(X, want, ws)
        got = torch.full((K,), -1.0, dtype=torch.float32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.act_stats_noalloc(X, got, dev_status=st)
        torch.cuda.synchronize()
        assert torch.allclose(got, want, rtol=1e-6, atol=0), (call, (got - want).abs().max())
        assert int(st.item()) == 0
        # accumulate = 1 adds to what is there
        binding.act_stats_noalloc(X, got, accumulate=True)
        torch.cuda.synchronize()
        assert torch.allclose(got, 2 * want, rtol=1e-6, atol=0)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    L = binding.lib()
    import ctypes as C
    ok = C.c_void_p(1 << 20)
    assert L.aaac_act_stats_noalloc(ok, 8, 32768 + 8, 32768 + 8, ok, 0, None, None) == 9
    assert b"capacity" in L.aaac_status_string(9)
    assert L.aaac_act_stats_noalloc(None, 8, 256, 256, ok, 0, None, None) == 1
    assert L.aaac_act_stats_noalloc(ok, 8, 250, 256, ok, 0, None, None) == 3
