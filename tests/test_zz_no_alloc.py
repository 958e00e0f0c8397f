"""aaac_act_stats_noalloc -- the entry point for callers that cannot allocate device memory
(a plugin that only receives its tensors, an engine whose pool is fixed at start-up) -- must
give Eq. 7's column sums of squares like aaac_act_stats does.  Called through the C ABI
several times in a row, on inputs of different widths and lengths so that partials left behind
by an earlier call would show up if they were ever read; expected values come from the CPU
oracle, and the existing entry point is compared as well.  Collected last on purpose: a failure
here cannot hide the other tests."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_08692_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


# (tokens, input channels): two ordinary calls in a row, the widest input the built-in scratch
# covers, and a narrow, long input for which the number of row strips is clamped to its maximum
CASES = [(1500, 4096), (37, 520), (300, 32768), (20000, 256)]


def test_noalloc_matches_oracle_and_workspace_entry_point_on_calls_in_a_row():
    build.build()
    free_after_first = None
    for call, (T, K) in enumerate(CASES):
        Xh = synth.activations(T, K, 4, f"noalloc/{call}", kind="loguniform", massive_frac=0.01)
        want = oracle.act_stats(Xh)
        X = _dev(Xh)
        ref = torch.empty(K, dtype=torch.float32, device="cuda")
        ws = binding.alloc_workspace(binding.NVFP4, 1, K)
        binding.act_stats(X, ref, ws)
        got = torch.full((K,), -1.0, dtype=torch.float32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.mem_get_info()[0]
        binding.act_stats_noalloc(X, got, dev_status=st)
        torch.cuda.synchronize()
        after = torch.cuda.mem_get_info()[0]
        if free_after_first is not None:
            # past the first call (which looks up the scratch array's address) the device's free
            # memory does not move: nothing is allocated
            assert after == before, (call, before, after)
        free_after_first = after
        g = got.cpu().numpy()
        assert np.allclose(g, want, rtol=1e-6, atol=0), (call, np.abs(g - want).max())
        assert torch.allclose(got, ref, rtol=1e-6, atol=0), call      # (the row strips may be cut differently)
        assert int(st.item()) == 0
        # accumulate = 1 adds to what is there
        binding.act_stats_noalloc(X, got, accumulate=True)
        torch.cuda.synchronize()
        assert np.allclose(got.cpu().numpy(), 2.0 * want.astype(np.float64), rtol=1e-6, atol=0)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    L = binding.lib()
    import ctypes as C
    ok = C.c_void_p(1 << 20)
    assert L.aaac_act_stats_noalloc(ok, 8, 32768 + 8, 32768 + 8, ok, 0, None, None) == 9
    assert b"capacity" in L.aaac_status_string(9)
    assert L.aaac_act_stats_noalloc(None, 8, 256, 256, ok, 0, None, None) == 1
    assert L.aaac_act_stats_noalloc(ok, 8, 250, 256, ok, 0, None, None) == 3
