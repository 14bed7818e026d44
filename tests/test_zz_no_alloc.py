"""lrsa_score_select_static: the variant for callers that have no device memory to lend as scratch
and may not allocate (for instance a plugin in a process whose allocator already holds the whole
GPU).  It must give the same indices and scores as lrsa_score_select, call after call, although every
call reuses the library's one fixed scratch array.  Collected last on purpose."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2506_11498_b200 import lrsa, workloads

W = workloads.Workload


def _static_vs_workspace(w, call_tag):
    host = workloads.generate(w, ("K", "V"))
    K, V = host["K"].cuda(), host["V"].cuda()
    p = lrsa.Params.from_workload(w)
    assert lrsa.lrsa_workspace_bytes(p)[0] <= lrsa.STATIC_SCRATCH_BYTES
    want_idx, want_sc = lrsa.lrsa_score_select(p, K, V, want_score=True)
    wsel = lrsa.lrsa_num_sel_windows(p)
    idx = torch.full((w.B, w.Hkv, wsel, w.K), -1, dtype=torch.int32, device="cuda")
    sc = torch.zeros((w.B, w.Hkv, wsel, w.L), dtype=torch.float32, device="cuda")
    for call in range(2):              # two calls in a row on the shared array
        idx.fill_(-1); sc.zero_()
        lrsa.lrsa_score_select_static(p, K, V, idx, sc)
        assert lrsa.lrsa_score_select_static_status() == 0
        assert torch.equal(idx, want_idx), (w.name, call_tag, call)
        np.testing.assert_allclose(sc.cpu().numpy(), want_sc.cpu().numpy(), rtol=2e-5, atol=0)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice():
    """Lag windows of up to 4096 tokens: the kernel keeps everything but the status word on chip."""
    cases = [W("na_a", 2, 4, 2, 4 + 6 * 256 + 50, 128, 256, 64, 4, seed=71),
             W("na_b", 1, 4, 4, 16 + 7 * 512, 64, 512, 128, 16, seed=72, values="channel_offset"),
             W("na_l4096", 1, 2, 2, 4 + 3 * 4096 + 9, 128, 4096, 1024, 4, seed=75)]
    for rep in range(2):               # alternating shapes between the pairs of calls
        for w in cases:
            _static_vs_workspace(w, rep)


@pytest.mark.gpu
def test_static_scratch_reused_by_the_long_window_kernel():
    """Lag windows beyond 4096 tokens: the ticket counter, the per-window counters and statistics and the
    per-token spreads live in the shared array; every call finds the previous call's contents there
    (of another shape, in this test) and must clear what has to start at zero."""
    cases = [W("na_long64", 1, 1, 1, 2 + 3 * 4608 + 11, 64, 4608, 100, 2, seed=73),
             W("na_long128", 1, 2, 2, 4 * 4160, 128, 4160, 1000, 0, seed=74)]
    for rep in range(2):
        for w in cases:
            assert lrsa.lrsa_workspace_bytes(lrsa.Params.from_workload(w))[0] > 4096   # really uses the array
            _static_vs_workspace(w, rep)


@pytest.mark.gpu
def test_static_scratch_refuses_problems_that_do_not_fit():
    # long windows on many heads: counters, statistics and spreads exceed the fixed array
    w = W("na_big", 2, 8, 8, 12 * 4608, 128, 4608, 1024, 0)
    p = lrsa.Params.from_workload(w)
    assert lrsa.lrsa_workspace_bytes(p)[0] > lrsa.STATIC_SCRATCH_BYTES
    K = torch.zeros(8, dtype=torch.bfloat16, device="cuda")     # never read: the call is refused first
    idx = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(lrsa.LrsaError) as e:
        lrsa.lrsa_score_select_static(p, K, K, idx)
    assert e.value.status == 3
    # the 128K-token benchmark shape (lag 4096) needs only the status word and is accepted
    big = lrsa.Params(2, 32, 8, 131072, 128, 4096, 1024, 4)
    assert lrsa.lrsa_workspace_bytes(big)[0] <= 4096


def test_static_entry_point_validates_on_the_host():
    L = lrsa.lib()
    cp = lrsa.Params(1, 4, 2, 1000, 128, 128, 32, 4).c()
    null, fake = ctypes.c_void_p(0), ctypes.c_void_p(0x10000)
    assert L.lrsa_score_select_static(ctypes.byref(cp), null, fake, fake, null, null) == 1
    assert L.lrsa_score_select_static(ctypes.byref(cp), fake, fake, null, null, null) == 1
    bad = lrsa.Params(1, 4, 2, 1000, 96, 128, 32, 4).c()
    assert L.lrsa_score_select_static(ctypes.byref(bad), fake, fake, fake, null, null) == 2
