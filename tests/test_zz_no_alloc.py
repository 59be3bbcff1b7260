"""pvt_vstep_select_noalloc against pvt_vstep_select.

The no-allocation variant exists for callers that cannot hand the library a
workspace because they cannot allocate device memory where the selection is
needed (a memory pool fixed at start-up, a host application that owns the
device memory, a thread that must stay out of allocators).  It must return
exactly the index list of the ordinary call.  Two calls in a row share the
library's built-in scratch, so the second one also checks that nothing left
behind by the first leaks into its result.  This file sorts last on purpose:
a run that stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2405_14852_b200 import binding as B


def _g(rows, cols, seed):
    return np.random.default_rng(seed).normal(0.0, 1e-3, size=(rows, cols)).astype(np.float32)


def _desc(g_dev, rows, cols, eta=1.0):
    # only g, the shape and eta are read by the selection
    return B.pvt_layer(rows, cols, 8, 1, 256, B.PVT_F16, B.PVT_U8, 8, float(eta), 0,
                       None, g_dev.data_ptr(), None, None, None)


@pytest.mark.gpu
def test_noalloc_select_matches_workspace_select_twice_in_a_row():
    cases = [(777, 520, 5050, 1.0, 11), (512, 1024, 655, 0.37, 12)]  # second call: other shape, k and step size
    for rows, cols, k, eta, seed in cases:
        g = torch.from_numpy(_g(rows, cols, seed)).cuda()
        desc = _desc(g, rows, cols, eta)
        want = torch.empty(k, dtype=torch.int32, device="cuda")
        ws = B.new_workspace(desc, k)
        B.pvt_vstep_select(desc, k, want, ws)
        got = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        status = torch.full((1,), 0x7F, dtype=torch.int32, device="cuda")
        B.pvt_vstep_select_noalloc(desc, k, got, status)
        torch.cuda.synchronize()
        assert B.pvt_status(ws) == 0
        assert int(status.item()) == 0
        assert torch.equal(got, want)  # index sets are integers: bit-exact
        assert bool((got[1:] > got[:-1]).all())


@pytest.mark.gpu
def test_noalloc_select_with_crafted_ties_after_a_previous_call():
    """All norms equal: the lowest indices win, also when the scratch still holds
    the keys and histograms of an unrelated earlier call."""
    g0 = torch.from_numpy(_g(256, 256, 13)).cuda()
    d0 = _desc(g0, 256, 256)
    tmp = torch.empty(100, dtype=torch.int32, device="cuda")
    B.pvt_vstep_select_noalloc(d0, 100, tmp)
    g = torch.full((128, 256), 1e-3, dtype=torch.float32, device="cuda")
    d = _desc(g, 128, 256)
    out = torch.empty(300, dtype=torch.int32, device="cuda")
    B.pvt_vstep_select_noalloc(d, 300, out)
    torch.cuda.synchronize()
    assert torch.equal(out.cpu(), torch.arange(300, dtype=torch.int32))


@pytest.mark.gpu
def test_noalloc_select_at_its_largest_layer_against_the_checker():
    """4096 x 4096 = 2^21 groups, the most the built-in scratch takes: the index list against the CPU
    checker's full sort, and no device memory taken or returned by the call (the first call on a device may
    make the array resident, so the free memory is compared across a second call)."""
    from oracle import pvt_oracle as oracle
    rows = cols = 4096
    assert rows * (cols // 8) == B.PVT_NOALLOC_MAX_GROUPS
    g_host = _g(rows, cols, 14)
    k = 20971
    want = oracle.select(oracle.group_norms(g_host, 1.0), k)
    g = torch.from_numpy(g_host).cuda()
    desc = _desc(g, rows, cols)
    got = torch.empty(k, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pvt_vstep_select_noalloc(desc, k, got, status)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    got.fill_(-1)
    B.pvt_vstep_select_noalloc(desc, k, got, status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert int(status.item()) == 0
    assert np.array_equal(got.cpu().numpy().astype(np.uint32), want)


def test_noalloc_select_rejects_layers_beyond_the_built_in_scratch():
    """Host-side check only: nothing is enqueued, so this runs without a GPU."""
    rows, cols = 4096, 4096 + 8  # one column group more than 2^21 groups
    assert rows * (cols // 8) > B.PVT_NOALLOC_MAX_GROUPS
    L = B.pvt_layer(rows, cols, 8, 1, 256, B.PVT_F16, B.PVT_U8, 8, 1.0, 0, None, 0x1000, None, None, None)
    rc = B.lib().pvt_vstep_select_noalloc(ctypes.byref(L), 10, 0x2000, None, None)
    assert rc == B.PVT_ETOOLARGE
    assert "scratch" in B.strerror(rc)
    # ordinary argument errors are reported as by pvt_vstep_select
    L = B.pvt_layer(16, 64, 8, 1, 256, B.PVT_F16, B.PVT_U8, 8, 1.0, 0, None, 0x1000, None, None, None)
    assert B.lib().pvt_vstep_select_noalloc(ctypes.byref(L), 0, 0x2000, None, None) == B.PVT_EINVAL
    assert B.lib().pvt_vstep_select_noalloc(ctypes.byref(L), 4, None, None, None) == B.PVT_EINVAL
