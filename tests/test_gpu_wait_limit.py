"""The give-up path of the search kernels' on-chip waits.

Every wait of the single-codebook search kernels on an on-chip barrier is bounded.  Here the bound is lowered
through the library's test hook and every thread block leaves out one codebook copy, so that a wait really runs
out: the call must come back and report PVT_DEV_WAIT_EXPIRED through the status word, and an
ordinary call right afterwards (same process, same context, same workspace) must match the CPU checker.  Nothing
here faults or blocks the device: the kernel stops polling, lets its issued copies and tensor-core work finish,
frees its tensor memory and returns."""
import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("engine,K,withhold", [
    # the codebook is large enough that every thread block streams more copies than the withheld number
    ("tensor", 65536, 5),   # a step in the middle of the second codebook stage
    ("tensor", 65536, 0),   # the very first step
    ("fp32", 65536, 3),
    ("fp32", 65536, 0),
])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(engine, K, withhold):
    L = synth.make_layer(1024, 1024, cfg=61, codebook_size=K, codebook_fp16=True)
    k = 3000
    idx_np = oracle.select(oracle.group_norms(L.g, L.eta), k)
    idx = torch.from_numpy(idx_np.astype(np.int32)).cuda()
    B.pvt_set_m1_search({"fp32": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR}[engine])
    try:
        dev = VStepLayer.from_host(L)
        B.pvt_test_wait_limit(20000, withhold)
        try:
            dev.encode(idx)
            torch.cuda.synchronize()
            status = dev.status()
        finally:
            B.pvt_test_wait_limit(0, -1)
        assert status & B.PVT_DEV_WAIT_EXPIRED  # (the codes of such a call are documented as invalid)
        # the context and the workspace are still good: the same call, unhindered, matches the checker
        dev.encode(idx)
        torch.cuda.synchronize()
        assert dev.status() == 0
    finally:
        B.pvt_set_m1_search(B.PVT_M1_AUTO)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx_np)
    enc = oracle.encode(t, L.codebooks, L.codes[idx_np.astype(np.int64)])
    got = dev.codes.cpu().numpy().reshape(-1, 1)
    helpers.check_codes_against_oracle(t, L.codebooks, got[idx_np.astype(np.int64)], enc, 1e-6)
