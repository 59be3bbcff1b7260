"""Parity at the benchmark's full layer sizes, through the same calls and launch
configuration that bench.py times (select -> encode -> dequantise on one stream):
selection compared in full, codes compared for every selected group where the
CPU checker finishes in seconds and on a seeded sample of the selected groups
otherwise, dequantised weights on sampled rows."""
import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu

REL = 1e-6
MAX_ORACLE_PAIRS = 3.0e9  # codeword pairs the CPU checker is asked to evaluate per case


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


CASES = [
    # (config, entry, tau, dequant dtype)
    (1, 0, "1.0", torch.float32),
    (2, 0, "0.01", torch.float32),
    (3, 0, "0.01", torch.float32),
    (3, 1, "0.001", torch.float32),
    (4, 0, "0.01", torch.float16),
    (4, 1, "0.01", torch.float16),
    (4, 2, "0.01", torch.float16),
    (5, 1, "0.01", torch.float32),
    (5, 3, "0.01", torch.float32),
    (5, 1, "1.0", torch.float32),   # every group re-encoded (1 048 576 targets): the selection is the index list
    # the remaining workload lines of the benchmark's table
    (3, 0, "0.001", torch.float32),
    (3, 0, "0.1", torch.float32),   # 563 609 targets: the compute-bound two-codebook case
    (3, 1, "0.01", torch.float32),
    (3, 1, "0.1", torch.float32),
    (4, 3, "0.01", torch.float16),
    (4, 4, "0.01", torch.float16),
    (4, 5, "0.01", torch.float16),
    (5, 0, "0.01", torch.float32),
    (5, 0, "1.0", torch.float32),   # 8 388 608 targets
    (5, 2, "0.01", torch.float32),
    (5, 2, "1.0", torch.float32),   # 29 360 128 targets
    (5, 3, "1.0", torch.float32),
]


@pytest.mark.parametrize("cfg,which,tau,wdtype", CASES)
def test_full_size_step_against_checker(cfg, which, tau, wdtype):
    L = synth.make_config_layer(cfg, which, nearest=oracle_nearest)
    M, G = L.num_codebooks, L.num_groups
    k = synth.subspace_size(tau, G)
    dev = VStepLayer.from_host(L)
    W_hat = torch.empty(L.rows, L.cols, dtype=wdtype, device="cuda")
    idx, _ = dev.step(k, W_hat=W_hat)
    torch.cuda.synchronize()
    assert dev.status() == 0

    # selection: every index
    want_idx = oracle.select(oracle.group_norms(L.g, L.eta), k)
    got_idx = idx.cpu().numpy().astype(np.uint32)
    assert np.array_equal(got_idx, want_idx)

    # codes: all selected groups, or a seeded sample of them
    got_codes = dev.codes.cpu().numpy().reshape(-1, M)
    n_check = int(min(k, max(256, MAX_ORACLE_PAIRS // L.pairs_per_group())))
    pick = np.sort(np.random.default_rng(900 + cfg).choice(k, size=n_check, replace=False)) if n_check < k else np.arange(k)
    sel = want_idx[pick]
    t = oracle.targets(L.W, L.g, L.scale, L.eta, sel)
    codes2 = L.codes.reshape(-1, M)
    enc = oracle.encode(t, L.codebooks, codes2[sel.astype(np.int64)], L.beam)
    exact, band = helpers.check_codes_against_oracle(t, L.codebooks, got_codes[sel.astype(np.int64)], enc, REL)
    assert exact >= n_check - max(4, n_check // 500)

    # locality: every code outside the selection is untouched
    mask = np.ones(G, bool)
    mask[want_idx.astype(np.int64)] = False
    assert np.array_equal(got_codes[mask], codes2[mask])

    # dequantised weights: sampled rows, bit-exact against the closed form applied to the GPU's codes
    rows = np.unique(np.random.default_rng(950 + cfg).integers(0, L.rows, size=16))
    gpr = L.cols // 8
    sub_codes = np.concatenate([got_codes[r * gpr:(r + 1) * gpr] for r in rows])
    want_W = oracle.dequant(sub_codes, L.codebooks, L.scale[rows], len(rows), L.cols)
    got_W = W_hat[torch.from_numpy(rows).cuda()].cpu().numpy()
    if wdtype == torch.float16:
        assert got_W.tobytes() == want_W.astype(np.float16).tobytes()
    else:
        assert got_W.tobytes() == want_W.tobytes()


@pytest.mark.parametrize("K,f16", [(256, False), (512, True)])
def test_fp32_engine_with_eight_targets_per_thread(K, f16):
    """More than 148 x 8192 targets on the FP32 engine: the variant of the search kernel that keeps eight
    targets per thread (tiles of 2048 targets).  4096 x 4096, every group re-encoded, a small codebook so that
    the checker evaluates every pair: all 2 097 152 codes compared."""
    from paper_2405_14852_b200 import binding as B
    L = synth.make_layer(4096, 4096, cfg=7, codebook_size=K, codebook_fp16=f16)
    G = L.num_groups
    assert G >= 148 * 8192 * 1.3
    B.pvt_set_m1_search(B.PVT_M1_FP32)
    try:
        dev = VStepLayer.from_host(L)
        idx = torch.arange(G, dtype=torch.int32, device="cuda")
        err = torch.empty(G, dtype=torch.float32, device="cuda")
        dev.encode(idx, err)
        torch.cuda.synchronize()
        assert dev.status() == 0
    finally:
        B.pvt_set_m1_search(B.PVT_M1_AUTO)
    sel = np.arange(G, dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, sel)
    enc = oracle.encode(t, L.codebooks, L.codes.reshape(G, 1))
    got = dev.codes.cpu().numpy().reshape(G, 1)
    exact, band = helpers.check_codes_against_oracle(t, L.codebooks, got, enc, REL)
    assert exact >= G - G // 500
    assert np.allclose(err.cpu().numpy(), enc.d_best, rtol=1e-5, atol=1e-30)


def test_full_size_trust_step_against_checker():
    """pvt_vstep_trust on the benchmark's default layer (4096 x 4096, one codebook of 65 536, k_max = 1 % of the
    groups): rank order in full, kept count, codes of the kept groups, everything else untouched."""
    L = synth.make_config_layer(2, 0)
    G = L.num_groups
    k_max = synth.subspace_size("0.01", G)
    ratio = 0.1  # the layer's previous codes are random, so every change is large: the cut falls inside k_max
    want = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, k_max=k_max)
    order = oracle.rank(oracle.group_norms(L.g, L.eta), k_max)
    dev = VStepLayer.from_host(L)
    idx, n, stats = dev.step_trust(k_max, ratio)
    torch.cuda.synchronize()
    assert dev.status() == 0
    n = int(n.item())
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), order)
    assert 1 < want.n_kept < k_max
    near_tie = np.any(want.gap_rel <= REL)
    if not near_tie:
        assert n == want.n_kept
        assert np.array_equal(dev.codes.cpu().numpy(), want.codes)
    else:
        assert abs(n - want.n_kept) <= 2
    got = dev.codes.cpu().numpy().reshape(G, 1)
    rest = np.setdiff1d(np.arange(G), order[:n].astype(np.int64))
    assert np.array_equal(got[rest], L.codes.reshape(G, 1)[rest])
    s = stats.cpu().numpy()
    # both sides add rows*cols non-negative binary64 terms, in different orders: each within n * 2^-53 of the sum
    assert abs(s[0] - want.sq_norm) <= (L.rows * L.cols) * 2.0 ** -52 * want.sq_norm
    assert s[1] < ratio ** 2 * s[0]


def test_full_size_step_with_groups_of_16():
    """4096 x 4096 in groups of 16 weights, one fp16 codebook of 65 536, tau = 0.01: the tensor engine's 48-half
    operand rows at the full codebook size; codes of a seeded sample against the checker."""
    L = synth.make_layer(4096, 4096, cfg=2, codebook_size=65536, codebook_fp16=True, group_dim=16)
    G = L.num_groups
    k = synth.subspace_size("0.01", G)
    dev = VStepLayer.from_host(L)
    W_hat = torch.empty(4096, 4096, device="cuda")
    idx, _ = dev.step(k, W_hat=W_hat)
    torch.cuda.synchronize()
    assert dev.status() == 0
    want_idx = oracle.select(oracle.group_norms(L.g, L.eta, 16), k)
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), want_idx)
    got = dev.codes.cpu().numpy().reshape(G, 1)
    pick = np.sort(np.random.default_rng(960).choice(k, size=4096, replace=False))
    sel = want_idx[pick]
    t = oracle.targets(L.W, L.g, L.scale, L.eta, sel, 16)
    enc = oracle.encode(t, L.codebooks, L.codes[sel.astype(np.int64)])
    exact, band = helpers.check_codes_against_oracle(t, L.codebooks, got[sel.astype(np.int64)], enc, REL)
    assert exact >= 4096 - 8
    mask = np.ones(G, bool)
    mask[want_idx.astype(np.int64)] = False
    assert np.array_equal(got[mask], L.codes.reshape(G, 1)[mask])
    rows = np.unique(np.random.default_rng(961).integers(0, 4096, size=8))
    sub = np.concatenate([got[r * 256:(r + 1) * 256] for r in rows])
    want_W = oracle.dequant(sub, L.codebooks, L.scale[rows], len(rows), 4096)
    assert W_hat[torch.from_numpy(rows).cuda()].cpu().numpy().tobytes() == want_W.tobytes()
