"""Parity of pvt_vstep_trust (subspace size from the trust ratio, Section 4.3 / Appendix J) with the CPU checker:
rank order and kept count exact, codes by the acceptance rule of the plain V step, reported norms to rounding."""
import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu

REL = 1e-6


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


def settle(L):
    """Previous codes = the nearest codes of W itself, so that the step changes few groups by little."""
    G = L.num_groups
    L.codes = oracle.vstep(L.W, np.zeros_like(L.g), L.scale, L.codebooks, L.codes, eta=0.0, k=G).codes
    return L


def run_case(L, k_max, ratio):
    G, M = L.num_groups, L.num_codebooks
    want = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, k_max=k_max, beam=L.beam)
    full_order = oracle.rank(oracle.group_norms(L.g, L.eta), k_max)
    dev = VStepLayer.from_host(L)
    idx, n, stats = dev.step_trust(k_max, ratio)
    torch.cuda.synchronize()
    assert dev.status() == 0
    idx = idx.cpu().numpy().astype(np.uint32)
    n = int(n.item())
    stats = stats.cpu().numpy()
    got = dev.codes.cpu().numpy().reshape(G, M)
    old = L.codes.reshape(G, M)
    # rank order: a total order, so exact
    assert np.array_equal(idx, full_order)
    # every group keeps its previous code except the first n of the order
    rest = np.setdiff1d(np.arange(G), idx[:n].astype(np.int64))
    assert np.array_equal(got[rest], old[rest])
    # the kept groups carry the search result (acceptance rule of the plain V step)
    kept = idx[:n].astype(np.int64)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx[:n])
    enc = oracle.encode(t, L.codebooks, old[kept], L.beam)
    exact, band = helpers.check_codes_against_oracle(t, L.codebooks, got[kept], enc, REL)
    # squared norm before: rows*cols non-negative binary64 terms added in different orders, each sum within
    # n * 2^-53 of the exact value
    assert abs(stats[0] - want.sq_norm) <= max(1e-12, (L.rows * L.cols) * 2.0 ** -52) * want.sq_norm
    # kept count: equal unless a running total sits within rounding of the bound, or a near-tie among the tried
    # groups let the two sides pick different codes (then their changes differ legitimately)
    limit = float(np.float64(np.float32(ratio)) ** 2) * want.sq_norm
    running = np.cumsum(want.change)
    touchy = np.any(np.abs(running - limit) <= 1e-9 * max(limit, 1e-300)) or np.any(want.gap_rel <= REL)
    if not touchy:
        assert n == want.n_kept
        assert np.array_equal(got, want.codes.reshape(G, M))
        kept_change = running[n - 1]
        assert abs(stats[1] - kept_change) <= 1e-12 * max(kept_change, 1e-300) + 1e-300
    else:
        assert abs(n - want.n_kept) <= 1
    return n, want


@pytest.mark.parametrize("M,K,f16,rows,cols,k_max,ratio", [
    (1, 256, False, 128, 1024, 2000, 0.03),
    (1, 256, False, 128, 1024, 16384, 0.05),    # every group ranked (selection skipped: k_max = G)
    (1, 2048, True, 256, 1024, 5000, 0.02),     # tensor-core search
    (1, 2048, True, 100, 264, 3300, 0.05),      # ragged sizes
    (2, 256, True, 128, 1024, 3000, 0.03),
    (2, 200, True, 96, 136, 1632, 0.1),
    (3, 64, True, 128, 512, 2000, 0.05),
    (4, 32, False, 64, 512, 1500, 0.05),
])
def test_trust_step_matches_checker(M, K, f16, rows, cols, k_max, ratio):
    L = settle(synth.make_layer(rows, cols, cfg=180 + M, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                                nearest=oracle_nearest))
    n, want = run_case(L, k_max, ratio)
    assert 1 < n < k_max, "the case should stop inside the ranked groups"


@pytest.mark.parametrize("M", [1, 2])
def test_trust_step_limits(M):
    L = synth.make_layer(64, 512, cfg=190 + M, num_codebooks=M, codebook_size=128, codebook_fp16=True,
                         nearest=oracle_nearest)  # random previous codes: every change is large
    n, _ = run_case(L, 500, 0.0)      # nothing satisfies the bound: one change goes through
    assert n == 1
    n, want = run_case(L, 500, 1e6)   # the cap binds: the plain V step on 500 groups
    assert n == 500


def test_trust_step_with_equal_norms_ranks_by_index():
    L = settle(synth.make_layer(64, 256, cfg=195, codebook_size=64, codebook_fp16=True))
    L.g[:] = np.tile(L.g[0, :8].copy(), 32)[None, :]   # every group has the same update: rank order = index order
    n, want = run_case(L, 700, 0.05)
    assert np.array_equal(want.order[:5], np.arange(5))


def test_trust_workspace_and_arguments():
    L = synth.make_layer(64, 256, cfg=196, codebook_size=64, codebook_fp16=True)
    dev = VStepLayer.from_host(L)
    need = B.pvt_trust_workspace_bytes(dev.desc, 100)
    assert need > B.pvt_workspace_bytes(dev.desc, 100)
    idx = torch.empty(100, dtype=torch.int32, device="cuda")
    n = torch.zeros(1, dtype=torch.int64, device="cuda")
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PvtError) as e:
        B.pvt_vstep_trust(dev.desc, 100, 0.01, idx, n, None, small)
    assert e.value.code == B.PVT_EWORKSPACE
    ws = B.new_trust_workspace(dev.desc, 100)
    for bad_ratio in (-0.1, float("nan"), float("inf")):
        with pytest.raises(B.PvtError) as e:
            B.pvt_vstep_trust(dev.desc, 100, bad_ratio, idx, n, None, ws)
        assert e.value.code == B.PVT_EINVAL
    with pytest.raises(B.PvtError):
        B.pvt_vstep_trust(dev.desc, 0, 0.01, idx, n, None, ws)
    B.pvt_vstep_trust(dev.desc, 100, 0.01, idx, n, None, ws)  # stats are optional
    torch.cuda.synchronize()
    assert 1 <= int(n.item()) <= 100
