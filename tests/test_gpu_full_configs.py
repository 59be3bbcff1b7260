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
