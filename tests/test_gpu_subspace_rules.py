"""The straight-through buffer (Appendix E) and the random subspace rules (small-scale experiments' appendix)
on the GPU against the CPU checker: buffers and index lists bit for bit, codes by the V step's acceptance rule."""
import os

import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


def to_np(t):
    return t.detach().cpu().numpy()


@pytest.mark.parametrize("rows,cols,M,K,gd,eta,tau", [
    (128, 256, 1, 512, 8, 1.0, "0.05"),
    (77, 520, 2, 64, 8, 0.37, "0.1"),      # ragged: 5005 groups
    (64, 512, 1, 2048, 16, 1.0, "0.05"),   # groups of 16
    (33, 72, 1, 16, 8, 1.0, "1.0"),        # every group: the buffer must still take the step
])
def test_step_with_a_straight_through_buffer(rows, cols, M, K, gd, eta, tau):
    L = synth.make_layer(rows, cols, cfg=70 + M, num_codebooks=M, codebook_size=K, codebook_fp16=True, eta=eta,
                         group_dim=gd, nearest=oracle_nearest)
    k = synth.subspace_size(tau, L.num_groups)
    # the buffer starts as a perturbed copy of the weights: it is its own tensor, never the dequantised codes
    buf0 = (L.W + np.random.default_rng(71).normal(0, 2e-3, size=L.W.shape)).astype(np.float32)
    want_buf, want = oracle.vstep_ste(buf0, L.g, L.scale, L.codebooks, L.codes, L.eta, k, L.beam)
    dev = VStepLayer.from_host(L)
    buf = torch.from_numpy(buf0).cuda()
    idx = dev.select_ste(buf, k)
    dev.encode_against(buf, idx)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert to_np(buf).tobytes() == want_buf.tobytes()
    assert np.array_equal(to_np(idx).astype(np.uint32), want.idx)
    got = to_np(dev.codes).reshape(-1, M)
    sel = want.idx.astype(np.int64)
    helpers.check_codes_against_oracle(want.t, L.codebooks, got[sel], want.enc, 1e-6)
    mask = np.ones(L.num_groups, bool)
    mask[sel] = False
    assert np.array_equal(got[mask], L.codes.reshape(-1, M)[mask])


def test_buffer_accumulates_over_steps_until_codes_change():
    """Four steps with the same small update on the worked example's scalar layer (one weight per group, padded
    to groups of 8): the code flips at the fourth step on the GPU as it does in the checker."""
    books = np.zeros((1, 2, 8), dtype=np.float32)
    books[0, 1, 0] = 1.0
    g = np.zeros((1, 8), dtype=np.float32)
    g[0, 0] = -0.125
    buf_host = np.zeros((1, 8), dtype=np.float32)
    buf_host[0, 0] = 0.125
    L = synth.SynthLayer(rows=1, cols=8, group_dim=8, num_codebooks=1, codebook_size=2, beam=8, eta=1.0,
                         W=np.zeros((1, 8), np.float32), g=g, scale=np.ones(1, np.float32), codebooks=books,
                         codes=np.zeros((1, 1), np.uint8))
    dev = VStepLayer.from_host(L)
    buf = torch.from_numpy(buf_host).cuda()
    seen = []
    for _ in range(4):
        idx = dev.select_ste(buf, 1)
        dev.encode_against(buf, idx)
        torch.cuda.synchronize()
        seen.append((float(buf[0, 0].item()), int(dev.codes[0, 0].item())))
    assert dev.status() == 0
    assert seen == [(0.25, 0), (0.375, 0), (0.5, 0), (0.625, 1)]


@pytest.mark.parametrize("rows,cols,gd,k,seed", [
    (64, 256, 8, 100, 1),
    (77, 520, 8, 1234, (7 << 32) | 5),   # ragged, a seed above 2^32
    (64, 512, 16, 300, 99),
    (8, 64, 8, 1, 3),
    (8, 64, 8, 63, 3),
    (8, 64, 8, 64, 3),                   # k = G
])
@pytest.mark.parametrize("rule", [B.PVT_SAMPLE_UNIFORM, B.PVT_SAMPLE_PROPORTIONAL])
def test_random_subspaces_equal_the_checkers(rows, cols, gd, k, seed, rule):
    g = np.random.default_rng(80 + gd).normal(0, 1e-3, size=(rows, cols)).astype(np.float32)
    g[3, :2 * gd] = 0.0  # two groups of weight zero
    G = rows * cols // gd
    L = synth.SynthLayer(rows=rows, cols=cols, group_dim=gd, num_codebooks=1, codebook_size=2, beam=8, eta=0.5,
                         W=np.zeros_like(g), g=g, scale=np.ones(rows, np.float32),
                         codebooks=np.zeros((1, 2, gd), np.float16), codes=np.zeros((G, 1), np.uint8))
    norms = oracle.group_norms(g, 0.5, gd)
    want = oracle.sample_subspace(G, k, rule, seed, norms if rule == B.PVT_SAMPLE_PROPORTIONAL else None)
    dev = VStepLayer.from_host(L)
    got = dev.sample(k, rule, seed)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(to_np(got).astype(np.uint32), want)


def test_stored_index_lists_are_reproduced_on_the_gpu():
    stored = {}
    with open(os.path.join(helpers.GOLDEN, "sampled_subspaces.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, vals = line.split(":")
                stored[name.strip()] = [int(v) for v in vals.split()]
    cases = [("uniform_g1000_k25_seed7", 1000, 25, B.PVT_SAMPLE_UNIFORM, 7),
             ("uniform_g4099_k40_seed2pow40", 4099, 40, B.PVT_SAMPLE_UNIFORM, 1 << 40),
             ("proportional_g1000_k25_seed7", 1000, 25, B.PVT_SAMPLE_PROPORTIONAL, 7),
             ("proportional_g4099_k40_seed123456789", 4099, 40, B.PVT_SAMPLE_PROPORTIONAL, 123456789)]
    for name, G, k, rule, seed in cases:
        g = np.random.default_rng(4242).normal(0.0, 1e-3, size=(G, 8)).astype(np.float32)  # the stored lists' recipe
        L = synth.SynthLayer(rows=G, cols=8, group_dim=8, num_codebooks=1, codebook_size=2, beam=8, eta=1.0,
                             W=np.zeros_like(g), g=g, scale=np.ones(G, np.float32),
                             codebooks=np.zeros((1, 2, 8), np.float16), codes=np.zeros((G, 1), np.uint8))
        dev = VStepLayer.from_host(L)
        got = dev.sample(k, rule, seed)
        torch.cuda.synchronize()
        assert [int(i) for i in to_np(got)] == stored[name]


def test_random_subspaces_at_full_size():
    """4096 x 4096 (2 097 152 groups), k = 20 971: both rules against the checker, every index."""
    g = np.random.default_rng(2001).normal(0, 1e-3, size=(4096, 4096)).astype(np.float32)
    G = 4096 * 512
    norms = oracle.group_norms(g, 1.0)
    g_dev = torch.from_numpy(g).cuda()  # only g, the shape and the step size are read by the sampling call
    dev = VStepLayer(4096, 4096, g_dev, g_dev, torch.ones(4096, device="cuda"),
                     torch.zeros(1, 2, 8, dtype=torch.float16, device="cuda"),
                     torch.zeros(G, 1, dtype=torch.uint8, device="cuda"))
    for rule in (B.PVT_SAMPLE_UNIFORM, B.PVT_SAMPLE_PROPORTIONAL):
        want = oracle.sample_subspace(G, 20971, rule, 31337, norms if rule == B.PVT_SAMPLE_PROPORTIONAL else None)
        got = dev.sample(20971, rule, 31337)
        torch.cuda.synchronize()
        assert dev.status() == 0
        assert np.array_equal(to_np(got).astype(np.uint32), want)
