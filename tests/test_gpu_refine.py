"""Parity of pvt_vstep_refine (local search over single-code changes, Appendix D) with the CPU checker.  Both
sides decide every move on the same binary64 errors under the same total order, so codes, move counts and
errors are compared exactly."""
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


def gpu_refine(L, idx_np, max_moves, encode_first=False):
    dev = VStepLayer.from_host(L)
    idx = torch.from_numpy(idx_np.astype(np.int32)).cuda()
    k = idx_np.size
    if encode_first:
        dev.encode(idx)
    err = torch.full((k,), -1.0, dtype=torch.float32, device="cuda")
    moves = torch.full((k,), 9999, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pvt_vstep_refine(dev.desc, idx, k, max_moves, err, moves, status)
    torch.cuda.synchronize()
    return dev.codes.cpu().numpy(), err.cpu().numpy(), moves.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("M,K,f16,rows,cols,k", [
    (2, 256, True, 64, 512, 1500),
    (2, 200, False, 33, 72, 297),      # every group, ragged sizes
    (1, 256, False, 64, 256, 900),
    (3, 64, True, 64, 256, 600),
    (4, 256, True, 32, 512, 300),      # codebooks read through L2 (1024 codewords)
    (4, 16, False, 32, 128, 512),
    (1, 2048, True, 64, 512, 333),     # two-byte codes; codebook read through L2 instead of shared memory
])
@pytest.mark.parametrize("max_moves", [0, 1, 64])
def test_refine_from_given_codes_matches_checker(M, K, f16, rows, cols, k, max_moves):
    L = synth.make_layer(rows, cols, cfg=200 + M, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         nearest=oracle_nearest)  # stored codes are random: several moves per group
    G = L.num_groups
    idx = np.sort(np.random.default_rng(k).choice(G, size=k, replace=False)).astype(np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    start = L.codes.reshape(G, M)[idx.astype(np.int64)]
    want, d, want_moves = oracle.local_search(t, L.codebooks, start, max_moves)
    codes, err, moves, status = gpu_refine(L, idx, max_moves)
    assert status == 0
    got = codes.reshape(G, M)
    assert np.array_equal(got[idx.astype(np.int64)].astype(np.int32), want)
    assert np.array_equal(moves, want_moves)
    assert np.array_equal(err, d.astype(np.float32))
    rest = np.setdiff1d(np.arange(G), idx.astype(np.int64))
    assert np.array_equal(got[rest], L.codes.reshape(G, M)[rest])
    if max_moves == 0:
        assert np.array_equal(got, L.codes.reshape(G, M))
    if M == 1 and max_moves >= 1:  # one move of a single codebook is the exhaustive search
        enc = oracle.encode(t, L.codebooks, start)
        assert np.array_equal(want, enc.codes)


def test_refine_after_the_beam_search_only_improves():
    L = synth.make_layer(96, 512, cfg=205, num_codebooks=2, codebook_size=256, codebook_fp16=True,
                         nearest=oracle_nearest, beam=1)  # greedy search: leaves improvable groups
    G = L.num_groups
    idx = oracle.select(oracle.group_norms(L.g, L.eta), 2000)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    enc = oracle.encode(t, L.codebooks, L.codes[idx.astype(np.int64)], L.beam)
    want, d, want_moves = oracle.local_search(t, L.codebooks, enc.codes)
    codes, err, moves, status = gpu_refine(L, idx, 64, encode_first=True)
    assert status == 0
    got = codes.reshape(G, 2)[idx.astype(np.int64)].astype(np.int32)
    decisive = (enc.d_second - enc.d_best) > 1e-6 * enc.d_second   # same start on both sides
    assert np.array_equal(got[decisive], want[decisive])
    assert np.array_equal(moves[decisive], want_moves[decisive])
    d_got = helpers.recon_error(t, L.codebooks, got)
    assert np.all(d_got <= enc.d_best * (1 + 1e-12))
    assert want_moves.sum() > 0, "the case should contain groups the beam search leaves improvable"


def test_refine_flags_bad_indices_and_codes():
    L = synth.make_layer(32, 128, cfg=206, num_codebooks=2, codebook_size=100, codebook_fp16=True,
                         nearest=oracle_nearest)
    L.codes[7, 1] = 100  # out of range
    idx = np.array([3, 7, 11, 5000], dtype=np.uint32)  # 5000 >= G = 512
    codes, err, moves, status = gpu_refine(L, idx, 8)
    assert status == (B.PVT_DEV_BAD_INDEX | B.PVT_DEV_BAD_CODE)
    assert np.array_equal(codes.reshape(-1, 2)[7], L.codes[7])


def test_refine_rejects_bad_arguments():
    L = synth.make_layer(32, 128, cfg=207, codebook_size=64, codebook_fp16=True)
    dev = VStepLayer.from_host(L)
    idx = torch.zeros(4, dtype=torch.int32, device="cuda")
    for k, mm in ((0, 1), (4, -1), (4, 70000), (10**6, 1)):
        with pytest.raises(B.PvtError) as e:
            B.pvt_vstep_refine(dev.desc, idx, k, mm)
        assert e.value.code == B.PVT_EINVAL
