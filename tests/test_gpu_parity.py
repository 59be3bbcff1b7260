"""Parity of the CUDA library (through the C ABI) with the CPU checker on the
same seeded inputs: selection bit-exact, codes bit-exact outside the 1e-6 gap
band (error within 1e-6 relative inside it), dequantised weights bit-exact."""
import contextlib

import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu

REL = 1e-6  # relative gap / error tolerance of the acceptance rule
DEQ_ABS = 1e-6  # absolute tolerance on dequantised fp32 weights (bit-exact expected)


@contextlib.contextmanager
def search_engine(name):
    """Run the single-codebook search on one engine (fp32 pipe / tensor cores)."""
    B.pvt_set_m1_search({"fp32": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR, "auto": B.PVT_M1_AUTO}[name])
    try:
        yield
    finally:
        B.pvt_set_m1_search(B.PVT_M1_AUTO)


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


def to_np(t):
    return t.detach().cpu().numpy()


def select_only_layer(rows, cols, cfg):
    """A layer of which only g matters (seeded like the generator's stream 1)."""
    g = np.random.default_rng(1000 * cfg + 1).normal(0.0, 1e-3, size=(rows, cols)).astype(np.float32)
    G = rows * cols // 8
    return synth.SynthLayer(rows=rows, cols=cols, group_dim=8, num_codebooks=1, codebook_size=2, beam=8, eta=1.0,
                            W=np.zeros_like(g), g=g, scale=np.ones(rows, np.float32),
                            codebooks=np.zeros((1, 2, 8), np.float16), codes=np.zeros((G, 1), np.uint8))


def run_select(L, k):
    dev = VStepLayer.from_host(L)
    idx = dev.select(k)
    torch.cuda.synchronize()
    assert dev.status() == 0
    return to_np(idx).astype(np.uint32)


def run_encode(L, idx_np, want_err=True):
    dev = VStepLayer.from_host(L)
    idx = torch.from_numpy(idx_np.astype(np.int32)).cuda()
    err = torch.full((idx_np.size,), -1.0, dtype=torch.float32, device="cuda") if want_err else None
    dev.encode(idx, err)
    torch.cuda.synchronize()
    status = dev.status()
    return to_np(dev.codes), (to_np(err) if want_err else None), status


def check_encode(L, idx_np, beam=None):
    """Run the GPU search on the groups idx_np and compare with the checker."""
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx_np)
    codes2 = L.codes.reshape(-1, L.num_codebooks)
    enc = oracle.encode(t, L.codebooks, codes2[idx_np.astype(np.int64)], L.beam)
    got_codes, err, status = run_encode(L, idx_np)
    assert status == 0
    got2 = got_codes.reshape(-1, L.num_codebooks)
    exact, band = helpers.check_codes_against_oracle(t, L.codebooks, got2[idx_np.astype(np.int64)], enc, REL)
    # locality: everything outside idx is untouched, bit for bit
    mask = np.ones(codes2.shape[0], bool)
    mask[idx_np.astype(np.int64)] = False
    assert np.array_equal(got2[mask], codes2[mask])
    # reported error: compared loosely, it is never trusted by the rule above
    assert np.allclose(err, enc.d_best, rtol=1e-5, atol=1e-30)
    # monotone (Lemma 3.3): never worse than the previous code
    d_prev = helpers.recon_error(t, L.codebooks, codes2[idx_np.astype(np.int64)])
    d_new = helpers.recon_error(t, L.codebooks, got2[idx_np.astype(np.int64)])
    assert np.all(d_new <= d_prev * (1 + 1e-12))
    return exact, band


# ------------------------------------------------------------------ dequantise


@pytest.mark.parametrize("M,K,f16,rows,cols", [
    (1, 256, False, 256, 256),
    (1, 2048, True, 100, 264),     # ragged: G = 3300
    (1, 65536, True, 512, 1024),
    (2, 256, True, 96, 136),       # ragged
    (2, 64, False, 33, 72),
    (1, 16, True, 300, 8),         # one group per row
    (1, 64, True, 70, 24),         # three groups per row
    (2, 16, True, 9, 8248),        # 1031 groups per row (a prime)
])
@pytest.mark.parametrize("out_f16", [False, True])
def test_dequant_bit_exact(M, K, f16, rows, cols, out_f16):
    L = synth.make_layer(rows, cols, cfg=40 + M, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         nearest=oracle_nearest)
    want = oracle.dequant(L.codes, L.codebooks, L.scale, rows, cols)
    dev = VStepLayer.from_host(L)
    out = dev.dequant(dtype=torch.float16 if out_f16 else torch.float32)
    torch.cuda.synchronize()
    got = to_np(out)
    if out_f16:
        assert got.tobytes() == want.astype(np.float16).tobytes()
    else:
        assert np.abs(got - want).max() <= DEQ_ABS
        assert got.tobytes() == want.tobytes()


def test_dequant_flags_out_of_range_codes():
    L = synth.make_layer(64, 64, cfg=43, codebook_size=100, codebook_fp16=True)
    L.codes[5, 0] = 200
    dev = VStepLayer.from_host(L)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty(64, 64, device="cuda")
    B.pvt_dequant(dev.desc, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.PVT_DEV_BAD_CODE


# ------------------------------------------------------------------ selection


@pytest.mark.parametrize("rows,cols,k", [
    (1, 8, 1), (3, 8, 2), (16, 64, 1), (16, 64, 128), (16, 64, 127), (100, 264, 33),
    (512, 1024, 655), (777, 520, 5050), (2048, 2048, 5242), (2048, 2048, 1), (64, 8, 10),
])
def test_select_bit_exact(rows, cols, k):
    L = select_only_layer(rows, cols, 50)
    want = oracle.select(oracle.group_norms(L.g, L.eta), k)
    assert np.array_equal(run_select(L, k), want)


def test_select_with_scaled_step_and_huge_row():
    L = synth.make_layer(300, 512, cfg=51, codebook_fp16=True)
    L.eta = 0.37
    L.g[123] *= 1000.0  # one row dominates: 64 groups far above the rest
    for k in (10, 64, 65, 1000):
        want = oracle.select(oracle.group_norms(L.g, L.eta), k)
        got = run_select(L, k)
        assert np.array_equal(got, want)
        if k <= 64:
            assert np.all(got // 64 == 123)


def test_select_pure_ties_take_lowest_indices():
    L = synth.make_layer(128, 256, cfg=52, codebook_fp16=True)
    L.g[:] = 1e-3  # every group has the same norm
    for k in (1, 100, 4095, 4096):
        assert np.array_equal(run_select(L, k), np.arange(k, dtype=np.uint32))
    # duplicated gradient groups straddling the threshold
    L.g[:] = 1e-3
    G = L.num_groups
    g2 = L.g.reshape(G, 8)
    g2[10] = 5e-3
    g2[3000:3010] = 2e-3
    want = oracle.select(oracle.group_norms(L.g, L.eta), 6)
    assert list(want) == [10, 3000, 3001, 3002, 3003, 3004]
    assert np.array_equal(run_select(L, 6), want)
    g2[3] = 0.0  # a zero key
    want = oracle.select(oracle.group_norms(L.g, L.eta), G - 1)
    assert np.array_equal(run_select(L, G - 1), want)


def test_select_denormal_and_zero_norms():
    L = synth.make_layer(64, 256, cfg=53, codebook_fp16=True)
    L.g *= 1e-19  # norms around 1e-44: subnormal keys, many exact zeros
    want = oracle.select(oracle.group_norms(L.g, L.eta), 77)
    assert np.array_equal(run_select(L, 77), want)


def _layer_with_a_block_of_equal_norms(rows, cols, gd, seed):
    """Norms: the first two fifths of the groups (at random positions) far above a value v, one fifth exactly v,
    the rest far below it."""
    G = rows * cols // gd
    r = np.random.default_rng(seed)
    g = np.zeros((G, gd), dtype=np.float32)
    perm = r.permutation(G)
    top, tie, low = perm[:2 * G // 5], perm[2 * G // 5:3 * G // 5], perm[3 * G // 5:]
    g[top] = r.uniform(2e-3, 4e-3, size=(top.size, gd)).astype(np.float32)
    g[tie] = np.float32(1e-3)
    g[low] = r.uniform(1e-5, 5e-4, size=(low.size, gd)).astype(np.float32)
    L = synth.SynthLayer(rows=rows, cols=cols, group_dim=gd, num_codebooks=1, codebook_size=2, beam=8, eta=1.0,
                         W=np.zeros((1, gd), np.float32), g=g.reshape(rows, cols), scale=np.ones(rows, np.float32),
                         codebooks=np.zeros((1, 2, gd), np.float16), codes=np.zeros((G, 1), np.uint8))
    return L, G


@pytest.mark.parametrize("rows,cols,gd", [(4096, 4096, 8), (2048, 8192, 16)])
def test_select_with_a_large_block_of_equal_norms_around_the_threshold(rows, cols, gd):
    """A fifth of a large layer shares one norm and the subspace ends just inside, at, or just beyond that block:
    the threshold bucket then holds far more keys than the candidate list takes, and hundreds of thousands of
    ties must be split by index.  The exact index set must come out, ties towards the lowest index."""
    L, G = _layer_with_a_block_of_equal_norms(rows, cols, gd, 55)
    norms = oracle.group_norms(L.g, L.eta, gd)
    g_dev = torch.from_numpy(L.g).cuda()
    dev = VStepLayer(rows, cols, g_dev, g_dev, torch.ones(rows, device="cuda"),
                     torch.zeros(1, 2, gd, dtype=torch.float16, device="cuda"),
                     torch.zeros(G, 1, dtype=torch.uint8, device="cuda"), group_dim=gd)
    top = 2 * G // 5
    for k in (top + G // 1000, top - G // 1000, top + G // 10, top, top + 1, 3 * G // 5 + G // 1000):
        want = oracle.select(norms, k)
        got = dev.select(k)
        torch.cuda.synchronize()
        assert dev.status() == 0
        assert np.array_equal(to_np(got).astype(np.uint32), want), k


def test_select_many_sizes_against_the_checker():
    """Subspace sizes from one group to all but one on three mid-size layers (one with a ragged last tile)."""
    for rows, cols in ((128, 1016), (129, 1024), (640, 1024)):
        L = select_only_layer(rows, cols, 56)
        G = L.num_groups
        norms = oracle.group_norms(L.g, L.eta)
        dev = VStepLayer.from_host(L)
        for k in (1, 2, 7, G // 1000 + 1, G // 100, G // 10, G // 3, G // 2, G - G // 100, G - 1):
            got = dev.select(k)
            torch.cuda.synchronize()
            assert dev.status() == 0
            assert np.array_equal(to_np(got).astype(np.uint32), oracle.select(norms, k)), (rows, cols, k)


# ------------------------------------------------------------------ M = 1 search


def test_config_1_all_groups():
    L = synth.make_config_layer(1)
    k = synth.subspace_size(synth.config_taus(1)[0], L.num_groups)
    idx = run_select(L, k)
    assert np.array_equal(idx, np.arange(k, dtype=np.uint32))
    exact, band = check_encode(L, idx)
    assert exact >= k - 8


@pytest.mark.parametrize("K,f16,rows,cols,k", [
    (2, False, 16, 64, 128),
    (37, True, 64, 64, 100),         # K not a multiple of anything
    (256, True, 128, 256, 4096),
    (1000, True, 256, 256, 1500),    # K pads to 1024; k spans two tiles with a ragged tail
    (4096, True, 256, 512, 3000),
    (65536, True, 1024, 1024, 2500),  # full 16-bit codebook, codebook split over many CTAs
])
@pytest.mark.parametrize("engine", ["fp32", "tensor"])
def test_single_codebook_search(K, f16, rows, cols, k, engine):
    L = synth.make_layer(rows, cols, cfg=60, codebook_size=K, codebook_fp16=f16)
    rng = np.random.default_rng(61)
    idx = np.sort(rng.choice(L.num_groups, size=k, replace=False)).astype(np.uint32)
    with search_engine(engine):
        exact, band = check_encode(L, idx)
    assert exact >= k - max(4, k // 500)


@pytest.mark.parametrize("engine", ["fp32", "tensor"])
def test_single_codebook_search_codewords_and_targets_at_extreme_scales(engine):
    """Codewords whose squared norm leaves the half-precision range, targets that
    sit next to them, targets far outside the codebook's range and vanishing
    targets: every one of them must still get its exact nearest codeword."""
    L = synth.make_layer(96, 256, cfg=75, codebook_size=3000, codebook_fp16=True, row_max_scale=False)
    cb = L.codebooks[0]
    cb[5] = np.array([250, 250, 0, 0, 0, 0, 0, 0], np.float16)       # ||c||^2 / 2 = 62500
    cb[2999] = np.array([-200, 0, 0, 180, 0, 0, 150, 0], np.float16)  # 47450 (representable) 
    cb[77] = np.array([30000, -30000, 0, 0, 0, 0, 0, 1], np.float16)  # far beyond
    G = L.num_groups
    Wg = L.W.reshape(G, 8)
    Wg[0:40] = cb[5].astype(np.float32) + np.random.default_rng(76).normal(0, 1.0, (40, 8)).astype(np.float32)
    Wg[40:80] = cb[2999].astype(np.float32) * np.float32(0.98)
    Wg[80:120] = cb[77].astype(np.float32) * np.float32(1.01)          # |t| far above 256
    Wg[120:160] *= np.float32(1e4)                                     # |t| ~ 200 .. 800: partly out of range
    Wg[160:200] *= np.float32(1e-9)                                    # vanishing targets
    L.g[:] = 0
    idx = np.arange(400, dtype=np.uint32)
    with search_engine(engine):
        exact, band = check_encode(L, idx)
    assert exact >= 396


def test_single_codebook_unsorted_indices_and_scaled_step():
    L = synth.make_layer(128, 256, cfg=62, codebook_size=512, codebook_fp16=True)
    L.eta = 0.25
    idx = np.random.default_rng(63).permutation(L.num_groups)[:777].astype(np.uint32)
    check_encode(L, idx)


def test_single_codebook_exact_ties_and_zero_distance():
    """Duplicate codewords and targets that coincide with codewords: the lower
    code must win and the reported error must be exactly zero."""
    L = synth.make_layer(64, 128, cfg=64, codebook_size=300, codebook_fp16=True, row_max_scale=False)
    L.codebooks[0, 200:300] = L.codebooks[0, 0:100]  # duplicates of the first hundred
    cb = L.codebooks[0].astype(np.float32)
    G = L.num_groups
    pick = np.random.default_rng(65).integers(0, 300, size=G)
    L.W[:] = cb[pick].reshape(L.W.shape)
    L.g[:] = 0.0
    L.eta = 0.0
    idx = np.arange(G, dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    enc = oracle.encode(t, L.codebooks, L.codes)
    got, err, status = run_encode(L, idx)
    assert status == 0
    assert np.array_equal(got[:, 0], enc.codes[:, 0])  # exact ties resolved identically
    assert np.all(err == 0.0)
    assert np.all(got[:, 0] < 200)


def test_fixed_point_round_trip():
    """encode(dequant(codes), eta = 0) returns the codes (small steps leave y
    itself optimal, Section 3.2)."""
    L = synth.make_layer(128, 128, cfg=66, codebook_size=1024, codebook_fp16=True, row_max_scale=False)
    L.scale[:] = np.exp2(np.random.default_rng(67).integers(-3, 3, size=L.rows)).astype(np.float32)
    dev = VStepLayer.from_host(L)
    What = dev.dequant()
    dev.W.copy_(What)
    dev.desc.eta = 0.0
    idx = torch.arange(L.num_groups, dtype=torch.int32, device="cuda")
    dev.encode(idx)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(to_np(dev.codes), L.codes)


def test_out_of_range_index_is_flagged_and_skipped():
    L = synth.make_layer(64, 64, cfg=68, codebook_size=64, codebook_fp16=True)
    idx = np.array([3, 7, L.num_groups + 5, 11], dtype=np.uint32)
    got, err, status = run_encode(L, idx)
    assert status == B.PVT_DEV_BAD_INDEX
    good = np.array([3, 7, 11], dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, good)
    enc = oracle.encode(t, L.codebooks, L.codes[good.astype(np.int64)])
    assert np.array_equal(got[good.astype(np.int64), 0], enc.codes[:, 0])
    mask = np.ones(L.num_groups, bool)
    mask[good.astype(np.int64)] = False
    assert np.array_equal(got[mask], L.codes[mask])


# ------------------------------------------------------------------ M = 2 beam search


@pytest.mark.parametrize("K,beam,f16,rows,cols,k", [
    (256, 8, True, 128, 256, 4096),
    (256, 8, True, 344, 128, 555),
    (256, 1, True, 64, 128, 300),
    (256, 3, False, 64, 128, 300),
    (100, 8, True, 64, 128, 1024),
    (4, 8, True, 16, 64, 128),       # beam wider than the codebook
])
def test_two_codebook_beam_search(K, beam, f16, rows, cols, k):
    L = synth.make_layer(rows, cols, cfg=70, num_codebooks=2, codebook_size=K, codebook_fp16=f16, beam=beam,
                         nearest=oracle_nearest)
    idx = np.sort(np.random.default_rng(71).choice(L.num_groups, size=k, replace=False)).astype(np.uint32)
    exact, band = check_encode(L, idx)
    assert exact >= k - max(4, k // 200)


def test_two_codebooks_zero_second_book_all_ties():
    L = synth.make_layer(64, 128, cfg=72, num_codebooks=2, codebook_size=64, codebook_fp16=True,
                         nearest=oracle_nearest)
    L.codebooks[1] = 0
    idx = np.arange(L.num_groups, dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    enc = oracle.encode(t, L.codebooks, L.codes, L.beam)
    got, err, status = run_encode(L, idx)
    assert status == 0
    assert np.array_equal(got, enc.codes)  # every second code ties: the lowest pair wins on both sides
    assert np.all(got[:, 1] == 0)


def test_two_codebooks_previous_pair_kept_when_better():
    """Give every group the exhaustive optimum as its previous pair and search
    with beam 1: the pool contains the previous pair, so it must survive."""
    L = synth.make_layer(32, 64, cfg=73, num_codebooks=2, codebook_size=16, codebook_fp16=True, beam=1,
                         nearest=oracle_nearest)
    L.codebooks[1] = L.codebooks[0][::-1]  # equal-energy books: greedy is often wrong
    idx = np.arange(L.num_groups, dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    opt, dist = helpers.brute_force_tuples(t, L.codebooks.astype(np.float32))
    L.codes[:] = opt.astype(np.uint8)
    enc = oracle.encode(t, L.codebooks, L.codes, 1)
    assert np.allclose(enc.d_best, dist, rtol=1e-13, atol=0)
    got, err, status = run_encode(L, idx)
    assert status == 0
    helpers.check_codes_against_oracle(t, L.codebooks, got, enc, REL)


def test_two_codebooks_bad_previous_code_is_flagged():
    L = synth.make_layer(32, 64, cfg=74, num_codebooks=2, codebook_size=50, codebook_fp16=True,
                         nearest=oracle_nearest)
    L.codes[9, 1] = 77
    idx = np.array([9], dtype=np.uint32)
    got, err, status = run_encode(L, idx)
    assert status == B.PVT_DEV_BAD_CODE
    assert got[9, 0] < 50 and got[9, 1] < 50


# ------------------------------------------------------------------ whole step


@pytest.mark.parametrize("M", [1, 2])
def test_whole_step_select_encode_dequant(M):
    K = 2048 if M == 1 else 256
    L = synth.make_layer(512, 512, cfg=80 + M, num_codebooks=M, codebook_size=K, codebook_fp16=True,
                         nearest=oracle_nearest)
    k = synth.subspace_size("0.01", L.num_groups)
    ref = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k, L.beam)
    dev = VStepLayer.from_host(L)
    W_hat = torch.empty(L.rows, L.cols, dtype=torch.float32, device="cuda")
    idx, _ = dev.step(k, W_hat=W_hat)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(to_np(idx).astype(np.uint32), ref.idx)
    got_codes = to_np(dev.codes).reshape(-1, M)
    helpers.check_codes_against_oracle(ref.t, L.codebooks, got_codes[ref.idx.astype(np.int64)], ref.enc, REL)
    want_W = oracle.dequant(got_codes, L.codebooks, L.scale, L.rows, L.cols)
    assert np.abs(to_np(W_hat) - want_W).max() <= DEQ_ABS


# ------------------------------------------------------------------ ragged sizes of the work decomposition


@pytest.mark.parametrize("engine", ["fp32", "tensor"])
@pytest.mark.parametrize("k", [1, 2, 255, 257, 1023, 1025])
def test_single_codebook_ragged_target_counts(engine, k):
    """Target counts around the tile sizes of both engines (256 and 1024), down to a single group."""
    L = synth.make_layer(64, 512, cfg=130, codebook_size=2048 + 37, codebook_fp16=True)  # K not a multiple of 128
    idx = np.sort(np.random.default_rng(131 + k).choice(L.num_groups, size=k, replace=False)).astype(np.uint32)
    with search_engine(engine):
        check_encode(L, idx)


@pytest.mark.parametrize("k", [1, 2, 3, 5, 31, 33])
def test_two_codebook_ragged_target_counts(k):
    """The beam search takes four targets per warp: counts that leave partial groups of four."""
    L = synth.make_layer(32, 256, cfg=132, num_codebooks=2, codebook_size=200, codebook_fp16=True, nearest=oracle_nearest)
    idx = np.sort(np.random.default_rng(133 + k).choice(L.num_groups, size=k, replace=False)).astype(np.uint32)
    check_encode(L, idx)


# ------------------------------------------------------------------ three and four codebooks


@pytest.mark.parametrize("M,K,f16,rows,cols,k,beam", [
    (3, 64, True, 64, 256, 700, 8),
    (3, 256, True, 64, 512, 600, 8),
    (4, 32, False, 33, 72, 297, 8),     # every group, ragged sizes
    (4, 256, True, 32, 512, 300, 4),
    (3, 16, True, 32, 128, 512, 1),     # greedy
    (3, 100, True, 64, 256, 900, 8),    # codebook sizes that leave the last tile of 16 codewords ragged
    (4, 23, True, 48, 128, 500, 8),
    (3, 5, True, 32, 128, 300, 8),      # fewer codewords than the beam: three to eight kept tuples per stage
])
def test_three_and_four_codebooks_match_checker(M, K, f16, rows, cols, k, beam):
    L = synth.make_layer(rows, cols, cfg=210 + M, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         nearest=oracle_nearest, beam=beam)
    idx = np.sort(np.random.default_rng(k + M).choice(L.num_groups, size=k, replace=False)).astype(np.uint32)
    exact, band = check_encode(L, idx)
    assert band == 0  # every decision is taken on the checker's own binary64 values


@pytest.mark.parametrize("M", [2, 3, 4])
@pytest.mark.parametrize("f16", [True, False])
def test_beam_search_with_targets_of_very_different_magnitude(M, f16):
    """Rows of W scaled over twelve decades while the row scales stay put: neighbouring selected groups
    (which share a warp, and on fp16 codebooks one power-of-two scale of the tensor-pipe operands) have
    targets from 1e-6 to 1e6 times the codewords."""
    rows, cols = 48, 256
    L = synth.make_layer(rows, cols, cfg=230 + M, num_codebooks=M, codebook_size=256, codebook_fp16=f16,
                         nearest=oracle_nearest)
    decades = np.random.default_rng(231).uniform(-6.0, 6.0, size=(rows, 1))
    L.W = (L.W * (10.0 ** decades)).astype(np.float32)
    # every fourth group: consecutive selected groups come from different rows every few entries
    idx = np.arange(0, L.num_groups, 5, dtype=np.uint32)
    exact, band = check_encode(L, idx)
    assert exact >= len(idx) - max(4, len(idx) // 100)


@pytest.mark.parametrize("M", [2, 3, 4])
def test_beam_search_with_a_codebook_of_equal_codewords(M):
    """The second codebook holds one codeword 256 times: every extension of a stage ties exactly, far more than
    any shortlist holds, and the lowest tuple must win on both sides."""
    L = synth.make_layer(32, 256, cfg=240 + M, num_codebooks=M, codebook_size=256, codebook_fp16=True,
                         nearest=oracle_nearest)
    L.codebooks[1, :] = L.codebooks[1, 7]
    idx = np.arange(L.num_groups, dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    enc = oracle.encode(t, L.codebooks, L.codes.reshape(-1, M), L.beam)
    got, err, status = run_encode(L, idx)
    assert status == 0
    assert np.array_equal(got.reshape(-1, M), enc.codes.reshape(-1, M))


@pytest.mark.parametrize("M,K,f16,rows,cols", [(3, 100, True, 96, 136), (4, 256, True, 64, 512), (4, 50, False, 33, 72)])
@pytest.mark.parametrize("out_f16", [False, True])
def test_dequant_three_and_four_codebooks_bit_exact(M, K, f16, rows, cols, out_f16):
    L = synth.make_layer(rows, cols, cfg=220 + M, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         nearest=oracle_nearest)
    want = oracle.dequant(L.codes, L.codebooks, L.scale, rows, cols)
    dev = VStepLayer.from_host(L)
    out = dev.dequant(dtype=torch.float16 if out_f16 else torch.float32)
    torch.cuda.synchronize()
    got = to_np(out)
    assert got.tobytes() == (want.astype(np.float16) if out_f16 else want).tobytes()


def test_whole_step_with_three_codebooks():
    L = synth.make_layer(64, 512, cfg=225, num_codebooks=3, codebook_size=128, codebook_fp16=True,
                         nearest=oracle_nearest)
    k = 400
    want = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k, L.beam)
    dev = VStepLayer.from_host(L)
    idx, W_hat = dev.step(k, W_hat=torch.empty(64, 512, device="cuda"))
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(to_np(idx).astype(np.uint32), want.idx)
    assert np.array_equal(to_np(dev.codes), want.codes)
    assert to_np(W_hat).tobytes() == oracle.dequant(want.codes, L.codebooks, L.scale, 64, 512).tobytes()


# ------------------------------------------------------------------ repeatability and graph replay


@pytest.mark.parametrize("M,K", [(1, 4096), (2, 256)])
def test_step_is_repeatable_and_replays_from_a_cuda_graph(M, K):
    """The three calls of a step give the same indices, codes and weights when run again on the same inputs, and
    when captured once into a CUDA graph and replayed (the calls only enqueue work on the given stream)."""
    L = synth.make_layer(128, 1024, cfg=250 + M, num_codebooks=M, codebook_size=K, codebook_fp16=True,
                         nearest=oracle_nearest)
    k = 900
    results = []
    for _ in range(2):
        dev = VStepLayer.from_host(L, max_k=k)
        idx, W_hat = dev.step(k, W_hat=torch.empty(128, 1024, device="cuda"))
        torch.cuda.synchronize()
        assert dev.status() == 0
        results.append((to_np(idx), to_np(dev.codes), to_np(W_hat)))
    for a, b in zip(results[0], results[1]):
        assert a.tobytes() == b.tobytes()

    dev = VStepLayer.from_host(L, max_k=k)
    codes0 = dev.codes.clone()
    idx = torch.empty(k, dtype=torch.int32, device="cuda")
    W_hat = torch.empty(128, 1024, device="cuda")
    ws = dev.reserve(k)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        # one eager pass first: anything the library sets up lazily happens outside the capture
        B.pvt_vstep_select(dev.desc, k, idx, ws, stream=stream)
        B.pvt_vstep_encode(dev.desc, idx, k, None, ws, stream=stream)
        B.pvt_dequant(dev.desc, W_hat, stream=stream)
        stream.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            B.pvt_vstep_select(dev.desc, k, idx, ws, stream=stream)
            B.pvt_vstep_encode(dev.desc, idx, k, None, ws, stream=stream)
            B.pvt_dequant(dev.desc, W_hat, stream=stream)
    for _ in range(2):
        dev.codes.copy_(codes0)
        idx.zero_()
        W_hat.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert dev.status() == 0
        assert to_np(idx).tobytes() == results[0][0].tobytes()
        assert to_np(dev.codes).tobytes() == results[0][1].tobytes()
        assert to_np(W_hat).tobytes() == results[0][2].tobytes()


# ------------------------------------------------------------------ small codebooks on the tensor engine, negative scales


@pytest.mark.parametrize("K", [2, 3, 100, 129])
def test_tiny_codebooks_on_the_tensor_engine(K):
    """Codebooks far below one 128-codeword step: padding rows must never win."""
    L = synth.make_layer(64, 256, cfg=260, codebook_size=K, codebook_fp16=True)
    idx = np.arange(0, L.num_groups, 2, dtype=np.uint32)
    with search_engine("tensor"):
        check_encode(L, idx)


@pytest.mark.parametrize("engine", ["fp32", "tensor"])
def test_negative_row_scales(engine):
    """Row scales only have to be finite and non-zero: the target divides by them, the dequantised weight
    multiplies by them."""
    L = synth.make_layer(64, 512, cfg=261, codebook_size=2048, codebook_fp16=True)
    L.scale[::3] *= -1.0
    idx = oracle.select(oracle.group_norms(L.g, L.eta), 700)
    with search_engine(engine):
        check_encode(L, idx)
    dev = VStepLayer.from_host(L)
    out = dev.dequant()
    torch.cuda.synchronize()
    assert to_np(out).tobytes() == oracle.dequant(L.codes, L.codebooks, L.scale, 64, 512).tobytes()
