"""Groups of 16 weights with one codebook (Appendix J's representations with group size 16): selection, search and
dequantisation of the CUDA library against the CPU checker.  The search scores every codeword in binary64, so
codes are compared exactly."""
import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu


def layer(rows, cols, K, f16, cfg=240):
    return synth.make_layer(rows, cols, cfg=cfg, codebook_size=K, codebook_fp16=f16, group_dim=16)


@pytest.mark.parametrize("rows,cols,k", [(64, 512, 1), (64, 512, 100), (100, 272, 333), (256, 4096, 655), (33, 48, 99)])
def test_select_group_size_16(rows, cols, k):
    L = layer(rows, cols, 16, True)
    want = oracle.select(oracle.group_norms(L.g, L.eta, 16), k)
    dev = VStepLayer.from_host(L)
    idx = dev.select(k)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), want)


def test_select_group_size_16_ties_take_lowest_index():
    L = layer(64, 512, 16, True)
    L.g[:] = np.tile(L.g[0, :16].copy(), 32)[None, :]
    dev = VStepLayer.from_host(L)
    idx = dev.select(77)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), np.arange(77))


ENGINE = {"binary64": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR, "auto": B.PVT_M1_AUTO}


@pytest.mark.parametrize("K,f16,rows,cols,k,engine", [
    (256, False, 64, 256, 500, "auto"),
    (300, True, 64, 512, 700, "binary64"),     # two-byte codes, K not a multiple of the staged chunk
    (300, True, 64, 512, 700, "tensor"),       # K not a multiple of the 128-codeword step
    (1500, True, 100, 272, 333, "auto"),       # ragged sizes; tensor cores from 1024 codewords on
    (1500, True, 100, 272, 333, "binary64"),
    (4096, True, 256, 4096, 3000, "tensor"),   # several tiles of 256 targets and a ragged last one
    (65536, True, 256, 4096, 40, "auto"),      # the full-size codebook, a few targets
    (200, True, 64, 512, 1, "tensor"),         # a single target
])
def test_encode_group_size_16_matches_checker(K, f16, rows, cols, k, engine):
    B.pvt_set_m1_search(ENGINE[engine])
    try:
        _encode_case(K, f16, rows, cols, k)
    finally:
        B.pvt_set_m1_search(B.PVT_M1_AUTO)


def test_encode_group_size_16_extreme_scales_on_the_tensor_engine():
    """Targets outside the range the operand scaling serves (huge, tiny, zero) and a codeword whose norm does not
    fit the operand image: the tensor engine must hand these to exact rescoring."""
    L = layer(64, 512, 2048, True, cfg=241)
    L.W[3] *= 1e4      # |t| >= 256 after the division by the (unchanged) scale
    L.W[5] *= 1e-12    # tiny targets
    L.W[7] = 0.0
    L.g[7] = 0.0       # zero targets
    L.codebooks[0, 17] = 300.0   # half squared norm 16 * 300^2 / 2 > 60000: an exception row
    idx = np.arange(0, L.num_groups, 3, dtype=np.uint32)
    B.pvt_set_m1_search(B.PVT_M1_TENSOR)
    try:
        _encode_case(None, None, None, None, idx.size, L=L, idx=idx)
    finally:
        B.pvt_set_m1_search(B.PVT_M1_AUTO)


def _encode_case(K, f16, rows, cols, k, L=None, idx=None):
    L = layer(rows, cols, K, f16) if L is None else L
    G = L.num_groups
    if idx is None:
        idx = np.sort(np.random.default_rng(K + k).choice(G, size=k, replace=False)).astype(np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx, 16)
    enc = oracle.encode(t, L.codebooks, L.codes[idx.astype(np.int64)])
    dev = VStepLayer.from_host(L)
    err = torch.full((k,), -1.0, device="cuda")
    dev.encode(torch.from_numpy(idx.astype(np.int32)).cuda(), err)
    torch.cuda.synchronize()
    assert dev.status() == 0
    got = dev.codes.cpu().numpy().reshape(G, 1)
    helpers.check_codes_against_oracle(t, L.codebooks, got[idx.astype(np.int64)], enc, 1e-6)
    decisive = (enc.d_second - enc.d_best) > 1e-6 * enc.d_second
    assert np.array_equal(got[idx.astype(np.int64), 0].astype(np.int32)[decisive], enc.codes[decisive, 0])
    assert np.allclose(err.cpu().numpy(), enc.d_best, rtol=1e-5, atol=1e-30)
    rest = np.setdiff1d(np.arange(G), idx.astype(np.int64))
    assert np.array_equal(got[rest], L.codes.reshape(G, 1)[rest])


@pytest.mark.parametrize("K,f16,rows,cols", [(256, False, 64, 256), (200, True, 100, 272), (65536, True, 256, 4096)])
@pytest.mark.parametrize("out_f16", [False, True])
def test_dequant_group_size_16_bit_exact(K, f16, rows, cols, out_f16):
    L = layer(rows, cols, K, f16)
    want = oracle.dequant(L.codes, L.codebooks, L.scale, rows, cols)
    dev = VStepLayer.from_host(L)
    out = dev.dequant(dtype=torch.float16 if out_f16 else torch.float32)
    torch.cuda.synchronize()
    assert out.cpu().numpy().tobytes() == (want.astype(np.float16) if out_f16 else want).tobytes()


def test_whole_step_group_size_16():
    L = layer(128, 1024, 2048, True)
    k = 300
    want = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k)
    dev = VStepLayer.from_host(L)
    idx, W_hat = dev.step(k, W_hat=torch.empty(128, 1024, device="cuda"))
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), want.idx)
    assert np.array_equal(dev.codes.cpu().numpy(), want.codes)
    assert W_hat.cpu().numpy().tobytes() == oracle.dequant(want.codes, L.codebooks, L.scale, 128, 1024).tobytes()


def settle(L):
    L.codes = oracle.vstep(L.W, np.zeros_like(L.g), L.scale, L.codebooks, L.codes, eta=0.0, k=L.num_groups).codes
    return L


@pytest.mark.parametrize("K,f16,rows,cols,k_max,ratio", [(256, False, 128, 1024, 2000, 0.05), (2048, True, 128, 2048, 3000, 0.03)])
def test_trust_step_group_size_16(K, f16, rows, cols, k_max, ratio):
    L = settle(layer(rows, cols, K, f16, cfg=242))
    G = L.num_groups
    want = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, k_max=k_max)
    order = oracle.rank(oracle.group_norms(L.g, L.eta, 16), k_max)
    dev = VStepLayer.from_host(L)
    idx, n, stats = dev.step_trust(k_max, ratio)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), order)
    assert 1 < want.n_kept < k_max
    if not np.any(want.gap_rel <= 1e-6):
        assert int(n.item()) == want.n_kept
        assert np.array_equal(dev.codes.cpu().numpy(), want.codes)
    s = stats.cpu().numpy()
    assert abs(s[0] - want.sq_norm) <= max(1e-12, rows * cols * 2.0 ** -52) * want.sq_norm


@pytest.mark.parametrize("K,f16,rows,cols", [(256, False, 64, 256), (1500, True, 100, 272)])
def test_pstep_grad_group_size_16(K, f16, rows, cols):
    L = layer(rows, cols, K, f16, cfg=243)
    want_b, want_s = oracle.pstep_grad(L.g, L.scale, L.codes, L.codebooks, rows, cols)
    dev = VStepLayer.from_host(L)
    gb = torch.full((1, K, 16), 7.0, dtype=torch.float64, device="cuda")
    gs = torch.full((rows,), 7.0, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pvt_pstep_grad(dev.desc, gb, gs, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    a_b = float(np.abs(L.scale).max()) * float(np.abs(L.g).max())
    a_s = float(np.abs(L.g).max()) * float(np.abs(L.codebooks.astype(np.float32)).max())
    assert np.abs(gb.cpu().numpy() - want_b).max() <= L.num_groups * a_b * 2.0 ** -50
    assert np.abs(gs.cpu().numpy() - want_s).max() <= cols * a_s * 2.0 ** -50


def test_group_size_16_rejections():
    L = layer(64, 256, 64, True)
    dev = VStepLayer.from_host(L)
    idx = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(B.PvtError) as e:
        B.pvt_vstep_refine(dev.desc, idx, 4, 1)
    assert e.value.code == B.PVT_EUNSUPPORTED
    with pytest.raises(B.PvtError) as e:
        B.pvt_vstep_select_noalloc(dev.desc, 4, idx)
    assert e.value.code == B.PVT_EUNSUPPORTED
