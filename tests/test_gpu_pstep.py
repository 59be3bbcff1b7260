"""P-step kernels against the CPU checker: the chain rule of dequantisation to codebooks and scales
(binary64 sums: equal up to the order of binary64 roundings) and one Adam update (binary32, fixed operation
order: bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


@pytest.mark.parametrize("M,K,f16,rows,cols", [
    (1, 256, False, 64, 72),       # shared-memory accumulation, a warp straddles rows (9 groups per row)
    (1, 300, True, 100, 264),      # K not a power of two
    (1, 65536, True, 512, 1024),   # accumulation straight in L2
    (2, 256, True, 96, 136),
    (2, 64, False, 33, 72),
    (3, 128, True, 64, 256),       # three codebooks, sorted tiles (384 codewords)
    (4, 256, True, 64, 512),       # four codebooks: 1024 codewords, accumulation straight in L2
    (4, 64, False, 33, 72),
])
def test_pstep_grad_matches_checker(M, K, f16, rows, cols):
    L = synth.make_layer(rows, cols, cfg=110 + M, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         nearest=oracle_nearest)
    want_b, want_s = oracle.pstep_grad(L.g, L.scale, L.codes, L.codebooks, rows, cols)
    dev = VStepLayer.from_host(L)
    gb = torch.full((M, K, 8), 7.0, dtype=torch.float64, device="cuda")  # must be overwritten
    gs = torch.full((rows,), 7.0, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pvt_pstep_grad(dev.desc, gb, gs, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got_b, got_s = gb.cpu().numpy(), gs.cpu().numpy()
    # only the order of the binary64 additions differs: n terms of magnitude <= a carry an error <= n^2 a 2^-53
    n_terms = L.num_groups
    a_b = float(np.abs(L.scale).max()) * float(np.abs(L.g).max())
    a_s = float(np.abs(L.g).max()) * float(np.abs(L.codebooks.astype(np.float32)).max()) * M
    assert np.abs(got_b - want_b).max() <= n_terms * a_b * 2.0 ** -50
    assert np.abs(got_s - want_s).max() <= cols * a_s * 2.0 ** -50
    # codewords nobody uses get exactly zero
    used = np.zeros((M, K), bool)
    c2 = L.codes.reshape(-1, M)
    for m in range(M):
        used[m, c2[:, m]] = True
    assert not got_b[~used].any()


def test_pstep_grad_without_scale_output_and_bad_codes():
    L = synth.make_layer(64, 64, cfg=113, codebook_size=100, codebook_fp16=True)
    L.codes[5, 0] = 200
    dev = VStepLayer.from_host(L)
    gb = torch.empty((1, 100, 8), dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pvt_pstep_grad(dev.desc, gb, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.PVT_DEV_BAD_CODE
    L.codes[5, 0] = 0
    g2 = L.g.copy().reshape(-1, 8)
    g2[5] = 0  # the flagged group contributes nothing
    want_b, _ = oracle.pstep_grad(g2.reshape(L.g.shape), L.scale, L.codes, L.codebooks, 64, 64)
    assert np.allclose(gb.cpu().numpy(), want_b, rtol=0, atol=1e-12)


@pytest.mark.parametrize("n", [1, 1000, 65536 * 8 + 3])
def test_adam_update_bit_exact(n):
    rng = np.random.default_rng(120)
    p0 = rng.normal(size=n).astype(np.float32)
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    dp, dm, dv = torch.from_numpy(p0.copy()).cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    d16 = torch.zeros(n, dtype=torch.float16, device="cuda")
    for step in range(1, 4):
        grad = rng.normal(size=n) * 10.0 ** rng.integers(-4, 2, n)
        oracle.adam(p, grad, m, v, step, 3e-4, 0.9, 0.95, 1e-8)
        B.pvt_adam_update(dp, torch.from_numpy(grad).cuda(), dm, dv, step, 3e-4, 0.9, 0.95, 1e-8, param_f16=d16)
        torch.cuda.synchronize()
        assert dp.cpu().numpy().tobytes() == p.tobytes()
        assert dm.cpu().numpy().tobytes() == m.tobytes()
        assert dv.cpu().numpy().tobytes() == v.tobytes()
        assert d16.cpu().numpy().tobytes() == p.astype(np.float16).tobytes()


def test_p_step_then_v_step_round_trip():
    """A whole step in the paper's order: gradient to the codebook, Adam on the fp32 master codebook with its
    fp16 copy refreshed, then the V step against the refreshed codebook; compared with the checker doing the
    same."""
    L = synth.make_layer(256, 512, cfg=121, codebook_size=2048, codebook_fp16=True)
    dev = VStepLayer.from_host(L)
    K = 2048
    master = dev.codebooks.float().reshape(-1).clone()
    gb = torch.empty((1, K, 8), dtype=torch.float64, device="cuda")
    m, v = torch.zeros_like(master), torch.zeros_like(master)
    B.pvt_pstep_grad(dev.desc, gb)
    B.pvt_adam_update(master, gb.reshape(-1), m, v, 1, 3e-4, param_f16=dev.codebooks.reshape(-1))
    k = synth.subspace_size("0.02", L.num_groups)
    idx, _ = dev.step(k)
    torch.cuda.synchronize()
    assert dev.status() == 0
    # checker
    want_b, _ = oracle.pstep_grad(L.g, L.scale, L.codes, L.codebooks, L.rows, L.cols)
    pm = L.codebooks.astype(np.float32).reshape(-1).copy()
    om, ov = np.zeros_like(pm), np.zeros_like(pm)
    oracle.adam(pm, want_b.reshape(-1), om, ov, 1, 3e-4)
    new_books = pm.astype(np.float16).reshape(1, K, 8)
    got_books = dev.codebooks.cpu().numpy()
    # the gradient sums may differ in the last binary64 bits, which can flip a binary32 rounding of the update
    assert np.abs(got_books.astype(np.float32) - new_books.astype(np.float32)).max() <= 2.0 ** -10 * np.abs(new_books.astype(np.float32)).max()
    ref = oracle.vstep(L.W, L.g, L.scale, got_books, L.codes, L.eta, k, L.beam)
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), ref.idx)
    import helpers
    got_codes = dev.codes.cpu().numpy().reshape(-1, 1)
    helpers.check_codes_against_oracle(ref.t, got_books, got_codes[ref.idx.astype(np.int64)], ref.enc, 1e-6)


def test_adam_direction_bit_exact_and_v_step_on_it():
    """Section 3.4: the V step runs on the Adam-normalised update.  The direction kernel is bit-exact against
    the checker; a V step with g := direction and eta := the learning rate of the codes matches the checker's
    V step on the same direction."""
    L = synth.make_layer(256, 512, cfg=122, codebook_size=2048, codebook_fp16=True)
    n = L.g.size
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    dm, dv = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    dgrad = torch.from_numpy(L.g.reshape(-1).copy()).cuda()
    ddir = torch.empty(n, device="cuda")
    rng = np.random.default_rng(123)
    for step in (1, 2, 3):
        grad = (L.g.reshape(-1) * rng.uniform(0.5, 1.5, n)).astype(np.float32)
        want = oracle.adam_direction(grad, m, v, step)
        dgrad.copy_(torch.from_numpy(grad))
        B.pvt_adam_direction(dgrad, dm, dv, ddir, step)
        torch.cuda.synchronize()
        assert ddir.cpu().numpy().tobytes() == want.tobytes()
        assert dm.cpu().numpy().tobytes() == m.tobytes() and dv.cpu().numpy().tobytes() == v.tobytes()
    # V step on the direction with the codes' learning rate (Appendix J: 3e-3)
    L.g = want.reshape(L.g.shape)
    L.eta = 3e-3
    k = synth.subspace_size("0.01", L.num_groups)
    ref = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k, L.beam)
    dev = VStepLayer.from_host(L)
    idx, _ = dev.step(k)
    torch.cuda.synchronize()
    assert dev.status() == 0
    assert np.array_equal(idx.cpu().numpy().astype(np.uint32), ref.idx)
    import helpers
    got = dev.codes.cpu().numpy().reshape(-1, 1)
    helpers.check_codes_against_oracle(ref.t, L.codebooks, got[ref.idx.astype(np.int64)], ref.enc, 1e-6)
