"""Randomised configurations (seeded): layer shape, codebook count and size, group size, search engine, step size
and subspace size are drawn at random and every call is compared with the CPU checker.  Complements the fixed
cases of the other files; each seed is a fixed list of cases."""
import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu

ENGINES = {"auto": B.PVT_M1_AUTO, "fp32": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR}


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


def draw_layer(rng, case, max_rows, max_groups_per_row, big_codebooks=True):
    M = int(rng.choice([1, 1, 1, 2, 2, 3, 4]))
    dg = 16 if (M == 1 and rng.random() < 0.3) else 8
    rows = int(rng.integers(1, max_rows))
    cols = dg * int(rng.integers(1, max_groups_per_row))
    G = rows * (cols // dg)
    sizes = [2, 5, 64, 255, 256] + ([257, 1000, 1024, 2049, 5000] if (M == 1 and big_codebooks) else [])
    K = min(int(rng.choice(sizes)), G)
    if K < 2:
        return None
    L = synth.make_layer(rows, cols, cfg=5000 + case, num_codebooks=M, codebook_size=K,
                         codebook_fp16=bool(rng.random() < 0.7), nearest=oracle_nearest, beam=int(rng.choice([1, 3, 8])),
                         group_dim=dg, eta=float(rng.choice([1.0, 0.5, 0.0])))
    if rng.random() < 0.2:
        L.g[rng.integers(0, rows)] *= 100.0  # one row dominates the selection
    return L


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_whole_steps(seed):
    rng = np.random.default_rng(seed)
    for case in range(60):
        L = draw_layer(rng, 100 * seed + case, 400, 120)
        if L is None:
            continue
        G, M, dg = L.num_groups, L.num_codebooks, L.group_dim
        k = int(rng.integers(1, G + 1)) if rng.random() < 0.7 else G
        engine = str(rng.choice(list(ENGINES)))
        what = f"seed {seed} case {case}: M={M} dg={dg} {L.rows}x{L.cols} K={L.codebook_size} k={k} {engine}"
        B.pvt_set_m1_search(ENGINES[engine])
        try:
            want = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k, L.beam)
            dev = VStepLayer.from_host(L)
            W_hat = torch.empty(L.rows, L.cols, device="cuda")
            idx, _ = dev.step(k, W_hat=W_hat)
            torch.cuda.synchronize()
            assert dev.status() == 0, what
            assert np.array_equal(idx.cpu().numpy().astype(np.uint32), want.idx), what
            got = dev.codes.cpu().numpy().reshape(G, M)
            t = oracle.targets(L.W, L.g, L.scale, L.eta, want.idx, dg)
            helpers.check_codes_against_oracle(t, L.codebooks, got[want.idx.astype(np.int64)], want.enc, 1e-6)
            rest = np.ones(G, bool)
            rest[want.idx.astype(np.int64)] = False
            assert np.array_equal(got[rest], L.codes.reshape(G, M)[rest]), what
            assert W_hat.cpu().numpy().tobytes() == oracle.dequant(got, L.codebooks, L.scale, L.rows, L.cols).tobytes(), what
        finally:
            B.pvt_set_m1_search(B.PVT_M1_AUTO)


@pytest.mark.parametrize("seed", [21, 22])
def test_random_trust_refine_pstep(seed):
    rng = np.random.default_rng(seed)
    for case in range(60):
        L = draw_layer(rng, 100 * seed + case, 250, 80, big_codebooks=bool(rng.random() < 0.3))
        if L is None:
            continue
        G, M, dg, K = L.num_groups, L.num_codebooks, L.group_dim, L.codebook_size
        kind = str(rng.choice(["trust", "refine", "pstep"]))
        if kind == "refine" and dg == 16:
            kind = "pstep"
        what = f"seed {seed} case {case}: {kind} M={M} dg={dg} {L.rows}x{L.cols} K={K}"
        if kind == "trust":
            if rng.random() < 0.6:  # previous codes that already fit: small changes
                L.codes = oracle.vstep(L.W, np.zeros_like(L.g), L.scale, L.codebooks, L.codes, eta=0.0, k=G).codes
            dev = VStepLayer.from_host(L)
            k_max = int(rng.integers(1, G + 1))
            ratio = float(rng.choice([0.0, 0.003, 0.01, 0.05, 0.3, 10.0]))
            want = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, k_max=k_max,
                                      beam=L.beam)
            order = oracle.rank(oracle.group_norms(L.g, L.eta, dg), k_max)
            idx, n, _ = dev.step_trust(k_max, ratio)
            torch.cuda.synchronize()
            assert dev.status() == 0, what
            assert np.array_equal(idx.cpu().numpy().astype(np.uint32), order), what
            limit = float(np.float64(np.float32(ratio)) ** 2) * want.sq_norm
            running = np.cumsum(want.change)
            touchy = np.any(np.abs(running - limit) <= 1e-9 * max(limit, 1e-300)) or np.any(want.gap_rel <= 1e-6)
            if not touchy:
                assert int(n.item()) == want.n_kept, what
                assert np.array_equal(dev.codes.cpu().numpy().reshape(G, M), want.codes.reshape(G, M)), what
        elif kind == "refine":
            dev = VStepLayer.from_host(L)
            k = int(rng.integers(1, G + 1))
            moves_cap = int(rng.choice([0, 1, 3, 64]))
            idx_np = np.sort(rng.choice(G, size=k, replace=False)).astype(np.uint32)
            t = oracle.targets(L.W, L.g, L.scale, L.eta, idx_np, dg)
            want, d, want_moves = oracle.local_search(t, L.codebooks, L.codes.reshape(G, M)[idx_np.astype(np.int64)],
                                                      moves_cap)
            idx = torch.from_numpy(idx_np.astype(np.int32)).cuda()
            err = torch.zeros(k, device="cuda")
            moves = torch.zeros(k, dtype=torch.int32, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            B.pvt_vstep_refine(dev.desc, idx, k, moves_cap, err, moves, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, what
            got = dev.codes.cpu().numpy().reshape(G, M)[idx_np.astype(np.int64)].astype(np.int32)
            assert np.array_equal(got, want), what
            assert np.array_equal(moves.cpu().numpy(), want_moves), what
            assert np.array_equal(err.cpu().numpy(), d.astype(np.float32)), what
        else:
            dev = VStepLayer.from_host(L)
            want_b, want_s = oracle.pstep_grad(L.g, L.scale, L.codes, L.codebooks, L.rows, L.cols)
            gb = torch.full((M, K, dg), 3.0, dtype=torch.float64, device="cuda")
            gs = torch.full((L.rows,), 3.0, dtype=torch.float64, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            B.pvt_pstep_grad(dev.desc, gb, gs, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, what
            a_b = float(np.abs(L.scale).max()) * float(np.abs(L.g).max())
            a_s = float(np.abs(L.g).max()) * float(np.abs(L.codebooks.astype(np.float32)).max()) * M
            assert np.abs(gb.cpu().numpy() - want_b).max() <= G * a_b * 2.0 ** -50, what
            assert np.abs(gs.cpu().numpy() - want_s).max() <= L.cols * a_s * 2.0 ** -50, what
