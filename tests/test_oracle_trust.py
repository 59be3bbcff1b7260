"""Pins of the CPU checker's trust-ratio subspace rule (Section 4.3 and the hyper-parameter paragraph of Appendix J):
a worked example done by hand, the bound and its maximality recomputed from dequantised matrices, the limits
ratio -> 0 and ratio -> infinity, and independence of the portion size.  No GPU needed."""
import numpy as np
import pytest

from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import synth


def oracle_nearest(X, C):
    enc = oracle.encode(X, C[None], np.zeros((X.shape[0], 1), np.int32))
    return enc.codes[:, 0]


def settled_layer(cfg, M, rows=128, cols=1024, K=256):
    """A synthetic layer whose previous codes are a V step's result (not random), so that a further step moves
    few groups by little, as in fine-tuning."""
    L = synth.make_layer(rows, cols, cfg=cfg, num_codebooks=M, codebook_size=K, codebook_fp16=True,
                         nearest=oracle_nearest)
    G = L.num_groups
    first = oracle.vstep(L.W, np.zeros_like(L.g), L.scale, L.codebooks, L.codes, eta=0.0, k=G)
    L.codes = first.codes
    return L


# ---------------------------------------------------------------- worked example (one weight per group)


def hand_example():
    # six scalar weights, value set {0, 1, 2, 3}, every weight currently 1: ||x_old||^2 = 6.
    # update eta*g moves the targets to 3.2, 2.1, 2.05, 1.2, 1, 1 -> values 3, 2, 2, 1, 1, 1;
    # squared changes in the order of decreasing |update|: 4, 1, 1, 0, 0, 0 (running total 4, 5, 6, 6, 6, 6).
    W = np.ones((1, 6), np.float32)
    g = np.array([[-2.2, -1.1, -1.05, -0.2, 0.0, 0.0]], np.float32)
    book = np.arange(4, dtype=np.float32).reshape(1, 4, 1)
    codes = np.ones((6, 1), np.uint8)
    return W, g, np.ones(1, np.float32), book, codes


@pytest.mark.parametrize("portion", [0.17, 0.34, 0.5, 1.0])
@pytest.mark.parametrize("ratio,kept,values", [
    (1.0, 2, [3, 2, 1, 1, 1, 1]),     # bound 6: totals 4 and 5 pass, 6 is not below 6
    (0.5, 1, [3, 1, 1, 1, 1, 1]),     # bound 1.5: already the first change (4) breaks it, yet one change goes through
    (0.9, 1, [3, 1, 1, 1, 1, 1]),     # bound 4.86
    (0.92, 2, [3, 2, 1, 1, 1, 1]),    # bound 5.08
    (1.01, 6, [3, 2, 2, 1, 1, 1]),    # bound 6.12: everything passes
])
def test_hand_worked_example(ratio, kept, values, portion):
    W, g, s, book, codes = hand_example()
    res = oracle.vstep_trust(W, g, s, book, codes, eta=1.0, ratio=ratio, portion=portion)
    assert res.n_kept == kept
    assert list(book[0, res.codes[:, 0].astype(int), 0]) == values
    assert res.sq_norm == 6.0
    tried = len(res.order)  # portions are taken whole: the procedure stops with the portion that breaks the bound
    assert kept <= tried <= 6 and list(res.order) == list(range(tried))
    assert list(res.change) == [4.0, 1.0, 1.0, 0.0, 0.0, 0.0][:tried]


def test_hand_example_with_a_cap_on_the_groups_tried():
    W, g, s, book, codes = hand_example()
    res = oracle.vstep_trust(W, g, s, book, codes, eta=1.0, ratio=1.01, portion=0.34, k_max=2)
    assert res.n_kept == 2 and len(res.order) == 2
    assert list(book[0, res.codes[:, 0].astype(int), 0]) == [3, 2, 1, 1, 1, 1]


# ---------------------------------------------------------------- order and per-group change


@pytest.mark.parametrize("G,k", [(50, 50), (4096, 1), (4096, 700)])
def test_rank_is_the_sorted_order_and_extends_select(G, k):
    rng = np.random.default_rng(G + k)
    norms = rng.choice(rng.random(G // 3 + 1).astype(np.float32), size=G)  # many exact ties
    got = oracle.rank(norms, k)
    expect = np.lexsort((np.arange(G), -norms.astype(np.float64)))[:k]
    assert np.array_equal(got, expect.astype(np.uint32))
    assert np.array_equal(np.sort(got), oracle.select(norms, k))


@pytest.mark.parametrize("M", [1, 2])
def test_group_change_equals_difference_of_dequantised_matrices(M):
    L = synth.make_layer(32, 128, cfg=140 + M, num_codebooks=M, codebook_size=32, codebook_fp16=True,
                         nearest=oracle_nearest)
    rng = np.random.default_rng(3)
    G = L.num_groups
    idx = np.sort(rng.choice(G, size=100, replace=False)).astype(np.uint32)
    new = L.codes.copy()
    new[idx.astype(int)] = rng.integers(0, 32, size=(100, M))
    change, own = oracle.group_change(L.codes[idx.astype(int)], new[idx.astype(int)], L.codebooks, L.scale, L.cols, idx)
    X0 = oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols).astype(np.float64).reshape(G, 8)
    X1 = oracle.dequant(new, L.codebooks, L.scale, L.rows, L.cols).astype(np.float64).reshape(G, 8)
    per_group = ((X1 - X0) ** 2).sum(axis=1)
    assert np.allclose(change, per_group[idx.astype(int)], rtol=1e-14, atol=0)
    assert np.allclose(own, (X0 ** 2).sum(axis=1)[idx.astype(int)], rtol=1e-14, atol=0)
    untouched = np.setdiff1d(np.arange(G), idx.astype(int))
    assert not per_group[untouched].any()


# ---------------------------------------------------------------- the bound, maximality, limits


def realised(L, codes_new):
    X0 = oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols).astype(np.float64)
    X1 = oracle.dequant(codes_new, L.codebooks, L.scale, L.rows, L.cols).astype(np.float64)
    return np.linalg.norm(X1 - X0) / np.linalg.norm(X0)


@pytest.mark.parametrize("M", [1, 2])
@pytest.mark.parametrize("ratio", [0.01, 0.03, 0.1])
def test_bound_holds_and_is_maximal(M, ratio):
    L = settled_layer(150 + M, M)
    res = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, portion=0.01)
    assert 1 <= res.n_kept <= len(res.order)
    kept = res.order[: res.n_kept].astype(int)
    # locality: only kept groups may differ from the previous codes, and they carry the search result
    rest = np.setdiff1d(np.arange(L.num_groups), kept)
    assert np.array_equal(res.codes[rest], L.codes[rest])
    assert np.array_equal(res.codes[kept].astype(np.int32), res.enc_codes[: res.n_kept])
    r = realised(L, res.codes)
    if res.n_kept > 1:
        assert r < ratio * (1 + 1e-6)
    # maximality: letting the next group of the order through breaks the bound
    assert res.n_kept < len(res.order), "pick a ratio that stops before every group is taken"
    more = res.codes.copy()
    nxt = int(res.order[res.n_kept])
    more[nxt] = res.enc_codes[res.n_kept]
    assert realised(L, more) >= ratio * (1 - 1e-6)
    assert res.n_kept > 1 or ratio < 0.03, "the test layer should let several groups through at ratio 0.03"


@pytest.mark.parametrize("M", [1, 2])
def test_longest_prefix_and_portion_independence(M):
    L = settled_layer(160 + M, M)
    G = L.num_groups
    ratio = 0.05
    # independent route: one V step over ALL groups, per-group change from dequantised matrices,
    # longest prefix of the sorted order whose running change stays below the bound
    full = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k=G)
    X0 = oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols).astype(np.float64).reshape(G, 8)
    X1 = oracle.dequant(full.codes, L.codebooks, L.scale, L.rows, L.cols).astype(np.float64).reshape(G, 8)
    norms = oracle.group_norms(L.g, L.eta)
    order = np.lexsort((np.arange(G), -norms.astype(np.float64)))
    running = np.cumsum(((X1 - X0) ** 2).sum(axis=1)[order])
    ok = running < (ratio ** 2) * (X0 ** 2).sum()
    n_expect = max(1, int(np.argmin(ok)) if not ok.all() else G)
    for portion in (0.01, 0.05, 0.3, 1.0):
        res = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, portion=portion)
        assert res.n_kept == n_expect
        expect = L.codes.copy()
        expect[order[:n_expect]] = full.codes[order[:n_expect]]
        assert np.array_equal(res.codes, expect)
    capped = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=ratio, k_max=max(1, n_expect // 2))
    assert capped.n_kept == max(1, n_expect // 2)


@pytest.mark.parametrize("M", [1, 2])
def test_limits_of_the_ratio(M):
    L = synth.make_layer(32, 256, cfg=170 + M, num_codebooks=M, codebook_size=64, codebook_fp16=True,
                         nearest=oracle_nearest)  # random previous codes: every re-encoding changes a lot
    k_max = 200
    wide = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=1e6, k_max=k_max)
    plain = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k=k_max)
    assert wide.n_kept == k_max and np.array_equal(wide.codes, plain.codes)
    none = oracle.vstep_trust(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, ratio=0.0, k_max=k_max)
    assert none.n_kept == 1
    first = int(none.order[0])
    rest = np.setdiff1d(np.arange(L.num_groups), [first])
    assert np.array_equal(none.codes[rest], L.codes[rest])
    assert np.array_equal(none.codes[first].astype(np.int32), plain.codes[first].astype(np.int32))
