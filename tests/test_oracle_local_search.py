"""Pins of the CPU checker's local search over single-code changes (Appendix D).  No GPU needed."""
import itertools

import numpy as np
import pytest

import helpers
from oracle import pvt_oracle as oracle


def scalar_books(*value_sets):
    K = max(len(v) for v in value_sets)
    assert all(len(v) == K for v in value_sets)
    return np.array(value_sets, dtype=np.float32).reshape(len(value_sets), K, 1)


# ---------------------------------------------------------------- worked by hand


def test_hand_example_two_moves_to_the_optimum():
    # sums of {0, 10} and {0, 1, 2}; target 11.2.  From (0, 0) (error 125.44) the best single change is
    # the first code -> (1, 0) (error 1.44); then the second code -> (1, 1) (error 0.04); then nothing helps.
    books = scalar_books([0, 10, 10], [0, 1, 2])  # first set padded with a duplicate: the lower code wins ties
    t = np.array([[11.2]], np.float32)
    codes, d, moves = oracle.local_search(t, books, [[0, 0]])
    assert codes.tolist() == [[1, 1]] and moves.tolist() == [2]
    assert d[0] == pytest.approx((float(np.float32(11.2)) - 11.0) ** 2, rel=1e-12)
    one, d1, m1 = oracle.local_search(t, books, [[0, 0]], max_moves=1)
    assert one.tolist() == [[1, 0]] and m1.tolist() == [1]
    assert d1[0] == pytest.approx((float(np.float32(11.2)) - 10.0) ** 2, rel=1e-12)
    none, _, m0 = oracle.local_search(t, books, [[0, 0]], max_moves=0)
    assert none.tolist() == [[0, 0]] and m0.tolist() == [0]


def test_hand_example_stuck_in_a_local_optimum():
    # sums of {0, 3} and {0, 2}: 0, 2, 3, 5.  Target 2.6: the optimum is 3 = (1, 0), but from 2 = (0, 1) every
    # single change is worse (0 -> 6.76, 5 -> 5.76 against 0.36), so the search stays.
    books = scalar_books([0, 3], [0, 2])
    t = np.array([[2.6]], np.float32)
    codes, d, moves = oracle.local_search(t, books, [[0, 1]])
    assert codes.tolist() == [[0, 1]] and moves.tolist() == [0]
    best, _, _ = oracle.local_search(t, books, [[1, 1]])
    assert best.tolist() == [[1, 0]]


def test_move_choice_matches_the_difference_formula_of_the_appendix():
    # scalar case, one value set: phi(x^) - phi(x) = x^_k^2 - x_k^2 - 2 (x^_k - x_k) B_k  (Appendix D)
    rng = np.random.default_rng(5)
    values = np.sort(rng.normal(size=16)).astype(np.float32)
    books = values.reshape(1, 16, 1)
    B = rng.normal(size=(200, 1)).astype(np.float32)
    start = rng.integers(0, 16, size=(200, 1))
    codes, d, moves = oracle.local_search(B, books, start, max_moves=1)
    v = values.astype(np.float64)
    x = v[start[:, 0]]
    delta = v[None, :] ** 2 - x[:, None] ** 2 - 2.0 * (v[None, :] - x[:, None]) * B.astype(np.float64)
    want = delta.argmin(axis=1)
    improves = delta.min(axis=1) < 0
    assert np.array_equal(codes[improves, 0], want[improves])
    assert np.array_equal(codes[~improves, 0], start[~improves, 0])
    assert np.array_equal(moves, improves.astype(np.int32))


# ---------------------------------------------------------------- against independent enumeration


def neighbours(code, K):
    for m, q in itertools.product(range(len(code)), range(K)):
        if q != code[m]:
            c = list(code)
            c[m] = q
            yield c


@pytest.mark.parametrize("M,K", [(1, 50), (2, 12), (3, 6)])
def test_result_has_no_better_neighbour_and_never_gets_worse(M, K):
    rng = np.random.default_rng(10 * M + K)
    books = rng.normal(size=(M, K, 8)).astype(np.float32)
    t = rng.normal(size=(60, 8)).astype(np.float32) * 1.5
    start = rng.integers(0, K, size=(60, M))
    codes, d, moves = oracle.local_search(t, books, start)
    assert np.allclose(d, helpers.recon_error(t, books, codes), rtol=1e-12)
    assert np.all(d <= helpers.recon_error(t, books, start) * (1 + 1e-15))
    for n in range(60):
        nb = np.array(list(neighbours(codes[n].tolist(), K)))
        dn = helpers.recon_error(np.repeat(t[n:n + 1], len(nb), axis=0), books, nb)
        assert dn.min() >= d[n] * (1 - 1e-12)
    # the global optimum is a fixed point, and no result beats it
    tuples = np.array(list(itertools.product(range(K), repeat=M)))
    for n in range(10):
        dall = helpers.recon_error(np.repeat(t[n:n + 1], len(tuples), axis=0), books, tuples)
        opt = tuples[dall.argmin()]
        kept, dk, mk = oracle.local_search(t[n:n + 1], books, opt[None])
        assert kept.tolist() == [opt.tolist()] and mk.tolist() == [0]
        assert d[n] >= dall.min() * (1 - 1e-12)


def test_single_codebook_one_move_is_the_exhaustive_search():
    rng = np.random.default_rng(77)
    books = rng.normal(size=(1, 100, 8)).astype(np.float32)
    t = rng.normal(size=(300, 8)).astype(np.float32)
    start = rng.integers(0, 100, size=(300, 1))
    codes, d, moves = oracle.local_search(t, books, start)
    enc = oracle.encode(t, books, start)
    assert np.array_equal(codes, enc.codes)
    assert np.array_equal(d, enc.d_best)
    assert np.all(moves <= 1)


def test_each_move_takes_the_best_neighbour():
    rng = np.random.default_rng(78)
    K = 9
    books = rng.normal(size=(2, K, 8)).astype(np.float32)
    t = rng.normal(size=(40, 8)).astype(np.float32) * 2
    cur = rng.integers(0, K, size=(40, 2))
    for _ in range(4):  # follow the search move by move
        nxt, d, moves = oracle.local_search(t, books, cur, max_moves=1)
        for n in range(40):
            nb = np.array(list(neighbours(cur[n].tolist(), K)))
            dn = helpers.recon_error(np.repeat(t[n:n + 1], len(nb), axis=0), books, nb)
            d_cur = helpers.recon_error(t[n:n + 1], books, cur[n:n + 1])[0]
            if dn.min() < d_cur * (1 - 1e-12):
                assert nxt[n].tolist() == nb[dn.argmin()].tolist() and moves[n] == 1
            elif dn.min() > d_cur * (1 + 1e-12):
                assert nxt[n].tolist() == cur[n].tolist() and moves[n] == 0
        cur = nxt


def test_rejects_codes_out_of_range():
    books = np.zeros((2, 4, 8), np.float32)
    with pytest.raises(ValueError):
        oracle.local_search(np.zeros((1, 8), np.float32), books, [[0, 4]])
