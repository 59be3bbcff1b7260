"""Pins of the CPU checker against what the paper and the mathematics fix:
printed examples, brute-force enumeration, library routines, identities,
special cases and invariants.  None of these tests needs a GPU."""
import itertools

import numpy as np
import pytest
from scipy.cluster.vq import vq

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import synth


def _rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- printed examples


def test_paper_example_clipping_nearest_value():
    ex = helpers.read_golden("example_clipping_nearest_value.txt")
    book = ex["codebook"].reshape(1, -1, 1)
    t = ex["targets"].reshape(-1, 1)
    enc = oracle.encode(t, book, np.zeros((t.shape[0], 1)))
    assert np.array_equal(book[0, enc.codes[:, 0], 0], ex["result"])
    # same example embedded in group dim 8 by zero padding
    book8 = np.zeros((1, 2, 8), np.float32)
    book8[0, :, 3] = ex["codebook"]
    t8 = np.zeros((5, 8), np.float32)
    t8[:, 3] = ex["targets"]
    enc8 = oracle.encode(t8, book8, np.zeros((5, 1)))
    assert np.array_equal(book8[0, enc8.codes[:, 0], 3], ex["result"])


@pytest.mark.parametrize("k", [4, 2])
def test_paper_example_linearized_v_step(k):
    ex = helpers.read_golden("example_vstep_degradation.txt")
    y = ex["y0"].astype(np.float32).reshape(1, 4)
    grad = (2.0 * (ex["y0"] - ex["xstar"])).astype(np.float32).reshape(1, 4)
    values = ex["values"].astype(np.float32).reshape(1, 3, 1)
    prev = np.array([[0], [1], [1], [2]], dtype=np.uint8)  # y0 in terms of the value set
    res = oracle.vstep(y, grad, np.ones(1, np.float32), values, prev, eta=0.5, k=k)
    if k == 2:  # only the two entries with a non-zero gradient are in the subspace
        assert list(res.idx) == [1, 2]
    x1 = values[0, res.codes[:, 0].astype(int), 0]
    assert np.array_equal(x1, ex["x1"])
    # the same step embedded in group dim 8 (4 rows, one group per row)
    y8 = np.zeros((4, 8), np.float32)
    g8 = np.zeros((4, 8), np.float32)
    v8 = np.zeros((1, 3, 8), np.float32)
    y8[:, 5], g8[:, 5], v8[0, :, 5] = y[0], grad[0], values[0, :, 0]
    res8 = oracle.vstep(y8, g8, np.ones(4, np.float32), v8, prev, eta=0.5, k=k)
    assert np.array_equal(v8[0, res8.codes[:, 0].astype(int), 5], ex["x1"])


def test_wrong_sign_of_update_would_fail_the_printed_example():
    """The printed example separates W - eta*g from W + eta*g: with the other
    sign the targets are {2, 0, 10, 11} and the result differs."""
    ex = helpers.read_golden("example_vstep_degradation.txt")
    t_wrong = (ex["y0"] + 0.5 * 2.0 * (ex["y0"] - ex["xstar"])).reshape(-1, 1)
    enc = oracle.encode(t_wrong, ex["values"].reshape(1, 3, 1), np.zeros((4, 1)))
    assert not np.array_equal(ex["values"][enc.codes[:, 0]], ex["x1"])


# ---------------------------------------------------------------- norms, targets (bit pins)


def test_group_norm_is_the_stated_fp32_sequence():
    g = (_rng(1).normal(0, 1e-3, size=(6, 16)) * np.array([1, 1e-18, 1e3, 1, 1e-20, 7])[:, None]).astype(np.float32)
    for eta in (1.0, 0.37, 3e-3):
        n = oracle.group_norms(g, eta)
        for j in range(n.size):
            r, c = divmod(j, 2)
            want = helpers.exact_group_norm(g[r, 8 * c:8 * c + 8], eta)
            assert n[j].tobytes() == want.tobytes(), (eta, j)


def test_group_norm_layout_and_group_dim():
    g = np.zeros((3, 24), np.float32)
    g[1, 8:16] = 2.0  # row 1, second group -> j = 1*3 + 1
    n = oracle.group_norms(g, 0.5)
    assert n.shape == (9,) and n[4] == 8.0 and n.sum() == 8.0
    n4 = oracle.group_norms(g, 0.5, group_dim=4)
    assert n4.shape == (18,) and n4[8] == 4.0 and n4[9] == 4.0


def test_targets_are_the_stated_fp32_sequence():
    r = _rng(2)
    W = r.normal(0, 0.02, size=(5, 32)).astype(np.float32)
    g = r.normal(0, 0.02, size=(5, 32)).astype(np.float32)  # comparable magnitudes: fused and unfused differ
    s = np.array([1.0, 0.071, 3.0, 0.5, 0.0123], np.float32)
    idx = np.arange(20, dtype=np.uint32)
    for eta in (1.0, 0.3):
        t = oracle.targets(W, g, s, eta, idx)
        unfused = ((W - np.float32(eta) * g) / s[:, None]).astype(np.float32).reshape(20, 8)
        if eta != 1.0:
            assert (unfused != t).any()  # the pin can tell the two apart
        for n, j in enumerate(idx):
            row, c = divmod(int(j), 4)
            for i in range(8):
                want = helpers.exact_target(W[row, 8 * c + i], g[row, 8 * c + i], eta, s[row])
                assert t[n, i].tobytes() == want.tobytes()


def test_targets_divide_by_the_row_scale():
    W = np.full((2, 8), 6.0, np.float32)
    g = np.full((2, 8), 2.0, np.float32)
    t = oracle.targets(W, g, np.array([1.0, 4.0], np.float32), 1.0, np.array([0, 1], np.uint32))
    assert np.all(t[0] == 4.0) and np.all(t[1] == 1.0)


# ---------------------------------------------------------------- selection


def _sort_select(norms, k):
    order = np.lexsort((np.arange(norms.size), -norms.astype(np.float64)))
    return np.sort(order[:k]).astype(np.uint32)


@pytest.mark.parametrize("G,k", [(1, 1), (17, 1), (17, 17), (1000, 10), (4096, 41), (50000, 500)])
def test_select_equals_full_sort(G, k):
    n = (_rng(G + k).chisquare(8, size=G) * 1e-6).astype(np.float32)
    assert np.array_equal(oracle.select(n, k), _sort_select(n, k))


def test_select_ties_take_the_lowest_index():
    n = np.ones(100, np.float32)
    assert list(oracle.select(n, 7)) == list(range(7))
    n[50:60] = 2.0
    assert list(oracle.select(n, 12)) == [0, 1] + list(range(50, 60))
    # duplicated gradient groups straddling the threshold
    n = np.array([3, 1, 2, 2, 2, 0, 2], np.float32)
    assert list(oracle.select(n, 3)) == [0, 2, 3]


def test_select_rejects_bad_arguments():
    n = np.ones(4, np.float32)
    for k in (0, 5):
        with pytest.raises(ValueError):
            oracle.select(n, k)
    n[2] = np.nan
    with pytest.raises(ValueError):
        oracle.select(n, 1)


# ---------------------------------------------------------------- M = 1 search


def test_single_codebook_equals_brute_force():
    r = _rng(3)
    t = r.normal(size=(200, 8)).astype(np.float32)
    book = r.normal(size=(1, 37, 8)).astype(np.float32)
    enc = oracle.encode(t, book, np.zeros((200, 1)))
    best, dist = helpers.brute_force_tuples(t, book)
    assert np.array_equal(enc.codes, best)
    assert np.allclose(enc.d_best, dist, rtol=1e-14, atol=0)
    # d_second is the smallest distance over the other codewords
    d = ((t[:, None, :].astype(np.float64) - book[0][None].astype(np.float64)) ** 2).sum(-1)
    d[np.arange(200), best[:, 0]] = np.inf
    assert np.allclose(enc.d_second, d.min(1), rtol=1e-14, atol=0)


def test_single_codebook_equals_library_kmeans_assignment_on_config_1():
    L = synth.make_config_layer(1)
    idx = np.arange(L.num_groups, dtype=np.uint32)
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    enc = oracle.encode(t, L.codebooks, L.codes)
    lib_codes, lib_dist = vq(t.astype(np.float64), L.codebooks[0].astype(np.float64))
    decisive = (enc.d_second - enc.d_best) > 1e-9 * enc.d_second
    assert decisive.mean() > 0.99
    assert np.array_equal(enc.codes[decisive, 0], lib_codes[decisive])
    assert np.allclose(np.sqrt(enc.d_best), lib_dist, rtol=1e-10)


def test_distance_expansion_identity():
    r = _rng(4)
    t = r.normal(size=(64, 8)).astype(np.float32)
    book = r.normal(size=(1, 50, 8)).astype(np.float32)
    enc = oracle.encode(t, book, np.zeros((64, 1)))
    t64, c64 = t.astype(np.float64), book[0].astype(np.float64)
    score = (c64 ** 2).sum(1)[None, :] - 2.0 * t64 @ c64.T  # ||c||^2 - 2 t.c
    assert np.array_equal(score.argmin(1), enc.codes[:, 0])
    assert np.allclose(score.min(1) + (t64 ** 2).sum(1), enc.d_best, rtol=1e-10, atol=1e-12)


def test_equidistant_codewords_take_the_lower_code():
    book = np.zeros((1, 4, 8), np.float32)
    book[0, 1, 0] = 1.0
    book[0, 2, 0] = -1.0
    book[0, 3, 0] = 1.0  # duplicate of codeword 1
    t = np.zeros((3, 8), np.float32)
    t[1, 0] = 0.9
    t[2, 0] = -0.9
    enc = oracle.encode(t, book, np.full((3, 1), 3))
    assert list(enc.codes[:, 0]) == [0, 1, 2]
    assert enc.d_second[1] == enc.d_best[1]  # the duplicate is the runner-up


def test_transposed_codebook_would_fail():
    """A codebook read as [dg][K] instead of [K][dg] gives different codes on a
    non-symmetric example; the brute force reads [K][dg]."""
    r = _rng(5)
    book = r.normal(size=(1, 8, 8)).astype(np.float32)
    t = book[0].copy() + 0.01 * r.normal(size=(8, 8)).astype(np.float32)
    enc = oracle.encode(t, book, np.zeros((8, 1)))
    assert list(enc.codes[:, 0]) == list(range(8))


# ---------------------------------------------------------------- M = 2 beam search


def _two_books(seed, K, dg=8, scale2=0.3):
    r = _rng(seed)
    return np.stack([r.normal(size=(K, dg)), scale2 * r.normal(size=(K, dg))]).astype(np.float32)


def test_beam_at_least_K_equals_exhaustive_enumeration():
    books = _two_books(6, 12)
    t = _rng(7).normal(size=(150, 8)).astype(np.float32)
    prev = _rng(8).integers(0, 12, size=(150, 2))
    best, dist = helpers.brute_force_tuples(t, books)
    for beam in (12, 40):
        enc = oracle.encode(t, books, prev, beam=beam)
        assert np.array_equal(enc.codes, best)
        assert np.allclose(enc.d_best, dist, rtol=1e-13, atol=0)


def test_beam_one_equals_greedy_residual_quantisation():
    books = _two_books(9, 31)
    t = _rng(10).normal(size=(300, 8)).astype(np.float32)
    t64, b64 = t.astype(np.float64), books.astype(np.float64)
    k1 = ((t64[:, None] - b64[0][None]) ** 2).sum(-1).argmin(1)
    res = t64 - b64[0][k1]
    k2 = ((res[:, None] - b64[1][None]) ** 2).sum(-1).argmin(1)
    greedy = np.stack([k1, k2], 1)
    enc = oracle.encode(t, books, greedy, beam=1)  # previous tuple = greedy result: adds nothing
    assert np.array_equal(enc.codes, greedy)
    assert np.allclose(enc.d_best, helpers.recon_error(t, books, greedy), rtol=1e-13, atol=0)


def test_zero_second_codebook_reduces_to_single_codebook():
    books = _two_books(11, 20)
    books[1] = 0.0
    t = _rng(12).normal(size=(100, 8)).astype(np.float32)
    enc2 = oracle.encode(t, books, np.zeros((100, 2)), beam=8)
    enc1 = oracle.encode(t, books[:1], np.zeros((100, 1)))
    assert np.array_equal(enc2.codes[:, 0], enc1.codes[:, 0])
    assert np.all(enc2.codes[:, 1] == 0)  # all second codes tie; lowest wins
    assert np.array_equal(enc2.d_best, enc1.d_best)


def test_beam_result_between_optimum_and_previous_tuple():
    books = _two_books(13, 64, scale2=1.0)  # equal-energy books: the beam is a real heuristic here
    t = _rng(14).normal(size=(400, 8)).astype(np.float32)
    prev = _rng(15).integers(0, 64, size=(400, 2))
    enc = oracle.encode(t, books, prev, beam=2)
    opt_codes, opt = helpers.brute_force_tuples(t, books)
    d_prev = helpers.recon_error(t, books, prev)
    d_got = helpers.recon_error(t, books, enc.codes)
    assert np.allclose(d_got, enc.d_best, rtol=1e-13, atol=0)
    assert np.all(d_got >= opt * (1 - 1e-13))
    assert np.all(d_got <= d_prev * (1 + 1e-13))
    assert (d_got > opt * (1 + 1e-9)).any()  # the heuristic is not secretly exhaustive


def test_previous_tuple_is_kept_when_it_beats_the_beam():
    """Put the exhaustive optimum in as the previous tuple: the pool contains
    it, so the result must reach the optimum even with beam 1."""
    books = _two_books(16, 32, scale2=1.0)
    t = _rng(17).normal(size=(200, 8)).astype(np.float32)
    opt_codes, opt = helpers.brute_force_tuples(t, books)
    enc = oracle.encode(t, books, opt_codes, beam=1)
    assert np.allclose(enc.d_best, opt, rtol=1e-13, atol=0)
    assert np.array_equal(enc.codes, opt_codes)


def test_beam_boundary_distances_are_the_8th_and_9th_stage_one_candidates():
    books = _two_books(18, 40)
    t = _rng(19).normal(size=(50, 8)).astype(np.float32)
    enc = oracle.encode(t, books, np.zeros((50, 2)), beam=8)
    d1 = np.sort(((t[:, None].astype(np.float64) - books[0][None].astype(np.float64)) ** 2).sum(-1), axis=1)
    assert np.allclose(enc.beam_d_in, d1[:, 7], rtol=1e-13, atol=0)
    assert np.allclose(enc.beam_d_out, d1[:, 8], rtol=1e-13, atol=0)


def test_three_codebooks_with_wide_beam_equal_enumeration():
    r = _rng(20)
    books = np.stack([r.normal(size=(5, 4)), 0.5 * r.normal(size=(5, 4)), 0.25 * r.normal(size=(5, 4))]).astype(np.float32)
    t = r.normal(size=(40, 4)).astype(np.float32)
    enc = oracle.encode(t, books, np.zeros((40, 3)), beam=25)
    best, dist = helpers.brute_force_tuples(t, books)
    assert np.array_equal(enc.codes, best)


def _residual_books(seed, M, K, dg=8, decay=0.5):
    r = _rng(seed)
    return np.stack([(decay ** m) * r.normal(size=(K, dg)) for m in range(M)]).astype(np.float32)


@pytest.mark.parametrize("M", [3, 4])
@pytest.mark.parametrize("K", [4, 7, 12])
@pytest.mark.parametrize("beam", [1, 2, 3, 5])
def test_narrow_beam_over_three_and_four_codebooks_against_a_stagewise_search(M, K, beam):
    """Beams that really drop partial tuples at the second and third stage (beam < kept x K): every tuple
    and distance against an independent stage-by-stage search that shares nothing with the checker."""
    books = _residual_books(100 + 10 * M + K, M, K)
    r = _rng(200 + beam)
    t = r.normal(size=(25, 8)).astype(np.float32)
    prev = r.integers(0, K, size=(25, M))
    enc = oracle.encode(t, books, prev, beam=beam)
    want_codes, want_d = helpers.stagewise_beam(t, books, beam, prev)
    assert np.array_equal(enc.codes, want_codes)
    assert np.array_equal(enc.d_best, want_d)
    # without the previous tuple in the pool (previous tuple := the result, which adds nothing)
    free_codes, free_d = helpers.stagewise_beam(t, books, beam)
    enc_free = oracle.encode(t, books, free_codes, beam=beam)
    assert np.array_equal(enc_free.codes, free_codes)
    assert np.array_equal(enc_free.d_best, free_d)


def test_narrow_beam_really_truncates_and_is_a_heuristic():
    """The cases above are not secretly exhaustive: with three codebooks of 7 and beam 2 some targets end
    above the enumerated optimum, and widening the beam to all tuples reaches it."""
    books = _residual_books(131, 3, 7, decay=0.9)
    t = _rng(132).normal(size=(60, 8)).astype(np.float32)
    narrow, d_narrow = helpers.stagewise_beam(t, books, 2)
    best, d_best = helpers.brute_force_tuples(t, books)
    assert (d_narrow > d_best * (1 + 1e-9)).any()
    enc = oracle.encode(t, books, narrow, beam=2)
    assert np.array_equal(enc.codes, narrow)
    wide = oracle.encode(t, books, narrow, beam=49)
    assert np.array_equal(wide.codes, best)


@pytest.mark.parametrize("M", [3, 4])
def test_beam_one_over_more_codebooks_equals_greedy_residual_quantisation(M):
    K = 9
    books = _residual_books(140 + M, M, K)
    t = _rng(150 + M).normal(size=(120, 8)).astype(np.float32)
    res = t.astype(np.float64)
    greedy = []
    for m in range(M):
        km = ((res[:, None] - books[m].astype(np.float64)[None]) ** 2).sum(-1).argmin(1)
        res = res - books[m].astype(np.float64)[km]
        greedy.append(km)
    greedy = np.stack(greedy, 1)
    enc = oracle.encode(t, books, greedy, beam=1)
    assert np.array_equal(enc.codes, greedy)
    assert np.allclose(enc.d_best, (res ** 2).sum(1), rtol=1e-13, atol=0)


def test_equal_partial_distances_keep_the_smaller_tuple_at_a_truncating_stage():
    """Duplicate codewords make exact ties among partial tuples; the kept ones must be the
    lexicographically smaller tuples, which decides the final code when the beam is narrow."""
    r = _rng(160)
    b1 = r.normal(size=(6, 8)).astype(np.float32)
    b1[4] = b1[1]  # codes 1 and 4 of the first codebook are the same vector
    b2 = (0.5 * r.normal(size=(6, 8))).astype(np.float32)
    b2[5] = b2[2]
    b3 = (0.25 * r.normal(size=(6, 8))).astype(np.float32)
    books = np.stack([b1, b2, b3])
    t = (b1[1] + b2[2] + 0.01 * r.normal(size=(30, 8))).astype(np.float32)
    for beam in (1, 2, 3):
        want_codes, want_d = helpers.stagewise_beam(t, books, beam)
        enc = oracle.encode(t, books, want_codes, beam=beam)
        assert np.array_equal(enc.codes, want_codes)
        assert np.all(enc.codes[:, 0] != 4)  # the duplicate with the larger code never wins


def test_tuple_error_matches_independent_formula():
    books = _two_books(21, 16)
    t = _rng(22).normal(size=(30, 8)).astype(np.float32)
    codes = _rng(23).integers(0, 16, size=(30, 2))
    assert np.allclose(oracle.tuple_error(t, books, codes), helpers.recon_error(t, books, codes), rtol=1e-13, atol=0)


# ---------------------------------------------------------------- whole step: invariants


def _small_layer(M, K=32, rows=16, cols=64, fp16=True, seed=30):
    r = _rng(seed)
    W = r.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    g = r.normal(0, 1e-3, size=(rows, cols)).astype(np.float32)
    s = np.abs(W).max(1).astype(np.float32)
    G = rows * cols // 8
    grp = (W / s[:, None]).reshape(G, 8)
    dt = np.float16 if fp16 else np.float32
    books = [grp[r.choice(G, K, replace=False)].astype(dt)]
    if M == 2:
        books.append((0.3 * grp[r.choice(G, K, replace=False)]).astype(dt))
    books = np.stack(books)
    codes = r.integers(0, K, size=(G, M)).astype(np.uint8)
    return W, g, s, books, codes


@pytest.mark.parametrize("M", [1, 2])
def test_monotone_and_local(M):
    W, g, s, books, codes = _small_layer(M)
    G = codes.shape[0]
    k = 13
    res = oracle.vstep(W, g, s, books, codes, eta=1.0, k=k)
    # locality: exactly k distinct in-range indices, everything else untouched
    assert res.idx.size == k and np.unique(res.idx).size == k and res.idx.max() < G
    assert np.all(np.diff(res.idx.astype(np.int64)) > 0)
    untouched = np.ones(G, bool)
    untouched[res.idx] = False
    assert np.array_equal(res.codes[untouched], codes[untouched])
    # monotone: new error <= error of the previous code (Lemma 3.3), from an independent formula
    d_prev = helpers.recon_error(res.t, books, codes[res.idx])
    d_new = helpers.recon_error(res.t, books, res.codes[res.idx])
    assert np.all(d_new <= d_prev * (1 + 1e-13))
    assert (d_new < d_prev).any()
    # the selected groups are those with the largest ||eta g||^2, from an independent formula
    n64 = (g.astype(np.float64).reshape(G, 8) ** 2).sum(1)
    assert n64[res.idx].min() >= np.delete(n64, res.idx).max() * (1 - 1e-6)


@pytest.mark.parametrize("M", [1, 2])
def test_fixed_point_and_round_trip(M):
    """W := dequant(codes) and eta = 0: the step leaves every code unchanged with
    zero error (for small steps the optimal solution is y itself, Section 3.2)."""
    W, g, s, books, codes = _small_layer(M, K=32, fp16=True, seed=31)
    # power-of-two scales make W/s exact, so the fixed point holds bit for bit
    s = np.exp2(_rng(32).integers(-4, 3, size=s.shape)).astype(np.float32)
    rows, cols = W.shape
    if M == 2:
        # keep only tuples whose reconstruction is unique enough: use the tuple the search itself returns
        W0 = oracle.dequant(codes, books, s, rows, cols)
        codes = oracle.vstep(W0, g, s, books, codes, eta=0.0, k=codes.shape[0]).codes
    What = oracle.dequant(codes, books, s, rows, cols)
    res = oracle.vstep(What, g, s, books, codes, eta=0.0, k=codes.shape[0])
    if M == 1:
        assert np.array_equal(res.codes, codes)
        assert np.all(res.enc.d_best == 0.0)
    else:
        assert np.array_equal(res.codes, codes)
        assert np.all(res.enc.d_best <= 1e-12)


def test_dequant_closed_form_and_fp16_rounding():
    W, g, s, books, codes = _small_layer(2, seed=33)
    rows, cols = W.shape
    What = oracle.dequant(codes, books, s, rows, cols)
    b32 = books.astype(np.float32)
    want = (b32[0][codes[:, 0]] + b32[1][codes[:, 1]]).reshape(rows, cols) * s[:, None]
    assert What.dtype == np.float32 and What.tobytes() == want.astype(np.float32).tobytes()
    # M = 1: the codeword itself times the scale
    What1 = oracle.dequant(codes[:, :1], books[:1], s, rows, cols)
    assert np.array_equal(What1, b32[0][codes[:, 0]].reshape(rows, cols) * s[:, None])
    # a wrong row/column mapping of the scale would show on a non-square layer
    assert rows != cols


def test_config_1_all_groups_reencoded_matches_brute_force():
    L = synth.make_config_layer(1)
    k = synth.subspace_size("1.0", L.num_groups)
    assert k == L.num_groups == 8192
    res = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k)
    assert np.array_equal(res.idx, np.arange(k))
    t = (L.W.astype(np.float64) - L.g.astype(np.float64)).reshape(k, 8)  # s = 1, eta = 1
    d = ((t[:, None] - L.codebooks[0][None].astype(np.float64)) ** 2).sum(-1)
    decisive = (res.enc.d_second - res.enc.d_best) > 1e-6 * res.enc.d_second
    assert np.array_equal(d.argmin(1)[decisive], res.enc.codes[decisive, 0])


# ------------------------------------------------------------------ P step: backprop to codebooks / scales, Adam


def _pstep_case(seed, rows=12, cols=40, K=9, M=2):
    rng = np.random.default_rng(seed)
    g = rng.normal(size=(rows, cols)).astype(np.float32)
    s = rng.uniform(0.5, 2.0, rows).astype(np.float32)
    books = rng.normal(size=(M, K, 8)).astype(np.float32)
    codes = rng.integers(0, K, (rows * cols // 8, M))
    return g, s, books, codes, rows, cols


def test_pstep_grad_equals_library_autodiff_of_dequantisation():
    """Algorithm 3: grad_codebooks = backprop(grad_phi).  Differentiate <g, W_hat(codebooks, scales)> with a
    library's reverse mode and compare (for M = 1 the forward map has no rounding, so the match is to fp64
    accuracy; for M = 2 the checker differentiates through the binary32 sum of the two codewords)."""
    import torch
    for M, tol_s in ((1, 1e-12), (2, 1e-5)):
        g, s, books, codes, rows, cols = _pstep_case(3 + M, M=M)
        gb, gs = oracle.pstep_grad(g, s, codes, books, rows, cols)
        Bk = torch.tensor(books, dtype=torch.float64, requires_grad=True)
        S = torch.tensor(s, dtype=torch.float64, requires_grad=True)
        c = torch.tensor(codes)
        v = sum(Bk[m][c[:, m]] for m in range(M)).reshape(rows, cols // 8, 8)
        W = (S[:, None, None] * v).reshape(rows, cols)
        (W * torch.tensor(g, dtype=torch.float64)).sum().backward()
        assert np.abs(gb - Bk.grad.numpy()).max() <= 1e-12 * np.abs(gb).max()
        assert np.abs(gs - S.grad.numpy()).max() <= tol_s * np.abs(gs).max()


def test_pstep_grad_matches_finite_differences_of_a_quadratic():
    """phi(W_hat) = 1/2 ||W_hat - Z||^2 has gradient W_hat - Z; perturb single codebook entries and scales."""
    g0, s, books, codes, rows, cols = _pstep_case(11, M=1)
    Z = g0  # any matrix
    def phi(bk, sc):
        W = oracle.dequant(codes, bk, sc, rows, cols).astype(np.float64)
        return 0.5 * ((W - Z) ** 2).sum()
    W0 = oracle.dequant(codes, books, s, rows, cols)
    g = (W0.astype(np.float64) - Z).astype(np.float32)
    gb, gs = oracle.pstep_grad(g, s, codes, books, rows, cols)
    h = 1e-2  # phi is quadratic: the central difference is exact up to rounding
    for (kap, i) in ((0, 0), (3, 5), (8, 7)):
        bp, bm = books.copy(), books.copy()
        bp[0, kap, i] += h
        bm[0, kap, i] -= h
        fd = (phi(bp, s) - phi(bm, s)) / (float(bp[0, kap, i]) - float(bm[0, kap, i]))
        assert abs(fd - gb[0, kap, i]) <= 2e-3 * max(1.0, abs(fd))
    for r in (0, 7):
        sp, sm = s.copy(), s.copy()
        sp[r] += h
        sm[r] -= h
        fd = (phi(books, sp) - phi(books, sm)) / (float(sp[r]) - float(sm[r]))
        assert abs(fd - gs[r]) <= 2e-3 * max(1.0, abs(fd))


def test_pstep_grad_linearity_and_single_code():
    g, s, books, codes, rows, cols = _pstep_case(13, M=2)
    gb1, gs1 = oracle.pstep_grad(g, s, codes, books, rows, cols)
    gb2, gs2 = oracle.pstep_grad(2 * g, s, codes, books, rows, cols)  # doubling is exact in binary32
    assert np.array_equal(gb2, 2 * gb1) and np.array_equal(gs2, 2 * gs1)
    # every group uses code (4, 4): the gradient of that codeword is the scaled column-group sum, all others zero
    codes[:] = 4
    gb, _ = oracle.pstep_grad(g, s, codes, books, rows, cols)
    want = (s[:, None].astype(np.float64) * g.astype(np.float64)).reshape(rows, cols // 8, 8).sum(axis=(0, 1))
    assert np.allclose(gb[0, 4], want, rtol=1e-13, atol=1e-13) and np.allclose(gb[1, 4], want, rtol=1e-13, atol=1e-13)
    gb[:, 4] = 0
    assert not gb.any()


def test_adam_first_step_closed_form_and_library():
    """First step from zero moments: update = lr * g / (|g| + eps) whatever the betas; further steps against
    a library Adam (Appendix J: beta1 = 0.9, beta2 = 0.95)."""
    import torch
    rng = np.random.default_rng(17)
    n = 1000
    p0 = rng.normal(size=n).astype(np.float32)
    grads = [rng.normal(size=n) * 10.0 ** rng.integers(-3, 2, n) for _ in range(4)]
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    oracle.adam(p, grads[0], m, v, 1, 3e-4)
    g32 = grads[0].astype(np.float32).astype(np.float64)
    want = p0 - 3e-4 * g32 / (np.abs(g32) + 1e-8)
    assert np.allclose(p, want, rtol=0, atol=2e-7 * np.abs(p0).max() + 1e-9)
    tp = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([tp], lr=3e-4, betas=(0.9, 0.95), eps=1e-8)
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t, gr in enumerate(grads, 1):
        oracle.adam(p, gr, m, v, t, 3e-4)
        tp.grad = torch.tensor(gr.astype(np.float32).astype(np.float64))
        opt.step()
    assert np.allclose(p, tp.detach().numpy(), rtol=0, atol=4e-7 * np.abs(p0).max() + 1e-8)


def test_adam_direction_first_step_and_library():
    """Section 3.4: the V step's gradient is replaced by one Adam update.  First step: g / (|g| + eps); over
    several steps a library Adam with learning rate 1 started at zero accumulates minus the directions."""
    import torch
    rng = np.random.default_rng(19)
    n = 500
    grads = [(rng.normal(size=n) * 10.0 ** rng.integers(-3, 2, n)).astype(np.float32) for _ in range(4)]
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    u = oracle.adam_direction(grads[0], m, v, 1)
    g64 = grads[0].astype(np.float64)
    assert np.allclose(u, g64 / (np.abs(g64) + 1e-8), rtol=3e-7, atol=0)
    tp = torch.zeros(n, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([tp], lr=1.0, betas=(0.9, 0.95), eps=1e-8)
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    acc = np.zeros(n)
    for t, gr in enumerate(grads, 1):
        acc += oracle.adam_direction(gr, m, v, t).astype(np.float64)
        tp.grad = torch.tensor(gr.astype(np.float64))
        opt.step()
    # directions are O(1) and each carries a few binary32 roundings; their sum may cancel, so the bound is absolute
    assert np.allclose(-acc, tp.detach().numpy(), rtol=0, atol=2e-6)


# ---------------------------------------------------------------- groups of 16 weights


def test_group_size_16_norm_is_one_chain_over_sixteen_elements():
    g = (_rng(31).normal(0, 1e-3, size=(4, 48)) * np.array([1, 1e-19, 1e3, 7])[:, None]).astype(np.float32)
    for eta in (1.0, 0.3):
        n = oracle.group_norms(g, eta, group_dim=16)
        assert n.shape == (12,)
        for j in range(12):
            r, c = divmod(j, 3)
            want = helpers.exact_group_norm(g[r, 16 * c:16 * c + 16], eta)
            assert n[j].tobytes() == want.tobytes(), (eta, j)


def test_group_size_16_search_equals_brute_force_and_library():
    r = _rng(32)
    book = r.normal(size=(1, 300, 16)).astype(np.float32)
    t = r.normal(size=(200, 16)).astype(np.float32)
    enc = oracle.encode(t, book, np.zeros((200, 1)))
    d = ((t[:, None, :].astype(np.float64) - book[0][None].astype(np.float64)) ** 2).sum(axis=2)
    assert np.array_equal(enc.codes[:, 0], d.argmin(axis=1))
    assert np.allclose(enc.d_best, d.min(axis=1), rtol=1e-13)
    lib_codes, _ = vq(t.astype(np.float64), book[0].astype(np.float64))
    assert np.array_equal(enc.codes[:, 0], lib_codes)


def test_group_size_16_step_dequant_and_fixed_point():
    L = synth.make_layer(32, 256, cfg=230, codebook_size=128, codebook_fp16=True, group_dim=16)
    G = L.num_groups
    assert G == 32 * 16 and L.codebooks.shape == (1, 128, 16)
    W_hat = oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols)
    want = L.scale[:, None, None] * L.codebooks[0].astype(np.float32)[L.codes[:, 0].astype(int)].reshape(32, 16, 16)
    assert W_hat.tobytes() == want.reshape(32, 256).astype(np.float32).tobytes()
    # the dequantised matrix is its own nearest assignment (distinct codewords), and the step is local
    again = oracle.vstep(W_hat, np.zeros_like(W_hat), L.scale, L.codebooks, L.codes, eta=0.0, k=G)
    assert np.array_equal(again.codes, L.codes) and np.all(again.enc.d_best < 1e-12)
    res = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k=40)
    rest = np.setdiff1d(np.arange(G), res.idx.astype(int))
    assert np.array_equal(res.codes[rest], L.codes[rest])
    t = oracle.targets(L.W, L.g, L.scale, L.eta, res.idx, 16)
    assert np.all(helpers.recon_error(t, L.codebooks, res.codes[res.idx.astype(int)]) <=
                  helpers.recon_error(t, L.codebooks, L.codes[res.idx.astype(int)]) * (1 + 1e-12))
