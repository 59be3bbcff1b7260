"""Pins of the CPU checker's straight-through buffer (Appendix E) and random subspace rules (the small-scale
experiments' appendix: uniform and gradient-proportional sampling of the subspace)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import helpers
from oracle import pvt_oracle as oracle


# ------------------------------------------------------------------ straight-through buffer


def test_buffer_update_is_one_fused_operation_per_weight():
    r = np.random.default_rng(1)
    buf = r.normal(0, 0.02, size=200).astype(np.float32)
    g = r.normal(0, 1e-3, size=200).astype(np.float32)
    eta = np.float32(0.37)
    got = oracle.ste_accumulate(buf, g, float(eta))
    for i in range(200):
        exact = Fraction(float(buf[i])) - Fraction(float(eta)) * Fraction(float(g[i]))
        assert got[i] == helpers.round_to_f32(exact)
    assert np.array_equal(oracle.ste_accumulate(buf, g, 0.0), buf)


def test_small_updates_add_up_in_the_buffer_until_the_code_flips():
    """Scalar weights (embedded in groups of 8 by zero padding), value set {0, 1}, eta = 1 and the same update
    -0.125 every step (all values are exact in binary32).  The plain V step restarts from the dequantised weight
    0 each time: its target 0.125 is nearest to 0 for ever.  The buffer goes 0.25, 0.375, 0.5 (a tie: the lower
    code stays), 0.625: the code flips at the fourth step -- the appendix's argument why the buffer prevents
    stalling."""
    books = np.zeros((1, 2, 8), dtype=np.float32)
    books[0, 1, 0] = 1.0
    scale = np.ones(1, dtype=np.float32)
    g = np.zeros((1, 8), dtype=np.float32)
    g[0, 0] = -0.125
    codes = np.zeros((1, 1), dtype=np.uint8)
    buf = np.zeros((1, 8), dtype=np.float32)
    buf[0, 0] = 0.125
    seen = []
    for step in range(4):
        buf, res = oracle.vstep_ste(buf, g, scale, books, codes, eta=1.0, k=1)
        codes = res.codes
        seen.append((float(buf[0, 0]), int(codes[0, 0])))
    assert seen == [(0.25, 0), (0.375, 0), (0.5, 0), (0.625, 1)]
    # without the buffer: W is the dequantised weight of code 0 every step
    plain = np.zeros((1, 1), dtype=np.uint8)
    for step in range(8):
        W = oracle.dequant(plain, books, scale, 1, 8)
        plain = oracle.vstep(W, g, scale, books, plain, 1.0, 1).codes
    assert int(plain[0, 0]) == 0


def test_step_against_the_buffer_equals_a_plain_step_on_the_moved_weights():
    r = np.random.default_rng(2)
    rows, cols, K = 16, 64, 32
    W = r.normal(0, 0.02, size=(rows, cols)).astype(np.float32)
    g = r.normal(0, 1e-3, size=(rows, cols)).astype(np.float32)
    s = np.abs(W).max(1).astype(np.float32)
    G = rows * cols // 8
    books = (W / s[:, None]).reshape(G, 8)[r.choice(G, K, replace=False)][None].astype(np.float16)
    codes = r.integers(0, K, size=(G, 1)).astype(np.uint8)
    new_buf, res = oracle.vstep_ste(W, g, s, books, codes, eta=0.5, k=20)
    assert np.array_equal(res.idx, oracle.select(oracle.group_norms(g, 0.5), 20))
    # targets are the buffer over the scale, exactly (a zero step changes no value)
    want_t = (new_buf.reshape(G, 8)[res.idx.astype(np.int64)] / s[res.idx.astype(np.int64) // (cols // 8)][:, None])
    assert np.array_equal(res.t, want_t.astype(np.float32))
    untouched = np.setdiff1d(np.arange(G), res.idx.astype(np.int64))
    assert np.array_equal(res.codes[untouched], codes[untouched])


# ------------------------------------------------------------------ the generator


def _hex_words(a):
    return [int(x) for x in a]


def test_philox_known_answers():
    vec = {}
    with open(os.path.join(helpers.GOLDEN, "philox4x32_10_known_answers.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, vals = line.split(":")
                vec[key.strip()] = [int(v, 16) for v in vals.split()]
    for case in ("zero", "ones", "pi"):
        got = oracle.philox4x32_10(vec[f"counter_{case}"], vec[f"key_{case}"])
        assert _hex_words(got) == vec[f"output_{case}"]


def test_fixed_logarithm_sequence_against_the_c_library():
    rs = [0, 1, 2, 3, 5, 255, 256, 12345, 0x7fffffff, 0x80000000, 0xb504f333, 0xb504f334, 0xfffffffe, 0xffffffff]
    rs += [int(x) for x in np.random.default_rng(3).integers(0, 2 ** 32, size=2000)]
    for r in rs:
        want = -math.log((r + 0.5) * 2.0 ** -32)
        got = oracle.neglog_u32(r)
        assert got > 0.0
        assert abs(got - want) <= 4e-16 * max(want, 1.0)  # a few units in the last place of the logarithm


# ------------------------------------------------------------------ uniform rule


def test_uniform_keys_are_the_top_24_bits_of_the_generators_first_word():
    seed = (5 << 32) | 77
    keys = oracle.sample_keys(300, oracle.SAMPLE_UNIFORM, seed)
    for j in (0, 1, 17, 299):
        r = int(oracle.philox4x32_10([j, 0, 0, 0], [77, 5])[0])
        assert keys[j] == np.float32(r >> 8)


@pytest.mark.parametrize("G,k", [(1, 1), (10, 1), (10, 10), (1000, 25), (4099, 4098)])
def test_uniform_subspace_is_a_k_subset(G, k):
    idx = oracle.sample_subspace(G, k, oracle.SAMPLE_UNIFORM, seed=9)
    assert idx.size == k and np.unique(idx).size == k and idx.max() < G
    assert np.all(idx[1:] > idx[:-1]) or k == 1
    keys = oracle.sample_keys(G, oracle.SAMPLE_UNIFORM, 9)
    order = sorted(range(G), key=lambda j: (-float(keys[j]), j))  # full sort: largest key, then lowest index
    assert sorted(order[:k]) == [int(i) for i in idx]


def test_uniform_inclusion_frequencies():
    """Every group is in the subspace with probability k/G: 2000 seeds, G = 40, k = 10; each count within five
    standard deviations of the binomial mean, and the mean count exact (every draw has k members)."""
    G, k, n = 40, 10, 2000
    counts = np.zeros(G)
    for seed in range(n):
        counts[oracle.sample_subspace(G, k, oracle.SAMPLE_UNIFORM, seed).astype(np.int64)] += 1
    p = k / G
    assert counts.sum() == n * k
    assert np.all(np.abs(counts - n * p) <= 5 * math.sqrt(n * p * (1 - p)))
    # different seeds give different subspaces
    assert not np.array_equal(oracle.sample_subspace(1000, 25, 0, 1), oracle.sample_subspace(1000, 25, 0, 2))


# ------------------------------------------------------------------ proportional rule


def test_proportional_keys_follow_their_definition():
    norms = np.array([0.0, 1.0, 3.0, 2.5e-7, 7.0], dtype=np.float32)
    keys = oracle.sample_keys(5, oracle.SAMPLE_PROPORTIONAL, 11, norms)
    assert keys[0] == 0.0
    for j in range(1, 5):
        r = int(oracle.philox4x32_10([j, 0, 0, 0], [11, 0])[0])
        want = np.float32(float(norms[j]) / oracle.neglog_u32(r))  # binary64 quotient rounded once to binary32
        assert keys[j] == want


def test_one_draw_is_proportional_to_the_weights():
    """k = 1: the group with the earliest exponential clock; P(j) = w_j / sum w.  Weights 1 : 3 : 0 : 4."""
    norms = np.array([1.0, 3.0, 0.0, 4.0], dtype=np.float32)
    n = 4000
    counts = np.zeros(4)
    for seed in range(n):
        counts[int(oracle.sample_subspace(4, 1, oracle.SAMPLE_PROPORTIONAL, seed, norms)[0])] += 1
    assert counts[2] == 0  # weight 0 is never drawn while positive weights remain
    for j, p in ((0, 1 / 8), (1, 3 / 8), (3, 4 / 8)):
        assert abs(counts[j] - n * p) <= 5 * math.sqrt(n * p * (1 - p))


def test_second_draw_is_proportional_among_the_rest():
    """k = 2 of three groups with weights 1 : 2 : 3 (drawing without replacement): P(group 0 left out) =
    sum over first picks of P(first) P(second | first) with group 0 never picked = (2/6)(3/4) + (3/6)(2/3)."""
    norms = np.array([1.0, 2.0, 3.0], dtype=np.float32)
    n = 6000
    left_out = np.zeros(3)
    for seed in range(n):
        idx = set(int(i) for i in oracle.sample_subspace(3, 2, oracle.SAMPLE_PROPORTIONAL, seed, norms))
        left_out[list({0, 1, 2} - idx)[0]] += 1
    p0 = (2 / 6) * (3 / 4) + (3 / 6) * (2 / 3)
    assert abs(left_out[0] - n * p0) <= 5 * math.sqrt(n * p0 * (1 - p0))
    assert left_out[0] > left_out[1] > left_out[2]


def test_equal_weights_are_drawn_uniformly_and_zero_weights_last():
    G, k, n = 30, 6, 1500
    norms = np.full(G, 2.0, dtype=np.float32)
    counts = np.zeros(G)
    for seed in range(n):
        counts[oracle.sample_subspace(G, k, oracle.SAMPLE_PROPORTIONAL, seed, norms).astype(np.int64)] += 1
    p = k / G
    assert np.all(np.abs(counts - n * p) <= 5 * math.sqrt(n * p * (1 - p)))
    # more draws than positive weights: the zero-weight groups fill up in index order (all their keys tie at 0)
    norms = np.array([0, 5, 0, 0, 1, 0], dtype=np.float32)
    assert [int(i) for i in oracle.sample_subspace(6, 4, oracle.SAMPLE_PROPORTIONAL, 3, norms)] == [0, 1, 2, 4]


def test_stored_index_lists_are_reproduced():
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_sampled_subspaces",
                                                  os.path.join(helpers.GOLDEN, "make_sampled_subspaces.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = {}
    with open(os.path.join(helpers.GOLDEN, "sampled_subspaces.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, vals = line.split(":")
                stored[name.strip()] = [int(v) for v in vals.split()]
    for name, groups, k, mode, seed in mod.CASES:
        norms = mod.norms_for(groups) if mode == oracle.SAMPLE_PROPORTIONAL else None
        assert [int(i) for i in oracle.sample_subspace(groups, k, mode, seed, norms)] == stored[name]
