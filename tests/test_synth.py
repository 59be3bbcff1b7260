"""The seeded input generator: determinism, shapes, recipe."""
import numpy as np
import pytest

from paper_2405_14852_b200 import synth


def test_subspace_size_is_exact():
    assert synth.subspace_size("0.01", 2097152) == 20971
    assert synth.subspace_size("0.001", 5636096) == 5636
    assert synth.subspace_size("0.1", 5636096) == 563609
    assert synth.subspace_size("1.0", 8192) == 8192
    assert synth.subspace_size("0.01", 10) == 1  # at least one group


def test_layer_is_deterministic_and_shaped():
    a = synth.make_layer(64, 128, cfg=7, codebook_size=64, codebook_fp16=True)
    b = synth.make_layer(64, 128, cfg=7, codebook_size=64, codebook_fp16=True)
    for f in ("W", "g", "scale", "codebooks", "codes"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert a.W.dtype == np.float32 and a.codebooks.dtype == np.float16 and a.codes.dtype == np.uint8
    assert a.codebooks.shape == (1, 64, 8) and a.codes.shape == (a.num_groups, 1)
    assert np.array_equal(a.scale, np.abs(a.W).max(1))
    # codewords are distinct scaled weight groups, so no component exceeds 1 in magnitude
    assert np.abs(a.codebooks.astype(np.float32)).max() <= 1.0
    assert np.unique(a.codebooks[0], axis=0).shape[0] == 64
    assert abs(a.W.std() - 0.02) < 2e-3 and abs(a.g.std() - 1e-3) < 1e-4


def test_second_codebook_uses_the_supplied_assignment():
    calls = []

    def first_codeword(X, C):
        calls.append((X.shape, C.shape))
        return np.zeros(X.shape[0], dtype=np.int64)

    L = synth.make_layer(64, 128, cfg=8, num_codebooks=2, codebook_size=32, codebook_fp16=True, nearest=first_codeword)
    assert calls == [((32, 8), (32, 8))]
    assert L.codebooks.shape == (2, 32, 8) and L.codes.shape == (L.num_groups, 2)
    assert L.pairs_per_group() == 32 + 8 * 32
    with pytest.raises(ValueError):
        synth.make_layer(64, 128, cfg=8, num_codebooks=2, codebook_size=32)
