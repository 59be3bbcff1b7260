"""The single-codebook search on the tensor engine against the CPU checker on randomly drawn (seeded) shapes:
codebook sizes that pad, fill or exceed whole 128-codeword steps and stages, target counts that leave ragged
tiles, sorted and unsorted index lists, groups of 8 and of 16 weights."""
import numpy as np
import pytest

import test_gpu_g16 as g16
import test_gpu_parity as parity
from paper_2405_14852_b200 import synth

pytestmark = pytest.mark.gpu

CODEBOOK_SIZES = [130, 256, 1000, 1024, 1500, 2048, 4096, 5000, 16384, 40000, 65536]


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_tensor_search_random_shapes(seed):
    rng = np.random.default_rng(seed)
    for case in range(24):
        gd = int(rng.choice([8, 8, 16]))
        K = int(rng.choice(CODEBOOK_SIZES))
        rows = int(rng.choice([64, 128, 256, 512, 1024]))
        cols = gd * int(rng.integers(8, 129))
        G = rows * cols // gd
        K = min(K, max(2, G // 2))
        k = int(rng.integers(1, min(G, 6000) + 1))
        L = synth.make_layer(rows, cols, cfg=300 + 100 * seed + case, codebook_size=K, codebook_fp16=True, group_dim=gd)
        idx = rng.choice(G, size=k, replace=False).astype(np.uint32)
        if rng.random() < 0.5:
            idx = np.sort(idx)
        with parity.search_engine("tensor"):
            if gd == 8:
                exact, _ = parity.check_encode(L, idx)
                assert exact >= k - max(4, k // 500), (case, gd, K, rows, cols, k)
            else:
                g16._encode_case(K, True, rows, cols, k, L=L, idx=idx)
