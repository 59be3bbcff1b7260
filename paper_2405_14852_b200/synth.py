"""Seeded synthetic layers for the V step (inputs only).

This module only draws random numbers and lays them out; it performs none of
the V step's own arithmetic (no norms, no selection, no codeword search, no
dequantisation).  Where the recipe of an input needs a nearest-codeword
assignment (the second residual codebook, "nearest" previous codes) the caller
passes that routine in as ``nearest``; the CPU checker's tests pass theirs and
the benchmark passes the GPU library's.

Recipe (stand-ins for Llama-2 linear layers: only their shapes are real):

* ``W ~ N(0, 0.02^2)`` fp32, ``g ~ N(0, (1e-3)^2)`` fp32, iid.
* per-row scale ``s``: all ones, or ``s_r = max_j |W[r, j]|``.
* codebook: K distinct weight groups of ``W / s`` drawn without replacement
  (rounded to fp16 when the codebook is fp16).
* second residual codebook (M = 2): 256 further groups X of ``W / s``;
  ``C2 = 0.3 * (X - C1[nearest(X, C1)])`` rounded to the codebook dtype.
* previous codes: uniform random in ``[0, K)`` per codebook.

Each array has its own generator: ``numpy.random.default_rng(1000 * cfg +
stream)`` with streams 0 = W, 1 = g, 2 = codebook sample, 3 = previous codes,
4 = second codebook sample.
"""
from __future__ import annotations

import dataclasses
from fractions import Fraction
from typing import Callable, Optional

import numpy as np

PVT_F32 = 0
PVT_F16 = 1
PVT_U8 = 0
PVT_U16 = 1


@dataclasses.dataclass
class SynthLayer:
    """Host arrays of one quantised linear layer plus its update direction."""

    rows: int
    cols: int
    group_dim: int
    num_codebooks: int  # M
    codebook_size: int  # K
    beam: int
    eta: float
    W: np.ndarray  # [rows, cols] fp32
    g: np.ndarray  # [rows, cols] fp32
    scale: np.ndarray  # [rows] fp32
    codebooks: np.ndarray  # [M, K, group_dim] fp32 or fp16
    codes: np.ndarray  # [G, M] uint8 or uint16
    name: str = ""

    @property
    def num_groups(self) -> int:
        return self.rows * (self.cols // self.group_dim)

    @property
    def codebook_dtype(self) -> int:
        return PVT_F16 if self.codebooks.dtype == np.float16 else PVT_F32

    @property
    def code_dtype(self) -> int:
        return PVT_U8 if self.codes.dtype == np.uint8 else PVT_U16

    def pairs_per_group(self) -> int:
        """Codeword-pair evaluations the search spends on one group."""
        K = self.codebook_size
        if self.num_codebooks == 1:
            return K
        return K + self.beam * K * (self.num_codebooks - 1)


def subspace_size(tau, num_groups: int) -> int:
    """k = max(1, floor(tau * G)) in exact rational arithmetic."""
    t = Fraction(str(tau))
    if t < 0 or t > 1:
        raise ValueError("tau must lie in [0, 1]")
    return max(1, (t.numerator * num_groups) // t.denominator)


def _scaled_groups(W: np.ndarray, scale: np.ndarray, group_ids: np.ndarray, dg: int) -> np.ndarray:
    rows, cols = W.shape
    gpr = cols // dg
    r = group_ids // gpr
    c = group_ids % gpr
    cols_idx = c[:, None] * dg + np.arange(dg)[None, :]
    vals = W[r[:, None], cols_idx]
    return (vals / scale[r][:, None]).astype(np.float32)


def make_layer(
    rows: int,
    cols: int,
    *,
    cfg: int,
    num_codebooks: int = 1,
    codebook_size: int = 256,
    codebook_fp16: bool = False,
    row_max_scale: bool = True,
    eta: float = 1.0,
    group_dim: int = 8,
    beam: int = 8,
    nearest: Optional[Callable[[np.ndarray, np.ndarray], np.ndarray]] = None,
    name: str = "",
) -> SynthLayer:
    """Draw one layer.  ``nearest(X, C)`` -> index of the codeword of ``C``
    ([K, dg] fp32) closest to each row of ``X`` ([n, dg] fp32); required only
    when ``num_codebooks == 2``."""
    if cols % group_dim:
        raise ValueError("cols must be a multiple of group_dim")
    G = rows * (cols // group_dim)
    K = codebook_size
    if K > G:
        raise ValueError("codebook larger than the number of groups")
    seed = 1000 * cfg
    W = np.random.default_rng(seed + 0).normal(0.0, 0.02, size=(rows, cols)).astype(np.float32)
    g = np.random.default_rng(seed + 1).normal(0.0, 1e-3, size=(rows, cols)).astype(np.float32)
    if row_max_scale:
        scale = np.abs(W).max(axis=1).astype(np.float32)
    else:
        scale = np.ones(rows, dtype=np.float32)
    cb_dtype = np.float16 if codebook_fp16 else np.float32

    pick = np.random.default_rng(seed + 2).choice(G, size=K, replace=False)
    C1 = _scaled_groups(W, scale, pick, group_dim).astype(cb_dtype)
    books = [C1]
    if num_codebooks >= 2:
        if nearest is None:
            raise ValueError("a nearest(X, C) routine is needed to build the further codebooks")
        if num_codebooks > 4:
            raise ValueError("num_codebooks must be 1..4")
        # codebook m+1 = 0.3 x what is left of K further sampled groups after their greedy assignment to
        # codebooks 1..m (streams 4, 5, 6 for codebooks 2, 3, 4)
        for m in range(1, num_codebooks):
            pick_m = np.random.default_rng(seed + 3 + m).choice(G, size=K, replace=False)
            X = _scaled_groups(W, scale, pick_m, group_dim)
            for Cq in books:
                Cq32 = Cq.astype(np.float32)
                X = X - Cq32[np.asarray(nearest(X, Cq32), dtype=np.int64)]
            books.append((np.float32(0.3) * X).astype(cb_dtype))
    codebooks = np.stack(books, axis=0)

    code_np = np.uint8 if K <= 256 else np.uint16
    codes = np.random.default_rng(seed + 3).integers(0, K, size=(G, num_codebooks)).astype(code_np)
    return SynthLayer(
        rows=rows, cols=cols, group_dim=group_dim, num_codebooks=num_codebooks,
        codebook_size=K, beam=beam, eta=float(eta), W=W, g=g, scale=scale,
        codebooks=np.ascontiguousarray(codebooks), codes=np.ascontiguousarray(codes), name=name,
    )


# The benchmark configurations: (name, rows, cols, M, K, fp16 codebook, row-max scale, taus).
CONFIGS = {
    1: [("tiny_256x256_1x8", 256, 256, 1, 256, False, False, ("1.0",))],
    2: [("llama2_7b_attn_4096x4096_1x16", 4096, 4096, 1, 65536, True, True, ("0.01",))],
    3: [
        ("llama2_7b_mlp_11008x4096_2x8", 11008, 4096, 2, 256, True, True, ("0.001", "0.01", "0.1")),
        ("llama2_7b_mlp_4096x11008_2x8", 4096, 11008, 2, 256, True, True, ("0.001", "0.01", "0.1")),
    ],
    4: [
        ("llama2_13b_5120x5120_1x16", 5120, 5120, 1, 65536, True, True, ("0.01",)),
        ("llama2_13b_5120x5120_2x8", 5120, 5120, 2, 256, True, True, ("0.01",)),
        ("llama2_13b_13824x5120_1x16", 13824, 5120, 1, 65536, True, True, ("0.01",)),
        ("llama2_13b_13824x5120_2x8", 13824, 5120, 2, 256, True, True, ("0.01",)),
        ("llama2_13b_5120x13824_1x16", 5120, 13824, 1, 65536, True, True, ("0.01",)),
        ("llama2_13b_5120x13824_2x8", 5120, 13824, 2, 256, True, True, ("0.01",)),
    ],
    5: [
        ("llama2_70b_8192x8192_1x16", 8192, 8192, 1, 65536, True, True, ("0.01", "1.0")),
        ("llama2_70b_8192x1024_1x16", 8192, 1024, 1, 65536, True, True, ("0.01", "1.0")),
        ("llama2_70b_28672x8192_1x16", 28672, 8192, 1, 65536, True, True, ("0.01", "1.0")),
        ("llama2_70b_8192x28672_1x16", 8192, 28672, 1, 65536, True, True, ("0.01", "1.0")),
    ],
}


# One transformer block of the largest model of the benchmark table: the seven linear layers of a
# Llama-2-70B decoder block (grouped-query attention: key / value projections are 8192 x 1024), as
# (layer name, entry of CONFIGS[5]).
BLOCK_70B = (("q_proj", 0), ("o_proj", 0), ("k_proj", 1), ("v_proj", 1), ("gate_proj", 2), ("up_proj", 2),
             ("down_proj", 3))
BLOCK_SEED_BASE = 50  # layer i of the block draws from the seed family cfg = BLOCK_SEED_BASE + i


def block_layer_shapes():
    """(name, rows, cols, M, K, fp16 codebook, row-max scale) of every layer of the block."""
    return [(name,) + tuple(CONFIGS[5][which][1:7]) for name, which in BLOCK_70B]


def make_block_layer(i: int, *, seed_offset: int = 0) -> SynthLayer:
    """Layer i of the 70B block (its own seed family, so no two layers share weights or codebooks)."""
    name, rows, cols, M, K, f16, rowmax = block_layer_shapes()[i]
    return make_layer(rows, cols, cfg=BLOCK_SEED_BASE + i + seed_offset, num_codebooks=M, codebook_size=K,
                      codebook_fp16=f16, row_max_scale=rowmax, name=f"llama2_70b_{name}_{rows}x{cols}_1x16")


def make_config_layer(cfg: int, which: int = 0, *, nearest=None) -> SynthLayer:
    name, rows, cols, M, K, f16, rowmax, _ = CONFIGS[cfg][which]
    return make_layer(rows, cols, cfg=cfg, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                      row_max_scale=rowmax, nearest=nearest, name=name)


def config_taus(cfg: int, which: int = 0):
    return CONFIGS[cfg][which][7]
