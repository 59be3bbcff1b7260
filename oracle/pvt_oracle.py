"""ctypes binding of the CPU checker (``pvt_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg; never by the GPU library or its Python binding.
The checker is compiled on first use with ``gcc -O2 -ffp-contract=off
-fopenmp`` (no fused operations other than its explicit ``fmaf`` calls).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pvt_oracle.c")
_LIB = os.path.join(_HERE, "libpvt_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker into ``libpvt_oracle.so`` next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-Wall",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.pvt_oracle_num_threads.restype = ctypes.c_int
        L.pvt_oracle_select.restype = ctypes.c_int
        L.pvt_oracle_encode.restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().pvt_oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().pvt_oracle_set_num_threads(ctypes.c_int(n))


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def group_norms(g, eta: float, group_dim: int = 8) -> np.ndarray:
    """Squared update norm per group, fp32 [G]."""
    g = _f32(g)
    rows, cols = g.shape
    out = np.empty(rows * (cols // group_dim), dtype=np.float32)
    lib().pvt_oracle_group_norms(_p(g, ctypes.c_float), ctypes.c_int64(rows), ctypes.c_int64(cols),
                                 ctypes.c_int32(group_dim), ctypes.c_float(eta), _p(out, ctypes.c_float))
    return out


def select(norms, k: int) -> np.ndarray:
    """Indices of the k largest norms (ties: lowest index), ascending, uint32 [k]."""
    norms = _f32(norms)
    out = np.empty(k, dtype=np.uint32)
    rc = lib().pvt_oracle_select(_p(norms, ctypes.c_float), ctypes.c_int64(norms.size), ctypes.c_int64(k),
                                 _p(out, ctypes.c_uint32))
    if rc != 0:
        raise ValueError("pvt_oracle_select rejected its arguments")
    return out


def targets(W, g, scale, eta: float, idx, group_dim: int = 8) -> np.ndarray:
    """t = (W - eta g) / s for the groups in idx, fp32 [k, group_dim]."""
    W, g, scale = _f32(W), _f32(g), _f32(scale)
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    rows, cols = W.shape
    out = np.empty((idx.size, group_dim), dtype=np.float32)
    lib().pvt_oracle_targets(_p(W, ctypes.c_float), _p(g, ctypes.c_float), _p(scale, ctypes.c_float),
                             ctypes.c_int64(rows), ctypes.c_int64(cols), ctypes.c_int32(group_dim),
                             ctypes.c_float(eta), _p(idx, ctypes.c_uint32), ctypes.c_int64(idx.size),
                             _p(out, ctypes.c_float))
    return out


@dataclass
class EncodeResult:
    codes: np.ndarray  # int32 [k, M]
    d_best: np.ndarray  # float64 [k]
    d_second: np.ndarray  # float64 [k]
    beam_d_in: np.ndarray  # float64 [k]
    beam_d_out: np.ndarray  # float64 [k]


def encode(t, codebooks, prev, beam: int = 8) -> EncodeResult:
    """Nearest-codeword search of targets t [k, dg] against codebooks [M, K, dg]
    (any float dtype, widened exactly to fp32); prev: previous tuples [k, M]."""
    t = _f32(t)
    books = _f32(codebooks)
    M, K, dg = books.shape
    k = t.shape[0]
    prev = np.ascontiguousarray(np.asarray(prev).reshape(k, M), dtype=np.int32)
    codes = np.zeros((k, M), dtype=np.int32)
    d1 = np.zeros(k)
    d2 = np.zeros(k)
    gi = np.zeros(k)
    go = np.zeros(k)
    rc = lib().pvt_oracle_encode(_p(t, ctypes.c_float), ctypes.c_int64(k), ctypes.c_int32(dg),
                                 ctypes.c_int32(M), ctypes.c_int32(K), _p(books, ctypes.c_float),
                                 ctypes.c_int32(beam), _p(prev, ctypes.c_int32), _p(codes, ctypes.c_int32),
                                 _p(d1, ctypes.c_double), _p(d2, ctypes.c_double),
                                 _p(gi, ctypes.c_double), _p(go, ctypes.c_double))
    if rc != 0:
        raise ValueError("pvt_oracle_encode rejected its arguments")
    return EncodeResult(codes, d1, d2, gi, go)


def tuple_error(t, codebooks, codes) -> np.ndarray:
    """||t - sum_m C_m[code_m]||^2 in fp64 for given tuples [k, M]."""
    t = _f32(t)
    books = _f32(codebooks)
    M, K, dg = books.shape
    k = t.shape[0]
    codes = np.ascontiguousarray(np.asarray(codes).reshape(k, M), dtype=np.int32)
    if codes.size and (codes.min() < 0 or codes.max() >= K):
        raise ValueError("code out of range")
    out = np.zeros(k)
    lib().pvt_oracle_tuple_error(_p(t, ctypes.c_float), ctypes.c_int64(k), ctypes.c_int32(dg),
                                 ctypes.c_int32(M), ctypes.c_int32(K), _p(books, ctypes.c_float),
                                 _p(codes, ctypes.c_int32), _p(out, ctypes.c_double))
    return out


def dequant(codes, codebooks, scale, rows: int, cols: int) -> np.ndarray:
    """W_hat = s * sum_m C_m[b_m], fp32 [rows, cols]."""
    books = _f32(codebooks)
    M, K, dg = books.shape
    G = rows * (cols // dg)
    codes = np.ascontiguousarray(np.asarray(codes).reshape(G, M), dtype=np.int32)
    if codes.min() < 0 or codes.max() >= K:
        raise ValueError("code out of range")
    scale = _f32(scale)
    out = np.empty((rows, cols), dtype=np.float32)
    lib().pvt_oracle_dequant(_p(codes, ctypes.c_int32), _p(books, ctypes.c_float), _p(scale, ctypes.c_float),
                             ctypes.c_int64(rows), ctypes.c_int64(cols), ctypes.c_int32(dg),
                             ctypes.c_int32(M), ctypes.c_int32(K), _p(out, ctypes.c_float))
    return out


@dataclass
class VStepResult:
    idx: np.ndarray  # uint32 [k] ascending
    t: np.ndarray  # fp32 [k, dg]
    enc: EncodeResult
    codes: np.ndarray  # full code array after the step, same dtype/shape as the input


def vstep(W, g, scale, codebooks, codes, eta: float, k: int, beam: int = 8, idx=None) -> VStepResult:
    """One V step on one layer (Algorithm 3, V-step lines): norms -> top-k ->
    targets -> search -> write the selected codes, leave the rest."""
    dg = np.asarray(codebooks).shape[2]
    if idx is None:
        idx = select(group_norms(g, eta, dg), k)
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    t = targets(W, g, scale, eta, idx, dg)
    codes = np.asarray(codes)
    M = np.asarray(codebooks).shape[0]
    codes2 = codes.reshape(-1, M)
    enc = encode(t, codebooks, codes2[idx.astype(np.int64)], beam)
    new_codes = codes2.copy()
    new_codes[idx.astype(np.int64)] = enc.codes.astype(codes.dtype)
    return VStepResult(idx, t, enc, new_codes.reshape(codes.shape))


def pstep_grad(g, scale, codes, codebooks, rows: int, cols: int):
    """Chain rule of dequantize_weights: (grad_codebooks fp64 [M, K, dg], grad_scale fp64 [rows])."""
    g = _f32(g)
    books = _f32(codebooks)
    M, K, dg = books.shape
    G = rows * (cols // dg)
    codes = np.ascontiguousarray(np.asarray(codes).reshape(G, M), dtype=np.int32)
    if codes.min() < 0 or codes.max() >= K:
        raise ValueError("code out of range")
    scale = _f32(scale)
    gb = np.zeros((M, K, dg))
    gs = np.zeros(rows)
    lib().pvt_oracle_pstep_grad(_p(g, ctypes.c_float), _p(scale, ctypes.c_float), _p(codes, ctypes.c_int32),
                                _p(books, ctypes.c_float), ctypes.c_int64(rows), ctypes.c_int64(cols),
                                ctypes.c_int32(dg), ctypes.c_int32(M), ctypes.c_int32(K),
                                _p(gb, ctypes.c_double), _p(gs, ctypes.c_double))
    return gb, gs


def adam(param, grad, exp_avg, exp_avg_sq, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.95,
         eps: float = 1e-8):
    """One Adam update in place on fp32 arrays; returns (bias1, bias2) as used."""
    assert param.dtype == np.float32 and exp_avg.dtype == np.float32 and exp_avg_sq.dtype == np.float32
    grad = np.ascontiguousarray(grad, dtype=np.float64)
    bias1, bias2 = adam_bias(step, beta1, beta2)
    lib().pvt_oracle_adam(_p(param, ctypes.c_float), _p(grad, ctypes.c_double), _p(exp_avg, ctypes.c_float),
                          _p(exp_avg_sq, ctypes.c_float), ctypes.c_int64(param.size), ctypes.c_float(lr),
                          ctypes.c_float(beta1), ctypes.c_float(beta2), ctypes.c_float(eps),
                          ctypes.c_float(bias1), ctypes.c_float(bias2))
    return bias1, bias2


def adam_bias(step: int, beta1: float, beta2: float):
    """Bias corrections 1 - beta^t of step t >= 1: powers of the binary32 betas in binary64, rounded to binary32."""
    b1, b2 = float(np.float32(beta1)), float(np.float32(beta2))
    return float(np.float32(1.0 - b1 ** step)), float(np.float32(1.0 - b2 ** step))


def adam_direction(grad, exp_avg, exp_avg_sq, step: int, beta1: float = 0.9, beta2: float = 0.95,
                   eps: float = 1e-8) -> np.ndarray:
    """Adam-normalised update direction (fp32), moments updated in place."""
    grad = _f32(grad)
    assert exp_avg.dtype == np.float32 and exp_avg_sq.dtype == np.float32
    out = np.empty(grad.shape, dtype=np.float32)
    bias1, bias2 = adam_bias(step, beta1, beta2)
    lib().pvt_oracle_adam_direction(_p(grad, ctypes.c_float), _p(exp_avg, ctypes.c_float),
                                    _p(exp_avg_sq, ctypes.c_float), _p(out, ctypes.c_float),
                                    ctypes.c_int64(grad.size), ctypes.c_float(beta1), ctypes.c_float(beta2),
                                    ctypes.c_float(eps), ctypes.c_float(bias1), ctypes.c_float(bias2))
    return out
