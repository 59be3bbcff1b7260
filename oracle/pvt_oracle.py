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
        L.pvt_oracle_rank.restype = ctypes.c_int
        L.pvt_oracle_local_search.restype = ctypes.c_int
        L.pvt_oracle_sample_keys.restype = ctypes.c_int
        L.pvt_oracle_neglog_u32.restype = ctypes.c_double
        L.pvt_oracle_neglog_u32.argtypes = [ctypes.c_uint32]
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


def rank(norms, k: int) -> np.ndarray:
    """The k groups of largest norm in the order (norm descending, index ascending), uint32 [k]."""
    norms = _f32(norms)
    out = np.empty(k, dtype=np.uint32)
    rc = lib().pvt_oracle_rank(_p(norms, ctypes.c_float), ctypes.c_int64(norms.size), ctypes.c_int64(k),
                               _p(out, ctypes.c_uint32))
    if rc != 0:
        raise ValueError("pvt_oracle_rank rejected its arguments")
    return out


def group_change(codes_old, codes_new, codebooks, scale, cols: int, idx):
    """Per listed group: squared change of its dequantised weights, and their squared norm before (float64 [k] each)."""
    books = _f32(codebooks)
    M, K, dg = books.shape
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    k = idx.size
    co = np.ascontiguousarray(np.asarray(codes_old).reshape(k, M), dtype=np.int32)
    cn = np.ascontiguousarray(np.asarray(codes_new).reshape(k, M), dtype=np.int32)
    for c in (co, cn):
        if k and (c.min() < 0 or c.max() >= K):
            raise ValueError("code out of range")
    scale = _f32(scale)
    change = np.empty(k, dtype=np.float64)
    own = np.empty(k, dtype=np.float64)
    lib().pvt_oracle_group_change(_p(co, ctypes.c_int32), _p(cn, ctypes.c_int32), _p(books, ctypes.c_float),
                                  _p(scale, ctypes.c_float), ctypes.c_int64(cols), ctypes.c_int32(dg),
                                  ctypes.c_int32(M), ctypes.c_int32(K), _p(idx, ctypes.c_uint32), ctypes.c_int64(k),
                                  _p(change, ctypes.c_double), _p(own, ctypes.c_double))
    return change, own


@dataclass
class TrustResult:
    order: np.ndarray  # uint32 [tried]: the groups that were re-encoded, in the order they were taken
    n_kept: int  # how many of them (a prefix of ``order``) keep their new code
    codes: np.ndarray  # full code array after the step
    change: np.ndarray  # float64 [tried]: squared change of each tried group's dequantised weights
    sq_norm: float  # ||x_old||^2 of the whole matrix
    enc_codes: np.ndarray  # int32 [tried, M]: what the search returned for each tried group
    gap_rel: np.ndarray  # float64 [tried]: (second - best) / second of each search (near-tie indicator)


def vstep_trust(W, g, scale, codebooks, codes, eta: float, ratio: float = 0.01, portion: float = 0.01,
                k_max: int | None = None, beam: int = 8) -> TrustResult:
    """V step whose subspace size comes from the trust ratio (Section 4.3, Appendix J).

    Groups are taken in the order of decreasing update norm, ``portion`` of all groups at a time, and
    re-encoded; after each portion the total squared change of the dequantised matrix is compared with
    ``ratio**2 * ||x_old||**2`` (the bound ``||x_new - x_old|| / ||x_old|| < ratio`` without the division and
    the roots, in float64).  Once the bound fails, codes are put back one group at a time from the end of the
    last portion until it holds; at least one group keeps its new code.  ``k_max`` stops the procedure after
    that many groups (default: all of them).
    """
    books = _f32(codebooks)
    M, K, dg = books.shape
    W = _f32(W)
    rows, cols = W.shape
    G = rows * (cols // dg)
    k_max = G if k_max is None else int(k_max)
    codes = np.asarray(codes)
    codes2 = codes.reshape(G, M)
    order = rank(group_norms(g, eta, dg), k_max)
    x_old = dequant(codes2, books, scale, rows, cols)
    sq_norm = float(np.cumsum(x_old.astype(np.float64).ravel() ** 2)[-1]) if G else 0.0
    limit = float(np.float64(np.float32(ratio)) * np.float64(np.float32(ratio))) * sq_norm
    step = max(1, int(portion * G))
    new_codes = codes2.copy()
    changes, enc_all, gaps = [], [], []
    total = 0.0
    n_kept = 0
    tried = 0
    while tried < k_max:
        part = order[tried:min(tried + step, k_max)]
        j = part.astype(np.int64)
        enc = encode(targets(W, g, scale, eta, part, dg), books, codes2[j], beam)
        ch, _ = group_change(codes2[j], enc.codes, books, scale, cols, part)
        new_codes[j] = enc.codes.astype(codes.dtype)
        enc_all.append(enc.codes.reshape(-1, M))
        gaps.append(np.where(enc.d_second > 0, (enc.d_second - enc.d_best) / np.where(enc.d_second > 0, enc.d_second, 1.0), 0.0))
        running = total + np.cumsum(ch)  # total change after each group of this portion, in order
        changes.append(ch)
        tried += part.size
        if running[-1] < limit:
            total = float(running[-1])
            n_kept = tried
            continue
        # the bound fails inside this portion: undo its groups from the end until it holds again
        keep = part.size
        while keep > 0 and not (running[keep - 1] < limit):
            keep -= 1
        n_kept = tried - part.size + keep
        break
    n_kept = max(n_kept, 1)  # one change is always let through
    undo = order[n_kept:tried].astype(np.int64)
    new_codes[undo] = codes2[undo]
    return TrustResult(order[:tried], n_kept, new_codes.reshape(codes.shape), np.concatenate(changes), sq_norm,
                       np.concatenate(enc_all), np.concatenate(gaps))


def local_search(t, codebooks, codes, max_moves: int = 64):
    """Local search over single-code changes (Appendix D) from the given code tuples: returns
    (codes int32 [k, M], error float64 [k], moves int32 [k])."""
    books = _f32(codebooks)
    M, K, dg = books.shape
    t = _f32(t).reshape(-1, dg)
    k = t.shape[0]
    out = np.ascontiguousarray(np.asarray(codes).reshape(k, M), dtype=np.int32).copy()
    d = np.empty(k, dtype=np.float64)
    moves = np.empty(k, dtype=np.int32)
    rc = lib().pvt_oracle_local_search(_p(t, ctypes.c_float), ctypes.c_int64(k), ctypes.c_int32(dg),
                                       ctypes.c_int32(M), ctypes.c_int32(K), _p(books, ctypes.c_float),
                                       _p(out, ctypes.c_int32), ctypes.c_int32(max_moves), _p(d, ctypes.c_double),
                                       _p(moves, ctypes.c_int32))
    if rc != 0:
        raise ValueError("pvt_oracle_local_search rejected its arguments")
    return out, d, moves


SAMPLE_UNIFORM, SAMPLE_PROPORTIONAL = 0, 1


def ste_accumulate(buffer, g, eta: float) -> np.ndarray:
    """Straight-through buffer after one step: fmaf(-eta, g, buffer) per weight (Appendix E); returns a new array."""
    out = np.ascontiguousarray(buffer, dtype=np.float32).copy()
    g = _f32(g)
    assert out.shape == g.shape
    lib().pvt_oracle_ste_accumulate(_p(out, ctypes.c_float), _p(g, ctypes.c_float), ctypes.c_int64(out.size),
                                    ctypes.c_float(eta))
    return out


def philox4x32_10(ctr, key) -> np.ndarray:
    """One block of the Philox-4x32-10 generator: four 32-bit words."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    assert c.size == 4 and k.size == 2
    out = np.zeros(4, dtype=np.uint32)
    lib().pvt_oracle_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32), _p(out, ctypes.c_uint32))
    return out


def neglog_u32(r: int) -> float:
    """-ln((r + 1/2) 2^-32) by the sampler's fixed binary64 sequence."""
    return float(lib().pvt_oracle_neglog_u32(ctypes.c_uint32(r)))


def sample_keys(num_groups: int, mode: int, seed: int, norms=None) -> np.ndarray:
    """Sampling keys (binary32, >= 0) of every group for the random subspace rules."""
    keys = np.empty(num_groups, dtype=np.float32)
    nptr = None
    if norms is not None:
        norms = _f32(norms)
        assert norms.size == num_groups
        nptr = _p(norms, ctypes.c_float)
    rc = lib().pvt_oracle_sample_keys(nptr, ctypes.c_int64(num_groups), ctypes.c_int32(mode), ctypes.c_uint64(seed),
                                      _p(keys, ctypes.c_float))
    if rc != 0:
        raise ValueError("pvt_oracle_sample_keys rejected its arguments")
    return keys


def sample_subspace(num_groups: int, k: int, mode: int, seed: int, norms=None) -> np.ndarray:
    """A random subspace of k groups (uniform, or in proportion to the squared update norms), ascending uint32 [k]."""
    return select(sample_keys(num_groups, mode, seed, norms), k)


def vstep_ste(buffer, g, scale, codebooks, codes, eta: float, k: int, beam: int = 8):
    """Subspace V step combined with a straight-through buffer: the buffer takes the whole step, the subspace is
    chosen by the size of this step's update, the chosen groups are re-encoded against the buffer.  Returns
    (new buffer, VStepResult)."""
    dg = np.asarray(codebooks).shape[2]
    new_buffer = ste_accumulate(buffer, g, eta)
    idx = select(group_norms(g, eta, dg), k)
    return new_buffer, vstep(new_buffer, g, scale, codebooks, codes, 0.0, k, beam, idx=idx)
