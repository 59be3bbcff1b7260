"""Test-side helpers: an independent brute-force enumerator (numpy, fp64), an
exact binary32 rounding routine, golden-file reader and the acceptance rule
that compares a code assignment with the CPU checker's result."""
from __future__ import annotations

import itertools
import os
from fractions import Fraction

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":")
            out[key.strip()] = np.array([float(v) for v in vals.split()])
    return out


def round_to_f32(x: Fraction) -> np.float32:
    """Round an exact rational to the nearest binary32 (ties to even)."""
    if x == 0:
        return np.float32(0.0)
    sign = -1 if x < 0 else 1
    x = abs(x)
    e = 0
    while x >= 2:
        x /= 2
        e += 1
    while x < 1:
        x *= 2
        e -= 1
    if e < -126:  # subnormal: fixed quantum 2^-149
        x = x * Fraction(2) ** (e + 126)
        e = -126
    scaled = x * (1 << 23)
    q = scaled.numerator // scaled.denominator
    rem = scaled - q
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and q % 2 == 1):
        q += 1
    val = Fraction(q, 1 << 23) * (Fraction(2) ** e)
    return np.float32(sign * float(val))


def exact_group_norm(g_group, eta):
    """The fp32 norm sequence of the V step evaluated with exact rationals and
    one rounding per stated operation: u = fl(eta*g); acc = fl(u*u + acc)."""
    acc = Fraction(0)
    eta = Fraction(float(np.float32(eta)))
    for v in g_group:
        u = Fraction(float(round_to_f32(eta * Fraction(float(np.float32(v))))))
        acc = Fraction(float(round_to_f32(u * u + acc)))
    return np.float32(float(acc))


def exact_target(w, g, eta, s):
    """fl(fl(w - eta*g) / s) with exact rationals."""
    w, g, eta, s = (Fraction(float(np.float32(v))) for v in (w, g, eta, s))
    num = Fraction(float(round_to_f32(w - eta * g)))
    return round_to_f32(num / s)


def brute_force_tuples(t, codebooks):
    """Enumerate every code tuple: returns (best tuples [k, M], best distance
    [k]) under (distance, tuple) lexicographic order, in fp64."""
    t = np.asarray(t, dtype=np.float64)
    books = np.asarray(codebooks, dtype=np.float64)
    M, K, dg = books.shape
    tuples = list(itertools.product(range(K), repeat=M))  # lexicographic order
    recon = np.zeros((len(tuples), dg))
    for n, tup in enumerate(tuples):
        for m, c in enumerate(tup):
            recon[n] += books[m, c]
    best = np.zeros((t.shape[0], M), dtype=np.int64)
    dist = np.zeros(t.shape[0])
    for n in range(t.shape[0]):
        d = ((t[n][None, :] - recon) ** 2).sum(axis=1)
        a = int(np.argmin(d))  # first minimum = lexicographically smallest tuple
        best[n] = tuples[a]
        dist[n] = d[a]
    return best, dist


def recon_error(t, codebooks, codes):
    """||t - sum_m C_m[code_m]||^2 in fp64, independent of the checker."""
    t = np.asarray(t, dtype=np.float64)
    books = np.asarray(codebooks, dtype=np.float64)
    codes = np.asarray(codes, dtype=np.int64).reshape(t.shape[0], books.shape[0])
    recon = np.zeros_like(t)
    for m in range(books.shape[0]):
        recon += books[m, codes[:, m]]
    return ((t - recon) ** 2).sum(axis=1)


def check_codes_against_oracle(t, codebooks, got_codes, enc, rel=1e-6):
    """Acceptance rule: where the checker's best-vs-second gap exceeds `rel`
    (relative to the second distance) the code tuple must be identical;
    elsewhere the reconstruction error must agree within `rel` relative.
    Returns (number of exact matches, number accepted inside the gap band)."""
    got = np.asarray(got_codes, dtype=np.int64).reshape(enc.codes.shape)
    same = (got == enc.codes).all(axis=1)
    decisive = (enc.d_second - enc.d_best) > rel * enc.d_second
    wrong = decisive & ~same
    assert not wrong.any(), f"{int(wrong.sum())} code tuples differ outside the gap band, first at {np.flatnonzero(wrong)[:5]}"
    band = ~same
    if band.any():
        K = np.asarray(codebooks).shape[1]
        assert got[band].min() >= 0 and got[band].max() < K
        d_got = recon_error(np.asarray(t)[band], codebooks, got[band])
        d_ref = enc.d_best[band]
        ok = np.abs(d_got - d_ref) <= rel * np.maximum(d_got, d_ref)
        assert ok.all(), "reconstruction error differs by more than the relative tolerance inside the gap band"
    return int(same.sum()), int(band.sum())


def stagewise_beam(t, codebooks, beam, prev=None):
    """Greedy residual beam search written stage by stage on whole arrays (numpy, fp64), with no call
    into the CPU checker: after stage m the `beam` partial tuples with the smallest
    ||t - c^1 - ... - c^m||^2 are kept, ties resolved towards the lexicographically smaller tuple; the
    last stage's extensions (plus `prev`, if given) form the pool, whose smallest member under
    (distance, tuple) is returned.  The residual is carried codebook by codebook and the squared
    distance summed element by element, so that equal operands give the checker's binary64 values.
    Returns (tuples int64 [k, M], distances float64 [k])."""
    t = np.asarray(t, dtype=np.float32).astype(np.float64)
    books = np.asarray(codebooks).astype(np.float32).astype(np.float64)
    M, K, dg = books.shape
    out_codes = np.zeros((t.shape[0], M), dtype=np.int64)
    out_dist = np.zeros(t.shape[0])
    for n in range(t.shape[0]):
        partial = [((), t[n].copy())]  # (tuple so far, residual)
        scored = []
        for m in range(M):
            scored = []
            for tup, res in partial:
                diff = res[None, :] - books[m]
                d = np.zeros(K)
                for i in range(dg):  # element order, one rounding per addition
                    d = d + diff[:, i] * diff[:, i]
                for q in range(K):
                    scored.append((float(d[q]), tup + (q,)))
            if m == M - 1:
                break
            scored.sort()  # python tuples compare as (distance, then code tuple) -- the stated order
            partial = []
            for d_, tup in scored[:beam]:
                res = t[n].copy()
                for mm, q in enumerate(tup):
                    res = res - books[mm, q]
                partial.append((tup, res))
        if prev is not None:
            p = tuple(int(x) for x in np.asarray(prev)[n])
            if p not in {tup for _, tup in scored}:
                res = t[n].copy()
                for mm in range(M - 1):
                    res = res - books[mm, p[mm]]
                diff = res - books[M - 1, p[M - 1]]
                d = 0.0
                for i in range(dg):
                    d = d + diff[i] * diff[i]
                scored.append((float(d), p))
        best = min(scored)
        out_codes[n] = best[1]
        out_dist[n] = best[0]
    return out_codes, out_dist
