"""Pure-Python brute force of the LagKV scoring and selection, for tiny inputs only.

TEST INFRASTRUCTURE ONLY.  A second, independent statement of Section 2.2 of
arXiv 2504.04704 (Eq. 7-12) on nested Python lists of floats, written without numpy
and without the C oracle, so that the two can be held against each other on inputs
small enough to check by hand (S ~ 40, D = 4).
"""
from __future__ import annotations

import math


def lagkv_cache_len(Ls: int, S: int, L: int, k: int) -> int:
    """Eq. 12 with rL = k; unchanged length when Ls < S + 2L."""
    if Ls < S + 2 * L:
        return Ls
    return S + k * ((Ls - S) // L - 1) + L + (Ls - S) % L


def _column(rows, c):
    return [row[c] for row in rows]


def _std(values, ddof):
    m = sum(values) / len(values)
    return math.sqrt(sum((v - m) ** 2 for v in values) / (len(values) - ddof))


def _softmax(values):
    top = max(values)
    e = [math.exp(v - top) for v in values]
    z = sum(e)
    return [v / z for v in e]


def tensor_score(cur, ref, ddof):
    """Eq. 7-10: normalise ``cur`` by the per-channel min/max of ``ref``; per-token std
    over channels; softmax over the tokens of the partition."""
    D = len(cur[0])
    lo = [min(_column(ref, c)) for c in range(D)]
    hi = [max(_column(ref, c)) for c in range(D)]
    sig = []
    for token in cur:
        y = [(token[c] - lo[c]) / (hi[c] - lo[c]) if hi[c] > lo[c] else 0.0 for c in range(D)]
        sig.append(_std(y, ddof))
    return _softmax(sig)


def partition_score(Kcur, Vcur, Kref, Vref, ddof=1):
    """Eq. 11."""
    return [a + b for a, b in zip(tensor_score(Kcur, Kref, ddof), tensor_score(Vcur, Vref, ddof))]


def keep_indices(score, k):
    """k largest, lower index first among equals, returned ascending."""
    order = sorted(range(len(score)), key=lambda t: (-score[t], t))
    return sorted(order[:k])


def compress_head(K, V, S, L, k, ddof=1):
    """Whole pass for one head: ``K``, ``V`` are ``[Ls][D]`` lists.  Returns the list of
    kept source rows (sink, kept rows of every partition but the last, window)."""
    Ls = len(K)
    if Ls - S < 2 * L:
        return list(range(Ls))
    n = (Ls - S) // L
    kept = list(range(S))
    for p in range(n - 1):
        a, b = S + p * L, S + (p + 1) * L
        score = partition_score(K[a:b], V[a:b], K[b:b + L], V[b:b + L], ddof)
        kept += [a + t for t in keep_indices(score, k)]
    kept += list(range(S + (n - 1) * L, Ls))
    return kept
