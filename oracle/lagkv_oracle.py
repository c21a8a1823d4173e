"""ctypes front end of the float64 CPU oracle (``lagkv_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  Nothing here is part of the CUDA library, and the CUDA
library imports nothing from here.

All arrays are numpy; K and V are 16-bit patterns (bf16 by default, fp16 with
``storage=STORAGE_FP16``) held as ``uint16`` with shape
``[B, H, seq_len, D]`` (C-contiguous).  The arithmetic lives in the C file; this
module only compiles it (gcc, on first use), marshals arguments and implements the
append bookkeeping of Section 2.2 (bullets 2-4) on top of ``compress``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "lagkv_oracle.c"
_LIB = _HERE / "liblagkv_oracle.so"

VARIANT_LAGKV, VARIANT_LOCALKV, VARIANT_L2NORM = 0, 1, 2
STORAGE_BF16, STORAGE_FP16, STORAGE_FP8_E4M3 = 0, 1, 2

_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle into a shared object next to its source."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(str(build()))
    i64, dbl, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_int
    vp = ctypes.c_void_p
    lib.lagkv_oracle_num_threads.restype = ci
    lib.lagkv_oracle_set_threads.argtypes = [ci]
    lib.lagkv_oracle_keep_count.restype = i64
    lib.lagkv_oracle_keep_count.argtypes = [dbl, i64]
    lib.lagkv_oracle_compressed_len.restype = i64
    lib.lagkv_oracle_compressed_len.argtypes = [i64, i64, i64, i64]
    lib.lagkv_oracle_partition_scores.restype = None
    lib.lagkv_oracle_partition_scores.argtypes = [vp, vp, vp, vp, i64, i64, i64, ci, ci, ci, vp, vp, vp]
    lib.lagkv_oracle_topk.restype = None
    lib.lagkv_oracle_topk.argtypes = [vp, i64, i64, vp]
    lib.lagkv_oracle_compress.restype = i64
    lib.lagkv_oracle_compress.argtypes = [vp, vp, i64, i64, i64, i64, i64, i64, i64, ci, ci, ci, vp, vp, vp, vp]
    lib.lagkv_oracle_decode.restype = None
    lib.lagkv_oracle_decode.argtypes = [vp, i64, ci, vp]
    lib.lagkv_oracle_gather.restype = None
    lib.lagkv_oracle_gather.argtypes = [vp, i64, i64, i64, vp, i64, vp]
    _lib = lib
    return lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    """Bit patterns as the C side takes them: uint16 per element.  fp8 bytes (uint8) are
    zero-extended: a change of container, not of value."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint8:
        return a.astype(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("K/V must be bit patterns: uint16 (bf16, fp16) or uint8 (fp8 e4m3)")
    return a


def num_threads() -> int:
    return int(_load().lagkv_oracle_num_threads())


def set_threads(n: int) -> None:
    _load().lagkv_oracle_set_threads(int(n))


def keep_count(r: float, L: int) -> int:
    """k = ceil(r*L) clamped to [1, L] (text before Eq. 12)."""
    return int(_load().lagkv_oracle_keep_count(float(r), int(L)))


def compressed_len(seq_len: int, static_len: int, L: int, k: int) -> int:
    """Eq. 12 with the skip rule of Section 2.2 (rest < 2L leaves the cache alone)."""
    return int(_load().lagkv_oracle_compressed_len(int(seq_len), int(static_len), int(L), int(k)))


def decode(bits, storage: int = STORAGE_BF16) -> np.ndarray:
    """The float64 value of every 16-bit pattern, as the oracle reads it."""
    bits = _u16(bits)
    out = np.zeros(bits.shape, np.float64)
    _load().lagkv_oracle_decode(_ptr(bits), bits.size, int(storage), _ptr(out))
    return out


def partition_scores(Kcur, Vcur, Kref, Vref, ddof: int = 1, variant: int = VARIANT_LAGKV,
                     storage: int = STORAGE_BF16):
    """Eq. 7-11 for one partition.  Inputs ``[L, D]`` uint16.  Returns (score, sK, sV)."""
    Kcur, Vcur, Kref, Vref = map(_u16, (Kcur, Vcur, Kref, Vref))
    L, D = Kcur.shape
    score, sK, sV = (np.zeros(L, np.float64) for _ in range(3))
    _load().lagkv_oracle_partition_scores(
        _ptr(Kcur), _ptr(Vcur), _ptr(Kref), _ptr(Vref), L, D, D, int(ddof), int(variant), int(storage),
        _ptr(score), _ptr(sK), _ptr(sV))
    return score, sK, sV


def topk(score, k: int) -> np.ndarray:
    """Indices of the k largest scores, ties to the lower index, ascending order."""
    score = np.ascontiguousarray(score, dtype=np.float64)
    out = np.zeros(int(k), np.int32)
    _load().lagkv_oracle_topk(_ptr(score), score.shape[0], int(k), _ptr(out))
    return out


def compress(K, V, static_len: int, L: int, k: int, ddof: int = 1,
             variant: int = VARIANT_LAGKV, want_rows: bool = True, want_scores: bool = True,
             storage: int = STORAGE_BF16):
    """One compress pass (Section 2.2) over ``[B, H, seq_len, D]`` caches.

    Returns a dict with ``L_R``, ``idx`` ``[B,H,L_R]`` int32, and optionally ``K_out`` /
    ``V_out`` ``[B,H,L_R,D]`` uint16 and ``scores`` ``[B,H,n_c,L]`` float64.
    """
    K, V = _u16(K), _u16(V)
    B, H, S, D = K.shape
    assert V.shape == K.shape
    L_R = compressed_len(S, static_len, L, k)
    rest = S - static_len
    n_c = rest // L - 1 if rest >= 2 * L else 0
    idx = np.zeros((B, H, L_R), np.int32)
    K_out = np.zeros((B, H, L_R, D), np.uint16) if want_rows else None
    V_out = np.zeros((B, H, L_R, D), np.uint16) if want_rows else None
    scores = np.zeros((B, H, n_c, L), np.float64) if want_scores else None
    got = _load().lagkv_oracle_compress(
        _ptr(K), _ptr(V), B, H, S, D, int(static_len), int(L), int(k), int(ddof), int(variant),
        int(storage), _ptr(idx), _ptr(K_out), _ptr(V_out), _ptr(scores))
    assert got == L_R
    if storage == STORAGE_FP8_E4M3 and want_rows:     # back to bytes
        K_out, V_out = K_out.astype(np.uint8), V_out.astype(np.uint8)
    return {"L_R": L_R, "n_c": n_c, "idx": idx, "K_out": K_out, "V_out": V_out, "scores": scores}


def gather(X, idx) -> np.ndarray:
    """out[b,h,j,:] = X[b,h,idx[b,h,j],:]."""
    X = _u16(X)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    B, H, S, D = X.shape
    n_idx = idx.shape[-1]
    out = np.zeros((B, H, n_idx, D), np.uint16)
    _load().lagkv_oracle_gather(_ptr(X), B * H, S, D, _ptr(idx), n_idx, _ptr(out))
    return out


def compress_append(K_cache, V_cache, seq_len, static_len, L: int, k: int, ddof: int = 1,
                    variant: int = VARIANT_LAGKV, storage: int = STORAGE_BF16):
    """Incremental pass on a ``[B, H, S_cap, D]`` cache with per-sequence lengths.

    For every sequence b the rows ``[0, static_len[b])`` are the sink plus everything
    kept by earlier passes; if the rows after them number at least 2L the pass of
    ``compress`` runs on ``[0, seq_len[b])`` and the cache is rewritten in place
    (Section 2.2, bullets 2-4).  Returns new ``(K, V, seq_len, static_len, kept)`` where
    ``kept[b]`` is ``[H, n_c*k]`` int32 positions (pre-call) of the newly kept rows, or an
    empty array when the sequence was skipped.
    """
    K_cache, V_cache = np.array(K_cache, copy=True), np.array(V_cache, copy=True)
    B = K_cache.shape[0]
    seq_len = np.array(seq_len, dtype=np.int64).copy()
    static_len = np.array(static_len, dtype=np.int64).copy()
    kept = []
    for b in range(B):
        s, st = int(seq_len[b]), int(static_len[b])
        if s - st < 2 * L:
            kept.append(np.zeros((K_cache.shape[1], 0), np.int32))
            continue
        res = compress(K_cache[b:b + 1, :, :s], V_cache[b:b + 1, :, :s], st, L, k, ddof, variant,
                       want_scores=False, storage=storage)
        L_R, n_c = res["L_R"], res["n_c"]
        K_cache[b, :, :L_R] = res["K_out"][0]
        V_cache[b, :, :L_R] = res["V_out"][0]
        kept.append(res["idx"][0, :, st:st + n_c * k].copy())
        static_len[b] = st + n_c * k
        seq_len[b] = L_R
    return K_cache, V_cache, seq_len, static_len, kept
