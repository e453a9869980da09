"""ctypes front end of the fp64 CPU oracle (``curdkv_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests, the smoke check and the
benchmark's cpu-baseline leg may import this module.  It holds no arithmetic of
its own -- every number comes from the C file, which restates Algorithm 1 and
the AdaCurDKV paragraph of Sec. 3.2 of the CurDKV paper in naive fp64 loops.

All arrays are host numpy arrays.  bf16 tensors travel as ``uint16`` bit
patterns with layout ``[B, H, n_max, d]`` (C-contiguous); G is fp32 ``[d, r]``
or ``[H, d, r]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "curdkv_oracle.c"
_LIB = _HERE / "libcurdkv_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (OpenMP across problems only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
    return _lib


def _p(a, ctype):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    lib = _load()
    lib.oracle_num_threads.restype = ctypes.c_int
    return int(lib.oracle_num_threads())


def score(K, V, G, seqlens=None, score_mode=0, use_projection=1, return_factors=False):
    """Alg. 1 (scoring steps).  Returns (scores [B,H,n] f64, head_sums [B,H] f64[, lK, lV])."""
    K = np.ascontiguousarray(K, dtype=np.uint16)
    V = np.ascontiguousarray(V, dtype=np.uint16)
    G = np.ascontiguousarray(G, dtype=np.float32)
    B, H, n, d = K.shape
    assert V.shape == K.shape
    g_per_head = int(G.ndim == 3)
    r = G.shape[-1]
    assert G.shape[-2] == d and (not g_per_head or G.shape[0] == H)
    seqlens = _i32(seqlens)
    scores = np.empty((B, H, n), dtype=np.float64)
    sums = np.empty((B, H), dtype=np.float64)
    lK = np.empty((B, H, n), dtype=np.float64) if return_factors else None
    lV = np.empty((B, H, n), dtype=np.float64) if return_factors else None
    sb, sh, sn = H * n * d, n * d, d
    i64 = ctypes.c_int64
    _load().oracle_score(
        _p(K, ctypes.c_uint16), _p(V, ctypes.c_uint16), B, H, n, d,
        i64(sb), i64(sh), i64(sn), i64(sb), i64(sh), i64(sn),
        _p(seqlens, ctypes.c_int32), _p(G, ctypes.c_float), r, g_per_head,
        int(score_mode), int(use_projection),
        _p(scores, ctypes.c_double), _p(sums, ctypes.c_double),
        _p(lK, ctypes.c_double), _p(lV, ctypes.c_double),
    )
    if return_factors:
        return scores, sums, lK, lV
    return scores, sums


def select_fixed(scores, budget, num_sink=0, window=0, seqlens=None, head_budgets=None):
    """Alg. 1 (sinks, top-k, union).  Returns (idx [B,H,budget] int32 ascending, tail -1; counts [B,H])."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    B, H, n = scores.shape
    seqlens = _i32(seqlens)
    head_budgets = _i32(head_budgets)
    idx = np.empty((B, H, max(budget, 0)), dtype=np.int32)
    counts = np.empty((B, H), dtype=np.int32)
    _load().oracle_select_fixed(
        _p(scores, ctypes.c_double), B, H, n, _p(seqlens, ctypes.c_int32), int(budget),
        _p(head_budgets, ctypes.c_int32), int(num_sink), int(window),
        _p(idx, ctypes.c_int32), _p(counts, ctypes.c_int32),
    )
    return idx, counts


def select_adaptive(scores, budget, num_sink=0, window=0, alpha=0.2, seqlens=None):
    """AdaCurDKV.  Returns (idx packed [total] int32, counts [B,H], offsets [B*H+1])."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    B, H, n = scores.shape
    seqlens = _i32(seqlens)
    idx = np.full((B * H * max(min(budget, n), 1),), -1, dtype=np.int32)
    counts = np.empty((B, H), dtype=np.int32)
    offsets = np.empty((B * H + 1,), dtype=np.int32)
    _load().oracle_select_adaptive(
        _p(scores, ctypes.c_double), B, H, n, _p(seqlens, ctypes.c_int32), int(budget),
        int(num_sink), int(window), ctypes.c_double(alpha),
        _p(idx, ctypes.c_int32), _p(counts, ctypes.c_int32), _p(offsets, ctypes.c_int32),
    )
    return idx[: offsets[-1]].copy(), counts, offsets


def compact(K, V, idx, counts, offsets=None):
    """Alg. 1 (gather step).  Fixed layout (idx [B,H,budget]) -> [B,H,budget,d] (unused rows 0);
    packed layout (idx [total] with offsets) -> [total, d]."""
    K = np.ascontiguousarray(K, dtype=np.uint16)
    V = np.ascontiguousarray(V, dtype=np.uint16)
    B, H, n, d = K.shape
    idx = _i32(idx)
    counts = _i32(counts)
    sb, sh, sn = H * n * d, n * d, d
    i64 = ctypes.c_int64
    if offsets is None:
        budget = idx.shape[-1]
        Ko = np.zeros((B, H, budget, d), dtype=np.uint16)
        Vo = np.zeros((B, H, budget, d), dtype=np.uint16)
        out_stride_h, idx_stride = budget, budget
    else:
        offsets = _i32(offsets)
        total = int(offsets[-1])
        Ko = np.zeros((total, d), dtype=np.uint16)
        Vo = np.zeros((total, d), dtype=np.uint16)
        out_stride_h, idx_stride = 0, 0
    _load().oracle_compact(
        _p(K, ctypes.c_uint16), _p(V, ctypes.c_uint16), B, H, d,
        i64(sb), i64(sh), i64(sn), i64(sb), i64(sh), i64(sn),
        _p(idx, ctypes.c_int32), i64(idx_stride), _p(counts, ctypes.c_int32),
        _p(offsets, ctypes.c_int32), _p(Ko, ctypes.c_uint16), _p(Vo, ctypes.c_uint16),
        i64(out_stride_h),
    )
    return Ko, Vo


def kv_head_of_query(q_head: int, q_heads: int, kv_heads: int) -> int:
    lib = _load()
    lib.oracle_kv_head_of_query.restype = ctypes.c_int
    return int(lib.oracle_kv_head_of_query(int(q_head), int(q_heads), int(kv_heads)))
