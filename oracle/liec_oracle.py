"""ctypes front end of ``liec_oracle.c`` (test infrastructure, see that file's header).

Argument marshalling only: every number is computed by the C file.  The shared
object is compiled with gcc on first use (``-O2 -ffp-contract=off``, no fast-math)
into ``oracle/_build/``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

IDENTITY, SIGN, TOPK, RANDK = 0, 1, 2, 3

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "liec_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_OUT = os.path.join(_OUT_DIR, "libliec_oracle.so")
_LIB: Optional[C.CDLL] = None

CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
          "-Wall", "-Wextra"]


def build(force: bool = False, extra_flags=(), out: Optional[str] = None) -> str:
    """Compile the oracle; returns the path of the shared object."""
    target = out or _OUT
    os.makedirs(os.path.dirname(target), exist_ok=True)
    stale = (not os.path.exists(target)) or os.path.getmtime(target) < os.path.getmtime(_SRC)
    if force or stale or extra_flags:
        tmp = target + f".tmp{os.getpid()}"
        subprocess.run(["gcc", *CFLAGS, *extra_flags, _SRC, "-o", tmp], check=True)
        os.replace(tmp, target)
    return target


def _bind(lib: C.CDLL) -> C.CDLL:
    p = C.c_void_p
    lib.liec_oracle_widen_bf16.argtypes = [p, p, C.c_int64]
    lib.liec_oracle_widen_bf16.restype = None
    lib.liec_oracle_tree_abs_sum.argtypes = [p, C.c_int64]
    lib.liec_oracle_tree_abs_sum.restype = C.c_double
    lib.liec_oracle_tree_sumsq.argtypes = [p, C.c_int64]
    lib.liec_oracle_tree_sumsq.restype = C.c_double
    lib.liec_oracle_scale.argtypes = [p, C.c_int64]
    lib.liec_oracle_scale.restype = C.c_float
    lib.liec_oracle_sign.argtypes = [p, C.c_int32, p, p, p, p]
    lib.liec_oracle_sign.restype = None
    lib.liec_oracle_topk.argtypes = [p, C.c_int32, p, p, p, p, p]
    lib.liec_oracle_topk.restype = C.c_int
    lib.liec_oracle_randk.argtypes = [p, C.c_int32, p, p, p, p, p, p]
    lib.liec_oracle_randk.restype = C.c_int
    lib.liec_oracle_step_sets.argtypes = [C.c_int32, C.c_int64, C.c_int32, p, C.c_int32, C.c_int32, p, p, p,
                                          p, C.c_float, p, p] + [p] * 9
    lib.liec_oracle_step_sets.restype = C.c_int
    lib.liec_oracle_step.argtypes = [C.c_int32, C.c_int64, C.c_int32, p, C.c_int32, C.c_int32, p,
                                     p, C.c_float, p, p] + [p] * 9
    lib.liec_oracle_step.restype = C.c_int
    lib.liec_oracle_philox4x32_10.argtypes = [p, p, p]
    lib.liec_oracle_philox4x32_10.restype = None
    lib.liec_oracle_subset_scores.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_int64, p]
    lib.liec_oracle_subset_scores.restype = None
    lib.liec_oracle_subset_from_scores.argtypes = [p, C.c_int64, C.c_int64, p]
    lib.liec_oracle_subset_from_scores.restype = C.c_int
    lib.liec_oracle_draw_subsets.argtypes = [C.c_uint64, C.c_uint32, C.c_int32, C.c_int32, p, p, p]
    lib.liec_oracle_draw_subsets.restype = C.c_int
    lib.liec_oracle_mean_params.argtypes = [C.c_int32, C.c_int64, p, p]
    lib.liec_oracle_mean_params.restype = None
    lib.liec_oracle_average_step.argtypes = [C.c_int32, C.c_int64, p, C.c_float, p, p, p, p]
    lib.liec_oracle_average_step.restype = C.c_int
    return lib


def lib(path: Optional[str] = None) -> C.CDLL:
    global _LIB
    if path is not None:
        return _bind(C.CDLL(path))
    if _LIB is None:
        _LIB = _bind(C.CDLL(build()))
    return _LIB


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _off(off) -> np.ndarray:
    return np.ascontiguousarray(off, dtype=np.int64)


def num_words(off) -> int:
    off = _off(off)
    return int(((np.diff(off) + 31) // 32).sum())


def widen_bf16(bits_u16: np.ndarray, _lib=None) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32, exactly."""
    a = np.ascontiguousarray(bits_u16, dtype=np.uint16)
    out = np.empty(a.shape, dtype=np.float32)
    (_lib or lib()).liec_oracle_widen_bf16(_ptr(a), _ptr(out), a.size)
    return out


def tree_abs_sum(x, _lib=None) -> float:
    x = _f32(x)
    return float((_lib or lib()).liec_oracle_tree_abs_sum(_ptr(x), x.size))


def tree_sumsq(x, _lib=None) -> float:
    """||x||_2^2 in binary64 (balanced tree)."""
    x = _f32(x)
    return float((_lib or lib()).liec_oracle_tree_sumsq(_ptr(x), x.size))


def scale(x, _lib=None) -> np.float32:
    x = _f32(x)
    return np.float32((_lib or lib()).liec_oracle_scale(_ptr(x), x.size))


def sign_compress(x, off, _lib=None):
    """(words, scales, decoded) of the segment-wise scaled sign of x (Def. 4 / Def. 5)."""
    x, off = _f32(x), _off(off)
    T = off.size - 1
    words = np.empty(num_words(off), dtype=np.uint32)
    scales = np.empty(T, dtype=np.float32)
    dec = np.empty_like(x)
    (_lib or lib()).liec_oracle_sign(_ptr(x), T, _ptr(off), _ptr(words), _ptr(scales), _ptr(dec))
    return words, scales, dec


def topk_compress(x, off, k, _lib=None):
    """(idx, val, decoded) of the segment-wise top-k of x (Def. 2)."""
    x, off = _f32(x), _off(off)
    k = np.ascontiguousarray(k, dtype=np.int64)
    T = off.size - 1
    K = int(k.sum())
    idx = np.empty(K, dtype=np.uint32)
    val = np.empty(K, dtype=np.float32)
    dec = np.empty_like(x)
    rc = (_lib or lib()).liec_oracle_topk(_ptr(x), T, _ptr(off), _ptr(k), _ptr(idx), _ptr(val), _ptr(dec))
    if rc:
        raise MemoryError("oracle top-k out of memory")
    return idx, val, dec


def randk_compress(x, off, k, subset, _lib=None):
    """(idx, val, decoded) of the segment-wise random-k of x (Def. 3) for the given subset:
    flat indices, k_t per segment, ascending inside each segment."""
    x, off = _f32(x), _off(off)
    k = np.ascontiguousarray(k, dtype=np.int64)
    subset = np.ascontiguousarray(subset, dtype=np.uint32)
    T = off.size - 1
    K = int(k.sum())
    assert subset.shape == (K,)
    idx = np.empty(K, dtype=np.uint32)
    val = np.empty(K, dtype=np.float32)
    dec = np.empty_like(x)
    rc = (_lib or lib()).liec_oracle_randk(_ptr(x), T, _ptr(off), _ptr(k), _ptr(subset), _ptr(idx), _ptr(val), _ptr(dec))
    if rc:
        raise ValueError(f"oracle random-k rejected the subset (code {rc})")
    return idx, val, dec


@dataclass
class StepResult:
    up_words: Optional[np.ndarray]
    up_scales: Optional[np.ndarray]
    up_idx: Optional[np.ndarray]
    up_val: Optional[np.ndarray]
    down_words: Optional[np.ndarray]
    down_scales: Optional[np.ndarray]
    down_idx: Optional[np.ndarray]
    down_val: Optional[np.ndarray]
    v: np.ndarray


def step(X: np.ndarray, e: np.ndarray, G: np.ndarray, lr: float, off, up: int, down: int,
         k=None, _lib=None, up_sets=None, down_set=None) -> StepResult:
    """One compressed iteration; X [N,d] and e [d] (float32, contiguous) are updated in place.

    G is [N,d] float32 (widen bf16 with ``widen_bf16`` first).  A random-k side takes its
    subsets from ``up_sets`` [N,K] / ``down_set`` [K] (uint32 flat indices, ascending inside each
    segment).  Returns the messages and v.
    """
    assert X.dtype == np.float32 and X.flags.c_contiguous and X.ndim == 2
    assert e.dtype == np.float32 and e.flags.c_contiguous
    G = _f32(G)
    off = _off(off)
    N, d = X.shape
    assert G.shape == (N, d) and e.shape == (d,) and off[0] == 0 and off[-1] == d
    T = off.size - 1
    W = num_words(off)
    karr = None
    K = 0
    sparse = (TOPK, RANDK)
    if up in sparse or down in sparse:
        karr = np.ascontiguousarray(k, dtype=np.int64)
        assert karr.shape == (T,)
        K = int(karr.sum())
    r = StepResult(
        up_words=np.zeros((N, W), np.uint32) if up == SIGN else None,
        up_scales=np.zeros((N, T), np.float32) if up == SIGN else None,
        up_idx=np.zeros((N, K), np.uint32) if up in sparse else None,
        up_val=np.zeros((N, K), np.float32) if up in sparse else None,
        down_words=np.zeros(W, np.uint32) if down == SIGN else None,
        down_scales=np.zeros(T, np.float32) if down == SIGN else None,
        down_idx=np.zeros(K, np.uint32) if down in sparse else None,
        down_val=np.zeros(K, np.float32) if down in sparse else None,
        v=np.zeros(d, np.float32),
    )
    if up == RANDK:
        up_sets = np.ascontiguousarray(up_sets, dtype=np.uint32)
        assert up_sets.shape == (N, K)
    else:
        up_sets = None
    if down == RANDK:
        down_set = np.ascontiguousarray(down_set, dtype=np.uint32)
        assert down_set.shape == (K,)
    else:
        down_set = None
    rc = (_lib or lib()).liec_oracle_step_sets(
        N, d, T, _ptr(off), up, down, _ptr(karr), _ptr(up_sets), _ptr(down_set), _ptr(G), C.c_float(lr), _ptr(X), _ptr(e),
        _ptr(r.up_words), _ptr(r.up_scales), _ptr(r.up_idx), _ptr(r.up_val),
        _ptr(r.down_words), _ptr(r.down_scales), _ptr(r.down_idx), _ptr(r.down_val), _ptr(r.v))
    if rc:
        raise RuntimeError(f"liec_oracle_step failed with code {rc}")
    return r


def mean_params(X: np.ndarray, _lib=None) -> np.ndarray:
    """xbar = (1/N) sum_i x^i, the output of Algorithm 1 and the model sent back by an averaging iteration."""
    assert X.dtype == np.float32 and X.flags.c_contiguous and X.ndim == 2
    out = np.empty(X.shape[1], np.float32)
    (_lib or lib()).liec_oracle_mean_params(X.shape[0], X.shape[1], _ptr(X), _ptr(out))
    return out


def average_step(X: np.ndarray, e: np.ndarray, G: np.ndarray, lr: float, _lib=None):
    """Model-averaging iteration of Algorithm 1; X and e updated in place; returns (v, xbar)."""
    assert X.dtype == np.float32 and X.flags.c_contiguous and X.ndim == 2
    assert e.dtype == np.float32 and e.flags.c_contiguous
    G = _f32(G)
    N, d = X.shape
    assert G.shape == (N, d) and e.shape == (d,)
    v = np.empty(d, np.float32)
    xbar = np.empty(d, np.float32)
    rc = (_lib or lib()).liec_oracle_average_step(N, d, _ptr(G), C.c_float(lr), _ptr(X), _ptr(e), _ptr(v), _ptr(xbar))
    if rc:
        raise MemoryError("oracle average step out of memory")
    return v, xbar


def philox4x32_10(ctr, key, _lib=None) -> np.ndarray:
    """One block of the counter-based generator behind the seeded subset draw."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    assert c.shape == (4,) and k.shape == (2,)
    out = np.empty(4, np.uint32)
    (_lib or lib()).liec_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def subset_scores(seed: int, epoch: int, row: int, t: int, n: int, _lib=None) -> np.ndarray:
    out = np.empty(n, np.uint32)
    (_lib or lib()).liec_oracle_subset_scores(int(seed), int(epoch), int(row), int(t), int(n), _ptr(out))
    return out


def subset_from_scores(scores, k: int, _lib=None) -> np.ndarray:
    """Positions of the k highest scores (equal scores: lower index first), ascending."""
    sc = np.ascontiguousarray(scores, dtype=np.uint32)
    out = np.empty(int(k), np.uint32)
    rc = (_lib or lib()).liec_oracle_subset_from_scores(_ptr(sc), sc.size, int(k), _ptr(out))
    if rc:
        raise MemoryError("oracle subset selection out of memory")
    return out


def draw_subsets(seed: int, epoch: int, rows: int, off, k, _lib=None) -> np.ndarray:
    """Seeded random-k subsets (Def. 3) of `rows` rows: [rows, K] flat indices, ascending inside
    each segment.  Row i < N is worker i's subset, row N the server's."""
    off = _off(off)
    k = np.ascontiguousarray(k, dtype=np.int64)
    T = off.size - 1
    out = np.empty((int(rows), int(k.sum())), np.uint32)
    rc = (_lib or lib()).liec_oracle_draw_subsets(int(seed), int(epoch), int(rows), T, _ptr(off), _ptr(k), _ptr(out))
    if rc:
        raise MemoryError("oracle subset draw out of memory")
    return out
