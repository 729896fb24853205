"""ctypes loader for the plain-C oracle in ``stream_oracle.c``.

Test infrastructure only. It is compiled with gcc on the machine that uses it (the object is
keyed by the source text, the flags and the CPU model, so a copy built elsewhere is never
reused) and holds no arithmetic of its own: every number comes from the C file.

Arrays are numpy, contiguous: Q ``[batch, n_q_heads, T, d]``, K/V ``[batch, n_kv_heads, T, d]``,
dtype float32, or uint16 holding bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import platform
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stream_oracle.c")
_FLAGS = ["-O3", "-march=native", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11"]

SCORE_CACHE = 1  # so_build_mask_rows flag: reuse s(q, r) within a row (same values, fewer tiles)


class _CProblem(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("T", ctypes.c_int64),
        ("d", ctypes.c_int32), ("block_q", ctypes.c_int32), ("block_k", ctypes.c_int32),
        ("k_top", ctypes.c_int32), ("causal", ctypes.c_int32), ("dtype", ctypes.c_int32),
    ]


@dataclass(frozen=True)
class OracleProblem:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    T: int
    d: int
    block_q: int
    block_k: int
    k_top: int
    causal: bool = True
    dtype: str = "f32"  # "f32" or "bf16"

    def c(self) -> _CProblem:
        return _CProblem(self.batch, self.n_q_heads, self.n_kv_heads, self.T, self.d, self.block_q,
                         self.block_k, self.k_top, int(self.causal), {"f32": 0, "bf16": 1}[self.dtype])


def _cpu_tag() -> str:
    model = platform.processor()
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.startswith(("model name", "flags")):
                    model += line
                    if line.startswith("flags"):
                        break
    except OSError:
        pass
    return model


def _lib_path() -> str:
    with open(_SRC, "rb") as fh:
        key = hashlib.sha256(fh.read() + " ".join(_FLAGS).encode() + _cpu_tag().encode()).hexdigest()[:16]
    return os.path.join(_HERE, "_build", f"libstream_oracle_{key}.so")


def build() -> str:
    """Compile the oracle for this machine if that has not been done; return the library path."""
    path = _lib_path()
    if not os.path.exists(path):
        os.makedirs(os.path.dirname(path), exist_ok=True)
        tmp = f"{path}.{os.getpid()}.tmp"
        subprocess.run(["gcc", *_FLAGS, _SRC, "-o", tmp, "-lm"], check=True)
        os.replace(tmp, path)
    return path


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64p = ctypes.c_void_p, ctypes.c_void_p
        lib.so_num_query_blocks.restype = ctypes.c_int64
        lib.so_num_query_blocks.argtypes = [ctypes.POINTER(_CProblem)]
        lib.so_num_rows.restype = ctypes.c_int64
        lib.so_num_rows.argtypes = [ctypes.POINTER(_CProblem)]
        lib.so_threads.restype = ctypes.c_int
        lib.so_tile_score.restype = ctypes.c_float
        lib.so_tile_score.argtypes = [ctypes.POINTER(_CProblem), vp, vp] + [ctypes.c_int64] * 4
        lib.so_build_mask_rows.restype = ctypes.c_int
        lib.so_build_mask_rows.argtypes = [ctypes.POINTER(_CProblem), vp, vp, i64p, ctypes.c_int64,
                                           vp, vp, vp, vp, ctypes.c_int, ctypes.c_int]
        lib.so_build_mask_rows_var.restype = ctypes.c_int
        lib.so_build_mask_rows_var.argtypes = [ctypes.POINTER(_CProblem), vp, vp, vp, i64p, ctypes.c_int64,
                                               vp, vp, vp, vp, ctypes.c_int]
        lib.so_build_mask_rows_multi.restype = ctypes.c_int
        lib.so_build_mask_rows_multi.argtypes = [ctypes.POINTER(_CProblem), vp, vp, ctypes.c_int32, vp, i64p,
                                                 ctypes.c_int64, vp, vp, vp, vp, ctypes.c_int]
        lib.so_effective_k.restype = ctypes.c_int64
        lib.so_effective_k.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_double]
        lib.so_k_schedule.restype = ctypes.c_int
        lib.so_k_schedule.argtypes = [ctypes.POINTER(_CProblem), ctypes.c_double, vp]
        lib.so_sparse_attention_rows.restype = ctypes.c_int
        lib.so_sparse_attention_rows.argtypes = [ctypes.POINTER(_CProblem), vp, vp, vp, i64p, ctypes.c_int64,
                                                 vp, ctypes.c_double, vp]
        lib.so_mask_difference.restype = ctypes.c_int
        lib.so_mask_difference.argtypes = [ctypes.c_int64, ctypes.c_int32, vp, vp, ctypes.c_int32, vp, vp, vp]
        lib.so_vertical_scores.restype = ctypes.c_int
        lib.so_vertical_scores.argtypes = [ctypes.POINTER(_CProblem), vp, vp, vp, vp]
        _lib = lib
    return _lib


def _check(p: OracleProblem, x: np.ndarray, heads: int, name: str) -> np.ndarray:
    want = np.float32 if p.dtype == "f32" else np.uint16
    if x.dtype != want or not x.flags["C_CONTIGUOUS"] or x.shape != (p.batch, heads, p.T, p.d):
        raise ValueError(f"{name}: need contiguous {np.dtype(want)} array of shape {(p.batch, heads, p.T, p.d)}")
    return x


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def threads() -> int:
    return int(_load().so_threads())


def num_query_blocks(p: OracleProblem) -> int:
    return int(_load().so_num_query_blocks(ctypes.byref(p.c())))


def num_rows(p: OracleProblem) -> int:
    return int(_load().so_num_rows(ctypes.byref(p.c())))


def tile_score(p: OracleProblem, q: np.ndarray, k: np.ndarray, b: int, h: int, qb: int, r: int) -> float:
    _check(p, q, p.n_q_heads, "q"), _check(p, k, p.n_kv_heads, "k")
    return float(_load().so_tile_score(ctypes.byref(p.c()), _ptr(q), _ptr(k), b, h, qb, r))


def build_mask_rows(p: OracleProblem, q: np.ndarray, k: np.ndarray, rows=None, *, n_it: int = -1,
                    score_cache: bool = False, want_scores: bool = False):
    """Algorithm 2 for ``rows`` (flat row ids; ``None`` = every row).

    Returns a dict: ``mask`` int32 [n, k_top] (ascending block indices, -1 padded), ``min_gap``
    float32 [n], ``tiles`` int64 [n] and, if asked, ``scores`` float32 [n, k_top].
    """
    _check(p, q, p.n_q_heads, "q"), _check(p, k, p.n_kv_heads, "k")
    lib = _load()
    rows_arr = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = num_rows(p) if rows_arr is None else rows_arr.shape[0]
    mask = np.empty((n, p.k_top), np.int32)
    gap = np.empty((n,), np.float32)
    tiles = np.empty((n,), np.int64)
    scores = np.empty((n, p.k_top), np.float32) if want_scores else None
    rc = lib.so_build_mask_rows(ctypes.byref(p.c()), _ptr(q), _ptr(k), _ptr(rows_arr), n, _ptr(mask),
                                _ptr(scores), _ptr(gap), _ptr(tiles), n_it, SCORE_CACHE if score_cache else 0)
    if rc:
        raise RuntimeError(f"so_build_mask_rows failed with {rc}")
    out = {"mask": mask, "min_gap": gap, "tiles": tiles}
    if want_scores:
        out["scores"] = scores
    return out


def build_mask_rows_var(p: OracleProblem, q: np.ndarray, k: np.ndarray, k_row: np.ndarray, rows=None, *,
                        score_cache: bool = False, want_scores: bool = False):
    """Algorithm 2 with ``k = k_row[query block]`` per row (clamped to 1 .. k_top); same returns as
    :func:`build_mask_rows`, rows ``k_top`` wide."""
    _check(p, q, p.n_q_heads, "q"), _check(p, k, p.n_kv_heads, "k")
    lib = _load()
    k_row = np.ascontiguousarray(k_row, dtype=np.int32)
    if k_row.shape != (num_query_blocks(p),):
        raise ValueError(f"k_row: need shape {(num_query_blocks(p),)}, got {k_row.shape}")
    rows_arr = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = num_rows(p) if rows_arr is None else rows_arr.shape[0]
    mask = np.empty((n, p.k_top), np.int32)
    gap = np.empty((n,), np.float32)
    tiles = np.empty((n,), np.int64)
    scores = np.empty((n, p.k_top), np.float32) if want_scores else None
    rc = lib.so_build_mask_rows_var(ctypes.byref(p.c()), _ptr(q), _ptr(k), _ptr(k_row), _ptr(rows_arr), n,
                                    _ptr(mask), _ptr(scores), _ptr(gap), _ptr(tiles),
                                    SCORE_CACHE if score_cache else 0)
    if rc:
        raise RuntimeError(f"so_build_mask_rows_var failed with {rc}")
    out = {"mask": mask, "min_gap": gap, "tiles": tiles}
    if want_scores:
        out["scores"] = scores
    return out


def build_mask_rows_multi(p: OracleProblem, q: np.ndarray, k: np.ndarray, k_list, rows=None, *,
                          score_cache: bool = False, want_scores: bool = False):
    """Algorithm 2 for every k in ``k_list`` (each 1 .. k_top). Returns ``mask`` int32
    [n_k, n, k_top], ``min_gap`` [n_k, n], ``tiles`` int64 [n] (distinct tiles over all k of a row)
    and, if asked, ``scores`` [n_k, n, k_top]."""
    _check(p, q, p.n_q_heads, "q"), _check(p, k, p.n_kv_heads, "k")
    lib = _load()
    ks = np.ascontiguousarray(k_list, dtype=np.int32)
    rows_arr = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = num_rows(p) if rows_arr is None else rows_arr.shape[0]
    mask = np.empty((len(ks), n, p.k_top), np.int32)
    gap = np.empty((len(ks), n), np.float32)
    tiles = np.empty((n,), np.int64)
    scores = np.empty((len(ks), n, p.k_top), np.float32) if want_scores else None
    rc = lib.so_build_mask_rows_multi(ctypes.byref(p.c()), _ptr(q), _ptr(k), len(ks), _ptr(ks), _ptr(rows_arr), n,
                                      _ptr(mask), _ptr(scores), _ptr(gap), _ptr(tiles),
                                      SCORE_CACHE if score_cache else 0)
    if rc:
        raise RuntimeError(f"so_build_mask_rows_multi failed with {rc}")
    out = {"mask": mask, "min_gap": gap, "tiles": tiles}
    if want_scores:
        out["scores"] = scores
    return out


def k_schedule(p: OracleProblem, s: float) -> np.ndarray:
    """``k`` per query block from the effective sparsity ``s`` (0 < s < 1) and the row's own number
    of allowed key blocks; int32 [ceil(T / block_q)], clamped to 1 .. k_top."""
    out = np.empty((num_query_blocks(p),), np.int32)
    rc = _load().so_k_schedule(ctypes.byref(p.c()), float(s), _ptr(out))
    if rc:
        raise RuntimeError(f"so_k_schedule failed with {rc}")
    return out


def effective_k(T: int, block_q: int, s: float) -> int:
    """The printed effective-sparsity formula (Section 4.2): ``floor(1 + (T / b_q - 1) s)`` in 1 .. floor(T / b_q)."""
    k = int(_load().so_effective_k(int(T), int(block_q), float(s)))
    if k < 0:
        raise ValueError("need T, block_q >= 1 and 0 <= s <= 1")
    return k


def sparse_attention_rows(p: OracleProblem, q: np.ndarray, k: np.ndarray, v: np.ndarray, mask: np.ndarray,
                          rows=None, *, scale: float | None = None) -> np.ndarray:
    """Eq. 2 restricted to the blocks in ``mask`` ([n, k_top]); returns fp64 [n, block_q, d]."""
    _check(p, q, p.n_q_heads, "q"), _check(p, k, p.n_kv_heads, "k"), _check(p, v, p.n_kv_heads, "v")
    lib = _load()
    rows_arr = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = num_rows(p) if rows_arr is None else rows_arr.shape[0]
    mask = np.ascontiguousarray(mask, dtype=np.int32)
    if mask.shape != (n, p.k_top):
        raise ValueError(f"mask: need shape {(n, p.k_top)}, got {mask.shape}")
    out = np.empty((n, p.block_q, p.d), np.float64)
    s = float(scale) if scale is not None else 1.0 / float(np.sqrt(p.d))
    rc = lib.so_sparse_attention_rows(ctypes.byref(p.c()), _ptr(q), _ptr(k), _ptr(v), _ptr(rows_arr), n,
                                      _ptr(mask), s, _ptr(out))
    if rc:
        raise RuntimeError(f"so_sparse_attention_rows failed with {rc}")
    return out


def vertical_scores(p: OracleProblem, mask: np.ndarray, scores: np.ndarray | None = None):
    """Column sums of a block mask (binary, or weighted by ``scores``) per head and their kurtosis.

    ``mask`` (and ``scores``) cover every row: [num_rows, k_top]. Returns (vertical fp64
    [batch * n_q_heads, ceil(T / block_k)], kurtosis fp64 [batch * n_q_heads]).
    """
    lib = _load()
    n = num_rows(p)
    mask = np.ascontiguousarray(mask, dtype=np.int32)
    if mask.shape != (n, p.k_top):
        raise ValueError(f"mask: need shape {(n, p.k_top)}, got {mask.shape}")
    if scores is not None:
        scores = np.ascontiguousarray(scores, dtype=np.float32)
        if scores.shape != mask.shape:
            raise ValueError("scores must have the mask's shape")
    heads, nk = p.batch * p.n_q_heads, -(-p.T // p.block_k)
    vert = np.empty((heads, nk), np.float64)
    kurt = np.empty((heads,), np.float64)
    rc = lib.so_vertical_scores(ctypes.byref(p.c()), _ptr(mask), _ptr(scores), _ptr(vert), _ptr(kurt))
    if rc:
        raise RuntimeError(f"so_vertical_scores failed with {rc}")
    return vert, kurt


def mask_difference(mask_a: np.ndarray, mask_b: np.ndarray, scores_a: np.ndarray | None = None):
    """Row-wise ``mask_a`` minus ``mask_b`` ([n, k_a], [n, k_b]); returns (diff [n, k_a], scores or None)."""
    lib = _load()
    mask_a = np.ascontiguousarray(mask_a, dtype=np.int32)
    mask_b = np.ascontiguousarray(mask_b, dtype=np.int32)
    if mask_a.ndim != 2 or mask_b.ndim != 2 or mask_a.shape[0] != mask_b.shape[0]:
        raise ValueError("masks must be [n, k_a] and [n, k_b]")
    if scores_a is not None:
        scores_a = np.ascontiguousarray(scores_a, dtype=np.float32)
    diff = np.empty_like(mask_a)
    dsc = np.empty(mask_a.shape, np.float32) if scores_a is not None else None
    rc = lib.so_mask_difference(mask_a.shape[0], mask_a.shape[1], _ptr(mask_a), _ptr(scores_a), mask_b.shape[1],
                                _ptr(mask_b), _ptr(diff), _ptr(dsc))
    if rc:
        raise RuntimeError(f"so_mask_difference failed with {rc}")
    return diff, dsc
