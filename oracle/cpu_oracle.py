"""ctypes loader for the plain-C oracle (`ivfpq_oracle.c`).  TEST INFRASTRUCTURE ONLY.

Compiles the C file on first use with strict fp32 flags (`-O2 -ffp-contract=off`,
no fast-math; `-mfma` only when the host CPU has it, so that `fmaf` is a single
instruction instead of a library call - the value is the same either way) and
exposes `coarse()` and `search()` on numpy arrays.  The index argument is any
object with the attributes of `ivfpq_inputs.IvfPqIndex`.
"""

from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ivfpq_oracle.c")
_LIB: Optional[ctypes.CDLL] = None


def _cpu_has_fma() -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    return " fma " in line + " "
    except OSError:
        pass
    return False


def build() -> str:
    """Compile the oracle if its shared object is missing or stale; return its path."""
    flags = ["-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared"]
    if _cpu_has_fma():
        flags.append("-mfma")
    with open(_SRC, "rb") as f:
        tag = hashlib.sha1(f.read() + " ".join(flags).encode()).hexdigest()[:12]
    out_dir = os.path.join(_HERE, "_build")
    os.makedirs(out_dir, exist_ok=True)
    out = os.path.join(out_dir, f"libivfpq_oracle_{tag}.so")
    if not os.path.exists(out):
        tmp = out + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *flags, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, out)
    return out


def _lib() -> ctypes.CDLL:
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build())
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
        lib.oracle_coarse.argtypes = [vp, i64, i32, vp, i32, i32, vp, vp]
        lib.oracle_coarse.restype = i32
        lib.oracle_search.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp,      # index
                                      vp, i64, i32, i32,                               # queries
                                      vp, i32, f32, f32, i32,                          # radius, k
                                      vp, vp,                                          # outputs
                                      vp, vp, vp, vp, i64, vp, vp, vp]                 # dumps
        lib.oracle_search.restype = i32
        lib.oracle_search_scored.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp,
                                             vp, i64, i32, i32,
                                             vp, i32, f32, f32, i32, i32,             # ..., score, k
                                             vp, vp,
                                             vp, vp, vp, vp, i64, vp, vp, vp]
        lib.oracle_search_scored.restype = i32
        lib.oracle_entry_stats.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i64, vp, i32, vp, vp]
        lib.oracle_entry_stats.restype = i32
        lib.oracle_search_ip.argtypes = list(lib.oracle_search.argtypes)
        lib.oracle_search_ip.restype = i32
        lib.oracle_thresholds.argtypes = [i32, i32, i32, vp, i64, i32, i32, vp, vp, vp, vp, vp]
        lib.oracle_thresholds.restype = i32
        lib.oracle_thresholds_knn.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, i64, i32, i32, vp, vp]
        lib.oracle_thresholds_knn.restype = i32
        lib.oracle_num_threads.restype = i32
        lib.oracle_set_num_threads.argtypes = [i32]
        _LIB = lib
    return _LIB


def num_threads() -> int:
    return int(_lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _lib().oracle_set_num_threads(int(n))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def coarse(index, queries: np.ndarray, nprobe: int):
    """S1 only: (probe_ids [nq, nprobe] int32, probe_d [nq, nprobe] fp32)."""
    q = _c(queries, np.float32)
    cent = _c(index.coarse_centroids, np.float32)
    nq = q.shape[0]
    pid = np.empty((nq, nprobe), np.int32)
    pd = np.empty((nq, nprobe), np.float32)
    rc = _lib().oracle_coarse(_p(q), nq, index.d, _p(cent), index.nlist, nprobe, _p(pid), _p(pd))
    if rc != 0:
        raise ValueError(f"oracle_coarse failed: {rc}")
    return pid, pd


def search(index, queries: np.ndarray, nprobe: int, k: int, *, dense: bool = False,
           radius: Optional[np.ndarray] = None, scale: float = 1.0, miss_penalty: float = -1.0,
           dumps: bool = False, visit_stride: int = 0, score: int = 0, metric: Optional[int] = None) -> dict:
    """Dense (`dense=True`) or sparsity-aware search.  `radius` is [nsub] (one
    threshold per subspace) or [nq, nsub] (per query and subspace).  Returns a dict
    with `dist` [nq, k] fp32 and `ids` [nq, k] int32; with `dumps=True` also
    `probe_ids`, `probe_d`, `masks` [nq, nprobe, nsub, 8] uint32 and `visit_count`;
    with `visit_stride > 0` also per-visited-point `visit_hits` (uint64 bit sets),
    `visit_dist` and `visit_ids`, each [nq, visit_stride] in visiting order.
    `score`: 0 = distances; 1 = hit count (reported value: subspaces missed); 2 = reward/penalty
    with an inner sphere of half the radius (reported value: nsub - score).
    `metric` (default: the index's): 0 = squared L2; 1 = inner product, where `dist`, `probe_d`
    and `visit_dist` hold similarities, larger first, padded with -inf."""
    q = _c(queries, np.float32)
    nq = q.shape[0]
    cent = _c(index.coarse_centroids, np.float32)
    cb = _c(index.codebooks, np.float32)
    off = _c(index.list_offsets, np.int64)
    codes = _c(index.codes, np.uint8)
    ids = _c(index.ids, np.int32)
    rad, mode = None, 0
    if not dense:
        if radius is None:
            raise ValueError("sparse search needs radius")
        rad = _c(radius, np.float32)
        if rad.shape == (index.nsub,):
            mode = 0
        elif rad.shape == (nq, index.nsub):
            mode = 1
        else:
            raise ValueError("radius must be [nsub] or [nq, nsub]")
    out_d = np.empty((nq, k), np.float32)
    out_i = np.empty((nq, k), np.int32)
    res = {"dist": out_d, "ids": out_i}
    pid = pd = masks = vcount = vh = vd = vi = None
    if dumps or visit_stride > 0:
        pid = np.empty((nq, nprobe), np.int32)
        pd = np.empty((nq, nprobe), np.float32)
        masks = np.zeros((nq, nprobe, index.nsub, 8), np.uint32)
        vcount = np.zeros(nq, np.int64)
        res.update(probe_ids=pid, probe_d=pd, masks=masks, visit_count=vcount)
    if visit_stride > 0:
        vh = np.zeros((nq, visit_stride), np.uint64)
        vd = np.full((nq, visit_stride), np.inf, np.float32)
        vi = np.full((nq, visit_stride), -1, np.int32)
        res.update(visit_hits=vh, visit_dist=vd, visit_ids=vi)
    metric = int(getattr(index, "metric", 0)) if metric is None else int(metric)
    if metric == 1:
        if score != 0:
            raise ValueError("the count scores are defined for the L2 metric only")
        if visit_stride > 0:
            vd.fill(-np.inf)
        rc = _lib().oracle_search_ip(index.d, index.nlist, index.nsub, index.dsub, index.ksub,
                                     _p(cent), _p(cb), _p(off), _p(codes), _p(ids),
                                     _p(q), nq, nprobe, 1 if dense else 0,
                                     _p(rad), mode, float(scale), float(miss_penalty), k,
                                     _p(out_d), _p(out_i),
                                     _p(pid), _p(pd), _p(masks), _p(vcount), int(visit_stride),
                                     _p(vh), _p(vd), _p(vi))
        if rc != 0:
            raise ValueError(f"oracle_search_ip failed: {rc}")
        return res
    rc = _lib().oracle_search_scored(index.d, index.nlist, index.nsub, index.dsub, index.ksub,
                                     _p(cent), _p(cb), _p(off), _p(codes), _p(ids),
                                     _p(q), nq, nprobe, 1 if dense else 0,
                                     _p(rad), mode, float(scale), float(miss_penalty), int(score), k,
                                     _p(out_d), _p(out_i),
                                     _p(pid), _p(pd), _p(masks), _p(vcount), int(visit_stride),
                                     _p(vh), _p(vd), _p(vi))
    if rc != 0:
        raise ValueError(f"oracle_search failed: {rc}")
    return res


def thresholds(d: int, nsub: int, dsub: int, queries: np.ndarray, model) -> np.ndarray:
    """Dynamic thresholds [nq, nsub] fp32 from a density-map + polynomial model (an object with
    `grid`, `degree`, `density` [nsub, grid, grid], `origin` [nsub, 2], `inv_cell` [nsub, 2] and
    `coef` [nsub, degree + 1], as `ivfpq_inputs.ThresholdModel`)."""
    q = _c(queries, np.float32)
    dens = _c(model.density, np.float32)
    org = _c(model.origin, np.float32)
    inv = _c(model.inv_cell, np.float32)
    cf = _c(model.coef, np.float32)
    out = np.empty((q.shape[0], nsub), np.float32)
    rc = _lib().oracle_thresholds(d, nsub, dsub, _p(q), q.shape[0], int(model.grid), int(model.degree),
                                  _p(dens), _p(org), _p(inv), _p(cf), _p(out))
    if rc != 0:
        raise ValueError(f"oracle_thresholds failed: {rc}")
    return out


def thresholds_knn(index, queries: np.ndarray, kth: int, coef: np.ndarray) -> np.ndarray:
    """Dynamic thresholds [nq, nsub] fp32 for subspaces of any width: a per-subspace polynomial
    (`coef` [nsub, degree + 1], ascending powers) of the distance from the query's residual
    projection (against its nearest cluster) to its `kth`-nearest codebook entry."""
    q = _c(queries, np.float32)
    cent = _c(index.coarse_centroids, np.float32)
    cb = _c(index.codebooks, np.float32)
    cf = _c(coef, np.float32)
    if cf.ndim != 2 or cf.shape[0] != index.nsub:
        raise ValueError("coef must be [nsub, degree + 1]")
    out = np.empty((q.shape[0], index.nsub), np.float32)
    rc = _lib().oracle_thresholds_knn(index.d, index.nlist, index.nsub, index.dsub, index.ksub, _p(cent), _p(cb),
                                      _p(q), q.shape[0], int(kth), cf.shape[1] - 1, _p(cf), _p(out))
    if rc != 0:
        raise ValueError(f"oracle_thresholds_knn failed: {rc}")
    return out


def entry_stats(index, queries: np.ndarray, neighbor_pos: np.ndarray):
    """Entry usage and locality statistics of each query's neighbours (`neighbor_pos` [nq, k] int64
    positions into the list-contiguous codes, -1 = none).  Returns (usage [nq, nsub] int32: distinct
    entries used per subspace; rank_hist [nsub, ksub] int64: how often a neighbour's entry was the
    r-th closest entry to the query's residual projection)."""
    q = _c(queries, np.float32)
    pos = _c(neighbor_pos, np.int64)
    nq, k = pos.shape
    cent = _c(index.coarse_centroids, np.float32)
    cb = _c(index.codebooks, np.float32)
    off = _c(index.list_offsets, np.int64)
    codes = _c(index.codes, np.uint8)
    usage = np.zeros((nq, index.nsub), np.int32)
    hist = np.zeros((index.nsub, index.ksub), np.int64)
    rc = _lib().oracle_entry_stats(index.d, index.nlist, index.nsub, index.dsub, index.ksub, _p(cent), _p(cb),
                                   _p(off), _p(codes), _p(q), nq, _p(pos), k, _p(usage), _p(hist))
    if rc != 0:
        raise ValueError(f"oracle_entry_stats failed: {rc}")
    return usage, hist
