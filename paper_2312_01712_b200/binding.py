"""Thin ctypes binding of `libivfpq_b200.so` (declared in `include/ivfpq.h`).

Argument marshalling only: every step of the search runs in the CUDA library.
torch is used for device memory and for the current stream.  There is no CPU
path: loading fails loudly when the shared object is missing, and every compute
call fails when no CUDA device is present.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libivfpq_b200.so")

IVFPQ_OK = 0
IVFPQ_ERR_INVALID_ARGUMENT = -1
IVFPQ_ERR_UNSUPPORTED = -2
IVFPQ_ERR_WORKSPACE = -3
IVFPQ_ERR_CUDA = -4
IVFPQ_ERR_DEVICE_FLAG = -5
IVFPQ_ERR_STATIC_LIMIT = -6
IVFPQ_STATIC_SCRATCH_BYTES = 8 << 20
IVFPQ_STATIC_MAX_NLIST = 16384
IVFPQ_OPT_NSPLIT = 1
IVFPQ_OPT_TIMING = 2
IVFPQ_OPT_SPARSE_SCAN = 3
IVFPQ_OPT_TEST_FAULT = 4
IVFPQ_SPARSE_SCAN_AUTO = 0
IVFPQ_SPARSE_SCAN_STREAM = 1
IVFPQ_SPARSE_SCAN_MAP = 2
IVFPQ_METRIC_L2 = 0
IVFPQ_METRIC_IP = 1
IVFPQ_SCORE_DISTANCE = 0
IVFPQ_SCORE_HIT_COUNT = 1
IVFPQ_SCORE_REWARD_PENALTY = 2

EXPORTS = (
    "ivfpq_index_derived_bytes", "ivfpq_index_load", "ivfpq_index_free",
    "ivfpq_search_workspace_bytes", "ivfpq_search_dense", "ivfpq_search_sparse",
    "ivfpq_search_host_workspace_bytes", "ivfpq_search_host", "ivfpq_sync_status",
    "ivfpq_index_set_option", "ivfpq_last_launch_count", "ivfpq_last_stage_ms", "ivfpq_error_string",
    "ivfpq_debug_probes", "ivfpq_debug_search", "ivfpq_probe_static", "ivfpq_static_status", "ivfpq_query_thresholds",
    "ivfpq_query_thresholds_knn",
    "ivfpq_entry_stats",
)


class IvfpqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {error_string(code)} ({code})")


class ivfpq_index_desc_t(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("nlist", ctypes.c_int32), ("nsub", ctypes.c_int32),
                ("dsub", ctypes.c_int32), ("ksub", ctypes.c_int32), ("metric", ctypes.c_int32),
                ("ntotal", ctypes.c_int64),
                ("coarse_centroids", ctypes.c_void_p), ("codebooks", ctypes.c_void_p),
                ("list_offsets", ctypes.c_void_p), ("codes", ctypes.c_void_p), ("ids", ctypes.c_void_p)]


class ivfpq_radius_t(ctypes.Structure):
    _fields_ = [("radius", ctypes.c_void_p), ("mode", ctypes.c_int32), ("scale", ctypes.c_float),
                ("miss_penalty", ctypes.c_float), ("score", ctypes.c_int32)]


class ivfpq_threshold_model_t(ctypes.Structure):
    _fields_ = [("grid", ctypes.c_int32), ("degree", ctypes.c_int32), ("density", ctypes.c_void_p),
                ("origin", ctypes.c_void_p), ("inv_cell", ctypes.c_void_p), ("coef", ctypes.c_void_p)]


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """dlopen the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2312_01712_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t, ctypes.c_float
    lib.ivfpq_index_derived_bytes.argtypes = [ctypes.POINTER(ivfpq_index_desc_t)]
    lib.ivfpq_index_derived_bytes.restype = sz
    lib.ivfpq_index_load.argtypes = [ctypes.POINTER(ivfpq_index_desc_t), vp, sz, vp, ctypes.POINTER(vp)]
    lib.ivfpq_index_load.restype = ctypes.c_int
    lib.ivfpq_index_free.argtypes = [vp]
    lib.ivfpq_index_free.restype = ctypes.c_int
    lib.ivfpq_search_workspace_bytes.argtypes = [vp, i64, i32, i32]
    lib.ivfpq_search_workspace_bytes.restype = sz
    lib.ivfpq_search_dense.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, sz, vp]
    lib.ivfpq_search_dense.restype = ctypes.c_int
    lib.ivfpq_search_sparse.argtypes = [vp, vp, i64, i32, ctypes.POINTER(ivfpq_radius_t), i32, vp, vp, vp, sz, vp]
    lib.ivfpq_search_sparse.restype = ctypes.c_int
    lib.ivfpq_search_host_workspace_bytes.argtypes = [vp, i64, i32, i32]
    lib.ivfpq_search_host_workspace_bytes.restype = sz
    lib.ivfpq_search_host.argtypes = [vp, vp, i64, i32, ctypes.POINTER(ivfpq_radius_t), i32, vp, vp, vp, sz, vp]
    lib.ivfpq_search_host.restype = ctypes.c_int
    lib.ivfpq_sync_status.argtypes = [vp, vp, vp]
    lib.ivfpq_sync_status.restype = ctypes.c_int
    lib.ivfpq_index_set_option.argtypes = [vp, i32, i64]
    lib.ivfpq_index_set_option.restype = ctypes.c_int
    lib.ivfpq_last_launch_count.argtypes = [vp]
    lib.ivfpq_last_launch_count.restype = i64
    lib.ivfpq_last_stage_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.ivfpq_last_stage_ms.restype = ctypes.c_int
    lib.ivfpq_error_string.argtypes = [ctypes.c_int]
    lib.ivfpq_error_string.restype = ctypes.c_char_p
    lib.ivfpq_debug_probes.argtypes = [vp, vp, i64, i32, vp, vp, vp, sz, vp]
    lib.ivfpq_debug_probes.restype = ctypes.c_int
    lib.ivfpq_debug_search.argtypes = [vp, vp, i64, i32, ctypes.POINTER(ivfpq_radius_t), i32, vp, vp,
                                       vp, vp, vp, vp, i64, vp, vp, vp, vp, sz, vp]
    lib.ivfpq_debug_search.restype = ctypes.c_int
    lib.ivfpq_query_thresholds.argtypes = [vp, vp, i64, ctypes.POINTER(ivfpq_threshold_model_t), vp, vp]
    lib.ivfpq_query_thresholds.restype = ctypes.c_int
    lib.ivfpq_query_thresholds_knn.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, ctypes.c_size_t, vp]
    lib.ivfpq_query_thresholds_knn.restype = ctypes.c_int
    lib.ivfpq_entry_stats.argtypes = [vp, vp, vp, i64, vp, i32, vp, vp, vp, vp]
    lib.ivfpq_entry_stats.restype = ctypes.c_int
    lib.ivfpq_probe_static.argtypes = [vp, vp, i64, i32, vp, vp, vp]
    lib.ivfpq_probe_static.restype = ctypes.c_int
    lib.ivfpq_static_status.argtypes = [vp]
    lib.ivfpq_static_status.restype = ctypes.c_int
    _lib = lib
    return lib


def error_string(code: int) -> str:
    return load_library().ivfpq_error_string(int(code)).decode()


def _check(rc: int, where: str) -> None:
    if rc != IVFPQ_OK:
        raise IvfpqError(rc, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


class IndexHandle:
    """Owns the device copies of an index and the library handle built on them."""

    def __init__(self, handle: int, tensors: dict, meta: dict):
        self.handle = handle
        self.tensors = tensors          # keeps the device memory alive
        self.__dict__.update(meta)      # d, nlist, nsub, dsub, ksub, ntotal
        self._ws: Optional[torch.Tensor] = None

    def workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.tensors["cent"].device)
        return self._ws

    def close(self) -> None:
        if self.handle:
            load_library().ivfpq_index_free(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ivfpq_index_load(index, device="cuda") -> IndexHandle:
    """Copies an `ivfpq_inputs.IvfPqIndex`-like object (numpy arrays) to the device
    and calls ivfpq_index_load on it."""
    lib = load_library()
    if not torch.cuda.is_available():
        raise RuntimeError("ivfpq_index_load: no CUDA device (there is no CPU fallback)")
    dev = torch.device(device)
    cent = torch.from_numpy(np.ascontiguousarray(index.coarse_centroids, np.float32)).to(dev)
    cb = torch.from_numpy(np.ascontiguousarray(index.codebooks, np.float32)).to(dev)
    codes = torch.from_numpy(np.ascontiguousarray(index.codes, np.uint8)).to(dev)
    ids = torch.from_numpy(np.ascontiguousarray(index.ids, np.int32)).to(dev)
    off = np.ascontiguousarray(index.list_offsets, np.int64)
    metric = int(getattr(index, "metric", IVFPQ_METRIC_L2))
    desc = ivfpq_index_desc_t(index.d, index.nlist, index.nsub, index.dsub, index.ksub, metric, index.ntotal,
                              cent.data_ptr(), cb.data_ptr(), off.ctypes.data, codes.data_ptr(), ids.data_ptr())
    nbytes = lib.ivfpq_index_derived_bytes(ctypes.byref(desc))
    if nbytes == 0:
        raise IvfpqError(IVFPQ_ERR_INVALID_ARGUMENT, "ivfpq_index_derived_bytes")
    derived = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    handle = ctypes.c_void_p()
    with torch.cuda.device(dev):
        _check(lib.ivfpq_index_load(ctypes.byref(desc), derived.data_ptr(), nbytes, _stream(), ctypes.byref(handle)),
               "ivfpq_index_load")
        torch.cuda.current_stream().synchronize()   # the source codes may be released now
    meta = dict(d=index.d, nlist=index.nlist, nsub=index.nsub, dsub=index.dsub, ksub=index.ksub,
                ntotal=index.ntotal, metric=metric)
    return IndexHandle(handle.value, {"cent": cent, "cb": cb, "ids": ids, "derived": derived}, meta)


def ivfpq_index_free(ix: IndexHandle) -> None:
    ix.close()


def ivfpq_index_set_option(ix: IndexHandle, option: int, value: int) -> None:
    _check(load_library().ivfpq_index_set_option(ix.handle, option, value), "ivfpq_index_set_option")


def ivfpq_last_launch_count(ix: IndexHandle) -> int:
    return int(load_library().ivfpq_last_launch_count(ix.handle))


def ivfpq_last_stage_ms(ix: IndexHandle) -> Tuple[float, float]:
    """(filtering ms, LUT+scan+merge ms) of the last search timed with IVFPQ_OPT_TIMING."""
    ms = (ctypes.c_float * 2)()
    _check(load_library().ivfpq_last_stage_ms(ix.handle, ms), "ivfpq_last_stage_ms")
    return float(ms[0]), float(ms[1])


def ivfpq_search_workspace_bytes(ix: IndexHandle, nq: int, nprobe: int, k: int) -> int:
    return int(load_library().ivfpq_search_workspace_bytes(ix.handle, nq, nprobe, k))


def _radius_struct(ix: IndexHandle, nq: int, radius: torch.Tensor, scale: float, miss_penalty: float,
                   score: int = IVFPQ_SCORE_DISTANCE):
    if radius.dtype != torch.float32 or not radius.is_cuda or not radius.is_contiguous():
        raise ValueError("radius must be a contiguous fp32 CUDA tensor")
    if tuple(radius.shape) == (ix.nsub,):
        mode = 0
    elif tuple(radius.shape) == (nq, ix.nsub):
        mode = 1
    else:
        raise ValueError("radius must be [nsub] or [nq, nsub]")
    return ivfpq_radius_t(radius.data_ptr(), mode, float(scale), float(miss_penalty), int(score))


def _prep(ix: IndexHandle, queries: torch.Tensor, nprobe: int, k: int):
    if queries.dtype != torch.float32 or not queries.is_cuda or not queries.is_contiguous() or queries.dim() != 2 \
            or queries.shape[1] != ix.d:
        raise ValueError("queries must be a contiguous fp32 CUDA tensor [nq, d]")
    nq = queries.shape[0]
    nbytes = ivfpq_search_workspace_bytes(ix, nq, nprobe, k)
    if nbytes == 0:
        # let the library name the reason
        _check(load_library().ivfpq_search_dense(ix.handle, queries.data_ptr(), nq, nprobe, k, None, None, None, 0,
                                                 None), "ivfpq_search")
    ws = ix.workspace(nbytes)
    out_d = torch.empty((nq, k), dtype=torch.float32, device=queries.device)
    out_i = torch.empty((nq, k), dtype=torch.int32, device=queries.device)
    return nq, ws, out_d, out_i


def ivfpq_search_dense(ix: IndexHandle, queries: torch.Tensor, nprobe: int, k: int,
                       out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None):
    """Conventional IVFPQ search.  Returns (dist [nq, k] fp32, ids [nq, k] int32) on the device."""
    nq, ws, out_d, out_i = _prep(ix, queries, nprobe, k)
    if out is not None:
        out_d, out_i = out
    _check(load_library().ivfpq_search_dense(ix.handle, queries.data_ptr(), nq, nprobe, k, out_d.data_ptr(),
                                             out_i.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "ivfpq_search_dense")
    return out_d, out_i


def ivfpq_search_sparse(ix: IndexHandle, queries: torch.Tensor, nprobe: int, radius: torch.Tensor, k: int,
                        scale: float = 1.0, miss_penalty: float = -1.0,
                        out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None,
                        score: int = IVFPQ_SCORE_DISTANCE):
    """Sparsity-aware search with per-subspace threshold radii; `score` = IVFPQ_SCORE_DISTANCE,
    IVFPQ_SCORE_HIT_COUNT or IVFPQ_SCORE_REWARD_PENALTY."""
    nq, ws, out_d, out_i = _prep(ix, queries, nprobe, k)
    if out is not None:
        out_d, out_i = out
    rs = _radius_struct(ix, nq, radius, scale, miss_penalty, score)
    _check(load_library().ivfpq_search_sparse(ix.handle, queries.data_ptr(), nq, nprobe, ctypes.byref(rs), k,
                                              out_d.data_ptr(), out_i.data_ptr(), ws.data_ptr(), ws.numel(),
                                              _stream()), "ivfpq_search_sparse")
    return out_d, out_i


def ivfpq_search_host(ix: IndexHandle, queries_host: torch.Tensor, nprobe: int, k: int,
                      out_dist_host: torch.Tensor, out_ids_host: torch.Tensor,
                      radius: Optional[torch.Tensor] = None, scale: float = 1.0, miss_penalty: float = -1.0,
                      score: int = IVFPQ_SCORE_DISTANCE):
    """End-to-end call with host (ideally pinned) query and result buffers; asynchronous on
    the current stream: synchronise before reading the results."""
    lib = load_library()
    nq = queries_host.shape[0]
    for t, dt in ((queries_host, torch.float32), (out_dist_host, torch.float32), (out_ids_host, torch.int32)):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise ValueError("host buffers must be contiguous CPU tensors of the right dtype")
    nbytes = int(lib.ivfpq_search_host_workspace_bytes(ix.handle, nq, nprobe, k))
    ws = ix.workspace(nbytes)
    rs = None if radius is None else _radius_struct(ix, nq, radius, scale, miss_penalty, score)
    _check(lib.ivfpq_search_host(ix.handle, queries_host.data_ptr(), nq, nprobe,
                                 None if rs is None else ctypes.byref(rs), k, out_dist_host.data_ptr(),
                                 out_ids_host.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "ivfpq_search_host")


def ivfpq_sync_status(ix: IndexHandle) -> int:
    """Synchronises the current stream and returns the device status of the last search."""
    if ix._ws is None:
        return IVFPQ_OK
    return int(load_library().ivfpq_sync_status(ix.handle, ix._ws.data_ptr(), _stream()))


def ivfpq_debug_probes(ix: IndexHandle, queries: torch.Tensor, nprobe: int):
    nq, ws, _, _ = _prep(ix, queries, nprobe, 1)
    pid = torch.empty((nq, nprobe), dtype=torch.int32, device=queries.device)
    pd = torch.empty((nq, nprobe), dtype=torch.float32, device=queries.device)
    _check(load_library().ivfpq_debug_probes(ix.handle, queries.data_ptr(), nq, nprobe, pid.data_ptr(),
                                             pd.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "ivfpq_debug_probes")
    return pid, pd


def ivfpq_debug_search(ix: IndexHandle, queries: torch.Tensor, nprobe: int, k: int,
                       radius: Optional[torch.Tensor] = None, scale: float = 1.0, miss_penalty: float = -1.0,
                       visit_stride: int = 0, score: int = IVFPQ_SCORE_DISTANCE) -> dict:
    """Search with stage dumps (test-only): probe lists, selected-entry masks and,
    per visited point, hit sets, distances and ids."""
    nq, ws, out_d, out_i = _prep(ix, queries, nprobe, k)
    dev = queries.device
    pid = torch.empty((nq, nprobe), dtype=torch.int32, device=dev)
    pd = torch.empty((nq, nprobe), dtype=torch.float32, device=dev)
    masks = torch.zeros((nq, nprobe, ix.nsub, 8), dtype=torch.int32, device=dev)
    vcount = torch.zeros(nq, dtype=torch.int64, device=dev)
    vh = vd = vi = None
    if visit_stride > 0:
        vh = torch.zeros((nq, visit_stride), dtype=torch.int64, device=dev)
        vd = torch.full((nq, visit_stride), float("inf"), dtype=torch.float32, device=dev)
        vi = torch.full((nq, visit_stride), -1, dtype=torch.int32, device=dev)
    rs = None if radius is None else _radius_struct(ix, nq, radius, scale, miss_penalty, score)
    _check(load_library().ivfpq_debug_search(ix.handle, queries.data_ptr(), nq, nprobe,
                                             None if rs is None else ctypes.byref(rs), k,
                                             out_d.data_ptr(), out_i.data_ptr(), pid.data_ptr(), pd.data_ptr(),
                                             masks.data_ptr(), vcount.data_ptr(), visit_stride,
                                             _ptr(vh), _ptr(vd), _ptr(vi), ws.data_ptr(), ws.numel(), _stream()),
           "ivfpq_debug_search")
    res = dict(dist=out_d, ids=out_i, probe_ids=pid, probe_d=pd, masks=masks, visit_count=vcount)
    if visit_stride > 0:
        res.update(visit_hits=vh, visit_dist=vd, visit_ids=vi)
    return res


def ivfpq_probe_static(ix: IndexHandle, queries: torch.Tensor, nprobe: int,
                       out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None):
    """Filtering stage through the entry point that needs no workspace: the distance tile lives
    in an array built into the library (see `ivfpq_probe_static` in ivfpq.h for who needs this
    and for its limits).  Pass `out=(probe_ids, probe_d)` to keep even the outputs out of the
    allocator; otherwise they are new torch tensors.  Returns (probe_ids [nq, nprobe] int32,
    probe_d [nq, nprobe] fp32)."""
    if queries.dtype != torch.float32 or not queries.is_cuda or not queries.is_contiguous() or queries.dim() != 2 \
            or queries.shape[1] != ix.d:
        raise ValueError("queries must be a contiguous fp32 CUDA tensor [nq, d]")
    nq = queries.shape[0]
    if out is None:
        pid = torch.empty((nq, nprobe), dtype=torch.int32, device=queries.device)
        pd = torch.empty((nq, nprobe), dtype=torch.float32, device=queries.device)
    else:
        pid, pd = out
    _check(load_library().ivfpq_probe_static(ix.handle, queries.data_ptr(), nq, nprobe, pid.data_ptr(),
                                             pd.data_ptr(), _stream()), "ivfpq_probe_static")
    return pid, pd


def ivfpq_static_status() -> int:
    """Waits for the current stream and returns IVFPQ_OK or IVFPQ_ERR_DEVICE_FLAG for the most recent
    `ivfpq_probe_static` call on the current device (that call has no workspace to ask)."""
    rc = load_library().ivfpq_static_status(_stream())
    if rc not in (IVFPQ_OK, IVFPQ_ERR_DEVICE_FLAG):
        _check(rc, "ivfpq_static_status")
    return rc


def ivfpq_query_thresholds_knn(ix: IndexHandle, queries: torch.Tensor, kth: int, coef: torch.Tensor,
                               out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Query-specific thresholds [nq, nsub] from the distance to the kth-nearest codebook entry
    (`coef` [nsub, degree + 1] fp32 on the device, ascending powers)."""
    if queries.dtype != torch.float32 or not queries.is_cuda or not queries.is_contiguous() or queries.dim() != 2 \
            or queries.shape[1] != ix.d:
        raise ValueError("queries must be a contiguous fp32 CUDA tensor [nq, d]")
    if coef.dtype != torch.float32 or not coef.is_cuda or not coef.is_contiguous() or coef.dim() != 2 \
            or coef.shape[0] != ix.nsub:
        raise ValueError("coef must be a contiguous fp32 CUDA tensor [nsub, degree + 1]")
    nq = queries.shape[0]
    lib = load_library()
    ws = ix.workspace(int(lib.ivfpq_search_workspace_bytes(ix.handle, nq, 1, 1)))
    if out is None:
        out = torch.empty((nq, ix.nsub), dtype=torch.float32, device=queries.device)
    _check(lib.ivfpq_query_thresholds_knn(ix.handle, queries.data_ptr(), nq, int(kth), coef.shape[1] - 1, coef.data_ptr(),
                                          out.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "ivfpq_query_thresholds_knn")
    return out


class ThresholdModelHandle:
    """Device copies of a dynamic threshold model (an object with grid, degree, density
    [nsub, grid, grid], origin [nsub, 2], inv_cell [nsub, 2], coef [nsub, degree + 1])."""

    def __init__(self, model, device="cuda"):
        f = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(device)
        self.grid, self.degree = int(model.grid), int(model.degree)
        self.density, self.origin, self.inv_cell, self.coef = f(model.density), f(model.origin), f(model.inv_cell), f(model.coef)
        self.struct = ivfpq_threshold_model_t(self.grid, self.degree, self.density.data_ptr(), self.origin.data_ptr(),
                                              self.inv_cell.data_ptr(), self.coef.data_ptr())


def ivfpq_query_thresholds(ix: IndexHandle, queries: torch.Tensor, model: ThresholdModelHandle,
                           out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Query-specific thresholds [nq, nsub] fp32 on the device (the mode-1 radius of the sparse search)."""
    if queries.dtype != torch.float32 or not queries.is_cuda or not queries.is_contiguous() or queries.dim() != 2 \
            or queries.shape[1] != ix.d:
        raise ValueError("queries must be a contiguous fp32 CUDA tensor [nq, d]")
    nq = queries.shape[0]
    if out is None:
        out = torch.empty((nq, ix.nsub), dtype=torch.float32, device=queries.device)
    _check(load_library().ivfpq_query_thresholds(ix.handle, queries.data_ptr(), nq, ctypes.byref(model.struct),
                                                 out.data_ptr(), _stream()), "ivfpq_query_thresholds")
    return out


def ivfpq_entry_stats(ix: IndexHandle, codes: torch.Tensor, queries: torch.Tensor, neighbor_pos: torch.Tensor,
                      rank_hist: Optional[torch.Tensor] = None):
    """Entry usage and locality statistics of each query's neighbours.  `codes` [ntotal, nsub] uint8
    (list-contiguous, on the device), `neighbor_pos` [nq, k] int64 positions into it (-1 = none).
    Returns (usage [nq, nsub] int32, rank_hist [nsub, ksub] int64, accumulated into when given,
    flags: non-zero when an out-of-range position or code was skipped)."""
    nq, k = neighbor_pos.shape
    if codes.dtype != torch.uint8 or not codes.is_cuda or not codes.is_contiguous() or tuple(codes.shape) != (ix.ntotal, ix.nsub):
        raise ValueError("codes must be a contiguous uint8 CUDA tensor [ntotal, nsub]")
    if neighbor_pos.dtype != torch.int64 or not neighbor_pos.is_cuda or not neighbor_pos.is_contiguous():
        raise ValueError("neighbor_pos must be a contiguous int64 CUDA tensor [nq, k]")
    if queries.dtype != torch.float32 or not queries.is_cuda or not queries.is_contiguous() or tuple(queries.shape) != (nq, ix.d):
        raise ValueError("queries must be a contiguous fp32 CUDA tensor [nq, d]")
    dev = queries.device
    usage = torch.empty((nq, ix.nsub), dtype=torch.int32, device=dev)
    if rank_hist is None:
        rank_hist = torch.zeros((ix.nsub, ix.ksub), dtype=torch.int64, device=dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(load_library().ivfpq_entry_stats(ix.handle, codes.data_ptr(), queries.data_ptr(), nq, neighbor_pos.data_ptr(),
                                            k, usage.data_ptr(), rank_hist.data_ptr(), flags.data_ptr(), _stream()),
           "ivfpq_entry_stats")
    return usage, rank_hist, int(flags.item())
