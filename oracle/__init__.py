"""CPU oracle for the KV block save/restore path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``gk_oracle.c`` (plain C, compiled with gcc).  The
oracle defines what pack / restore must produce, byte for byte; see the header
of ``gk_oracle.h`` for the passages of the paper it follows (Section 2.2 for
save, load, check-on-load and the recompute-on-any-failure rule; Table 1 for
bit-identical restoration).  It imports nothing from the CUDA package and the
CUDA package imports nothing from here.  Only tests, the smoke check and the
benchmark's CPU-baseline leg may use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgk_oracle.so")
_SRCS = [os.path.join(_HERE, "gk_oracle.c"), os.path.join(_HERE, "gk_sha256_oracle.c")]
_HDRS = [os.path.join(_HERE, "gk_oracle.h"), os.path.join(_HERE, "gk_sha256_oracle.h")]

CODE_OK, CODE_CHECKSUM, CODE_PAGE_TABLE, CODE_MISSING = 0, 1, 2, 3
FLAG_SKIP_VERIFY = 1
FLAG_SINGLE_PASS = 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB_PATH)
             or os.path.getmtime(_LIB_PATH) < max(os.path.getmtime(f) for f in _SRCS + _HDRS))
    if force or stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fPIC", "-shared",
                               "-o", tmp] + _SRCS)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


class _CGeom(ctypes.Structure):
    _fields_ = [("layers", ctypes.c_uint32), ("kv_heads", ctypes.c_uint32),
                ("head_dim", ctypes.c_uint32), ("page_tokens", ctypes.c_uint32),
                ("elem_bytes", ctypes.c_uint32), ("scale_kv", ctypes.c_uint32),
                ("head_major", ctypes.c_uint32)]


class _CCache(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("num_pages", ctypes.c_uint64),
                ("layer_stride", ctypes.c_uint64), ("kv_stride", ctypes.c_uint64),
                ("page_stride", ctypes.c_uint64), ("scales", ctypes.c_void_p),
                ("s_layer_stride", ctypes.c_uint64), ("s_kv_stride", ctypes.c_uint64),
                ("s_page_stride", ctypes.c_uint64)]


class _CJob(ctypes.Structure):
    _fields_ = [("blob", ctypes.c_void_p), ("checksums", ctypes.c_void_p),
                ("page_table", ctypes.c_void_p), ("n_tokens", ctypes.c_uint32)]


_WINDOW_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                              ctypes.POINTER(ctypes.c_uint32))

_GROUP_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32)

_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.ok_crc64_bitwise.restype = ctypes.c_uint64
        L.ok_crc64_bitwise.argtypes = [ctypes.c_void_p, ctypes.c_size_t]
        L.ok_crc64.restype = ctypes.c_uint64
        L.ok_crc64.argtypes = [ctypes.c_void_p, ctypes.c_size_t]
        L.ok_crc64_continue.restype = ctypes.c_uint64
        L.ok_crc64_continue.argtypes = [ctypes.c_uint64, ctypes.c_void_p, ctypes.c_size_t]
        L.ok_blob_size.restype = ctypes.c_int
        L.ok_blob_size.argtypes = [ctypes.POINTER(_CGeom), ctypes.c_uint32,
                                   ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint32)]
        L.ok_record_bytes.restype = ctypes.c_uint64
        L.ok_record_bytes.argtypes = [ctypes.POINTER(_CGeom), ctypes.c_uint32, ctypes.c_uint32]
        L.ok_record_offset.restype = ctypes.c_uint64
        L.ok_record_offset.argtypes = [ctypes.POINTER(_CGeom), ctypes.c_uint32]
        L.ok_pack.restype = ctypes.c_int
        L.ok_pack.argtypes = [ctypes.POINTER(_CGeom), ctypes.POINTER(_CCache), ctypes.c_void_p,
                              ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p,
                              ctypes.POINTER(ctypes.c_int32)]
        L.ok_restore.restype = None
        L.ok_restore.argtypes = [ctypes.POINTER(_CGeom), ctypes.POINTER(_CCache),
                                 ctypes.POINTER(_CJob), ctypes.c_uint32, ctypes.c_uint32,
                                 ctypes.c_void_p, ctypes.c_void_p]
        L.ok_restore_stream.restype = ctypes.c_int
        L.ok_restore_stream.argtypes = [ctypes.POINTER(_CGeom), ctypes.POINTER(_CCache),
                                        ctypes.POINTER(_CJob), ctypes.c_uint32, ctypes.c_uint32,
                                        ctypes.c_void_p, ctypes.c_void_p, _WINDOW_FN, ctypes.c_void_p]
        L.ok_pack_layerwise.restype = ctypes.c_int
        L.ok_pack_layerwise.argtypes = [ctypes.POINTER(_CGeom), ctypes.c_uint32, ctypes.POINTER(_CCache),
                                        ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.POINTER(ctypes.c_int32)]
        L.ok_restore_layerwise.restype = None
        L.ok_restore_layerwise.argtypes = [ctypes.POINTER(_CGeom), ctypes.c_uint32, ctypes.POINTER(_CCache),
                                           ctypes.POINTER(_CJob), ctypes.c_uint32, ctypes.c_uint32,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, _GROUP_FN,
                                           ctypes.c_void_p]
        L.ok_sha256.restype = None
        L.ok_sha256.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.ok_sha256_constants.restype = None
        L.ok_sha256_constants.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.ok_fingerprints.restype = ctypes.c_int
        L.ok_fingerprints.argtypes = [ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.ok_blob_digest.restype = None
        L.ok_blob_digest.argtypes = [ctypes.POINTER(_CGeom), ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_void_p]
        _lib = L
    return _lib


def _as_u8(data) -> np.ndarray:
    if isinstance(data, (bytes, bytearray, memoryview)):
        return np.frombuffer(bytes(data), dtype=np.uint8)
    arr = np.ascontiguousarray(data)
    return arr.view(np.uint8).reshape(-1)


def crc64_bitwise(data) -> int:
    a = _as_u8(data)
    return int(lib().ok_crc64_bitwise(a.ctypes.data, a.size))


def crc64(data) -> int:
    a = _as_u8(data)
    return int(lib().ok_crc64(a.ctypes.data, a.size))


def crc64_continue(crc_so_far: int, data) -> int:
    a = _as_u8(data)
    return int(lib().ok_crc64_continue(ctypes.c_uint64(crc_so_far), a.ctypes.data, a.size))


@dataclass(frozen=True)
class Geom:
    """Cache geometry as the oracle sees it (element size in bytes, not a dtype tag)."""
    layers: int
    kv_heads: int
    head_dim: int
    page_tokens: int
    elem_bytes: int = 2
    scale_kv: int = 0
    head_major: int = 0

    def c(self) -> _CGeom:
        return _CGeom(self.layers, self.kv_heads, self.head_dim, self.page_tokens,
                      self.elem_bytes, self.scale_kv, self.head_major)


@dataclass
class Cache:
    """A paged cache held in host memory as flat byte arrays plus byte strides."""
    data: np.ndarray                  # uint8, flat
    num_pages: int
    layer_stride: int
    kv_stride: int
    page_stride: int
    scales: Optional[np.ndarray] = None   # uint8, flat (fp32 values as bytes)
    s_layer_stride: int = 0
    s_kv_stride: int = 0
    s_page_stride: int = 0

    def c(self) -> _CCache:
        assert self.data.dtype == np.uint8 and self.data.flags.c_contiguous
        sp = 0
        if self.scales is not None:
            assert self.scales.dtype == np.uint8 and self.scales.flags.c_contiguous
            sp = self.scales.ctypes.data
        return _CCache(self.data.ctypes.data, self.num_pages, self.layer_stride, self.kv_stride,
                       self.page_stride, sp, self.s_layer_stride, self.s_kv_stride,
                       self.s_page_stride)


def blob_size(g: Geom, n_tokens: int) -> tuple[int, int]:
    nb, npg = ctypes.c_uint64(0), ctypes.c_uint32(0)
    cg = g.c()
    rc = lib().ok_blob_size(ctypes.byref(cg), n_tokens, ctypes.byref(nb), ctypes.byref(npg))
    if rc != 0:
        raise ValueError("bad geometry or n_tokens == 0")
    return int(nb.value), int(npg.value)


def record_bytes(g: Geom, n_tokens: int, p: int) -> int:
    cg = g.c()
    return int(lib().ok_record_bytes(ctypes.byref(cg), n_tokens, p))


def record_offset(g: Geom, p: int) -> int:
    cg = g.c()
    return int(lib().ok_record_offset(ctypes.byref(cg), p))


def pack(g: Geom, src: Cache, page_table, n_tokens: int):
    """Returns (blob uint8[blob_bytes], checksums uint64[P], code, bad_index)."""
    nbytes, npages = blob_size(g, n_tokens)
    pt = np.ascontiguousarray(page_table, dtype=np.int32)
    assert pt.size >= npages
    blob = np.zeros(nbytes, dtype=np.uint8)
    sums = np.zeros(npages, dtype=np.uint64)
    bad = ctypes.c_int32(-1)
    cg, cc = g.c(), src.c()
    code = lib().ok_pack(ctypes.byref(cg), ctypes.byref(cc), pt.ctypes.data, n_tokens,
                         blob.ctypes.data, sums.ctypes.data, ctypes.byref(bad))
    return blob, sums, int(code), int(bad.value)


@dataclass
class Job:
    blob: Optional[np.ndarray]        # uint8 flat, or None for a missing record
    checksums: Optional[np.ndarray]   # uint64[P], or None
    page_table: np.ndarray            # int32[P]
    n_tokens: int


def _c_jobs(jobs: Sequence[Job], with_tables: bool = True):
    n = len(jobs)
    arr = (_CJob * max(n, 1))()
    keep = []
    for i, jb in enumerate(jobs):
        pt = np.ascontiguousarray(jb.page_table if with_tables else np.zeros(1), dtype=np.int32)
        keep.append(pt)
        bp = cp = 0
        if jb.blob is not None:
            b = jb.blob
            assert b.dtype == np.uint8 and b.flags.c_contiguous
            bp = b.ctypes.data
        if jb.checksums is not None:
            c = np.ascontiguousarray(jb.checksums, dtype=np.uint64)
            keep.append(c)
            cp = c.ctypes.data
        arr[i] = _CJob(bp, cp, pt.ctypes.data, jb.n_tokens)
    return arr, keep


def restore(g: Geom, dst: Cache, jobs: Sequence[Job], flags: int = 0):
    """Mutates ``dst``; returns (mask uint8[n_jobs], first_bad int32[n_jobs])."""
    n = len(jobs)
    arr, keep = _c_jobs(jobs)
    mask = np.zeros(n, dtype=np.uint8)
    first_bad = np.zeros(n, dtype=np.int32)
    cg, cc = g.c(), dst.c()
    lib().ok_restore(ctypes.byref(cg), ctypes.byref(cc), arr, n, flags,
                     mask.ctypes.data, first_bad.ctypes.data)
    return mask, first_bad


def restore_stream(g: Geom, ring: Cache, jobs: Sequence[Job], consume=None, flags: int = 0):
    """Streams ``jobs`` (their page tables are ignored) through ``ring`` window by window.
    ``consume(first_job, n_jobs, first_pages)`` runs after each window, while the window's
    pages are still in ``ring``.  Returns (mask, first_bad), or raises ValueError if one job
    alone does not fit the ring."""
    n = len(jobs)
    arr, keep = _c_jobs(jobs, with_tables=False)
    mask = np.zeros(n, dtype=np.uint8)
    first_bad = np.zeros(n, dtype=np.int32)

    def _cb(_user, first_job, count, first_page):
        if consume is not None:
            consume(int(first_job), int(count), [int(first_page[i]) for i in range(count)])

    cb = _WINDOW_FN(_cb)
    cg, cc = g.c(), ring.c()
    rc = lib().ok_restore_stream(ctypes.byref(cg), ctypes.byref(cc), arr, n, flags,
                                 mask.ctypes.data, first_bad.ctypes.data, cb, None)
    if rc != 0:
        raise ValueError("a job has more pages than the ring")
    return mask, first_bad


def pack_layerwise(g: Geom, n_groups: int, src: Cache, page_table, n_tokens: int):
    """``g`` describes one layer group; ``src`` holds n_groups * g.layers layers.
    Returns (blob, checksums uint64[n_groups * P], code, bad_index)."""
    group_bytes, npages = blob_size(g, n_tokens)
    pt = np.ascontiguousarray(page_table, dtype=np.int32)
    blob = np.zeros(n_groups * group_bytes, dtype=np.uint8)
    sums = np.zeros(n_groups * npages, dtype=np.uint64)
    bad = ctypes.c_int32(-1)
    cg, cc = g.c(), src.c()
    code = lib().ok_pack_layerwise(ctypes.byref(cg), n_groups, ctypes.byref(cc), pt.ctypes.data, n_tokens,
                                   blob.ctypes.data, sums.ctypes.data, ctypes.byref(bad))
    return blob, sums, int(code), int(bad.value)


def restore_layerwise(g: Geom, n_groups: int, dst: Cache, jobs: Sequence[Job], consume=None, flags: int = 0):
    """Mutates ``dst``; ``consume(group, first_layer, n_layers)`` runs after each group.
    Returns (mask, first_bad, group_mask uint8[n_groups, n_jobs])."""
    n = len(jobs)
    arr, keep = _c_jobs(jobs)
    mask = np.zeros(n, dtype=np.uint8)
    first_bad = np.zeros(n, dtype=np.int32)
    group_mask = np.zeros((n_groups, max(n, 1)), dtype=np.uint8)

    def _cb(_user, group, first_layer, n_layers):
        if consume is not None:
            consume(int(group), int(first_layer), int(n_layers))

    cb = _GROUP_FN(_cb)
    cg, cc = g.c(), dst.c()
    lib().ok_restore_layerwise(ctypes.byref(cg), n_groups, ctypes.byref(cc), arr, n, flags, mask.ctypes.data,
                               first_bad.ctypes.data, group_mask.ctypes.data, cb, None)
    return mask, first_bad, group_mask[:, :n]


# ---------------------------------------------------------------------------
# fingerprints and blob digests (gk_sha256_oracle.c)
# ---------------------------------------------------------------------------
DIGEST_CHUNK = 4096


def sha256(data) -> bytes:
    a = _as_u8(data)
    out = np.zeros(32, dtype=np.uint8)
    lib().ok_sha256(a.ctypes.data if a.size else None, a.size, out.ctypes.data)
    return out.tobytes()


def sha256_constants():
    k = np.zeros(64, dtype=np.uint32)
    h0 = np.zeros(8, dtype=np.uint32)
    lib().ok_sha256_constants(k.ctypes.data, h0.ctypes.data)
    return k, h0


def fingerprints(data, offsets, parent, model: bytes, tenant: bytes) -> np.ndarray:
    """Keys (uint8[n, 32]) of the messages data[offsets[i]:offsets[i+1]]; parent may be None."""
    d = _as_u8(data)
    off = np.ascontiguousarray(offsets, dtype=np.uint64)
    n = off.size - 1
    par = None if parent is None else np.ascontiguousarray(parent, dtype=np.int32)
    m, t = _as_u8(model), _as_u8(tenant)
    assert m.size == 32 and t.size == 32 and (par is None or par.size == n)
    keys = np.zeros((max(n, 1), 32), dtype=np.uint8)
    rc = lib().ok_fingerprints(n, d.ctypes.data if d.size else None, off.ctypes.data,
                               None if par is None else par.ctypes.data, m.ctypes.data, t.ctypes.data,
                               keys.ctypes.data)
    if rc != 0:
        raise ValueError("parent[i] must be < i")
    return keys[:n]


def blob_digest(g: Geom, blob: np.ndarray, n_tokens: int, key: bytes):
    """Returns (digest bytes[32], page digests uint8[P, 32])."""
    nbytes, npages = blob_size(g, n_tokens)
    b = _as_u8(blob)
    assert b.size == nbytes
    k = _as_u8(key)
    assert k.size == 32
    pages = np.zeros((npages, 32), dtype=np.uint8)
    out = np.zeros(32, dtype=np.uint8)
    cg = g.c()
    lib().ok_blob_digest(ctypes.byref(cg), b.ctypes.data, n_tokens, k.ctypes.data, pages.ctypes.data,
                         out.ctypes.data)
    return out.tobytes(), pages
