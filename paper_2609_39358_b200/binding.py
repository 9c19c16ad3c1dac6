"""ctypes binding of libgk: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/gk.h``.
Tensors are torch tensors used purely as device (or pinned host) memory; the
binding passes their addresses and sizes through and raises ``GkError`` on a
negative return code.  There is no fallback: if ``libgk.so`` is missing, or no
sm_100 device is present, calls fail loudly.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Callable, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("GK_LIB_PATH") or os.path.join(_HERE, "libgk.so")

GK_OK = 0
GK_BF16, GK_FP8_E4M3 = 0, 1
GK_FLAG_SKIP_VERIFY = 1
GK_FLAG_HEAD_MAJOR = 2
GK_FLAG_SINGLE_PASS = 4
JOB_OK, JOB_CHECKSUM, JOB_PAGE_TABLE, JOB_MISSING, JOB_TIMEOUT = 0, 1, 2, 3, 4

EXPORTS = ["gk_blob_size", "gk_ctx_create", "gk_ctx_destroy", "gk_last_error", "gk_pack_batch", "gk_pack",
           "gk_page_checksums", "gk_restore", "gk_restore_host", "gk_get_stats", "gk_ctx_set_tuning", "gk_get_kernel_times",
           "gk_page_checksums_noalloc", "gk_pack_host", "gk_verify", "gk_commit", "gk_restore_stream",
           "gk_fingerprints", "gk_blob_digests", "gk_pack_layerwise", "gk_pack_layerwise_host",
           "gk_restore_layerwise", "gk_restore_layerwise_host", "gk_ctx_reserve", "gk_ctx_clear_error",
           "gk_debug_status", "gk_debug_range_ok", "gk_measure_logic_rate"]


class GkError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        super().__init__(f"{where} failed with code {code}" + (f": {detail}" if detail else ""))
        self.code = code


class CGeom(ctypes.Structure):
    _fields_ = [("layers", ctypes.c_uint32), ("kv_heads", ctypes.c_uint32), ("head_dim", ctypes.c_uint32),
                ("page_tokens", ctypes.c_uint32), ("dtype", ctypes.c_uint32), ("scale_kv", ctypes.c_uint32),
                ("flags", ctypes.c_uint32), ("reserved", ctypes.c_uint32)]


class CCache(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("num_pages", ctypes.c_uint64), ("layer_stride", ctypes.c_uint64),
                ("kv_stride", ctypes.c_uint64), ("page_stride", ctypes.c_uint64), ("scales", ctypes.c_void_p),
                ("s_layer_stride", ctypes.c_uint64), ("s_kv_stride", ctypes.c_uint64),
                ("s_page_stride", ctypes.c_uint64)]


class CJob(ctypes.Structure):
    _fields_ = [("blob", ctypes.c_void_p), ("checksums", ctypes.c_void_p), ("page_table", ctypes.c_void_p),
                ("n_tokens", ctypes.c_uint32), ("request_id", ctypes.c_uint32)]


class CStats(ctypes.Structure):
    _fields_ = [("calls_pack", ctypes.c_uint64), ("calls_restore", ctypes.c_uint64),
                ("calls_restore_host", ctypes.c_uint64), ("jobs", ctypes.c_uint64), ("pages", ctypes.c_uint64),
                ("bytes_blob", ctypes.c_uint64), ("kernels_launched", ctypes.c_uint64),
                ("device_wait_expired", ctypes.c_uint32), ("allocations", ctypes.c_uint32),
                ("calls_restore_stream", ctypes.c_uint64), ("quartet_launches", ctypes.c_uint64)]


class CWindowBlock(ctypes.Structure):
    _fields_ = [("job", ctypes.c_uint32), ("n_tokens", ctypes.c_uint32), ("page_table", ctypes.c_void_p)]


GROUP_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p,
                            ctypes.c_void_p)
WINDOW_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.POINTER(CWindowBlock), ctypes.c_uint32, ctypes.c_void_p,
                             ctypes.c_void_p)


@dataclass(frozen=True)
class WindowBlock:
    """One block of a streaming-restore window, as handed to the consumer."""
    job: int          # index into the call's job list
    n_tokens: int
    page_table: int   # device address of the block's int32 ring page ids


def _marshal_jobs(jobs: Sequence["Job"]):
    arr = (CJob * max(len(jobs), 1))()
    for i, j in enumerate(jobs):
        arr[i] = CJob(_ptr(j.blob), _ptr(j.checksums), _ptr(j.page_table), j.n_tokens, j.request_id)
    return arr


class JobArray:
    """A job list marshalled once, for callers that submit the same jobs repeatedly: every
    method that takes a job list also takes a JobArray.  Keeps the jobs' tensors alive."""

    def __init__(self, jobs: Sequence["Job"]):
        self.jobs = list(jobs)
        self.arr = _marshal_jobs(self.jobs)

    def __len__(self):
        return len(self.jobs)

    def __getitem__(self, i):
        return self.jobs[i]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libgk.so (built in-tree by ``paper_2609_39358_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        # not built yet in this tree: compile it now with nvcc (in-tree); there is no other path
        try:
            from . import build as _build
            _build.build()
        except Exception as e:
            raise ImportError(f"{LIB_PATH} not found and building it failed ({e}); build it with "
                              "`python -m paper_2609_39358_b200.build` (there is no CPU fallback)") from e
    L = ctypes.CDLL(LIB_PATH)
    vp, u32, u64p = ctypes.c_void_p, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint64)
    L.gk_blob_size.restype = ctypes.c_int
    L.gk_blob_size.argtypes = [ctypes.POINTER(CGeom), u32, u64p, ctypes.POINTER(u32)]
    L.gk_ctx_create.restype = ctypes.c_int
    L.gk_ctx_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(CGeom), ctypes.c_int]
    L.gk_ctx_destroy.restype = ctypes.c_int
    L.gk_ctx_destroy.argtypes = [vp]
    L.gk_last_error.restype = ctypes.c_char_p
    L.gk_last_error.argtypes = [vp]
    L.gk_pack_batch.restype = ctypes.c_int
    L.gk_pack_batch.argtypes = [vp, ctypes.POINTER(CCache), ctypes.POINTER(CJob), u32, vp, vp]
    L.gk_pack_host.restype = ctypes.c_int
    L.gk_pack_host.argtypes = [vp, ctypes.POINTER(CCache), ctypes.POINTER(CJob), u32, vp, vp]
    L.gk_pack.restype = ctypes.c_int
    L.gk_pack.argtypes = [vp, ctypes.POINTER(CCache), vp, u32, vp, vp, vp, vp]
    L.gk_page_checksums.restype = ctypes.c_int
    L.gk_page_checksums.argtypes = [vp, vp, u32, vp, vp]
    L.gk_restore.restype = ctypes.c_int
    L.gk_restore.argtypes = [vp, ctypes.POINTER(CJob), u32, ctypes.POINTER(CCache), vp, vp, vp]
    L.gk_verify.restype = ctypes.c_int
    L.gk_verify.argtypes = [vp, ctypes.POINTER(CJob), u32, ctypes.POINTER(CCache), vp, vp, vp]
    L.gk_commit.restype = ctypes.c_int
    L.gk_commit.argtypes = [vp, ctypes.POINTER(CJob), u32, ctypes.POINTER(CCache), vp, vp]
    L.gk_restore_host.restype = ctypes.c_int
    L.gk_restore_host.argtypes = [vp, ctypes.POINTER(CJob), u32, ctypes.POINTER(CCache), vp, vp, vp]
    L.gk_restore_stream.restype = ctypes.c_int
    L.gk_restore_stream.argtypes = [vp, ctypes.POINTER(CJob), u32, ctypes.POINTER(CCache), vp, vp, WINDOW_FN, vp, vp]
    for name in ("gk_pack_layerwise", "gk_pack_layerwise_host"):
        getattr(L, name).restype = ctypes.c_int
        getattr(L, name).argtypes = [vp, u32, ctypes.POINTER(CCache), ctypes.POINTER(CJob), u32, vp, vp]
    for name in ("gk_restore_layerwise", "gk_restore_layerwise_host"):
        getattr(L, name).restype = ctypes.c_int
        getattr(L, name).argtypes = [vp, u32, ctypes.POINTER(CJob), u32, ctypes.POINTER(CCache), vp, vp, vp, GROUP_FN,
                                     vp, vp]
    L.gk_fingerprints.restype = ctypes.c_int
    L.gk_fingerprints.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_int32), u32, ctypes.c_char_p, ctypes.c_char_p, vp, vp]
    L.gk_blob_digests.restype = ctypes.c_int
    L.gk_blob_digests.argtypes = [vp, ctypes.POINTER(CJob), u32, vp, vp, vp, vp]
    L.gk_get_stats.restype = ctypes.c_int
    L.gk_get_stats.argtypes = [vp, ctypes.POINTER(CStats)]
    L.gk_get_kernel_times.restype = ctypes.c_int
    L.gk_get_kernel_times.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_uint64)]
    L.gk_page_checksums_noalloc.restype = ctypes.c_int
    L.gk_page_checksums_noalloc.argtypes = [ctypes.POINTER(CGeom), vp, u32, vp, ctypes.c_int, vp]
    L.gk_ctx_set_tuning.restype = ctypes.c_int
    L.gk_ctx_set_tuning.argtypes = [vp, ctypes.c_char_p, u32]
    L.gk_ctx_reserve.restype = ctypes.c_int
    L.gk_ctx_reserve.argtypes = [vp, u32, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64]
    L.gk_ctx_clear_error.restype = ctypes.c_int
    L.gk_ctx_clear_error.argtypes = [vp, vp]
    L.gk_measure_logic_rate.restype = ctypes.c_int
    L.gk_measure_logic_rate.argtypes = [vp, ctypes.POINTER(ctypes.c_double), vp]
    L.gk_debug_status.restype = ctypes.c_int
    L.gk_debug_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    L.gk_debug_range_ok.restype = ctypes.c_int
    L.gk_debug_range_ok.argtypes = [ctypes.c_uint64] * 4
    _lib = L
    return L


@dataclass(frozen=True)
class Geom:
    layers: int
    kv_heads: int
    head_dim: int
    page_tokens: int
    dtype: int = GK_BF16
    scale_kv: int = 0
    flags: int = 0

    def c(self) -> CGeom:
        return CGeom(self.layers, self.kv_heads, self.head_dim, self.page_tokens, self.dtype, self.scale_kv,
                     self.flags, 0)


@dataclass
class Cache:
    """A paged cache: a uint8 device tensor plus byte strides (see gk.h)."""
    data: torch.Tensor
    num_pages: int
    layer_stride: int
    kv_stride: int
    page_stride: int
    scales: Optional[torch.Tensor] = None
    s_layer_stride: int = 0
    s_kv_stride: int = 0
    s_page_stride: int = 0

    def c(self) -> CCache:
        return CCache(self.data.data_ptr(), self.num_pages, self.layer_stride, self.kv_stride, self.page_stride,
                      0 if self.scales is None else self.scales.data_ptr(), self.s_layer_stride,
                      self.s_kv_stride, self.s_page_stride)


@dataclass
class Job:
    blob: Optional[torch.Tensor]        # uint8; device (pinned host for restore_host); None = missing
    checksums: Optional[torch.Tensor]   # int64/uint64 storage of P entries; None = missing
    page_table: torch.Tensor            # int32, device
    n_tokens: int
    request_id: int = 0


def _ptr(t) -> int:
    """Address of a tensor's storage; an int is taken as a raw address, None as NULL."""
    if t is None:
        return 0
    return t if isinstance(t, int) else t.data_ptr()


def _stream_handle(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def gk_blob_size(geom: Geom, n_tokens: int) -> tuple[int, int]:
    nb, npg = ctypes.c_uint64(0), ctypes.c_uint32(0)
    cg = geom.c()
    rc = load_library().gk_blob_size(ctypes.byref(cg), n_tokens, ctypes.byref(nb), ctypes.byref(npg))
    if rc != GK_OK:
        raise GkError(rc, "gk_blob_size")
    return int(nb.value), int(npg.value)


GK_NOALLOC_MAX_PAGES = 8192
GK_NOALLOC_MAX_PAGE_TOKENS = 256


def gk_debug_range_ok(addr: int, nbytes: int, base: int, extent: int) -> bool:
    return bool(load_library().gk_debug_range_ok(addr, nbytes, base, extent))


def gk_page_checksums_noalloc(geom: Geom, blob: torch.Tensor, n_tokens: int, checksums: torch.Tensor,
                              device: int = 0, stream=None) -> None:
    """Page checksums of a device blob through the entry point that allocates
    nothing and needs no context (see gk.h: fixed scratch, at most
    GK_NOALLOC_MAX_PAGES pages per call, calls on one device must not overlap)."""
    cg = geom.c()
    sh = 0 if stream is None and not torch.cuda.is_available() else _stream_handle(stream)
    rc = load_library().gk_page_checksums_noalloc(ctypes.byref(cg), _ptr(blob), n_tokens, _ptr(checksums),
                                                  device, sh)
    if rc != GK_OK:
        raise GkError(rc, "gk_page_checksums_noalloc")


class Context:
    """Owns a ``gk_ctx``.  One context per concurrently used stream."""

    def __init__(self, geom: Geom, device: int = 0):
        self._lib = load_library()
        self.geom = geom
        self.device = device
        h = ctypes.c_void_p(0)
        cg = geom.c()
        rc = self._lib.gk_ctx_create(ctypes.byref(h), ctypes.byref(cg), device)
        if rc != GK_OK:
            raise GkError(rc, "gk_ctx_create")
        self._h = h
        # GK_TUNING="key=value,key=value": tuning keys applied to every new context of the process
        # (gk_ctx_set_tuning; e.g. quad=2 makes every pack and fused restore use page quartets)
        for kv in filter(None, os.environ.get("GK_TUNING", "").split(",")):
            key, _, value = kv.partition("=")
            rc = self._lib.gk_ctx_set_tuning(self._h, key.strip().encode(), int(value))
            if rc != GK_OK:
                raise GkError(rc, f"GK_TUNING: {kv}")

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
        return False

    def close(self):
        if getattr(self, "_h", None):
            status = self.gk_debug_status()
            self._lib.gk_ctx_destroy(self._h)
            self._h = None
            if status is not None and status[0] != 0:
                raise GkError(-8, "bounds-checked build",
                              f"an access outside its object was refused: kind/role {status[0]:#x}, offset "
                              f"{status[1] | (status[2] << 32)}, {status[3]} bytes")

    def gk_debug_status(self):
        """(kind/role, offset low, offset high, bytes) of the first refused access with the bounds-checked
        library (all zero if there was none); None with the ordinary library."""
        out = (ctypes.c_uint32 * 4)()
        rc = self._lib.gk_debug_status(self._h, out)
        return None if rc != GK_OK else tuple(int(x) for x in out)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != GK_OK:
            raise GkError(rc, where, self._lib.gk_last_error(self._h).decode(errors="replace"))

    def _jobs(self, jobs):
        return jobs.arr if isinstance(jobs, JobArray) else _marshal_jobs(jobs)

    def set_tuning(self, key: str, value: int):
        self._check(self._lib.gk_ctx_set_tuning(self._h, key.encode(), value), "gk_ctx_set_tuning")

    def gk_ctx_reserve(self, max_jobs: int, max_pages: int, num_pages: int, max_host_batch_bytes: int = 0):
        self._check(self._lib.gk_ctx_reserve(self._h, max_jobs, max_pages, num_pages, max_host_batch_bytes),
                    "gk_ctx_reserve")

    def gk_ctx_clear_error(self, stream=None):
        self._check(self._lib.gk_ctx_clear_error(self._h, _stream_handle(stream)), "gk_ctx_clear_error")

    def gk_pack_batch(self, src: Cache, jobs: Sequence[Job], status: Optional[torch.Tensor] = None, stream=None):
        cc = src.c()
        self._check(self._lib.gk_pack_batch(self._h, ctypes.byref(cc), self._jobs(jobs), len(jobs), _ptr(status),
                                            _stream_handle(stream)), "gk_pack_batch")

    def gk_pack_host(self, src: Cache, jobs: Sequence[Job], status: Optional[torch.Tensor] = None, stream=None):
        cc = src.c()
        self._check(self._lib.gk_pack_host(self._h, ctypes.byref(cc), self._jobs(jobs), len(jobs), _ptr(status),
                                           _stream_handle(stream)), "gk_pack_host")

    def gk_pack(self, src: Cache, page_table: torch.Tensor, n_tokens: int, blob: torch.Tensor,
                checksums: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None):
        cc = src.c()
        self._check(self._lib.gk_pack(self._h, ctypes.byref(cc), _ptr(page_table), n_tokens, _ptr(blob),
                                      _ptr(checksums), _ptr(status), _stream_handle(stream)), "gk_pack")

    def gk_page_checksums(self, blob: torch.Tensor, n_tokens: int, checksums: torch.Tensor, stream=None):
        self._check(self._lib.gk_page_checksums(self._h, _ptr(blob), n_tokens, _ptr(checksums),
                                                _stream_handle(stream)), "gk_page_checksums")

    def gk_restore(self, jobs: Sequence[Job], dst: Cache, mask: torch.Tensor, first_bad_page: torch.Tensor,
                   stream=None):
        cc = dst.c()
        self._check(self._lib.gk_restore(self._h, self._jobs(jobs), len(jobs), ctypes.byref(cc), _ptr(mask),
                                         _ptr(first_bad_page), _stream_handle(stream)), "gk_restore")

    def gk_verify(self, jobs: Sequence[Job], dst: Cache, mask: torch.Tensor, first_bad_page: torch.Tensor,
                  stream=None):
        cc = dst.c()
        self._check(self._lib.gk_verify(self._h, self._jobs(jobs), len(jobs), ctypes.byref(cc), _ptr(mask),
                                        _ptr(first_bad_page), _stream_handle(stream)), "gk_verify")

    def gk_commit(self, jobs: Sequence[Job], dst: Cache, mask: torch.Tensor, stream=None):
        cc = dst.c()
        self._check(self._lib.gk_commit(self._h, self._jobs(jobs), len(jobs), ctypes.byref(cc), _ptr(mask),
                                        _stream_handle(stream)), "gk_commit")

    def gk_restore_host(self, jobs: Sequence[Job], dst: Cache, mask: torch.Tensor, first_bad_page: torch.Tensor,
                        stream=None):
        cc = dst.c()
        self._check(self._lib.gk_restore_host(self._h, self._jobs(jobs), len(jobs), ctypes.byref(cc), _ptr(mask),
                                              _ptr(first_bad_page), _stream_handle(stream)), "gk_restore_host")

    def gk_restore_stream(self, jobs: Sequence[Job], ring: Cache, mask: torch.Tensor, first_bad_page: torch.Tensor,
                          consume: Optional[Callable] = None, stream=None):
        """``consume(blocks: list[WindowBlock], stream_handle: int)`` runs on the host after each window has
        been enqueued; it may only enqueue work on that stream.  An exception it raises is re-raised here
        after the call has returned (the remaining windows still run)."""
        cc = ring.c()
        raised = []

        def _cb(_user, blocks, n, _mask, st):
            if consume is None:
                return
            try:
                consume([WindowBlock(blocks[i].job, blocks[i].n_tokens, blocks[i].page_table or 0) for i in range(n)],
                        st or 0)
            except BaseException as e:  # must not unwind through the C frames
                raised.append(e)

        cb = WINDOW_FN(_cb)
        rc = self._lib.gk_restore_stream(self._h, self._jobs(jobs), len(jobs), ctypes.byref(cc), _ptr(mask),
                                         _ptr(first_bad_page), cb, None, _stream_handle(stream))
        if raised:
            raise raised[0]
        self._check(rc, "gk_restore_stream")

    def gk_pack_layerwise(self, n_groups: int, src: Cache, jobs, status: Optional[torch.Tensor] = None, stream=None,
                          host: bool = False):
        """The context's geometry describes one layer group; ``src`` holds n_groups of them."""
        cc = src.c()
        fn = self._lib.gk_pack_layerwise_host if host else self._lib.gk_pack_layerwise
        self._check(fn(self._h, n_groups, ctypes.byref(cc), self._jobs(jobs), len(jobs), _ptr(status),
                       _stream_handle(stream)), "gk_pack_layerwise")

    def gk_restore_layerwise(self, n_groups: int, jobs, dst: Cache, mask: torch.Tensor, first_bad_page: torch.Tensor,
                             group_mask: Optional[torch.Tensor] = None, on_group: Optional[Callable] = None,
                             stream=None, host: bool = False):
        """``on_group(group, first_layer, n_layers, stream_handle)`` runs on the host after the work of
        each group has been enqueued; it may only enqueue work on that stream."""
        cc = dst.c()
        raised = []

        def _cb(_user, group, first_layer, n_layers, _gm, st):
            if on_group is None:
                return
            try:
                on_group(int(group), int(first_layer), int(n_layers), st or 0)
            except BaseException as e:  # must not unwind through the C frames
                raised.append(e)

        cb = GROUP_FN(_cb)
        fn = self._lib.gk_restore_layerwise_host if host else self._lib.gk_restore_layerwise
        rc = fn(self._h, n_groups, self._jobs(jobs), len(jobs), ctypes.byref(cc), _ptr(mask), _ptr(first_bad_page),
                _ptr(group_mask), cb, None, _stream_handle(stream))
        if raised:
            raise raised[0]
        self._check(rc, "gk_restore_layerwise")

    def gk_fingerprints(self, data: torch.Tensor, offsets: torch.Tensor, parent: Optional[Sequence[int]],
                        model: bytes, tenant: bytes, keys: torch.Tensor, stream=None):
        """data: device bytes; offsets: device int64/uint64 [n+1]; parent: host ints or None; keys: device uint8 [n, 32]."""
        n = offsets.numel() - 1
        assert len(model) == 32 and len(tenant) == 32 and keys.numel() >= 32 * n
        par = None
        if parent is not None:
            assert len(parent) == n
            par = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in parent])
        self._check(self._lib.gk_fingerprints(self._h, _ptr(data), _ptr(offsets), par, n, bytes(model), bytes(tenant),
                                              _ptr(keys), _stream_handle(stream)), "gk_fingerprints")

    def gk_blob_digests(self, jobs: Sequence[Job], keys: torch.Tensor, digests: torch.Tensor,
                        page_digests: Optional[torch.Tensor] = None, stream=None):
        self._check(self._lib.gk_blob_digests(self._h, self._jobs(jobs), len(jobs), _ptr(keys), _ptr(digests),
                                              _ptr(page_digests), _stream_handle(stream)), "gk_blob_digests")

    def gk_measure_logic_rate(self, stream=None) -> float:
        """Three-input logic operations per second (lanes x instructions) of this GPU, measured."""
        out = ctypes.c_double(0.0)
        self._check(self._lib.gk_measure_logic_rate(self._h, ctypes.byref(out), _stream_handle(stream)),
                    "gk_measure_logic_rate")
        return float(out.value)

    def gk_get_kernel_times(self) -> dict:
        """{'verify'|'pack'|'commit'|'restore': (ms, launches)} since the previous call (needs tuning key profile=1)."""
        ms = (ctypes.c_double * 4)()
        n = (ctypes.c_uint64 * 4)()
        self._check(self._lib.gk_get_kernel_times(self._h, ms, n), "gk_get_kernel_times")
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(("verify", "pack", "commit", "restore"))}

    def gk_get_stats(self) -> dict:
        st = CStats()
        self._check(self._lib.gk_get_stats(self._h, ctypes.byref(st)), "gk_get_stats")
        return {name: int(getattr(st, name)) for name, _ in CStats._fields_ }
