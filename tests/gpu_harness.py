"""Helpers for the GPU parity tests: the same bytes go to the oracle (numpy, host)
and to libgk (torch tensors as device memory), through each side's own API."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2609_39358_b200 as gk


def gk_geom(og: oracle.Geom, flags: int = 0) -> gk.Geom:
    dtype = gk.GK_BF16 if og.elem_bytes == 2 else gk.GK_FP8_E4M3
    if og.head_major:
        flags |= gk.GK_FLAG_HEAD_MAJOR
    return gk.Geom(og.layers, og.kv_heads, og.head_dim, og.page_tokens, dtype, og.scale_kv, flags)


def dev_cache(oc: oracle.Cache, device="cuda") -> gk.Cache:
    """Device copy of an oracle-side cache with identical strides."""
    data = torch.from_numpy(oc.data).to(device)
    scales = None if oc.scales is None else torch.from_numpy(oc.scales).to(device)
    return gk.Cache(data, oc.num_pages, oc.layer_stride, oc.kv_stride, oc.page_stride, scales,
                    oc.s_layer_stride, oc.s_kv_stride, oc.s_page_stride)


def dev_i32(a, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)


def sums_to_dev(sums: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(sums.view(np.int64).copy()).to(device)


def sums_to_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint64)


def gpu_pack(ctx: gk.Context, og: oracle.Geom, dcache: gk.Cache, tables, n_tokens_list):
    """Packs blocks with one batched call; returns [(blob np.uint8, sums np.uint64)], status."""
    jobs, keep = [], []
    for pt, n in zip(tables, n_tokens_list):
        nbytes, npages = oracle.blob_size(og, n)
        blob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        sums = torch.zeros(npages, dtype=torch.int64, device="cuda")
        t = dev_i32(pt)
        keep.append((blob, sums, t))
        jobs.append(gk.Job(blob, sums, t, n))
    status = torch.full((len(jobs),), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_batch(dcache, jobs, status)
    torch.cuda.synchronize()
    return [(b.cpu().numpy(), sums_to_np(s)) for b, s, _ in keep], status.cpu().numpy()


def gpu_restore(ctx: gk.Context, dcache: gk.Cache, ojobs, host_tier: bool = False):
    """Runs gk_restore (or gk_restore_host) on device copies of oracle-side jobs.
    Returns mask, first_bad as numpy."""
    jobs, keep = [], []
    for jb in ojobs:
        if host_tier:
            blob = None if jb.blob is None else torch.from_numpy(jb.blob).pin_memory()
            sums = None if jb.checksums is None else torch.from_numpy(jb.checksums.view(np.int64).copy()).pin_memory()
        else:
            blob = None if jb.blob is None else torch.from_numpy(jb.blob).cuda()
            sums = None if jb.checksums is None else sums_to_dev(jb.checksums)
        pt = dev_i32(jb.page_table)
        keep.append((blob, sums, pt))
        jobs.append(gk.Job(blob, sums, pt, jb.n_tokens))
    mask = torch.full((len(jobs),), 255, dtype=torch.uint8, device="cuda")
    first_bad = torch.full((len(jobs),), -7, dtype=torch.int32, device="cuda")
    if host_tier:
        ctx.gk_restore_host(jobs, dcache, mask, first_bad)
    else:
        ctx.gk_restore(jobs, dcache, mask, first_bad)
    torch.cuda.synchronize()
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    return mask.cpu().numpy(), first_bad.cpu().numpy()


def assert_cache_equal(dcache: gk.Cache, oc: oracle.Cache):
    got = dcache.data.cpu().numpy()
    assert np.array_equal(got, oc.data), f"cache data differs at {np.flatnonzero(got != oc.data)[:8]}"
    if oc.scales is not None:
        gs = dcache.scales.cpu().numpy()
        assert np.array_equal(gs, oc.scales), f"scales differ at {np.flatnonzero(gs != oc.scales)[:8]}"
