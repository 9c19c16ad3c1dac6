"""Shared test plumbing: cache descriptors for the oracle side, small utilities."""
from __future__ import annotations

import numpy as np

import oracle
import synth


def oracle_geom(w: synth.Workload) -> oracle.Geom:
    return oracle.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, w.elem_bytes, w.scale_kv)


def slab_bytes(g: oracle.Geom) -> int:
    return g.page_tokens * g.kv_heads * g.head_dim * g.elem_bytes


def layer_major_strides(g: oracle.Geom, num_pages: int):
    """[L][2][N][T][H][D]: (layer_stride, kv_stride, page_stride) in bytes."""
    s = slab_bytes(g)
    return 2 * num_pages * s, num_pages * s, s


def page_major_strides(g: oracle.Geom):
    """[N][L][2][T][H][D]"""
    s = slab_bytes(g)
    return 2 * s, s, 2 * g.layers * s


def cache_bytes(g: oracle.Geom, num_pages: int) -> int:
    return 2 * g.layers * num_pages * slab_bytes(g)


def scale_bytes(g: oracle.Geom, num_pages: int) -> int:
    return g.layers * g.scale_kv * num_pages * g.kv_heads * 4


def scale_strides(g: oracle.Geom, num_pages: int):
    """[L][scale_kv][N][H] fp32: (layer, kv, page) strides in bytes."""
    h4 = g.kv_heads * 4
    return g.scale_kv * num_pages * h4, num_pages * h4, h4


def make_cache(g: oracle.Geom, num_pages: int, data: np.ndarray, scales: np.ndarray | None = None,
               layout: str = "layer_major") -> oracle.Cache:
    assert data.dtype == np.uint8 and data.size == cache_bytes(g, num_pages)
    if layout == "layer_major":
        ls, ks, ps = layer_major_strides(g, num_pages)
    else:
        ls, ks, ps = page_major_strides(g)
    c = oracle.Cache(data, num_pages, ls, ks, ps)
    if g.scale_kv:
        assert scales is not None and scales.dtype == np.uint8 and scales.size == scale_bytes(g, num_pages)
        c.scales = scales
        c.s_layer_stride, c.s_kv_stride, c.s_page_stride = scale_strides(g, num_pages)
    return c


def random_cache(g: oracle.Geom, num_pages: int, seed: int, layout: str = "layer_major") -> oracle.Cache:
    rng = np.random.default_rng(seed)
    data = rng.integers(0, 256, size=cache_bytes(g, num_pages), dtype=np.uint8)
    scales = None
    if g.scale_kv:
        scales = rng.integers(0, 256, size=scale_bytes(g, num_pages), dtype=np.uint8)
    return make_cache(g, num_pages, data, scales, layout)


def clone_cache(c: oracle.Cache) -> oracle.Cache:
    return oracle.Cache(c.data.copy(), c.num_pages, c.layer_stride, c.kv_stride, c.page_stride,
                        None if c.scales is None else c.scales.copy(),
                        c.s_layer_stride, c.s_kv_stride, c.s_page_stride)


def n_pages(g: oracle.Geom, n_tokens: int) -> int:
    return -(-n_tokens // g.page_tokens)
