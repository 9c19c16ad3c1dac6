"""Seeded synthetic inputs for the KV block save/restore path.

This module serves both the CUDA library's callers and the CPU oracle's
callers.  It holds workload shapes and random draws only: no checksum, no blob
layout, no commit rule.  Anything that depends on the method (blob sizes, page
counts of a record) is passed in by the caller.

The five workloads stand in for the paper's own (its corpus, datasets and
model weights are not available): a tiny case, a GQA 7B-like serving case, the
97k-token recall corpus (Section 4.1 / storage-footprint paragraph of Section
4.3), an fp8 cache, and a stress mix shaped like the seven-dataset evaluation
with deliberately failed loads (Sections 4.2, 4.3).  The base seed is the one
the paper states for its dataset evaluation.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

BASE_SEED = 20260927


@dataclass(frozen=True)
class Workload:
    name: str
    index: int
    layers: int
    kv_heads: int
    head_dim: int
    page_tokens: int
    dtype: str            # "bf16" | "fp8_e4m3"
    sigma: float
    scale_kv: int = 0     # fp8: 2 = one K scale and one V scale per (layer, head, page)

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 1

    def seed(self, k: int = 0) -> int:
        return BASE_SEED + 1000 * self.index + k


TINY = Workload("tiny", 0, layers=2, kv_heads=2, head_dim=64, page_tokens=16, dtype="bf16", sigma=1.0)
GQA7B = Workload("gqa7b", 1, layers=32, kv_heads=8, head_dim=128, page_tokens=16, dtype="bf16", sigma=0.5)
CORPUS = Workload("corpus", 2, layers=48, kv_heads=8, head_dim=128, page_tokens=16, dtype="bf16", sigma=1.0)
FP8 = Workload("fp8", 3, layers=60, kv_heads=16, head_dim=128, page_tokens=32, dtype="fp8_e4m3",
               sigma=1.0, scale_kv=2)
STRESS = Workload("stress", 4, layers=24, kv_heads=4, head_dim=128, page_tokens=16, dtype="bf16", sigma=1.0)

WORKLOADS = {w.name: w for w in (TINY, GQA7B, CORPUS, FP8, STRESS)}

# block structure of the workloads (tokens per block)
TINY_BLOCKS = [256] * 4
TINY_DST_PAGES = 128
GQA7B_BLOCK_TOKENS = 4096
GQA7B_POOL_BLOCKS = 64
GQA7B_REQUESTS = 8
GQA7B_BLOCKS_PER_REQUEST = 2
GQA7B_DST_PAGES = 16384
CORPUS_BLOCKS = [1024] * 95 + [280]
CORPUS_DST_PAGES = 6200
FP8_BLOCKS = [2048] * 32
STRESS_POOL_BLOCKS = 20000
STRESS_REQUESTS = 256


def _torch_gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def kv_bytes_bf16(n_elems: int, sigma: float, seed: int, device="cpu") -> torch.Tensor:
    """uint8 tensor of 2*n_elems bytes: bf16 bit patterns of N(0, sigma) draws."""
    g = _torch_gen(seed, device)
    out = torch.empty(n_elems, dtype=torch.bfloat16, device=device)
    chunk = 1 << 26
    for lo in range(0, n_elems, chunk):
        hi = min(n_elems, lo + chunk)
        x = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32)
        out[lo:hi] = (x * sigma).to(torch.bfloat16)
    return out.view(torch.uint8)


def kv_bytes_fp8(layers: int, num_pages: int, page_tokens: int, kv_heads: int, head_dim: int,
                 sigma: float, seed: int, device="cpu"):
    """fp8 e4m3 cache of shape [L][2][N][T][H][D] (as uint8) and fp32 scales
    [L][2][N][H]: N(0, sigma) draws divided by amax/448 of their (l, kv, page,
    head) group, rounded to e4m3 by torch."""
    g = _torch_gen(seed, device)
    data = torch.empty((layers, 2, num_pages, page_tokens, kv_heads, head_dim),
                       dtype=torch.uint8, device=device)
    scales = torch.empty((layers, 2, num_pages, kv_heads), dtype=torch.float32, device=device)
    for l in range(layers):
        x = torch.randn((2, num_pages, page_tokens, kv_heads, head_dim), generator=g,
                        device=device, dtype=torch.float32) * sigma
        amax = x.abs().amax(dim=(2, 4)).clamp_min(1e-12)       # [2][N][H]
        s = amax / 448.0
        q = (x / s[:, :, None, :, None]).to(torch.float8_e4m3fn)
        data[l] = q.view(torch.uint8)
        scales[l] = s
    return data.reshape(-1), scales


def sentinel_bytes(n_bytes: int, seed: int, device="cpu") -> torch.Tensor:
    """Pseudo-random fill for a destination cache, so that stray writes (zeros
    included) show up in a byte comparison."""
    g = _torch_gen(seed, device)
    n8 = (n_bytes + 7) // 8
    out = torch.empty(n8, dtype=torch.int64, device=device)
    chunk = 1 << 25
    for lo in range(0, n8, chunk):
        hi = min(n8, lo + chunk)
        out[lo:hi] = torch.randint(-(1 << 62), 1 << 62, (hi - lo,), generator=g, device=device,
                                   dtype=torch.int64)
    return out.view(torch.uint8)[:n_bytes]


def page_permutation(num_pages: int, seed: int) -> np.ndarray:
    return np.random.default_rng(seed).permutation(num_pages).astype(np.int32)


def bit_flip_positions(total_bits: int, count: int, seed: int) -> np.ndarray:
    """``count`` distinct bit positions in [0, total_bits)."""
    rng = np.random.default_rng(seed)
    pos = set()
    while len(pos) < count:
        pos.add(int(rng.integers(0, total_bits)))
    return np.array(sorted(pos), dtype=np.int64)


def byte_run_corruption(start_lo: int, start_hi: int, length: int, seed: int):
    """A run of ``length`` consecutive byte offsets starting in [start_lo,
    start_hi) and one non-zero XOR value per byte."""
    rng = np.random.default_rng(seed)
    start = int(rng.integers(start_lo, max(start_lo + 1, start_hi - length)))
    xors = rng.integers(1, 256, size=length).astype(np.uint8)
    return start, xors


# ---------------------------------------------------------------------------
# Stress workload: block lengths, request mix, corrupted set.
# ---------------------------------------------------------------------------
def stress_block_lengths(seed: int, n_blocks: int = STRESS_POOL_BLOCKS) -> np.ndarray:
    """round(lognormal(mu=6, sigma=0.8)) clipped to [17, 4096] tokens."""
    rng = np.random.default_rng(seed)
    x = np.rint(rng.lognormal(mean=6.0, sigma=0.8, size=n_blocks))
    return np.clip(x, 17, 4096).astype(np.int64)


def stress_requests(seed: int, n_requests: int = STRESS_REQUESTS,
                    n_blocks: int = STRESS_POOL_BLOCKS, max_blocks: int = 40) -> list[np.ndarray]:
    """Each request draws uniform[1, max_blocks] distinct block ids; ranks follow
    p(r) ~ r^-1.1 on 1..n_blocks and map to ids through a seeded permutation."""
    rng = np.random.default_rng(seed)
    ranks = np.arange(1, n_blocks + 1, dtype=np.float64)
    prob = ranks ** -1.1
    prob /= prob.sum()
    rank_to_id = rng.permutation(n_blocks)
    out = []
    for _ in range(n_requests):
        k = int(rng.integers(1, max_blocks + 1))
        r = rng.choice(n_blocks, size=k, replace=False, p=prob)
        out.append(rank_to_id[r].astype(np.int64))
    return out


def stress_corrupted_blocks(seed: int, n_blocks: int = STRESS_POOL_BLOCKS, frac: float = 0.01):
    """Ids of the corrupted blobs (exactly frac*n_blocks of them) and the
    number of flipped bits, uniform in [1, 8], for each."""
    rng = np.random.default_rng(seed)
    ids = np.sort(rng.choice(n_blocks, size=int(round(frac * n_blocks)), replace=False))
    flips = rng.integers(1, 9, size=ids.size)
    return ids.astype(np.int64), flips.astype(np.int64)
