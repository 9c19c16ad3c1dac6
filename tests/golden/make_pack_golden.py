#!/usr/bin/env python3
"""Writes pack_golden.txt: expected outputs of save (pack) for two small fixed
inputs, computed by the CPU oracle only.

The paper prints no worked example for its record format (it withholds the
format), so these stored values are not the paper's: they freeze what the pinned
oracle produces today, so that a later change to the oracle's arithmetic cannot
go unnoticed, and they give the CUDA path a stored target that was not produced
by the CUDA path.  Inputs are derived from SHA-256 in counter mode so that they
do not depend on any random-number library.

    python tests/golden/make_pack_golden.py      # rewrites pack_golden.txt
"""
import hashlib
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

CASES = [
    # name, layers, kv_heads, head_dim, page_tokens, elem_bytes, scale_kv, src_pages, n_tokens, page table
    ("bf16_ragged", 5, 4, 64, 16, 2, 0, 6, 2 * 16 + 5, [4, 1, 3]),
    ("fp8_scales", 6, 4, 32, 8, 1, 2, 5, 3 * 8 + 1, [0, 4, 2, 2]),
]


def counter_bytes(tag: str, n: int) -> np.ndarray:
    out = bytearray()
    i = 0
    while len(out) < n:
        out += hashlib.sha256(f"{tag}:{i}".encode()).digest()
        i += 1
    return np.frombuffer(bytes(out[:n]), dtype=np.uint8).copy()


def case_inputs(case):
    name, L, H, D, T, E, K, N, n_tokens, table = case
    slab = T * H * D * E
    data = counter_bytes(name + ":data", 2 * L * N * slab)
    scales = counter_bytes(name + ":scales", L * K * N * H * 4) if K else None
    return data, scales


def main():
    import oracle
    lines = ["# written by make_pack_golden.py from the CPU oracle; do not edit by hand",
             "# name blob_sha256 checksum_0 checksum_1 ..."]
    for case in CASES:
        name, L, H, D, T, E, K, N, n_tokens, table = case
        g = oracle.Geom(L, H, D, T, E, K)
        slab = T * H * D * E
        data, scales = case_inputs(case)
        cache = oracle.Cache(data, N, 2 * N * slab, N * slab, slab)
        if K:
            cache.scales = scales
            cache.s_layer_stride, cache.s_kv_stride, cache.s_page_stride = K * N * H * 4, N * H * 4, H * 4
        blob, sums, code, _ = oracle.pack(g, cache, np.array(table, dtype=np.int32), n_tokens)
        assert code == 0
        lines.append(" ".join([name, hashlib.sha256(blob.tobytes()).hexdigest()] + [f"{int(s):016x}" for s in sums]))
    with open(os.path.join(HERE, "pack_golden.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
