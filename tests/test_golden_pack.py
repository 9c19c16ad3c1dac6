"""Stored expected values (tests/golden/pack_golden.txt, written by a committed
script that calls only the oracle): the oracle must still reproduce them, and
the CUDA path must reproduce them too."""
import hashlib
import importlib.util
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _maker():
    spec = importlib.util.spec_from_file_location("make_pack_golden", os.path.join(HERE, "golden", "make_pack_golden.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


def _golden():
    out = {}
    with open(os.path.join(HERE, "golden", "pack_golden.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            out[parts[0]] = (parts[1], [int(x, 16) for x in parts[2:]])
    return out


def test_oracle_reproduces_stored_values():
    mk, gold = _maker(), _golden()
    for case in mk.CASES:
        name, L, H, D, T, E, K, N, n_tokens, table = case
        g = oracle.Geom(L, H, D, T, E, K)
        slab = T * H * D * E
        data, scales = mk.case_inputs(case)
        cache = oracle.Cache(data, N, 2 * N * slab, N * slab, slab)
        if K:
            cache.scales = scales
            cache.s_layer_stride, cache.s_kv_stride, cache.s_page_stride = K * N * H * 4, N * H * 4, H * 4
        blob, sums, code, _ = oracle.pack(g, cache, np.array(table, dtype=np.int32), n_tokens)
        assert code == 0
        assert hashlib.sha256(blob.tobytes()).hexdigest() == gold[name][0]
        assert [int(s) for s in sums] == gold[name][1]


@pytest.mark.gpu
def test_gpu_reproduces_stored_values():
    import torch
    import paper_2609_39358_b200 as gk
    mk, gold = _maker(), _golden()
    for case in mk.CASES:
        name, L, H, D, T, E, K, N, n_tokens, table = case
        geom = gk.Geom(L, H, D, T, gk.GK_BF16 if E == 2 else gk.GK_FP8_E4M3, K)
        slab = T * H * D * E
        data, scales = mk.case_inputs(case)
        cache = gk.Cache(torch.from_numpy(data).cuda(), N, 2 * N * slab, N * slab, slab)
        if K:
            cache.scales = torch.from_numpy(scales).cuda()
            cache.s_layer_stride, cache.s_kv_stride, cache.s_page_stride = K * N * H * 4, N * H * 4, H * 4
        ctx = gk.Context(geom, 0)
        nbytes, P = gk.gk_blob_size(geom, n_tokens)
        blob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        sums = torch.zeros(P, dtype=torch.int64, device="cuda")
        ctx.gk_pack(cache, torch.tensor(table, dtype=torch.int32, device="cuda"), n_tokens, blob, sums)
        torch.cuda.synchronize()
        assert hashlib.sha256(blob.cpu().numpy().tobytes()).hexdigest() == gold[name][0]
        assert [int(x) for x in sums.cpu().numpy().view(np.uint64)] == gold[name][1]
        ctx.close()
