"""GPU parity of the layer-wise save and load against the oracle: blobs, checksums, block and
group codes, and the destination image after every group."""
import numpy as np
import pytest
import torch

import oracle
from helpers import clone_cache, n_pages, random_cache

pytestmark = pytest.mark.gpu

GROUP_GEOMS = [oracle.Geom(2, 4, 64, 16, 2, 0),             # bf16, 2 layers per group: records of 32 KiB
               oracle.Geom(4, 8, 128, 16, 2, 0),            # 4 layers per group: records of 256 KiB
               oracle.Geom(3, 8, 64, 32, 1, 2),             # fp8 with scales
               oracle.Geom(2, 4, 64, 16, 2, 0, head_major=1)]


@pytest.fixture(scope="module")
def gk():
    import paper_2609_39358_b200 as m
    assert torch.cuda.is_available()
    return m


def _full(g, G):
    return oracle.Geom(g.layers * G, g.kv_heads, g.head_dim, g.page_tokens, g.elem_bytes, g.scale_kv, g.head_major)


@pytest.mark.parametrize("og", GROUP_GEOMS)
@pytest.mark.parametrize("host", [False, True])
def test_layerwise_pack_and_restore_parity(gk, og, host):
    from gpu_harness import dev_cache, dev_i32, gk_geom
    G = 3
    full = _full(og, G)
    T = og.page_tokens
    src = random_cache(full, 11, seed=600)
    rng = np.random.default_rng(601)
    lens = [2 * T + 1, T, 4 * T - 1, 1]
    tables = [rng.integers(0, 11, size=n_pages(og, n)).astype(np.int32) for n in lens]
    Nd = 14
    perm = rng.permutation(Nd).astype(np.int32)
    ctx = gk.Context(gk_geom(og), 0)
    dsrc = dev_cache(src)

    # save
    jobs, keep = [], []
    for pt, n in zip(tables, lens):
        gb, P = oracle.blob_size(og, n)
        if host:
            blob = torch.zeros(G * gb, dtype=torch.uint8).pin_memory()
            sums = torch.zeros(G * P, dtype=torch.int64).pin_memory()
        else:
            blob = torch.zeros(G * gb, dtype=torch.uint8, device="cuda")
            sums = torch.zeros(G * P, dtype=torch.int64, device="cuda")
        keep.append((blob, sums))
        jobs.append(gk.Job(blob, sums, dev_i32(pt), n))
    status = torch.full((len(lens),), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_layerwise(G, dsrc, jobs, status, host=host)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * len(lens)
    ojobs, used = [], 0
    for (blob, sums), pt, n in zip(keep, tables, lens):
        wb, ws, code, _ = oracle.pack_layerwise(og, G, src, pt, n)
        assert code == 0
        assert np.array_equal(blob.cpu().numpy(), wb)
        assert np.array_equal(sums.cpu().numpy().view(np.uint64), ws)
        P = n_pages(og, n)
        ojobs.append(oracle.Job(wb.copy(), ws.copy(), perm[used:used + P].copy(), n))
        used += P

    # load: job 0 damaged in group 1, job 2 in groups 0 and 2, job 3 missing
    gb0, _ = oracle.blob_size(og, lens[0])
    gb2, P2 = oracle.blob_size(og, lens[2])
    ojobs[0].blob[gb0 + 9] ^= 0x02
    ojobs[2].blob[5] ^= 0x40
    ojobs[2].checksums[2 * P2 + 1] ^= np.uint64(1 << 33)
    ojobs[3] = oracle.Job(None, None, ojobs[3].page_table, lens[3])
    clean = random_cache(full, Nd, seed=602)
    want = clone_cache(clean)
    osnaps = []
    wmask, wfb, wgm = oracle.restore_layerwise(og, G, want, ojobs, lambda k, l0, nl: osnaps.append(want.data.copy()))
    assert wmask.tolist() == [1, 0, 1, 3] and wgm.tolist() == [[0, 0, 1, 3], [1, 0, 0, 3], [0, 0, 1, 3]]

    d = dev_cache(clean)
    djobs, dkeep = [], []
    for jb in ojobs:
        if jb.blob is None:
            b = s_ = None
        elif host:
            b = torch.from_numpy(jb.blob).pin_memory()
            s_ = torch.from_numpy(jb.checksums.view(np.int64).copy()).pin_memory()
        else:
            b = torch.from_numpy(jb.blob).cuda()
            s_ = torch.from_numpy(jb.checksums.view(np.int64).copy()).cuda()
        dkeep.append((b, s_))
        djobs.append(gk.Job(b, s_, dev_i32(jb.page_table), jb.n_tokens))
    for with_gm in (True, False):
        d.data.copy_(torch.from_numpy(clean.data))
        if d.scales is not None:
            d.scales.copy_(torch.from_numpy(clean.scales))
        mask = torch.full((4,), 255, dtype=torch.uint8, device="cuda")
        fb = torch.full((4,), -7, dtype=torch.int32, device="cuda")
        gm = torch.full((G, 4), 255, dtype=torch.uint8, device="cuda") if with_gm else None
        gsnaps, calls = [], []

        def on_group(group, first_layer, n_layers, st):
            assert st == torch.cuda.current_stream().cuda_stream
            calls.append((group, first_layer, n_layers))
            gsnaps.append(d.data.clone())

        ctx.gk_restore_layerwise(G, djobs, d, mask, fb, gm, on_group, host=host)
        torch.cuda.synchronize()
        assert calls == [(k, k * og.layers, og.layers) for k in range(G)]
        assert mask.cpu().tolist() == wmask.tolist() and fb.cpu().tolist() == wfb.tolist()
        if with_gm:
            assert gm.cpu().tolist() == wgm.tolist()
        for k in range(G):
            assert np.array_equal(gsnaps[k].cpu().numpy(), osnaps[k]), f"image after group {k} differs"
        assert np.array_equal(d.data.cpu().numpy(), want.data)
        if want.scales is not None:
            assert np.array_equal(d.scales.cpu().numpy(), want.scales)
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()
