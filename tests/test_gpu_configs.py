"""The workload configurations at full size on the GPU, in the launch
configuration bench.py times.  The oracle cannot process tens of GB in a test,
so these tests check (a) sampled page records, checksums and destination pages
one by one against the oracle, and (b) properties that hold at any size,
evaluated over ALL pages with torch on the device: every committed page equals
its source page on the valid token range, every other byte of the destination
equals the pre-call sentinel image, masks are exactly as the injected damage
dictates."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import oracle_geom

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gk():
    import paper_2609_39358_b200 as m
    assert torch.cuda.is_available()
    return m


@pytest.fixture(autouse=True)
def _release_device_memory():
    yield
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def _slab(w):
    return w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes


def _dev_cache(gk, w, num_pages, data, scales=None):
    s = _slab(w)
    c = gk.Cache(data, num_pages, 2 * num_pages * s, num_pages * s, s)
    if scales is not None:
        h4 = w.kv_heads * 4
        c.scales = scales
        c.s_layer_stride, c.s_kv_stride, c.s_page_stride = w.scale_kv * num_pages * h4, num_pages * h4, h4
    return c


def _view(w, cache):
    """[L][2][N][T][row] uint8 view of a layer-major cache."""
    return cache.data.view(w.layers, 2, cache.num_pages, w.page_tokens, -1)


def _scale_view(w, cache):
    return cache.scales.view(torch.uint8).view(w.layers, w.scale_kv, cache.num_pages, -1)


def _oracle_record(w, src_cache, phys, t_tokens):
    """Record bytes and checksum of one page, by the oracle, from the page's slabs."""
    og = oracle_geom(w)
    page = _view(w, src_cache)[:, :, phys].contiguous().cpu().numpy().reshape(-1)
    s = _slab(w)
    oc = oracle.Cache(page, 1, 2 * s, s, s)
    if w.scale_kv:
        sc = _scale_view(w, src_cache)[:, :, phys].contiguous().cpu().numpy().reshape(-1)
        oc.scales = sc
        h4 = w.kv_heads * 4
        oc.s_layer_stride, oc.s_kv_stride, oc.s_page_stride = w.scale_kv * h4, h4, h4
    blob, sums, code, _ = oracle.pack(og, oc, np.zeros(1, dtype=np.int32), t_tokens)
    assert code == 0
    return blob, int(sums[0])


def _check_sampled_records(w, src, jobs_meta, rng, n_samples):
    """jobs_meta: list of (blob tensor, sums tensor, src table (np), n_tokens)."""
    og = oracle_geom(w)
    for _ in range(n_samples):
        j = int(rng.integers(0, len(jobs_meta)))
        blob, sums, spt, n = jobs_meta[j]
        P = -(-n // w.page_tokens)
        p = int(rng.integers(0, P)) if rng.random() < 0.7 else P - 1
        t = min(w.page_tokens, n - p * w.page_tokens)
        want, crc = _oracle_record(w, src, int(spt[p]), t)
        lo = oracle.record_offset(og, p)
        got = blob[lo:lo + want.size].cpu().numpy()
        assert np.array_equal(got, want), f"record {p} of job {j} differs"
        assert int(sums[p].item()) & 0xFFFFFFFFFFFFFFFF == crc, f"checksum {p} of job {j} differs"


def _check_all_checksums(w, blobs, sums, lens):
    """EVERY checksum of every block against the oracle's CRC-64 of the record bytes as the
    GPU packed them (blobs copied to the host block by block; the oracle runs on a few
    host threads, ctypes releases the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    import os
    og = oracle_geom(w)
    with ThreadPoolExecutor(max_workers=max(1, min(16, os.cpu_count() or 1))) as pool:
        for blob, sm, n in zip(blobs, sums, lens):
            host = blob.cpu().numpy()
            got = sm.cpu().numpy().view(np.uint64)
            P = -(-n // w.page_tokens)
            offs = [oracle.record_offset(og, p) for p in range(P)] + [host.size]
            want = list(pool.map(lambda p: oracle.crc64(host[offs[p]:offs[p + 1]]), range(P)))
            assert [int(x) for x in got] == want, "a checksum differs from the oracle's"


def _check_whole_block(w, src, blob, sums, spt, n):
    """All bytes and all checksums of one block against oracle.pack over the block's source pages."""
    og = oracle_geom(w)
    idx = torch.from_numpy(np.ascontiguousarray(spt).astype(np.int64)).cuda()
    P = idx.numel()
    pages = _view(w, src)[:, :, idx].contiguous().cpu().numpy().reshape(-1)   # [L][2][P][T][row]
    s = _slab(w)
    oc = oracle.Cache(pages, P, 2 * P * s, P * s, s)
    if w.scale_kv:
        oc.scales = _scale_view(w, src)[:, :, idx].contiguous().cpu().numpy().reshape(-1)
        h4 = w.kv_heads * 4
        oc.s_layer_stride, oc.s_kv_stride, oc.s_page_stride = w.scale_kv * P * h4, P * h4, h4
    want_blob, want_sums, code, _ = oracle.pack(og, oc, np.arange(P, dtype=np.int32), n)
    assert code == 0
    assert np.array_equal(blob.cpu().numpy(), want_blob), "blob bytes differ from the oracle's"
    assert np.array_equal(sums.cpu().numpy().view(np.uint64), want_sums), "checksums differ from the oracle's"


def _check_destination(w, src, dst, sentinel, jobs, masks):
    """jobs: list of (src table np, dst table np, n_tokens).  Every committed page
    equals its source on the valid range; everything else equals the sentinel."""
    T = w.page_tokens
    sv, dv, zv = _view(w, src), _view(w, dst), sentinel.view(w.layers, 2, dst.num_pages, T, -1)
    expected_untouched = torch.ones(dst.num_pages, dtype=torch.bool, device="cuda")
    for (spt, dpt, n), code in zip(jobs, masks):
        if code != 0:
            continue
        P = -(-n // T)
        full = P if n % T == 0 else P - 1
        s_idx = torch.from_numpy(np.ascontiguousarray(spt[:full]).astype(np.int64)).cuda()
        d_idx = torch.from_numpy(np.ascontiguousarray(dpt[:full]).astype(np.int64)).cuda()
        assert torch.equal(dv[:, :, d_idx], sv[:, :, s_idx])
        expected_untouched[d_idx] = False
        if w.scale_kv:
            assert torch.equal(_scale_view(w, dst)[:, :, d_idx], _scale_view(w, src)[:, :, s_idx])
        if full < P:
            t = n - full * T
            sp, dp = int(spt[full]), int(dpt[full])
            assert torch.equal(dv[:, :, dp, :t], sv[:, :, sp, :t])
            assert torch.equal(dv[:, :, dp, t:], zv[:, :, dp, t:])          # tail of the partial page
            expected_untouched[dp] = False
            if w.scale_kv:
                assert torch.equal(_scale_view(w, dst)[:, :, dp], _scale_view(w, src)[:, :, sp])
    rest = torch.nonzero(expected_untouched).flatten()
    for lo in range(0, rest.numel(), 512):
        idx = rest[lo:lo + 512]
        assert torch.equal(dv[:, :, idx], zv[:, :, idx]), "a page outside the committed set was written"


# ---------------------------------------------------------------------------
def test_gqa7b_full(gk):
    """8 requests x 2 blocks of 4,096 tokens into a 16,384-page cache; no corruption."""
    w = synth.GQA7B
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens)
    ctx = gk.Context(geom, 0)
    n_tok, NB = synth.GQA7B_BLOCK_TOKENS, synth.GQA7B_REQUESTS * synth.GQA7B_BLOCKS_PER_REQUEST
    nbytes, P = gk.gk_blob_size(geom, n_tok)
    s = _slab(w)
    src_pages, dst_pages = NB * P, synth.GQA7B_DST_PAGES
    src = _dev_cache(gk, w, src_pages, synth.kv_bytes_bf16(w.layers * src_pages * s, w.sigma, w.seed(0), "cuda"))
    sentinel = synth.sentinel_bytes(2 * w.layers * dst_pages * s, w.seed(1), "cuda")
    dst = _dev_cache(gk, w, dst_pages, sentinel.clone())
    sperm = synth.page_permutation(src_pages, w.seed(2))
    dperm = synth.page_permutation(dst_pages, w.seed(3))
    blobs = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(NB)]
    sums = [torch.zeros(P, dtype=torch.int64, device="cuda") for _ in range(NB)]
    spts = [sperm[i * P:(i + 1) * P] for i in range(NB)]
    dpts = [dperm[i * P:(i + 1) * P] for i in range(NB)]
    d_spts = [torch.from_numpy(x.copy()).cuda() for x in spts]
    d_dpts = [torch.from_numpy(x.copy()).cuda() for x in dpts]
    status = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_batch(src, [gk.Job(blobs[i], sums[i], d_spts[i], n_tok) for i in range(NB)], status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * NB
    rng = np.random.default_rng(w.seed(4))
    _check_sampled_records(w, src, [(blobs[i], sums[i], spts[i], n_tok) for i in range(NB)], rng, 24)
    # all 4,096 checksums of the batch, and every byte of two whole blocks, against the oracle
    _check_all_checksums(w, blobs, sums, [n_tok] * NB)
    for i in (0, NB - 1):
        _check_whole_block(w, src, blobs[i], sums[i], spts[i], n_tok)
    mask = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(NB, dtype=torch.int32, device="cuda")
    ctx.gk_restore([gk.Job(blobs[i], sums[i], d_dpts[i], n_tok, i // 2) for i in range(NB)], dst, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == [0] * NB and fb.cpu().tolist() == [-1] * NB
    _check_destination(w, src, dst, sentinel, [(spts[i], dpts[i], n_tok) for i in range(NB)], [0] * NB)
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_small_records_full(gk):
    """The gqa7b geometry with ONE layer per record (64 KiB records, the layer-wise format's smallest group):
    8 blocks of 32,768 tokens = 16,384 pages, 1 GiB of blobs.  Calls of this size take the page-quartet form
    of the packing and of the fused restore kernel (one record per warp).  All 16,384 checksums and every
    byte of two blocks against the oracle; one blob damaged; full destination check."""
    import dataclasses
    w = dataclasses.replace(synth.GQA7B, layers=1)
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens)
    ctx = gk.Context(geom, 0)
    n_tok, NB = 32768, 8
    nbytes, P = gk.gk_blob_size(geom, n_tok)
    s = _slab(w)
    src_pages, dst_pages = NB * P, NB * P + 100
    src = _dev_cache(gk, w, src_pages, synth.kv_bytes_bf16(w.layers * src_pages * s, w.sigma, w.seed(40), "cuda"))
    sentinel = synth.sentinel_bytes(2 * w.layers * dst_pages * s, w.seed(41), "cuda")
    dst = _dev_cache(gk, w, dst_pages, sentinel.clone())
    sperm = synth.page_permutation(src_pages, w.seed(42))
    dperm = synth.page_permutation(dst_pages, w.seed(43))
    blobs = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(NB)]
    sums = [torch.zeros(P, dtype=torch.int64, device="cuda") for _ in range(NB)]
    spts = [sperm[i * P:(i + 1) * P] for i in range(NB)]
    dpts = [dperm[i * P:(i + 1) * P] for i in range(NB)]
    d_spts = [torch.from_numpy(x.copy()).cuda() for x in spts]
    d_dpts = [torch.from_numpy(x.copy()).cuda() for x in dpts]
    status = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_batch(src, [gk.Job(blobs[i], sums[i], d_spts[i], n_tok) for i in range(NB)], status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * NB
    assert ctx.gk_get_stats()["quartet_launches"] == 1
    _check_all_checksums(w, blobs, sums, [n_tok] * NB)
    for i in (0, NB - 1):
        _check_whole_block(w, src, blobs[i], sums[i], spts[i], n_tok)
    # one byte of block 5 flipped, in the third page of a quartet
    bad_page = 4 * 277 + 2
    blobs[5][bad_page * (nbytes // P) + 12345] ^= 0x10
    mask = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(NB, dtype=torch.int32, device="cuda")
    ctx.gk_restore([gk.Job(blobs[i], sums[i], d_dpts[i], n_tok) for i in range(NB)], dst, mask, fb)
    torch.cuda.synchronize()
    want = [0] * NB
    want[5] = 1
    assert mask.cpu().tolist() == want
    assert fb.cpu().tolist() == [-1 if m == 0 else bad_page for m in want]
    assert ctx.gk_get_stats()["quartet_launches"] == 2
    _check_destination(w, src, dst, sentinel, [(spts[i], dpts[i], n_tok) for i in range(NB)], want)
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_corpus_full_device_and_host_tier(gk):
    """95 blocks of 1,024 tokens + a 280-token tail block (partial last page) into a
    6,200-page cache: once from device blobs, once from pinned host memory."""
    w = synth.CORPUS
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens)
    ctx = gk.Context(geom, 0)
    lens = synth.CORPUS_BLOCKS
    s = _slab(w)
    pages = [-(-n // w.page_tokens) for n in lens]
    src_pages, dst_pages = sum(pages), synth.CORPUS_DST_PAGES
    assert src_pages == 6098
    src = _dev_cache(gk, w, src_pages, synth.kv_bytes_bf16(w.layers * src_pages * s, w.sigma, w.seed(0), "cuda"))
    sentinel = synth.sentinel_bytes(2 * w.layers * dst_pages * s, w.seed(1), "cuda")
    dst = _dev_cache(gk, w, dst_pages, sentinel.clone())
    sperm = synth.page_permutation(src_pages, w.seed(2))
    dperm = synth.page_permutation(dst_pages, w.seed(3))
    blobs, sums, spts, dpts, off = [], [], [], [], 0
    for n, P in zip(lens, pages):
        blobs.append(torch.empty(gk.gk_blob_size(geom, n)[0], dtype=torch.uint8, device="cuda"))
        sums.append(torch.zeros(P, dtype=torch.int64, device="cuda"))
        spts.append(sperm[off:off + P])
        dpts.append(dperm[off:off + P])
        off += P
    assert sum(b.numel() for b in blobs) == 19_181_076_480
    d_spts = [torch.from_numpy(x.copy()).cuda() for x in spts]
    d_dpts = [torch.from_numpy(x.copy()).cuda() for x in dpts]
    NB = len(lens)
    status = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_batch(src, [gk.Job(blobs[i], sums[i], d_spts[i], lens[i]) for i in range(NB)], status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * NB
    rng = np.random.default_rng(w.seed(4))
    meta = [(blobs[i], sums[i], spts[i], lens[i]) for i in range(NB)]
    _check_sampled_records(w, src, meta, rng, 16)
    _check_sampled_records(w, src, meta[-1:], rng, 6)          # the tail block, its partial page included
    # the 280-token tail block whole (its 8-token last page included) and one full block, byte for byte
    _check_whole_block(w, src, blobs[-1], sums[-1], spts[-1], lens[-1])
    _check_whole_block(w, src, blobs[40], sums[40], spts[40], lens[40])
    _check_all_checksums(w, blobs[-3:], sums[-3:], lens[-3:])
    jobs_meta = [(spts[i], dpts[i], lens[i]) for i in range(NB)]
    mask = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(NB, dtype=torch.int32, device="cuda")
    # run A: device-resident blobs
    ctx.gk_restore([gk.Job(blobs[i], sums[i], d_dpts[i], lens[i]) for i in range(NB)], dst, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == [0] * NB
    _check_destination(w, src, dst, sentinel, jobs_meta, [0] * NB)
    # run B: save the corpus to pinned host memory with gk_pack_host (many staging batches),
    # check it is byte-identical to the device-packed blobs, damage one blob on the host,
    # restore from the host tier
    dst.data.copy_(sentinel)
    host = []
    for i in range(NB):
        hb = torch.empty(blobs[i].numel(), dtype=torch.uint8, pin_memory=True)
        hs = torch.empty(pages[i], dtype=torch.int64, pin_memory=True)
        host.append((hb, hs))
    status.fill_(255)
    ctx.gk_pack_host(src, [gk.Job(host[i][0], host[i][1], d_spts[i], lens[i]) for i in range(NB)], status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * NB
    for i in range(NB):
        assert torch.equal(host[i][0], blobs[i].cpu()) and torch.equal(host[i][1], sums[i].cpu())
    del blobs
    victim = 37
    host[victim][0][123_456_789] ^= 0x04
    mask.fill_(255)
    ctx.gk_restore_host([gk.Job(host[i][0], host[i][1], d_dpts[i], lens[i]) for i in range(NB)], dst, mask, fb)
    torch.cuda.synchronize()
    want = [0] * NB
    want[victim] = 1
    assert mask.cpu().tolist() == want
    og = oracle_geom(w)
    assert fb.cpu().tolist()[victim] == 123_456_789 // oracle.record_bytes(og, 1024, 0)
    _check_destination(w, src, dst, sentinel, jobs_meta, want)
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_fp8_full(gk):
    """32 blocks of 2,048 tokens, fp8 with per-(layer, head, page) K and V scales in
    the record; damage in a scale section of one blob and in the K data of another."""
    w = synth.FP8
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_FP8_E4M3, w.scale_kv)
    ctx = gk.Context(geom, 0)
    lens = synth.FP8_BLOCKS
    NB, n_tok = len(lens), lens[0]
    nbytes, P = gk.gk_blob_size(geom, n_tok)
    assert nbytes == 64 * 7_872_000
    src_pages = NB * P
    dst_pages = src_pages + 100
    data, scales = synth.kv_bytes_fp8(w.layers, src_pages, w.page_tokens, w.kv_heads, w.head_dim, w.sigma,
                                      w.seed(0), "cuda")
    src = _dev_cache(gk, w, src_pages, data, scales)
    s = _slab(w)
    sentinel = synth.sentinel_bytes(2 * w.layers * dst_pages * s, w.seed(1), "cuda")
    sent_scales = synth.sentinel_bytes(w.layers * 2 * dst_pages * w.kv_heads * 4, w.seed(5), "cuda")
    dst = _dev_cache(gk, w, dst_pages, sentinel.clone(), sent_scales.clone().view(torch.float32))
    sperm = synth.page_permutation(src_pages, w.seed(2))
    dperm = synth.page_permutation(dst_pages, w.seed(3))
    blobs = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(NB)]
    sums = [torch.zeros(P, dtype=torch.int64, device="cuda") for _ in range(NB)]
    spts = [sperm[i * P:(i + 1) * P] for i in range(NB)]
    dpts = [dperm[i * P:(i + 1) * P] for i in range(NB)]
    d_spts = [torch.from_numpy(x.copy()).cuda() for x in spts]
    d_dpts = [torch.from_numpy(x.copy()).cuda() for x in dpts]
    status = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_batch(src, [gk.Job(blobs[i], sums[i], d_spts[i], n_tok) for i in range(NB)], status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * NB
    rng = np.random.default_rng(w.seed(4))
    _check_sampled_records(w, src, [(blobs[i], sums[i], spts[i], n_tok) for i in range(NB)], rng, 12)
    # seeded damage: 8 consecutive bytes, each xored with a non-zero value
    og = oracle_geom(w)
    R = oracle.record_bytes(og, n_tok, 0)
    S = w.layers * w.scale_kv * w.kv_heads * 4
    job_a, job_b = (int(x) for x in rng.choice(NB, size=2, replace=False))
    page_a, page_b = int(rng.integers(0, P)), int(rng.integers(0, P))
    start, xors = synth.byte_run_corruption(page_a * R, page_a * R + S, 8, w.seed(6))
    blobs[job_a][start:start + 8] ^= torch.from_numpy(xors).cuda()
    start, xors = synth.byte_run_corruption(page_b * R + S, page_b * R + S + s, 8, w.seed(7))
    blobs[job_b][start:start + 8] ^= torch.from_numpy(xors).cuda()
    mask = torch.full((NB,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(NB, dtype=torch.int32, device="cuda")
    ctx.gk_restore([gk.Job(blobs[i], sums[i], d_dpts[i], n_tok) for i in range(NB)], dst, mask, fb)
    torch.cuda.synchronize()
    want = [0] * NB
    want[job_a] = want[job_b] = 1
    assert mask.cpu().tolist() == want
    assert fb.cpu().tolist()[job_a] == page_a and fb.cpu().tolist()[job_b] == page_b
    _check_destination(w, src, dst, sentinel, [(spts[i], dpts[i], n_tok) for i in range(NB)], want)
    # scale entries of rejected jobs and of unmapped pages keep the sentinel
    untouched = np.ones(dst_pages, dtype=bool)
    for i in range(NB):
        if want[i] == 0:
            untouched[dpts[i]] = False
    idx = torch.from_numpy(np.flatnonzero(untouched)).cuda()
    zs = sent_scales.view(w.layers, w.scale_kv, dst_pages, -1)
    assert torch.equal(_scale_view(w, dst)[:, :, idx], zs[:, :, idx])
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


@pytest.mark.parametrize("bad_frac", [0.01, 1.0 / 3.0])
def test_stress_waves(gk, bad_frac):
    """(bad_frac = 1/3 mirrors the paper's experiment with one in three loads
    deliberately failed, Section 4.3 / Section 5: every request still completes.)
    20,000-block pool (lengths lognormal, clipped to [17, 4096]), 256 requests of
    1..40 blocks drawn Zipf(1.1) without replacement, 1% of the blobs with 1..8
    flipped bits.  Only referenced blocks are materialised; requests run in
    waves that fit the destination cache; page tables never reuse a page within
    a wave.  Every job on a damaged blob must come back rejected, every other
    job committed, and the destination must say the same byte for byte."""
    w = synth.STRESS
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens)
    ctx = gk.Context(geom, 0)
    T, s = w.page_tokens, _slab(w)
    lengths = synth.stress_block_lengths(w.seed(0))
    requests = synth.stress_requests(w.seed(1))
    bad_ids, bad_flips = synth.stress_corrupted_blocks(w.seed(2), frac=bad_frac)
    bad = dict(zip(bad_ids.tolist(), bad_flips.tolist()))
    unique = sorted({int(b) for r in requests for b in r})
    n_jobs = sum(len(r) for r in requests)
    assert 1000 < len(unique) < 3000 and 4000 < n_jobs < 6500

    # pool: each referenced block is generated from its own seed into a scratch
    # source cache and packed once
    max_pages = -(-4096 // T)
    scratch_tab = torch.arange(max_pages, dtype=torch.int32, device="cuda")
    pool = {}
    for b in unique:
        n = int(lengths[b])
        P = -(-n // T)
        data = synth.kv_bytes_bf16(w.layers * P * s, w.sigma, w.seed(10_000 + b), "cuda")
        src = _dev_cache(gk, w, P, data)
        blob = torch.empty(gk.gk_blob_size(geom, n)[0], dtype=torch.uint8, device="cuda")
        sums = torch.zeros(P, dtype=torch.int64, device="cuda")
        ctx.gk_pack(src, scratch_tab[:P], n, blob, sums)
        if b in bad:
            torch.cuda.synchronize()
            for pos in synth.bit_flip_positions(blob.numel() * 8, bad[b], w.seed(50_000 + b)):
                blob[int(pos) >> 3] ^= 1 << (int(pos) & 7)
        pool[b] = (blob, sums, n, P)
    torch.cuda.synchronize()

    dst_pages = 32768
    sentinel = synth.sentinel_bytes(2 * w.layers * dst_pages * s, w.seed(3), "cuda")
    dst = _dev_cache(gk, w, dst_pages, sentinel.clone())
    # waves: requests in order while their pages fit
    waves, cur, cur_pages = [], [], 0
    for r in requests:
        need = sum(pool[int(b)][3] for b in r)
        if cur and cur_pages + need > dst_pages:
            waves.append(cur)
            cur, cur_pages = [], 0
        cur.append(r)
        cur_pages += need
    waves.append(cur)
    rng = np.random.default_rng(w.seed(4))
    total_rejected = 0
    for wi, wave in enumerate(waves):
        perm = synth.page_permutation(dst_pages, w.seed(100 + wi))
        jobs, meta, off = [], [], 0
        for ri, r in enumerate(wave):
            for b in r:
                blob, sums, n, P = pool[int(b)]
                dpt = perm[off:off + P]
                off += P
                jobs.append(gk.Job(blob, sums, torch.from_numpy(dpt.copy()).cuda(), n, ri))
                meta.append((int(b), dpt, n, P))
        mask = torch.full((len(jobs),), 255, dtype=torch.uint8, device="cuda")
        fb = torch.zeros(len(jobs), dtype=torch.int32, device="cuda")
        if wi > 0:
            dst.data.copy_(sentinel)
        ctx.gk_restore(jobs, dst, mask, fb)
        torch.cuda.synchronize()
        got = mask.cpu().numpy()
        want = np.array([1 if m[0] in bad else 0 for m in meta], dtype=np.uint8)
        assert np.array_equal(got, want)
        total_rejected += int(want.sum())
        # committed pages: regenerate a sample of blocks from their seeds and compare all their pages;
        # rejected and unmapped pages: all of them against the sentinel
        dv = _view(w, dst)
        zv = sentinel.view(w.layers, 2, dst_pages, T, -1)
        untouched = np.ones(dst_pages, dtype=bool)
        for (b, dpt, n, P), code in zip(meta, got):
            if code == 0:
                untouched[dpt] = False
        idx_all = torch.from_numpy(np.flatnonzero(untouched)).cuda()
        for lo in range(0, idx_all.numel(), 1024):
            idx = idx_all[lo:lo + 1024]
            assert torch.equal(dv[:, :, idx], zv[:, :, idx])
        for k in rng.choice(len(meta), size=min(40, len(meta)), replace=False):
            b, dpt, n, P = meta[int(k)]
            if got[int(k)] != 0:
                continue
            data = synth.kv_bytes_bf16(w.layers * P * s, w.sigma, w.seed(10_000 + b), "cuda")
            sv = data.view(w.layers, 2, P, T, -1)
            d_idx = torch.from_numpy(dpt.astype(np.int64)).cuda()
            full = P if n % T == 0 else P - 1
            assert torch.equal(dv[:, :, d_idx[:full]], sv[:, :, :full])
            if full < P:
                t = n - full * T
                assert torch.equal(dv[:, :, d_idx[full], :t], sv[:, :, full, :t])
                assert torch.equal(dv[:, :, d_idx[full], t:], zv[:, :, d_idx[full], t:])
        # two sampled jobs of the wave against the oracle end to end (blob, checksums, mask)
        og = oracle_geom(w)
        for k in rng.choice(len(meta), size=2, replace=False):
            b, dpt, n, P = meta[int(k)]
            blob, sums, _, _ = pool[b]
            hb = blob.cpu().numpy()
            hs = sums.cpu().numpy().view(np.uint64)
            oc = oracle.Cache(np.zeros(2 * w.layers * P * s, dtype=np.uint8), P, 2 * P * s, P * s, s)
            om, ofb = oracle.restore(og, oc, [oracle.Job(hb, hs, np.arange(P, dtype=np.int32), n)])
            assert om[0] == got[int(k)] and ofb[0] == fb.cpu().numpy()[int(k)]
    assert total_rejected > 0
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_long_window_stream_restore(gk):
    """Blocks of 30,000 tokens (the block size of the paper's flat-memory experiment,
    Section 4.3) in the GQA-7B geometry, streamed from pinned host memory through a ring of
    two blocks: sampled records against the oracle, and, inside the consumer of every
    window, every page of the ring against the source caches on the device."""
    w = synth.GQA7B
    T = w.page_tokens
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens)
    ctx = gk.Context(geom, 0)
    s = _slab(w)
    lens3 = [30000, 29999, 30000]                       # A, B (partial last page), C (will be damaged)
    P = 1875
    srcs, host, tables = [], [], []
    rng = np.random.default_rng(w.seed(40))
    for k, n in enumerate(lens3):
        src = _dev_cache(gk, w, P, synth.kv_bytes_bf16(w.layers * P * s, w.sigma, w.seed(41 + k), "cuda"))
        spt = synth.page_permutation(P, w.seed(45 + k))
        hb = torch.empty(gk.gk_blob_size(geom, n)[0], dtype=torch.uint8, pin_memory=True)
        hs = torch.empty(P, dtype=torch.int64, pin_memory=True)
        status = torch.full((1,), 255, dtype=torch.uint8, device="cuda")
        ctx.gk_pack_host(src, [gk.Job(hb, hs, torch.from_numpy(spt.copy()).cuda(), n)], status)
        torch.cuda.synchronize()
        assert status.item() == 0
        _check_sampled_records(w, src, [(hb, hs, spt, n)], rng, 6)
        srcs.append(src)
        host.append((hb, hs))
        tables.append(spt)
    host[2][0][2_000_000_001] ^= 0x40                   # C: one flipped bit, in page 953
    order = [0, 1, 2, 0, 1, 2, 1]                       # windows: {A,B} {C,A} {B,C} {B}
    jobs = [gk.Job(host[k][0], host[k][1], None, lens3[k]) for k in order]
    ring_pages = 2 * P + 10
    sentinel = synth.sentinel_bytes(2 * w.layers * ring_pages * s, w.seed(49), "cuda")
    ring = _dev_cache(gk, w, ring_pages, sentinel.clone())
    rv = _view(w, ring)
    mask = torch.full((len(order),), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((len(order),), -7, dtype=torch.int32, device="cuda")
    checks, windows = [], []
    prev = {"img": sentinel.clone()}

    def consume(blocks, st):
        windows.append([b.job for b in blocks])
        pv = prev["img"].view(w.layers, 2, ring_pages, T, -1)
        first = 0
        for b in blocks:
            assert (b.page_table - blocks[0].page_table) // 4 == first
            k = order[b.job]
            n = lens3[k]
            if k == 2:      # damaged: its pages keep what the previous window left there
                checks.append(torch.equal(rv[:, :, first:first + P], pv[:, :, first:first + P]))
            else:
                full = n // T
                idx = torch.from_numpy(tables[k][:full].astype(np.int64)).cuda()
                checks.append(torch.equal(rv[:, :, first:first + full], _view(w, srcs[k])[:, :, idx]))
                if full < P:
                    t, sp = n - full * T, int(tables[k][full])
                    checks.append(torch.equal(rv[:, :, first + full, :t], _view(w, srcs[k])[:, :, sp, :t]))
                    checks.append(torch.equal(rv[:, :, first + full, t:], pv[:, :, first + full, t:]))
            first += P
        checks.append(torch.equal(rv[:, :, first:], pv[:, :, first:]))      # pages beyond the window
        prev["img"] = ring.data.clone()

    ctx.gk_restore_stream(jobs, ring, mask, fb, consume)
    torch.cuda.synchronize()
    assert windows == [[0, 1], [2, 3], [4, 5], [6]]
    assert mask.cpu().tolist() == [1 if k == 2 else 0 for k in order]
    og = oracle_geom(w)
    bad_page = 2_000_000_001 // oracle.record_bytes(og, 30000, 0)
    assert [fb.cpu().tolist()[i] for i, k in enumerate(order) if k == 2] == [bad_page] * 2
    assert all(checks) and len(checks) >= 12
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_gqa7b_full_digests_and_keys(gk):
    """The second tier at the headline batch size: 16 blocks of 4,096 tokens (8 GiB).  Sampled
    page digests against the oracle; every root recomputed with hashlib from the page
    digests the GPU reports; keys of the 16 token-id blocks against the oracle."""
    import hashlib
    import struct
    w = synth.GQA7B
    og = oracle_geom(w)
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens)
    ctx = gk.Context(geom, 0)
    n_tok, NB = synth.GQA7B_BLOCK_TOKENS, synth.GQA7B_REQUESTS * synth.GQA7B_BLOCKS_PER_REQUEST
    nbytes, P = gk.gk_blob_size(geom, n_tok)
    blobs = [synth.kv_bytes_bf16(nbytes // 2, w.sigma, w.seed(60 + j), "cuda") for j in range(NB)]
    # keys
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed(80))
    ids = torch.randint(0, 128000, (NB * n_tok,), generator=g, device="cuda", dtype=torch.int32)
    offsets = torch.arange(NB + 1, dtype=torch.int64, device="cuda") * (4 * n_tok)
    parent = [(-1 if j % 2 == 0 else j - 1) for j in range(NB)]
    model, tenant = bytes(range(32)), bytes(range(64, 96))
    keys = torch.zeros(NB, 32, dtype=torch.uint8, device="cuda")
    ctx.gk_fingerprints(ids.view(torch.uint8), offsets, parent, model, tenant, keys)
    torch.cuda.synchronize()
    want_keys = oracle.fingerprints(ids.cpu().numpy().view(np.uint8), offsets.cpu().numpy().astype(np.uint64), parent,
                                    model, tenant)
    assert np.array_equal(keys.cpu().numpy(), want_keys)
    # digests
    digests = torch.zeros(NB, 32, dtype=torch.uint8, device="cuda")
    pages = torch.zeros(NB * P, 32, dtype=torch.uint8, device="cuda")
    ctx.gk_blob_digests([gk.Job(b, None, None, n_tok) for b in blobs], keys, digests, pages)
    torch.cuda.synchronize()
    hp, hd, hk = pages.cpu().numpy(), digests.cpu().numpy(), keys.cpu().numpy()
    rng = np.random.default_rng(w.seed(81))
    R = oracle.record_bytes(og, n_tok, 0)
    for _ in range(12):
        j, p = int(rng.integers(0, NB)), int(rng.integers(0, P))
        rec = blobs[j][p * R:(p + 1) * R].cpu().numpy()
        _, one = oracle.blob_digest(og, rec, w.page_tokens, bytes(32))        # a one-page blob: its page node
        assert np.array_equal(hp[j * P + p], one[0]), (j, p)
    for j in range(NB):
        root = hashlib.sha256(hp[j * P:(j + 1) * P].tobytes() + hk[j].tobytes() + struct.pack("<II", n_tok, P)
                              + b"GKB0").digest()
        assert hd[j].tobytes() == root
    ctx.close()


@pytest.mark.parametrize("host_tier", [True, False])
def test_layerwise_full_size(gk, host_tier):
    """GQA-7B geometry cut into 8 groups of 4 layers, 3 blocks of 4,096 / 4,096 / 5,200 tokens,
    saved and loaded group by group -- to and from pinned host memory, and on the device tier, where
    the groups alternate between the context and its twin on two streams; one (block, group) damaged."""
    w = synth.GQA7B
    T = w.page_tokens
    gl, G = 4, w.layers // 4
    g_geom = gk.Geom(gl, w.kv_heads, w.head_dim, w.page_tokens)
    og_group = oracle.Geom(gl, w.kv_heads, w.head_dim, w.page_tokens, 2, 0)
    ctx = gk.Context(g_geom, 0)
    s = _slab(w)
    lens = [4096, 4096, 5200]
    pages = [-(-n // T) for n in lens]
    N = sum(pages)
    src = _dev_cache(gk, w, N, synth.kv_bytes_bf16(w.layers * N * s, w.sigma, w.seed(70), "cuda"))
    Nd = N + 50
    sentinel = synth.sentinel_bytes(2 * w.layers * Nd * s, w.seed(71), "cuda")
    dst = _dev_cache(gk, w, Nd, sentinel.clone())
    sperm, dperm = synth.page_permutation(N, w.seed(72)), synth.page_permutation(Nd, w.seed(73))
    jobs_s, jobs_d, spts, dpts, host, off = [], [], [], [], [], 0
    for n, P in zip(lens, pages):
        gb, _ = gk.gk_blob_size(g_geom, n)
        if host_tier:
            hb = torch.empty(G * gb, dtype=torch.uint8, pin_memory=True)
            hs = torch.empty(G * P, dtype=torch.int64, pin_memory=True)
        else:
            hb = torch.empty(G * gb, dtype=torch.uint8, device="cuda")
            hs = torch.empty(G * P, dtype=torch.int64, device="cuda")
        spts.append(sperm[off:off + P])
        dpts.append(dperm[off:off + P])
        host.append((hb, hs, gb))
        jobs_s.append(gk.Job(hb, hs, torch.from_numpy(spts[-1].copy()).cuda(), n))
        jobs_d.append(gk.Job(hb, hs, torch.from_numpy(dpts[-1].copy()).cuda(), n))
        off += P
    status = torch.full((3,), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_layerwise(G, src, jobs_s, status, host=host_tier)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0, 0]
    # sampled (block, group, page) records against the oracle
    rng = np.random.default_rng(w.seed(74))
    sv = _view(w, src)
    for _ in range(12):
        j, k = int(rng.integers(0, 3)), int(rng.integers(0, G))
        P = pages[j]
        p = int(rng.integers(0, P)) if rng.random() < 0.6 else P - 1
        t = min(T, lens[j] - p * T)
        page = sv[k * gl:(k + 1) * gl, :, int(spts[j][p])].contiguous().cpu().numpy().reshape(-1)
        blob, sums, code, _ = oracle.pack(og_group, oracle.Cache(page, 1, 2 * s, s, s), np.zeros(1, dtype=np.int32), t)
        assert code == 0
        hb, hs, gb = host[j]
        lo = k * gb + oracle.record_offset(og_group, p)
        assert np.array_equal(hb[lo:lo + blob.size].cpu().numpy(), blob), (j, k, p)
        assert int(hs[k * P + p].item()) & 0xFFFFFFFFFFFFFFFF == int(sums[0])
    # damage block 1 inside group 5, then load
    host[1][0][5 * host[1][2] + 1_000_003] ^= 0x20
    mask = torch.full((3,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((3,), -7, dtype=torch.int32, device="cuda")
    gm = torch.full((G, 3), 255, dtype=torch.uint8, device="cuda")
    seen = []
    ctx.gk_restore_layerwise(G, jobs_d, dst, mask, fb, gm, lambda k, l0, nl, st: seen.append((k, l0, nl)),
                             host=host_tier)
    torch.cuda.synchronize()
    assert seen == [(k, k * gl, gl) for k in range(G)]
    want_gm = [[0, 0, 0] for _ in range(G)]
    want_gm[5][1] = 1
    assert gm.cpu().tolist() == want_gm and mask.cpu().tolist() == [0, 1, 0]
    assert fb.cpu().tolist()[1] == 1_000_003 // oracle.record_bytes(og_group, 4096, 0)
    dv, zv = _view(w, dst), sentinel.view(w.layers, 2, Nd, T, -1)
    untouched = torch.ones(Nd, dtype=torch.bool, device="cuda")
    for j, (n, P) in enumerate(zip(lens, pages)):
        full = n // T
        s_idx = torch.from_numpy(spts[j][:full].astype(np.int64)).cuda()
        d_idx = torch.from_numpy(dpts[j][:full].astype(np.int64)).cuda()
        untouched[torch.from_numpy(dpts[j].astype(np.int64)).cuda()] = False
        for k in range(G):
            ls = slice(k * gl, (k + 1) * gl)
            if want_gm[k][j]:
                assert torch.equal(dv[ls][:, :, d_idx], zv[ls][:, :, d_idx])        # the failing group wrote nothing
            else:
                assert torch.equal(dv[ls][:, :, d_idx], sv[ls][:, :, s_idx])
        if full < P:
            t, sp, dp = n - full * T, int(spts[j][full]), int(dpts[j][full])
            assert torch.equal(dv[:, :, dp, :t], sv[:, :, sp, :t])
            assert torch.equal(dv[:, :, dp, t:], zv[:, :, dp, t:])
    rest = torch.nonzero(untouched).flatten()
    assert torch.equal(dv[:, :, rest], zv[:, :, rest])
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()
