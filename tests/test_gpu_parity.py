"""GPU parity: libgk (through its C ABI) against the CPU oracle, bit for bit --
blob bytes, page checksums, result codes, first failing page, and the full
destination cache image (so that "nothing written" is checked byte by byte).
Sizes here are small enough for the oracle to finish in seconds yet span
several 32 KiB granules, several segments and ragged tails."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import (cache_bytes, clone_cache, make_cache, n_pages, oracle_geom, random_cache)

pytestmark = pytest.mark.gpu

G_TINY = oracle.Geom(2, 2, 64, 16, 2, 0)           # record 16 KiB: half a granule
G_MID = oracle.Geom(5, 4, 64, 16, 2, 0)            # record 80 KiB: 2.5 granules
G_BIG = oracle.Geom(16, 8, 128, 16, 2, 0)          # record 1 MiB
G_FP8_S = oracle.Geom(6, 4, 32, 8, 1, 2)           # record 12,480 B, scale section 192 B
G_FP8_M = oracle.Geom(10, 8, 64, 32, 1, 2)         # record 328,320 B, scale section 640 B
G_FP8_1 = oracle.Geom(4, 4, 64, 16, 1, 1)          # shared K/V scale
G_FP8_W = oracle.Geom(40, 64, 16, 8, 1, 2)         # scale section 20,480 B: spans several tiles
ALL_GEOMS = [G_TINY, G_MID, G_BIG, G_FP8_S, G_FP8_M, G_FP8_1, G_FP8_W]


@pytest.fixture(scope="module")
def gk():
    import paper_2609_39358_b200 as m
    assert torch.cuda.is_available()
    return m


def _ctx(gk, og, flags=0, **tuning):
    from gpu_harness import gk_geom
    ctx = gk.Context(gk_geom(og, flags), 0)
    for k, v in tuning.items():
        ctx.set_tuning(k, v)
    return ctx


# ---------------------------------------------------------------------------
# checksums of an existing blob
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("og", ALL_GEOMS)
@pytest.mark.parametrize("seg", [0, 1, 2])
def test_page_checksums(gk, og, seg):
    from gpu_harness import sums_to_np
    ctx = _ctx(gk, og, seg_granules=seg)
    rng = np.random.default_rng(100 + seg)
    for n_tokens in [1, og.page_tokens, 3 * og.page_tokens + 1, 5 * og.page_tokens - 1]:
        nbytes, P = oracle.blob_size(og, n_tokens)
        blob = rng.integers(0, 256, size=nbytes, dtype=np.uint8)
        want = np.array([oracle.crc64(blob[oracle.record_offset(og, p):
                                           oracle.record_offset(og, p) + oracle.record_bytes(og, n_tokens, p)])
                         for p in range(P)], dtype=np.uint64)
        d_blob = torch.from_numpy(blob).cuda()
        d_sums = torch.zeros(P, dtype=torch.int64, device="cuda")
        ctx.gk_page_checksums(d_blob, n_tokens, d_sums)
        torch.cuda.synchronize()
        assert np.array_equal(sums_to_np(d_sums), want)
    ctx.close()


def test_page_checksums_special_contents(gk):
    """All-zero and all-ones records (the init and final-xor terms must be right
    even when the data contribute nothing), and the catalogue check string
    embedded at the very end of a record."""
    from gpu_harness import sums_to_np
    og = G_MID
    ctx = _ctx(gk, og)
    nbytes, P = oracle.blob_size(og, og.page_tokens)
    for fill in (0x00, 0xFF):
        blob = np.full(nbytes, fill, dtype=np.uint8)
        d_sums = torch.zeros(P, dtype=torch.int64, device="cuda")
        ctx.gk_page_checksums(torch.from_numpy(blob).cuda(), og.page_tokens, d_sums)
        torch.cuda.synchronize()
        assert int(sums_to_np(d_sums)[0]) == oracle.crc64(blob)
    blob = np.zeros(nbytes, dtype=np.uint8)
    blob[-9:] = np.frombuffer(b"123456789", dtype=np.uint8)
    d_sums = torch.zeros(P, dtype=torch.int64, device="cuda")
    ctx.gk_page_checksums(torch.from_numpy(blob).cuda(), og.page_tokens, d_sums)
    torch.cuda.synchronize()
    assert int(sums_to_np(d_sums)[0]) == oracle.crc64(blob)
    ctx.close()


# ---------------------------------------------------------------------------
# pack
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("og", ALL_GEOMS)
@pytest.mark.parametrize("layout", ["layer_major", "page_major"])
def test_pack_parity(gk, og, layout):
    from gpu_harness import dev_cache, gpu_pack
    N = 23
    src = random_cache(og, N, seed=200, layout=layout)
    dsrc = dev_cache(src)
    rng = np.random.default_rng(201)
    T = og.page_tokens
    lens = [1, T, T + 1, 4 * T, 6 * T - 1, 2 * T]
    tables = [rng.integers(0, N, size=n_pages(og, n)).astype(np.int32) for n in lens]   # duplicates allowed
    for seg in (0, 1):
        ctx = _ctx(gk, og, seg_granules=seg)
        got, status = gpu_pack(ctx, og, dsrc, tables, lens)
        assert status.tolist() == [0] * len(lens)
        for (blob, sums), pt, n in zip(got, tables, lens):
            wb, ws, code, _ = oracle.pack(og, src, pt, n)
            assert code == 0
            assert np.array_equal(blob, wb), f"blob differs at {np.flatnonzero(blob != wb)[:8]}"
            assert np.array_equal(sums, ws)
        ctx.close()


def test_pack_single_entry_point_and_bad_table(gk):
    from gpu_harness import dev_cache, dev_i32, sums_to_np
    og, N = G_MID, 9
    src = random_cache(og, N, seed=210)
    dsrc = dev_cache(src)
    ctx = _ctx(gk, og)
    n = 2 * og.page_tokens + 3
    nbytes, P = oracle.blob_size(og, n)
    pt = np.array([4, 0, 8], dtype=np.int32)
    blob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    sums = torch.zeros(P, dtype=torch.int64, device="cuda")
    status = torch.full((1,), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack(dsrc, dev_i32(pt), n, blob, sums, status)
    torch.cuda.synchronize()
    wb, ws, _, _ = oracle.pack(og, src, pt, n)
    assert status.item() == 0
    assert np.array_equal(blob.cpu().numpy(), wb) and np.array_equal(sums_to_np(sums), ws)
    # an id outside the cache: nothing written, status 2
    for bad_id in (-1, N):
        blob.fill_(0x5A)
        sums.fill_(0x5A5A)
        status.fill_(255)
        ctx.gk_pack(dsrc, dev_i32(np.array([4, bad_id, 8])), n, blob, sums, status)
        torch.cuda.synchronize()
        assert status.item() == 2
        assert bool((blob == 0x5A).all()) and bool((sums == 0x5A5A).all())
    ctx.close()


@pytest.mark.parametrize("og", [G_MID, G_FP8_M])
def test_pack_host_parity(gk, og):
    """Save to pinned host memory: same bytes and checksums as the oracle."""
    from gpu_harness import dev_cache, dev_i32
    N = 19
    src = random_cache(og, N, seed=220)
    dsrc = dev_cache(src)
    rng = np.random.default_rng(221)
    T = og.page_tokens
    lens = [3 * T + 2, 1, 5 * T, T]
    tables = [rng.integers(0, N, size=n_pages(og, n)).astype(np.int32) for n in lens]
    tables[2][1] = N + 5                                   # job 2: an id outside the cache
    ctx = _ctx(gk, og)
    jobs, keep = [], []
    for pt, n in zip(tables, lens):
        nbytes, P = oracle.blob_size(og, n)
        hb = torch.zeros(nbytes, dtype=torch.uint8).pin_memory()
        hs = torch.zeros(P, dtype=torch.int64).pin_memory()
        keep.append((hb, hs))
        jobs.append(gk.Job(hb, hs, dev_i32(pt), n))
    status = torch.full((len(jobs),), 255, dtype=torch.uint8, device="cuda")
    ctx.gk_pack_host(dsrc, jobs, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0, 2, 0]
    for i, (pt, n) in enumerate(zip(tables, lens)):
        if i == 2:
            continue
        wb, ws, code, _ = oracle.pack(og, src, pt, n)
        assert code == 0
        assert np.array_equal(keep[i][0].numpy(), wb)
        assert np.array_equal(keep[i][1].numpy().view(np.uint64), ws)
    # pageable outputs are refused
    with pytest.raises(gk.GkError) as e:
        ctx.gk_pack_host(dsrc, [gk.Job(torch.zeros(oracle.blob_size(og, 1)[0], dtype=torch.uint8),
                                       torch.zeros(1, dtype=torch.int64), dev_i32(np.zeros(1)), 1)], None)
    assert e.value.code == -3
    ctx.close()


# ---------------------------------------------------------------------------
# head-major slabs: partial pages are gathered / scattered head by head
# ---------------------------------------------------------------------------
HM_MID = oracle.Geom(5, 4, 64, 16, 2, 0, head_major=1)       # 128 B per token and head
HM_BIG = oracle.Geom(16, 8, 128, 16, 2, 0, head_major=1)     # chunks of t*256 B, 256 chunks per partial page
HM_FP8 = oracle.Geom(10, 8, 64, 32, 1, 2, head_major=1)      # 64 B per token and head, with scales
HM_MIN = oracle.Geom(3, 2, 8, 4, 2, 0, head_major=1)         # 16 B per token and head: the smallest allowed
HM_GEOMS = [HM_MID, HM_BIG, HM_FP8, HM_MIN]


@pytest.mark.parametrize("og", HM_GEOMS)
def test_head_major_pack_parity(gk, og):
    from gpu_harness import dev_cache, gpu_pack
    N = 19
    src = random_cache(og, N, seed=210)
    dsrc = dev_cache(src)
    rng = np.random.default_rng(211)
    T = og.page_tokens
    lens = [1, T - 1, T, T + 1, 3 * T + T // 2, 2 * T, 5 * T - 1]
    tables = [rng.integers(0, N, size=n_pages(og, n)).astype(np.int32) for n in lens]
    for seg in (0, 1):
        ctx = _ctx(gk, og, seg_granules=seg)
        got, status = gpu_pack(ctx, og, dsrc, tables, lens)
        assert status.tolist() == [0] * len(lens)
        for (blob, sums), pt, n in zip(got, tables, lens):
            wb, ws, code, _ = oracle.pack(og, src, pt, n)
            assert code == 0
            assert np.array_equal(blob, wb), f"blob differs at {np.flatnonzero(blob != wb)[:8]}"
            assert np.array_equal(sums, ws)
        ctx.close()


@pytest.mark.parametrize("og", HM_GEOMS)
@pytest.mark.parametrize("host_tier", [False, True])
def test_head_major_restore_parity(gk, og, host_tier):
    """Partial pages must land head by head and leave every head's tail as it was;
    a damaged block leaves everything as it was."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_restore
    T = og.page_tokens
    src = random_cache(og, 13, seed=310)
    lens = [2 * T + 1, 1, T - 1, 4 * T, 3 * T + T // 2, T + 2]
    Nd = 31
    jobs = _oracle_jobs(og, src, lens, 311, Nd)
    jobs[4].blob[-3] ^= 0x20                 # damage inside the partial page of job 4
    clean = random_cache(og, Nd, seed=312)
    for tuning in ({}, {"seg_granules": 1, "commit_seg_tiles": 1}, {"fused": 0}):
        ctx = _ctx(gk, og, **tuning)
        want = clone_cache(clean)
        wmask, wfb = oracle.restore(og, want, jobs)
        assert wmask.tolist() == [0, 0, 0, 0, 1, 0]
        d = dev_cache(clean)
        mask, fb = gpu_restore(ctx, d, jobs, host_tier=host_tier)
        assert mask.tolist() == wmask.tolist()
        assert fb.tolist() == wfb.tolist()
        assert_cache_equal(d, want)
        ctx.close()


def test_head_major_needs_16_byte_head_rows(gk):
    with pytest.raises(gk.GkError) as e:
        gk.gk_blob_size(gk.Geom(2, 4, 4, 16, gk.GK_BF16, 0, gk.GK_FLAG_HEAD_MAJOR), 16)   # 8 B per token and head
    assert e.value.code == -2
    assert gk.gk_blob_size(gk.Geom(2, 4, 4, 16, gk.GK_BF16, 0, 0), 16)[1] == 1            # fine token-major


# ---------------------------------------------------------------------------
# restore
# ---------------------------------------------------------------------------
def _oracle_jobs(og, src, lens, seed, dst_pages):
    rng = np.random.default_rng(seed)
    perm = rng.permutation(dst_pages).astype(np.int32)
    jobs, used = [], 0
    for n in lens:
        P = n_pages(og, n)
        spt = rng.integers(0, src.num_pages, size=P).astype(np.int32)
        blob, sums, code, _ = oracle.pack(og, src, spt, n)
        assert code == 0
        jobs.append(oracle.Job(blob, sums, perm[used:used + P].copy(), n))
        used += P
    assert used <= dst_pages
    return jobs


@pytest.mark.parametrize("og", ALL_GEOMS)
@pytest.mark.parametrize("host_tier", [False, True])
def test_restore_parity_with_corruption(gk, og, host_tier):
    from gpu_harness import assert_cache_equal, dev_cache, gpu_restore
    T = og.page_tokens
    src = random_cache(og, 17, seed=300)
    lens = [3 * T, 1, 2 * T + 1, 5 * T, T, 4 * T - 1]
    Nd = 40
    jobs = _oracle_jobs(og, src, lens, 301, Nd)
    # job 1: one flipped bit in the blob; job 3: one flipped bit in a checksum;
    # job 5: damage in the last (partial) page only
    jobs[1].blob[len(jobs[1].blob) // 2] ^= 0x10
    jobs[3].checksums[2] ^= np.uint64(1 << 40)
    jobs[5].blob[-1] ^= 0x01
    clean = random_cache(og, Nd, seed=302)
    for tuning in ({}, {"seg_granules": 1, "commit_seg_tiles": 1}, {"grid_cap": 3}):
        ctx = _ctx(gk, og, **tuning)
        want = clone_cache(clean)
        wmask, wfb = oracle.restore(og, want, jobs)
        assert wmask.tolist() == [0, 1, 0, 1, 0, 1]
        d = dev_cache(clean)
        mask, fb = gpu_restore(ctx, d, jobs, host_tier=host_tier)
        assert mask.tolist() == wmask.tolist()
        assert fb.tolist() == wfb.tolist()
        assert_cache_equal(d, want)
        ctx.close()


# ---------------------------------------------------------------------------
# streaming restore through a ring of pages
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("og", [G_MID, G_FP8_M, HM_MID])
@pytest.mark.parametrize("ring_pages", [6, 9, 64])
def test_stream_restore_parity(gk, og, ring_pages):
    """Window by window: same windows, same ring image after every window, same codes.
    The consumer also packs every block back out of the ring through the page table it
    was handed, which must give the saved blob again."""
    from gpu_harness import dev_cache, sums_to_np
    T = og.page_tokens
    src = random_cache(og, 17, seed=320)
    rng = np.random.default_rng(321)
    lens = [2 * T, 1, 3 * T + 1, T, 6 * T, 2 * T - 1, T + 1, 4 * T, 1, 3 * T, 5 * T + 2]
    ojobs = []
    for n in lens:
        spt = rng.integers(0, src.num_pages, size=n_pages(og, n)).astype(np.int32)
        blob, sums, code, _ = oracle.pack(og, src, spt, n)
        assert code == 0
        ojobs.append(oracle.Job(blob, sums, None, n))
    pristine = [jb.blob.copy() for jb in ojobs]
    ojobs[3].blob[7] ^= 0x04
    ojobs[7].checksums[1] ^= np.uint64(2)
    ojobs[8] = oracle.Job(None, None, None, lens[8])
    bad = {3, 7, 8}
    clean = random_cache(og, ring_pages, seed=322)

    want_ring = clone_cache(clean)
    owin = []

    def oconsume(first, count, first_pages):
        owin.append((first, count, first_pages, want_ring.data.copy(),
                     None if want_ring.scales is None else want_ring.scales.copy()))

    wmask, wfb = oracle.restore_stream(og, want_ring, ojobs, oconsume)
    assert [int(m) for m in wmask] == [1 if j in (3, 7) else 3 if j == 8 else 0 for j in range(len(lens))]

    ctx, ctx2 = _ctx(gk, og), _ctx(gk, og)
    d = dev_cache(clean)
    jobs, keep = [], []
    for jb in ojobs:
        hb = None if jb.blob is None else torch.from_numpy(jb.blob).pin_memory()
        hs = None if jb.checksums is None else torch.from_numpy(jb.checksums.view(np.int64).copy()).pin_memory()
        keep.append((hb, hs))
        jobs.append(gk.Job(hb, hs, None, jb.n_tokens))
    mask = torch.full((len(jobs),), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((len(jobs),), -7, dtype=torch.int32, device="cuda")
    gwin = []

    def consume(blocks, st):
        assert st == torch.cuda.current_stream().cuda_stream
        packed = []
        for b in blocks:
            nbytes, P = oracle.blob_size(og, b.n_tokens)
            ob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
            os_ = torch.zeros(P, dtype=torch.int64, device="cuda")
            ctx2.gk_pack_batch(d, [gk.Job(ob, os_, b.page_table, b.n_tokens)])
            packed.append((b.job, ob, os_))
        gwin.append(([b.job for b in blocks], [b.page_table for b in blocks], d.data.clone(),
                     None if d.scales is None else d.scales.clone(), packed))

    ctx.gk_restore_stream(jobs, d, mask, fb, consume)
    torch.cuda.synchronize()
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    assert mask.cpu().tolist() == wmask.tolist()
    assert fb.cpu().tolist() == wfb.tolist()
    assert len(gwin) == len(owin)
    for (first, count, first_pages, odata, oscales), (gjobs, gtables, gdata, gscales, packed) in zip(owin, gwin):
        assert gjobs == list(range(first, first + count))
        assert [(a - gtables[0]) // 4 for a in gtables] == first_pages
        assert np.array_equal(gdata.cpu().numpy(), odata)
        if oscales is not None:
            assert np.array_equal(gscales.cpu().numpy(), oscales)
        for j, ob, os_ in packed:
            if j in bad:
                continue
            assert np.array_equal(ob.cpu().numpy(), pristine[j])
            assert np.array_equal(sums_to_np(os_), ojobs[j].checksums)
    if ring_pages == 64:
        assert len(gwin) == 1
    ctx.close()
    ctx2.close()


def test_stream_restore_on_a_side_stream_and_refusals(gk):
    from gpu_harness import assert_cache_equal, dev_cache
    og = G_MID
    T = og.page_tokens
    src = random_cache(og, 9, seed=330)
    lens = [3 * T, 2 * T + 1, 4 * T, T]
    ojobs = []
    for i, n in enumerate(lens):
        blob, sums, code, _ = oracle.pack(og, src, np.arange(n_pages(og, n), dtype=np.int32) + i, n)
        ojobs.append(oracle.Job(blob, sums, None, n))
    clean = random_cache(og, 5, seed=331)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore_stream(og, want, ojobs)
    ctx = _ctx(gk, og)
    d = dev_cache(clean)
    keep = [(torch.from_numpy(j.blob).pin_memory(), torch.from_numpy(j.checksums.view(np.int64).copy()).pin_memory())
            for j in ojobs]
    jobs = [gk.Job(b, s, None, j.n_tokens) for (b, s), j in zip(keep, ojobs)]
    mask = torch.full((4,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((4,), -7, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    seen = []
    with torch.cuda.stream(side):
        ctx.gk_restore_stream(jobs, d, mask, fb, lambda blocks, st: seen.append((len(blocks), st)))
    side.synchronize()
    h = side.cuda_stream
    assert seen == [(1, h), (1, h), (2, h)]            # pages 3 | 3 | 4 + 1 through a 5-page ring
    assert mask.cpu().tolist() == wmask.tolist() == [0, 0, 0, 0]
    assert_cache_equal(d, want)                        # the final image: what the last window left
    assert ctx.gk_get_stats()["calls_restore_stream"] == 1

    # a job that alone does not fit: refused before anything runs
    d2 = dev_cache(clean)
    big, bs, _, _ = oracle.pack(og, src, np.arange(6, dtype=np.int32), 6 * T)
    hb, hs = torch.from_numpy(big).pin_memory(), torch.from_numpy(bs.view(np.int64).copy()).pin_memory()
    with pytest.raises(gk.GkError) as e:
        ctx.gk_restore_stream([jobs[0], gk.Job(hb, hs, None, 6 * T)], d2, mask, fb)
    assert e.value.code == -7
    torch.cuda.synchronize()
    assert_cache_equal(d2, clean)
    # an exception in the consumer surfaces after the call
    def boom(blocks, st):
        raise KeyError("consumer failed")
    with pytest.raises(KeyError):
        ctx.gk_restore_stream(jobs[:1], d2, mask, fb, boom)
    torch.cuda.synchronize()
    ctx.close()


def test_job_array_marshalled_once_gives_the_same_result(gk):
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, sums_to_dev
    og = G_MID
    T = og.page_tokens
    src = random_cache(og, 9, seed=340)
    ojobs = _oracle_jobs(og, src, [2 * T, T + 3, 1], 341, 12)
    clean = random_cache(og, 12, seed=342)
    want = clone_cache(clean)
    wmask, _ = oracle.restore(og, want, ojobs)
    ctx = _ctx(gk, og)
    jobs = gk.JobArray([gk.Job(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table), j.n_tokens)
                        for j in ojobs])
    assert len(jobs) == 3 and jobs[1].n_tokens == T + 3
    for _ in range(3):                                   # the same marshalled array, call after call
        d = dev_cache(clean)
        mask = torch.full((3,), 255, dtype=torch.uint8, device="cuda")
        fb = torch.full((3,), -7, dtype=torch.int32, device="cuda")
        ctx.gk_restore(jobs, d, mask, fb)
        torch.cuda.synchronize()
        assert mask.cpu().tolist() == wmask.tolist()
        assert_cache_equal(d, want)
    ctx.close()


# ---------------------------------------------------------------------------
# single-pass restore (GK_FLAG_SINGLE_PASS)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("og", ALL_GEOMS + [HM_MID, HM_FP8])
@pytest.mark.parametrize("host_tier", [False, True])
def test_single_pass_restore_parity(gk, og, host_tier):
    """Same report as the two-phase restore; the pages of a block that fails only its checksum
    hold the unverified bytes, everything else is byte-identical to the strict result."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_restore
    T = og.page_tokens
    src = random_cache(og, 17, seed=350)
    lens = [3 * T, 1, 2 * T + 1, 5 * T, T, 4 * T - 1, 2 * T]
    Nd = 44
    jobs = _oracle_jobs(og, src, lens, 351, Nd)
    jobs[1].blob[len(jobs[1].blob) // 2] ^= 0x10           # checksum failure
    jobs[3].checksums[2] ^= np.uint64(1 << 40)             # checksum failure (damaged checksum)
    jobs[4] = oracle.Job(None, None, jobs[4].page_table, T)  # missing
    jobs[5].page_table[1] = jobs[0].page_table[0]          # page claimed twice: jobs 0 and 5 write nothing
    clean = random_cache(og, Nd, seed=352)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs, flags=oracle.FLAG_SINGLE_PASS)
    assert wmask.tolist() == [2, 1, 0, 1, 3, 2, 0]
    strict = clone_cache(clean)
    smask, sfb = oracle.restore(og, strict, jobs)
    assert smask.tolist() == wmask.tolist() and sfb.tolist() == wfb.tolist()
    assert not np.array_equal(strict.data, want.data)
    for tuning in ({}, {"seg_granules": 1}, {"grid_cap": 3}):
        ctx = _ctx(gk, og, flags=gk.GK_FLAG_SINGLE_PASS, **tuning)
        d = dev_cache(clean)
        mask, fb = gpu_restore(ctx, d, jobs, host_tier=host_tier)
        assert mask.tolist() == wmask.tolist()
        assert fb.tolist() == wfb.tolist()
        assert_cache_equal(d, want)
        ctx.close()


def test_restore_host_is_ordered_after_earlier_work_on_the_stream(gk):
    """The pinned blob is still being filled by an asynchronous copy on the caller's stream
    when gk_restore_host is called: its copies must wait for that work."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32
    og = G_BIG                                             # 1 MiB records
    T = og.page_tokens
    n = 96 * T                                             # a 96 MiB blob: the fill takes milliseconds
    src = random_cache(og, 96, seed=360)
    spt = np.random.default_rng(361).permutation(96).astype(np.int32)
    blob, sums, code, _ = oracle.pack(og, src, spt, n)
    assert code == 0
    dpt = np.random.default_rng(362).permutation(100).astype(np.int32)[:96]
    clean = random_cache(og, 100, seed=363)
    want = clone_cache(clean)
    wmask, _ = oracle.restore(og, want, [oracle.Job(blob, sums, dpt, n)])
    assert wmask.tolist() == [0]
    ctx = _ctx(gk, og)
    d = dev_cache(clean)
    d_blob = torch.from_numpy(blob).cuda()
    d_sums = torch.from_numpy(sums.view(np.int64).copy()).cuda()
    h_blob = torch.zeros(blob.size, dtype=torch.uint8).pin_memory()        # zeros: a premature copy fails its checksums
    h_sums = torch.zeros(sums.size, dtype=torch.int64).pin_memory()
    mask = torch.full((1,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    h_blob.copy_(d_blob, non_blocking=True)                # device -> pinned host, on the current stream
    h_sums.copy_(d_sums, non_blocking=True)
    ctx.gk_restore_host([gk.Job(h_blob, h_sums, dev_i32(dpt), n)], d, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == [0]
    assert_cache_equal(d, want)
    ctx.close()


def test_small_calls_replay_from_a_cuda_graph(gk):
    """A small save + restore captured once and replayed: every replay does the real work
    (the work-item counters start from zero in every call), so damage done to the source
    cache or to a blob between replays shows up exactly as in a direct call."""
    from gpu_harness import dev_cache, dev_i32
    og = G_MID
    T = og.page_tokens
    lens = [2 * T + 3, T, 3 * T]
    src = random_cache(og, 9, seed=370)
    rng = np.random.default_rng(371)
    tables = [rng.integers(0, 9, size=n_pages(og, n)).astype(np.int32) for n in lens]
    Nd = 12
    dperm = rng.permutation(Nd).astype(np.int32)
    clean = random_cache(og, Nd, seed=372)
    ctx = _ctx(gk, og)
    dsrc, ddst = dev_cache(src), dev_cache(clean)
    pack_jobs, restore_jobs, used = [], [], 0
    for pt, n in zip(tables, lens):
        nbytes, P = oracle.blob_size(og, n)
        blob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        sums = torch.zeros(P, dtype=torch.int64, device="cuda")
        pack_jobs.append(gk.Job(blob, sums, dev_i32(pt), n))
        restore_jobs.append(gk.Job(blob, sums, dev_i32(dperm[used:used + P]), n))
        used += P
    pack_jobs, restore_jobs = gk.JobArray(pack_jobs), gk.JobArray(restore_jobs)
    status = torch.full((3,), 255, dtype=torch.uint8, device="cuda")
    mask = torch.full((3,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((3,), -7, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                       # warm-up outside the capture: workspace allocation
        ctx.gk_pack_batch(dsrc, pack_jobs, status)
        ctx.gk_restore(restore_jobs, ddst, mask, fb)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        ctx.gk_pack_batch(dsrc, pack_jobs, status)
        ctx.gk_restore(restore_jobs, ddst, mask, fb)

    def expect(src_cache):
        ojobs, used = [], 0
        for pt, n in zip(tables, lens):
            b, s_, code, _ = oracle.pack(og, src_cache, pt, n)
            assert code == 0
            P = n_pages(og, n)
            ojobs.append(oracle.Job(b, s_, dperm[used:used + P].copy(), n))
            used += P
        want = clone_cache(clean)
        wmask, _ = oracle.restore(og, want, ojobs)
        return ojobs, want, wmask

    for round_ in range(4):
        if round_ % 2 == 1:                             # new cache contents: the replay must save and restore them
            src = random_cache(og, 9, seed=373 + round_)
            dsrc.data.copy_(torch.from_numpy(src.data))
        ddst.data.copy_(torch.from_numpy(clean.data))
        mask.fill_(255)
        graph.replay()
        torch.cuda.synchronize()
        ojobs, want, wmask = expect(src)
        assert status.cpu().tolist() == [0, 0, 0] and mask.cpu().tolist() == wmask.tolist() == [0, 0, 0]
        for jb, oj in zip(pack_jobs.jobs, ojobs):
            assert np.array_equal(jb.blob.cpu().numpy(), oj.blob)
            assert np.array_equal(jb.checksums.cpu().numpy().view(np.uint64), oj.checksums)
        assert np.array_equal(ddst.data.cpu().numpy(), want.data)
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_restore_codes_and_first_bad_page(gk):
    from gpu_harness import assert_cache_equal, dev_cache, gpu_restore
    og, N = G_MID, 12
    src = random_cache(og, N, seed=310)
    T = og.page_tokens
    n = 3 * T
    blob, sums, _, _ = oracle.pack(og, src, np.array([0, 1, 2], dtype=np.int32), n)
    blob1, sums1, _, _ = oracle.pack(og, src, np.array([0], dtype=np.int32), 1)
    bad2 = blob.copy()
    bad2[oracle.record_offset(og, 1) + 5] ^= 1
    bad2[oracle.record_offset(og, 2) + 5] ^= 1
    clean = random_cache(og, N, seed=311)
    i32 = lambda *v: np.array(v, dtype=np.int32)
    jobs = [
        oracle.Job(blob, sums, i32(0, 1, 2), n),
        oracle.Job(bad2, sums, i32(3, 4, 5), n),
        oracle.Job(None, sums, i32(6, 7, 8), n),
        oracle.Job(blob, None, i32(6, 7, 8), n),
        oracle.Job(blob, sums, i32(9, 12, -1), n),
        oracle.Job(blob, sums, i32(6, 10, 11), n),
        oracle.Job(blob, sums, i32(8, 7, 10), n),
        oracle.Job(blob1, sums1, i32(9), 1),
    ]
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs)
    assert wmask.tolist() == [0, 1, 3, 3, 2, 2, 2, 0]
    ctx = _ctx(gk, og)
    for host_tier in (False, True):
        d = dev_cache(clean)
        mask, fb = gpu_restore(ctx, d, jobs, host_tier=host_tier)
        assert mask.tolist() == wmask.tolist()
        assert fb.tolist() == wfb.tolist()
        assert_cache_equal(d, want)
    # a page claimed twice inside one job, and by three jobs
    jobs2 = [
        oracle.Job(blob, sums, i32(0, 1, 0), n),
        oracle.Job(blob, sums, i32(2, 3, 4), n),
        oracle.Job(blob, sums, i32(5, 4, 6), n),
        oracle.Job(blob, sums, i32(7, 8, 4), n),
        oracle.Job(blob, sums, i32(9, 10, 11), n),
    ]
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs2)
    assert wmask.tolist() == [2, 2, 2, 2, 0] and wfb.tolist() == [0, 2, 1, 2, -1]
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, jobs2)
    assert mask.tolist() == wmask.tolist() and fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    ctx.close()


def test_sabotage_triple_on_gpu(gk):
    """Defence on: rejected and untouched.  Defence off: the damaged bytes land.
    Defence on again: rejected and untouched."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_restore
    og = G_MID
    src = random_cache(og, 8, seed=320)
    n = 2 * og.page_tokens + 5
    jobs = _oracle_jobs(og, src, [n], 321, 8)
    jobs[0].blob[12345] ^= 0x80
    clean = random_cache(og, 8, seed=322)
    for flags, want_code in ((0, 1), (oracle.FLAG_SKIP_VERIFY, 0), (0, 1)):
        ctx = _ctx(gk, og, flags=flags)
        want = clone_cache(clean)
        wmask, _ = oracle.restore(og, want, jobs, flags=flags)
        assert wmask.tolist() == [want_code]
        d = dev_cache(clean)
        mask, _ = gpu_restore(ctx, d, jobs)
        assert mask.tolist() == [want_code]
        assert_cache_equal(d, want)
        changed = not np.array_equal(want.data, clean.data)
        assert changed == (want_code == 0)
        ctx.close()


def test_tiny_workload(gk):
    """4 blocks of 256 tokens, one flipped bit: 3 ok, 1 rejected with its pages untouched."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_pack, gpu_restore
    w = synth.TINY
    og = oracle_geom(w)
    src_pages = 64
    src = make_cache(og, src_pages,
                     synth.kv_bytes_bf16(cache_bytes(og, src_pages) // 2, w.sigma, w.seed(0)).numpy())
    dsrc = dev_cache(src)
    ctx = _ctx(gk, og)
    tables = [np.arange(16 * i, 16 * i + 16, dtype=np.int32) for i in range(4)]
    packed, status = gpu_pack(ctx, og, dsrc, tables, synth.TINY_BLOCKS)
    assert status.tolist() == [0, 0, 0, 0]
    perm = synth.page_permutation(synth.TINY_DST_PAGES, w.seed(1))
    jobs = []
    for i, ((blob, sums), n) in enumerate(zip(packed, synth.TINY_BLOCKS)):
        wb, ws, _, _ = oracle.pack(og, src, tables[i], n)
        assert np.array_equal(blob, wb) and np.array_equal(sums, ws)
        jobs.append(oracle.Job(blob.copy(), sums.copy(), perm[16 * i:16 * i + 16], n))
    victim = int(np.random.default_rng(w.seed(2)).integers(0, 4))
    bit = int(synth.bit_flip_positions(jobs[victim].blob.size * 8, 1, w.seed(3))[0])
    jobs[victim].blob[bit >> 3] ^= 1 << (bit & 7)
    clean = make_cache(og, synth.TINY_DST_PAGES,
                       synth.sentinel_bytes(cache_bytes(og, synth.TINY_DST_PAGES), w.seed(4)).numpy().copy())
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs)
    assert sorted(wmask.tolist()) == [0, 0, 0, 1]
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, jobs)
    assert mask.tolist() == wmask.tolist() and fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    ctx.close()


def test_fp8_scale_and_data_corruption(gk):
    """A run of damaged bytes inside a scale section of one blob and inside a K
    slab of another: both rejected, their pages and scale entries untouched."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_restore
    og = G_FP8_M
    T = og.page_tokens
    Ns = 12
    data, scales = synth.kv_bytes_fp8(og.layers, Ns, T, og.kv_heads, og.head_dim, 1.0, synth.FP8.seed(0))
    src = make_cache(og, Ns, data.numpy().copy(), scales.view(torch.uint8).reshape(-1).numpy().copy())
    lens = [2 * T] * 5
    jobs = _oracle_jobs(og, src, lens, 331, 16)
    S = og.layers * og.scale_kv * og.kv_heads * 4
    rec = oracle.record_bytes(og, 2 * T, 0)
    start, xors = synth.byte_run_corruption(rec, rec + S, 8, synth.FP8.seed(1))       # scale section of page 1
    jobs[1].blob[start:start + 8] ^= xors
    start, xors = synth.byte_run_corruption(S, S + T * og.kv_heads * og.head_dim, 8, synth.FP8.seed(2))  # K slab, layer 0, page 0
    jobs[3].blob[start:start + 8] ^= xors
    clean = random_cache(og, 16, seed=332)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs)
    assert wmask.tolist() == [0, 1, 0, 1, 0] and wfb.tolist() == [-1, 1, -1, 0, -1]
    ctx = _ctx(gk, og)
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, jobs)
    assert mask.tolist() == wmask.tolist() and fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    ctx.close()


def test_round_trip_on_gpu_only_path(gk):
    """restore(pack(x)) == x through libgk alone, then checked against the source bytes."""
    from gpu_harness import dev_cache, dev_i32
    og = G_BIG
    N = 24
    src = random_cache(og, N, seed=340)
    dsrc = dev_cache(src)
    ctx = _ctx(gk, og)
    n = 10 * og.page_tokens + 7
    P = n_pages(og, n)
    nbytes, _ = oracle.blob_size(og, n)
    spt = np.random.default_rng(341).permutation(N)[:P].astype(np.int32)
    dpt = np.random.default_rng(342).permutation(N)[:P].astype(np.int32)
    blob = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    sums = torch.zeros(P, dtype=torch.int64, device="cuda")
    ctx.gk_pack(dsrc, dev_i32(spt), n, blob, sums)
    clean = random_cache(og, N, seed=343)
    d = dev_cache(clean)
    mask = torch.full((1,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.gk_restore([gk.Job(blob, sums, dev_i32(dpt), n)], d, mask, fb)
    torch.cuda.synchronize()
    assert mask.item() == 0 and fb.item() == -1
    L, T = og.layers, og.page_tokens
    got = d.data.cpu().numpy().reshape(L, 2, N, T, -1)
    s = src.data.reshape(L, 2, N, T, -1)
    c = clean.data.reshape(L, 2, N, T, -1)
    touched = np.zeros(N, dtype=bool)
    for p in range(P):
        t = min(T, n - p * T)
        assert np.array_equal(got[:, :, dpt[p], :t], s[:, :, spt[p], :t])
        assert np.array_equal(got[:, :, dpt[p], t:], c[:, :, dpt[p], t:])
        touched[dpt[p]] = True
    assert np.array_equal(got[:, :, ~touched], c[:, :, ~touched])
    ctx.close()


def test_verify_then_commit_matches_restore(gk):
    """gk_verify writes nothing and reports what gk_restore would; gk_commit with that
    mask produces gk_restore's destination; a job failed from outside (another rank's
    verdict) is not committed."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, sums_to_dev
    from paper_2609_39358_b200 import tp
    og = G_FP8_M
    T = og.page_tokens
    src = random_cache(og, 9, seed=380)
    jobs = _oracle_jobs(og, src, [2 * T, T + 3, 3 * T, 1], 381, 20)
    jobs[1].blob[77] ^= 0x02
    used = set(int(x) for j in jobs for x in j.page_table)
    free_page = next(g for g in range(20) if g not in used)
    jobs.append(oracle.Job(jobs[0].blob, jobs[0].checksums, np.array([free_page, 25], dtype=np.int32), 2 * T))  # id 25 out of range
    clean = random_cache(og, 20, seed=382)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs)
    assert wmask.tolist() == [0, 1, 0, 0, 2]
    ctx = _ctx(gk, og)
    keep = [(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table)) for j in jobs]
    gjobs = [gk.Job(b, s, t, j.n_tokens) for (b, s, t), j in zip(keep, jobs)]
    d = dev_cache(clean)
    mask = torch.full((5,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(5, dtype=torch.int32, device="cuda")
    ctx.gk_verify(gjobs, d, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == wmask.tolist() and fb.cpu().tolist() == wfb.tolist()
    assert_cache_equal(d, clean)                               # verify commits nothing
    ctx.gk_commit(gjobs, d, mask)
    torch.cuda.synchronize()
    assert_cache_equal(d, want)
    # another rank rejected job 2: with the merged mask it must stay out
    d = dev_cache(clean)
    merged = mask.clone()
    merged[2] = 1
    ctx.gk_commit(gjobs, d, merged)
    torch.cuda.synchronize()
    want2 = clone_cache(clean)
    oracle.restore(og, want2, [jobs[0], jobs[3]])
    assert_cache_equal(d, want2)
    # a mask that claims "ok" for the job with the bad table does not get it written
    d = dev_cache(clean)
    ctx.gk_commit(gjobs, d, torch.zeros(5, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    got = d.data.cpu().numpy().reshape(og.layers, 2, 20, T, -1)
    c = clean.data.reshape(og.layers, 2, 20, T, -1)
    assert np.array_equal(got[:, :, free_page], c[:, :, free_page])
    # single-rank tp_restore is verify + commit
    d = dev_cache(clean)
    mask.fill_(255)
    tp.tp_restore(ctx, gjobs, d, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == wmask.tolist()
    assert_cache_equal(d, want)
    ctx.close()


def test_device_wait_time_out_is_fail_closed(gk):
    """Failure detection without a GPU fault: the commit side's bounded wait for
    "all pages of the job verified" is made to run out (test hook: nothing gets
    verified, limit 50 ms).  The kernel must return by itself, report code 4 for
    every job, write nothing, and leave the context refusing to commit until the
    error is cleared; after gk_ctx_clear_error the SAME context restores the same
    jobs correctly."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, sums_to_dev
    og = G_MID
    src = random_cache(og, 8, seed=360)
    jobs = _oracle_jobs(og, src, [3 * og.page_tokens, og.page_tokens + 1], 361, 12)
    clean = random_cache(og, 12, seed=362)
    ctx = _ctx(gk, og, wait_limit_ms=50, test_drop_verify=1)
    d = dev_cache(clean)
    keep = [(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table)) for j in jobs]
    gjobs = [gk.Job(b, s, t, j.n_tokens) for (b, s, t), j in zip(keep, jobs)]
    mask = torch.full((2,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(2, dtype=torch.int32, device="cuda")
    ctx.gk_restore(gjobs, d, mask, fb)
    torch.cuda.synchronize()                       # returns: the wait was bounded
    assert mask.cpu().tolist() == [4, 4] and fb.cpu().tolist() == [-1, -1]
    assert_cache_equal(d, clean)
    assert ctx.gk_get_stats()["device_wait_expired"] != 0
    # the error is sticky: with the hook off the same context still commits nothing
    ctx.set_tuning("test_drop_verify", 0)
    mask.fill_(255)
    ctx.gk_restore(gjobs, d, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == [4, 4]
    assert_cache_equal(d, clean)
    # the unfused path (separate verify and commit launches) refuses as well
    ctx.set_tuning("fused", 0)
    mask.fill_(255)
    ctx.gk_restore(gjobs, d, mask, fb)
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == [4, 4]
    assert_cache_equal(d, clean)
    ctx.set_tuning("fused", 1)
    # cleared: the same context commits the same jobs, bit-exact
    want = clone_cache(clean)
    wmask, _ = oracle.restore(og, want, jobs)
    ctx.gk_ctx_clear_error()
    mask.fill_(255)
    ctx.gk_restore(gjobs, d, mask, fb)
    torch.cuda.synchronize()
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    assert mask.cpu().tolist() == wmask.tolist() == [0, 0]
    assert_cache_equal(d, want)
    ctx.close()


def test_partial_time_out_commits_whole_jobs_or_nothing(gk):
    """A wait that runs out for SOME jobs of a fused restore: the hook leaves the jobs
    from index 3 on unverified (limit 50 ms, no fault, no hang).  The jobs before them
    have verified and must be committed whole with code 0 -- the decision of a job is
    taken once and does not change when another job's wait runs out later -- and the
    others must report code 4 with not one byte written.  Several segments and commit
    items per page, so that every job's items are spread over many CTAs."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, sums_to_dev
    og = G_BIG
    T = og.page_tokens
    lens = [5 * T, 2 * T + 3, 7 * T, 4 * T, 3 * T + 1, 6 * T]
    n_pages = sum(-(-n // T) for n in lens)
    src = random_cache(og, n_pages, seed=370)
    jobs = _oracle_jobs(og, src, lens, 371, n_pages + 6)
    jobs[1].blob[12345] ^= 0x40                     # a job that verified as damaged keeps its code 1
    clean = random_cache(og, n_pages + 6, seed=372)
    # expectation: the oracle's result for the jobs that were verified, nothing for the rest
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs[:3])
    assert wmask.tolist() == [0, 1, 0]
    for seg, cst in ((0, 0), (1, 2)):
        ctx = _ctx(gk, og, wait_limit_ms=50, test_drop_verify=4, seg_granules=seg, commit_seg_tiles=cst)
        d = dev_cache(clean)
        keep = [(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table)) for j in jobs]
        gjobs = [gk.Job(b, s, t, j.n_tokens) for (b, s, t), j in zip(keep, jobs)]
        mask = torch.full((6,), 255, dtype=torch.uint8, device="cuda")
        fb = torch.full((6,), -9, dtype=torch.int32, device="cuda")
        ctx.gk_restore(gjobs, d, mask, fb)
        torch.cuda.synchronize()
        assert mask.cpu().tolist() == [0, 1, 0, 4, 4, 4]
        assert fb.cpu().tolist() == wfb.tolist() + [-1, -1, -1]
        assert_cache_equal(d, want)
        assert ctx.gk_get_stats()["device_wait_expired"] != 0
        ctx.close()


def test_one_segment_per_page_on_1_mib_records(gk):
    """The tiling every full-size call takes -- a whole page record as ONE checksum segment
    (many tiles per work item, no segment merge) -- forced on a small case of 1 MiB records
    and compared in full: pack, checksums alone, verify + commit as separate calls, and the
    fused restore, with damage in a full page and in the short last page."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, gpu_pack, gpu_restore, sums_to_dev
    og = oracle.Geom(16, 8, 128, 16)               # 64 KiB per token, 1 MiB per full page record
    T = og.page_tokens
    assert oracle.record_bytes(og, 4 * T, 0) == 1 << 20
    lens = [3 * T + 5, 2 * T, T + 15]
    total = sum(n_pages(og, n) for n in lens)
    src = random_cache(og, total + 2, seed=380)
    rng = np.random.default_rng(381)
    tables = [rng.integers(0, total + 2, size=n_pages(og, n)).astype(np.int32) for n in lens]
    granules = (1 << 20) // 32768
    for seg in (granules, 2 * granules):           # exactly one record, and "longer than any record"
        ctx = _ctx(gk, og, seg_granules=seg)
        got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
        assert status.tolist() == [0, 0, 0]
        ojobs, perm, used = [], rng.permutation(total + 3).astype(np.int32), 0
        for (blob, sums), pt, n in zip(got, tables, lens):
            wb, ws, code, _ = oracle.pack(og, src, pt, n)
            assert code == 0 and np.array_equal(blob, wb) and np.array_equal(sums, ws)
            # the checksums alone, from the blob
            sums2 = torch.zeros(ws.size, dtype=torch.int64, device="cuda")
            ctx.gk_page_checksums(torch.from_numpy(wb).cuda(), n, sums2)
            torch.cuda.synchronize()
            assert np.array_equal(sums2.cpu().numpy().view(np.uint64), ws)
            P = n_pages(og, n)
            ojobs.append(oracle.Job(wb.copy(), ws.copy(), perm[used:used + P].copy(), n))
            used += P
        ojobs[0].blob[oracle.record_offset(og, 3) + 77] ^= 0x01      # in the 5-token last page of job 0
        ojobs[2].blob[(1 << 20) - 1] ^= 0x80                          # last byte of a full page of job 2
        clean = random_cache(og, total + 3, seed=382)
        want = clone_cache(clean)
        wmask, wfb = oracle.restore(og, want, ojobs)
        assert wmask.tolist() == [1, 0, 1] and wfb.tolist() == [3, -1, 0]
        for host_tier in (False, True):
            d = dev_cache(clean)
            mask, fb = gpu_restore(ctx, d, ojobs, host_tier=host_tier)
            assert mask.tolist() == wmask.tolist() and fb.tolist() == wfb.tolist()
            assert_cache_equal(d, want)
        # the two halves as separate calls (verify-only kernel, then commit-only kernel)
        d = dev_cache(clean)
        keep = [(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table)) for j in ojobs]
        gjobs = [gk.Job(b, s_, t, j.n_tokens) for (b, s_, t), j in zip(keep, ojobs)]
        mask = torch.full((3,), 255, dtype=torch.uint8, device="cuda")
        fb = torch.full((3,), -9, dtype=torch.int32, device="cuda")
        ctx.gk_verify(gjobs, d, mask, fb)
        torch.cuda.synchronize()
        assert mask.cpu().tolist() == wmask.tolist() and fb.cpu().tolist() == wfb.tolist()
        assert_cache_equal(d, clean)
        ctx.gk_commit(gjobs, d, mask)
        torch.cuda.synchronize()
        assert_cache_equal(d, want)
        assert ctx.gk_get_stats()["device_wait_expired"] == 0
        ctx.close()


@pytest.mark.parametrize("n_jobs", [65, 96])
def test_device_tier_call_of_many_tiny_jobs(gk, n_jobs):
    """More than 64 jobs in ONE device-tier call: gk_pack_batch and gk_restore then take the
    staged job-table upload followed by the validation and claim kernels (smaller calls pass
    the table as kernel arguments).  Every kind of damage the random suite knows, several of
    each, full destination image against the oracle."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_pack, gpu_restore
    og = G_MID
    T = og.page_tokens
    rng = np.random.default_rng(8800 + n_jobs)
    lens = [int(rng.integers(1, 3 * T + 1)) for _ in range(n_jobs)]
    Ns = 40
    src = random_cache(og, Ns, seed=8801)
    tables = [rng.integers(0, Ns, size=n_pages(og, n)).astype(np.int32) for n in lens]
    tables[7][0] = Ns + 1                           # save: an id out of range -> status 2, nothing written
    for fused in (1, 0):
        ctx = _ctx(gk, og, fused=fused)
        got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
        wstatus = [0] * n_jobs
        wstatus[7] = 2
        assert status.tolist() == wstatus
        total = sum(n_pages(og, n) for n in lens)
        Nd = total + 5
        perm = rng.permutation(Nd).astype(np.int32)
        ojobs, used = [], 0
        for j, ((blob, sums), pt, n) in enumerate(zip(got, tables, lens)):
            P = n_pages(og, n)
            if j == 7:
                assert not blob.any() and not sums.any()        # left as the harness zeroed them
                pt = tables[7].copy()
                pt[0] = 0
                wb, ws, code, _ = oracle.pack(og, src, pt, n)
            else:
                wb, ws, code, _ = oracle.pack(og, src, pt, n)
                assert code == 0 and np.array_equal(blob, wb) and np.array_equal(sums, ws)
            ojobs.append(oracle.Job(wb.copy(), ws.copy(), perm[used:used + P].copy(), n))
            used += P
        for j, jb in enumerate(ojobs):
            kind = j % 8
            if kind == 1:
                for _ in range(1 + j % 4):
                    jb.blob[int(rng.integers(0, jb.blob.size))] ^= np.uint8(1 << int(rng.integers(0, 8)))
            elif kind == 2:
                jb.checksums[int(rng.integers(0, jb.checksums.size))] ^= np.uint64(1) << np.uint64(int(rng.integers(0, 64)))
            elif kind == 3:
                ojobs[j] = oracle.Job(None, None, jb.page_table, jb.n_tokens)
            elif kind == 4:
                jb.page_table[int(rng.integers(0, jb.page_table.size))] = Nd + 2 if j % 16 == 4 else -1
            elif kind == 5:
                jb.page_table[0] = ojobs[(j + 1) % n_jobs].page_table[0]
        clean = random_cache(og, Nd, seed=8802)
        want = clone_cache(clean)
        wmask, wfb = oracle.restore(og, want, ojobs)
        assert set(wmask.tolist()) == {0, 1, 2, 3}
        d = dev_cache(clean)
        mask, fb = gpu_restore(ctx, d, ojobs, host_tier=False)
        assert mask.tolist() == wmask.tolist()
        assert fb.tolist() == wfb.tolist()
        assert_cache_equal(d, want)
        ctx.close()


def test_reserve_sizes_everything_once(gk):
    """After gk_ctx_reserve no call within the stated bounds allocates (and so none frees or
    synchronises the device): the context's allocation counter stays where reserve left it
    across small and large calls of every kind, on both tiers, and the results stay bit-exact."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, gpu_pack, gpu_restore, sums_to_dev
    og = G_MID
    T = og.page_tokens
    rng = np.random.default_rng(8900)
    ctx = _ctx(gk, og)
    max_jobs, max_pages, num_pages = 100, 320, 400
    blob_max = oracle.blob_size(og, 3 * T)[0]
    ctx.gk_ctx_reserve(max_jobs, max_pages, num_pages, max_jobs * blob_max)
    base = ctx.gk_get_stats()["allocations"]
    assert base > 0
    src = random_cache(og, 60, seed=8901)
    for n_jobs in (1, 4, 64, 65, 100):
        lens = [int(rng.integers(1, 3 * T + 1)) for _ in range(n_jobs)]
        tables = [rng.integers(0, 60, size=n_pages(og, n)).astype(np.int32) for n in lens]
        got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
        assert not status.any()
        total = sum(n_pages(og, n) for n in lens)
        perm = rng.permutation(num_pages).astype(np.int32)
        ojobs, used = [], 0
        for (blob, sums), pt, n in zip(got, tables, lens):
            wb, ws, code, _ = oracle.pack(og, src, pt, n)
            assert np.array_equal(blob, wb) and np.array_equal(sums, ws)
            P = n_pages(og, n)
            ojobs.append(oracle.Job(wb, ws, perm[used:used + P].copy(), n))
            used += P
        ojobs[0].blob[5] ^= 1
        clean = random_cache(og, num_pages, seed=8902 + n_jobs)
        want = clone_cache(clean)
        wmask, wfb = oracle.restore(og, want, ojobs)
        for host_tier in (False, True):
            d = dev_cache(clean)
            mask, fb = gpu_restore(ctx, d, ojobs, host_tier=host_tier)
            assert mask.tolist() == wmask.tolist() and fb.tolist() == wfb.tolist()
            assert_cache_equal(d, want)
        # the two halves and the checksum-only call
        d = dev_cache(clean)
        keep = [(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table)) for j in ojobs]
        gjobs = [gk.Job(b, s_, t, j.n_tokens) for (b, s_, t), j in zip(keep, ojobs)]
        mask = torch.full((n_jobs,), 255, dtype=torch.uint8, device="cuda")
        fb = torch.zeros(n_jobs, dtype=torch.int32, device="cuda")
        ctx.gk_verify(gjobs, d, mask, fb)
        ctx.gk_commit(gjobs, d, mask)
        sums2 = torch.zeros(ojobs[1 % n_jobs].checksums.size, dtype=torch.int64, device="cuda")
        ctx.gk_page_checksums(keep[1 % n_jobs][0], ojobs[1 % n_jobs].n_tokens, sums2)
        torch.cuda.synchronize()
        assert_cache_equal(d, want)
        # save to the host tier
        hjobs, hkeep = [], []
        for (blob, sums), pt, n in zip(got, tables, lens):
            hb = torch.empty(blob.size, dtype=torch.uint8, pin_memory=True)
            hs = torch.empty(sums.size, dtype=torch.int64, pin_memory=True)
            hkeep.append((hb, hs))
            hjobs.append(gk.Job(hb, hs, dev_i32(pt), n))
        ctx.gk_pack_host(dev_cache(src), hjobs)
        torch.cuda.synchronize()
        for (hb, hs), (blob, sums) in zip(hkeep, got):
            assert np.array_equal(hb.numpy(), blob) and np.array_equal(hs.numpy().view(np.uint64), sums)
        assert ctx.gk_get_stats()["allocations"] == base, f"a call of {n_jobs} jobs allocated after reserve"
    ctx.close()
    # without reserve the same calls do allocate: the counter means something
    ctx = _ctx(gk, og)
    got, _ = gpu_pack(ctx, og, dev_cache(src), [np.zeros(1, dtype=np.int32)] * 70, [T] * 70)
    assert ctx.gk_get_stats()["allocations"] > 0
    ctx.close()


def test_restore_beside_another_kernel_that_occupies_the_gpu(gk):
    """The fused restore kernel must not depend on all of its CTAs being resident at once:
    while a side stream keeps the SMs busy with large matrix products, a multi-job restore
    still completes, bit-exact, without any wait running out."""
    from gpu_harness import assert_cache_equal, dev_cache, dev_i32, sums_to_dev
    og = G_BIG
    T = og.page_tokens
    src = random_cache(og, 40, seed=390)
    jobs = _oracle_jobs(og, src, [12 * T, 9 * T + 1, 15 * T, 3 * T], 391, 48)
    jobs[2].blob[1 << 20] ^= 0x08
    clean = random_cache(og, 48, seed=392)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs)
    ctx = _ctx(gk, og)
    keep = [(torch.from_numpy(j.blob).cuda(), sums_to_dev(j.checksums), dev_i32(j.page_table)) for j in jobs]
    gjobs = [gk.Job(b, s, t, j.n_tokens) for (b, s, t), j in zip(keep, jobs)]
    mask = torch.full((4,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(4, dtype=torch.int32, device="cuda")
    a = torch.randn(8192, 8192, device="cuda", dtype=torch.bfloat16)
    side = torch.cuda.Stream()
    for rep in range(3):
        d = dev_cache(clean)
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            for _ in range(6):
                a @ a                                   # a few ms each, all SMs
        ctx.gk_restore(gjobs, d, mask, fb)
        torch.cuda.synchronize()
        assert mask.cpu().tolist() == wmask.tolist() and fb.cpu().tolist() == wfb.tolist()
        assert_cache_equal(d, want)
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    ctx.close()


def test_logic_rate_measurement_is_plausible(gk):
    """The measured rate of three-input logic operations (the denominator of the checksum kernels'
    roofline): between 32 and 128 lanes per clock per SM at the device's maximum clock."""
    ctx = _ctx(gk, G_MID)
    rate = ctx.gk_measure_logic_rate()
    props = torch.cuda.get_device_properties(0)
    per_sm_clk = rate / (props.multi_processor_count * getattr(props, "clock_rate", 1965000) * 1e3)
    assert 32.0 <= per_sm_clk <= 128.0, per_sm_clk
    ctx.close()


def test_padded_strides_leave_the_padding_alone(gk):
    """Caches whose pages, K/V planes and layers are separated by padding: pack reads
    only slab bytes, restore writes only slab bytes."""
    from gpu_harness import gpu_pack, gpu_restore
    import paper_2609_39358_b200 as m
    og = G_MID
    T, N = og.page_tokens, 9
    slab = T * og.kv_heads * og.head_dim * og.elem_bytes
    ps, ks, ls = slab + 256, N * (slab + 256) + 512, 2 * (N * (slab + 256) + 512) + 1024
    total = og.layers * ls
    rng = np.random.default_rng(370)
    src = oracle.Cache(rng.integers(0, 256, size=total, dtype=np.uint8), N, ls, ks, ps)
    clean = oracle.Cache(rng.integers(0, 256, size=total, dtype=np.uint8), N, ls, ks, ps)
    lens = [2 * T + 3, T]
    tables = [np.array([7, 2, 5], dtype=np.int32), np.array([0], dtype=np.int32)]
    ctx = _ctx(gk, og)
    dsrc = m.Cache(torch.from_numpy(src.data).cuda(), N, ls, ks, ps)
    got, status = gpu_pack(ctx, og, dsrc, tables, lens)
    assert status.tolist() == [0, 0]
    jobs = []
    for (blob, sums), pt, n, dpt in zip(got, tables, lens, [np.array([1, 8, 3], dtype=np.int32),
                                                              np.array([6], dtype=np.int32)]):
        wb, ws, _, _ = oracle.pack(og, src, pt, n)
        assert np.array_equal(blob, wb) and np.array_equal(sums, ws)
        jobs.append(oracle.Job(blob, sums, dpt, n))
    want = clone_cache(clean)
    wmask, _ = oracle.restore(og, want, jobs)
    d = m.Cache(torch.from_numpy(clean.data).cuda(), N, ls, ks, ps)
    mask, _ = gpu_restore(ctx, d, jobs)
    assert mask.tolist() == wmask.tolist() == [0, 0]
    assert np.array_equal(d.data.cpu().numpy(), want.data)
    ctx.close()


@pytest.mark.parametrize("og", [
    oracle.Geom(3, 2, 16, 1, 1, 2),      # 32-byte slabs (one token per page, fp8): a tile is hundreds of copies
    oracle.Geom(7, 1, 8, 3, 2, 0),       # 48-byte slabs, odd page size, odd layer count
    oracle.Geom(1, 1, 8, 1, 2, 0),       # the smallest geometry the library accepts: 32-byte records
    oracle.Geom(2, 3, 40, 5, 2, 0),      # nothing is a power of two
])
def test_extreme_small_geometries(gk, og):
    from gpu_harness import assert_cache_equal, dev_cache, gpu_pack, gpu_restore
    T = og.page_tokens
    N = 37
    src = random_cache(og, N, seed=400)
    lens = [1, T, 5 * T + (1 if T > 1 else 0), 11 * T]
    rng = np.random.default_rng(401)
    tables = [rng.integers(0, N, size=n_pages(og, n)).astype(np.int32) for n in lens]
    ctx = _ctx(gk, og)
    got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
    assert status.tolist() == [0] * len(lens)
    for (blob, sums), pt, n in zip(got, tables, lens):
        wb, ws, _, _ = oracle.pack(og, src, pt, n)
        assert np.array_equal(blob, wb) and np.array_equal(sums, ws)
    jobs = _oracle_jobs(og, src, lens, 402, 64)
    jobs[2].blob[len(jobs[2].blob) - 1] ^= 0x40
    clean = random_cache(og, 64, seed=403)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, jobs)
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, jobs)
    assert mask.tolist() == wmask.tolist() == [0, 0, 1, 0] and fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    ctx.close()


def test_guard_bands_around_every_output_buffer(gk):
    """Every buffer the library writes (blob, checksums, status, destination cache, scales,
    mask, first_bad_page) sits inside a larger allocation filled with a sentinel: after
    pack and restore the slack on both sides must be untouched."""
    from gpu_harness import dev_i32
    import paper_2609_39358_b200 as m
    og = G_FP8_M
    T, N, G = og.page_tokens, 13, 4096                      # G = guard bytes on each side
    src = random_cache(og, N, seed=410)
    lens = [2 * T + 1, T, 3 * T]
    rng = np.random.default_rng(411)
    tables = [rng.permutation(N)[:n_pages(og, n)].astype(np.int32) for n in lens]
    ctx = _ctx(gk, og)

    def guarded(nbytes, dtype=torch.uint8):
        raw = torch.full((nbytes + 2 * G,), 0xA5, dtype=torch.uint8, device="cuda")
        return raw, raw[G:G + nbytes].view(dtype)

    def slack_ok(raw, nbytes):
        return bool((raw[:G] == 0xA5).all()) and bool((raw[G + nbytes:] == 0xA5).all())

    dsrc = m.Cache(torch.from_numpy(src.data).cuda(), N, src.layer_stride, src.kv_stride, src.page_stride,
                   torch.from_numpy(src.scales).cuda(), src.s_layer_stride, src.s_kv_stride, src.s_page_stride)
    bufs, jobs = [], []
    for pt, n in zip(tables, lens):
        nbytes, P = oracle.blob_size(og, n)
        braw, blob = guarded(nbytes)
        sraw, sums = guarded(8 * P, torch.int64)
        bufs.append((braw, nbytes, sraw, 8 * P))
        jobs.append(m.Job(blob, sums, dev_i32(pt), n))
    straw, status = guarded(len(jobs))
    ctx.gk_pack_batch(dsrc, jobs, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0, 0]
    for (braw, nb, sraw, ns), job, pt, n in zip(bufs, jobs, tables, lens):
        assert slack_ok(braw, nb) and slack_ok(sraw, ns)
        wb, ws, _, _ = oracle.pack(og, src, pt, n)
        assert np.array_equal(job.blob.cpu().numpy(), wb)
    assert slack_ok(straw, len(jobs))
    # restore into a guarded destination
    Nd = 16
    clean = random_cache(og, Nd, seed=412)
    draw, ddata = guarded(clean.data.size)
    ddata.copy_(torch.from_numpy(clean.data))
    scraw, dscales = guarded(clean.scales.size)
    dscales.copy_(torch.from_numpy(clean.scales))
    dst = m.Cache(ddata, Nd, clean.layer_stride, clean.kv_stride, clean.page_stride, dscales,
                  clean.s_layer_stride, clean.s_kv_stride, clean.s_page_stride)
    perm = rng.permutation(Nd).astype(np.int32)
    rjobs, ojobs, off = [], [], 0
    for job, n in zip(jobs, lens):
        P = n_pages(og, n)
        dpt = perm[off:off + P]
        off += P
        rjobs.append(m.Job(job.blob, job.checksums, dev_i32(dpt), n))
        ojobs.append(oracle.Job(job.blob.cpu().numpy(), job.checksums.cpu().numpy().view(np.uint64), dpt, n))
    mraw, mask = guarded(len(rjobs))
    fraw, fb = guarded(4 * len(rjobs), torch.int32)
    ctx.gk_restore(rjobs, dst, mask, fb)
    torch.cuda.synchronize()
    want = clone_cache(clean)
    wmask, _ = oracle.restore(og, want, ojobs)
    assert mask.cpu().tolist() == wmask.tolist() == [0, 0, 0]
    assert np.array_equal(ddata.cpu().numpy(), want.data) and np.array_equal(dscales.cpu().numpy(), want.scales)
    assert slack_ok(draw, clean.data.size) and slack_ok(scraw, clean.scales.size)
    assert slack_ok(mraw, len(rjobs)) and slack_ok(fraw, 4 * len(rjobs))
    ctx.close()


def test_argument_errors(gk):
    from gpu_harness import dev_cache
    og = G_MID
    ctx = _ctx(gk, og)
    clean = random_cache(og, 4, seed=350)
    d = dev_cache(clean)
    mask = torch.zeros(1, dtype=torch.uint8, device="cuda")
    fb = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.gk_restore([], d, mask, fb)                       # n_jobs == 0: no-op
    pt = torch.zeros(1, dtype=torch.int32, device="cuda")
    blob = torch.zeros(oracle.blob_size(og, 1)[0], dtype=torch.uint8)          # pageable host memory
    sums = torch.zeros(1, dtype=torch.int64)
    with pytest.raises(gk.GkError) as e:
        ctx.gk_restore_host([gk.Job(blob, sums, pt, 1)], d, mask, fb)
    assert e.value.code == -3
    with pytest.raises(gk.GkError) as e:
        ctx.gk_restore([gk.Job(blob.cuda(), sums.cuda(), pt, 0)], d, mask, fb)
    assert e.value.code == -1
    with pytest.raises(gk.GkError):
        gk.Context(gk.Geom(2, 1, 4, 16), 0)               # row of 8 bytes: not a multiple of 16
    ctx.close()


def test_round_trip_from_plain_c(gk, tmp_path):
    """The C ABI used from a C program that knows nothing of Python or torch."""
    import os
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    libdir = os.path.join(root, "paper_2609_39358_b200")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = tmp_path / "roundtrip_gpu"
    build = subprocess.run(["gcc", "-std=c11", "-O1", "-Wall", "-Wextra", "-Werror", os.path.join(root, "tests", "c", "roundtrip_gpu.c"),
                            "-o", str(exe), "-I" + os.path.join(cuda, "include"), "-L" + libdir, "-l:libgk.so",
                            "-L" + os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + libdir,
                            "-Wl,-rpath," + os.path.join(cuda, "lib64")], capture_output=True, text=True)
    assert build.returncode == 0, build.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and "roundtrip ok" in run.stdout, (run.returncode, run.stdout, run.stderr)
