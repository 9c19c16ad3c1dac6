"""Seeded random cases on the GPU against the oracle: random geometries (both dtypes, both
slab layouts), block lengths, page tables, kinds of damage, flags, tunings and tiers.  Every
case compares the blob, the checksums, the codes, the first bad pages and the full
destination image."""
import numpy as np
import pytest
import torch

import oracle
from helpers import clone_cache, n_pages, random_cache

import os

pytestmark = pytest.mark.gpu

# more cases for a soak run: GK_FUZZ_CASES=3000 python -m pytest tests/test_gpu_fuzz.py -m gpu
N_CASES = int(os.environ.get("GK_FUZZ_CASES", "128"))


@pytest.fixture(scope="module")
def gk():
    import paper_2609_39358_b200 as m
    assert torch.cuda.is_available()
    return m


def _random_geom(rng):
    fp8 = bool(rng.integers(0, 2))
    head_major = int(rng.integers(0, 2))
    elem = 1 if fp8 else 2
    while True:
        layers = int(rng.integers(1, 7))
        heads = int(rng.choice([1, 2, 3, 4, 8]))
        dim = int(rng.choice([16, 32, 64, 128]))
        T = int(rng.choice([1, 2, 4, 8, 16, 32]))
        scale_kv = int(rng.integers(1, 3)) if fp8 else 0
        row = heads * dim * elem
        S = layers * scale_kv * heads * 4
        if row % 16 or S % 16:
            continue
        return oracle.Geom(layers, heads, dim, T, elem, scale_kv, head_major)


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_case(gk, case):
    from gpu_harness import assert_cache_equal, dev_cache, gk_geom, gpu_pack, gpu_restore
    rng = np.random.default_rng(9000 + case)
    og = _random_geom(rng)
    T = og.page_tokens
    n_jobs = int(rng.integers(1, 9))
    lens = [int(rng.integers(1, 6 * T + 1)) for _ in range(n_jobs)]
    Ns = int(rng.integers(4, 24))
    src = random_cache(og, Ns, seed=9100 + case, layout=str(rng.choice(["layer_major", "page_major"])))
    tables = [rng.integers(0, Ns, size=n_pages(og, n)).astype(np.int32) for n in lens]
    single = bool(rng.integers(0, 2))
    flags = gk.GK_FLAG_SINGLE_PASS if single else 0
    tuning = [{}, {"seg_granules": 1}, {"seg_granules": 2, "commit_seg_tiles": 1}, {"grid_cap": int(rng.integers(1, 9))},
              {"fused": 0}][int(rng.integers(0, 5))]
    ctx = gk.Context(gk_geom(og, flags), 0)
    for k, v in tuning.items():
        ctx.set_tuning(k, v)

    # save: every blob and checksum against the oracle
    got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
    assert status.tolist() == [0] * n_jobs
    ojobs = []
    total = sum(n_pages(og, n) for n in lens)
    Nd = total + int(rng.integers(0, 6))
    perm = rng.permutation(Nd).astype(np.int32)
    used = 0
    for (blob, sums), pt, n in zip(got, tables, lens):
        wb, ws, code, _ = oracle.pack(og, src, pt, n)
        assert code == 0 and np.array_equal(blob, wb) and np.array_equal(sums, ws)
        P = n_pages(og, n)
        ojobs.append(oracle.Job(wb.copy(), ws.copy(), perm[used:used + P].copy(), n))
        used += P

    # damage: each job independently gets nothing, bit flips, a damaged checksum, a missing record,
    # an out-of-range id, or a page shared with another job
    for j, jb in enumerate(ojobs):
        kind = int(rng.integers(0, 8))
        if kind == 1:
            for _ in range(int(rng.integers(1, 5))):
                jb.blob[int(rng.integers(0, jb.blob.size))] ^= np.uint8(1 << int(rng.integers(0, 8)))
        elif kind == 2:
            jb.checksums[int(rng.integers(0, jb.checksums.size))] ^= np.uint64(1) << np.uint64(int(rng.integers(0, 64)))
        elif kind == 3:
            ojobs[j] = oracle.Job(None, None, jb.page_table, jb.n_tokens)
        elif kind == 4:
            jb.page_table[int(rng.integers(0, jb.page_table.size))] = Nd + int(rng.integers(0, 3)) if rng.random() < 0.5 else -1
        elif kind == 5 and n_jobs > 1:
            other = ojobs[(j + 1) % n_jobs]
            jb.page_table[0] = other.page_table[0]
    clean = random_cache(og, Nd, seed=9200 + case, layout=str(rng.choice(["layer_major", "page_major"])))
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, ojobs, flags=oracle.FLAG_SINGLE_PASS if single else 0)
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, ojobs, host_tier=bool(rng.integers(0, 2)))
    assert mask.tolist() == wmask.tolist(), (og, lens, tuning, single)
    assert fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    ctx.close()


@pytest.mark.parametrize("case", range(max(N_CASES // 4, 1)))
def test_random_stream_restore_case(gk, case):
    """Random corpora through random rings: windows, ring image after every window, codes."""
    from gpu_harness import dev_cache, gk_geom
    rng = np.random.default_rng(9500 + case)
    og = _random_geom(rng)
    T = og.page_tokens
    n_jobs = int(rng.integers(1, 12))
    lens = [int(rng.integers(1, 5 * T + 1)) for _ in range(n_jobs)]
    src = random_cache(og, 9, seed=9600 + case)
    ojobs = []
    for n in lens:
        blob, sums, code, _ = oracle.pack(og, src, rng.integers(0, 9, size=n_pages(og, n)).astype(np.int32), n)
        assert code == 0
        kind = int(rng.integers(0, 6))
        if kind == 1:
            blob[int(rng.integers(0, blob.size))] ^= np.uint8(1 << int(rng.integers(0, 8)))
        if kind == 2:
            ojobs.append(oracle.Job(None, None, None, n))
        else:
            ojobs.append(oracle.Job(blob, sums, None, n))
    ring_pages = max(n_pages(og, n) for n in lens) + int(rng.integers(0, 8))
    single = bool(rng.integers(0, 2))
    clean = random_cache(og, ring_pages, seed=9700 + case)
    want = clone_cache(clean)
    owin = []
    wmask, wfb = oracle.restore_stream(og, want, ojobs,
                                       lambda first, count, pages: owin.append((first, count, want.data.copy())),
                                       flags=oracle.FLAG_SINGLE_PASS if single else 0)
    ctx = gk.Context(gk_geom(og, gk.GK_FLAG_SINGLE_PASS if single else 0), 0)
    d = dev_cache(clean)
    jobs, keep = [], []
    for jb in ojobs:
        hb = None if jb.blob is None else torch.from_numpy(jb.blob).pin_memory()
        hs = None if jb.checksums is None else torch.from_numpy(jb.checksums.view(np.int64).copy()).pin_memory()
        keep.append((hb, hs))
        jobs.append(gk.Job(hb, hs, None, jb.n_tokens))
    mask = torch.full((n_jobs,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((n_jobs,), -7, dtype=torch.int32, device="cuda")
    gwin = []
    ctx.gk_restore_stream(jobs, d, mask, fb, lambda blocks, st: gwin.append((blocks[0].job, len(blocks), d.data.clone())))
    torch.cuda.synchronize()
    assert mask.cpu().tolist() == wmask.tolist() and fb.cpu().tolist() == wfb.tolist()
    assert [(a, b) for a, b, _ in gwin] == [(a, b) for a, b, _ in owin]
    for (_, _, gimg), (_, _, oimg) in zip(gwin, owin):
        assert np.array_equal(gimg.cpu().numpy(), oimg)
    ctx.close()


@pytest.mark.parametrize("case", range(12))
def test_random_medium_case(gk, case):
    """Records of 0.25 to 3 MiB and up to a few hundred pages per call: adaptive segment
    tiling, many CTAs drawing items at once, jobs finishing out of order."""
    from gpu_harness import assert_cache_equal, dev_cache, gk_geom, gpu_pack, gpu_restore
    rng = np.random.default_rng(9800 + case)
    fp8 = bool(rng.integers(0, 2))
    og = oracle.Geom(int(rng.choice([8, 16, 24, 48])), int(rng.choice([4, 8])), 128, int(rng.choice([16, 32])),
                     1 if fp8 else 2, 2 if fp8 else 0, int(rng.integers(0, 2)))
    T = og.page_tokens
    rec = oracle.record_bytes(og, T, 0)
    budget_pages = max(int(160e6 // rec), 8)
    n_jobs = int(rng.integers(1, 10))
    lens = []
    for _ in range(n_jobs):
        lens.append(int(rng.integers(1, max(2, budget_pages // n_jobs) * T + 1)))
    Ns = 12
    src = random_cache(og, Ns, seed=9900 + case)
    tables = [rng.integers(0, Ns, size=n_pages(og, n)).astype(np.int32) for n in lens]
    single = bool(rng.integers(0, 2))
    ctx = gk.Context(gk_geom(og, gk.GK_FLAG_SINGLE_PASS if single else 0), 0)
    got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
    assert status.tolist() == [0] * n_jobs
    total = sum(n_pages(og, n) for n in lens)
    Nd = total + 3
    perm = rng.permutation(Nd).astype(np.int32)
    ojobs, used = [], 0
    for (blob, sums), pt, n in zip(got, tables, lens):
        wb, ws, code, _ = oracle.pack(og, src, pt, n)
        assert code == 0 and np.array_equal(blob, wb) and np.array_equal(sums, ws)
        P = n_pages(og, n)
        ojobs.append(oracle.Job(wb.copy(), ws.copy(), perm[used:used + P].copy(), n))
        used += P
    for jb in ojobs:
        if rng.random() < 0.3:
            jb.blob[int(rng.integers(0, jb.blob.size))] ^= np.uint8(1 << int(rng.integers(0, 8)))
    clean = random_cache(og, Nd, seed=9950 + case)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, ojobs, flags=oracle.FLAG_SINGLE_PASS if single else 0)
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, ojobs, host_tier=bool(rng.integers(0, 2)))
    assert mask.tolist() == wmask.tolist() and fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    ctx.close()
