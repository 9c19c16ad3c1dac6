"""Page quartets: packing and fused-restore launches over SMALL page records reduce one
record per warp, four consecutive pages of the launch to a work item (tuning key "quad").
Checked here against the oracle, bit for bit: calls large enough for the library to choose
the form by itself, the form forced on small and ragged calls (quartets that straddle jobs,
short last pages, jobs that are skipped, damage of every kind), and the rest of the GPU
suites once more with the form forced on everything."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from helpers import clone_cache, n_pages, random_cache

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

G_8K = oracle.Geom(1, 2, 64, 16, 2, 0)      # record 8 KiB: one granule of a warp
G_20K = oracle.Geom(5, 1, 64, 16, 2, 0)     # record 20 KiB: 2.5 granules, front padding in every record
G_HM = oracle.Geom(2, 2, 64, 16, 2, 0, head_major=1)  # head-major slabs: short pages are gathered head by head
G_FP8 = oracle.Geom(6, 4, 32, 8, 1, 2)      # scale sections: restore may use quartets, pack may not


@pytest.fixture(scope="module")
def gk():
    import paper_2609_39358_b200 as m
    assert torch.cuda.is_available()
    return m


def _ctx(gk, og, **tuning):
    from gpu_harness import gk_geom
    ctx = gk.Context(gk_geom(og), 0)
    for k, v in tuning.items():
        ctx.set_tuning(k, v)
    return ctx


def _round_trip(gk, og, lens, seed, quad, expect_quartets, damage=True, host_tier=False, **tuning):
    """Packs blocks of the given lengths, checks blobs and checksums against the oracle, damages
    some, restores, and compares codes, first bad pages and the whole destination image."""
    from gpu_harness import assert_cache_equal, dev_cache, gpu_pack, gpu_restore
    rng = np.random.default_rng(seed)
    n_jobs = len(lens)
    Ns = 48
    src = random_cache(og, Ns, seed=seed + 1)
    tables = [rng.integers(0, Ns, size=n_pages(og, n)).astype(np.int32) for n in lens]
    ctx = _ctx(gk, og, quad=quad, **tuning)
    got, status = gpu_pack(ctx, og, dev_cache(src), tables, lens)
    assert status.tolist() == [0] * n_jobs
    total = sum(n_pages(og, n) for n in lens)
    Nd = total + 7
    perm = rng.permutation(Nd).astype(np.int32)
    ojobs, used = [], 0
    for (blob, sums), pt, n in zip(got, tables, lens):
        wb, ws, code, _ = oracle.pack(og, src, pt, n)
        assert code == 0
        assert np.array_equal(sums, ws), f"checksums differ at pages {np.flatnonzero(sums != ws)[:8]}"
        assert np.array_equal(blob, wb)
        P = n_pages(og, n)
        ojobs.append(oracle.Job(wb.copy(), ws.copy(), perm[used:used + P].copy(), n))
        used += P
    if damage:
        for j, jb in enumerate(ojobs):
            kind = j % 9
            if kind == 1:      # a flipped bit somewhere in the blob
                jb.blob[int(rng.integers(0, jb.blob.size))] ^= np.uint8(1 << int(rng.integers(0, 8)))
            elif kind == 2:    # a flipped bit in a stored checksum
                jb.checksums[int(rng.integers(0, jb.checksums.size))] ^= np.uint64(1) << np.uint64(int(rng.integers(0, 64)))
            elif kind == 3:    # nothing stored
                ojobs[j] = oracle.Job(None, None, jb.page_table, jb.n_tokens)
            elif kind == 4:    # a table entry out of range
                jb.page_table[int(rng.integers(0, jb.page_table.size))] = Nd + 2 if j % 2 else -1
            elif kind == 5:    # a destination page claimed twice
                jb.page_table[0] = ojobs[(j + 1) % n_jobs].page_table[0]
            elif kind == 6:    # the LAST page of the block (the short one) damaged
                jb.blob[jb.blob.size - 1] ^= np.uint8(0x80)
    clean = random_cache(og, Nd, seed=seed + 2)
    want = clone_cache(clean)
    wmask, wfb = oracle.restore(og, want, ojobs)
    d = dev_cache(clean)
    mask, fb = gpu_restore(ctx, d, ojobs, host_tier=host_tier)
    assert mask.tolist() == wmask.tolist()
    assert fb.tolist() == wfb.tolist()
    assert_cache_equal(d, want)
    q = ctx.gk_get_stats()["quartet_launches"]
    if expect_quartets is not None:
        assert q == expect_quartets, q
    ctx.close()
    return wmask


@pytest.mark.parametrize("og", [G_8K, G_20K, G_HM])
def test_forced_on_small_ragged_calls(gk, og):
    """Lengths from one token to a few pages, so that quartets straddle jobs, hold short last
    pages next to full ones, and whole quartets belong to skipped jobs."""
    T = og.page_tokens
    rng = np.random.default_rng(4100)
    lens = [int(rng.integers(1, 5 * T + 1)) for _ in range(40)] + [1, T, T + 1, 4 * T, 4 * T - 1, 7]
    wmask = _round_trip(gk, og, lens, 4200, quad=2, expect_quartets=2)
    assert set(wmask.tolist()) == {0, 1, 2, 3}
    # one block alone, one page alone
    _round_trip(gk, og, [1], 4300, quad=2, expect_quartets=2, damage=False)
    _round_trip(gk, og, [9 * T + 3], 4400, quad=2, expect_quartets=2, damage=False)


def test_scale_sections_restore_only(gk):
    """Records with scale sections: the restore may take quartets (a record is read as it lies in the
    blob), the pack may not (its scale values are gathered by a whole warp per record)."""
    og = G_FP8
    T = og.page_tokens
    rng = np.random.default_rng(4500)
    lens = [int(rng.integers(1, 6 * T + 1)) for _ in range(30)]
    _round_trip(gk, og, lens, 4600, quad=2, expect_quartets=1)


@pytest.mark.parametrize("og", [G_8K, G_20K])
def test_chosen_for_large_calls_of_small_records(gk, og):
    """Enough pages for two quartets per resident CTA: the library takes the form by itself; with the
    key at 1 it does not, and the results are the same."""
    T = og.page_tokens
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    want_pages = 8 * 2 * sm + 300
    rng = np.random.default_rng(4700)
    lens = []
    while sum(n_pages(og, n) for n in lens) < want_pages:
        lens.append(int(rng.integers(1, 400 * T)))
    _round_trip(gk, og, lens, 4800, quad=0, expect_quartets=2)
    _round_trip(gk, og, lens, 4800, quad=1, expect_quartets=0)


def test_verify_alone_and_page_checksums(gk):
    """The verifying kernel on its own (restore with the tuning key fused = 0: a verify launch, a compare
    launch, a commit launch; and gk_page_checksums) takes the same form."""
    from gpu_harness import gk_geom
    og = G_20K
    T = og.page_tokens
    rng = np.random.default_rng(5100)
    lens = [int(rng.integers(1, 5 * T + 1)) for _ in range(40)]
    _round_trip(gk, og, lens, 5200, quad=2, expect_quartets=2, fused=0)
    # checksums of an existing blob
    n = 37 * T + 5
    src = random_cache(og, n_pages(og, n), seed=5300)
    blob, sums, code, _ = oracle.pack(og, src, np.arange(n_pages(og, n), dtype=np.int32), n)
    assert code == 0
    ctx = gk.Context(gk_geom(og), 0)
    ctx.set_tuning("quad", 2)
    out = torch.zeros(n_pages(og, n), dtype=torch.int64, device="cuda")
    ctx.gk_page_checksums(torch.from_numpy(blob).cuda(), n, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint64), sums)
    assert ctx.gk_get_stats()["quartet_launches"] == 1
    ctx.close()


def test_host_tier_in_batches(gk):
    """Host-tier calls launch per staging batch: quartets are counted from the first page of each launch."""
    og = G_20K
    T = og.page_tokens
    rng = np.random.default_rng(4900)
    lens = [int(rng.integers(1, 30 * T)) for _ in range(24)]
    _round_trip(gk, og, lens, 5000, quad=2, expect_quartets=None, host_tier=True)


def test_other_suites_with_quartets_forced(gk):
    """The random, parity and layer-wise suites once more, in a child process whose every context
    has quad=2, against the ordinary and against the bounds-checked library."""
    from paper_2609_39358_b200 import build
    for lib in (build.build(), build.build(debug=True)):
        env = dict(os.environ, GK_LIB_PATH=lib, GK_TUNING="quad=2", GK_FUZZ_CASES="48")
        r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                            "tests/test_gpu_fuzz.py", "tests/test_gpu_parity.py", "tests/test_gpu_layerwise.py",
                            "-k", "not plain_c and not reserve_sizes"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
        assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
