"""GPU parity of the SHA-256 paths (block fingerprints, blob digests) against the CPU
oracle, byte for byte, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import n_pages, random_cache

pytestmark = pytest.mark.gpu

MODEL = bytes((7 * i + 1) & 0xFF for i in range(32))
TENANT = bytes((11 * i + 3) & 0xFF for i in range(32))


@pytest.fixture(scope="module")
def gk():
    import paper_2609_39358_b200 as m
    assert torch.cuda.is_available()
    return m


def _ctx(gk, og):
    from gpu_harness import gk_geom
    return gk.Context(gk_geom(og), 0)


def _gpu_keys(ctx, data, off, parent):
    d = torch.from_numpy(data).cuda() if data.size else torch.zeros(16, dtype=torch.uint8, device="cuda")
    o = torch.from_numpy(off.astype(np.int64)).cuda()
    keys = torch.full((off.size - 1, 32), 0xEE, dtype=torch.uint8, device="cuda")
    ctx.gk_fingerprints(d, o, parent, MODEL, TENANT, keys)
    torch.cuda.synchronize()
    return keys.cpu().numpy()


def test_fingerprints_all_padding_cases_alignments_and_chains(gk):
    ctx = _ctx(gk, oracle.Geom(2, 2, 64, 16, 2, 0))
    rng = np.random.default_rng(500)
    lens = [0, 1, 3, 4, 55, 56, 63, 64, 65, 100, 119, 120, 127, 128, 4096, 16384, 17, 16384 + 13, 5, 0, 64]
    parent = [-1, -1, 0, 2, -1, 4, 5, 6, 1, -1, 9, 10, 11, 12, 13, 14, -1, 16, 17, 18, 19]
    data = rng.integers(0, 256, size=sum(lens), dtype=np.uint8)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    want = oracle.fingerprints(data, off, parent, MODEL, TENANT)
    assert np.array_equal(_gpu_keys(ctx, data, off, parent), want)
    want0 = oracle.fingerprints(data, off, None, MODEL, TENANT)
    assert np.array_equal(_gpu_keys(ctx, data, off, None), want0)
    # 16-byte aligned starts (token ids): the vector-load path
    lens = [16 * k for k in (1, 4, 5, 256, 1024, 3)]
    data = rng.integers(0, 256, size=sum(lens), dtype=np.uint8)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    par = [-1, 0, 1, 2, -1, 4]
    assert np.array_equal(_gpu_keys(ctx, data, off, par), oracle.fingerprints(data, off, par, MODEL, TENANT))
    ctx.close()


def test_fingerprints_many_messages_and_deep_chains(gk):
    ctx = _ctx(gk, oracle.Geom(2, 2, 64, 16, 2, 0))
    rng = np.random.default_rng(501)
    n = 2500                                           # more messages than threads of the chain kernel
    lens = rng.integers(0, 300, size=n)
    parent = [-1] * n
    for i in range(1, n):
        r = rng.random()
        if r < 0.7:
            parent[i] = i - 1 if rng.random() < 0.6 else int(rng.integers(0, i))
    data = rng.integers(0, 256, size=int(lens.sum()), dtype=np.uint8)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    want = oracle.fingerprints(data, off, parent, MODEL, TENANT)
    assert np.array_equal(_gpu_keys(ctx, data, off, parent), want)
    with pytest.raises(gk.GkError) as e:
        _gpu_keys(ctx, data, off, [-1, 1] + [-1] * (n - 2))
    assert e.value.code == -1
    ctx.close()


DIGEST_GEOMS = [oracle.Geom(2, 2, 64, 16, 2, 0),            # record 16 KiB: 4 full leaves
                oracle.Geom(5, 4, 64, 16, 2, 0),            # record 80 KiB: 20 leaves
                oracle.Geom(6, 4, 32, 8, 1, 2),             # record 12,480 B: 3 full leaves + 192 B
                oracle.Geom(10, 8, 64, 32, 1, 2),           # record 328,320 B: 80 full leaves + 640 B
                oracle.Geom(3, 2, 8, 4, 2, 0)]              # record 768 B: one short leaf


@pytest.mark.parametrize("og", DIGEST_GEOMS)
def test_blob_digests_parity(gk, og):
    T = og.page_tokens
    src = random_cache(og, 13, seed=510)
    rng = np.random.default_rng(511)
    lens = [3 * T, 1, 2 * T + 1, T, 4 * T - 1]
    blobs = []
    for n in lens:
        blob, _, code, _ = oracle.pack(og, src, rng.integers(0, 13, size=n_pages(og, n)).astype(np.int32), n)
        assert code == 0
        blobs.append(blob)
    blobs[2][len(blobs[2]) // 3] ^= 0x40               # a damaged copy is digested like any other bytes
    keys = rng.integers(0, 256, size=(len(lens), 32), dtype=np.uint8)
    want, want_pages = [], []
    for blob, n, key in zip(blobs, lens, keys):
        d, pages = oracle.blob_digest(og, blob, n, key.tobytes())
        want.append(np.frombuffer(d, dtype=np.uint8))
        want_pages.append(pages)
    want, want_pages = np.stack(want), np.concatenate(want_pages)

    ctx = _ctx(gk, og)
    dblobs = [torch.from_numpy(b).cuda() for b in blobs]
    jobs = [gk.Job(b, None, None, n) for b, n in zip(dblobs, lens)]
    dkeys = torch.from_numpy(keys).cuda()
    for with_pages in (True, False):
        digests = torch.full((len(lens), 32), 0xEE, dtype=torch.uint8, device="cuda")
        pages = torch.full((want_pages.shape[0], 32), 0xEE, dtype=torch.uint8, device="cuda") if with_pages else None
        ctx.gk_blob_digests(jobs, dkeys, digests, pages)
        torch.cuda.synchronize()
        assert np.array_equal(digests.cpu().numpy(), want)
        if with_pages:
            assert np.array_equal(pages.cpu().numpy(), want_pages)
    # a single job, and a call after a restore on the same context (shared workspace)
    one = torch.zeros(32, dtype=torch.uint8, device="cuda")
    ctx.gk_blob_digests(jobs[3:4], dkeys[3:4].contiguous(), one)
    torch.cuda.synchronize()
    assert np.array_equal(one.cpu().numpy(), want[3])
    with pytest.raises(gk.GkError):
        ctx.gk_blob_digests([gk.Job(None, None, None, T)], dkeys, one)
    ctx.close()


def test_confirmation_hash_sabotage_triple(gk):
    """Section 3, sabotage testing: the attack -- an intact record of one block filed under
    another block's key -- must succeed with the defence off and fail with it on.  The page
    checksums cannot see this attack (every record byte is intact); the digest, which is
    bound to the key, can."""
    from gpu_harness import dev_cache, gpu_restore
    og = oracle.Geom(5, 4, 64, 16, 2, 0)
    T = og.page_tokens
    n = 2 * T + 3
    src = random_cache(og, 9, seed=520)
    blob_a, sums_a, _, _ = oracle.pack(og, src, np.array([0, 1, 2], dtype=np.int32), n)
    blob_b, sums_b, _, _ = oracle.pack(og, src, np.array([3, 4, 5], dtype=np.int32), n)
    ctx = _ctx(gk, og)
    # keys of two different texts, and the digests stored with each record at save time
    text = np.frombuffer(b"first block of text " * 8 + b"another block, other text " * 8, dtype=np.uint8).copy()
    off = np.array([0, 160, text.size], dtype=np.uint64)
    keys = torch.from_numpy(_gpu_keys(ctx, text, off, None)).cuda()
    assert not torch.equal(keys[0], keys[1])
    stored = torch.zeros(2, 32, dtype=torch.uint8, device="cuda")
    da, db = torch.from_numpy(blob_a).cuda(), torch.from_numpy(blob_b).cuda()
    ctx.gk_blob_digests([gk.Job(da, None, None, n), gk.Job(db, None, None, n)], keys, stored)

    def load_under_key_a(record_blob, record_sums, record_digest, defence_on):
        """What a loader does with the record it found under key A."""
        if defence_on:
            got = torch.zeros(1, 32, dtype=torch.uint8, device="cuda")
            ctx.gk_blob_digests([gk.Job(torch.from_numpy(record_blob).cuda(), None, None, n)], keys[0:1].contiguous(), got)
            torch.cuda.synchronize()
            if not torch.equal(got[0], record_digest):
                return None                       # reported for recompute; nothing restored
        dst = random_cache(og, 6, seed=521)
        d = dev_cache(dst)
        mask, _ = gpu_restore(ctx, d, [oracle.Job(record_blob, record_sums, np.array([1, 3, 5], dtype=np.int32), n)])
        assert mask.tolist() == [0]               # the checksums see nothing wrong
        return d

    def holds(d, blob):
        back = torch.zeros(blob.size, dtype=torch.uint8, device="cuda")
        sums = torch.zeros(3, dtype=torch.int64, device="cuda")
        ctx.gk_pack_batch(d, [gk.Job(back, sums, torch.tensor([1, 3, 5], dtype=torch.int32, device="cuda"), n)])
        torch.cuda.synchronize()
        return np.array_equal(back.cpu().numpy(), blob)

    # attack: B's record (blob, checksums, digest) is filed under key A
    assert load_under_key_a(blob_b, sums_b, stored[1], defence_on=True) is None        # defence on: refused
    served = load_under_key_a(blob_b, sums_b, stored[1], defence_on=False)             # defence off: B's state is served for A
    assert served is not None and holds(served, blob_b)
    assert load_under_key_a(blob_b, sums_b, stored[1], defence_on=True) is None        # defence restored: refused again
    ok = load_under_key_a(blob_a, sums_a, stored[0], defence_on=True)                  # the honest record loads
    assert ok is not None and holds(ok, blob_a)
    ctx.close()
