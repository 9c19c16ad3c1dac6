"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself -- catalogue values, a library routine (stdlib lzma), long
division of polynomials written independently in Python, closed forms, textbook
special cases (memcpy), invariants and brute force on tiny inputs."""
import lzma
import os
import struct

import numpy as np
import pytest

import oracle
import synth
from helpers import (cache_bytes, clone_cache, make_cache, n_pages, oracle_geom, random_cache,
                     slab_bytes)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# CRC-64/XZ
# --------------------------------------------------------------------------
def _golden_vectors():
    out = []
    with open(os.path.join(GOLDEN, "crc64_xz_vectors.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            msg, crc = line.split()
            out.append((b"" if msg == "-" else bytes.fromhex(msg), int(crc, 16)))
    return out


def test_crc_catalogue_vectors():
    vecs = _golden_vectors()
    assert (b"123456789", 0x995DC9BBDF1939FA) in vecs
    for msg, crc in vecs:
        assert oracle.crc64_bitwise(msg) == crc
        assert oracle.crc64(msg) == crc


def _crc_by_long_division(msg: bytes) -> int:
    """CRC-64/XZ from the polynomial definition: message bits (least significant
    bit of each byte first) are the coefficients, highest degree first; the
    register is (M*x^64 + ones*x^n) mod P, xored with ones, bit-reversed."""
    P = (1 << 64) | 0x42F0E1EBA9EA3693
    n = 8 * len(msg)
    M = 0
    for i, b in enumerate(msg):
        for k in range(8):
            if (b >> k) & 1:
                M |= 1 << (n - 1 - (8 * i + k))
    ones = (1 << 64) - 1
    V = (M << 64) ^ (ones << n)
    for d in range(V.bit_length() - 1, 63, -1):
        if (V >> d) & 1:
            V ^= P << (d - 64)
    V ^= ones
    return int(format(V, "064b")[::-1], 2)


def test_crc_against_polynomial_long_division():
    rng = np.random.default_rng(1)
    for n in [0, 1, 2, 7, 8, 9, 63, 64, 65, 200, 1000]:
        msg = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
        assert oracle.crc64(msg) == _crc_by_long_division(msg)
    assert _crc_by_long_division(b"\x00") == 0x1FADA17364673F59


def _crc_from_xz_container(data: bytes) -> int:
    """The CRC-64 that liblzma stores for a one-block .xz stream."""
    x = lzma.compress(data, format=lzma.FORMAT_XZ, check=lzma.CHECK_CRC64)
    backward = struct.unpack("<I", x[-8:-4])[0]
    end = len(x) - 12 - 4 * (backward + 1)
    return int.from_bytes(x[end - 8:end], "little")


def test_crc_against_liblzma():
    rng = np.random.default_rng(2)
    for n in [1, 3, 16, 255, 256, 257, 4096, 16384, 100003]:
        msg = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
        want = _crc_from_xz_container(msg)
        assert oracle.crc64(msg) == want
        assert oracle.crc64_bitwise(msg) == want


def test_crc_table_equals_bitwise_and_streams():
    rng = np.random.default_rng(3)
    for n in [0, 1, 5, 64, 1023, 70001]:
        msg = rng.integers(0, 256, size=n, dtype=np.uint8)
        full = oracle.crc64_bitwise(msg)
        assert oracle.crc64(msg) == full
        for cut in {0, n // 3, n // 2, n}:
            assert oracle.crc64_continue(oracle.crc64(msg[:cut]), msg[cut:]) == full


def test_crc_residue():
    rng = np.random.default_rng(4)
    for n in [0, 1, 17, 4096]:
        msg = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
        tail = oracle.crc64(msg).to_bytes(8, "little")
        # register residue 0x49958C9ABD7D353F, i.e. CRC value = its complement
        assert oracle.crc64(msg + tail) == 0x49958C9ABD7D353F ^ 0xFFFFFFFFFFFFFFFF


def test_crc_affine_law():
    """crc(a^b) ^ crc(a) ^ crc(b) == crc(zeros) for equal lengths."""
    rng = np.random.default_rng(5)
    for n in [1, 8, 333, 4096]:
        a = rng.integers(0, 256, size=n, dtype=np.uint8)
        b = rng.integers(0, 256, size=n, dtype=np.uint8)
        z = np.zeros(n, dtype=np.uint8)
        assert oracle.crc64(a ^ b) ^ oracle.crc64(a) ^ oracle.crc64(b) == oracle.crc64(z)


def test_crc_detects_every_single_bit_flip_of_a_tiny_record():
    """Exhaustive over a 16 KiB record (131,072 bits) and over the checksum word."""
    rng = np.random.default_rng(6)
    rec = rng.integers(0, 256, size=16384, dtype=np.uint8)
    good = oracle.crc64(rec)
    seen = set()
    for byte in range(rec.size):
        for bit in range(8):
            rec[byte] ^= 1 << bit
            c = oracle.crc64(rec)
            rec[byte] ^= 1 << bit
            assert c != good
            seen.add(c)
    assert len(seen) == rec.size * 8          # all syndromes distinct as well
    for bit in range(64):
        assert (good ^ (1 << bit)) != good


def test_crc_detects_every_double_bit_flip_of_a_64_byte_record():
    rng = np.random.default_rng(7)
    rec = rng.integers(0, 256, size=64, dtype=np.uint8)
    good = oracle.crc64(rec)
    nb = rec.size * 8
    for i in range(nb):
        rec[i >> 3] ^= 1 << (i & 7)
        for j in range(i + 1, nb):
            rec[j >> 3] ^= 1 << (j & 7)
            assert oracle.crc64(rec) != good
            rec[j >> 3] ^= 1 << (j & 7)
        rec[i >> 3] ^= 1 << (i & 7)


# --------------------------------------------------------------------------
# Sizes: closed form blob_bytes = P*S + n*tokB, and the workloads' figures
# --------------------------------------------------------------------------
@pytest.mark.parametrize("w,n,want_bytes,want_pages", [
    (synth.TINY, 256, 256 * 1024, 16),
    (synth.GQA7B, 4096, 512 << 20, 256),
    (synth.CORPUS, 1024, 64 * (3 << 20), 64),
    (synth.CORPUS, 280, 17 * (3 << 20) + 8 * 192 * 1024, 18),
    (synth.FP8, 2048, 64 * 7872000, 64),
    (synth.STRESS, 17, 768 * 1024 + 48 * 1024, 2),
])
def test_blob_size_closed_form(w, n, want_bytes, want_pages):
    g = oracle_geom(w)
    nbytes, P = oracle.blob_size(g, n)
    S = g.layers * g.scale_kv * g.kv_heads * 4
    tokB = 2 * g.layers * g.kv_heads * g.head_dim * g.elem_bytes
    assert P == -(-n // g.page_tokens) == want_pages
    assert nbytes == P * S + n * tokB == want_bytes
    assert sum(oracle.record_bytes(g, n, p) for p in range(P)) == nbytes
    assert oracle.record_offset(g, P - 1) + oracle.record_bytes(g, n, P - 1) == nbytes


def test_corpus_total_bytes():
    g = oracle_geom(synth.CORPUS)
    total = sum(oracle.blob_size(g, n)[0] for n in synth.CORPUS_BLOCKS)
    pages = sum(oracle.blob_size(g, n)[1] for n in synth.CORPUS_BLOCKS)
    assert total == 19_181_076_480 and pages == 6098


# --------------------------------------------------------------------------
# pack
# --------------------------------------------------------------------------
SMALL = oracle.Geom(layers=3, kv_heads=2, head_dim=8, page_tokens=4, elem_bytes=2, scale_kv=0)
SMALL_FP8 = oracle.Geom(layers=3, kv_heads=4, head_dim=8, page_tokens=4, elem_bytes=1, scale_kv=2)


def test_pack_identity_table_page_major_is_memcpy():
    g, N = SMALL, 7
    src = random_cache(g, N, seed=10, layout="page_major")
    blob, sums, code, bad = oracle.pack(g, src, np.arange(N), N * g.page_tokens)
    assert code == 0 and bad == -1
    assert np.array_equal(blob, src.data)
    rec = 2 * g.layers * slab_bytes(g)
    for p in range(N):
        assert int(sums[p]) == _crc_from_xz_container(src.data[p * rec:(p + 1) * rec].tobytes())


def _pack_by_numpy_indexing(g, src, pt, n_tokens, layer_major_pages):
    """Independent statement of the record layout with numpy views."""
    L, H, D, T, E = g.layers, g.kv_heads, g.head_dim, g.page_tokens, g.elem_bytes
    arr = src.data.reshape(L, 2, layer_major_pages, T, H * D * E)
    sc = None if src.scales is None else src.scales.reshape(L, g.scale_kv, layer_major_pages, H * 4)
    out = []
    for p in range(n_pages(g, n_tokens)):
        t = min(T, n_tokens - p * T)
        if sc is not None:
            out.append(sc[:, :, pt[p], :].reshape(-1))
        out.append(arr[:, :, pt[p], :t, :].reshape(-1))
    return np.concatenate(out)


@pytest.mark.parametrize("g", [SMALL, SMALL_FP8])
@pytest.mark.parametrize("n_tokens", [1, 4, 5, 17, 20])
def test_pack_layout_against_numpy_views(g, n_tokens):
    N = 11
    src = random_cache(g, N, seed=11)
    pt = np.random.default_rng(12).permutation(N).astype(np.int32)
    blob, sums, code, _ = oracle.pack(g, src, pt, n_tokens)
    assert code == 0
    want = _pack_by_numpy_indexing(g, src, pt, n_tokens, N)
    assert np.array_equal(blob, want)
    for p in range(n_pages(g, n_tokens)):
        lo = oracle.record_offset(g, p)
        hi = lo + oracle.record_bytes(g, n_tokens, p)
        assert int(sums[p]) == _crc_by_long_division(blob[lo:hi].tobytes())


# head-major slabs ([head][token][dim]): full pages are the slab as it is, partial pages
# keep the first t tokens of every head
SMALL_HM = oracle.Geom(layers=3, kv_heads=4, head_dim=8, page_tokens=4, elem_bytes=2, scale_kv=0, head_major=1)
SMALL_HM_FP8 = oracle.Geom(layers=2, kv_heads=4, head_dim=16, page_tokens=8, elem_bytes=1, scale_kv=2, head_major=1)


@pytest.mark.parametrize("g", [SMALL_HM, SMALL_HM_FP8])
def test_head_major_full_pages_equal_token_major(g):
    """A full slab is opaque contiguous bytes in either layout, so on full pages the two
    layouts must give the same blob and checksums."""
    N = 9
    src = random_cache(g, N, seed=60)
    pt = np.random.default_rng(61).permutation(N)[:5].astype(np.int32)
    n = 5 * g.page_tokens
    g_tm = oracle.Geom(g.layers, g.kv_heads, g.head_dim, g.page_tokens, g.elem_bytes, g.scale_kv, 0)
    b1, s1, c1, _ = oracle.pack(g, src, pt, n)
    b2, s2, c2, _ = oracle.pack(g_tm, src, pt, n)
    assert c1 == c2 == 0 and np.array_equal(b1, b2) and np.array_equal(s1, s2)


@pytest.mark.parametrize("g", [SMALL_HM, SMALL_HM_FP8])
@pytest.mark.parametrize("n_tokens", [1, 3, 9, 14])
def test_head_major_layout_against_numpy_views(g, n_tokens):
    N = 7
    src = random_cache(g, N, seed=62)
    pt = np.random.default_rng(63).permutation(N).astype(np.int32)
    blob, sums, code, _ = oracle.pack(g, src, pt, n_tokens)
    assert code == 0
    L, H, D, T, E = g.layers, g.kv_heads, g.head_dim, g.page_tokens, g.elem_bytes
    arr = src.data.reshape(L, 2, N, H, T, D * E)
    sc = None if src.scales is None else src.scales.reshape(L, g.scale_kv, N, H * 4)
    parts = []
    for p in range(n_pages(g, n_tokens)):
        t = min(T, n_tokens - p * T)
        if sc is not None:
            parts.append(sc[:, :, pt[p], :].reshape(-1))
        parts.append(arr[:, :, pt[p], :, :t, :].reshape(-1))
    assert np.array_equal(blob, np.concatenate(parts))
    # round trip into a sentinel cache: valid tokens of every head restored, every other byte kept
    Nd = 9
    dst = random_cache(g, Nd, seed=64)
    before = clone_cache(dst)
    dpt = np.random.default_rng(65).permutation(Nd).astype(np.int32)[:n_pages(g, n_tokens)]
    mask, _ = oracle.restore(g, dst, [oracle.Job(blob, sums, dpt, n_tokens)])
    assert mask.tolist() == [0]
    d = dst.data.reshape(L, 2, Nd, H, T, D * E)
    b = before.data.reshape(L, 2, Nd, H, T, D * E)
    touched = np.zeros(Nd, dtype=bool)
    for p in range(n_pages(g, n_tokens)):
        t = min(T, n_tokens - p * T)
        assert np.array_equal(d[:, :, dpt[p], :, :t], arr[:, :, pt[p], :, :t])
        assert np.array_equal(d[:, :, dpt[p], :, t:], b[:, :, dpt[p], :, t:])
        touched[dpt[p]] = True
    assert np.array_equal(d[:, :, ~touched], b[:, :, ~touched])


def test_pack_is_a_permutation_of_the_valid_bytes():
    g, N = SMALL, 9
    src = random_cache(g, N, seed=13)
    pt = np.array([8, 0, 3], dtype=np.int32)
    n = 2 * g.page_tokens + 1
    blob, _, _, _ = oracle.pack(g, src, pt, n)
    arr = src.data.reshape(g.layers, 2, N, g.page_tokens, -1)
    valid = np.concatenate([arr[:, :, 8].reshape(-1), arr[:, :, 0].reshape(-1),
                            arr[:, :, 3, :1].reshape(-1)])
    assert np.array_equal(np.sort(blob), np.sort(valid))


def test_pack_duplicates_allowed_out_of_range_rejected():
    g, N = SMALL, 4
    src = random_cache(g, N, seed=14)
    blob, sums, code, bad = oracle.pack(g, src, np.array([1, 1], dtype=np.int32), 8)
    assert code == 0 and np.array_equal(blob[:blob.size // 2], blob[blob.size // 2:])
    for bad_id in (-1, N):
        blob, sums, code, bad = oracle.pack(g, src, np.array([0, bad_id, 2], dtype=np.int32), 12)
        assert code == oracle.CODE_PAGE_TABLE and bad == 1
        assert not blob.any() and not sums.any()


# --------------------------------------------------------------------------
# restore: round trip, fail-closed, codes
# --------------------------------------------------------------------------
def _sentinel_cache(g, N, seed):
    return random_cache(g, N, seed)


@pytest.mark.parametrize("g", [SMALL, SMALL_FP8])
@pytest.mark.parametrize("n_tokens", [3, 4, 9, 16])
def test_round_trip_and_untouched_rest(g, n_tokens):
    Ns, Nd = 6, 10
    src = random_cache(g, Ns, seed=20)
    P = n_pages(g, n_tokens)
    spt = np.random.default_rng(21).permutation(Ns).astype(np.int32)[:P]
    blob, sums, _, _ = oracle.pack(g, src, spt, n_tokens)
    dst = _sentinel_cache(g, Nd, seed=22)
    before = clone_cache(dst)
    dpt = np.random.default_rng(23).permutation(Nd).astype(np.int32)[:P]
    mask, fb = oracle.restore(g, dst, [oracle.Job(blob, sums, dpt, n_tokens)])
    assert mask.tolist() == [0] and fb.tolist() == [-1]
    L, T = g.layers, g.page_tokens
    s = src.data.reshape(L, 2, Ns, T, -1)
    d = dst.data.reshape(L, 2, Nd, T, -1)
    b = before.data.reshape(L, 2, Nd, T, -1)
    touched = np.zeros(Nd, dtype=bool)
    for p in range(P):
        t = min(T, n_tokens - p * T)
        assert np.array_equal(d[:, :, dpt[p], :t], s[:, :, spt[p], :t])      # restored == saved
        assert np.array_equal(d[:, :, dpt[p], t:], b[:, :, dpt[p], t:])      # tail of a partial page
        touched[dpt[p]] = True
    assert np.array_equal(d[:, :, ~touched], b[:, :, ~touched])              # unmapped pages
    if g.scale_kv:
        ss = src.scales.reshape(L, g.scale_kv, Ns, -1)
        ds = dst.scales.reshape(L, g.scale_kv, Nd, -1)
        bs = before.scales.reshape(L, g.scale_kv, Nd, -1)
        for p in range(P):
            assert np.array_equal(ds[:, :, dpt[p]], ss[:, :, spt[p]])
        assert np.array_equal(ds[:, :, ~touched], bs[:, :, ~touched])
    # a second pack from the destination reproduces the record bytes and checksums
    blob2, sums2, _, _ = oracle.pack(g, dst, dpt, n_tokens)
    assert np.array_equal(blob2, blob) and np.array_equal(sums2, sums)


@pytest.mark.parametrize("g", [oracle.Geom(1, 1, 8, 2, 2, 0), oracle.Geom(1, 2, 4, 2, 1, 2)])
def test_every_single_bit_flip_is_rejected_and_nothing_is_written(g):
    N = 3
    src = random_cache(g, N, seed=30)
    n_tokens = 3                                # one full page and one partial page
    blob, sums, _, _ = oracle.pack(g, src, np.array([2, 0], dtype=np.int32), n_tokens)
    dpt = np.array([1, 2], dtype=np.int32)
    clean = _sentinel_cache(g, N, seed=31)
    rec0 = oracle.record_bytes(g, n_tokens, 0)
    for bit in range(blob.size * 8):
        bad = blob.copy()
        bad[bit >> 3] ^= 1 << (bit & 7)
        dst = clone_cache(clean)
        mask, fb = oracle.restore(g, dst, [oracle.Job(bad, sums, dpt, n_tokens)])
        assert mask[0] == oracle.CODE_CHECKSUM
        assert fb[0] == (0 if (bit >> 3) < rec0 else 1)
        assert np.array_equal(dst.data, clean.data)
        if g.scale_kv:
            assert np.array_equal(dst.scales, clean.scales)
    for bit in range(sums.size * 64):           # damage in the checksum array instead
        bad = sums.copy()
        bad[bit // 64] ^= np.uint64(1) << np.uint64(bit % 64)
        dst = clone_cache(clean)
        mask, fb = oracle.restore(g, dst, [oracle.Job(blob, bad, dpt, n_tokens)])
        assert mask[0] == oracle.CODE_CHECKSUM and fb[0] == bit // 64
        assert np.array_equal(dst.data, clean.data)


def test_sabotage_triple_defence_on_off_on():
    """Section 3, sabotage testing: the attack must fail with the defence on,
    succeed with it off, and fail again with it restored."""
    g, N = SMALL, 8
    src = random_cache(g, N, seed=40)
    n = 10
    spt = np.array([5, 1, 2], dtype=np.int32)
    blob, sums, _, _ = oracle.pack(g, src, spt, n)
    bad = blob.copy()
    bad[100] ^= 0x40
    dpt = np.array([0, 7, 3], dtype=np.int32)
    clean = _sentinel_cache(g, N, seed=41)

    dst = clone_cache(clean)
    mask, _ = oracle.restore(g, dst, [oracle.Job(bad, sums, dpt, n)])
    assert mask[0] == oracle.CODE_CHECKSUM and np.array_equal(dst.data, clean.data)

    dst = clone_cache(clean)
    mask, _ = oracle.restore(g, dst, [oracle.Job(bad, sums, dpt, n)], flags=oracle.FLAG_SKIP_VERIFY)
    assert mask[0] == 0 and not np.array_equal(dst.data, clean.data)
    good_dst = clone_cache(clean)
    oracle.restore(g, good_dst, [oracle.Job(blob, sums, dpt, n)])
    assert not np.array_equal(dst.data, good_dst.data)      # the wrong bytes really landed

    dst = clone_cache(clean)
    mask, _ = oracle.restore(g, dst, [oracle.Job(bad, sums, dpt, n)])
    assert mask[0] == oracle.CODE_CHECKSUM and np.array_equal(dst.data, clean.data)


@pytest.mark.parametrize("g", [SMALL, SMALL_FP8])
def test_single_pass_reading(g):
    """Optional reading: a block whose only fault is a checksum mismatch is reported but its
    own pages receive the unverified bytes; every other rule stands."""
    N = 14
    T = g.page_tokens
    src = random_cache(g, 9, seed=55)
    lens = [2 * T + 1, T, 3 * T, 1, 2 * T]
    rng = np.random.default_rng(56)
    perm = rng.permutation(N).astype(np.int32)
    jobs, used = [], 0
    for n in lens:
        P = n_pages(g, n)
        blob, sums, _, _ = oracle.pack(g, src, rng.integers(0, 9, size=P).astype(np.int32), n)
        jobs.append(oracle.Job(blob, sums, perm[used:used + P].copy(), n))
        used += P
    clean = _sentinel_cache(g, N, seed=57)
    # all good: the flag changes nothing
    a, b = clone_cache(clean), clone_cache(clean)
    ma, fa = oracle.restore(g, a, jobs)
    mb, fb_ = oracle.restore(g, b, jobs, flags=oracle.FLAG_SINGLE_PASS)
    assert ma.tolist() == mb.tolist() == [0] * 5 and fa.tolist() == fb_.tolist()
    assert np.array_equal(a.data, b.data)
    # job 0 damaged in its partial page, job 2 with an out-of-range id, job 3 missing, job 4 damaged
    jobs[0].blob[-1] ^= 0x01
    jobs[2].page_table[1] = N + 3
    jobs[3] = oracle.Job(None, None, jobs[3].page_table, 1)
    jobs[4].checksums[0] ^= np.uint64(1)
    strict, single, forced = clone_cache(clean), clone_cache(clean), clone_cache(clean)
    ms, fs = oracle.restore(g, strict, jobs)
    m1, f1 = oracle.restore(g, single, jobs, flags=oracle.FLAG_SINGLE_PASS)
    assert ms.tolist() == m1.tolist() == [1, 0, 2, 3, 1]             # same report either way
    assert fs.tolist() == f1.tolist() == [2, -1, 1, -1, 0]
    # what differs are exactly the pages of the two checksum failures, which hold what a
    # restore without any check would have put there
    oracle.restore(g, forced, [jobs[0], jobs[4]], flags=oracle.FLAG_SKIP_VERIFY)
    expect = clone_cache(strict)
    L = g.layers
    for jb in (jobs[0], jobs[4]):
        for page in jb.page_table[:n_pages(g, jb.n_tokens)]:
            for arr_e, arr_f, per_page in ((expect.data, forced.data, slab_bytes(g)),) + (
                    ((expect.scales, forced.scales, g.kv_heads * 4),) if g.scale_kv else ()):
                kvn = 2 if per_page == slab_bytes(g) else g.scale_kv
                ve = arr_e.reshape(L, kvn, N, per_page)
                vf = arr_f.reshape(L, kvn, N, per_page)
                ve[:, :, page] = vf[:, :, page]
    assert np.array_equal(single.data, expect.data)
    if g.scale_kv:
        assert np.array_equal(single.scales, expect.scales)
    assert not np.array_equal(single.data, strict.data)


def test_codes_and_first_bad_page():
    g, N = SMALL, 12
    src = random_cache(g, N, seed=50)
    n = 3 * g.page_tokens
    blob, sums, _, _ = oracle.pack(g, src, np.array([0, 1, 2], dtype=np.int32), n)
    bad2 = blob.copy()
    bad2[oracle.record_offset(g, 1) + 5] ^= 1
    bad2[oracle.record_offset(g, 2) + 5] ^= 1
    clean = _sentinel_cache(g, N, seed=51)
    blob1, sums1, _, _ = oracle.pack(g, src, np.array([0], dtype=np.int32), 1)
    jobs = [
        oracle.Job(blob, sums, np.array([0, 1, 2], dtype=np.int32), n),       # ok
        oracle.Job(bad2, sums, np.array([3, 4, 5], dtype=np.int32), n),       # checksum, page 1 first
        oracle.Job(None, sums, np.array([6, 7, 8], dtype=np.int32), n),       # missing
        oracle.Job(blob, None, np.array([6, 7, 8], dtype=np.int32), n),       # missing
        oracle.Job(blob, sums, np.array([9, 12, -1], dtype=np.int32), n),     # out of range at 1
        oracle.Job(blob, sums, np.array([6, 10, 11], dtype=np.int32), n),     # dup with next at 1
        oracle.Job(blob, sums, np.array([8, 7, 10], dtype=np.int32), n),      # dup with previous at 2
        oracle.Job(blob1, sums1, np.array([9], dtype=np.int32), 1),           # page 9: job 4 never claimed it
    ]
    dst = clone_cache(clean)
    mask, fb = oracle.restore(g, dst, jobs)
    assert mask.tolist() == [0, 1, 3, 3, 2, 2, 2, 0]
    assert fb.tolist() == [-1, 1, -1, -1, 1, 1, 2, -1]
    d = dst.data.reshape(g.layers, 2, N, g.page_tokens, -1)
    c = clean.data.reshape(g.layers, 2, N, g.page_tokens, -1)
    s = src.data.reshape(g.layers, 2, N, g.page_tokens, -1)
    assert np.array_equal(d[:, :, [0, 1, 2]], s[:, :, [0, 1, 2]])
    assert np.array_equal(d[:, :, 9, :1], s[:, :, 0, :1])
    assert np.array_equal(d[:, :, 9, 1:], c[:, :, 9, 1:])
    for page in (3, 4, 5, 6, 7, 8, 10, 11):
        assert np.array_equal(d[:, :, page], c[:, :, page])


def test_one_failed_job_does_not_stop_the_others():
    """Tiny workload: 4 blocks, one flipped bit, 3 ok and 1 rejected."""
    w = synth.TINY
    g = oracle_geom(w)
    src_pages = 64
    src = make_cache(g, src_pages,
                     synth.kv_bytes_bf16(cache_bytes(g, src_pages) // 2, w.sigma, w.seed(0)).numpy())
    perm = synth.page_permutation(synth.TINY_DST_PAGES, w.seed(1))
    jobs = []
    for i, n in enumerate(synth.TINY_BLOCKS):
        blob, sums, code, _ = oracle.pack(g, src, np.arange(16 * i, 16 * i + 16, dtype=np.int32), n)
        assert code == 0
        jobs.append(oracle.Job(blob, sums, perm[16 * i:16 * i + 16], n))
    rng = np.random.default_rng(w.seed(2))
    victim = int(rng.integers(0, 4))
    bit = int(synth.bit_flip_positions(jobs[victim].blob.size * 8, 1, w.seed(3))[0])
    jobs[victim].blob[bit >> 3] ^= 1 << (bit & 7)
    clean = make_cache(g, synth.TINY_DST_PAGES,
                       synth.sentinel_bytes(cache_bytes(g, synth.TINY_DST_PAGES), w.seed(4)).numpy().copy())
    dst = clone_cache(clean)
    mask, fb = oracle.restore(g, dst, jobs)
    want = [0, 0, 0, 0]
    want[victim] = 1
    assert mask.tolist() == want
    assert fb[victim] == (bit >> 3) // oracle.record_bytes(g, 256, 0)
    d = dst.data.reshape(g.layers, 2, synth.TINY_DST_PAGES, g.page_tokens, -1)
    c = clean.data.reshape(g.layers, 2, synth.TINY_DST_PAGES, g.page_tokens, -1)
    s = src.data.reshape(g.layers, 2, src_pages, g.page_tokens, -1)
    for i in range(4):
        pages = perm[16 * i:16 * i + 16]
        if i == victim:
            assert np.array_equal(d[:, :, pages], c[:, :, pages])
        else:
            assert np.array_equal(d[:, :, pages], s[:, :, 16 * i:16 * i + 16])
    rest = perm[64:]
    assert np.array_equal(d[:, :, rest], c[:, :, rest])


# --------------------------------------------------------------------------
# streaming restore through a ring of pages (Section 4.3, long windows at flat memory)
# --------------------------------------------------------------------------
def _valid_prefix(g, cache, page, t):
    """Valid bytes (first t tokens, token-major) of every slab of a page, plus its scales."""
    L, H, D, T, E = g.layers, g.kv_heads, g.head_dim, g.page_tokens, g.elem_bytes
    arr = cache.data.reshape(L, 2, cache.num_pages, T, H * D * E)
    out = [arr[:, :, page, :t].reshape(-1)]
    if cache.scales is not None:
        out.append(cache.scales.reshape(L, g.scale_kv, cache.num_pages, H * 4)[:, :, page].reshape(-1))
    return np.concatenate(out)


@pytest.mark.parametrize("g", [oracle.Geom(3, 2, 8, 4, 2, 0), oracle.Geom(2, 4, 16, 8, 1, 2)])
@pytest.mark.parametrize("ring_pages", [5, 8, 64])
def test_stream_restore_windows_contents_and_fail_closed(g, ring_pages):
    T = g.page_tokens
    src = random_cache(g, 11, seed=70)
    rng = np.random.default_rng(71)
    lens = [2 * T, 1, 3 * T + 1, T, 5 * T, 2 * T - 1, T + 1, 4 * T, 1, 3 * T]
    tables = [rng.integers(0, 11, size=n_pages(g, n)).astype(np.int32) for n in lens]
    jobs = []
    for pt, n in zip(tables, lens):
        blob, sums, code, _ = oracle.pack(g, src, pt, n)
        assert code == 0
        jobs.append(oracle.Job(blob, sums, None, n))
    jobs[3].blob[0] ^= 0x80                       # damaged
    jobs[6] = oracle.Job(None, None, None, lens[6])  # missing
    ring = random_cache(g, ring_pages, seed=72)
    seen = []
    state = {"before": clone_cache(ring), "next_job": 0}

    def consume(first_job, count, first_pages):
        # windows arrive in order, are contiguous, and are maximal
        assert first_job == state["next_job"] and count >= 1
        pages = [n_pages(g, lens[first_job + k]) for k in range(count)]
        assert first_pages == [sum(pages[:k]) for k in range(count)]
        assert sum(pages) <= ring_pages
        nxt = first_job + count
        if nxt < len(lens):
            assert sum(pages) + n_pages(g, lens[nxt]) > ring_pages
        # contents: a good job's pages hold the saved bytes; every other byte of the ring
        # (bad jobs' pages, tails of partial pages, pages beyond the window) is as it was
        expect = clone_cache(state["before"])
        for k in range(count):
            j = first_job + k
            if j in (3, 6):
                continue
            for p in range(pages[k]):
                t = min(T, lens[j] - p * T)
                assert np.array_equal(_valid_prefix(g, ring, first_pages[k] + p, t),
                                      _valid_prefix(g, src, tables[j][p], t))
                # graft the saved bytes into the expectation through numpy views
                L, H, D, E = g.layers, g.kv_heads, g.head_dim, g.elem_bytes
                ev = expect.data.reshape(L, 2, ring_pages, T, H * D * E)
                sv = src.data.reshape(L, 2, 11, T, H * D * E)
                ev[:, :, first_pages[k] + p, :t] = sv[:, :, tables[j][p], :t]
                if g.scale_kv:
                    es = expect.scales.reshape(L, g.scale_kv, ring_pages, H * 4)
                    ss = src.scales.reshape(L, g.scale_kv, 11, H * 4)
                    es[:, :, first_pages[k] + p] = ss[:, :, tables[j][p]]
        assert np.array_equal(ring.data, expect.data)
        if g.scale_kv:
            assert np.array_equal(ring.scales, expect.scales)
        state["before"] = clone_cache(ring)
        state["next_job"] = nxt
        seen.append((first_job, count))

    mask, fb = oracle.restore_stream(g, ring, jobs, consume)
    assert state["next_job"] == len(lens)
    assert mask.tolist() == [0, 0, 0, 1, 0, 0, 3, 0, 0, 0]
    assert fb.tolist() == [-1, -1, -1, 0, -1, -1, -1, -1, -1, -1]
    if ring_pages == 64:
        assert seen == [(0, len(lens))]            # everything fits: one window
    if ring_pages == 5:
        assert (4, 1) in seen                      # the 5-page job fills a window alone


def test_stream_restore_refuses_a_job_larger_than_the_ring():
    g = oracle.Geom(3, 2, 8, 4, 2, 0)
    src = random_cache(g, 6, seed=73)
    blob, sums, _, _ = oracle.pack(g, src, np.arange(6, dtype=np.int32), 6 * g.page_tokens)
    small, _s, _, _ = oracle.pack(g, src, np.arange(1, dtype=np.int32), 1)
    ring = random_cache(g, 5, seed=74)
    before = clone_cache(ring)
    with pytest.raises(ValueError):
        oracle.restore_stream(g, ring, [oracle.Job(small, _s, None, 1), oracle.Job(blob, sums, None, 6 * g.page_tokens)])
    assert np.array_equal(ring.data, before.data)   # not even the first job was restored


# --------------------------------------------------------------------------
# layer-wise save and load (the ordinary format once per group of layers)
# --------------------------------------------------------------------------
def _full_geom(g, n_groups):
    return oracle.Geom(g.layers * n_groups, g.kv_heads, g.head_dim, g.page_tokens, g.elem_bytes, g.scale_kv, g.head_major)


@pytest.mark.parametrize("g", [oracle.Geom(2, 2, 8, 4, 2, 0), oracle.Geom(1, 4, 16, 8, 1, 2),
                               oracle.Geom(2, 4, 8, 4, 2, 0, head_major=1)])
@pytest.mark.parametrize("n_tokens_extra", [0, 1, 3])
def test_layerwise_blob_is_the_ordinary_blob_cut_by_layer_groups(g, n_tokens_extra):
    G = 3
    full = _full_geom(g, G)
    N, T = 7, g.page_tokens
    n = 2 * T + n_tokens_extra
    src = random_cache(full, N, seed=90)
    pt = np.random.default_rng(91).permutation(N)[:n_pages(full, n)].astype(np.int32)
    whole, _, code, _ = oracle.pack(full, src, pt, n)
    assert code == 0
    lw, sums, code, _ = oracle.pack_layerwise(g, G, src, pt, n)
    assert code == 0 and lw.size == whole.size
    P = n_pages(full, n)
    group_bytes, _ = oracle.blob_size(g, n)
    S_full = full.layers * full.scale_kv * full.kv_heads * 4
    S_g = S_full // G
    for k in range(G):
        for p in range(P):
            rec_full = whole[oracle.record_offset(full, p):][:oracle.record_bytes(full, n, p)]
            data_full = rec_full[S_full:]
            dg = data_full.size // G
            want = np.concatenate([rec_full[k * S_g:(k + 1) * S_g], data_full[k * dg:(k + 1) * dg]])
            got = lw[k * group_bytes + oracle.record_offset(g, p):][:oracle.record_bytes(g, n, p)]
            assert np.array_equal(got, want), (k, p)
            assert int(sums[k * P + p]) == oracle.crc64(want)
    # every byte of the ordinary blob appears exactly once
    assert np.array_equal(np.sort(lw), np.sort(whole))


@pytest.mark.parametrize("g", [oracle.Geom(2, 2, 8, 4, 2, 0), oracle.Geom(1, 4, 16, 8, 1, 2)])
def test_layerwise_restore_groups_are_independent_and_in_order(g):
    G = 3
    full = _full_geom(g, G)
    T, N = g.page_tokens, 12
    src = random_cache(full, 8, seed=92)
    lens = [2 * T + 1, T, 3 * T - 1]
    rng = np.random.default_rng(93)
    perm = rng.permutation(N).astype(np.int32)
    lw_jobs, std_jobs, used = [], [], 0
    for n in lens:
        P = n_pages(full, n)
        spt = rng.integers(0, 8, size=P).astype(np.int32)
        b, s_, _, _ = oracle.pack_layerwise(g, G, src, spt, n)
        wb, ws, _, _ = oracle.pack(full, src, spt, n)
        lw_jobs.append(oracle.Job(b, s_, perm[used:used + P].copy(), n))
        std_jobs.append(oracle.Job(wb, ws, perm[used:used + P].copy(), n))
        used += P
    clean = _sentinel_cache(full, N, seed=94)
    # all good: same destination as the ordinary restore of the ordinary blobs
    a, b_ = clone_cache(clean), clone_cache(clean)
    oracle.restore(full, a, std_jobs)
    seen = []
    mask, fb, gm = oracle.restore_layerwise(g, G, b_, lw_jobs, lambda k, l0, nl: seen.append((k, l0, nl)))
    assert mask.tolist() == [0, 0, 0] and fb.tolist() == [-1, -1, -1] and gm.tolist() == [[0, 0, 0]] * 3
    assert seen == [(0, 0, g.layers), (1, g.layers, g.layers), (2, 2 * g.layers, g.layers)]
    assert np.array_equal(a.data, b_.data)
    if g.scale_kv:
        assert np.array_equal(a.scales, b_.scales)
    # job 0 damaged inside group 1 (second page), job 2 inside groups 0 and 2
    gb0, P0 = oracle.blob_size(g, lens[0])
    gb2, P2 = oracle.blob_size(g, lens[2])
    lw_jobs[0].blob[gb0 + oracle.record_offset(g, 1) + 5] ^= 0x01
    lw_jobs[2].blob[3] ^= 0x80
    lw_jobs[2].checksums[2 * P2 + 2] ^= np.uint64(4)
    c = clone_cache(clean)
    snapshots = []
    mask, fb, gm = oracle.restore_layerwise(g, G, c, lw_jobs, lambda k, l0, nl: snapshots.append(c.data.copy()))
    assert mask.tolist() == [1, 0, 1] and fb.tolist() == [1, -1, 0]
    assert gm.tolist() == [[0, 0, 1], [1, 0, 0], [0, 0, 1]]
    # layer by layer: a (job, group) that verified holds the ordinary result, one that failed the sentinel
    L_full = full.layers
    va = a.data.reshape(L_full, -1)
    vz = clean.data.reshape(L_full, -1)
    vc = c.data.reshape(L_full, -1)
    per_layer = va.shape[1]
    slab = slab_bytes(full)
    for k in range(G):
        for l in range(k * g.layers, (k + 1) * g.layers):
            expect = vz[l].copy().reshape(2, N, slab)
            good = va[l].reshape(2, N, slab)
            for j, jb in enumerate(lw_jobs):
                if gm[k][j] == 0:
                    for page in jb.page_table:
                        expect[:, page] = good[:, page]
            assert np.array_equal(vc[l].reshape(2, N, slab), expect), (k, l)
    # in order: after the call-back of group k the layers of the groups up to k are final
    for k in range(G):
        snap = snapshots[k].reshape(L_full, per_layer)
        assert np.array_equal(snap[:(k + 1) * g.layers], vc[:(k + 1) * g.layers])
        assert np.array_equal(snap[(k + 1) * g.layers:], vz[(k + 1) * g.layers:])
