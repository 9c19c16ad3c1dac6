"""Pins for the fingerprint / digest oracle: SHA-256 against the standard's published
example values and against the standard library's implementation, its derived constants
against floating-point roots of the primes, the message layouts against messages built
here byte by byte and hashed with hashlib, plus sensitivity and independence properties."""
import hashlib
import os
import struct

import numpy as np
import pytest

import oracle
from helpers import n_pages, random_cache

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _vectors():
    out = []
    with open(os.path.join(GOLDEN, "sha256_vectors.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            msg, digest = line.split()
            if msg == "-":
                data = b""
            elif msg.startswith("repeat:"):
                _, byte, count = msg.split(":")
                data = bytes.fromhex(byte) * int(count)
            else:
                data = bytes.fromhex(msg)
            out.append((data, digest))
    return out


def test_sha256_published_examples():
    vecs = _vectors()
    assert len(vecs) == 4
    for data, digest in vecs:
        assert oracle.sha256(data).hex() == digest


def test_sha256_against_hashlib_over_all_padding_cases():
    rng = np.random.default_rng(1)
    # every length around the 55/56/64-byte padding boundaries, then some long ones
    for n in list(range(0, 200)) + [1000, 4095, 4096, 4097, 65536 + 3]:
        data = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
        assert oracle.sha256(data) == hashlib.sha256(data).digest(), n


def test_sha256_constants_are_the_roots_of_the_primes():
    k, h0 = oracle.sha256_constants()
    primes = [p for p in range(2, 320) if all(p % d for d in range(2, int(p ** 0.5) + 1))][:64]
    assert primes[-1] == 311
    for i, p in enumerate(primes):
        # float64 carries ~52 bits; compare the top 20 fractional bits, then a few exact known values
        frac = (p ** (1.0 / 3.0)) % 1.0
        assert int(k[i]) >> 12 == int(frac * (1 << 20)), i
    for i, p in enumerate(primes[:8]):
        frac = (p ** 0.5) % 1.0
        assert int(h0[i]) >> 12 == int(frac * (1 << 20)), i
    assert int(k[0]) == 0x428A2F98 and int(k[63]) == 0xC67178F2      # first and last printed in FIPS 180-4, 4.2.2
    assert int(h0[0]) == 0x6A09E667 and int(h0[7]) == 0x5BE0CD19     # FIPS 180-4, 5.3.3
    # exactness: k is floor(cuberoot(p) * 2^32) mod 2^32, so (whole*2^32 + k)^3 <= p*2^96 < (.. + 1)^3
    for i, p in enumerate(primes):
        whole = int(round(p ** (1.0 / 3.0) - 0.5))
        x = (whole << 32) + int(k[i])
        assert x ** 3 <= p << 96 < (x + 1) ** 3, i


MODEL = bytes(range(32))
TENANT = bytes(range(100, 132))


def _key(msg: bytes, parent_key: bytes, model=MODEL, tenant=TENANT) -> bytes:
    inner = hashlib.sha256(msg + model + tenant + struct.pack("<Q", len(msg)) + b"GKF1").digest()
    return hashlib.sha256(parent_key + inner + b"GKF2").digest()


def test_fingerprints_against_messages_built_here():
    rng = np.random.default_rng(2)
    lens = [0, 1, 3, 4, 55, 56, 64, 100, 4096 * 4, 17, 16384, 5]
    parent = [-1, -1, 0, 2, -1, 4, 5, 6, 1, -1, 9, 10]
    data = rng.integers(0, 256, size=sum(lens), dtype=np.uint8)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    keys = oracle.fingerprints(data, off, parent, MODEL, TENANT)
    want = []
    for i, n in enumerate(lens):
        msg = data[int(off[i]):int(off[i + 1])].tobytes()
        pk = bytes(32) if parent[i] < 0 else want[parent[i]]
        want.append(_key(msg, pk))
    assert [k.tobytes() for k in keys] == want
    # no chains: parent None is the same as all -1
    k2 = oracle.fingerprints(data, off, None, MODEL, TENANT)
    k3 = oracle.fingerprints(data, off, [-1] * len(lens), MODEL, TENANT)
    assert np.array_equal(k2, k3)
    assert k2[0].tobytes() == want[0] and k2[2].tobytes() != want[2]
    with pytest.raises(ValueError):
        oracle.fingerprints(data, off, [-1, 1] + [-1] * 10, MODEL, TENANT)      # a block cannot follow itself


def test_fingerprint_separates_model_tenant_position_and_content():
    msg = np.frombuffer(b"the same block of prompt text, twice" * 10, dtype=np.uint8)
    data = np.concatenate([msg, msg])
    off = np.array([0, msg.size, 2 * msg.size], dtype=np.uint64)
    base = oracle.fingerprints(data, off, [-1, 0], MODEL, TENANT)
    assert base[0].tobytes() != base[1].tobytes()          # same text at another position: another key
    same = oracle.fingerprints(data, off, [-1, -1], MODEL, TENANT)
    assert same[0].tobytes() == same[1].tobytes()          # same text, same (first) position: same key
    other_model = oracle.fingerprints(data, off, [-1, 0], bytes(31) + b"\x01", TENANT)
    other_tenant = oracle.fingerprints(data, off, [-1, 0], MODEL, bytes(31) + b"\x01")
    flipped = data.copy()
    flipped[5] ^= 1
    other_text = oracle.fingerprints(flipped, off, [-1, 0], MODEL, TENANT)
    all_keys = {k.tobytes() for ks in (base, other_model, other_tenant, other_text) for k in ks}
    assert len(all_keys) == 8                              # a change in block 0 also moves block 1 through the chain
    # moving a byte across the boundary of two messages changes both keys (lengths are hashed)
    off2 = np.array([0, msg.size + 1, 2 * msg.size], dtype=np.uint64)
    moved = oracle.fingerprints(data, off2, [-1, -1], MODEL, TENANT)
    assert moved[0].tobytes() != same[0].tobytes() and moved[1].tobytes() != same[1].tobytes()


GEOMS = [oracle.Geom(3, 2, 8, 4, 2, 0),            # record 768 B: one short leaf per page
         oracle.Geom(6, 4, 32, 8, 1, 2),           # record 12,480 B: 3 full leaves + 192 B
         oracle.Geom(4, 4, 64, 16, 2, 0)]          # record 65,536 B: 16 full leaves exactly


@pytest.mark.parametrize("g", GEOMS)
@pytest.mark.parametrize("n_tokens_in_pages", [(0, 1), (1, 0), (2, 3), (3, -1)])
def test_blob_digest_against_messages_built_here(g, n_tokens_in_pages):
    full, extra = n_tokens_in_pages
    n = full * g.page_tokens + (extra if extra >= 0 else g.page_tokens - 1)
    src = random_cache(g, 7, seed=80)
    pt = np.random.default_rng(81).permutation(7)[:n_pages(g, n)].astype(np.int32)
    blob, _, code, _ = oracle.pack(g, src, pt, n)
    assert code == 0
    key = hashlib.sha256(b"some key").digest()
    digest, pages = oracle.blob_digest(g, blob, n, key)
    P = n_pages(g, n)
    want_pages = []
    for p in range(P):
        rec = blob[oracle.record_offset(g, p):oracle.record_offset(g, p) + oracle.record_bytes(g, n, p)].tobytes()
        leaves = b"".join(hashlib.sha256(rec[lo:lo + 4096] + b"GKL0").digest() for lo in range(0, len(rec), 4096))
        want_pages.append(hashlib.sha256(leaves + struct.pack("<Q", len(rec)) + b"GKP0").digest())
    assert [p.tobytes() for p in pages] == want_pages
    assert digest == hashlib.sha256(b"".join(want_pages) + key + struct.pack("<II", n, P) + b"GKB0").digest()


def test_blob_digest_moves_with_every_bit_key_order_and_length():
    g = GEOMS[0]
    n = 2 * g.page_tokens + 1
    src = random_cache(g, 5, seed=82)
    blob, _, _, _ = oracle.pack(g, src, np.array([3, 1, 4], dtype=np.int32), n)
    key = bytes(range(32))
    base, base_pages = oracle.blob_digest(g, blob, n, key)
    seen = {base}
    for byte in range(blob.size):                     # brute force: every bit of a 1,632-byte blob
        for bit in range(8):
            b = blob.copy()
            b[byte] ^= 1 << bit
            d, pages = oracle.blob_digest(g, b, n, key)
            assert d not in seen
            seen.add(d)
            page = min(byte // oracle.record_bytes(g, n, 0), 2)
            changed = [i for i in range(3) if pages[i].tobytes() != base_pages[i].tobytes()]
            assert changed == [page]                   # exactly the page that holds the byte
    assert oracle.blob_digest(g, blob, n, bytes(31) + b"\x01")[0] not in seen       # filed under another key
    swapped = blob.copy()
    R = oracle.record_bytes(g, n, 0)
    swapped[:R], swapped[R:2 * R] = blob[R:2 * R], blob[:R]
    assert oracle.blob_digest(g, swapped, n, key)[0] not in seen                    # pages in another order
    # same record bytes read as a different token count (full last page of a shorter layout is impossible
    # here, so compare n against n-? through the size fields): two full pages only
    d2, _ = oracle.blob_digest(g, blob[:2 * R], 2 * g.page_tokens, key)
    assert d2 not in seen
