"""CPU-side checks of the product: the shared library loads and exports every
entry point the public header declares, size arithmetic agrees with the oracle,
argument checks answer without a GPU, and the generated GF(2) tables are what
the kernels' algebra needs (checked with independent big-integer arithmetic)."""
import ctypes
import importlib.util
import os
import re

import numpy as np
import pytest

import oracle
import synth
from helpers import oracle_geom

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gk():
    from paper_2609_39358_b200 import build
    build.build()
    import paper_2609_39358_b200 as m
    return m


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gk_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(gk):
    lib = gk.load_library()
    names = _declared_functions()
    assert "gk_pack" in names and "gk_restore" in names and "gk_restore_host" in names
    for name in names:
        assert hasattr(lib, name), name
    from paper_2609_39358_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_header_is_plain_c_and_library_links_from_c(gk, tmp_path):
    import subprocess
    gk.load_library()
    libdir = os.path.join(ROOT, "paper_2609_39358_b200")
    exe = tmp_path / "abi_from_c"
    build = subprocess.run(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-pedantic",
                            os.path.join(ROOT, "tests", "c", "abi_from_c.c"), "-o", str(exe),
                            "-L" + libdir, "-l:libgk.so", "-Wl,-rpath," + libdir], capture_output=True, text=True)
    assert build.returncode == 0, build.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=60)
    assert run.returncode == 0 and "abi ok" in run.stdout, run.stdout + run.stderr


def test_blob_size_matches_oracle_on_all_workloads(gk):
    from gpu_harness import gk_geom
    cases = [(synth.TINY, 256), (synth.GQA7B, 4096), (synth.CORPUS, 1024), (synth.CORPUS, 280),
             (synth.FP8, 2048), (synth.STRESS, 17), (synth.STRESS, 4096), (synth.STRESS, 555)]
    for w, n in cases:
        og = oracle_geom(w)
        assert gk.gk_blob_size(gk_geom(og), n) == oracle.blob_size(og, n)


def test_blob_size_at_the_top_of_the_token_range(gk):
    """n_tokens = 2^32 - 1: the page count must not wrap (closed form P*S + n*tokB)."""
    from gpu_harness import gk_geom
    og = oracle.Geom(1, 1, 8, 16, 2, 0)
    n = 0xFFFFFFFF
    want_pages = -(-n // 16)
    want_bytes = n * 2 * 1 * 16
    assert gk.gk_blob_size(gk_geom(og), n) == (want_bytes, want_pages)
    assert oracle.blob_size(og, n) == (want_bytes, want_pages)


def test_argument_checks_without_gpu(gk):
    with pytest.raises(gk.GkError) as e:
        gk.gk_blob_size(gk.Geom(2, 2, 64, 16), 0)
    assert e.value.code == -1
    with pytest.raises(gk.GkError) as e:
        gk.gk_blob_size(gk.Geom(2, 2, 64, 16, dtype=7), 16)
    assert e.value.code == -2
    with pytest.raises(gk.GkError) as e:
        gk.gk_blob_size(gk.Geom(2, 1, 4, 16), 16)          # row = 8 bytes
    assert e.value.code == -2
    with pytest.raises(gk.GkError):
        gk.gk_blob_size(gk.Geom(2, 2, 64, 16, scale_kv=2), 16)   # bf16 has no scales
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(gk.GkError):                    # no device: fails loudly, no fallback
            gk.Context(gk.Geom(2, 2, 64, 16), 0)


# ---------------------------------------------------------------------------
# generated tables
# ---------------------------------------------------------------------------
P_FULL = (1 << 64) | 0x42F0E1EBA9EA3693


def _mod(v):
    while v.bit_length() > 64:
        v ^= P_FULL << (v.bit_length() - 65)
    return v


def _clmul(a, b):
    r = 0
    while b:
        if b & 1:
            r ^= a
        a <<= 1
        b >>= 1
    return r


def _load_gen():
    spec = importlib.util.spec_from_file_location(
        "gen_tables", os.path.join(ROOT, "paper_2609_39358_b200", "csrc", "gen_tables.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


def test_frobenius_rows_are_repeated_squaring():
    gen = _load_gen()
    rng = np.random.default_rng(5)
    for e in (10, 11, 12, 13):
        rows = gen.frob_rows(e)
        for _ in range(20):
            r = int(rng.integers(0, 1 << 63)) | (int(rng.integers(0, 2)) << 63)
            want = r
            for _ in range(e):
                want = _mod(_clmul(want, want))
            got = 0
            for m in range(64):
                if bin(rows[m] & r).count("1") & 1:
                    got |= 1 << m
            assert got == want


def test_generated_file_is_current_and_g8_constants():
    gen = _load_gen()
    path = os.path.join(ROOT, "paper_2609_39358_b200", "csrc", "gk_gf2_generated.inc")
    text = open(path).read()
    assert text == gen.generate()
    vals = [int(v, 16) for v in re.findall(r"0x([0-9A-F]{16})ull", text.split("GK_G8_INIT")[1].split("\n")[0])]
    assert len(vals) == 8
    for j, v in enumerate(vals):
        assert v == _mod(1 << (64 + j))


def test_bit_sliced_scheme_reproduces_crc():
    """The kernels' algebra, restated with Python integers: 8 threads, streams of
    stride 32*8 bits reduced by a plain shift register, raised to the 2^8-th power,
    merged with x^(distance) factors, plus init and final-xor terms."""
    gen = _load_gen()
    NT, e = 8, 8
    rng = np.random.default_rng(6)
    data = rng.integers(0, 256, size=NT * 4 * 24, dtype=np.uint8).tobytes()
    words = [int.from_bytes(data[4 * i:4 * i + 4], "little") for i in range(len(data) // 4)]
    total = 0
    for t in range(NT):
        acc = 0
        for s in range(32):
            r = 0
            for w in words[t::NT]:
                r = _mod((r << 1) | ((w >> s) & 1))
            for _ in range(e):
                r = _mod(_clmul(r, r))
            acc ^= r << (31 - s)
        total ^= _mod(_clmul(_mod(acc), _mod(1 << (32 * (NT - 1 - t) + 64))))
    ones = (1 << 64) - 1
    init = _mod(_clmul(ones, gen.xpow(8 * len(data))))
    crc = int(format(total ^ init ^ ones, "064b")[::-1], 2)
    assert crc == oracle.crc64(data)


def test_word_slot_merge_of_the_thread_polynomials():
    """How the kernels merge the threads of a CTA, restated with Python integers.  Every
    thread holds an UNREDUCED polynomial of up to 95 bits (three 32-bit words a0, a1, a2)
    that sits 32 bits above its right-hand neighbour's.  Inside a warp the words that fall on
    the same 32-bit slot are XORed across lanes, so that each lane is left with ONE word to
    multiply by its constant x^(32*(NT-1-t)+64); the two words that stick out above a warp's
    first lane are multiplied by two constants of their own.  The sum must equal the plain
    definition: sum over threads of poly_t * x^(32*(NT-1-t)+64) mod P."""
    rng = np.random.default_rng(7)
    for NT, WS in ((8, 4), (16, 4), (12, 2), (128, 32)):
        NW = NT // WS
        polys = [int(rng.integers(0, 1 << 62)) | (int(rng.integers(0, 1 << 33)) << 62) for _ in range(NT)]
        assert max(p.bit_length() for p in polys) <= 95
        want = 0
        for t, p in enumerate(polys):
            want ^= _mod(_clmul(p, 1 << (32 * (NT - 1 - t) + 64)))
        M = 0xFFFFFFFF
        a0 = [p & M for p in polys]
        a1 = [(p >> 32) & M for p in polys]
        a2 = [p >> 64 for p in polys]
        got = 0
        for w in range(NW):
            def word(arr, lane):
                return arr[w * WS + lane] if lane < WS else 0
            for lane in range(WS):
                t = w * WS + lane
                slot_word = a0[t] ^ word(a1, lane + 1) ^ word(a2, lane + 2)
                got ^= _mod(_clmul(slot_word, _mod(1 << (32 * (NT - 1 - t) + 64))))
            over0 = word(a1, 0) ^ word(a2, 1)
            over1 = word(a2, 0)
            got ^= _mod(_clmul(over0, _mod(1 << (32 * WS * (NW - w) + 64))))
            got ^= _mod(_clmul(over1, _mod(1 << (32 * WS * (NW - w) + 96))))
        assert got == want, (NT, WS)


def test_sha256_round_constants_in_the_kernel_source_match_the_derived_ones():
    """The kernels carry the SHA-256 round constants and initial state as typed literals;
    the oracle derives them from the primes.  Neither reads the other: compare them here."""
    text = open(os.path.join(ROOT, "paper_2609_39358_b200", "csrc", "gk_sha256.cuh")).read()
    table = text.split("kShaK[64] = {")[1].split("}")[0]
    typed_k = [int(v, 16) for v in re.findall(r"0x([0-9a-f]{8})u", table)]
    init = text.split("void sha_init(uint32_t h[8])")[1].split("}")[0]
    typed_h = [int(v, 16) for v in re.findall(r"0x([0-9a-f]{8})u", init)]
    k, h0 = oracle.sha256_constants()
    assert typed_k == [int(v) for v in k]
    assert typed_h == [int(v) for v in h0]
