"""gk_page_checksums_noalloc: the context-free entry point that allocates nothing.

Some users of libgk cannot call cudaMalloc at the moment they need a checksum --
an engine whose KV-cache pool already owns all free HBM, or a scrubber running
beside it -- so this entry point keeps all of its scratch in a fixed array inside
the library.  The test checks it against gk_page_checksums (the context-based
entry point, itself checked against the CPU oracle elsewhere) on two calls in a
row that differ in length and content, because the shared scratch still holds the
first call's data when the second one starts.  The file name makes pytest collect
it last.
"""
import os
import re
import shutil

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _library_or_skip():
    """The library as built in-tree; without it and without nvcc there is nothing to test."""
    import paper_2609_39358_b200 as gk
    from paper_2609_39358_b200 import build
    if not os.path.exists(build.LIB_PATH) and not (shutil.which("nvcc") or os.path.exists("/usr/local/cuda/bin/nvcc")):
        pytest.skip("libgk.so is not built and nvcc is not available")
    build.build()
    return gk


def test_limits_in_the_binding_are_those_of_the_header():
    gk = _library_or_skip()
    text = open(os.path.join(ROOT, "include", "gk.h")).read()
    limits = {k: int(v) for k, v in re.findall(r"#define (GK_NOALLOC_MAX_[A-Z_]+) (\d+)u", text)}
    assert limits == {"GK_NOALLOC_MAX_PAGES": gk.binding.GK_NOALLOC_MAX_PAGES,
                      "GK_NOALLOC_MAX_PAGE_TOKENS": gk.binding.GK_NOALLOC_MAX_PAGE_TOKENS}


def test_too_large_requests_are_rejected_before_any_gpu_work():
    gk = _library_or_skip()
    geom = gk.Geom(2, 2, 64, 16)
    blob = torch.zeros(64, dtype=torch.uint8)
    sums = torch.zeros(8, dtype=torch.int64)
    with pytest.raises(gk.GkError) as e:
        gk.gk_page_checksums_noalloc(geom, blob, (gk.binding.GK_NOALLOC_MAX_PAGES + 1) * 16, sums, 0, 0)
    assert e.value.code == -7
    with pytest.raises(gk.GkError) as e:
        gk.gk_page_checksums_noalloc(gk.Geom(2, 2, 64, 512), blob, 512, sums, 0, 0)
    assert e.value.code == -7
    with pytest.raises(gk.GkError) as e:
        gk.gk_page_checksums_noalloc(geom, blob, 0, sums, 0, 0)
    assert e.value.code == -1


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [
    (5, 4, 64, 16, 0, 0),      # bf16, 80 KiB records
    (10, 8, 64, 32, 1, 2),     # fp8 with a scale section, ragged record length
])
def test_noalloc_matches_context_entry_point_twice_in_a_row(shape):
    import paper_2609_39358_b200 as gk
    L, H, D, T, dtype, scale_kv = shape
    geom = gk.Geom(L, H, D, T, dtype, scale_kv)
    ctx = gk.Context(geom, 0)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(20260927)
    # second call is shorter than the first and ends in a partial page: stale
    # remainders or counters from call one would show up here
    import oracle
    cases = []
    for n_tokens in (7 * T + 3, 2 * T + 1):
        nbytes, P = gk.gk_blob_size(geom, n_tokens)
        blob = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda", generator=gen)
        want = torch.zeros(P, dtype=torch.int64, device="cuda")
        ctx.gk_page_checksums(blob, n_tokens, want)
        got = torch.full((P,), -1, dtype=torch.int64, device="cuda")
        cases.append((n_tokens, blob, want, got))
    torch.cuda.synchronize()
    ctx.close()
    # what the entry point exists for: with everything the test needs already in place, the two
    # calls leave the device's free memory exactly where it was (the first call on a device does
    # the one-time set-up, so warm that up before measuring)
    gk.gk_page_checksums_noalloc(geom, cases[0][1], cases[0][0], cases[0][3], 0)
    torch.cuda.synchronize()
    cases[0][3].fill_(-1)
    free_before = torch.cuda.mem_get_info()[0]
    for n_tokens, blob, want, got in cases:
        gk.gk_page_checksums_noalloc(geom, blob, n_tokens, got, 0)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    for n_tokens, blob, want, got in cases:
        assert torch.equal(got, want)          # integer work: bit-exact
        # and every page against the CPU oracle's CRC-64 of the record bytes
        host = blob.cpu().numpy()
        rec = gk.gk_blob_size(geom, T)[0]
        sums = got.cpu().numpy().view(np.uint64)
        for p in range(sums.size):
            assert int(sums[p]) == oracle.crc64(host[p * rec:(p + 1) * rec])


@pytest.mark.gpu
def test_noalloc_at_its_page_limit_and_against_the_oracle():
    import oracle
    import paper_2609_39358_b200 as gk
    geom = gk.Geom(1, 1, 64, 16)               # 4 KiB records
    n_tokens = gk.binding.GK_NOALLOC_MAX_PAGES * 16
    nbytes, P = gk.gk_blob_size(geom, n_tokens)
    assert P == gk.binding.GK_NOALLOC_MAX_PAGES
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7)
    blob = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda", generator=gen)
    got = torch.zeros(P, dtype=torch.int64, device="cuda")
    gk.gk_page_checksums_noalloc(geom, blob, n_tokens, got, 0)
    torch.cuda.synchronize()
    host = blob.cpu().numpy()
    sums = got.cpu().numpy().view(np.uint64)
    rec = nbytes // P
    for p in range(P):                          # every page of the 32 MiB blob
        assert int(sums[p]) == oracle.crc64(host[p * rec:(p + 1) * rec])


@pytest.mark.gpu
def test_noalloc_at_its_page_size_limit():
    """256 tokens per page (the largest the fixed table of initial-register terms holds) with a
    partial last page, against the oracle."""
    import oracle
    import paper_2609_39358_b200 as gk
    T = gk.binding.GK_NOALLOC_MAX_PAGE_TOKENS
    geom = gk.Geom(2, 2, 64, T)                # 1 KiB per token, 256 KiB records
    n_tokens = 3 * T + 37
    nbytes, P = gk.gk_blob_size(geom, n_tokens)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(11)
    blob = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda", generator=gen)
    got = torch.zeros(P, dtype=torch.int64, device="cuda")
    gk.gk_page_checksums_noalloc(geom, blob, n_tokens, got, 0)
    torch.cuda.synchronize()
    host = blob.cpu().numpy()
    sums = got.cpu().numpy().view(np.uint64)
    rec = gk.gk_blob_size(geom, T)[0]
    for p in range(P):
        assert int(sums[p]) == oracle.crc64(host[p * rec:min((p + 1) * rec, nbytes)])
