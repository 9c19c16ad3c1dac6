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
import numpy as np
import pytest
import torch


def test_too_large_requests_are_rejected_before_any_gpu_work():
    import paper_2609_39358_b200 as gk
    from paper_2609_39358_b200 import build
    build.build()
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
    for n_tokens in (7 * T + 3, 2 * T + 1):
        nbytes, P = gk.gk_blob_size(geom, n_tokens)
        blob = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda", generator=gen)
        want = torch.zeros(P, dtype=torch.int64, device="cuda")
        ctx.gk_page_checksums(blob, n_tokens, want)
        got = torch.full((P,), -1, dtype=torch.int64, device="cuda")
        gk.gk_page_checksums_noalloc(geom, blob, n_tokens, got, 0)
        torch.cuda.synchronize()
        assert torch.equal(got, want)          # integer work: bit-exact
    ctx.close()


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
    for p in (0, 1, P // 2, P - 1):
        assert int(sums[p]) == oracle.crc64(host[p * rec:(p + 1) * rec])
