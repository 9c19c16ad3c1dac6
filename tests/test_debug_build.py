"""The bounds-checked build of the library (libgk_debug.so, -DGK_DEBUG).

With compute-sanitizer unavailable, stray accesses of the kernels are looked for
by the kernels themselves: every bulk copy, scale access and checksum access is
compared with the extent of the object it belongs to, a refused access is
skipped and recorded, nothing traps.  The range predicate is unit-tested on the
host; on the GPU the random suite and the small parity suite run once more, in a
child process, against the debug library -- VALID inputs only -- and every
context of that run checks on close that nothing was refused.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gk():
    from paper_2609_39358_b200 import build
    build.build()
    import paper_2609_39358_b200 as m
    return m


def test_range_predicate(gk):
    ok = gk.gk_debug_range_ok
    base, extent = 0x7f00_0000_1000, 4096
    assert ok(base, 4096, base, extent)                      # exact fit
    assert ok(base + 4095, 1, base, extent)
    assert ok(base + 4096, 0, base, extent)                  # empty range at the end
    assert not ok(base + 4096, 1, base, extent)              # one past the end
    assert not ok(base - 1, 1, base, extent)                 # before the start
    assert not ok(base - 16, 32, base, extent)               # straddles the start
    assert not ok(base + 4000, 97, base, extent)             # straddles the end
    assert not ok(base, 4097, base, extent)
    assert not ok(base + 8192, 16, base, extent)
    # sizes near 2^64 must not wrap around into "inside"
    assert not ok(base + 16, 0xFFFF_FFFF_FFFF_FFF0, base, extent)
    assert not ok(0xFFFF_FFFF_FFFF_FFF0, 32, 0xFFFF_FFFF_FFFF_F000, 4096)
    assert ok(0xFFFF_FFFF_FFFF_FFF0, 15, 0xFFFF_FFFF_FFFF_F000, 4095)


def test_debug_library_builds_and_exports_the_same_interface(gk):
    import ctypes
    from paper_2609_39358_b200 import binding, build
    path = build.build(debug=True)
    lib = ctypes.CDLL(path)
    for name in binding.EXPORTS:
        assert hasattr(lib, name), name


@pytest.mark.gpu
def test_parity_suites_under_the_bounds_checked_build(gk):
    """Every context closed during the child run raises if the debug status word is non-zero."""
    from paper_2609_39358_b200 import build
    env = dict(os.environ, GK_LIB_PATH=build.build(debug=True), GK_FUZZ_CASES="48")
    # the sanity check first: the child really runs the debug library and sees a clean status
    probe = ("import torch, paper_2609_39358_b200 as gk\n"
             "ctx = gk.Context(gk.Geom(2, 2, 64, 16), 0)\n"
             "assert ctx.gk_debug_status() == (0, 0, 0, 0), ctx.gk_debug_status()\n"
             "ctx.close(); print('debug library in use')\n")
    out = subprocess.run([sys.executable, "-c", probe], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "debug library in use" in out.stdout, out.stdout + out.stderr
    # the reporting path, without any access outside an object: the cache's extent is UNDERSTATED by one
    # slab, so that the (valid) reads of the last page are refused; the call must still complete, the
    # record must say "cache, loader", and closing the context must raise
    refuse = ("import torch, paper_2609_39358_b200 as gk\n"
              "geom = gk.Geom(2, 2, 64, 16); slab = 16 * 2 * 64 * 2; N = 8\n"
              "ctx = gk.Context(geom, 0); ctx.set_tuning('debug_extent_cut', slab)\n"
              "data = torch.zeros(2 * 2 * N * slab, dtype=torch.uint8, device='cuda')\n"
              "cache = gk.Cache(data, N, 2 * N * slab, N * slab, slab)\n"
              "nb, P = gk.gk_blob_size(geom, 16 * N)\n"
              "blob = torch.zeros(nb, dtype=torch.uint8, device='cuda'); sums = torch.zeros(P, dtype=torch.int64, device='cuda')\n"
              "ctx.gk_pack(cache, torch.arange(N, dtype=torch.int32, device='cuda'), 16 * N, blob, sums)\n"
              "torch.cuda.synchronize()\n"
              "st = ctx.gk_debug_status(); assert st[0] == (0 << 8 | 1) and st[3] > 0, st\n"
              "assert ctx.gk_get_stats()['device_wait_expired'] == 0\n"
              "try:\n    ctx.close()\nexcept gk.GkError as e:\n    assert e.code == -8; print('refused access reported')\n")
    out = subprocess.run([sys.executable, "-c", refuse], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "refused access reported" in out.stdout, out.stdout + out.stderr
    run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                          "tests/test_gpu_fuzz.py", "tests/test_gpu_parity.py", "tests/test_gpu_layerwise.py",
                          "-k", "not plain_c and not bounds_checked"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert run.returncode == 0, run.stdout[-4000:] + run.stderr[-2000:]
    assert " passed" in run.stdout
