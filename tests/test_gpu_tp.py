"""Tensor-parallel agreement on the GPU: two ranks (two processes on the one GPU, gloo for the
collective -- the ranks' kernels never wait on one another, the agreement is a host-level
all-reduce of n_jobs bytes) restore their own shards; a block damaged on either rank must be
written on neither."""
import os
import socket

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    import oracle
    import paper_2609_39358_b200 as gk
    from paper_2609_39358_b200.tp import tp_restore
    from gpu_harness import dev_cache, dev_i32, gk_geom, sums_to_dev
    from helpers import clone_cache, n_pages, random_cache

    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    og = oracle.Geom(5, 4, 64, 16, 2, 0)                 # this rank's shard: 4 of the model's 8 KV heads
    T = og.page_tokens
    lens = [2 * T + 1, 3 * T, T, 4 * T - 2]
    src = random_cache(og, 11, seed=400 + rank)          # every rank holds different bytes
    rng = np.random.default_rng(410)                     # same tables on all ranks
    Nd = 14
    perm = rng.permutation(Nd).astype(np.int32)
    jobs, used = [], 0
    for n in lens:
        P = n_pages(og, n)
        blob, sums, code, _ = oracle.pack(og, src, rng.integers(0, 11, size=P).astype(np.int32), n)
        assert code == 0
        jobs.append(oracle.Job(blob, sums, perm[used:used + P].copy(), n))
        used += P
    bad_here = 1 if rank == 0 else 3                     # rank 0 sees job 1 damaged, rank 1 sees job 3 damaged
    jobs[bad_here].blob[17] ^= 0x08
    clean = random_cache(og, Nd, seed=420 + rank)
    # expectation: jobs 1 and 3 are written on neither rank
    want = clone_cache(clean)
    agreed_bad = {1, 3}
    oracle.restore(og, want, [jb if j not in agreed_bad else oracle.Job(None, None, jb.page_table, jb.n_tokens)
                              for j, jb in enumerate(jobs)])
    ctx = gk.Context(gk_geom(og), 0)
    d = dev_cache(clean)
    djobs = [gk.Job(torch.from_numpy(jb.blob).cuda(), sums_to_dev(jb.checksums), dev_i32(jb.page_table), jb.n_tokens)
             for jb in jobs]
    mask = torch.full((4,), 255, dtype=torch.uint8, device="cuda")
    fb = torch.full((4,), -7, dtype=torch.int32, device="cuda")
    tp_restore(ctx, djobs, d, mask, fb)
    torch.cuda.synchronize()
    ok = (mask.cpu().tolist() == [0, 1, 0, 1]
          and fb.cpu().tolist()[bad_here] == 0
          and np.array_equal(d.data.cpu().numpy(), want.data)
          and ctx.gk_get_stats()["device_wait_expired"] == 0)
    ctx.close()
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write("ok" if ok else f"mismatch: mask {mask.cpu().tolist()} fb {fb.cpu().tolist()}")
    dist.destroy_process_group()


def test_two_ranks_agree_before_commit(tmp_path):
    import torch.multiprocessing as mp
    assert torch.cuda.is_available()
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        assert open(tmp_path / f"rank{r}.txt").read() == "ok"
