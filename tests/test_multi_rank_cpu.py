"""The N > 1 launch path on CPU: world_size-2 gloo ranks.  The data path has no
exchange step, so what is covered is what bench.py does across ranks: rendezvous
on 127.0.0.1, barrier, max / sum of per-rank timings, distinct per-rank seeds,
and that the reference arm runs on rank 0 only and prints exactly one line."""
import json
import os
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    sys.path.insert(0, ROOT)
    import bench
    import synth
    comm = bench.RankComm("gloo")
    comm.barrier()
    got = {"max": comm.max(10.0 + rank), "sum": comm.sum(1.0 + rank), "world": comm.world,
           "seed": bench.rank_seed(synth.GQA7B, rank)}
    comm.barrier()
    comm.close()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump(got, f)


def test_rank_comm_over_gloo(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["world"] == 2 and r["max"] == 11.0 and r["sum"] == 3.0
    assert res[0]["seed"] != res[1]["seed"]


class _FakeCtx:
    """Stands in for a gk context on CPU: verify reports this rank's verdicts,
    commit records which jobs it was allowed to write."""

    def __init__(self, verdicts):
        self.verdicts, self.committed = verdicts, None

    def gk_verify(self, jobs, dst, mask, first_bad_page, stream=None):
        mask.copy_(torch.tensor(self.verdicts, dtype=torch.uint8))

    def gk_commit(self, jobs, dst, mask, stream=None):
        self.committed = [i for i, c in enumerate(mask.tolist()) if c == 0]


def _tp_worker(rank, world, port, out_dir):
    os.environ.update({"RANK": str(rank), "WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1",
                       "MASTER_PORT": str(port)})
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2609_39358_b200 import tp
    dist.init_process_group("gloo", rank=rank, world_size=world)
    verdicts = [[0, 1, 0, 0, 3], [0, 0, 0, 2, 0]][rank]     # each rank sees different failures
    ctx = _FakeCtx(verdicts)
    mask = torch.zeros(5, dtype=torch.uint8)
    tp.tp_restore(ctx, [None] * 5, None, mask, torch.zeros(5, dtype=torch.int32))
    dist.destroy_process_group()
    with open(os.path.join(out_dir, f"tp{rank}.json"), "w") as f:
        json.dump({"mask": mask.tolist(), "committed": ctx.committed}, f)


def test_tp_restore_commits_a_block_on_all_ranks_or_none(tmp_path):
    mp.spawn(_tp_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    res = [json.load(open(tmp_path / f"tp{r}.json")) for r in range(2)]
    assert res[0] == res[1] == {"mask": [0, 1, 0, 2, 3], "committed": [0, 2]}


def test_reference_arm_under_torchrun_prints_one_line_on_rank0():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--reference-seconds", "1"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
