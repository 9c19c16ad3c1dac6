#!/usr/bin/env python3
"""Benchmark of the KV block save/restore hot path on B200.

One step = one pass of the whole path over one batch of synthetic input shaped
like the GQA-7B-like serving workload: gk_pack_batch saves the batch's 16 blocks
of 4,096 tokens (32 layers, 8 KV heads, head_dim 128, bf16, 16-token pages) from
a paged source cache into their slots of a 64-block device-resident pool, then
gk_restore validates the page tables, verifies every page record (CRC-64/XZ),
and scatters the 16 blocks (8 requests x 2 blocks) into a 16,384-page destination
cache through seeded random-permutation page tables.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line on rank 0.  `value` is the metric itself: restored KV GB/s,
counting the bytes the restore phase of a step must read plus the bytes it must
write (2 x blob bytes), over the device time of that phase, summed over all
GPUs; the save phase, the whole step, tokens/s, the per-kernel roofline (against
the measured copy peak and against the nominal 8,000 GB/s), the other workload
shapes, lone-block latencies, the host-tier end-to-end leg and the CPU oracle's
timings are reported beside it.  With N > 1 (launched by torch.distributed.run)
every rank runs its own batch on its own GPU: the path has no exchange step, so
this is weak scaling over independent request batches.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "restored KV GB/s (read+write)"
UNIT = "GB/s"

# DRAM bytes per blob byte of one launch of the fused restore kernel: ncu's
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the full-size
# (16-block) workload, a one-pass capture summarised under profiles/
# (17.18 GB read + 8.56 GB written for 8.59 GB of blobs); the full --set full
# capture of a 2-block launch gives 2.96.
RESTORE_DRAM_BYTES_PER_BLOB_BYTE = 25.74 / 8.59
NOMINAL_HBM_GBS = 8000.0   # the HBM peak the target is stated against


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="gqa7b", choices=["gqa7b", "tiny", "corpus", "fp8", "stress", "longwindow", "digest", "layerwise",
                                                            "latency", "records", "layerwise-device"],
                    help="gqa7b is the headline workload (full JSON line); the others print a shorter line "
                         "with the save and restore phases of that workload's shape")
    ap.add_argument("--window-blocks", type=int, default=48,
                    help="longwindow: blocks streamed per step (30,000 tokens each, through a 2-block ring)")
    ap.add_argument("--single-pass", action="store_true",
                    help="restore with GK_FLAG_SINGLE_PASS (one pass over the blob; pages of a block that fails "
                         "its checksum receive the unverified bytes); prints the short line, never the headline")
    ap.add_argument("--blocks", type=int, default=0,
                    help="restore this many blocks instead of the workload's 16 (small cases for profiling)")
    ap.add_argument("--unfused", action="store_true",
                    help="restore with a verify launch, a compare launch and a commit launch instead of the fused "
                         "kernel (the kernels gk_verify and gk_commit run; for profiling)")
    ap.add_argument("--tokens", type=int, default=0,
                    help="latency: restore one block of this many tokens (default: 256, 1,024, 5,200 and 24,018)")
    ap.add_argument("--layers", type=int, default=1,
                    help="records: layers per page record of the gqa7b geometry (64 KiB per layer), 8 GiB of blobs; "
                         "layerwise-device: layers per group (not given: groups of 32, 8, 4, 2 and 1 layers in turn)")
    ap.add_argument("--tune", default="", help="tuning keys for the context of the run, key=value[,key=value...]")
    ap.add_argument("--e2e-steps", type=int, default=3, help="steps of the one-step-at-a-time end-to-end leg")
    ap.add_argument("--e2e-pipelined-steps", type=int, default=10,
                    help="steps of the pipelined end-to-end leg (save of step k+1 overlaps restore of step k)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the other workload shapes and the latency cases")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-baseline-blocks", type=int, default=4)
    ap.add_argument("--reference-seconds", type=float, default=100.0,
                    help="--impl reference: target wall time of all steps together (sizes the sample)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ---------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.path = None
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            fd, self.path = tempfile.mkstemp(prefix="gk_clocks_", suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def wait_first_sample(self, limit_s: float = 8.0):
        if self.proc is None:
            return
        t0 = time.time()
        while time.time() - t0 < limit_s:
            try:
                if os.path.getsize(self.path) > 0:
                    return
            except OSError:
                return
            time.sleep(0.05)

    def stop(self):
        if self.proc is None:
            return None
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        self.out.close()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 7:
                        continue
                    try:
                        sm.append(float(parts[0]))
                        smax.append(float(parts[1]))
                    except ValueError:
                        continue
                    for name, val in zip(names, parts[3:7]):
                        if val.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            return None
        if not sm:
            return None
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------
# ranks: one process per GPU, no data-path collective
# ---------------------------------------------------------------------------
class RankComm:
    """Rendezvous, barrier and reductions of scalars over the ranks of a
    torch.distributed.run launch (env: RANK, LOCAL_RANK, WORLD_SIZE, MASTER_*).
    The data path itself never communicates; this is only for timing."""

    def __init__(self, backend: str, device=None):
        import torch
        import torch.distributed as dist
        self.torch, self.dist = torch, dist
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        # GK_FORCE_DIST=1 brings the process group up even for one rank (to try the NCCL path on one GPU)
        self.active = self.world > 1 or os.environ.get("GK_FORCE_DIST") == "1"
        if self.active:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29511")
            kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
            dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kw)

    def barrier(self):
        if self.active:
            self.dist.barrier()
        if self.device is not None:
            self.torch.cuda.synchronize(self.device)

    def _reduce(self, x: float, op) -> float:
        if not self.active:
            return float(x)
        t = self.torch.tensor([x], dtype=self.torch.float64,
                              device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=op)
        return float(t.item())

    def max(self, x: float) -> float:
        return self._reduce(x, self.dist.ReduceOp.MAX)

    def sum(self, x: float) -> float:
        return self._reduce(x, self.dist.ReduceOp.SUM)

    def close(self):
        if self.active:
            self.dist.destroy_process_group()


def rank_seed(workload, rank: int) -> int:
    """Every rank works on its own seeded batch (weak scaling over independent batches)."""
    return workload.seed(100 * rank)


# ---------------------------------------------------------------------------
# workload
# ---------------------------------------------------------------------------
def build_workload(args, device, rank):
    import torch
    import synth
    import paper_2609_39358_b200 as gk

    w = synth.GQA7B
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
    n_tok = synth.GQA7B_BLOCK_TOKENS
    blob_bytes, P = gk.gk_blob_size(geom, n_tok)
    if args.blocks:
        n_blocks = args.blocks
        pool_blocks = n_blocks
        dst_pages = max(2 * n_blocks * P, 512)
    else:
        n_blocks = synth.GQA7B_REQUESTS * synth.GQA7B_BLOCKS_PER_REQUEST
        pool_blocks = synth.GQA7B_POOL_BLOCKS
        dst_pages = synth.GQA7B_DST_PAGES
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    src_pages = n_blocks * P

    def cache(num_pages, data):
        return gk.Cache(data, num_pages, 2 * num_pages * slab, num_pages * slab, slab)

    seed0 = rank_seed(w, rank)
    rng = np.random.default_rng(seed0)
    pool = [torch.empty(blob_bytes, dtype=torch.uint8, device=device) for _ in range(pool_blocks)]
    sums = [torch.zeros(P, dtype=torch.int64, device=device) for _ in range(pool_blocks)]
    ctx = gk.Context(geom, device.index)
    src_perm = torch.from_numpy(synth.page_permutation(src_pages, seed0 + 1)).to(device)
    chosen = np.sort(rng.choice(pool_blocks, size=n_blocks, replace=False))

    # fill the pool: the source cache is refilled for every group of n_blocks blocks;
    # the last fill holds the blocks the timed steps save and restore
    groups = [list(range(g, min(g + n_blocks, pool_blocks))) for g in range(0, pool_blocks, n_blocks)]
    src = None
    for gi, group in enumerate(groups + [list(chosen)]):
        data = synth.kv_bytes_bf16(2 * w.layers * src_pages * slab // 2, w.sigma, seed0 + 10 + gi, device)
        src = cache(src_pages, data)
        jobs = [gk.Job(pool[b], sums[b], src_perm[i * P:(i + 1) * P].contiguous(), n_tok)
                for i, b in enumerate(group)]
        ctx.gk_pack_batch(src, jobs)
        torch.cuda.synchronize(device)
        if gi < len(groups):
            del data, src
    dst_data = synth.sentinel_bytes(2 * w.layers * dst_pages * slab, seed0 + 2, device)
    dst = cache(dst_pages, dst_data)
    dst_perm = torch.from_numpy(synth.page_permutation(dst_pages, seed0 + 3)).to(device)
    pack_jobs, restore_jobs = [], []
    for i, b in enumerate(chosen):
        pack_jobs.append(gk.Job(pool[b], sums[b], src_perm[i * P:(i + 1) * P].contiguous(), n_tok, i // 2))
        restore_jobs.append(gk.Job(pool[b], sums[b], dst_perm[i * P:(i + 1) * P].contiguous(), n_tok, i // 2))
    pack_jobs, restore_jobs = gk.JobArray(pack_jobs), gk.JobArray(restore_jobs)   # marshalled once
    return dict(gk=gk, ctx=ctx, geom=geom, w=w, n_tok=n_tok, blob_bytes=blob_bytes, P=P, n_blocks=n_blocks,
                pool_blocks=pool_blocks, dst_pages=dst_pages, src=src, dst=dst, pack_jobs=pack_jobs,
                restore_jobs=restore_jobs, chosen=chosen, src_perm=src_perm, dst_perm=dst_perm, slab=slab,
                src_pages=src_pages)


def oracle_sample(wl, n_blocks):
    """Times the CPU oracle, as it stands, on blocks of the batch: pack from a host copy of
    the source cache, then restore into a host destination cache.  Two legs: one thread over
    the first n_blocks blocks, and one thread per block over as many blocks as the box has
    cores (at most the batch), every thread calling the unchanged oracle through ctypes on its
    own block and its own destination pages.  Returns the times (whole and restore phase
    alone) of both legs and the oracle's checksums of the sampled blocks."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    w = wl["w"]
    og = oracle.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, w.elem_bytes, 0)
    P, n_tok, slab = wl["P"], wl["n_tok"], wl["slab"]
    src_pages = wl["src_pages"]
    src_host = wl["src"].data.cpu().numpy()
    src = oracle.Cache(src_host, src_pages, 2 * src_pages * slab, src_pages * slab, slab)
    src_perm = wl["src_perm"].cpu().numpy()

    def one_block(i, dst, dperm, slot):
        t_begin = time.perf_counter()
        blob, sums, code, _ = oracle.pack(og, src, src_perm[i * P:(i + 1) * P], n_tok)
        assert code == 0
        t = time.perf_counter()
        mask, _ = oracle.restore(og, dst, [oracle.Job(blob, sums, dperm[slot * P:(slot + 1) * P], n_tok)])
        assert not mask.any()
        t_end = time.perf_counter()
        return sums, t_end - t, t_end - t_begin

    def dst_for(blocks):
        dpages = blocks * P
        return (oracle.Cache(np.zeros(2 * w.layers * dpages * slab, dtype=np.uint8), dpages, 2 * dpages * slab,
                             dpages * slab, slab),
                np.random.default_rng(7).permutation(dpages).astype(np.int32))

    dst, dperm = dst_for(n_blocks)
    t0 = time.perf_counter()
    res = [one_block(i, dst, dperm, i) for i in range(n_blocks)]
    t_single = time.perf_counter() - t0
    sums_out = [r[0] for r in res]
    t_single_restore = sum(r[1] for r in res)
    del dst
    threads = max(1, min(os.cpu_count() or 1, wl["n_blocks"]))
    dst, dperm = dst_for(threads)
    with ThreadPoolExecutor(max_workers=threads) as pool:
        t0 = time.perf_counter()
        res = list(pool.map(lambda i: one_block(i, dst, dperm, i), range(threads)))
        t_multi = time.perf_counter() - t0
    # the threads' restore phases overlap one another's save phases: the restore's share of the wall time
    t_multi_restore = t_multi * sum(r[1] for r in res) / max(sum(r[2] for r in res), 1e-9)
    return dict(t_single=t_single, t_single_restore=t_single_restore, t_multi=t_multi, t_multi_restore=t_multi_restore,
                threads=threads, blob_bytes=wl["blob_bytes"], n_tok=n_tok, sums=sums_out)


# ---------------------------------------------------------------------------
# reference arm: the oracle on the host cores
# ---------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    import synth
    w = synth.GQA7B
    og = oracle.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, w.elem_bytes, 0)
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    # size the sample so that the whole run stays within about two minutes
    probe_pages = 8
    rng = np.random.default_rng(w.seed(900))
    n_iter = max(1, args.steps + args.warmup)
    per_page = None
    pages = probe_pages
    for _ in range(2):
        N = pages
        data = rng.integers(0, 256, size=2 * w.layers * N * slab, dtype=np.uint8)
        src = oracle.Cache(data, N, 2 * N * slab, N * slab, slab)
        dst = oracle.Cache(np.zeros_like(data), N, 2 * N * slab, N * slab, slab)
        spt = rng.permutation(N).astype(np.int32)
        dpt = rng.permutation(N).astype(np.int32)
        n_tok = N * w.page_tokens
        if per_page is None:
            t0 = time.perf_counter()
            blob, sums, _, _ = oracle.pack(og, src, spt, n_tok)
            oracle.restore(og, dst, [oracle.Job(blob, sums, dpt, n_tok)])
            per_page = (time.perf_counter() - t0) / N
            pages = int(min(1024, max(8, args.reference_seconds / (per_page * n_iter))))
    times, rtimes = [], []
    blob_bytes = oracle.blob_size(og, n_tok)[0]
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        blob, sums, code, _ = oracle.pack(og, src, spt, n_tok)
        t1 = time.perf_counter()
        mask, _ = oracle.restore(og, dst, [oracle.Job(blob, sums, dpt, n_tok)])
        t2 = time.perf_counter()
        assert code == 0 and not mask.any()
        if it >= args.warmup:
            times.append(t2 - t0)
            rtimes.append(t2 - t1)
    t, tr = float(np.mean(times)), float(np.median(rtimes))
    value = 2 * blob_bytes / tr / 1e9       # the metric: restored bytes read + written over the restore phase
    hi = host_info()
    sample = (f"one block of {n_tok} tokens ({pages} pages, {blob_bytes / 2**20:.0f} MiB blob) saved and restored per "
              f"step by the CPU oracle, one thread ({hi['cpu_model']}, {hi['nproc']} cores in the box)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": "gqa7b (32 layers, 8 KV heads, head_dim 128, bf16, 16-token pages), bounded sample",
                       "sample": sample,
                       "value_definition": "restored KV bytes read + written (2 x blob bytes) / time of the restore "
                                           "phase of a step (median over the timed steps)"},
            "tokens_per_s": n_tok / tr,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                             "nproc": hi["nproc"], "cpu_model": hi["cpu_model"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------
def run_ours(args):
    import torch

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgk has no CPU fallback")
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    comm = RankComm("nccl", device)
    world, rank = comm.world, comm.rank
    barrier, max_over_ranks = comm.barrier, comm.max

    wl = build_workload(args, device, rank)
    gk, ctx = wl["gk"], wl["ctx"]
    n_blocks, blob_bytes, n_tok = wl["n_blocks"], wl["blob_bytes"], wl["n_tok"]
    batch_bytes = n_blocks * blob_bytes
    mask = torch.zeros(n_blocks, dtype=torch.uint8, device=device)
    first_bad = torch.zeros(n_blocks, dtype=torch.int32, device=device)
    status = torch.zeros(n_blocks, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device)

    def step(events=None):
        if events:
            events[0].record(stream)
        ctx.gk_pack_batch(wl["src"], wl["pack_jobs"], status)
        if events:
            events[1].record(stream)
        ctx.gk_restore(wl["restore_jobs"], wl["dst"], mask, first_bad)
        if events:
            events[2].record(stream)

    if args.unfused:
        ctx.set_tuning("fused", 0)
    for kv in filter(None, args.tune.split(",")):
        key, val = kv.split("=")
        ctx.set_tuning(key, int(val))
    # warm-up: the per-kernel timing events are created here, not in the timed region
    ctx.set_tuning("profile", 1)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize(device)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.wait_first_sample()   # nvidia-smi start-up would otherwise stall CUDA calls of step 0
    step()
    torch.cuda.synchronize(device)
    ctx.gk_get_kernel_times()
    launches0 = ctx.gk_get_stats()["kernels_launched"]
    phase_events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin.record(stream)
    for k in range(args.steps):
        step(phase_events[k])
    t_end.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    step_ms = max_over_ranks(t_begin.elapsed_time(t_end) / max(args.steps, 1))
    kt = ctx.gk_get_kernel_times()
    ctx.set_tuning("profile", 0)
    stats = ctx.gk_get_stats()
    launches = stats["kernels_launched"] - launches0
    assert int(mask.sum().item()) == 0 and int(status.sum().item()) == 0, "a clean block was rejected"
    assert stats["device_wait_expired"] == 0
    pack_all = [e[0].elapsed_time(e[1]) for e in phase_events]
    restore_all = [e[1].elapsed_time(e[2]) for e in phase_events]
    pack_ms, restore_ms = float(np.median(pack_all)), float(np.median(restore_all))
    # the slowest rank's restore phase decides the job's rate (weak scaling over independent batches)
    restore_ms_job = max_over_ranks(restore_ms)

    value = world * 2 * batch_bytes / (restore_ms_job * 1e-3) / 1e9
    peak, peak_kind = measured_peak()

    def kernel_entry(name, alg_bytes_per_launch):
        ms, n = kt[name]
        if n == 0:
            return None
        per = ms / n
        ach = alg_bytes_per_launch / (per * 1e-3) / 1e9
        return {"launches": n, "ms_per_launch": per, "algorithmic_bytes_per_launch": alg_bytes_per_launch,
                "achieved": ach, "unit": "GB/s", "frac": ach / peak, "frac_of_nominal_8000": ach / NOMINAL_HBM_GBS}

    # algorithmic bytes: the fused restore kernel reads every blob byte twice (verify, then
    # commit -- a block may be written only after all of it has verified, and blocks are larger
    # than L2) and writes it once; pack reads and writes every byte once
    kernels = {"restore": kernel_entry("restore", 3 * batch_bytes),
               "pack": kernel_entry("pack", 2 * batch_bytes),
               "verify": kernel_entry("verify", batch_bytes),
               "commit": kernel_entry("commit", 2 * batch_bytes)}
    kernels = {k: v for k, v in kernels.items() if v is not None}
    if "restore" in kernels:
        dom = kernels["restore"]
        roofline = {"bound": "hbm", "kernel": "restore_kernel (fused verify + commit: blob -> CRC check -> paged cache)",
                    "achieved": dom["achieved"], "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                    "frac": dom["frac"], "frac_of_nominal_8000": dom["achieved"] / NOMINAL_HBM_GBS,
                    "traffic": RESTORE_DRAM_BYTES_PER_BLOB_BYTE * batch_bytes,
                    "traffic_note": "ncu dram read+write per blob byte of a launch of this workload (one-pass capture), "
                                    "times the blob bytes of the launch",
                    "algorithmic_bytes_per_launch": 3 * batch_bytes, "ms_per_launch": dom["ms_per_launch"],
                    "achieved_useful_2x": 2 * batch_bytes / (dom["ms_per_launch"] * 1e-3) / 1e9}
    else:
        # a lone job of 256 MiB or more is restored by the two dedicated kernels (it cannot overlap its
        # own verify and commit); the commit kernel moves the most bytes
        dom = kernels["commit"]
        roofline = {"bound": "hbm", "kernel": "stream_kernel<kCommit> (blob -> paged cache), after stream_kernel<kVerify>",
                    "achieved": dom["achieved"], "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                    "frac": dom["frac"], "frac_of_nominal_8000": dom["achieved"] / NOMINAL_HBM_GBS, "traffic": None,
                    "algorithmic_bytes_per_launch": 2 * batch_bytes, "ms_per_launch": dom["ms_per_launch"]}

    # ---- end to end: the same step with HOST buffers -- gk_pack_host saves the batch into pinned
    # host memory (D2H inside), gk_restore_host restores it from there (H2D inside), and the
    # result masks are read back ----
    e2e = None
    if not args.no_e2e:
        host_pack, host_restore, keep = [], [], []
        for pj, rj in zip(wl["pack_jobs"], wl["restore_jobs"]):
            hb = torch.empty(blob_bytes, dtype=torch.uint8, pin_memory=True)
            hs = torch.empty(wl["P"], dtype=torch.int64, pin_memory=True)
            keep.append((hb, hs))
            host_pack.append(gk.Job(hb, hs, pj.page_table, n_tok, pj.request_id))
            host_restore.append(gk.Job(hb, hs, rj.page_table, n_tok, rj.request_id))
        mask_h = torch.empty(n_blocks, dtype=torch.uint8, pin_memory=True)
        fb_h = torch.empty(n_blocks, dtype=torch.int32, pin_memory=True)
        status_h = torch.empty(n_blocks, dtype=torch.uint8, pin_memory=True)
        torch.cuda.synchronize(device)
        e2e_events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.e2e_steps)]

        def e2e_step(ev=None):
            if ev:
                ev[0].record(stream)
            ctx.gk_pack_host(wl["src"], host_pack, status)
            status_h.copy_(status, non_blocking=True)
            if ev:
                ev[1].record(stream)
            ctx.gk_restore_host(host_restore, wl["dst"], mask, first_bad)
            mask_h.copy_(mask, non_blocking=True)
            fb_h.copy_(first_bad, non_blocking=True)
            if ev:
                ev[2].record(stream)

        # the link's own rate on this machine: plain pinned copies of one blob each way, for the host-tier roofline
        tmp = torch.empty(blob_bytes, dtype=torch.uint8, device=device)
        link_rate = {}
        for name, (d, s_) in {"h2d": (tmp, keep[0][0]), "d2h": (keep[0][0], tmp)}.items():
            d.copy_(s_, non_blocking=True)
            torch.cuda.synchronize(device)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            for _ in range(3):
                d.copy_(s_, non_blocking=True)
            c1.record(stream)
            torch.cuda.synchronize(device)
            link_rate[name] = 3 * blob_bytes / (c0.elapsed_time(c1) * 1e-3) / 1e9
        # both directions at once (two streams): the ceiling of the pipelined save + restore below
        if len(keep) >= 2:
            tmp2 = torch.empty(blob_bytes, dtype=torch.uint8, device=device)
            s_a, s_b = torch.cuda.Stream(device), torch.cuda.Stream(device)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(device)
            c0.record(stream)
            s_a.wait_event(c0)
            s_b.wait_event(c0)
            for _ in range(3):
                with torch.cuda.stream(s_a):
                    tmp.copy_(keep[0][0], non_blocking=True)       # host -> device
                with torch.cuda.stream(s_b):
                    keep[1][0].copy_(tmp2, non_blocking=True)      # device -> host (the step below packs it afresh)
            stream.wait_stream(s_a)
            stream.wait_stream(s_b)
            c1.record(stream)
            torch.cuda.synchronize(device)
            link_rate["each_direction_when_both_run"] = 3 * blob_bytes / (c0.elapsed_time(c1) * 1e-3) / 1e9
            del tmp2
        del tmp
        e2e_step()
        torch.cuda.synchronize(device)
        for i in range(min(4, n_blocks)):      # what went over the link is what the device pool holds
            assert torch.equal(keep[i][1], wl["pack_jobs"][i].checksums.cpu())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for k in range(args.e2e_steps):
            e2e_step(e2e_events[k])
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / max(args.e2e_steps, 1))
        assert int(mask_h.sum().item()) == 0 and int(status_h.sum().item()) == 0
        save_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in e2e_events]))
        load_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in e2e_events]))
        link = batch_bytes + n_blocks * wl["P"] * 8

        # ---- the same steps pipelined: a second context restores step k on its own stream while the
        # first saves step k+1 (two sets of pinned buffers), so that both directions of the host link
        # are busy at once.  Every step still copies its whole batch out and in and reads its results.
        keep2, host_pack2, host_restore2 = [], [], []
        # the second buffer set needs batch_bytes more pinned memory on every rank of this host
        try:
            import psutil
            room = psutil.virtual_memory().available > 1.5 * world * batch_bytes
        except Exception:
            room = True
        try:
            for pj, rj in zip(wl["pack_jobs"], wl["restore_jobs"]):
                if not room:
                    break
                hb = torch.empty(blob_bytes, dtype=torch.uint8, pin_memory=True)
                hs = torch.empty(wl["P"], dtype=torch.int64, pin_memory=True)
                keep2.append((hb, hs))
                host_pack2.append(gk.Job(hb, hs, pj.page_table, n_tok, pj.request_id))
                host_restore2.append(gk.Job(hb, hs, rj.page_table, n_tok, rj.request_id))
        except RuntimeError:
            room = False
            keep2, host_pack2, host_restore2 = [], [], []
        room = bool(comm.max(0.0 if room else 1.0) == 0.0)      # all ranks or none
        sets = [(host_pack, host_restore), (host_pack2, host_restore2)]
        ctx_r = gk.Context(wl["geom"], device.index)
        s_save, s_rest = torch.cuda.Stream(device), torch.cuda.Stream(device)
        status2 = torch.zeros_like(status)

        def pipelined(n_steps):
            saved = [torch.cuda.Event() for _ in range(n_steps)]
            restored = [torch.cuda.Event() for _ in range(n_steps)]
            b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            b0.record(stream)
            s_save.wait_event(b0)
            s_rest.wait_event(b0)
            for k in range(n_steps):
                hp, hr = sets[k % 2]
                with torch.cuda.stream(s_save):
                    if k >= 2:
                        s_save.wait_event(restored[k - 2])      # this buffer set has been read back in
                    ctx.gk_pack_host(wl["src"], hp, status2, stream=s_save)
                    status_h.copy_(status2, non_blocking=True)
                    saved[k].record(s_save)
                with torch.cuda.stream(s_rest):
                    s_rest.wait_event(saved[k])
                    ctx_r.gk_restore_host(hr, wl["dst"], mask, first_bad, stream=s_rest)
                    mask_h.copy_(mask, non_blocking=True)
                    fb_h.copy_(first_bad, non_blocking=True)
                    restored[k].record(s_rest)
            stream.wait_stream(s_save)
            stream.wait_stream(s_rest)
            b1.record(stream)
            return b0, b1

        if room:
            pipelined(2)
            torch.cuda.synchronize(device)
            barrier()
            b0, b1 = pipelined(args.e2e_pipelined_steps)
            barrier()
            pipe_ms = max_over_ranks(b0.elapsed_time(b1) / max(args.e2e_pipelined_steps, 1))
            pipe_steps = args.e2e_pipelined_steps
            pipe_note = ("save of step k+1 (context 1, stream 1) overlaps restore of step k (context 2, stream 2); "
                         "two sets of pinned buffers; both directions of the host link in use at once")
            assert int(mask_h.sum().item()) == 0 and int(status_h.sum().item()) == 0
            for i in range(min(4, n_blocks)):
                assert torch.equal(keep2[i][1], wl["pack_jobs"][i].checksums.cpu())
            assert ctx_r.gk_get_stats()["device_wait_expired"] == 0
        else:
            pipe_ms, pipe_steps = e2e_ms, args.e2e_steps
            pipe_note = "not pipelined: no room for a second set of pinned buffers on this host"
        ctx_r.close()
        del keep2, host_pack2, host_restore2, sets
        e2e = {"value": world * 4 * batch_bytes / (pipe_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": link + 2 * n_blocks * 40, "d2h_bytes_per_step": link + n_blocks * 6,
               "ms_per_step": pipe_ms, "steps": pipe_steps,
               "link_gbs": {"each_direction": link / (pipe_ms * 1e-3) / 1e9,
                            "note": "bytes that cross the host link per step in one direction / step time; value "
                                    "counts 2 x blob bytes for the save and 2 x for the restore (read + write), "
                                    "the link itself carries 1 x out and 1 x in"},
               "tokens_per_s": world * n_blocks * n_tok / (pipe_ms * 1e-3),
               "pipelining": pipe_note,
               "one_step_at_a_time": {"value": world * 4 * batch_bytes / (e2e_ms * 1e-3) / 1e9,
                                      "ms_per_step": e2e_ms, "steps": args.e2e_steps},
               "save": {"ms": save_ms, "host_link_gbs": link / (save_ms * 1e-3) / 1e9,
                        "frac_of_plain_d2h_copy": link / (save_ms * 1e-3) / 1e9 / link_rate["d2h"]},
               "restore": {"ms": load_ms, "host_link_gbs": link / (load_ms * 1e-3) / 1e9,
                           "frac_of_plain_h2d_copy": link / (load_ms * 1e-3) / 1e9 / link_rate["h2d"],
                           "tokens_per_s": n_blocks * n_tok / (load_ms * 1e-3)},
               "plain_pinned_copy_gbs": link_rate,
               "what": "gk_pack_host (save to pinned host) + gk_restore_host (restore from pinned host) + D2H read "
                       "of status, mask and first_bad_page; value counts 2 x blob bytes for each"}
        del keep, host_pack, host_restore

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        nb = min(args.cpu_baseline_blocks, n_blocks)
        o = oracle_sample(wl, nb)
        for i in range(nb):   # the pool blobs the GPU packed carry the same checksums
            got = wl["pack_jobs"][i].checksums.cpu().numpy().view(np.uint64)
            assert np.array_equal(got, o["sums"][i]), "GPU checksums differ from the oracle's"
        hi = host_info()
        bb, nt, th = o["blob_bytes"], o["n_tok"], o["threads"]
        cpu_baseline = {"value": 2 * nb * bb / o["t_single_restore"] / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": f"restore phase of save + restore of the first {nb} blocks of the batch ({nb * nt} "
                                  f"tokens, {nb * bb / 2**30:.1f} GiB of blobs) by one thread: {o['t_single_restore']:.1f} s "
                                  f"of {o['t_single']:.1f} s; value = 2 x blob bytes / restore time, as the headline",
                        "tokens_per_s": nb * nt / o["t_single_restore"],
                        "save_plus_restore_gbs": 4 * nb * bb / o["t_single"] / 1e9,
                        "threaded": {"value": 2 * th * bb / o["t_multi_restore"] / 1e9, "unit": UNIT, "cores": th,
                                     "sample": f"one thread per block over {th} blocks at once, {o['t_multi']:.1f} s for "
                                               f"save + restore; restore share {o['t_multi_restore']:.1f} s",
                                     "save_plus_restore_gbs": 4 * th * bb / o["t_multi"] / 1e9,
                                     "tokens_per_s": th * nt / o["t_multi_restore"]},
                        "nproc": hi["nproc"], "cpu_model": hi["cpu_model"]}

    # ---- the integer side: measured rate of three-input logic operations, and what it allows the checksum
    alu = None
    if rank == 0:
        rate = ctx.gk_measure_logic_rate()
        mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
        sms = torch.cuda.get_device_properties(device).multi_processor_count
        instr_per_byte = 3.05    # integer-pipe instructions per blob byte of the verify kernel (ncu, profiles/)
        alu = {"logic_lane_ops_per_s": rate, "lanes_per_clock_per_sm": rate / (sms * mhz * 1e6),
               "how": "one kernel of independent lop3 chains, 8 CTAs x 256 threads per SM, CUDA events, best of 3",
               "verify_alone_bound_gbs": rate / instr_per_byte / 1e9,
               "note": f"the checksum costs {instr_per_byte} integer-pipe instructions per byte, so verification "
                       "alone cannot stream faster than this; in the fused restore kernel it hides under the DRAM time"}

    # ---- the other workload shapes and the lone-block latencies (one GPU, after the headline's memory is free)
    workloads, latency = None, None
    if world == 1 and not args.no_workloads and not args.blocks:
        wl_keep = {k: wl[k] for k in ("n_blocks", "n_tok", "pool_blocks", "dst_pages")}
        ctx.close()
        wl.clear()
        import gc
        gc.collect()
        torch.cuda.empty_cache()
        wl.update(wl_keep)
        workloads = {}
        for name in ("tiny", "corpus", "corpus_host", "fp8", "stress_wave", "stress_wave_one_third_damaged"):
            workloads[name] = workload_case(name, device, steps=5, warmup=2)
        # small page records (the gqa7b geometry with one and two layers per record, 8 GiB of blobs)
        for layers in (1, 2):
            workloads[f"records_{64 * layers}_kib"] = workload_case("gqa7b", device, steps=5, warmup=2, layers=layers)
        latency = latency_cases(device)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {
                "workload": ("gqa7b: 32 layers, 8 KV heads, head_dim 128, bf16 N(0,0.5), 16-token pages; "
                             f"{n_blocks} blocks of {wl['n_tok']} tokens per step per GPU "
                             f"({synth_requests(n_blocks)}), pool of {wl['pool_blocks']} blocks, "
                             f"{wl['dst_pages']}-page destination cache, seeded random-permutation page tables"),
                "step": "gk_pack_batch (save) + gk_restore (validate, verify, commit) of the batch",
                "value_definition": "restored KV bytes read + written (2 x blob bytes of the batch) / device time of "
                                    "the restore phase of a step (median over the timed steps, slowest GPU), all GPUs",
                "batch_blob_bytes": batch_bytes, "l2": "inputs larger than L2 (8 GiB per phase vs 126 MB)",
                "parallelism": f"replicas x{world}, no collective"},
            "tokens_per_s": world * n_blocks * n_tok / (restore_ms_job * 1e-3),
            "north_star": {
                "what": "device-resident restore against the HBM peak, bytes read plus bytes written",
                "restore_useful_2_bytes_per_byte": fractions(2 * batch_bytes / (restore_ms * 1e-3) / 1e9, peak),
                "restore_dram_model_3_bytes_per_byte": fractions(3 * batch_bytes / (restore_ms * 1e-3) / 1e9, peak),
                "note": "a block is written only after all of it has verified and blocks exceed L2, so every blob "
                        "byte crosses DRAM three times (read to verify, read to commit, written): the DRAM-model "
                        "rate is the memory system's, the useful rate is two thirds of it"},
            "phases": {
                "save": dict(stats_ms(pack_all), **fractions(2 * batch_bytes / (pack_ms * 1e-3) / 1e9, peak)),
                "restore": dict(stats_ms(restore_all), tokens_per_s=n_blocks * wl["n_tok"] / (restore_ms * 1e-3)),
                "whole_step": {"ms_per_step": step_ms,
                               "gbs_save_plus_restore": world * 4 * batch_bytes / (step_ms * 1e-3) / 1e9}},
            "roofline": roofline, "kernels": kernels, "alu": alu, "workloads": workloads, "latency": latency,
            "cpu_baseline": cpu_baseline, "e2e": e2e,
            "gpu_launches": launches, "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    comm.close()


# ---------------------------------------------------------------------------
# the other workload shapes: save and restore phases, with the damage the
# configuration prescribes, and the mask census
# ---------------------------------------------------------------------------
def host_info():
    """Cores and CPU model of the box (for the CPU baseline record)."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count() or 1, "cpu_model": model}


def fractions(gbs, peak):
    return {"gbs": gbs, "frac_of_measured_peak": gbs / peak, "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS}


def stats_ms(xs):
    xs = [float(x) for x in xs]
    return {"median": float(np.median(xs)), "best": float(np.min(xs)), "mean": float(np.mean(xs)), "n": len(xs)}


def shape_of(synth, name, blocks=0):
    """(workload, block lengths, destination pages, block ids or None) of a named case."""
    if name in ("stress_wave", "stress_wave_one_third_damaged", "stress"):
        w = synth.STRESS
        # one wave of the stress mix: the blocks of the first requests that fit a 65,536-page cache
        all_len = synth.stress_block_lengths(w.seed(0))
        lens, ids, dst_pages, used = [], [], 65536, 0
        for req in synth.stress_requests(w.seed(1)):
            need = sum(-(-int(all_len[b]) // w.page_tokens) for b in req)
            if used + need > dst_pages:
                break
            lens += [int(all_len[b]) for b in req]
            ids += [int(b) for b in req]
            used += need
            if blocks and len(lens) >= blocks:   # a shorter wave (small cases for profiling)
                break
        return w, lens, dst_pages, ids
    w = synth.WORKLOADS[name.replace("_host", "")]
    if name == "gqa7b":
        return w, [synth.GQA7B_BLOCK_TOKENS] * (blocks or synth.GQA7B_REQUESTS * synth.GQA7B_BLOCKS_PER_REQUEST), synth.GQA7B_DST_PAGES, None
    if name == "tiny":
        return w, synth.TINY_BLOCKS, synth.TINY_DST_PAGES, None
    if name in ("corpus", "corpus_host"):
        return w, synth.CORPUS_BLOCKS, synth.CORPUS_DST_PAGES, None
    if name == "fp8":
        return w, synth.FP8_BLOCKS, sum(-(-n // w.page_tokens) for n in synth.FP8_BLOCKS) + 100, None
    raise ValueError(name)


def workload_case(name, device, steps=5, warmup=2, single_pass=False, blocks=0, layers=0, tune=""):
    """Save and restore phases of one workload shape, each timed on its own over `steps`
    calls (the damage the configuration prescribes is applied between the two, so the
    restore is timed with it in place).  Returns a record for the bench line."""
    import torch
    import synth
    import paper_2609_39358_b200 as gk

    w, lens, dst_pages, ids = shape_of(synth, name, blocks)
    if layers:
        # small page records: the gqa7b geometry with fewer layers per record, 8 GiB of blobs as in the headline
        import dataclasses
        w = dataclasses.replace(w, layers=layers)
        lens = [4096 * max(32 // layers, 1)] * (blocks or 16)
        dst_pages = sum(-(-n // w.page_tokens) for n in lens)
    host_tier = name.endswith("_host")
    dtype = gk.GK_BF16 if w.dtype == "bf16" else gk.GK_FP8_E4M3
    flags = gk.GK_FLAG_SINGLE_PASS if single_pass else 0
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, dtype, w.scale_kv, flags)
    ctx = gk.Context(geom, device.index)
    for kv in filter(None, tune.split(",")):
        key, val = kv.split("=")
        ctx.set_tuning(key, int(val))
    restore_traffic = 2 if single_pass else 3     # DRAM bytes per blob byte of the restore
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    pages = [-(-n // w.page_tokens) for n in lens]
    src_pages = sum(pages)

    def cache(num_pages, seed):
        if w.dtype == "bf16":
            data = synth.kv_bytes_bf16(2 * w.layers * num_pages * slab // 2, w.sigma, seed, device)
            return gk.Cache(data, num_pages, 2 * num_pages * slab, num_pages * slab, slab)
        data, scales = synth.kv_bytes_fp8(w.layers, num_pages, w.page_tokens, w.kv_heads, w.head_dim, w.sigma,
                                          seed, device)
        h4 = w.kv_heads * 4
        return gk.Cache(data, num_pages, 2 * num_pages * slab, num_pages * slab, slab, scales,
                        w.scale_kv * num_pages * h4, num_pages * h4, h4)

    src, dst = cache(src_pages, w.seed(10)), cache(dst_pages, w.seed(11))
    sperm = torch.from_numpy(synth.page_permutation(src_pages, w.seed(12))).to(device)
    dperm = torch.from_numpy(synth.page_permutation(dst_pages, w.seed(13))).to(device)
    pack_jobs, restore_jobs, blobs, off, total = [], [], [], 0, 0
    for n, P in zip(lens, pages):
        nb, _ = gk.gk_blob_size(geom, n)
        total += nb
        if host_tier:
            blob = torch.empty(nb, dtype=torch.uint8, pin_memory=True)
            sums = torch.zeros(P, dtype=torch.int64, pin_memory=True)
        else:
            blob = torch.empty(nb, dtype=torch.uint8, device=device)
            sums = torch.zeros(P, dtype=torch.int64, device=device)
        blobs.append(blob)
        pack_jobs.append(gk.Job(blob, sums, sperm[off:off + P].contiguous(), n))
        restore_jobs.append(gk.Job(blob, sums, dperm[off:off + P].contiguous(), n))
        off += P
    nj = len(lens)
    pack_jobs, restore_jobs = gk.JobArray(pack_jobs), gk.JobArray(restore_jobs)   # marshalled once
    mask = torch.zeros(nj, dtype=torch.uint8, device=device)
    fb = torch.zeros(nj, dtype=torch.int32, device=device)
    status = torch.zeros(nj, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device)
    do_pack = (lambda: ctx.gk_pack_host(src, pack_jobs, status)) if host_tier else (lambda: ctx.gk_pack_batch(src, pack_jobs, status))
    do_restore = ((lambda: ctx.gk_restore_host(restore_jobs, dst, mask, fb)) if host_tier
                  else (lambda: ctx.gk_restore(restore_jobs, dst, mask, fb)))
    if host_tier:
        steps, warmup = min(steps, 2), 1

    def timed(fn, reps):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize(device)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(reps)]
        for k in range(reps):
            ev[k][0].record(stream)
            fn()
            ev[k][1].record(stream)
        torch.cuda.synchronize(device)
        return [e[0].elapsed_time(e[1]) for e in ev]

    pack_ms = timed(do_pack, steps)
    assert int(status.sum().item()) == 0

    # damage, as the configuration prescribes it (seeded); expected number of rejected blocks
    expect_rejected, damage = 0, "none"
    rng = np.random.default_rng(w.seed(14))
    R = w.layers * w.scale_kv * w.kv_heads * 4 + w.page_tokens * 2 * w.layers * (slab // w.page_tokens)
    S = w.layers * w.scale_kv * w.kv_heads * 4
    if name == "tiny":
        j = int(rng.integers(0, nj))
        pos = int(synth.bit_flip_positions(blobs[j].numel() * 8, 1, w.seed(15))[0])
        blobs[j][pos >> 3] ^= 1 << (pos & 7)
        expect_rejected, damage = 1, "one flipped bit in one of the 4 blobs"
    elif name == "fp8":
        ja, jb_ = (int(x) for x in rng.choice(nj, size=2, replace=False))
        pa, pb = int(rng.integers(0, pages[ja])), int(rng.integers(0, pages[jb_]))
        start, xors = synth.byte_run_corruption(pa * R, pa * R + S, 8, w.seed(6))
        blobs[ja][start:start + 8] ^= torch.from_numpy(xors).to(device)
        start, xors = synth.byte_run_corruption(pb * R + S, pb * R + S + slab, 8, w.seed(7))
        blobs[jb_][start:start + 8] ^= torch.from_numpy(xors).to(device)
        expect_rejected, damage = 2, "8 consecutive bytes in a scale section of one blob and in the K data of another"
    elif name.startswith("stress"):
        frac = 1.0 / 3.0 if name.endswith("one_third_damaged") else 0.01
        bad_ids, bad_flips = synth.stress_corrupted_blocks(w.seed(2), frac=frac)
        bad = dict(zip(bad_ids.tolist(), bad_flips.tolist()))
        for j, b in enumerate(ids):
            if b in bad:
                for pos in synth.bit_flip_positions(blobs[j].numel() * 8, bad[b], w.seed(50_000 + b)):
                    blobs[j][int(pos) >> 3] ^= 1 << (int(pos) & 7)
                expect_rejected += 1
        damage = f"1 to 8 flipped bits in the blobs of a seeded {frac:.2%} of the pool's blocks"
    torch.cuda.synchronize(device)

    restore_ms = timed(do_restore, steps)
    mask_host = mask.cpu().numpy()
    committed = int(sum(b.numel() for b, m in zip(blobs, mask_host) if m == 0))
    codes = np.bincount(mask_host, minlength=5)
    census = {"ok": int(codes[0]), "checksum": int(codes[1]), "page_table": int(codes[2]), "missing": int(codes[3]),
              "wait_ran_out": int(codes[4]), "expected_rejected": expect_rejected}
    assert census["checksum"] == expect_rejected and census["ok"] == nj - expect_rejected, census
    assert ctx.gk_get_stats()["device_wait_expired"] == 0
    peak, peak_kind = measured_peak()
    pm, rm = float(np.median(pack_ms)), float(np.median(restore_ms))
    rec = {"workload": f"{name}: {w.layers} layers, {w.kv_heads} KV heads, head_dim {w.head_dim}, {w.dtype}, "
                       f"{w.page_tokens}-token pages; {nj} blocks, {sum(lens)} tokens, {total / 2**30:.2f} GiB of blobs, "
                       f"{dst_pages}-page destination" + (", blobs in pinned host memory" if host_tier else ""),
           "jobs": nj, "tokens": int(sum(lens)), "blob_bytes": int(total), "damage": damage, "mask_census": census,
           "save_ms": stats_ms(pack_ms), "restore_ms": stats_ms(restore_ms),
           "restored_tokens_per_s": sum(lens) / (rm * 1e-3)}
    if host_tier:
        rec["save_host_link_gbs"] = total / (pm * 1e-3) / 1e9
        rec["restore_host_link_gbs"] = total / (rm * 1e-3) / 1e9
    else:
        rec["save"] = fractions(2 * total / (pm * 1e-3) / 1e9, peak)
        # every blob is read once to be verified; only the accepted ones are read again and written
        rec["committed_blob_bytes"] = committed
        rec["restore_useful"] = fractions((total + committed) / (rm * 1e-3) / 1e9, peak)
        rec["restore_dram_model"] = dict(fractions((total + (restore_traffic - 1) * committed) / (rm * 1e-3) / 1e9, peak),
                                         dram_bytes="blob bytes read to verify + %d x the bytes of the accepted blobs"
                                                    % (restore_traffic - 1))
    ctx.close()
    del src, dst, blobs, pack_jobs, restore_jobs
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return rec


def latency_cases(device, token_counts=(256, 1024, 5200, 24018), reps=15):
    """Restore of ONE block of the GQA-7B geometry, the serving case of a single recurring
    prompt: device time per call, L2 flushed before every call (the blob is cold in HBM, as
    it is after sitting in the pool), median and best; beside it the time the bytes alone
    would take at the measured copy peak (blob read twice and written once, and read once)."""
    import torch
    import synth
    import paper_2609_39358_b200 as gk
    w = synth.GQA7B
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    peak, _ = measured_peak()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device)
    out = {}
    for n in token_counts:
        ctx = gk.Context(geom, device.index)
        nb, P = gk.gk_blob_size(geom, n)
        data = synth.kv_bytes_bf16(w.layers * P * slab, w.sigma, w.seed(600 + n), device)
        src = gk.Cache(data, P, 2 * P * slab, P * slab, slab)
        dst = gk.Cache(torch.zeros_like(data), P, 2 * P * slab, P * slab, slab)
        blob = torch.empty(nb, dtype=torch.uint8, device=device)
        sums = torch.zeros(P, dtype=torch.int64, device=device)
        spt = torch.from_numpy(synth.page_permutation(P, w.seed(601))).to(device)
        dpt = torch.from_numpy(synth.page_permutation(P, w.seed(602))).to(device)
        ctx.gk_pack(src, spt, n, blob, sums)
        jobs = gk.JobArray([gk.Job(blob, sums, dpt, n)])
        mask = torch.zeros(1, dtype=torch.uint8, device=device)
        fb = torch.zeros(1, dtype=torch.int32, device=device)
        for _ in range(3):
            ctx.gk_restore(jobs, dst, mask, fb)
        torch.cuda.synchronize(device)
        ts = []
        for _ in range(reps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            ctx.gk_restore(jobs, dst, mask, fb)
            e1.record(stream)
            torch.cuda.synchronize(device)
            ts.append(e0.elapsed_time(e1) * 1e3)
        assert int(mask.item()) == 0
        # back to back, without the flush: what a caller sees who restores the same block again at once
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b2b = max(reps, 50)   # enough calls for the first one's launch latency not to show
        e0.record(stream)
        for _ in range(b2b):
            ctx.gk_restore(jobs, dst, mask, fb)
        e1.record(stream)
        torch.cuda.synchronize(device)
        warm = e0.elapsed_time(e1) * 1e3 / b2b
        med = float(np.median(ts))
        bound3 = 3 * nb / (peak * 1e9) * 1e6
        out[f"{n}_tokens"] = {"blob_mib": nb / 2**20, "restore_us_median": med, "restore_us_best": float(np.min(ts)),
                              "restore_us_back_to_back": warm, "bound_us_3_bytes_per_byte": bound3,
                              "frac_of_bound": bound3 / med, "bound_us_2_bytes_per_byte": 2 * nb / (peak * 1e9) * 1e6,
                              "restored_tokens_per_s": n / (med * 1e-6)}
        ctx.close()
        del data, src, dst, blob
        torch.cuda.empty_cache()
    return out


def run_latency(args):
    import torch
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    cases = latency_cases(device, (args.tokens,) if args.tokens else (256, 1024, 5200, 24018),
                          reps=max(3, min(args.steps, 15)))
    first = next(iter(cases.values()))
    line = {"metric": "restore of one block, device time per call", "value": first["restore_us_median"], "unit": "us",
            "n_gpus": 1, "steps": max(3, min(args.steps, 15)), "warmup": 3, "ms_per_step": first["restore_us_median"] / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": "latency: gqa7b geometry, one block per call, L2 flushed before every call"},
            "latency": cases}
    print(json.dumps(line), flush=True)


def run_other_workload(args):
    import torch
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    name = {"stress": "stress_wave", "records": "gqa7b"}.get(args.workload, args.workload)
    rec = workload_case(name, device, steps=max(args.steps, 1) if args.steps < 50 else 10, warmup=max(args.warmup, 3),
                        single_pass=args.single_pass, blocks=args.blocks, tune=args.tune,
                        layers=args.layers if args.workload == "records" else 0)
    pm, rm = rec["save_ms"]["median"], rec["restore_ms"]["median"]
    line = {"metric": METRIC, "value": rec["restore_useful"]["gbs"], "unit": UNIT, "n_gpus": 1,
            "steps": rec["restore_ms"]["n"], "warmup": max(args.warmup, 3), "ms_per_step": pm + rm,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": rec["workload"],
                       "step": "gk_pack_batch, then gk_restore, of all blocks in one call each, timed separately"
                               + (" (restore in a single pass: GK_FLAG_SINGLE_PASS)" if args.single_pass else "")},
            "case": rec}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# long window at flat GPU memory: a corpus far larger than the cache streamed
# from pinned host memory through a ring of pages (gk_restore_stream)
# ---------------------------------------------------------------------------
def run_longwindow(args):
    import torch
    import synth
    import paper_2609_39358_b200 as gk

    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    w = synth.GQA7B
    block_tokens, pool_blocks, ring_blocks = 30000, 4, 2
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
    ctx = gk.Context(geom, device.index)
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    P = -(-block_tokens // w.page_tokens)
    nb, _ = gk.gk_blob_size(geom, block_tokens)

    def cache(num_pages, seed):
        data = synth.kv_bytes_bf16(2 * w.layers * num_pages * slab // 2, w.sigma, seed, device)
        return gk.Cache(data, num_pages, 2 * num_pages * slab, num_pages * slab, slab)

    # the saved corpus: pool_blocks distinct blobs in pinned host memory, visited round-robin
    pool = []
    ident = torch.arange(P, dtype=torch.int32, device=device)
    for k in range(pool_blocks):
        src = cache(P, w.seed(700 + k))
        hb = torch.empty(nb, dtype=torch.uint8, pin_memory=True)
        hs = torch.zeros(P, dtype=torch.int64, pin_memory=True)
        ctx.gk_pack_host(src, [gk.Job(hb, hs, ident, block_tokens)])
        torch.cuda.synchronize(device)
        pool.append((hb, hs))
        del src
    torch.cuda.empty_cache()
    ring = cache(ring_blocks * P, w.seed(710))
    n_jobs = args.window_blocks
    jobs = [gk.Job(pool[j % pool_blocks][0], pool[j % pool_blocks][1], None, block_tokens) for j in range(n_jobs)]
    mask = torch.zeros(n_jobs, dtype=torch.uint8, device=device)
    fb = torch.zeros(n_jobs, dtype=torch.int32, device=device)
    touched = torch.zeros(1, dtype=torch.int64, device=device)
    windows = []

    def consume(blocks, st):
        # stand-in for the reader of the window: one cheap stream-ordered pass over part of the ring
        windows.append(len(blocks))
        touched.add_(ring.data[:1 << 20].sum())

    stream = torch.cuda.current_stream(device)
    steps, warmup = max(1, min(args.steps, 3)), 1
    for _ in range(warmup):
        ctx.gk_restore_stream(jobs, ring, mask, fb, consume)
    torch.cuda.synchronize(device)
    free_before, total_mem = torch.cuda.mem_get_info(device)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    windows.clear()
    ev[0].record(stream)
    for _ in range(steps):
        ctx.gk_restore_stream(jobs, ring, mask, fb, consume)
    ev[1].record(stream)
    torch.cuda.synchronize(device)
    free_after, _ = torch.cuda.mem_get_info(device)
    assert int(mask.sum().item()) == 0
    ms = ev[0].elapsed_time(ev[1]) / steps
    total = n_jobs * nb
    line = {"metric": "streamed restore from pinned host memory, blob GB/s", "value": total / (ms * 1e-3) / 1e9,
            "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": f"longwindow: gqa7b geometry, {n_jobs} blocks x {block_tokens} tokens "
                                   f"({n_jobs * block_tokens / 1e6:.2f} M tokens, {total / 2**30:.1f} GiB of blobs, "
                                   f"{pool_blocks} distinct blobs visited round-robin) through a ring of "
                                   f"{ring_blocks} blocks ({ring_blocks * P} pages)",
                       "step": "one gk_restore_stream call; the consumer touches the ring after every window"},
            "tokens_per_s": n_jobs * block_tokens / (ms * 1e-3),
            "windows_per_step": len(windows) // steps,
            "device_memory": {"used_bytes": total_mem - free_after, "growth_during_timed_steps": free_before - free_after,
                              "ring_bytes": ring.data.numel(), "total_bytes": total_mem}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# second tier: block fingerprints and blob digests (SHA-256) on the headline batch
# ---------------------------------------------------------------------------
# Integer instructions per 64-byte SHA-256 block in the kernels (14 per round, 10 per
# message-schedule word, 16 byte swaps, 8 final adds, loads and loop overhead), all of
# which issue on the 64-lane integer pipe of an SM.
SHA_INSTR_PER_BLOCK = 64 * 14 + 48 * 10 + 16 + 8 + 10
INT_LANES_PER_SM_CLK = 64
SM_COUNT = 148


def run_digest(args):
    import torch
    import synth
    import paper_2609_39358_b200 as gk

    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    w = synth.GQA7B
    n_blocks = args.blocks or synth.GQA7B_REQUESTS * synth.GQA7B_BLOCKS_PER_REQUEST
    n_tok = synth.GQA7B_BLOCK_TOKENS
    geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
    ctx = gk.Context(geom, device.index)
    nb, P = gk.gk_blob_size(geom, n_tok)
    # blob bytes: any bytes do for a hash; bf16 N(0, sigma) patterns like the cache contents
    blobs = [synth.kv_bytes_bf16(nb // 2, w.sigma, w.seed(800 + j), device) for j in range(n_blocks)]
    jobs = [gk.Job(b, None, None, n_tok) for b in blobs]
    # token ids of the blocks (int32), two-block chains per request
    g = torch.Generator(device=device)
    g.manual_seed(w.seed(820))
    ids = torch.randint(0, 128000, (n_blocks * n_tok,), generator=g, device=device, dtype=torch.int32)
    offsets = torch.arange(n_blocks + 1, dtype=torch.int64, device=device) * (4 * n_tok)
    parent = [(-1 if j % synth.GQA7B_BLOCKS_PER_REQUEST == 0 else j - 1) for j in range(n_blocks)]
    model, tenant = bytes(range(32)), bytes(range(32, 64))
    keys = torch.zeros(n_blocks, 32, dtype=torch.uint8, device=device)
    digests = torch.zeros(n_blocks, 32, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device)
    steps, warmup = min(args.steps, 20), max(args.warmup, 3)

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        ctx.gk_fingerprints(ids.view(torch.uint8), offsets, parent, model, tenant, keys)
        if ev:
            ev[1].record(stream)
        ctx.gk_blob_digests(jobs, keys, digests)
        if ev:
            ev[2].record(stream)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize(device)
    sampler = ClockSampler(device.index)
    sampler.wait_first_sample()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for k in range(steps):
        step(events[k])
    torch.cuda.synchronize(device)
    clocks = sampler.stop() or {}
    fp_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in events]))
    dg_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in events]))
    total = n_blocks * nb
    sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965
    peak = SM_COUNT * INT_LANES_PER_SM_CLK * sm_mhz * 1e6 / (SHA_INSTR_PER_BLOCK / 64.0) / 1e9
    achieved = total / (dg_ms * 1e-3) / 1e9
    line = {"metric": "blob digest GB/s (SHA-256 tree)", "value": achieved, "unit": UNIT, "n_gpus": 1, "steps": steps,
            "warmup": warmup, "ms_per_step": fp_ms + dg_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": f"digest: gqa7b geometry, {n_blocks} blocks x {n_tok} tokens, {total / 2**30:.2f} GiB of "
                                   f"blobs, {n_blocks} keys over {4 * n_tok}-byte token-id blocks in chains of "
                                   f"{synth.GQA7B_BLOCKS_PER_REQUEST}",
                       "step": "gk_fingerprints + gk_blob_digests; inputs (8 GiB) larger than L2"},
            "phases": {"fingerprints": {"ms": fp_ms}, "blob_digests": {"ms": dg_ms, "gbs": achieved}},
            "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None,
                         "peak_kind": f"derived: {SM_COUNT} SMs x {INT_LANES_PER_SM_CLK} integer lanes per clock x "
                                      f"{sm_mhz} MHz (sampled) / {SHA_INSTR_PER_BLOCK / 64.0:.1f} instructions per byte"},
            "clocks": clocks}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# layer-wise load from the host tier: when is each group of layers ready?
# ---------------------------------------------------------------------------
def run_layerwise(args):
    import torch
    import synth
    import paper_2609_39358_b200 as gk

    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    w = synth.GQA7B
    group_layers, n_groups = 4, w.layers // 4
    g_geom = gk.Geom(group_layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
    f_geom = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
    ctx_g, ctx_f = gk.Context(g_geom, device.index), gk.Context(f_geom, device.index)
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    stream = torch.cuda.current_stream(device)
    out = {}
    for name, lens in (("prompt_5200_tokens", [5200]), ("batch_4_x_4096_tokens", [4096] * 4)):
        pages = [-(-n // w.page_tokens) for n in lens]
        N = sum(pages)
        data = synth.kv_bytes_bf16(2 * w.layers * N * slab // 2, w.sigma, w.seed(900), device)
        src = gk.Cache(data, N, 2 * N * slab, N * slab, slab)
        dst = gk.Cache(torch.zeros_like(data), N, 2 * N * slab, N * slab, slab)
        tables, off = [], 0
        perm = torch.from_numpy(synth.page_permutation(N, w.seed(901))).to(device)
        for P in pages:
            tables.append(perm[off:off + P].contiguous())
            off += P
        lw_jobs, std_jobs, total = [], [], 0
        for n, P, pt in zip(lens, pages, tables):
            nb, _ = gk.gk_blob_size(f_geom, n)
            total += nb
            lw_jobs.append(gk.Job(torch.empty(nb, dtype=torch.uint8, pin_memory=True),
                                  torch.empty(n_groups * P, dtype=torch.int64, pin_memory=True), pt, n))
            std_jobs.append(gk.Job(torch.empty(nb, dtype=torch.uint8, pin_memory=True),
                                   torch.empty(P, dtype=torch.int64, pin_memory=True), pt, n))
        ctx_g.gk_pack_layerwise(n_groups, src, lw_jobs, host=True)
        ctx_f.gk_pack_host(src, std_jobs)
        torch.cuda.synchronize(device)
        nj = len(lens)
        mask = torch.zeros(nj, dtype=torch.uint8, device=device)
        fb = torch.zeros(nj, dtype=torch.int32, device=device)
        reps = 5
        whole_ms, group_ms = [], []
        for r in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            ctx_f.gk_restore_host(std_jobs, dst, mask, fb)
            e1.record(stream)
            torch.cuda.synchronize(device)
            assert int(mask.sum().item()) == 0
            ready = []
            g0 = torch.cuda.Event(enable_timing=True)
            g0.record(stream)

            def on_group(group, first_layer, n_layers, st):
                ev = torch.cuda.Event(enable_timing=True)
                ev.record(stream)
                ready.append(ev)

            ctx_g.gk_restore_layerwise(n_groups, lw_jobs, dst, mask, fb, None, on_group, host=True)
            torch.cuda.synchronize(device)
            assert int(mask.sum().item()) == 0
            if r > 0:
                whole_ms.append(e0.elapsed_time(e1))
                group_ms.append([g0.elapsed_time(ev) for ev in ready])
        gm = np.mean(np.array(group_ms), axis=0)
        out[name] = {"blob_gib": total / 2**30, "ordinary_restore_host_ms": float(np.mean(whole_ms)),
                     "layerwise_group_ready_ms": [round(float(x), 3) for x in gm],
                     "layerwise_total_ms": float(gm[-1]),
                     "first_group_ready_after_fraction": float(gm[0] / np.mean(whole_ms)),
                     "host_link_gbs_layerwise": total / (float(gm[-1]) * 1e-3) / 1e9}
        del data, src, dst, lw_jobs, std_jobs
        torch.cuda.empty_cache()
    line = {"metric": "layer-wise restore from pinned host memory: ms until each group of layers is ready",
            "value": out["prompt_5200_tokens"]["layerwise_group_ready_ms"][0], "unit": "ms", "n_gpus": 1,
            "steps": 5, "warmup": 1, "ms_per_step": out["prompt_5200_tokens"]["layerwise_total_ms"],
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": f"layerwise: gqa7b geometry, {n_groups} groups of {group_layers} layers; a 5,200-token "
                                   "prompt block and a batch of 4 x 4,096 tokens, blobs in pinned host memory",
                       "step": "gk_restore_layerwise_host, an event recorded in the group call-back; beside it "
                               "gk_restore_host of the same blocks in the ordinary format"},
            "cases": out}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# layer-wise save and load on the device tier: what the smaller records cost
# ---------------------------------------------------------------------------
def run_layerwise_device(args):
    """The headline batch (16 blocks x 4,096 tokens of the gqa7b geometry, 8 GiB) saved and restored
    group of layers by group of layers with gk_pack_layerwise / gk_restore_layerwise, blobs on the device:
    one ordinary call per group, records `group_layers` layers tall."""
    import torch
    import synth
    import paper_2609_39358_b200 as gk

    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    w = synth.GQA7B
    peak, _ = measured_peak()
    slab = w.page_tokens * w.kv_heads * w.head_dim * w.elem_bytes
    n_blocks, n_tok = 16, 4096
    P = n_tok // w.page_tokens
    N = n_blocks * P
    data = synth.kv_bytes_bf16(2 * w.layers * N * slab // 2, w.sigma, w.seed(950), device)
    src = gk.Cache(data, N, 2 * N * slab, N * slab, slab)
    dst = gk.Cache(torch.zeros_like(data), N, 2 * N * slab, N * slab, slab)
    perm_s = torch.from_numpy(synth.page_permutation(N, w.seed(951))).to(device)
    perm_d = torch.from_numpy(synth.page_permutation(N, w.seed(952))).to(device)
    stream = torch.cuda.current_stream(device)
    reps = max(3, min(args.steps, 10))
    out = {}
    for g in ((args.layers,) if any(a.startswith("--layers") for a in sys.argv) else (32, 8, 4, 2, 1)):
        n_groups = w.layers // g
        geom = gk.Geom(g, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
        full = gk.Geom(w.layers, w.kv_heads, w.head_dim, w.page_tokens, gk.GK_BF16, 0)
        ctx = gk.Context(geom, device.index)
        nb, _ = gk.gk_blob_size(full, n_tok)
        sj, rj, keep = [], [], []
        for b in range(n_blocks):
            blob = torch.empty(nb, dtype=torch.uint8, device=device)
            sums = torch.zeros(n_groups * P, dtype=torch.int64, device=device)
            keep.append((blob, sums))
            sj.append(gk.Job(blob, sums, perm_s[b * P:(b + 1) * P].contiguous(), n_tok))
            rj.append(gk.Job(blob, sums, perm_d[b * P:(b + 1) * P].contiguous(), n_tok))
        sj, rj = gk.JobArray(sj), gk.JobArray(rj)
        mask = torch.zeros(n_blocks, dtype=torch.uint8, device=device)
        fb = torch.zeros(n_blocks, dtype=torch.int32, device=device)
        ts = {"save": [], "restore": []}
        for r in range(reps + 3):
            for name, fn in (("save", lambda: ctx.gk_pack_layerwise(n_groups, src, sj)),
                             ("restore", lambda: ctx.gk_restore_layerwise(n_groups, rj, dst, mask, fb))):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn()
                e1.record(stream)
                torch.cuda.synchronize(device)
                if r >= 3:
                    ts[name].append(e0.elapsed_time(e1))
        assert int(mask.sum().item()) == 0
        total = n_blocks * nb
        sm, rm = float(np.median(ts["save"])), float(np.median(ts["restore"]))
        out[f"{g}_layers_per_group"] = {
            "groups": n_groups, "record_kib": 2 * g * slab // 1024, "save_ms": stats_ms(ts["save"]),
            "restore_ms": stats_ms(ts["restore"]),
            "save_frac_of_measured_peak": 2 * total / (sm * 1e-3) / 1e9 / peak,
            "restore_frac_of_measured_peak_3_bytes": 3 * total / (rm * 1e-3) / 1e9 / peak,
            "quartet_launches": ctx.gk_get_stats()["quartet_launches"]}
        ctx.close()
        del sj, rj, keep
        torch.cuda.empty_cache()
    first = next(iter(out.values()))
    line = {"metric": METRIC, "value": 2 * n_blocks * nb / (first["restore_ms"]["median"] * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": 1, "steps": reps, "warmup": 3, "ms_per_step": first["save_ms"]["median"] + first["restore_ms"]["median"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": "layerwise-device: gqa7b geometry, 16 blocks x 4,096 tokens (8 GiB of blobs on the "
                                   "device), saved and restored one group of layers at a time",
                       "step": "gk_pack_layerwise, then gk_restore_layerwise, timed separately"},
            "cases": out}
    print(json.dumps(line), flush=True)


def synth_requests(n_blocks):
    return f"{max(n_blocks // 2, 1)} requests x {min(n_blocks, 2)} blocks"


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "longwindow":
        run_longwindow(args)
    elif args.workload == "digest":
        run_digest(args)
    elif args.workload == "layerwise":
        run_layerwise(args)
    elif args.workload == "layerwise-device":
        run_layerwise_device(args)
    elif args.workload == "latency":
        run_latency(args)
    elif args.workload != "gqa7b" or args.single_pass:
        run_other_workload(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
