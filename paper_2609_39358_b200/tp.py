"""Tensor-parallel restore: every rank holds its own shard (its KV heads) of each
block, with its own blobs, checksums and destination cache.  A block may be
written only if it verified on ALL ranks, otherwise the ranks' caches would
disagree.  The only exchange step is the agreement on the per-block result:

    gk_verify on every rank  ->  all-reduce(max) of the uint8 masks  ->  gk_commit

The all-reduce moves n_jobs bytes (NCCL over NVLink/NVSwitch: latency-bound).
All other work is the ordinary single-GPU path; no kernel touches a peer's memory.
The paper itself only reports that its library runs under the serving runtime's
tensor parallelism (Table 1, and Section 4.4); this helper is this build's way of
keeping the fail-closed rule intact across ranks.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch
import torch.distributed as dist


def tp_restore(ctx, jobs: Sequence, dst, mask: torch.Tensor, first_bad_page: torch.Tensor,
               group: Optional["dist.ProcessGroup"] = None, stream=None) -> None:
    """Verify on this rank, agree with the other ranks of ``group``, commit.

    ``mask`` ends up holding the agreed code of every job (the maximum over the
    ranks, so 0 only if all ranks verified the job); ``first_bad_page`` stays this
    rank's own finding.  The collective is issued through torch.distributed on the
    current stream, so pass ``stream=None`` (torch's current stream) unless the
    caller orders the streams itself.
    """
    ctx.gk_verify(jobs, dst, mask, first_bad_page, stream)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(mask, op=dist.ReduceOp.MAX, group=group)
    ctx.gk_commit(jobs, dst, mask, stream)
