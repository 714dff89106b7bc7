"""Data-parallel use of the encoder on several GPUs: one process per GPU, each with its own samples,
one exchange per step -- the all-reduce of the float32 parameter-gradient blob -- which is the paper's
own multi-GPU scheme (section 3.3: data parallelism, gradients summed across processes).

BatchNorm statistics stay per replica (each replica normalises over its own valid frames), so a
data-parallel step is NOT the single-GPU step on the concatenated batch; it is the sum (or mean) of the
per-replica gradients, which is what this module computes.  The collective is torch.distributed's
(NCCL over NVLink between GPUs, gloo on CPU for the tests); the compute stays in the library's kernels.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def shard(n_items: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of `n_items` batch items for `rank` (sizes differ by at most one)."""
    lo = n_items * rank // world
    hi = n_items * (rank + 1) // world
    return range(lo, hi)


def all_reduce_gradients(grads_blob: torch.Tensor, op: str = "sum", group: Optional[dist.ProcessGroup] = None,
                         async_op: bool = False):
    """All-reduces the flat gradient blob that encoder_fwd_bwd fills (uint8 view of float32 arrays, every
    array on a 256-byte boundary; the padding between arrays is zero on every rank and stays zero).
    op = "sum" | "mean".  In place; returns the work handle when async_op is set."""
    if op not in ("sum", "mean"):
        raise ValueError(op)
    if grads_blob.dtype != torch.uint8 or grads_blob.numel() % 4:
        raise ValueError("expected the uint8 gradient blob of an EncoderSpec")
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return None
    g = grads_blob.view(torch.float32)
    work = dist.all_reduce(g, op=dist.ReduceOp.SUM, group=group, async_op=async_op)
    if op == "mean":
        if async_op:
            work.wait()
            work = None
        g.div_(dist.get_world_size(group))
    return work


def data_parallel_step(api, ctx, spec, x, lengths, params_blob, dlogits, grads_blob, workspace, logits=None,
                       op: str = "sum", group=None):
    """One data-parallel training step on this rank's samples: encoder forward + backward through the C ABI,
    then the gradient exchange.  Returns (logits, out_lengths)."""
    logits, out_len, _, _ = api.encoder_fwd_bwd(ctx, spec, x, lengths, params_blob, dlogits, grads_blob=grads_blob,
                                                workspace=workspace, logits=logits)
    all_reduce_gradients(grads_blob, op=op, group=group)
    return logits, out_len
