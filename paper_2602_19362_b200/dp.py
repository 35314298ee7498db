"""Data-parallel plumbing for the LM-head step: shard a batch over ranks by prompt and
sum the per-rank results.

Eq. 2 and Eq. 3 of the paper couple only the rollouts of one prompt, so whole groups can
be placed on different ranks with the LM-head weight replicated.  Each rank then runs the
library's single-GPU path on its shard (with the *global* loss_scale), and the only
exchange is the sum of dW and of the scalar loss over the ranks; dH stays local because
its rows belong to the rank's own tokens.  torch.distributed does the transport (NCCL on
GPUs, gloo on CPU tensors); nothing here computes any part of the method.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

_ROW_KEYS = ("H", "targets", "mask", "seq_id", "logp_inf")
_SEQ_KEYS = ("group_id", "reward", "lengths")


def prompts_of_rank(P: int, rank: int, world: int) -> range:
    """Contiguous block of prompt (group) ids owned by `rank`; the first P % world ranks
    own one prompt more."""
    base, extra = divmod(P, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def shard_by_prompt(batch: dict, rank: int, world: int) -> dict:
    """The sub-batch of `batch` (see synth.make_batch) holding the rollouts of this rank's
    prompts: rows and sequences are filtered, sequence and group ids renumbered from 0,
    W shared, loss_scale unchanged (it normalises over the whole batch)."""
    mine = prompts_of_rank(batch["P"], rank, world)
    gid = batch["group_id"]
    seq_sel = (gid >= mine.start) & (gid < mine.stop)
    seq_idx = torch.nonzero(seq_sel).flatten()
    new_seq = torch.full((batch["S"],), -1, dtype=torch.int64, device=gid.device)
    new_seq[seq_idx] = torch.arange(seq_idx.numel(), device=gid.device)
    row_sel = seq_sel[batch["seq_id"].long()]
    out = dict(batch)
    for k in _ROW_KEYS:
        out[k] = batch[k][row_sel].contiguous()
    out["seq_id"] = new_seq[batch["seq_id"][row_sel].long()].to(torch.int32)
    for k in _SEQ_KEYS:
        if k in batch and torch.is_tensor(batch[k]):
            out[k] = batch[k].to(seq_sel.device)[seq_sel].contiguous()
    out["group_id"] = (out["group_id"] - mine.start).to(torch.int32)
    out["N"] = int(row_sel.sum())
    out["S"] = int(seq_idx.numel())
    out["P"] = len(mine)
    out["live_tokens"] = int(out["mask"].sum())
    return out


def allreduce_outputs(loss: torch.Tensor, dW: torch.Tensor, group=None) -> None:
    """Sum the per-rank loss and dW over the ranks, in place (no-op without a process group)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=group)


def start_allreduce_dW(dW: torch.Tensor, dW_ready=None, comm_stream=None, group=None):
    """Begin the sum of dW over the ranks while the step is still computing dH.

    dW is complete before the single call's last dH contraction starts; the call records
    `dW_ready` (a torch.cuda.Event) at that point.  On CUDA tensors the all-reduce is enqueued
    on `comm_stream` behind that event, so NCCL runs under the remaining compute; on CPU
    tensors (gloo) it is started asynchronously at once.  Returns a handle for
    finish_allreduce; None without a process group.  (A group of one rank still goes through the
    same streams and events; the sum is then the identity.)"""
    if not dist.is_available() or not dist.is_initialized():
        return None
    if dW.is_cuda:
        if dW_ready is None or comm_stream is None:
            raise ValueError("CUDA tensors need the dW-ready event and a communication stream")
        with torch.cuda.stream(comm_stream):
            comm_stream.wait_event(dW_ready)
            dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
        return ("cuda", comm_stream)
    return ("cpu", dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group, async_op=True))


def finish_allreduce(handle, loss: torch.Tensor, group=None) -> None:
    """Sum the scalar loss over the ranks (it is complete only when the step's last kernel is)
    and make the caller's stream wait for the dW exchange started by start_allreduce_dW."""
    if handle is None:
        return
    dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=group)
    kind, h = handle
    if kind == "cuda":
        torch.cuda.current_stream().wait_stream(h)
    else:
        h.wait()
