"""Token-data-parallel plumbing around libatgrpo (one process per GPU, torch.distributed).

The policy-update path shards by environment: every (environment, role, turn) group then lives on
one rank, so the grouped advantages (Eq. 1) need no communication.  The loss of Eq. 2 is a mean
over ALL tokens of policy m, so each rank weights its local loss and gradient by
T_m(local) / T_m(global) -- passed to the library as `grad_loss` -- and the only data-path exchange
is one sum all-reduce of each dW_m (NCCL over NVLink on GPUs, gloo in the CPU tests), which
`backward_overlapped` starts chunk by chunk while the backward kernels are still running.
Nothing here computes advantages, log-probs or losses.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

__all__ = ["shard_batch_by_env", "token_mean_scale", "allreduce_gradients", "chunk_row_ranges",
           "allreduce_gradient_rows", "backward_overlapped"]


def shard_batch_by_env(batch: dict, rank: int, world: int) -> dict:
    """Sub-batch of the environments e with e % world == rank (whole groups stay together).
    Candidate and token order is preserved; response indices are renumbered densely.  Environment
    ids are kept, so the group key space (n_env slots) is unchanged and merely sparser."""
    keep_resp = (batch["env_id"] % world) == rank
    new_index = torch.cumsum(keep_resp.to(torch.int64), 0) - 1
    keep_tok = keep_resp[batch["resp_of_token"].long()]
    out = dict(batch)
    for k in ("rewards", "env_id", "role_id", "turn_id", "resp_len"):
        out[k] = batch[k][keep_resp].contiguous()
    out["resp_of_token"] = new_index[batch["resp_of_token"].long()][keep_tok].to(torch.int32).contiguous()
    for k in ("role_of_token", "target", "H"):
        if k in batch:
            out[k] = batch[k][keep_tok].contiguous()
    out["T"] = int(keep_tok.sum())
    out["R"] = int(keep_resp.sum())
    out["token_index"] = torch.nonzero(keep_tok).squeeze(1)
    return out


def token_mean_scale(local_counts: torch.Tensor, group=None):
    """local_counts[m] = tokens of policy m on this rank.  Returns (scale[m] float32, global
    counts): scale = local / global (0 where the policy has no token anywhere), the weight that
    turns per-rank token means into the global token mean when summed over ranks."""
    total = local_counts.clone().to(torch.int64)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    scale = torch.where(total > 0, local_counts.double() / total.clamp(min=1).double(),
                        torch.zeros_like(total, dtype=torch.float64))
    return scale.to(torch.float32), total


def allreduce_gradients(dW, group=None):
    """Sums every dW_m over the ranks, in place (the one exchange step of the data-parallel path)."""
    if not (dist.is_available() and dist.is_initialized()):
        return
    for w in dW:
        dist.all_reduce(w, op=dist.ReduceOp.SUM, group=group)


def chunk_row_ranges(V: int, n_chunks: int, rows_per_chunk: int):
    """Row ranges [(lo, hi)] of the vocabulary chunks a backward call finishes one after the other."""
    return [(c * rows_per_chunk, min(V, (c + 1) * rows_per_chunk)) for c in range(n_chunks)]


def allreduce_gradient_rows(dW, lo: int, hi: int, group=None):
    """Sums rows [lo, hi) of every dW_m over the ranks, in place."""
    if not (dist.is_available() and dist.is_initialized()) or hi <= lo:
        return
    for w in dW:
        dist.all_reduce(w[lo:hi], op=dist.ReduceOp.SUM, group=group)


def backward_overlapped(A, bwd_kwargs: dict, comm_stream, group=None):
    """The backward call with the all-reduce of dW overlapped: the library records one CUDA event
    per vocabulary chunk as soon as that chunk's rows of every dW_m are final, and `comm_stream`
    waits for each event and then sums those rows over the ranks while the main stream goes on with
    the next chunk.  On return the main stream waits for `comm_stream`, so later work on it sees
    the summed gradient.  `A` is the paper_2510_11062_b200.atgrpo module, bwd_kwargs the keyword
    arguments of A.atgrpo_policy_loss_bwd (H, W, ..., dH, dW, device_status, workspace)."""
    H, W, dW = bwd_kwargs["H"], bwd_kwargs["W"], bwd_kwargs["dW"]
    V = W[0].shape[0]
    n_chunks, rows = A.atgrpo_policy_loss_bwd_chunks(H.shape[0], H.shape[1], V, len(W))
    events = [torch.cuda.Event() for _ in range(n_chunks)]
    A.atgrpo_policy_loss_bwd(**bwd_kwargs, chunk_events=events)
    main = torch.cuda.current_stream()
    with torch.cuda.stream(comm_stream):
        for (lo, hi), ev in zip(chunk_row_ranges(V, n_chunks, rows), events):
            comm_stream.wait_event(ev)
            allreduce_gradient_rows(dW, lo, hi, group)
    main.wait_stream(comm_stream)
