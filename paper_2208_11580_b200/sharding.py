"""Row sharding of one layer across ranks (one process per GPU).

Rows of W are independent problems that share one Hessian (Section 3 of "Optimal Brain Compression": no Hessian
interaction between rows), so a layer splits across GPUs by row range with no exchange during the elimination.
The only exchange step is before the global mask selection (Algorithm 2), which needs every row's loss trace
and order: one all-gather of 8 * d_row * d_col bytes, after which every rank runs the selection redundantly and
applies it to its own rows.  Each rank builds and inverts the Hessian itself (redundant, a few ms).

This module holds only the partition arithmetic and the collective; the kernels are reached through the package's
C-ABI binding.  It works with any torch.distributed backend (NCCL on GPUs; gloo on CPU tensors in the tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_range(d_row: int, world: int, rank: int) -> tuple[int, int]:
    """(row_begin, row_count) of `rank`: contiguous ranges, sizes differing by at most one, lower ranks first."""
    if d_row < 0 or world < 1 or not 0 <= rank < world:
        raise ValueError("bad partition arguments")
    base, extra = divmod(d_row, world)
    begin = rank * base + min(rank, extra)
    return begin, base + (1 if rank < extra else 0)


def gather_rows(local: torch.Tensor, d_row: int, group=None) -> torch.Tensor:
    """All-gather of a row-sharded 2-D tensor: `local` holds this rank's rows (row_range order); returns the full
    d_row x d_col tensor on every rank.  Ranges of unequal size are padded to the largest for the collective."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    begin, count = row_range(d_row, world, rank)
    if local.dim() != 2 or local.shape[0] != count:
        raise ValueError(f"rank {rank}: expected {count} local rows, got {tuple(local.shape)}")
    most = -(-d_row // world) if d_row else 0
    pad = local
    if count < most:
        pad = torch.cat([local, local.new_zeros(most - count, local.shape[1])], dim=0)
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad.contiguous(), group=group)
    return torch.cat([parts[r][:row_range(d_row, world, r)[1]] for r in range(world)], dim=0)


def gather_traces(loss_local: torch.Tensor, order_local: torch.Tensor, d_row: int, group=None):
    """The exchange step before Algorithm 2: every rank ends up with the loss traces and orders of all rows."""
    return gather_rows(loss_local, d_row, group), gather_rows(order_local, d_row, group)


def prune_layer_sharded(W, X, sparsities, damp_rel: float, prec: int = 2, group=None, keep_trace: bool = True):
    """One layer, rows sharded over the ranks of `group` (CUDA tensors, every rank holds all of W and X):
    Hessian and inverse on every rank, pruning trace on the rank's rows, all-gather of the traces, global masks for
    each sparsity on every rank, final weights of the rank's rows.  Returns a dict with the local row range, the
    global counts/masks per sparsity and the local final weights per sparsity (status: local rows)."""
    import paper_2208_11580_b200 as obc
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    R, d = W.shape
    begin, count = row_range(R, world, rank)
    dev = W.device
    H = torch.empty(d, d, dtype=torch.float32, device=dev)
    obc.obc_hessian(X, H, prec=prec)
    Hinv, info = obc.obc_hessian_inverse(H, damp_rel)
    # Per-rank buffers hold the LOCAL rows only (the weight trace is count x (d+1) x d, not R x ...): the rank's row
    # range is handed to the library as a layer of `count` rows of its own, which rows being independent allows.
    Wl = W[begin:begin + count]
    order_l = torch.zeros(count, d, dtype=torch.int32, device=dev)
    loss_l = torch.zeros(count, d, dtype=torch.float32, device=dev)
    status = torch.zeros(count, dtype=torch.int32, device=dev)
    trace = torch.empty(count, d + 1, d, dtype=torch.float32, device=dev) if (keep_trace and count) else None
    if count:
        obc.obc_prune_trace(Wl, Hinv, order_l, loss_l, status, w_trace=trace)
    if world > 1:
        loss, order = gather_traces(loss_l, order_l, R, group)
    else:
        loss, order = loss_l, order_l
    out = {"row_begin": begin, "row_count": count, "info": info, "status": status, "counts": [], "masks": [], "weights": []}
    for sp in sparsities:
        k = int(round(float(sp) * R * d))
        counts = torch.zeros(R, dtype=torch.int32, device=dev)
        mask = torch.zeros(R, d, dtype=torch.uint8, device=dev)
        obc.obc_select_global_mask(loss, order, k, counts, mask)
        What = torch.zeros(count, d, dtype=torch.float32, device=dev)
        if count:
            obc.obc_prune_apply(Wl, Hinv, order_l, counts[begin:begin + count], What, status, w_trace=trace,
                                trace_steps=d if keep_trace else 0)
        out["counts"].append(counts); out["masks"].append(mask); out["weights"].append(What)
    return out
