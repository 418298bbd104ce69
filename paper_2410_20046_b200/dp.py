"""Data-parallel training step of the embedding path (paper Appendix B.1): one process per
GPU, every rank holds all tables and takes its own samples; per step the ranks unify the
gradient quantisation scales (MAX all-reduce of T floats), quantise their sparse gradients to
INT8 with the unified scales, all-gather (rows, codes) and apply the exact integer sum, so
all replicas stay bit-identical.

The two collectives go through ``torch.distributed`` (NCCL over NVLink on GPUs; the same code
runs on CPU tensors with gloo, which is how the plumbing is tested without GPUs).  Everything
else is the CUDA library.  Nothing here computes gradients, codes or updates.
"""
from __future__ import annotations


def unify_absmax(absmax, group=None):
    """MAX all-reduce of the per-table abs-max values (in place); identity for one rank."""
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(absmax, op=dist.ReduceOp.MAX, group=group)
    return absmax


def gather_sparse(rows, uniq_off, codes, group=None):
    """All-gather of every rank's sparse INT8 gradient.

    rows int32 [>= U], uniq_off int32 [T+1], codes int8 [>= U, D] with U = uniq_off[T].
    Returns (rows_cat [W, stride], uoff_cat [W, T+1], codes_cat [W, stride, D], stride, n_entries,
    max_table_entries); stride is the largest U over the ranks (shorter lists are padded, the
    padding is never read)."""
    import torch
    import torch.distributed as dist

    W = dist.get_world_size(group) if (dist.is_available() and dist.is_initialized()) else 1
    T1 = uniq_off.numel()
    D = codes.shape[1]
    uoff_cat = torch.empty((W, T1), dtype=uniq_off.dtype, device=uniq_off.device)
    if W > 1:
        dist.all_gather_into_tensor(uoff_cat.view(-1), uniq_off.contiguous().view(-1), group=group)
    else:
        uoff_cat[0] = uniq_off
    uoff_h = uoff_cat.cpu()                                   # the sizes are needed on the host
    counts = uoff_h[:, -1]
    stride = max(int(counts.max()), 1)
    n_entries = int(counts.sum())
    per_table = (uoff_h[:, 1:] - uoff_h[:, :-1]).sum(dim=0)
    max_table = int(per_table.max()) if per_table.numel() else 0
    U = int(uoff_h[dist.get_rank(group) if W > 1 else 0, -1])
    my_rows = torch.zeros(stride, dtype=rows.dtype, device=rows.device)
    my_codes = torch.zeros((stride, D), dtype=codes.dtype, device=codes.device)
    my_rows[:U] = rows[:U]
    my_codes[:U] = codes[:U]
    rows_cat = torch.empty((W, stride), dtype=rows.dtype, device=rows.device)
    codes_cat = torch.empty((W, stride, D), dtype=codes.dtype, device=codes.device)
    if W > 1:
        dist.all_gather_into_tensor(rows_cat.view(-1), my_rows.view(-1), group=group)
        dist.all_gather_into_tensor(codes_cat.view(-1), my_codes.view(-1), group=group)
    else:
        rows_cat[0] = my_rows
        codes_cat[0] = my_codes
    return rows_cat, uoff_cat, codes_cat, stride, n_entries, max_table


class DataParallelStep:
    """Buffers and call sequence of one rank.  ``ctx`` is a ``Context``; ``max_lookups`` bounds L."""

    def __init__(self, ctx, B, max_lookups, world_size, group=None):
        import torch

        self.ctx, self.B, self.group, self.W = ctx, B, group, world_size
        T, D = ctx.T, ctx.D
        f32, i32, i8 = torch.float32, torch.int32, torch.int8
        self.out = torch.empty((B, T, D), dtype=f32, device="cuda")
        self.unique_rows = torch.empty(max_lookups, dtype=i32, device="cuda")
        self.uniq_off = torch.empty(T + 1, dtype=i32, device="cuda")
        self.grad_rows = torch.empty((max_lookups, D), dtype=f32, device="cuda")
        self.codes = torch.empty((max_lookups, D), dtype=i8, device="cuda")
        self.absmax = torch.empty(T, dtype=f32, device="cuda")
        self.grad_scales = torch.empty(T, dtype=f32, device="cuda")
        self.union_rows = torch.empty(max_lookups * world_size, dtype=i32, device="cuda")
        self.union_off = torch.empty(T + 1, dtype=i32, device="cuda")
        self.ws = ctx.dp_workspace(max_lookups * world_size)

    def step(self, tables, indices, offsets, grad_out, scales, bits, lr, L):
        c = self.ctx
        c.emb_fwd(tables, indices, offsets, scales, bits, self.out, None, B=self.B, L=L)
        c.emb_bwd(grad_out, indices, offsets, self.unique_rows, self.uniq_off, self.grad_rows, B=self.B, L=L)
        c.grad_absmax(self.grad_rows, self.uniq_off, self.absmax)
        unify_absmax(self.absmax, self.group)
        c.grad_quant_int8_unified(self.grad_rows, self.uniq_off, self.absmax, self.codes, self.grad_scales)
        rows_cat, uoff_cat, codes_cat, stride, n, max_table = gather_sparse(self.unique_rows, self.uniq_off, self.codes,
                                                                            self.group)
        c.dp_merge_update(tables, self.W, stride, rows_cat, uoff_cat, codes_cat, self.grad_scales, lr, n, max_table,
                          self.union_rows, self.union_off, None, self.ws)
        return self.out
