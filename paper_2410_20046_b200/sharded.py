"""Table-sharded (hybrid-parallel) embedding step: whole tables per rank, the samples' indices go
to the tables' owners, the owners send the looked-up rows back as bit-packed b-bit codes (the
all-to-all payload the paper's Section 4.3 remark is about: 32/b times smaller than FP32 vectors),
the upstream gradient returns to the owners, and backward, INT8 gradient quantisation and update
are local to the owner.  Refresh, unique, quantise and update need no communication.

This module is host-side plumbing only: the plan, the three exchanges and the call order.  All
arithmetic runs in the CUDA library (``GpuShardCompute``).  One index per bag (the Criteo shape).
"""
from __future__ import annotations

from typing import Callable, List, Sequence, Tuple


def plan_tables(rows: Sequence[int], world: int) -> List[Tuple[int, int]]:
    """Contiguous blocks of tables, one per rank, balanced by row count (greedy prefix cut).
    Every rank gets at least one table when there are at least `world` tables."""
    T = len(rows)
    assert world >= 1 and T >= world, "need at least one table per rank"
    total = float(sum(rows))
    plan, t0, acc = [], 0, 0.0
    for r in range(world):
        remaining_ranks = world - r
        if remaining_ranks == 1:
            t1 = T
        else:
            target = total * (r + 1) / world
            t1 = t0 + 1
            acc += rows[t0]
            while t1 < T - (remaining_ranks - 1) and acc + rows[t1] / 2.0 <= target:
                acc += rows[t1]
                t1 += 1
        plan.append((t0, t1))
        t0 = t1
    return plan


class P2PExchange:
    """send[q] goes to rank q, the result holds what every rank sent here (torch.distributed
    point-to-point, so it runs on NCCL and on gloo alike).  Shapes are known on both sides."""

    def __init__(self, group=None):
        import torch.distributed as dist

        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def __call__(self, send, recv_like):
        import torch

        recv = [torch.empty_like(x) for x in recv_like]
        recv[self.rank].copy_(send[self.rank])
        ops = []
        for q in range(self.world):
            if q != self.rank:
                ops.append(self.dist.P2POp(self.dist.isend, send[q].contiguous(), q, self.group))
                ops.append(self.dist.P2POp(self.dist.irecv, recv[q], q, self.group))
        if ops:
            for w in self.dist.batch_isend_irecv(ops):
                w.wait()
        return recv


class GpuShardCompute:
    """The owner-side and receiver-side calls of one rank on its GPU, through the C ABI."""

    def __init__(self, local_rows: Sequence[int], D: int, global_batch: int, bits: int, lr: float):
        import torch
        import numpy as np
        from . import binding

        self.torch = torch
        self.Tp, self.D, self.Bg, self.bits, self.lr = len(local_rows), D, global_batch, bits, lr
        row_off = np.zeros(self.Tp + 1, dtype=np.int64)
        row_off[1:] = np.cumsum(np.asarray(local_rows, dtype=np.int64))
        self.row_off = row_off
        G = self.Tp * self.Bg
        self.ctx = binding.Context(row_off, D, G, G)
        dev = "cuda"
        self.offsets = torch.arange(G + 1, dtype=torch.int32, device=dev)          # one index per bag
        self.bits_t = torch.full((self.Tp,), bits, dtype=torch.int32, device=dev)
        self.scales = torch.empty(self.Tp, dtype=torch.float32, device=dev)
        self.unique_rows = torch.empty(max(G, 1), dtype=torch.int32, device=dev)
        self.uniq_off = torch.empty(self.Tp + 1, dtype=torch.int32, device=dev)
        self.grad_rows = torch.empty((max(G, 1), D), dtype=torch.float32, device=dev)
        self.codes = torch.empty((max(G, 1), D), dtype=torch.int8, device=dev)
        self.grad_scales = torch.empty(self.Tp, dtype=torch.float32, device=dev)
        self.tables = None

    def refresh(self):
        self.ctx.scale_refresh(self.tables, self.bits_t, self.scales)
        return self.scales

    def fwd_codes(self, indices):
        payload = self.torch.empty((self.Bg, self.Tp, self.D * self.bits // 8), dtype=self.torch.uint8, device="cuda")
        self.ctx.emb_fwd_codes(self.tables, indices, self.offsets, self.scales, self.bits, payload, B=self.Bg,
                               L=self.Tp * self.Bg)
        return payload

    def decode(self, block, scales_block, t0, out):
        self.ctx.decode_payload(block, scales_block, self.bits, out, B=block.shape[0], T_blk=block.shape[1],
                                T_total=out.shape[1], t0=t0)

    def bwd_update(self, indices, grad_out):
        L = self.Tp * self.Bg
        self.ctx.emb_bwd(grad_out, indices, self.offsets, self.unique_rows, self.uniq_off, self.grad_rows, B=self.Bg, L=L)
        self.ctx.grad_quant_int8(self.grad_rows, self.uniq_off, self.codes, self.grad_scales)
        self.ctx.row_update(self.tables, self.unique_rows, self.uniq_off, self.codes, self.grad_scales, self.lr)


class TableShardedStep:
    """One rank of the table-sharded step.  `compute` does the arithmetic (GpuShardCompute in the
    product), `exchange(send, recv_like)` moves the blocks (P2PExchange in the product)."""

    def __init__(self, compute, plan: List[Tuple[int, int]], rank: int, B_local: int, D: int, bits: int,
                 exchange: Callable, empty: Callable):
        self.c, self.plan, self.rank, self.world = compute, plan, rank, len(plan)
        self.B, self.D, self.bits, self.exchange, self.empty = B_local, D, bits, exchange, empty
        self.T = plan[-1][1]
        self.t0, self.t1 = plan[rank]
        self.Tp = self.t1 - self.t0
        self.all_scales = None

    def refresh(self):
        """Local whole-table refresh, then every rank learns every table's scale (T floats)."""
        local = self.c.refresh()
        send = [local for _ in range(self.world)]
        like = [self.empty((p1 - p0,), "float32") for p0, p1 in self.plan]
        self.all_scales = self.exchange(send, like)

    def step(self, local_indices, grad_fn):
        """local_indices: [T][B_local] int32 (one index per bag); grad_fn(out [B_local][T][D]) gives this
        rank's upstream gradient.  Returns out."""
        W, B, D, rb = self.world, self.B, self.D, self.D * self.bits // 8
        # 1. indices to the tables' owners; the owner's global batch is rank-major: sample r*B + i
        send = [local_indices[p0:p1] for p0, p1 in self.plan]
        like = [self.empty((self.Tp, B), "int32") for _ in range(W)]
        got = self.exchange(send, like)
        g_idx = self._cat(got, dim=1).reshape(-1)                      # [Tp][W*B] table-major
        # 2. owners gather + quantise + pack; every rank gets its samples' codes of every table
        payload = self.c.fwd_codes(g_idx)                              # [W*B][Tp][rb]
        send = [payload[q * B:(q + 1) * B] for q in range(W)]
        like = [self.empty((B, p1 - p0, rb), "uint8") for p0, p1 in self.plan]
        blocks = self.exchange(send, like)
        # 3. decode with the owners' scales
        out = self.empty((B, self.T, D), "float32")
        for (p0, p1), blk, sc in zip(self.plan, blocks, self.all_scales):
            self.c.decode(blk, sc, p0, out)
        # 4. upstream gradient back to the owners
        grad_out = grad_fn(out)
        send = [grad_out[:, p0:p1, :] for p0, p1 in self.plan]
        like = [self.empty((B, self.Tp, D), "float32") for _ in range(W)]
        g_grad = self._cat(self.exchange(send, like), dim=0)           # [W*B][Tp][D]
        # 5. backward, INT8 gradient quantisation and update, local to the owner
        self.c.bwd_update(g_idx, g_grad)
        return out

    @staticmethod
    def _cat(parts, dim):
        if hasattr(parts[0], "numpy") or type(parts[0]).__module__.startswith("torch"):
            import torch

            return torch.cat([p.contiguous() for p in parts], dim=dim).contiguous()
        import numpy as np

        return np.ascontiguousarray(np.concatenate(parts, axis=dim))
