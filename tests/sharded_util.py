"""Shared pieces of the table-sharded tests: the problem every rank sees, an oracle-backed compute
object (CPU; what the gloo test runs) and the full-problem reference."""
import numpy as np

from dqrm_inputs import workloads as W


def problem(world, B_local, seed_step=0, bits=4):
    """A one-index workload with `world` * B_local samples; rank r owns samples r*B_local ..."""
    wl = W.scaled_down(W.kaggle(), total_rows=40_000, B=world * B_local, name="sharded")
    wl = type(wl)(**{**wl.__dict__, "bits": bits})
    tables = W.tables_np(wl)
    idx, off = W.make_batch(wl, seed_step)                 # table-major [T][Bg]
    go = W.grad_out_np(wl, seed_step)                      # [Bg][T][D]
    return wl, tables, idx.reshape(wl.T, wl.B), off, go


def reference(oracle, wl, tables, idx2d, off, go, bits):
    """Unsharded oracle step on the full problem (refresh first) -> out, updated tables."""
    t = tables.copy()
    b = np.full(wl.T, bits, dtype=np.int32)
    scales, _ = oracle.scale_refresh(t, wl.row_off(), wl.D, b)
    r = oracle.train_step(t, wl.row_off(), wl.D, wl.B, idx2d.reshape(-1), off, go, scales, b, wl.lr)
    return r["out"], t


class OracleShardCompute:
    """The compute interface of sharded.TableShardedStep on the CPU oracle (torch CPU tensors in and out)."""

    def __init__(self, oracle, local_tables, local_rows, D, global_batch, bits, lr):
        import torch

        self.o, self.torch = oracle, torch
        self.tables = np.ascontiguousarray(local_tables)
        self.Tp, self.D, self.Bg, self.bits, self.lr = len(local_rows), D, global_batch, bits, lr
        self.row_off = np.zeros(self.Tp + 1, dtype=np.int64)
        self.row_off[1:] = np.cumsum(local_rows)
        self.offsets = np.arange(self.Tp * self.Bg + 1, dtype=np.int32)
        self.bits_a = np.full(self.Tp, bits, dtype=np.int32)
        self.scales = None

    def refresh(self):
        self.scales, _ = self.o.scale_refresh(self.tables, self.row_off, self.D, self.bits_a)
        return self.torch.from_numpy(self.scales.copy())

    def fwd_codes(self, indices):
        p = self.o.emb_fwd_codes(self.tables, self.row_off, self.D, self.Bg, indices.numpy(), self.offsets, self.scales,
                                 self.bits)
        return self.torch.from_numpy(p)

    def decode(self, block, scales_block, t0, out):
        o = out.numpy()
        self.o.decode_payload(block.contiguous().numpy(), scales_block.numpy(), self.bits, self.D, o.shape[1], t0, out=o)

    def bwd_update(self, indices, grad_out):
        idx = indices.numpy()
        ur, uo, gr = self.o.emb_bwd(grad_out.contiguous().numpy(), self.Tp, self.D, self.Bg, idx, self.offsets)
        U = int(uo[-1])
        ur, gr = ur[:U], gr[:U]
        codes, gs = self.o.grad_quant_int8(gr, uo, self.D)
        self.o.row_update(self.tables, self.row_off, self.D, ur, uo, codes, gs, self.lr)
