"""GPU parity of the scale refresh fed from per-row (min, max) summaries that the update kernels keep current
(Section 3.2 gives the cost this removes: a table's range is found by reading the whole table).  The oracle
always scans the tables; scales and min/max must equal its result bit for bit at every refresh."""
from dataclasses import replace

import numpy as np
import pytest

from dqrm_inputs import workloads as W
from gpu_util import Case, bit_equal

pytestmark = pytest.mark.gpu


def _cases():
    kg = W.kaggle()
    return {
        "tiny": W.tiny(),
        "kaggle_small": W.scaled_down(kg, total_rows=300_000, B=2048, name="kaggle_small"),
        "terabyte_small": W.scaled_down(W.terabyte(), total_rows=200_000, B=700, name="terabyte_small"),
        "odd_d20": replace(W.scaled_down(kg, total_rows=50_000, B=333), D=20, name="odd_d20"),
        "wide_d384": W.Workload("wide_d384", (700, 90, 5000), D=384, B=257, alpha=1.1, bits=8),
        "one_row_tables": W.Workload("one_row_tables", (1, 1, 7, 1), D=16, B=100, alpha=1.05, bits=4),
        "d4": W.Workload("d4", (33, 1000, 5), D=4, B=200, alpha=1.1, bits=4),
        "multihot_small": W.scaled_down(W.multihot(), total_rows=26 * 3000, B=300, name="multihot_small"),
    }


CASES = _cases()


def _row_minmax(tables):
    return np.stack([tables.min(axis=1), tables.max(axis=1)], axis=1)


@pytest.mark.parametrize("name", sorted(CASES))
def test_summary_of_fresh_tables_and_refresh_from_it(name, oracle):
    c = Case(CASES[name])
    tables = W.tables_np(c.wl)
    # plant each table's extremes where a chunked scan would look last: first and last element
    for t in range(c.wl.T):
        flat = tables[c.row_off[t]:c.row_off[t + 1]].reshape(-1)
        flat[0 if t % 2 else flat.size - 1] = (-1) ** t * (2.0 + t)
    d_tables = c.dev(tables)
    summary = c.ctx.row_summary_attach(d_tables)
    assert (summary.cpu().numpy().reshape(-1, 2) == _row_minmax(tables)).all()
    scales, minmax = c.gpu_refresh(d_tables)
    o_scales, o_minmax = oracle.scale_refresh(tables, c.row_off, c.wl.D, c.bits_np)
    assert bit_equal(scales.cpu().numpy(), o_scales)
    assert (minmax.cpu().numpy() == o_minmax).all()
    c.ctx.row_summary_detach()
    scales2, minmax2 = c.gpu_refresh(d_tables)                 # scanning again gives the same
    assert bit_equal(scales2.cpu().numpy(), o_scales) and (minmax2.cpu().numpy() == o_minmax).all()
    c.ctx.close()


@pytest.mark.parametrize("name", sorted(CASES))
def test_trajectory_with_summaries_equals_oracle_with_scans(name, oracle):
    """Twelve steps, refresh every three.  The rows are written in the three ways the library has: the fused step,
    the step in two calls, and separate quantise + update calls.  The learning rate is raised so that the
    tables' ranges really move between refreshes."""
    import torch

    wl = replace(CASES[name], lr=CASES[name].lr * 50.0)
    c = Case(wl)
    o_tables = W.tables_np(wl)
    d_tables = c.dev(o_tables)
    summary = c.ctx.row_summary_attach(d_tables)
    Lmax = c.max_lookups
    out = c.empty((wl.B, wl.T, wl.D), torch.float32)
    ur = c.empty(Lmax, torch.int32)
    uo = c.empty(wl.T + 1, torch.int32)
    gr = c.empty((Lmax, wl.D), torch.float32)
    codes = c.empty((Lmax, wl.D), torch.int8)
    gs = c.empty(wl.T, torch.float32)
    scales = c.empty(wl.T, torch.float32)
    minmax = c.empty((wl.T, 2), torch.float32)
    o_scales = None
    moved = False
    for step in range(12):
        if step % 3 == 0:
            c.ctx.scale_refresh(d_tables, c.bits, scales, minmax)
            new_scales, o_minmax = oracle.scale_refresh(o_tables, c.row_off, wl.D, c.bits_np)
            moved |= o_scales is not None and not bit_equal(new_scales, o_scales)
            o_scales = new_scales
            assert bit_equal(scales.cpu().numpy(), o_scales), f"step {step}: scales"
            assert (minmax.cpu().numpy() == o_minmax).all(), f"step {step}: min/max"
        idx, off, go = c.batch(step)
        L = len(idx)
        d_idx = c.dev(idx) if L else c.empty(1, torch.int32)
        args = (d_tables, d_idx, c.dev(off), c.dev(go), scales, c.bits, out, ur, uo, gr, codes, gs, wl.lr)
        if step % 3 == 0:
            c.ctx.train_step(*args, B=wl.B, L=L)
        elif step % 3 == 1:
            c.ctx.sort_batch(args[1], args[2], ur, uo, B=wl.B, L=L, ws=1)
            c.ctx.train_step_sorted(*args, B=wl.B, L=L, ws=1)
        else:
            c.ctx.emb_fwd(d_tables, d_idx, args[2], scales, c.bits, out, None, B=wl.B, L=L)
            c.ctx.emb_bwd(args[3], d_idx, args[2], ur, uo, gr, B=wl.B, L=L)
            c.ctx.grad_quant_int8(gr, uo, codes, gs)
            c.ctx.row_update(d_tables, ur, uo, codes, gs, wl.lr)
        oracle.train_step(o_tables, c.row_off, wl.D, wl.B, idx, off, go, o_scales, c.bits_np, wl.lr)
    c.ctx.raise_on_device_error()
    assert bit_equal(d_tables.cpu().numpy(), o_tables)
    assert (summary.cpu().numpy().reshape(-1, 2) == _row_minmax(o_tables)).all()
    assert moved or name in ("one_row_tables",), "the scales never changed: the test would not see a stale summary"
    c.ctx.close()
