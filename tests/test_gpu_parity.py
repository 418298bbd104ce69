"""GPU parity: every call of the C ABI against the CPU oracle on the same seeded inputs.

Bars: integer outputs (weight codes, gradient codes, unique rows, offsets) and scales are
bit-exact; FP32 sums (pooled outputs, summed gradients) are within 1e-5 relative / 1e-6
absolute; the update, fed identical inputs, is bit-exact."""
from dataclasses import replace

import numpy as np
import pytest

from dqrm_inputs import workloads as W
from gpu_util import Case, assert_close_fp32, bit_equal

pytestmark = pytest.mark.gpu


def _cases():
    kg = W.kaggle()
    tb = W.terabyte()
    mh = W.multihot()
    return {
        "tiny": W.tiny(),
        # 26 tables, feature 16, 53,248 lookups = 26 sort tiles, the last one ragged
        "kaggle_small": W.scaled_down(kg, total_rows=300_000, B=2048, name="kaggle_small"),
        # feature 64, 26 * 1500 = 39,000 lookups: ragged tile and ragged 32-entry chunk
        "terabyte_small": W.scaled_down(tb, total_rows=400_000, B=1500, name="terabyte_small"),
        # multi-hot, duplicate heavy (Zipf 1.2 over 3000 rows, ~20 per bag)
        "multihot_small": W.scaled_down(mh, total_rows=26 * 3000, B=300, name="multihot_small"),
        "sweep_d16_b2_uniform": W.sweep(D=16, bits=2, zipf=False, rows=200_000, B=5000),
        "sweep_d32_b4_zipf": W.sweep(D=32, bits=4, zipf=True, rows=200_000, B=5000),
        "sweep_d64_b8_uniform": W.sweep(D=64, bits=8, zipf=False, rows=100_000, B=3000),
        "sweep_d128_b8_zipf": W.sweep(D=128, bits=8, zipf=True, rows=50_000, B=3000),
        # one table with enough lookups for the sixteen-block sort cluster; 20,000 is no multiple of 16 * 32
        "sweep_d16_b4_zipf_wide": W.sweep(D=16, bits=4, zipf=True, rows=300_000, B=20_000),
        # feature sizes that are not a power of two / need several vectors per lane
        "odd_d20": replace(W.scaled_down(kg, total_rows=50_000, B=333), D=20, name="odd_d20"),
        "wide_d384": W.Workload("wide_d384", (700, 90, 5000), D=384, B=257, alpha=1.1, bits=8),
        "one_row_tables": W.Workload("one_row_tables", (1, 1, 7, 1), D=16, B=100, alpha=1.05, bits=4),
        # a one-row table whose 6000 lookups span all blocks of its sort cluster and three 2048-entry tiles,
        # with other tables behind it (their unique rows must not shift)
        "one_row_wide": W.Workload("one_row_wide", (1, 3000, 1, 50), D=16, B=6000, alpha=1.05, bits=4),
    }


CASES = _cases()


@pytest.fixture(scope="module", params=sorted(CASES))
def case(request):
    c = Case(CASES[request.param])
    c.tables_np = W.tables_np(c.wl)
    yield c
    c.ctx.close()


def test_scale_refresh_bit_exact(case, oracle):
    d_tables = case.dev(case.tables_np)
    scales, minmax = case.gpu_refresh(d_tables)
    o_scales, o_minmax = oracle.scale_refresh(case.tables_np, case.row_off, case.wl.D, case.bits_np)
    assert bit_equal(scales.cpu().numpy(), o_scales)
    assert (minmax.cpu().numpy() == o_minmax).all()


def test_scale_refresh_extreme_positions(case, oracle):
    # plant the extreme at the first / last element of each table and mid-arena
    tables = case.tables_np.copy()
    off = case.row_off
    rng = np.random.default_rng(5)
    for t in range(case.wl.T):
        flat = tables[off[t]:off[t + 1]].reshape(-1)
        pos = [0, flat.size - 1, int(rng.integers(flat.size))][t % 3]
        flat[pos] = (-1) ** t * (3.0 + t)
    scales, minmax = case.gpu_refresh(case.dev(tables))
    o_scales, o_minmax = oracle.scale_refresh(tables, off, case.wl.D, case.bits_np)
    assert bit_equal(scales.cpu().numpy(), o_scales)
    assert (minmax.cpu().numpy() == o_minmax).all()


@pytest.mark.parametrize("step", [0, 1])
def test_forward(case, oracle, step):
    idx, off, _ = case.batch(step)
    o_scales, _ = oracle.scale_refresh(case.tables_np, case.row_off, case.wl.D, case.bits_np)
    if step == 1:
        o_scales = (o_scales * np.float32(0.37)).astype(np.float32)   # stale scale: clamp is live
    want_codes = case.wl.bits <= 8
    out, codes = case.gpu_fwd(case.dev(case.tables_np), idx, off, case.dev(o_scales), want_codes)
    if want_codes:
        o_out, o_codes = oracle.emb_fwd(case.tables_np, case.row_off, case.wl.D, case.wl.B, idx, off, o_scales,
                                        case.bits_np, want_codes=True)
        assert bit_equal(codes, o_codes)
    else:
        o_out = oracle.emb_fwd(case.tables_np, case.row_off, case.wl.D, case.wl.B, idx, off, o_scales, case.bits_np)
    assert_close_fp32(out, o_out, "pooled output")
    # same order, same FP64 accumulator: expected to agree to the bit
    assert bit_equal(out, o_out)


@pytest.mark.parametrize("step", [0, 2])
def test_backward(case, oracle, step):
    idx, off, go = case.batch(step)
    ur, uo, gr = case.gpu_bwd(idx, off, go)
    o_ur, o_uo, o_gr = oracle.emb_bwd(go, case.wl.T, case.wl.D, case.wl.B, idx, off)
    assert bit_equal(uo, o_uo)
    assert bit_equal(ur, o_ur)
    assert_close_fp32(gr, o_gr, "summed gradients")
    # determinism: a second run gives the same bits
    ur2, uo2, gr2 = case.gpu_bwd(idx, off, go)
    assert bit_equal(gr, gr2) and bit_equal(ur, ur2) and bit_equal(uo, uo2)
    # FP64 accumulation makes the rounded sums equal the oracle's except for double-rounding ties
    mism = int((gr.view(np.int32) != o_gr.view(np.int32)).sum())
    assert mism <= max(1, gr.size // 100_000), f"{mism} of {gr.size} summed gradients differ in the last bit"


def test_grad_quant_and_update_bit_exact(case, oracle):
    idx, off, go = case.batch(3)
    o_ur, o_uo, o_gr = oracle.emb_bwd(go, case.wl.T, case.wl.D, case.wl.B, idx, off)
    codes, gs = case.gpu_quant(o_gr, o_uo)
    o_codes, o_gs = oracle.grad_quant_int8(o_gr, o_uo, case.wl.D)
    assert bit_equal(gs, o_gs)
    assert bit_equal(codes, o_codes)
    d_tables = case.dev(case.tables_np)
    case.gpu_update(d_tables, o_ur, o_uo, o_codes, o_gs, case.wl.lr)
    o_tables = case.tables_np.copy()
    oracle.row_update(o_tables, case.row_off, case.wl.D, o_ur, o_uo, o_codes, o_gs, case.wl.lr)
    assert bit_equal(d_tables.cpu().numpy(), o_tables)


def test_train_step_equals_separate_calls_and_oracle(case, oracle):
    import torch

    wl = case.wl
    idx, off, go = case.batch(4)
    L = len(idx)
    o_tables = case.tables_np.copy()
    o_scales, _ = oracle.scale_refresh(o_tables, case.row_off, wl.D, case.bits_np)
    r = oracle.train_step(o_tables, case.row_off, wl.D, wl.B, idx, off, go, o_scales, case.bits_np, wl.lr)
    d_tables = case.dev(case.tables_np)
    out = case.empty((wl.B, wl.T, wl.D), torch.float32)
    ur = case.empty(max(L, 1), torch.int32)
    uo = case.empty(wl.T + 1, torch.int32)
    gr = case.empty((max(L, 1), wl.D), torch.float32)
    codes = case.empty((max(L, 1), wl.D), torch.int8)
    gs = case.empty(wl.T, torch.float32)
    case.ctx.train_step(d_tables, case.dev(idx), case.dev(off), case.dev(go), case.dev(o_scales), case.bits, out,
                        ur, uo, gr, codes, gs, wl.lr, B=wl.B, L=L)
    case.ctx.raise_on_device_error()
    U = int(r["uniq_off"][-1])
    assert bit_equal(uo.cpu().numpy(), r["uniq_off"])
    assert bit_equal(ur.cpu().numpy()[:U], r["unique_rows"])
    assert bit_equal(out.cpu().numpy(), r["out"])
    assert_close_fp32(gr.cpu().numpy()[:U], r["grad_rows"])
    if bit_equal(gr.cpu().numpy()[:U], r["grad_rows"]):
        assert bit_equal(gs.cpu().numpy(), r["grad_scales"])
        assert bit_equal(codes.cpu().numpy()[:U], r["codes"])
        assert bit_equal(d_tables.cpu().numpy(), o_tables)
    else:
        assert_close_fp32(d_tables.cpu().numpy(), o_tables, "updated weights")


def test_backward_sort_paths_agree(case, oracle):
    """The per-table cluster sort (default) and the global radix sort give the same bits."""
    idx, off, go = case.batch(5)
    case.ctx.set_sort_path(0)
    ur0, uo0, gr0 = case.gpu_bwd(idx, off, go)
    case.ctx.set_sort_path(1)
    try:
        ur1, uo1, gr1 = case.gpu_bwd(idx, off, go)
    finally:
        case.ctx.set_sort_path(0)
    assert bit_equal(ur0, ur1) and bit_equal(uo0, uo1) and bit_equal(gr0, gr1)
    o_ur, o_uo, o_gr = oracle.emb_bwd(go, case.wl.T, case.wl.D, case.wl.B, idx, off)
    assert bit_equal(ur1, o_ur) and bit_equal(uo1, o_uo)
    assert_close_fp32(gr1, o_gr)


def test_tiny_trajectory_100_steps_with_periodic_refresh(oracle):
    """The Tiny configuration end to end: 100 iterations, scale refresh every 10, GPU and oracle
    running free (no resynchronisation).  Integer outputs and scales must agree bit for bit at
    every step; a code may differ only where the oracle's pre-rounding quotient lies within 1e-4
    of a rounding boundary (a last-bit difference of an FP64-accumulated sum), and none is expected."""
    import torch

    wl = W.tiny()
    c = Case(wl)
    o_tables = W.tables_np(wl)
    d_tables = c.dev(o_tables)
    L = wl.T * wl.B
    out = c.empty((wl.B, wl.T, wl.D), torch.float32)
    ur = c.empty(L, torch.int32)
    uo = c.empty(wl.T + 1, torch.int32)
    gr = c.empty((L, wl.D), torch.float32)
    codes = c.empty((L, wl.D), torch.int8)
    gs = c.empty(wl.T, torch.float32)
    scales = c.empty(wl.T, torch.float32)
    o_scales = None
    flips = 0
    for step in range(wl.iters):
        if step % wl.period == 0:
            c.ctx.scale_refresh(d_tables, c.bits, scales)
            o_scales, _ = oracle.scale_refresh(o_tables, c.row_off, wl.D, c.bits_np)
            assert bit_equal(scales.cpu().numpy(), o_scales), f"step {step}: scales"
        idx, off, go = c.batch(step)
        c.ctx.train_step(d_tables, c.dev(idx), c.dev(off), c.dev(go), scales, c.bits, out, ur, uo, gr, codes, gs,
                         wl.lr, B=wl.B, L=len(idx))
        r = oracle.train_step(o_tables, c.row_off, wl.D, wl.B, idx, off, go, o_scales, c.bits_np, wl.lr)
        U = int(r["uniq_off"][-1])
        assert bit_equal(uo.cpu().numpy(), r["uniq_off"]), f"step {step}"
        assert bit_equal(ur.cpu().numpy()[:U], r["unique_rows"]), f"step {step}"
        assert_close_fp32(out.cpu().numpy(), r["out"], f"step {step}: pooled output")
        assert_close_fp32(gr.cpu().numpy()[:U], r["grad_rows"], f"step {step}: summed gradients")
        assert bit_equal(gs.cpu().numpy(), r["grad_scales"]), f"step {step}: gradient scales"
        diff = codes.cpu().numpy()[:U] != r["codes"]
        if diff.any():
            t_of = np.searchsorted(r["uniq_off"], np.nonzero(diff)[0], side="right") - 1
            q = r["grad_rows"][diff] / r["grad_scales"][t_of]
            assert (np.abs(np.abs(q - np.floor(q)) - 0.5) < 1e-4).all(), f"step {step}: unexplained code flips"
            flips += int(diff.sum())
    c.ctx.raise_on_device_error()
    assert_close_fp32(d_tables.cpu().numpy(), o_tables, "weights after 100 steps")
    assert flips == 0, f"{flips} explained code flips (expected none)"
    assert bit_equal(d_tables.cpu().numpy(), o_tables)
    c.ctx.close()


# ---------------------------------------------------------------------------
# edge cases and error paths of the ABI
# ---------------------------------------------------------------------------
def _mini():
    return W.Workload("mini", (50, 7, 300), D=16, B=64, alpha=1.1, bits=4)


def test_alternating_empty_and_double_bags_with_L_equal_G(oracle):
    """L == T*B selects the one-index forward kernel; bags of 0 and 2 indices must still pool right."""
    wl = _mini()
    c = Case(wl)
    tables = W.tables_np(wl)
    idx, _, go = c.batch(0)                                   # L = T*B indices
    lens = np.tile(np.array([0, 2], dtype=np.int64), wl.T * wl.B // 2)
    off = np.zeros(wl.T * wl.B + 1, dtype=np.int32)
    off[1:] = np.cumsum(lens)
    o_scales, _ = oracle.scale_refresh(tables, c.row_off, wl.D, c.bits_np)
    out, _ = c.gpu_fwd(c.dev(tables), idx, off, c.dev(o_scales), want_codes=False)
    o_out = oracle.emb_fwd(tables, c.row_off, wl.D, wl.B, idx, off, o_scales, c.bits_np)
    assert bit_equal(out, o_out)
    ur, uo, gr = c.gpu_bwd(idx, off, go)
    o_ur, o_uo, o_gr = oracle.emb_bwd(go, wl.T, wl.D, wl.B, idx, off)
    assert bit_equal(ur, o_ur) and bit_equal(uo, o_uo)
    assert_close_fp32(gr, o_gr)
    c.ctx.close()


def test_all_bags_empty(oracle):
    import torch

    wl = _mini()
    c = Case(wl)
    tables = W.tables_np(wl)
    off = np.zeros(wl.T * wl.B + 1, dtype=np.int32)
    idx = np.zeros(0, dtype=np.int32)
    go = W.grad_out_np(wl, 0)
    o_scales, _ = oracle.scale_refresh(tables, c.row_off, wl.D, c.bits_np)
    out, _ = c.gpu_fwd(c.dev(tables), idx, off, c.dev(o_scales), want_codes=False)
    assert not out.any()
    ur, uo, gr = c.gpu_bwd(idx, off, go)
    assert len(ur) == 0 and not uo.any()
    d_tables = c.dev(tables)
    gs = c.empty(wl.T, torch.float32)
    one = c.empty(1, torch.int32)
    c.ctx.train_step(d_tables, one, c.dev(off), c.dev(go), c.dev(o_scales), c.bits,
                     c.empty((wl.B, wl.T, wl.D), torch.float32), one, c.empty(wl.T + 1, torch.int32),
                     c.empty((1, wl.D), torch.float32), c.empty((1, wl.D), torch.int8), gs, wl.lr, B=wl.B, L=0)
    c.ctx.raise_on_device_error()
    assert bit_equal(d_tables.cpu().numpy(), tables)                       # nothing touched, nothing updated
    assert (gs.cpu().numpy() == oracle.scale_from_absmax(0.0, 8)).all()    # scale of an empty gradient
    c.ctx.close()


def test_out_of_range_index_is_reported_not_trapped(oracle):
    import paper_2410_20046_b200 as dq

    wl = _mini()
    c = Case(wl)
    tables = W.tables_np(wl)
    idx, off, go = c.batch(0)
    o_scales, _ = oracle.scale_refresh(tables, c.row_off, wl.D, c.bits_np)
    bad = idx.copy()
    bad[3] = wl.rows[0] + 5                   # beyond table 0
    bad[wl.B + 1] = -2                        # negative, table 1
    for call in ("fwd", "bwd"):
        if call == "fwd":
            with pytest.raises(dq.DqrmError) as e:
                c.gpu_fwd(c.dev(tables), bad, off, c.dev(o_scales), want_codes=False)
        else:
            with pytest.raises(dq.DqrmError) as e:
                c.gpu_bwd(bad, off, go)
        assert e.value.status == dq.ERR_INDEX_RANGE
        assert c.ctx.check_status() == dq.OK                 # the report cleared the status word
    # the context is still usable and correct
    out, _ = c.gpu_fwd(c.dev(tables), idx, off, c.dev(o_scales), want_codes=False)
    assert bit_equal(out, oracle.emb_fwd(tables, c.row_off, wl.D, wl.B, idx, off, o_scales, c.bits_np))
    c.ctx.close()


@pytest.mark.parametrize("sort_path", [0, 1])
def test_decreasing_offsets_are_reported_not_followed(oracle, sort_path):
    """Offsets that decrease inside a table are an error the device reports; nothing is read or written
    out of bounds and the context stays usable."""
    import paper_2410_20046_b200 as dq

    wl = W.Workload("mini_bags", (50, 7, 300), D=16, B=64, alpha=1.1, bits=4, bag_mean=3.0, bag_max=6)
    c = Case(wl)
    idx, off, go = c.batch(0)
    bad = off.copy()
    g = wl.B + 5                                  # a bag inside table 1
    bad[g], bad[g + 1] = off[g + 1], off[g]       # (only a decrease when that bag is not empty)
    assert bad[g] > bad[g + 1]
    c.ctx.set_sort_path(sort_path)
    with pytest.raises(dq.DqrmError) as e:
        c.gpu_bwd(idx, bad, go)
    assert e.value.status == dq.ERR_INDEX_RANGE
    assert c.ctx.check_status() == dq.OK
    ur, uo, gr = c.gpu_bwd(idx, off, go)          # still usable and correct
    o_ur, o_uo, o_gr = oracle.emb_bwd(go, wl.T, wl.D, wl.B, idx, off)
    assert bit_equal(ur, o_ur) and bit_equal(uo, o_uo)
    assert_close_fp32(gr, o_gr)
    c.ctx.close()


def test_table_boundary_beyond_the_lookups_is_reported_and_nothing_is_summed(oracle):
    """A table whose first offset points past the batch's lookups cannot be sorted at all: its cluster says so,
    the summation then touches nothing and reports zero unique rows, and the context stays usable."""
    import paper_2410_20046_b200 as dq

    wl = W.Workload("mini_bags", (50, 7, 300), D=16, B=64, alpha=1.1, bits=4, bag_mean=3.0, bag_max=6)
    c = Case(wl)
    idx, off, go = c.batch(0)
    bad = off.copy()
    bad[wl.B] = len(idx) + 3                      # where table 1 begins
    c.ctx.set_sort_path(0)
    L = len(idx)
    ur = c.torch.full((L,), -1, dtype=c.torch.int32, device="cuda")
    uo = c.torch.full((wl.T + 1,), -1, dtype=c.torch.int32, device="cuda")
    gr = c.torch.full((L, wl.D), 7.0, dtype=c.torch.float32, device="cuda")
    c.ctx.emb_bwd(c.dev(go), c.dev(idx), c.dev(bad), ur, uo, gr, B=wl.B, L=L)
    with pytest.raises(dq.DqrmError) as e:
        c.ctx.raise_on_device_error()
    assert e.value.status == dq.ERR_INDEX_RANGE
    assert (uo.cpu().numpy() == 0).all()
    assert (gr.cpu().numpy() == 7.0).all() and (ur.cpu().numpy() == -1).all()
    assert c.ctx.check_status() == dq.OK
    g_ur, g_uo, g_gr = c.gpu_bwd(idx, off, go)    # still usable and correct
    o_ur, o_uo, o_gr = oracle.emb_bwd(go, wl.T, wl.D, wl.B, idx, off)
    assert bit_equal(g_ur, o_ur) and bit_equal(g_uo, o_uo)
    assert_close_fp32(g_gr, o_gr)
    c.ctx.close()


def test_bad_arguments_are_refused_on_the_host():
    import ctypes
    import torch
    import paper_2410_20046_b200 as dq

    wl = _mini()
    c = Case(wl)
    lib = c.ctx.lib
    t = c.empty((wl.total_rows, wl.D), torch.float32)
    i32 = c.empty(wl.T * wl.B + 1, torch.int32)
    f32 = c.empty((wl.B, wl.T, wl.D), torch.float32)
    st = torch.cuda.current_stream().cuda_stream
    # null output pointer
    assert lib.dqrm_emb_fwd(c.ctx._h, t.data_ptr(), i32.data_ptr(), i32.data_ptr(), f32.data_ptr(), c.bits.data_ptr(),
                            None, None, wl.B, wl.T * wl.B, st) == dq.ERR_INVALID_ARG
    # negative batch
    assert lib.dqrm_emb_fwd(c.ctx._h, t.data_ptr(), i32.data_ptr(), i32.data_ptr(), f32.data_ptr(), c.bits.data_ptr(),
                            f32.data_ptr(), None, -1, 10, st) == dq.ERR_INVALID_ARG
    # workspace too small / misaligned
    args = (c.ctx._h, f32.data_ptr(), i32.data_ptr(), i32.data_ptr(), i32.data_ptr(), i32.data_ptr(), f32.data_ptr(),
            wl.B, wl.T * wl.B)
    assert lib.dqrm_emb_bwd(*args, c.ctx._ws_ptr, 1024, st) == dq.ERR_WORKSPACE
    assert lib.dqrm_emb_bwd(*args, c.ctx._ws_ptr + 8, c.ctx.workspace_bytes - 8, st) == dq.ERR_WORKSPACE
    assert lib.dqrm_emb_bwd(*args, None, c.ctx.workspace_bytes, st) == dq.ERR_WORKSPACE
    torch.cuda.synchronize()
    c.ctx.close()
