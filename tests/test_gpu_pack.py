"""GPU parity of the bit-packed export and the packed inference lookup (paper Appendix C)
against the CPU oracle: packed bytes bit-exact; packed lookups bit-equal to the oracle's packed
lookup and to the training forward of the CUDA path on the same weights and scales."""
from dataclasses import replace

import numpy as np
import pytest

from dqrm_inputs import workloads as W
from gpu_util import Case, bit_equal

pytestmark = pytest.mark.gpu


def _cases():
    kg, tb, mh = W.kaggle(), W.terabyte(), W.multihot()
    return {
        "tiny": W.tiny(),
        "kaggle_small": W.scaled_down(kg, total_rows=300_000, B=2048, name="kaggle_small"),
        "terabyte_small": W.scaled_down(tb, total_rows=400_000, B=1500, name="terabyte_small"),
        "multihot_small": W.scaled_down(mh, total_rows=26 * 3000, B=300, name="multihot_small"),
        "odd_d20": replace(W.scaled_down(kg, total_rows=50_000, B=333), D=20, name="odd_d20"),
        "d4": W.Workload("d4", (5, 1, 1000), D=4, B=64, alpha=1.05, bits=4),
        "wide_d384": W.Workload("wide_d384", (700, 90, 5000), D=384, B=257, alpha=1.1, bits=8),
    }


CASES = _cases()


@pytest.fixture(scope="module", params=sorted(CASES))
def case(request):
    c = Case(CASES[request.param])
    c.tables_np = W.tables_np(c.wl)
    yield c
    c.ctx.close()


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("stale", [False, True])
def test_pack_and_packed_lookup(case, oracle, bits, stale):
    t = case.torch
    wl = case.wl
    b = np.full(wl.T, bits, dtype=np.int32)
    scales, _ = oracle.scale_refresh(case.tables_np, case.row_off, wl.D, b)
    if stale:
        scales = (scales * np.float32(0.41)).astype(np.float32)     # the clamp is live
    want_packed = oracle.pack_tables(case.tables_np, case.row_off, wl.D, scales, bits)

    d_tables, d_scales = case.dev(case.tables_np), case.dev(scales)
    nbytes = case.ctx.packed_bytes(bits)
    assert nbytes == want_packed.size
    guard = 64
    d_packed = t.full((nbytes + guard,), 0xA5, dtype=t.uint8, device="cuda")
    case.ctx.pack_tables(d_tables, d_scales, bits, d_packed)
    case.ctx.raise_on_device_error()
    got = d_packed.cpu().numpy()
    assert (got[nbytes:] == 0xA5).all()
    assert bit_equal(got[:nbytes].reshape(want_packed.shape), want_packed)

    idx, off, _ = case.batch(0)
    L = len(idx)
    out = case.empty((wl.B, wl.T, wl.D), t.float32)
    case.ctx.packed_fwd(d_packed, case.dev(idx), case.dev(off), d_scales, bits, out, B=wl.B, L=L)
    case.ctx.raise_on_device_error()
    want = oracle.packed_fwd(want_packed, case.row_off, wl.D, wl.B, idx, off, scales, bits)
    assert bit_equal(out.cpu().numpy(), want)

    # the training forward of the CUDA path (same bag order, same FP64 accumulator) gives the same bits
    out2 = case.empty((wl.B, wl.T, wl.D), t.float32)
    case.ctx.emb_fwd(d_tables, case.dev(idx), case.dev(off), d_scales, case.dev(b), out2, None, B=wl.B, L=L)
    case.ctx.raise_on_device_error()
    assert bit_equal(out2.cpu().numpy(), out.cpu().numpy())


def test_packed_lookup_reports_bad_index(oracle):
    import paper_2410_20046_b200 as dq

    c = Case(W.tiny())
    t = c.torch
    wl = c.wl
    tables = W.tables_np(wl)
    scales, _ = oracle.scale_refresh(tables, c.row_off, wl.D, np.full(wl.T, 4, dtype=np.int32))
    d_scales = c.dev(scales)
    d_packed = t.zeros(c.ctx.packed_bytes(4), dtype=t.uint8, device="cuda")
    c.ctx.pack_tables(c.dev(tables), d_scales, 4, d_packed)
    idx, off, _ = c.batch(0)
    idx = idx.copy()
    idx[3] = 1 << 30
    out = c.empty((wl.B, wl.T, wl.D), t.float32)
    c.ctx.packed_fwd(d_packed, c.dev(idx), c.dev(off), d_scales, 4, out, B=wl.B, L=len(idx))
    with pytest.raises(dq.DqrmError):
        c.ctx.raise_on_device_error()
    c.ctx.close()


def test_pack_rejects_unsupported_width():
    import paper_2410_20046_b200 as dq

    c = Case(W.tiny())
    t = c.torch
    assert c.ctx.packed_bytes(3) == 0
    with pytest.raises(dq.DqrmError):
        c.ctx.pack_tables(c.empty((c.wl.total_rows, c.wl.D), t.float32), c.empty(c.wl.T, t.float32), 3,
                          c.empty(16, t.uint8))
    c.ctx.close()


def test_packed_lookup_uneven_bags_with_one_index_per_bag_on_average(oracle):
    # L == T*B sends the call down the one-index path; bags of zero and two indices must still pool right
    wl = W.scaled_down(W.kaggle(), total_rows=20_000, B=200, name="uneven")
    c = Case(wl)
    t = c.torch
    tables = W.tables_np(wl)
    scales, _ = oracle.scale_refresh(tables, c.row_off, wl.D, np.full(wl.T, 4, dtype=np.int32))
    idx, off, _ = c.batch(0)
    assert len(idx) == wl.T * wl.B
    off = off.copy()
    rng = np.random.default_rng(3)
    for g in rng.choice(np.arange(1, wl.T * wl.B - 1), size=150, replace=False):
        if g % wl.B:                       # keep each table's range: only move boundaries inside a table
            off[g] += 1 if off[g + 1] - off[g] >= 1 and g % 2 else 0
    off = np.minimum.accumulate(off[::-1])[::-1].astype(np.int32)
    packed = oracle.pack_tables(tables, c.row_off, wl.D, scales, 4)
    want = oracle.packed_fwd(packed, c.row_off, wl.D, wl.B, idx, off, scales, 4)
    lens = np.diff(off)
    assert (lens == 0).any() and (lens == 2).any()
    out = c.empty((wl.B, wl.T, wl.D), t.float32)
    c.ctx.packed_fwd(c.dev(packed), c.dev(idx), c.dev(off), c.dev(scales), 4, out, B=wl.B, L=len(idx))
    c.ctx.raise_on_device_error()
    assert bit_equal(out.cpu().numpy(), want)
    c.ctx.close()
