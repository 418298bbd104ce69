"""Pins for the oracle's array steps: refresh, forward, backward, gradient
quantiser, update.  Expected values come from hand-built examples, numpy library
routines (min/max/unique/add.at), exact rational sums and dense brute force, not
from the oracle itself."""
from fractions import Fraction

import numpy as np
import pytest

from dqrm_inputs import workloads as W


def f32(x):
    return np.asarray(x, dtype=np.float32)


# ---------------------------------------------------------------------------
# scale refresh: whole-table min/max, one scale per table
# ---------------------------------------------------------------------------
def test_refresh_matches_numpy_minmax(oracle):
    wl = W.tiny()
    tables = W.tables_np(wl)
    off = wl.row_off()
    bits = np.array([4, 8, 2, 16], dtype=np.int32)
    scales, minmax = oracle.scale_refresh(tables, off, wl.D, bits)
    for t in range(wl.T):
        w = tables[off[t]:off[t + 1]]
        assert minmax[t, 0] == w.min() and minmax[t, 1] == w.max()
        a = max(abs(w.min()), abs(w.max()))
        n = np.float32(2 ** (int(bits[t]) - 1) - 1)
        assert scales[t] == np.float32(a) / n


def test_refresh_extremes_at_table_edges_do_not_leak(oracle):
    D = 4
    rows = [3, 5, 2]
    off = np.array([0, 3, 8, 10], dtype=np.int64)
    tables = np.zeros((10, D), dtype=np.float32)
    tables[0, 0] = -7.0          # first element of table 0
    tables[2, 3] = 3.5           # last element of table 0
    tables[3, 0] = 14.0          # first element of table 1
    tables[7, 3] = -2.0          # last element of table 1
    tables[8:10] = 0.25          # all-equal table 2
    scales, minmax = oracle.scale_refresh(tables, off, D, np.array([4, 4, 8], dtype=np.int32))
    assert minmax.tolist() == [[-7.0, 3.5], [-2.0, 14.0], [0.25, 0.25]]
    assert scales.tolist() == [1.0, 2.0, float(np.float32(0.25) / np.float32(127))]


def test_refresh_finds_the_extreme_at_every_position(oracle):
    D, R = 4, 3
    for pos in range(R * D):
        for val in (-9.0, 9.0):
            tables = np.full((2 * R, D), 0.5, dtype=np.float32)
            tables.reshape(-1)[R * D + pos] = val        # inside table 1
            _, minmax = oracle.scale_refresh(tables, np.array([0, R, 2 * R]), D,
                                             np.array([4, 4], dtype=np.int32))
            assert minmax[0].tolist() == [0.5, 0.5]
            assert minmax[1].tolist() == ([val, 0.5] if val < 0 else [0.5, val])


def test_refresh_all_zero_table_uses_floor(oracle):
    tables = np.zeros((6, 4), dtype=np.float32)
    scales, minmax = oracle.scale_refresh(tables, np.array([0, 6]), 4, np.array([4], dtype=np.int32))
    assert minmax.tolist() == [[0.0, 0.0]]
    assert scales[0] == np.float32(1e-8) / np.float32(7)


def test_refresh_negative_only_table(oracle):
    tables = -np.arange(1, 9, dtype=np.float32).reshape(2, 4)
    scales, minmax = oracle.scale_refresh(tables, np.array([0, 2]), 4, np.array([8], dtype=np.int32))
    assert minmax.tolist() == [[-8.0, -1.0]]
    assert scales[0] == np.float32(8.0) / np.float32(127)


# ---------------------------------------------------------------------------
# forward: gather, quantise each row with the table's scale, sum-pool
# ---------------------------------------------------------------------------
def _small_case():
    # T=2 tables (3 and 2 rows), D=4, B=2.  Integer-valued weights and scale 1
    # make the fake-quantiser the identity inside [-8, 7].
    D = 4
    off = np.array([0, 3, 5], dtype=np.int64)
    tables = f32([[1, 2, 3, 4], [-1, -2, -3, -4], [5, 6, 7, -8],      # table 0
                  [0, 1, 0, 1], [2, 2, 2, 2]])                        # table 1
    return D, off, tables


def test_forward_hand_example_layout_and_pooling(oracle):
    D, off, tables = _small_case()
    B = 2
    # table 0: sample 0 -> rows {0, 2}; sample 1 -> row {1}
    # table 1: sample 0 -> {} (empty);  sample 1 -> rows {1, 1, 0}
    indices = np.array([0, 2, 1, 1, 1, 0], dtype=np.int32)
    offsets = np.array([0, 2, 3, 3, 6], dtype=np.int32)
    scales = f32([1.0, 1.0])
    bits = np.array([4, 4], dtype=np.int32)
    out, codes = oracle.emb_fwd(tables, off, D, B, indices, offsets, scales, bits, want_codes=True)
    want = np.zeros((B, 2, D), dtype=np.float32)
    want[0, 0] = [6, 8, 10, -4]
    want[1, 0] = [-1, -2, -3, -4]
    want[0, 1] = [0, 0, 0, 0]
    want[1, 1] = [4, 5, 4, 5]
    assert out.tolist() == want.tolist()
    assert codes.tolist() == [[1, 2, 3, 4], [5, 6, 7, -8], [-1, -2, -3, -4],
                              [2, 2, 2, 2], [2, 2, 2, 2], [0, 1, 0, 1]]


def test_forward_uses_each_tables_own_scale_and_bits(oracle):
    D, off, tables = _small_case()
    indices = np.array([2, 1], dtype=np.int32)       # table 0 row 2, table 1 row 1
    offsets = np.array([0, 1, 2], dtype=np.int32)
    # table 0: scale 2, 4 bits: [5,6,7,-8]/2 = [2.5,3,3.5,-4] -> [2,3,4,-4] -> *2
    # table 1: scale 4, 2 bits: [2,2,2,2]/4 = .5 -> 0
    out = oracle.emb_fwd(tables, off, D, 1, indices, offsets, f32([2.0, 4.0]),
                         np.array([4, 2], dtype=np.int32))
    assert out[0, 0].tolist() == [4, 6, 8, -8]
    assert out[0, 1].tolist() == [0, 0, 0, 0]
    # 2-bit clamp: scale 1 -> codes of [2,2,2,2] clamp to 1
    out = oracle.emb_fwd(tables, off, D, 1, indices, offsets, f32([2.0, 1.0]),
                         np.array([4, 2], dtype=np.int32))
    assert out[0, 1].tolist() == [1, 1, 1, 1]


def test_forward_single_index_bags_equal_elementwise_fake_quant(oracle):
    wl = W.tiny()
    tables = W.tables_np(wl)
    off = wl.row_off()
    bits = np.full(wl.T, 4, dtype=np.int32)
    scales, _ = oracle.scale_refresh(tables, off, wl.D, bits)
    indices, offsets = W.make_batch(wl, 0)
    out, codes = oracle.emb_fwd(tables, off, wl.D, wl.B, indices, offsets, scales, bits, want_codes=True)
    for t in range(wl.T):
        for i in range(0, wl.B, 7):
            row = tables[off[t] + indices[t * wl.B + i]]
            for d in range(wl.D):
                assert codes[t * wl.B + i, d] == oracle.quantize(row[d], scales[t], 4)
                assert out[i, t, d] == oracle.fake_quant(row[d], scales[t], 4)
    assert codes.min() >= -7 and codes.max() <= 7       # fresh scale
    # U(-a, a) values beyond 6.5/7 of the range quantise to +-7; 8192 gathered values hit both
    assert np.abs(codes).max() == 7

def test_forward_bags_against_exact_integer_route(oracle):
    wl = W.scaled_down(W.multihot(), total_rows=26 * 500, B=16, name="mh_small")
    tables = W.tables_np(wl)
    off = wl.row_off()
    bits = np.full(wl.T, 4, dtype=np.int32)
    scales, _ = oracle.scale_refresh(tables, off, wl.D, bits)
    indices, offsets = W.make_batch(wl, 0)
    assert (np.diff(offsets) > 1).any()
    out, codes = oracle.emb_fwd(tables, off, wl.D, wl.B, indices, offsets, scales, bits, want_codes=True)
    for t in range(0, wl.T, 5):
        s = Fraction(float(scales[t]))
        for i in range(wl.B):
            g = t * wl.B + i
            for d in range(0, wl.D, 9):
                # exact: (sum of integer codes) * s, then compare within FP32 rounding of each term
                qsum = sum(int(codes[j, d]) for j in range(offsets[g], offsets[g + 1]))
                exact = float(qsum * s)
                n = offsets[g + 1] - offsets[g]
                tol = n * 7 * float(scales[t]) * 2.0 ** -23 + 1e-12
                assert abs(float(out[i, t, d]) - exact) <= tol


# ---------------------------------------------------------------------------
# backward: lossless sparse gradient on the touched rows
# ---------------------------------------------------------------------------
def _dense_gradient(wl, indices, offsets, grad_out):
    """Brute force: scatter every lookup into a dense zero table, in double."""
    off = wl.row_off()
    dense = np.zeros((wl.total_rows, wl.D), dtype=np.float64)
    for t in range(wl.T):
        for i in range(wl.B):
            g = t * wl.B + i
            for j in range(offsets[g], offsets[g + 1]):
                dense[off[t] + indices[j]] += grad_out[i, t].astype(np.float64)
    return dense


@pytest.mark.parametrize("maker", [
    lambda: W.tiny(),
    lambda: W.scaled_down(W.multihot(), total_rows=26 * 300, B=24, name="mh_small"),
    lambda: W.scaled_down(W.kaggle(), total_rows=20000, B=200, name="kg_small"),
])
def test_backward_equals_dense_bruteforce(oracle, maker):
    wl = maker()
    off = wl.row_off()
    indices, offsets = W.make_batch(wl, 3)
    grad_out = W.grad_out_np(wl, 3)
    unique_rows, uniq_off, grad_rows = oracle.emb_bwd(grad_out, wl.T, wl.D, wl.B, indices, offsets)
    dense = _dense_gradient(wl, indices, offsets, grad_out)
    touched = np.zeros(wl.total_rows, dtype=bool)
    assert uniq_off[0] == 0 and uniq_off[-1] == len(unique_rows)
    for t in range(wl.T):
        lo, hi = offsets[t * wl.B], offsets[(t + 1) * wl.B]
        want_rows = np.unique(indices[lo:hi])                 # sort then deduplicate
        got_rows = unique_rows[uniq_off[t]:uniq_off[t + 1]]
        assert got_rows.tolist() == want_rows.tolist()
        arena = off[t] + got_rows
        touched[arena] = True
        want = dense[arena].astype(np.float32)                # double sum rounded once
        got = grad_rows[uniq_off[t]:uniq_off[t + 1]]
        np.testing.assert_allclose(got, want, rtol=2e-7, atol=1e-30)
    assert not dense[~touched].any()                          # zero everywhere else
    # column sums: nothing lost, nothing double-counted
    total = np.zeros((wl.T, wl.D))
    for t in range(wl.T):
        cnt = np.diff(offsets[t * wl.B:(t + 1) * wl.B + 1]).astype(np.float64)
        total[t] = (grad_out[:, t].astype(np.float64) * cnt[:, None]).sum(0)
        got = grad_rows[uniq_off[t]:uniq_off[t + 1]].astype(np.float64).sum(0)
        np.testing.assert_allclose(got, total[t], rtol=1e-5, atol=1e-5)


def test_backward_hand_example(oracle):
    # T=2, B=3, D=2.  table 0: rows [4, 1, 4]; table 1: bags {2,2}, {}, {0}
    indices = np.array([4, 1, 4, 2, 2, 0], dtype=np.int32)
    offsets = np.array([0, 1, 2, 3, 5, 5, 6], dtype=np.int32)
    grad_out = f32([[[1, 2], [10, 20]],
                    [[3, 4], [30, 40]],
                    [[5, 6], [50, 60]]])          # [B=3][T=2][D=2]
    ur, uo, gr = oracle.emb_bwd(grad_out, 2, 2, 3, indices, offsets)
    assert ur.tolist() == [1, 4, 0, 2]
    assert uo.tolist() == [0, 2, 4]
    assert gr.tolist() == [[3, 4], [6, 8], [50, 60], [20, 40]]


def test_backward_same_row_number_in_two_tables_stays_separate(oracle):
    indices = np.array([7, 7], dtype=np.int32)
    offsets = np.array([0, 1, 2], dtype=np.int32)
    grad_out = f32([[[1, 1], [2, 2]]])
    ur, uo, gr = oracle.emb_bwd(grad_out, 2, 2, 1, indices, offsets)
    assert ur.tolist() == [7, 7] and uo.tolist() == [0, 1, 2]
    assert gr.tolist() == [[1, 1], [2, 2]]


# ---------------------------------------------------------------------------
# INT8 gradient quantiser: per-table abs-max scale, values only
# ---------------------------------------------------------------------------
def test_grad_quant_hand_example(oracle):
    D = 2
    grad_rows = f32([[127, -63.5], [1, 0],            # table 0: absmax 127 -> scale 1
                     [0.5, -0.25], [0.125, 0.5]])     # table 1: absmax 0.5 -> scale 0.5/127
    uniq_off = np.array([0, 2, 4, 4], dtype=np.int32)  # table 2 touched nothing
    codes, gs = oracle.grad_quant_int8(grad_rows, uniq_off, D)
    assert gs[0] == 1.0
    assert gs[1] == np.float32(0.5) / np.float32(127)
    assert gs[2] == np.float32(1e-8) / np.float32(127)
    assert codes[:2].tolist() == [[127, -64], [1, 0]]       # -63.5 is a tie -> even
    assert codes[2].tolist() == [127, -64]                  # 0.25/(0.5/127) = 63.5 -> 64
    assert codes[3].tolist() == [32, 127]                   # 31.75 -> 32


def test_grad_quant_properties(oracle):
    wl = W.tiny()
    indices, offsets = W.make_batch(wl, 1)
    grad_out = W.grad_out_np(wl, 1)
    ur, uo, gr = oracle.emb_bwd(grad_out, wl.T, wl.D, wl.B, indices, offsets)
    codes, gs = oracle.grad_quant_int8(gr, uo, wl.D)
    assert codes.dtype == np.int8 and codes.nbytes * 4 == gr.nbytes     # 1 byte per value
    for t in range(wl.T):
        g = gr[uo[t]:uo[t + 1]]
        c = codes[uo[t]:uo[t + 1]].astype(np.int32)
        a = np.abs(g).max()
        assert gs[t] == np.float32(a) / np.float32(127)
        assert np.abs(c).max() == 127 and c.min() >= -127
        k = np.unravel_index(np.abs(g).argmax(), g.shape)
        assert c[k] == (127 if g[k] > 0 else -127)
        deq = c.astype(np.float32) * gs[t]
        assert np.abs(deq - g).max() <= gs[t] / 2 * (1 + 1e-6)
    # order independence: the scale is a function of the values only
    perm = np.random.default_rng(0).permutation(uo[1] - uo[0])
    gr2 = gr.copy()
    gr2[uo[0]:uo[1]] = gr[uo[0]:uo[1]][perm]
    codes2, gs2 = oracle.grad_quant_int8(gr2, uo, wl.D)
    assert gs2.tobytes() == gs.tobytes()
    assert (codes2[uo[0]:uo[1]] == codes[uo[0]:uo[1]][perm]).all()


# ---------------------------------------------------------------------------
# touched-row update with the dequantised gradient
# ---------------------------------------------------------------------------
def test_update_hand_example(oracle):
    D = 2
    off = np.array([0, 3, 5], dtype=np.int64)
    tables = f32([[1, 1], [2, 2], [3, 3], [4, 4], [5, 5]])
    unique_rows = np.array([0, 2, 1], dtype=np.int32)      # table 0 rows 0,2 ; table 1 row 1
    uniq_off = np.array([0, 2, 3], dtype=np.int32)
    codes = np.array([[4, -4], [8, 0], [-128, 127]], dtype=np.int8)
    gs = f32([0.25, 0.5])
    oracle.row_update(tables, off, D, unique_rows, uniq_off, codes, gs, 0.5)
    # W - 0.5 * code * scale, all exactly representable
    assert tables.tolist() == [[0.5, 1.5], [2, 2], [2, 3], [4, 4], [5 + 32, 5 - 31.75]]


def test_update_touches_only_listed_rows_and_lr0_is_identity(oracle):
    wl = W.tiny()
    tables = W.tables_np(wl)
    off = wl.row_off()
    indices, offsets = W.make_batch(wl, 2)
    grad_out = W.grad_out_np(wl, 2)
    ur, uo, gr = oracle.emb_bwd(grad_out, wl.T, wl.D, wl.B, indices, offsets)
    codes, gs = oracle.grad_quant_int8(gr, uo, wl.D)
    before = tables.copy()
    oracle.row_update(tables, off, wl.D, ur, uo, codes, gs, 0.0)
    assert tables.tobytes() == before.tobytes()
    oracle.row_update(tables, off, wl.D, ur, uo, codes, gs, 0.1)
    touched = np.zeros(wl.total_rows, dtype=bool)
    for t in range(wl.T):
        touched[off[t] + ur[uo[t]:uo[t + 1]]] = True
    assert tables[~touched].tobytes() == before[~touched].tobytes()
    # three separately rounded FP32 operations
    for t in range(wl.T):
        rows = off[t] + ur[uo[t]:uo[t + 1]]
        deq = codes[uo[t]:uo[t + 1]].astype(np.float32) * gs[t]
        step = np.float32(0.1) * deq
        want = before[rows] - step
        assert tables[rows].tobytes() == want.astype(np.float32).tobytes()
    assert (tables[touched] != before[touched]).any()


# ---------------------------------------------------------------------------
# whole step: stale scales between refreshes, drift of the range
# ---------------------------------------------------------------------------
def test_train_steps_with_periodic_refresh(oracle):
    wl = W.tiny()
    tables = W.tables_np(wl)
    off = wl.row_off()
    bits = np.full(wl.T, 4, dtype=np.int32)
    samplers = W.make_samplers(wl)
    scales = None
    seen_scales = []
    for step in range(25):
        if step % wl.period == 0:
            scales, _ = oracle.scale_refresh(tables, off, wl.D, bits)
            seen_scales.append(scales.copy())
        indices, offsets = W.make_batch(wl, step, samplers)
        r = oracle.train_step(tables, off, wl.D, wl.B, indices, offsets,
                              W.grad_out_np(wl, step), scales, bits, wl.lr)
        assert np.isfinite(r["out"]).all()
        # forward output of a one-index bag is an integer multiple of the (stale) scale
        q = r["out"][:, 0, :] / scales[0]
        assert np.abs(q - np.rint(q)).max() < 1e-3 and np.abs(np.rint(q)).max() <= 8
    # the weight range spreads out as training goes on, so refreshed scales grow
    assert (seen_scales[-1] >= seen_scales[0]).all() and (seen_scales[-1] > seen_scales[0]).any()
