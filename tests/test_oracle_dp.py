"""Pins for the oracle's data-parallel gradient exchange (paper Appendix B.1): unify the
quantisation scales across ranks, quantise locally, sum the integer gradients, apply the
dequantised sum.  Expected values are hand-worked, come from numpy (unique, dense
accumulation) or from the single-rank path the exchange must reduce to."""
import numpy as np

from dqrm_inputs import workloads as W


def _local(oracle, wl, step):
    idx, off = W.make_batch(wl, step)
    go = W.grad_out_np(wl, step)
    return oracle.emb_bwd(go, wl.T, wl.D, wl.B, idx, off)


def test_merge_hand_example(oracle):
    rows = [np.array([1, 4, 2], np.int32), np.array([4, 0, 2], np.int32)]
    uoff = [np.array([0, 2, 3], np.int32), np.array([0, 1, 3], np.int32)]
    codes = [np.array([[1, -1], [2, -2], [3, -3]], np.int8), np.array([[10, 10], [20, 20], [127, -128]], np.int8)]
    r, o, s = oracle.dp_merge(rows, uoff, codes, 2, 2)
    assert r.tolist() == [1, 4, 0, 2]            # table 0: {1, 4}; table 1: {0, 2}
    assert o.tolist() == [0, 2, 4]
    assert s.tolist() == [[1, -1], [12, 8], [20, 20], [130, -131]]      # exact, beyond the int8 range


def test_merge_equals_dense_integer_accumulation(oracle):
    rng = np.random.default_rng(0)
    T, D, Wn = 5, 4, 4
    R = [7, 50, 3, 1000, 20]
    rows, uoff, codes = [], [], []
    for r in range(Wn):
        rr, uo = [], [0]
        for t in range(T):
            k = int(rng.integers(0, min(R[t], 12) + 1))
            rr.append(np.sort(rng.choice(R[t], size=k, replace=False)).astype(np.int32))
            uo.append(uo[-1] + k)
        rows.append(np.concatenate(rr).astype(np.int32))
        uoff.append(np.array(uo, np.int32))
        codes.append(rng.integers(-128, 128, size=(uo[-1], D)).astype(np.int8))
    out_rows, out_off, sums = oracle.dp_merge(rows, uoff, codes, T, D)
    for t in range(T):
        dense = np.zeros((R[t], D), dtype=np.int64)
        touched = np.zeros(R[t], dtype=bool)
        for r in range(Wn):
            sl = slice(uoff[r][t], uoff[r][t + 1])
            np.add.at(dense, rows[r][sl], codes[r][sl].astype(np.int64))
            touched[rows[r][sl]] = True
        want_rows = np.nonzero(touched)[0]
        got = out_rows[out_off[t]:out_off[t + 1]]
        assert got.tolist() == want_rows.tolist()
        assert (sums[out_off[t]:out_off[t + 1]] == dense[want_rows]).all()
    assert out_off[-1] == len(out_rows)


def test_scaled_quantiser_and_absmax(oracle):
    wl = W.tiny()
    ur, uo, gr = _local(oracle, wl, 0)
    a = oracle.grad_absmax(gr, uo, wl.D)
    for t in range(wl.T):
        assert a[t] == np.abs(gr[uo[t]:uo[t + 1]]).max()
    own_codes, own_scales = oracle.grad_quant_int8(gr, uo, wl.D)
    # with its own scale the scaled quantiser is the plain one
    assert oracle.grad_quant_int8_scaled(gr, uo, wl.D, own_scales).tobytes() == own_codes.tobytes()
    # with a scale twice as large every code is the code of half the value
    half = oracle.grad_quant_int8_scaled(gr, uo, wl.D, own_scales * np.float32(2))
    assert np.abs(half).max() == 64 and (np.abs(half.astype(int) * 2 - own_codes.astype(int)) <= 1).all()


def test_one_rank_reduces_to_the_single_gpu_update(oracle):
    wl = W.tiny()
    off = wl.row_off()
    ur, uo, gr = _local(oracle, wl, 1)
    a, b = W.tables_np(wl), W.tables_np(wl)
    codes, gs = oracle.grad_quant_int8(gr, uo, wl.D)
    oracle.row_update(a, off, wl.D, ur, uo, codes, gs, wl.lr)
    r = oracle.dp_exchange_update(b, off, wl.D, [(ur, uo, gr)], wl.lr)
    assert a.tobytes() == b.tobytes()
    assert r["scales"].tobytes() == gs.tobytes() and r["codes"][0].tobytes() == codes.tobytes()
    assert r["rows"].tobytes() == ur.tobytes() and r["off"].tobytes() == uo.tobytes()


def test_exchange_properties_two_and_four_ranks(oracle):
    wl = W.tiny()
    off = wl.row_off()
    for Wn in (2, 4):
        local = [_local(oracle, wl, 10 + r) for r in range(Wn)]
        tables = W.tables_np(wl)
        before = tables.copy()
        r = oracle.dp_exchange_update(tables, off, wl.D, local, wl.lr)
        # unified scale = max over ranks of the rank's own scale; nothing clips with it
        own = np.stack([oracle.grad_quant_int8(g, uo, wl.D)[1] for (_, uo, g) in local])
        assert r["scales"].tobytes() == own.max(axis=0).tobytes()
        for c in r["codes"]:
            assert c.min() >= -127 and c.max() <= 127
        assert max(np.abs(c).max() for c in r["codes"]) == 127
        # union of the ranks' rows, per table
        for t in range(wl.T):
            want = np.unique(np.concatenate([l[0][l[1][t]:l[1][t + 1]] for l in local]))
            assert r["rows"][r["off"][t]:r["off"][t + 1]].tolist() == want.tolist()
        assert np.abs(r["sums"]).max() <= 127 * Wn
        # the update: three rounded FP32 operations on the summed integers
        touched = np.zeros(wl.total_rows, dtype=bool)
        for t in range(wl.T):
            rows = off[t] + r["rows"][r["off"][t]:r["off"][t + 1]]
            touched[rows] = True
            g = r["sums"][r["off"][t]:r["off"][t + 1]].astype(np.float32) * r["scales"][t]
            want = before[rows] - np.float32(wl.lr) * g
            assert tables[rows].tobytes() == want.astype(np.float32).tobytes()
        assert tables[~touched].tobytes() == before[~touched].tobytes()


def test_two_identical_ranks_sum_not_mean(oracle):
    D = 2
    off = np.array([0, 4], dtype=np.int64)
    tables = np.zeros((4, D), dtype=np.float32)
    local = [(np.array([2], np.int32), np.array([0, 1], np.int32), np.array([[127.0, -63.5]], np.float32))] * 2
    r = oracle.dp_exchange_update(tables, off, D, local, 0.5)
    assert r["scales"][0] == 1.0 and r["sums"].tolist() == [[254, -128]]
    assert tables[2].tolist() == [-127.0, 64.0] and not tables[[0, 1, 3]].any()
