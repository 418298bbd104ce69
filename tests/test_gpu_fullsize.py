"""Parity at the full sizes of the benchmark configurations, through the timed entry points
(dqrm_train_step, and the two-call form dqrm_sort_batch + dqrm_train_step_sorted with the next
batch being sorted on a second stream meanwhile) in the launch configuration bench.py uses.

The tables (2.2 GB / 12.5 GB) are generated on the device by the shared counter-based
generator.  The oracle cannot hold them, but it does not need to: every row a batch
touches is regenerated on the host from the same generator, the batch is re-indexed onto
that compact set of rows, and the oracle runs the whole step on the compact problem.
That compares every output of the step, not a sample.  The scale refresh over the full
arena is checked against torch.aminmax (an independent reduction) fed through the
oracle's scale formula, and a sample of untouched rows is checked to be unchanged."""
import numpy as np
import pytest

from dqrm_inputs import workloads as W

pytestmark = pytest.mark.gpu


def _compact(wl, idx, off):
    """Touched rows per table (ascending) and the batch re-indexed onto them."""
    rows, new_idx = [], np.empty_like(idx)
    for t in range(wl.T):
        lo, hi = off[t * wl.B], off[(t + 1) * wl.B]
        u, inv = np.unique(idx[lo:hi], return_inverse=True)
        rows.append(u)
        new_idx[lo:hi] = inv.astype(np.int32)
    return rows, new_idx


def _workload(name):
    if name in W.BY_NAME:
        return W.BY_NAME[name]()
    d, b, dist = name.split("_")[1:]                  # sweep_d64_b8_zipf
    return W.sweep(D=int(d[1:]), bits=int(b[1:]), zipf=(dist == "zipf"))


@pytest.mark.parametrize("name", ["kaggle_b16384", "terabyte_b32768", "multihot_b16384", "kaggle_b128",
                                  "terabyte_b2048", "sweep_d16_b2_uniform", "sweep_d32_b4_zipf",
                                  "sweep_d64_b8_zipf", "sweep_d128_b8_uniform",
                                  "kaggle_b16384+two_calls", "terabyte_b32768+two_calls", "multihot_b16384+two_calls"])
def test_full_size_step_matches_oracle(name, oracle):
    import torch
    import paper_2410_20046_b200 as dq

    name, _, form = name.partition("+")
    wl = _workload(name)
    off_rows = wl.row_off()
    tables = W.tables_torch(wl, "cuda")
    bits_h = np.full(wl.T, wl.bits, dtype=np.int32)
    bits = torch.from_numpy(bits_h).cuda()
    samplers = W.make_samplers(wl)
    idx, off = W.make_batch(wl, 0, samplers)
    go = W.grad_out_np(wl, 0)
    L, G = len(idx), wl.T * wl.B

    ctx = dq.Context(off_rows, wl.D, L, G)
    scales = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    minmax = torch.empty((wl.T, 2), dtype=torch.float32, device="cuda")
    ctx.scale_refresh(tables, bits, scales, minmax)
    ctx.raise_on_device_error()
    # refresh against an independent reduction
    want_scales = np.empty(wl.T, dtype=np.float32)
    for t in range(wl.T):
        mn, mx = torch.aminmax(tables[off_rows[t]:off_rows[t + 1]])
        assert float(minmax[t, 0]) == float(mn) and float(minmax[t, 1]) == float(mx)
        want_scales[t] = oracle.scale_from_absmax(max(abs(float(mn)), abs(float(mx))), wl.bits)
    assert scales.cpu().numpy().tobytes() == want_scales.tobytes()

    # a sample of rows the batch does not touch, to be re-read after the step
    rng = np.random.default_rng(1)
    touched, new_idx = _compact(wl, idx, off)
    untouched = []
    for t in range(wl.T):
        cand = rng.integers(0, wl.rows[t], size=64)
        untouched.append(np.setdiff1d(cand, touched[t]))

    out = torch.empty((wl.B, wl.T, wl.D), dtype=torch.float32, device="cuda")
    ur = torch.empty(L, dtype=torch.int32, device="cuda")
    uo = torch.empty(wl.T + 1, dtype=torch.int32, device="cuda")
    gr = torch.empty((L, wl.D), dtype=torch.float32, device="cuda")
    codes = torch.empty((L, wl.D), dtype=torch.int8, device="cuda")
    gs = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    d_idx, d_off, d_go = torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda(), torch.from_numpy(go).cuda()
    if form == "two_calls":
        # what a pipelined loop does: this batch was sorted ahead into one workspace; while it trains, the
        # next batch is sorted on a second stream into the other workspace
        nidx, noff = W.make_batch(wl, 1, samplers)
        d_nidx, d_noff = torch.from_numpy(nidx).cuda(), torch.from_numpy(noff).cuda()
        ur2, uo2 = torch.empty(len(nidx), dtype=torch.int32, device="cuda"), torch.empty_like(uo)
        ctx2 = ctx if len(nidx) <= L else None
        ctx.sort_batch(d_idx, d_off, ur, uo, B=wl.B, L=L, ws=1)
        cur, side = torch.cuda.current_stream(), torch.cuda.Stream(priority=-1)
        side.wait_stream(cur)
        if ctx2 is not None:
            ctx.sort_batch(d_nidx, d_noff, ur2, uo2, B=wl.B, L=len(nidx), ws=0, stream=side)
        ctx.train_step_sorted(tables, d_idx, d_off, d_go, scales, bits, out, ur, uo, gr, codes, gs, wl.lr, B=wl.B,
                              L=L, ws=1)
        cur.wait_stream(side)
    else:
        ctx.train_step(tables, d_idx, d_off, d_go, scales, bits, out, ur, uo, gr, codes, gs, wl.lr, B=wl.B, L=L)
    ctx.raise_on_device_error()

    # the oracle on the compact problem: only the touched rows, regenerated on the host
    c_rows = np.array([len(r) for r in touched], dtype=np.int64)
    c_off = np.zeros(wl.T + 1, dtype=np.int64)
    c_off[1:] = np.cumsum(c_rows)
    c_tables = np.concatenate([W.table_rows_at_np(wl, t, touched[t]) for t in range(wl.T)])
    r = oracle.train_step(c_tables, c_off, wl.D, wl.B, new_idx, off, go, want_scales, bits_h, wl.lr)
    U = int(r["uniq_off"][-1])
    assert U == int(c_off[-1])

    assert uo.cpu().numpy().tobytes() == r["uniq_off"].tobytes()
    got_ur = ur.cpu().numpy()[:U]
    want_ur = np.concatenate(touched).astype(np.int32)          # compact rank u of table t is row touched[t][u]
    assert got_ur.tobytes() == want_ur.tobytes()
    assert out.cpu().numpy().tobytes() == r["out"].tobytes()     # same order, FP64 sums: bit for bit
    got_gr = gr.cpu().numpy()[:U]
    np.testing.assert_allclose(got_gr, r["grad_rows"], rtol=1e-5, atol=1e-6)
    mism = int((got_gr.view(np.int32) != r["grad_rows"].view(np.int32)).sum())
    assert mism <= max(2, got_gr.size // 1_000_000), f"{mism} summed gradients differ in the last bit"
    if mism == 0:
        assert gs.cpu().numpy().tobytes() == r["grad_scales"].tobytes()
        assert codes.cpu().numpy()[:U].tobytes() == r["codes"].tobytes()
    # updated rows: gather the touched rows from the device table
    for t in range(wl.T):
        rows_dev = tables[off_rows[t] + torch.from_numpy(touched[t].astype(np.int64)).cuda()].cpu().numpy()
        want = c_tables[c_off[t]:c_off[t + 1]]
        if mism == 0:
            assert rows_dev.tobytes() == want.tobytes(), f"table {t}: updated rows differ"
        else:
            np.testing.assert_allclose(rows_dev, want, rtol=1e-5, atol=1e-6)
        if len(untouched[t]):
            still = tables[off_rows[t] + torch.from_numpy(untouched[t].astype(np.int64)).cuda()].cpu().numpy()
            assert still.tobytes() == W.table_rows_at_np(wl, t, untouched[t]).tobytes(), f"table {t}: untouched rows changed"
    ctx.close()
    del tables
    torch.cuda.empty_cache()
