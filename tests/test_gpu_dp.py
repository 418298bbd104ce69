"""Data-parallel exchange of the sparse INT8 gradient (paper Appendix B.1) on one GPU: the W
ranks are emulated as W batches in one process, the two collectives (MAX all-reduce of the
abs-max values, all-gather of rows and codes) as torch.max / concatenation.  Every local call
gets the oracle's inputs and must reproduce the oracle bit for bit."""
import numpy as np
import pytest

from dqrm_inputs import workloads as W

pytestmark = pytest.mark.gpu

CASES = {
    "tiny": lambda: W.tiny(),
    "kaggle_small": lambda: W.scaled_down(W.kaggle(), total_rows=300_000, B=2048, name="kaggle_small"),
    "terabyte_small": lambda: W.scaled_down(W.terabyte(), total_rows=400_000, B=1500, name="terabyte_small"),
    "multihot_small": lambda: W.scaled_down(W.multihot(), total_rows=26 * 3000, B=300, name="multihot_small"),
}


@pytest.mark.parametrize("ranks", [1, 2, 4])
@pytest.mark.parametrize("name", sorted(CASES))
def test_exchange_matches_oracle(name, ranks, oracle):
    import torch
    import paper_2410_20046_b200 as dq

    wl = CASES[name]()
    off = wl.row_off()
    samplers = W.make_samplers(wl)
    local = []
    for r in range(ranks):
        idx, offs = W.make_batch(wl, 20 + r, samplers)
        local.append(oracle.emb_bwd(W.grad_out_np(wl, 20 + r), wl.T, wl.D, wl.B, idx, offs))
    o_tables = W.tables_np(wl)
    want = oracle.dp_exchange_update(o_tables, off, wl.D, local, wl.lr)

    ctx = dq.Context(off, wl.D, 16, wl.T)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    # local: abs-max per rank
    absmax = torch.empty((ranks, wl.T), dtype=torch.float32, device="cuda")
    d_local = []
    for r, (ur, uo, gr) in enumerate(local):
        d = (dev(ur), dev(uo), dev(gr))
        d_local.append(d)
        ctx.grad_absmax(d[2], d[1], absmax[r])
        assert absmax[r].cpu().numpy().tobytes() == oracle.grad_absmax(gr, uo, wl.D).tobytes()
    unified = absmax.max(dim=0).values.contiguous()            # stands in for the MAX all-reduce
    # local: quantise with the unified scale
    stride = max(len(l[0]) for l in local)
    rows_cat = torch.zeros((ranks, stride), dtype=torch.int32, device="cuda")
    codes_cat = torch.zeros((ranks, stride, wl.D), dtype=torch.int8, device="cuda")
    uoff_cat = torch.stack([d[1] for d in d_local]).contiguous()
    scales = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    for r, (ur, uo, gr) in enumerate(d_local):
        U = ur.numel()
        codes = torch.empty((U, wl.D), dtype=torch.int8, device="cuda")
        ctx.grad_quant_int8_unified(gr, uo, unified, codes, scales)
        assert codes.cpu().numpy().tobytes() == want["codes"][r].tobytes()
        rows_cat[r, :U] = ur                                   # stands in for the all-gather
        codes_cat[r, :U] = codes
    assert scales.cpu().numpy().tobytes() == want["scales"].tobytes()
    # merge + update
    uoff_h = uoff_cat.cpu().numpy()
    n_entries = int(sum(u[-1] for u in uoff_h))
    max_table = int(max(sum(u[t + 1] - u[t] for u in uoff_h) for t in range(wl.T)))
    ws = ctx.dp_workspace(n_entries)
    d_tables = dev(W.tables_np(wl))
    union_rows = torch.full((n_entries,), -7, dtype=torch.int32, device="cuda")
    union_off = torch.empty(wl.T + 1, dtype=torch.int32, device="cuda")
    sums = torch.zeros((n_entries, wl.D), dtype=torch.int32, device="cuda")
    ctx.dp_merge_update(d_tables, ranks, stride, rows_cat, uoff_cat, codes_cat, scales, wl.lr, n_entries, max_table,
                        union_rows, union_off, sums, ws)
    ctx.raise_on_device_error()
    U = int(want["off"][-1])
    assert union_off.cpu().numpy().tobytes() == want["off"].tobytes()
    assert union_rows.cpu().numpy()[:U].tobytes() == want["rows"].tobytes()
    assert sums.cpu().numpy()[:U].tobytes() == want["sums"].tobytes()
    assert d_tables.cpu().numpy().tobytes() == o_tables.tobytes()
    # the other sort path gives the same replica
    ctx.set_sort_path(1)
    d_tables2 = dev(W.tables_np(wl))
    ctx.dp_merge_update(d_tables2, ranks, stride, rows_cat, uoff_cat, codes_cat, scales, wl.lr, n_entries, max_table,
                        union_rows, union_off, None, ws)
    ctx.raise_on_device_error()
    assert d_tables2.cpu().numpy().tobytes() == o_tables.tobytes()
    # with a row summary attached the merged update keeps every written row's (min, max) current
    ctx.set_sort_path(0)
    d_tables3 = dev(W.tables_np(wl))
    summary = ctx.row_summary_attach(d_tables3)
    ctx.dp_merge_update(d_tables3, ranks, stride, rows_cat, uoff_cat, codes_cat, scales, wl.lr, n_entries, max_table,
                        union_rows, union_off, None, ws)
    ctx.raise_on_device_error()
    assert d_tables3.cpu().numpy().tobytes() == o_tables.tobytes()
    got = summary.cpu().numpy().reshape(-1, 2)
    assert (got[:, 0] == o_tables.min(axis=1)).all() and (got[:, 1] == o_tables.max(axis=1)).all()
    ctx.row_summary_detach()
    ctx.close()
