"""GPU parity of the training step split in two calls (dqrm_sort_batch on one stream for batch
k+1 while dqrm_train_step_sorted trains batch k on another, two workspaces used alternately):
the trajectory must equal the oracle's, and the single-call step's, bit for bit."""
import numpy as np
import pytest

from dqrm_inputs import workloads as W
from gpu_util import Case, assert_close_fp32, bit_equal

pytestmark = pytest.mark.gpu


def _cases():
    return {
        "tiny": W.tiny(),
        "kaggle_small": W.scaled_down(W.kaggle(), total_rows=300_000, B=2048, name="kaggle_small"),
        "multihot_small": W.scaled_down(W.multihot(), total_rows=26 * 3000, B=300, name="multihot_small"),
    }


@pytest.mark.parametrize("name", sorted(_cases()))
def test_pipelined_steps_equal_oracle(oracle, name):
    import torch

    wl = _cases()[name]
    steps = 12
    c = Case(wl)
    o_tables = W.tables_np(wl)
    d_tables = c.dev(o_tables)
    Lmax = c.max_lookups
    out = c.empty((wl.B, wl.T, wl.D), torch.float32)
    gr = c.empty((Lmax, wl.D), torch.float32)
    codes = c.empty((Lmax, wl.D), torch.int8)
    gs = c.empty(wl.T, torch.float32)
    scales = c.empty(wl.T, torch.float32)
    # per in-flight batch: its device inputs and the sort's outputs
    slots = [dict(ur=c.empty(Lmax, torch.int32), uo=c.empty(wl.T + 1, torch.int32)) for _ in range(2)]
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    sorted_ev = [torch.cuda.Event(), torch.cuda.Event()]
    trained_ev = [torch.cuda.Event(), torch.cuda.Event()]

    def stage(step):
        s = slots[step & 1]
        idx, off, go = c.batch(step)
        s.update(idx_h=idx, off_h=off, go_h=go, idx=c.dev(idx), off=c.dev(off), go=c.dev(go), L=len(idx))
        torch.cuda.current_stream().synchronize()
        with torch.cuda.stream(side):
            side.wait_event(trained_ev[step & 1])          # the workspace's previous batch is done
            c.ctx.sort_batch(s["idx"], s["off"], s["ur"], s["uo"], B=wl.B, L=s["L"], ws=step & 1, stream=side)
            sorted_ev[step & 1].record(side)

    trained_ev[0].record(main)
    trained_ev[1].record(main)
    c.ctx.scale_refresh(d_tables, c.bits, scales)
    torch.cuda.synchronize()
    o_scales, _ = oracle.scale_refresh(o_tables, c.row_off, wl.D, c.bits_np)
    stage(0)
    for step in range(steps):
        if step + 1 < steps:
            stage(step + 1)                                 # sorts batch k+1 while batch k trains
        s = slots[step & 1]
        if step and step % 4 == 0:
            # a scale refresh between the two halves of a step must leave the sorted batch alone
            with torch.cuda.stream(main):
                c.ctx.scale_refresh(d_tables, c.bits, scales, stream=main)
            o_scales, _ = oracle.scale_refresh(o_tables, c.row_off, wl.D, c.bits_np)
        with torch.cuda.stream(main):
            main.wait_event(sorted_ev[step & 1])
            c.ctx.train_step_sorted(d_tables, s["idx"], s["off"], s["go"], scales, c.bits, out, s["ur"], s["uo"], gr,
                                    codes, gs, wl.lr, B=wl.B, L=s["L"], ws=step & 1, stream=main)
            trained_ev[step & 1].record(main)
        main.synchronize()
        r = oracle.train_step(o_tables, c.row_off, wl.D, wl.B, s["idx_h"], s["off_h"], s["go_h"], o_scales, c.bits_np,
                              wl.lr)
        U = int(r["uniq_off"][-1])
        assert bit_equal(s["uo"].cpu().numpy(), r["uniq_off"]), f"step {step}"
        assert bit_equal(s["ur"].cpu().numpy()[:U], r["unique_rows"]), f"step {step}"
        assert_close_fp32(out.cpu().numpy(), r["out"], f"step {step}: pooled output")
        assert_close_fp32(gr.cpu().numpy()[:U], r["grad_rows"], f"step {step}: summed gradients")
        assert bit_equal(gs.cpu().numpy(), r["grad_scales"]), f"step {step}: gradient scales"
        assert bit_equal(codes.cpu().numpy()[:U], r["codes"]), f"step {step}: gradient codes"
    torch.cuda.synchronize()
    c.ctx.raise_on_device_error()
    assert bit_equal(d_tables.cpu().numpy(), o_tables)
    c.ctx.close()


def test_two_calls_equal_one_call():
    import torch

    wl = W.scaled_down(W.terabyte(), total_rows=400_000, B=1500, name="terabyte_small")
    c = Case(wl)
    tables = W.tables_np(wl)
    idx, off, go = c.batch(0)
    L = len(idx)
    res = []
    for split in (False, True):
        d_tables = c.dev(tables)
        scales = c.empty(wl.T, torch.float32)
        c.ctx.scale_refresh(d_tables, c.bits, scales)
        out = c.empty((wl.B, wl.T, wl.D), torch.float32)
        ur = torch.full((L,), -1, dtype=torch.int32, device="cuda")
        uo = c.empty(wl.T + 1, torch.int32)
        gr = torch.zeros((L, wl.D), dtype=torch.float32, device="cuda")
        codes = torch.zeros((L, wl.D), dtype=torch.int8, device="cuda")
        gs = c.empty(wl.T, torch.float32)
        args = (d_tables, c.dev(idx), c.dev(off), c.dev(go), scales, c.bits, out, ur, uo, gr, codes, gs, wl.lr)
        if split:
            c.ctx.sort_batch(args[1], args[2], ur, uo, B=wl.B, L=L, ws=1)
            c.ctx.train_step_sorted(*args, B=wl.B, L=L, ws=1)
        else:
            c.ctx.train_step(*args, B=wl.B, L=L)
        c.ctx.raise_on_device_error()
        res.append([x.cpu().numpy() for x in (d_tables, out, ur, uo, gr, codes, gs)])
    for a, b in zip(*res):
        assert bit_equal(a, b)
    c.ctx.close()


def test_step_on_a_workspace_without_a_fresh_sort_is_refused():
    """One sort serves one step: a workspace that was never sorted, was sorted for another batch size, or whose
    sorted batch a step has already taken is turned down on the host, before any launch."""
    import torch
    from paper_2410_20046_b200 import binding

    wl = W.scaled_down(W.kaggle(), total_rows=50_000, B=300, name="kaggle_small")
    c = Case(wl)
    d_tables = c.dev(W.tables_np(wl))
    scales = c.empty(wl.T, torch.float32)
    c.ctx.scale_refresh(d_tables, c.bits, scales)
    idx, off, go = c.batch(0)
    L = len(idx)
    out = c.empty((wl.B, wl.T, wl.D), torch.float32)
    ur = torch.full((L,), -1, dtype=torch.int32, device="cuda")
    uo = c.empty(wl.T + 1, torch.int32)
    gr = torch.zeros((L, wl.D), dtype=torch.float32, device="cuda")
    codes = torch.zeros((L, wl.D), dtype=torch.int8, device="cuda")
    gs = c.empty(wl.T, torch.float32)
    args = (d_tables, c.dev(idx), c.dev(off), c.dev(go), scales, c.bits, out, ur, uo, gr, codes, gs, wl.lr)

    def refused(**kw):
        with pytest.raises(binding.DqrmError) as e:
            c.ctx.train_step_sorted(*args, **kw)
        return e.value.status == binding.ERR_NOT_SORTED

    assert refused(B=wl.B, L=L, ws=1)                       # never sorted
    c.ctx.sort_batch(args[1], args[2], ur, uo, B=wl.B, L=L, ws=1)
    assert refused(B=wl.B, L=L, ws=0)                       # the other workspace was
    before = d_tables.clone()
    c.ctx.train_step_sorted(*args, B=wl.B, L=L, ws=1)
    c.ctx.raise_on_device_error()
    after = d_tables.clone()
    assert not torch.equal(before, after)
    assert refused(B=wl.B, L=L, ws=1)                       # already taken
    assert torch.equal(d_tables, after)                     # and nothing ran
    c.ctx.close()


def test_step_waits_for_its_sort_without_the_callers_help():
    """The gradient summation is ordered behind the sort by an event the context keeps with the workspace: the
    sort of the next batch runs on another stream, held back there by a long wait so that it is certainly late,
    and the step's stream never waits for that stream.  The trajectory must equal the single-call loop's."""
    import torch

    wl = W.scaled_down(W.terabyte(), total_rows=400_000, B=1500, name="terabyte_small")
    c = Case(wl)
    tables = W.tables_np(wl)
    steps = 5
    batches = [c.batch(s) for s in range(steps)]
    Lmax = max(len(b[0]) for b in batches)
    res = []
    for split in (False, True):
        d_tables = c.dev(tables)
        scales = c.empty(wl.T, torch.float32)
        c.ctx.scale_refresh(d_tables, c.bits, scales)
        out = c.empty((wl.B, wl.T, wl.D), torch.float32)
        urs = [torch.full((Lmax,), -1, dtype=torch.int32, device="cuda") for _ in range(2)]
        uos = [c.empty(wl.T + 1, torch.int32) for _ in range(2)]
        gr = torch.zeros((Lmax, wl.D), dtype=torch.float32, device="cuda")
        codes = torch.zeros((Lmax, wl.D), dtype=torch.int8, device="cuda")
        gs = c.empty(wl.T, torch.float32)
        dev = [(c.dev(i), c.dev(o), c.dev(g), len(i)) for i, o, g in batches]
        torch.cuda.synchronize()
        outs = []
        if not split:
            for i, o, g, L in dev:
                c.ctx.train_step(d_tables, i, o, g, scales, c.bits, out, urs[0], uos[0], gr, codes, gs, wl.lr, B=wl.B, L=L)
                outs.append(out.cpu().numpy().copy())
        else:
            main, side = torch.cuda.Stream(), torch.cuda.Stream()
            c.ctx.sort_batch(dev[0][0], dev[0][1], urs[0], uos[0], B=wl.B, L=dev[0][3], ws=0, stream=side)
            for k, (i, o, g, L) in enumerate(dev):
                slot = k & 1
                if k + 1 < steps:
                    ni, no, _, nL = dev[k + 1]
                    side.wait_stream(main)                  # the other workspace's previous batch has trained
                    with torch.cuda.stream(side):
                        torch.cuda._sleep(4_000_000)        # a few milliseconds: this sort is late
                    c.ctx.sort_batch(ni, no, urs[slot ^ 1], uos[slot ^ 1], B=wl.B, L=nL, ws=slot ^ 1, stream=side)
                c.ctx.train_step_sorted(d_tables, i, o, g, scales, c.bits, out, urs[slot], uos[slot], gr, codes, gs,
                                        wl.lr, B=wl.B, L=L, ws=slot, stream=main)
                main.synchronize()
                outs.append(out.cpu().numpy().copy())
            side.synchronize()
        c.ctx.raise_on_device_error()
        res.append((d_tables.cpu().numpy(), outs, gr.cpu().numpy()[:dev[-1][3]], codes.cpu().numpy()[:dev[-1][3]]))
    (ta, oa, ga, ca), (tb, ob, gb, cb) = res
    assert bit_equal(ta, tb)
    for x, y in zip(oa, ob):
        assert bit_equal(x, y)
    c.ctx.close()


def test_sort_held_until_the_forward_is_done_equals_one_call():
    """dqrm_stream_wait_forward: the next batch's sort starts only behind this batch's forward and runs
    beside the rest of the step; the trajectory must equal the single-call loop's bit for bit."""
    import torch

    wl = W.scaled_down(W.terabyte(), total_rows=400_000, B=1500, name="terabyte_small")
    c = Case(wl)
    tables = W.tables_np(wl)
    steps = 6
    batches = [c.batch(s) for s in range(steps)]
    res = []
    for held in (False, True):
        d_tables = c.dev(tables)
        scales = c.empty(wl.T, torch.float32)
        c.ctx.scale_refresh(d_tables, c.bits, scales)
        out = c.empty((wl.B, wl.T, wl.D), torch.float32)
        Lmax = max(len(b[0]) for b in batches)
        urs = [torch.full((Lmax,), -1, dtype=torch.int32, device="cuda") for _ in range(2)]
        uos = [c.empty(wl.T + 1, torch.int32) for _ in range(2)]
        gr = torch.zeros((Lmax, wl.D), dtype=torch.float32, device="cuda")
        codes = torch.zeros((Lmax, wl.D), dtype=torch.int8, device="cuda")
        gs = c.empty(wl.T, torch.float32)
        dev = [(c.dev(i), c.dev(o), c.dev(g), len(i)) for i, o, g in batches]
        torch.cuda.synchronize()
        outs = []
        if not held:
            for i, o, g, L in dev:
                c.ctx.train_step(d_tables, i, o, g, scales, c.bits, out, urs[0], uos[0], gr, codes, gs, wl.lr, B=wl.B, L=L)
                outs.append(out.cpu().numpy().copy())
        else:
            main, side = torch.cuda.Stream(), torch.cuda.Stream()
            c.ctx.sort_batch(dev[0][0], dev[0][1], urs[0], uos[0], B=wl.B, L=dev[0][3], ws=0, stream=main)
            for k, (i, o, g, L) in enumerate(dev):
                slot = k & 1
                side.wait_stream(main)                      # workspace slot^1: its previous batch has trained
                c.ctx.train_step_sorted(d_tables, i, o, g, scales, c.bits, out, urs[slot], uos[slot], gr, codes, gs,
                                        wl.lr, B=wl.B, L=L, ws=slot, stream=main)
                if k + 1 < steps:
                    ni, no, _, nL = dev[k + 1]
                    c.ctx.stream_wait_forward(side)
                    c.ctx.sort_batch(ni, no, urs[slot ^ 1], uos[slot ^ 1], B=wl.B, L=nL, ws=slot ^ 1, stream=side)
                main.wait_stream(side)
                main.synchronize()
                outs.append(out.cpu().numpy().copy())
        torch.cuda.synchronize()
        c.ctx.raise_on_device_error()
        res.append((d_tables.cpu().numpy(), outs, gs.cpu().numpy()))
    assert bit_equal(res[0][0], res[1][0])
    assert bit_equal(res[0][2], res[1][2])
    for a, b in zip(res[0][1], res[1][1]):
        assert bit_equal(a, b)
    c.ctx.close()
