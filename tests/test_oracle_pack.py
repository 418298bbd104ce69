"""Pins for the oracle's bit-packed export and packed inference lookup (paper Appendix C)."""
import os

import numpy as np
import pytest

from dqrm_inputs import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))


def test_paper_model_sizes_are_an_eighth():
    # Table "res_tab": the INT4 model is the FP32 model / 8; the packed layout must give that ratio
    for line in open(os.path.join(HERE, "golden", "paper_model_sizes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, fp32, int4 = line.split()
        assert abs(float(fp32) / 8 - float(int4)) < 0.002
    wl = W.tiny()
    assert wl.total_rows * (wl.D * 4 // 8) * 8 == wl.table_bytes()


def test_pack_hand_example(oracle):
    D = 4
    off = np.array([0, 2], dtype=np.int64)
    tables = np.array([[1, -1, 7, -8], [0, 3, -4, 100]], dtype=np.float32)
    p4 = oracle.pack_tables(tables, off, D, np.array([1.0], np.float32), 4)
    # element 2k in the low nibble, 2k+1 in the high nibble, two's complement: -1 = 0xF, -8 = 0x8, 100 clamps to 7
    assert p4.tolist() == [[0xF1, 0x87], [0x30, 0x7C]]
    p2 = oracle.pack_tables(tables, off, D, np.array([4.0], np.float32), 2)
    # codes with scale 4, 2 bits: [0,0,1(2->clamp 1),-2] and [0,1,-1,1]; -2 = 0b10, -1 = 0b11
    assert p2.tolist() == [[0b10010000], [0b01110100]]
    p8 = oracle.pack_tables(tables, off, D, np.array([0.5], np.float32), 8)
    assert p8.view(np.int8).tolist() == [[2, -2, 14, -16], [0, 6, -8, 127]]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_packed_lookup_equals_training_forward(oracle, bits):
    # inference from the packed table gives exactly what the QAT forward computes from the FP32 master table
    for wl in (W.tiny(), W.scaled_down(W.multihot(), total_rows=26 * 400, B=20, name="mh")):
        tables = W.tables_np(wl)
        off = wl.row_off()
        b = np.full(wl.T, bits, dtype=np.int32)
        scales, _ = oracle.scale_refresh(tables, off, wl.D, b)
        idx, offs = W.make_batch(wl, 0)
        packed = oracle.pack_tables(tables, off, wl.D, scales, bits)
        assert packed.shape == (wl.total_rows, wl.D * bits // 8)
        got = oracle.packed_fwd(packed, off, wl.D, wl.B, idx, offs, scales, bits)
        want = oracle.emb_fwd(tables, off, wl.D, wl.B, idx, offs, scales, b)
        assert got.tobytes() == want.tobytes()


def test_unpacked_codes_match_the_quantiser(oracle):
    wl = W.tiny()
    tables = W.tables_np(wl)
    off = wl.row_off()
    scales, _ = oracle.scale_refresh(tables, off, wl.D, np.full(wl.T, 4, dtype=np.int32))
    packed = oracle.pack_tables(tables, off, wl.D, scales, 4)
    lo = (packed & 0x0F).astype(np.int8)
    hi = (packed >> 4).astype(np.int8)
    codes = np.stack([lo, hi], axis=-1).reshape(wl.total_rows, wl.D)
    codes = np.where(codes >= 8, codes - 16, codes)
    for r in (0, 999, 1000, 25999, 125999):
        t = int(np.searchsorted(off, r, side="right") - 1)
        assert codes[r].tolist() == [oracle.quantize(x, scales[t], 4) for x in tables[r]]
