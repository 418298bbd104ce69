"""Pins for the oracle's table-sharded forward payload (Section 4.3's remark on hybrid parallelism:
the all-to-all of embedding vectors shrinks with the code width)."""
import numpy as np
import pytest

from dqrm_inputs import workloads as W


def _problem(bits):
    wl = W.tiny()
    tables = W.tables_np(wl)
    off = wl.row_off()
    b = np.full(wl.T, bits, dtype=np.int32)
    idx, offs = W.make_batch(wl, 0)
    return wl, tables, off, b, idx, offs


def test_payload_hand_example(oracle):
    D = 4
    off = np.array([0, 2, 3], dtype=np.int64)                     # two tables: 2 rows, 1 row
    tables = np.array([[1, -1, 7, -8], [0, 3, -4, 100], [2, 2, -2, 0]], dtype=np.float32)
    idx = np.array([1, 0, 0, 0], dtype=np.int32)                  # table 0: bags -> rows 1, 0; table 1: row 0 twice
    offs = np.arange(5, dtype=np.int32)
    p = oracle.emb_fwd_codes(tables, off, D, 2, idx, offs, np.array([1.0, 2.0], np.float32), 4)
    # [bag][table][bytes]; element 2k in the low nibble; 100 clamps to 7; table 1 has scale 2: codes 1, 1, -1, 0
    assert p.tolist() == [[[0x30, 0x7C], [0x11, 0x0F]], [[0xF1, 0x87], [0x11, 0x0F]]]
    out = oracle.decode_payload(p, np.array([1.0, 2.0], np.float32), 4, D, 2, 0)
    assert out.tolist() == [[[0, 3, -4, 7], [2, 2, -2, 0]], [[1, -1, 7, -8], [2, 2, -2, 0]]]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_payload_is_the_packed_row_and_decodes_to_the_forward(oracle, bits):
    wl, tables, off, b, idx, offs = _problem(bits)
    scales, _ = oracle.scale_refresh(tables, off, wl.D, b)
    payload = oracle.emb_fwd_codes(tables, off, wl.D, wl.B, idx, offs, scales, bits)
    assert payload.shape == (wl.B, wl.T, wl.D * bits // 8)
    # the payload of a bag is the row of the packed table it looks up (pack_tables is pinned by hand examples)
    packed = oracle.pack_tables(tables, off, wl.D, scales, bits)
    for t in range(wl.T):
        rows = off[t] + idx[offs[t * wl.B:(t + 1) * wl.B]]
        assert (payload[:, t, :] == packed[rows]).all()
    # decoding every sender's block gives exactly the training forward
    want = oracle.emb_fwd(tables, off, wl.D, wl.B, idx, offs, scales, b)
    got = np.zeros_like(want)
    for t0, t1 in ((0, 1), (1, wl.T)):
        oracle.decode_payload(payload[:, t0:t1, :], scales[t0:t1], bits, wl.D, wl.T, t0, out=got)
    assert got.tobytes() == want.tobytes()
    # the payload is 32/bits times smaller than the FP32 vectors
    assert payload.nbytes * (32 // bits) == want.nbytes


def test_payload_refuses_bags_that_are_not_one_index(oracle):
    wl = W.scaled_down(W.multihot(), total_rows=26 * 100, B=8, name="mh")
    tables = W.tables_np(wl)
    idx, offs = W.make_batch(wl, 0)
    with pytest.raises(ValueError):
        oracle.emb_fwd_codes(tables, wl.row_off(), wl.D, wl.B, idx, offs, np.ones(wl.T, np.float32), 4)
