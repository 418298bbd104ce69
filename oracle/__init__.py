"""ctypes front end of the DQRM embedding-path oracle (``dqrm_oracle.c``).

TEST INFRASTRUCTURE ONLY: a plain single-threaded CPU statement of the method,
used by the tests, the smoke check and the benchmark's CPU-baseline leg.  The
CUDA package never imports this module and this module never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dqrm_oracle.c")
_LIB = os.path.join(_HERE, "libdqrm_oracle.so")

CFLAGS = ["-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared"]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no FMA contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.dqrm_oracle_scale_from_absmax.restype = ctypes.c_float
        _lib.dqrm_oracle_scale_from_absmax.argtypes = [ctypes.c_float, ctypes.c_int]
        _lib.dqrm_oracle_quantize.restype = ctypes.c_int32
        _lib.dqrm_oracle_quantize.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int]
        _lib.dqrm_oracle_dequantize.restype = ctypes.c_float
        _lib.dqrm_oracle_dequantize.argtypes = [ctypes.c_int32, ctypes.c_float]
        _lib.dqrm_oracle_fake_quant.restype = ctypes.c_float
        _lib.dqrm_oracle_fake_quant.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int]
        _lib.dqrm_oracle_emb_bwd.restype = ctypes.c_int64
        _lib.dqrm_oracle_dp_merge.restype = ctypes.c_int64
    return _lib


def _p(a, dtype):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (
        f"expected contiguous {dtype} array")
    return a.ctypes.data_as(ctypes.c_void_p)


# ---- scalar quantiser ------------------------------------------------------
def scale_from_absmax(absmax: float, bits: int) -> np.float32:
    return np.float32(lib().dqrm_oracle_scale_from_absmax(float(np.float32(absmax)), int(bits)))


def quantize(x: float, s: float, bits: int) -> int:
    return int(lib().dqrm_oracle_quantize(float(np.float32(x)), float(np.float32(s)), int(bits)))


def dequantize(q: int, s: float) -> np.float32:
    return np.float32(lib().dqrm_oracle_dequantize(int(q), float(np.float32(s))))


def fake_quant(x: float, s: float, bits: int) -> np.float32:
    return np.float32(lib().dqrm_oracle_fake_quant(float(np.float32(x)), float(np.float32(s)), int(bits)))


# ---- array steps -----------------------------------------------------------
def scale_refresh(tables, row_off, D, bits):
    """-> (scales float32 [T], minmax float32 [T, 2])"""
    T = len(row_off) - 1
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    bits = np.ascontiguousarray(bits, dtype=np.int32)
    scales = np.empty(T, dtype=np.float32)
    minmax = np.empty((T, 2), dtype=np.float32)
    lib().dqrm_oracle_scale_refresh(_p(tables, np.float32), _p(row_off, np.int64), T, int(D),
                                    _p(bits, np.int32), _p(scales, np.float32), _p(minmax, np.float32))
    return scales, minmax


def emb_fwd(tables, row_off, D, B, indices, offsets, scales, bits, want_codes=False):
    """-> out float32 [B, T, D] (and codes int8 [L, D] if want_codes)"""
    T = len(row_off) - 1
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    bits = np.ascontiguousarray(bits, dtype=np.int32)
    out = np.empty((B, T, D), dtype=np.float32)
    codes = np.empty((len(indices), D), dtype=np.int8) if want_codes else None
    lib().dqrm_oracle_emb_fwd(_p(tables, np.float32), _p(row_off, np.int64), T, int(D), int(B),
                              _p(indices, np.int32), _p(offsets, np.int32),
                              _p(scales, np.float32), _p(bits, np.int32),
                              _p(out, np.float32), _p(codes, np.int8))
    return (out, codes) if want_codes else out


def emb_bwd(grad_out, T, D, B, indices, offsets):
    """-> (unique_rows int32 [U], uniq_off int32 [T+1], grad_rows float32 [U, D])"""
    L = len(indices)
    unique_rows = np.empty(max(L, 1), dtype=np.int32)
    uniq_off = np.empty(T + 1, dtype=np.int32)
    grad_rows = np.empty((max(L, 1), D), dtype=np.float32)
    U = lib().dqrm_oracle_emb_bwd(_p(grad_out, np.float32), int(T), int(D), int(B),
                                  _p(indices, np.int32), _p(offsets, np.int32),
                                  _p(unique_rows, np.int32), _p(uniq_off, np.int32),
                                  _p(grad_rows, np.float32))
    return unique_rows[:U].copy(), uniq_off, grad_rows[:U].copy()


def grad_quant_int8(grad_rows, uniq_off, D):
    """-> (codes int8 [U, D], grad_scales float32 [T])"""
    T = len(uniq_off) - 1
    codes = np.empty(grad_rows.shape, dtype=np.int8)
    grad_scales = np.empty(T, dtype=np.float32)
    gr = grad_rows if grad_rows.size else np.zeros((1, D), dtype=np.float32)
    cd = codes if codes.size else np.zeros((1, D), dtype=np.int8)
    lib().dqrm_oracle_grad_quant_int8(_p(gr, np.float32), _p(uniq_off, np.int32), T, int(D),
                                      _p(cd, np.int8), _p(grad_scales, np.float32))
    return codes, grad_scales


def row_update(tables, row_off, D, unique_rows, uniq_off, codes, grad_scales, lr):
    """Updates ``tables`` in place."""
    T = len(row_off) - 1
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    ur = unique_rows if unique_rows.size else np.zeros(1, dtype=np.int32)
    cd = codes if codes.size else np.zeros((1, D), dtype=np.int8)
    lib().dqrm_oracle_row_update(_p(tables, np.float32), _p(row_off, np.int64), T, int(D),
                                 _p(ur, np.int32), _p(uniq_off, np.int32),
                                 _p(cd, np.int8), _p(grad_scales, np.float32),
                                 ctypes.c_float(float(np.float32(lr))))


def train_step(tables, row_off, D, B, indices, offsets, grad_out, scales, bits, lr):
    """fwd -> bwd -> INT8 gradient quantisation -> touched-row update, in the order
    the paper's training iteration takes them.  Updates ``tables`` in place."""
    T = len(row_off) - 1
    out = emb_fwd(tables, row_off, D, B, indices, offsets, scales, bits)
    unique_rows, uniq_off, grad_rows = emb_bwd(grad_out, T, D, B, indices, offsets)
    codes, grad_scales = grad_quant_int8(grad_rows, uniq_off, D)
    row_update(tables, row_off, D, unique_rows, uniq_off, codes, grad_scales, lr)
    return dict(out=out, unique_rows=unique_rows, uniq_off=uniq_off, grad_rows=grad_rows,
                codes=codes, grad_scales=grad_scales)


# ---- data-parallel exchange of the sparse INT8 gradient (Appendix B.1) -----------------
def grad_absmax(grad_rows, uniq_off, D):
    T = len(uniq_off) - 1
    out = np.empty(T, dtype=np.float32)
    gr = grad_rows if grad_rows.size else np.zeros((1, D), dtype=np.float32)
    lib().dqrm_oracle_grad_absmax(_p(gr, np.float32), _p(uniq_off, np.int32), T, int(D), _p(out, np.float32))
    return out


def grad_quant_int8_scaled(grad_rows, uniq_off, D, scales):
    T = len(uniq_off) - 1
    codes = np.empty(grad_rows.shape, dtype=np.int8)
    gr = grad_rows if grad_rows.size else np.zeros((1, D), dtype=np.float32)
    cd = codes if codes.size else np.zeros((1, D), dtype=np.int8)
    lib().dqrm_oracle_grad_quant_int8_scaled(_p(gr, np.float32), _p(uniq_off, np.int32), T, int(D),
                                             _p(np.ascontiguousarray(scales, dtype=np.float32), np.float32),
                                             _p(cd, np.int8))
    return codes


def dp_merge(rows, uoffs, codes, T, D):
    """rows[r] int32 [U_r], uoffs[r] int32 [T+1], codes[r] int8 [U_r, D] -> (union rows, off [T+1], int32 sums)"""
    W = len(rows)
    n_in = sum(len(r) for r in rows)
    out_rows = np.empty(max(n_in, 1), dtype=np.int32)
    out_off = np.empty(T + 1, dtype=np.int32)
    out_sums = np.empty((max(n_in, 1), D), dtype=np.int32)
    pad = lambda a, shape, dt: a if a.size else np.zeros(shape, dtype=dt)
    keep = [[pad(np.ascontiguousarray(r, dtype=np.int32), 1, np.int32) for r in rows],
            [np.ascontiguousarray(u, dtype=np.int32) for u in uoffs],
            [pad(np.ascontiguousarray(c, dtype=np.int8), (1, D), np.int8) for c in codes]]
    arr = lambda lst: (ctypes.c_void_p * W)(*[a.ctypes.data for a in lst])
    n = lib().dqrm_oracle_dp_merge(W, int(T), int(D), arr(keep[0]), arr(keep[1]), arr(keep[2]),
                                   _p(out_rows, np.int32), _p(out_off, np.int32), _p(out_sums, np.int32))
    return out_rows[:n].copy(), out_off, out_sums[:n].copy()


def row_update_i32(tables, row_off, D, rows, off, sums, scales, lr):
    T = len(row_off) - 1
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    r = rows if rows.size else np.zeros(1, dtype=np.int32)
    s = sums if sums.size else np.zeros((1, D), dtype=np.int32)
    lib().dqrm_oracle_row_update_i32(_p(tables, np.float32), _p(row_off, np.int64), T, int(D), _p(r, np.int32),
                                     _p(off, np.int32), _p(s, np.int32),
                                     _p(np.ascontiguousarray(scales, dtype=np.float32), np.float32),
                                     ctypes.c_float(float(np.float32(lr))))


def dp_exchange_update(tables, row_off, D, local, lr):
    """`local` = per rank (unique_rows, uniq_off, grad_rows).  Unifies the scales by max, quantises every
    rank's gradient with them, sums the codes exactly and applies the dequantised sum to `tables`
    (one replica; all replicas are identical).  Returns what the ranks would hold afterwards."""
    T = len(row_off) - 1
    absmax = np.max(np.stack([grad_absmax(g, uo, D) for (_, uo, g) in local]), axis=0)
    scales = np.array([scale_from_absmax(a, 8) for a in absmax], dtype=np.float32)
    codes = [grad_quant_int8_scaled(g, uo, D, scales) for (_, uo, g) in local]
    rows, off, sums = dp_merge([l[0] for l in local], [l[1] for l in local], codes, T, D)
    row_update_i32(tables, row_off, D, rows, off, sums, scales, lr)
    return dict(scales=scales, codes=codes, rows=rows, off=off, sums=sums)


# ---- bit-packed export and inference (Appendix C) ---------------------------------------
def pack_tables(tables, row_off, D, scales, bits):
    """-> uint8 [sum R_t, D*bits/8]"""
    T = len(row_off) - 1
    assert bits in (2, 4, 8) and (D * bits) % 8 == 0
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    packed = np.empty((tables.shape[0], D * bits // 8), dtype=np.uint8)
    lib().dqrm_oracle_pack_tables(_p(tables, np.float32), _p(row_off, np.int64), T, int(D),
                                  _p(np.ascontiguousarray(scales, dtype=np.float32), np.float32), int(bits),
                                  _p(packed, np.uint8))
    return packed


def packed_fwd(packed, row_off, D, B, indices, offsets, scales, bits):
    T = len(row_off) - 1
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    out = np.empty((B, T, D), dtype=np.float32)
    lib().dqrm_oracle_packed_fwd(_p(packed, np.uint8), _p(row_off, np.int64), T, int(D), int(B),
                                 _p(indices, np.int32), _p(offsets, np.int32),
                                 _p(np.ascontiguousarray(scales, dtype=np.float32), np.float32), int(bits),
                                 _p(out, np.float32))
    return out


def emb_fwd_codes(tables, row_off, D, B, indices, offsets, scales, bits):
    """Packed codes of every one-index bag's row -> uint8 [B, T, D*bits/8]."""
    T = len(row_off) - 1
    assert bits in (2, 4, 8) and (D * bits) % 8 == 0
    row_off = np.ascontiguousarray(row_off, dtype=np.int64)
    payload = np.empty((B, T, D * bits // 8), dtype=np.uint8)
    f = lib().dqrm_oracle_emb_fwd_codes
    f.restype = ctypes.c_int
    rc = f(_p(tables, np.float32), _p(row_off, np.int64), T, int(D), int(B), _p(indices, np.int32),
           _p(offsets, np.int32), _p(np.ascontiguousarray(scales, dtype=np.float32), np.float32), int(bits),
           _p(payload, np.uint8))
    if rc != 0:
        raise ValueError("emb_fwd_codes needs exactly one index per bag")
    return payload


def decode_payload(payload, scales, bits, D, T_total, t0, out=None):
    """out[i, t0 + j, :] = code * scales[j] for payload [B, T_blk, D*bits/8]."""
    B, T_blk = payload.shape[0], payload.shape[1]
    if out is None:
        out = np.zeros((B, T_total, D), dtype=np.float32)
    lib().dqrm_oracle_decode_payload(_p(np.ascontiguousarray(payload), np.uint8),
                                     _p(np.ascontiguousarray(scales, dtype=np.float32), np.float32), int(bits), int(B),
                                     int(T_blk), int(T_total), int(t0), int(D), _p(out, np.float32))
    return out
