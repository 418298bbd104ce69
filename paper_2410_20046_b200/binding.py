"""ctypes binding of ``libdqrm_b200.so``: argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdqrm_b200.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_WORKSPACE = -2
ERR_CUDA = -3
ERR_INDEX_RANGE = -4
ERR_TIMEOUT = -5
ERR_STATIC_LIMIT = -6
ERR_NOT_SORTED = -7
STATIC_MAX_TABLES = 1024

_vp = ctypes.c_void_p
_i = ctypes.c_int
_i64 = ctypes.c_int64
_sz = ctypes.c_size_t
_f = ctypes.c_float

# name -> (restype, argtypes); mirrors include/dqrm.h
SIGNATURES = {
    "dqrm_create": (_i, [ctypes.POINTER(_vp), _i, _i, ctypes.POINTER(_i64)]),
    "dqrm_destroy": (_i, [_vp]),
    "dqrm_workspace_bytes": (_sz, [_vp, _i64, _i64]),
    "dqrm_check_status": (_i, [_vp, _vp]),
    "dqrm_last_cuda_error": (_i, [_vp]),
    "dqrm_status_string": (ctypes.c_char_p, [_i]),
    "dqrm_scale_refresh": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "dqrm_emb_fwd": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i64, _vp]),
    "dqrm_emb_bwd": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i64, _vp, _sz, _vp]),
    "dqrm_grad_quant_int8": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "dqrm_row_update": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _f, _vp]),
    "dqrm_sort_batch": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i64, _vp, _sz, _vp]),
    "dqrm_train_step_sorted": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _f, _i, _i64,
                                    _vp, _sz, _vp]),
    "dqrm_train_step": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _f, _i, _i64,
                             _vp, _sz, _vp]),
    "dqrm_stream_wait_forward": (_i, [_vp, _vp]),
    "dqrm_row_summary_bytes": (_sz, [_vp]),
    "dqrm_row_summary_attach": (_i, [_vp, _vp, _vp, _sz, _vp]),
    "dqrm_row_summary_detach": (_i, [_vp]),
    "dqrm_host_step_workspace_bytes": (_sz, [_vp, _i64, _i64]),
    "dqrm_train_step_host": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _f, _i, _i64, _vp, _sz, _vp]),
    "dqrm_grad_quant_int8_static": (_i, [_i, _i, _vp, _vp, _vp, _vp, _vp]),
    "dqrm_selfcheck_quantizer": (_i, [_vp, _f, _i, ctypes.c_uint32, ctypes.c_uint64, _vp, _vp]),
    "dqrm_grad_absmax": (_i, [_vp, _vp, _vp, _vp, _vp]),
    "dqrm_grad_quant_int8_unified": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dqrm_dp_workspace_bytes": (_sz, [_vp, _i64]),
    "dqrm_dp_merge_update": (_i, [_vp, _vp, _i, _i64, _vp, _vp, _vp, _vp, _f, _i64, _i64, _vp, _vp, _vp, _vp, _sz, _vp]),
    "dqrm_packed_bytes": (_sz, [_vp, _i]),
    "dqrm_pack_tables": (_i, [_vp, _vp, _vp, _i, _vp, _vp]),
    "dqrm_packed_fwd": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _i, _i64, _vp]),
    "dqrm_emb_fwd_codes": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _vp, _i, _i64, _vp]),
    "dqrm_decode_payload": (_i, [_vp, _vp, _vp, _i, _vp, _i, _i, _i, _i, _vp]),
    "dqrm_set_sort_path": (_i, [_vp, _i]),
    "dqrm_set_overlap": (_i, [_vp, _i]),
    "dqrm_launch_count": (_i64, [_vp]),
    "dqrm_profile_begin": (_i, [_vp, _vp]),
    "dqrm_profile_end": (_i, [_vp, _vp, ctypes.POINTER(_f), ctypes.POINTER(ctypes.c_int32), _i]),
    "dqrm_kernel_name": (ctypes.c_char_p, [_i]),
    "dqrm_kernel_count": (_i, []),
}

_lib = None


class DqrmError(RuntimeError):
    def __init__(self, call: str, status: int, text: str, cuda_error: int = 0):
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{call} failed: {status} {text}{extra}")
        self.status = status
        self.cuda_error = cuda_error


def load_library(path: Optional[str] = None):
    """Loads the CUDA library.  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise ImportError(
            f"{p} is missing: build it with `python -m paper_2410_20046_b200.build` "
            "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(p)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    if path is None:
        _lib = lib
    return lib


def _ptr(t, dtype=None, device="cuda"):
    """Device (or host) pointer of a contiguous torch tensor; None -> NULL."""
    if t is None:
        return None
    import torch

    assert isinstance(t, torch.Tensor), "expected a torch tensor"
    assert t.is_contiguous(), "tensor must be contiguous"
    if dtype is not None:
        assert t.dtype == dtype, f"expected {dtype}, got {t.dtype}"
    if device == "cuda":
        assert t.is_cuda, "expected a CUDA tensor"
    else:
        assert not t.is_cuda, "expected a host tensor"
    return t.data_ptr()


def _stream(stream=None):
    import torch

    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


class Context:
    """One ``dqrm_ctx`` plus a torch-allocated workspace.  Method names and argument
    order are those of the C ABI; tensors stand in for the pointers."""

    def __init__(self, row_off, D: int, max_lookups: int, max_bags: int, host_step: bool = False):
        import torch

        self.lib = load_library()
        self.T = len(row_off) - 1
        self.D = int(D)
        arr = (_i64 * (self.T + 1))(*[int(x) for x in row_off])
        h = _vp()
        rc = self.lib.dqrm_create(ctypes.byref(h), self.T, self.D, arr)
        self._h = h if rc == OK else None
        self._check("dqrm_create", rc)
        self.max_lookups = int(max_lookups)
        self.max_bags = int(max_bags)
        self.workspace_bytes = int(self.lib.dqrm_workspace_bytes(self._h, self.max_lookups, self.max_bags))
        self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device="cuda")
        self._ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        # scratch of the calls that carry nothing from one call to the next (scale refresh, gradient
        # quantiser): kept apart from the workspaces that hold a sorted batch between dqrm_sort_batch
        # and dqrm_train_step_sorted
        self.scratch_bytes = int(self.lib.dqrm_workspace_bytes(self._h, 0, 0))
        self.scratch = torch.empty(self.scratch_bytes + 256, dtype=torch.uint8, device="cuda")
        self._scratch_ptr = (self.scratch.data_ptr() + 255) // 256 * 256
        self.host_workspace = None
        if host_step:
            self.host_workspace_bytes = int(
                self.lib.dqrm_host_step_workspace_bytes(self._h, self.max_lookups, self.max_bags))
            self.host_workspace = torch.empty(self.host_workspace_bytes + 256, dtype=torch.uint8, device="cuda")
            self._hws_ptr = (self.host_workspace.data_ptr() + 255) // 256 * 256

    # ---- plumbing ----
    def _check(self, call: str, rc: int):
        if rc != OK:
            text = self.lib.dqrm_status_string(rc).decode()
            ce = self.lib.dqrm_last_cuda_error(self._h) if self._h else 0
            raise DqrmError(call, rc, text, ce)

    def close(self):
        if getattr(self, "_h", None):
            self.lib.dqrm_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check_status(self, stream=None) -> int:
        return int(self.lib.dqrm_check_status(self._h, _stream(stream)))

    def raise_on_device_error(self, stream=None):
        self._check("dqrm_check_status", self.check_status(stream))

    def selfcheck_quantizer(self, scale, bits, first_bits, count, mismatches, stream=None):
        import torch

        self._check("dqrm_selfcheck_quantizer", self.lib.dqrm_selfcheck_quantizer(
            self._h, float(scale), int(bits), int(first_bits) & 0xFFFFFFFF, int(count),
            _ptr(mismatches, torch.int64), _stream(stream)))

    # ---- data-parallel exchange (local pieces) ----
    def grad_absmax(self, grad_rows, uniq_off, absmax, stream=None):
        import torch

        self._check("dqrm_grad_absmax", self.lib.dqrm_grad_absmax(
            self._h, _ptr(grad_rows, torch.float32), _ptr(uniq_off, torch.int32), _ptr(absmax, torch.float32),
            _stream(stream)))

    def grad_quant_int8_unified(self, grad_rows, uniq_off, unified_absmax, codes, grad_scales, stream=None):
        import torch

        self._check("dqrm_grad_quant_int8_unified", self.lib.dqrm_grad_quant_int8_unified(
            self._h, _ptr(grad_rows, torch.float32), _ptr(uniq_off, torch.int32), _ptr(unified_absmax, torch.float32),
            _ptr(codes, torch.int8), _ptr(grad_scales, torch.float32), _stream(stream)))

    def dp_workspace(self, max_entries: int):
        """torch-allocated, 256-byte aligned workspace for dp_merge_update -> (tensor, pointer, bytes)"""
        import torch

        n = int(self.lib.dqrm_dp_workspace_bytes(self._h, int(max_entries)))
        buf = torch.empty(n + 256, dtype=torch.uint8, device="cuda")
        return buf, (buf.data_ptr() + 255) // 256 * 256, n

    def dp_merge_update(self, tables, W, rank_stride, rows_cat, uoff_cat, codes_cat, grad_scales, lr, n_entries,
                        max_table_entries, union_rows, union_off, sums_out, ws, stream=None):
        import torch

        _, ws_ptr, ws_bytes = ws
        self._check("dqrm_dp_merge_update", self.lib.dqrm_dp_merge_update(
            self._h, _ptr(tables, torch.float32), int(W), int(rank_stride), _ptr(rows_cat, torch.int32),
            _ptr(uoff_cat, torch.int32), _ptr(codes_cat, torch.int8), _ptr(grad_scales, torch.float32), float(lr),
            int(n_entries), int(max_table_entries), _ptr(union_rows, torch.int32), _ptr(union_off, torch.int32),
            _ptr(sums_out, torch.int32), ws_ptr, ws_bytes, _stream(stream)))

    # ---- bit-packed export and inference ----
    def packed_bytes(self, bits: int) -> int:
        return int(self.lib.dqrm_packed_bytes(self._h, int(bits)))

    def pack_tables(self, tables, scales, bits, packed, stream=None):
        import torch

        self._check("dqrm_pack_tables", self.lib.dqrm_pack_tables(
            self._h, _ptr(tables, torch.float32), _ptr(scales, torch.float32), int(bits), _ptr(packed, torch.uint8),
            _stream(stream)))

    def packed_fwd(self, packed, indices, offsets, scales, bits, out, *, B, L, stream=None):
        import torch

        self._check("dqrm_packed_fwd", self.lib.dqrm_packed_fwd(
            self._h, _ptr(packed, torch.uint8), _ptr(indices, torch.int32), _ptr(offsets, torch.int32),
            _ptr(scales, torch.float32), int(bits), _ptr(out, torch.float32), int(B), int(L), _stream(stream)))

    # ---- table-sharded forward payload ----
    def emb_fwd_codes(self, tables, indices, offsets, scales, bits, payload, *, B, L, stream=None):
        import torch

        self._check("dqrm_emb_fwd_codes", self.lib.dqrm_emb_fwd_codes(
            self._h, _ptr(tables, torch.float32), _ptr(indices, torch.int32), _ptr(offsets, torch.int32),
            _ptr(scales, torch.float32), int(bits), _ptr(payload, torch.uint8), int(B), int(L), _stream(stream)))

    def decode_payload(self, payload, scales, bits, out, *, B, T_blk, T_total, t0, stream=None):
        import torch

        self._check("dqrm_decode_payload", self.lib.dqrm_decode_payload(
            self._h, _ptr(payload, torch.uint8), _ptr(scales, torch.float32), int(bits), _ptr(out, torch.float32),
            int(B), int(T_blk), int(T_total), int(t0), _stream(stream)))

    def set_overlap(self, on: bool):
        self._check("dqrm_set_overlap", self.lib.dqrm_set_overlap(self._h, int(bool(on))))

    def set_sort_path(self, path: int):
        self._check("dqrm_set_sort_path", self.lib.dqrm_set_sort_path(self._h, int(path)))

    def launch_count(self) -> int:
        return int(self.lib.dqrm_launch_count(self._h))

    def profile_begin(self, stream=None):
        self._check("dqrm_profile_begin", self.lib.dqrm_profile_begin(self._h, _stream(stream)))

    def profile_end(self, stream=None):
        """-> {kernel name: (milliseconds, launches)} for the launches since profile_begin"""
        n = int(self.lib.dqrm_kernel_count())
        ms = (_f * n)()
        cnt = (ctypes.c_int32 * n)()
        self._check("dqrm_profile_end", self.lib.dqrm_profile_end(self._h, _stream(stream), ms, cnt, n))
        return {self.lib.dqrm_kernel_name(k).decode(): (float(ms[k]), int(cnt[k])) for k in range(n) if cnt[k]}

    # ---- the calls of include/dqrm.h ----
    def scale_refresh(self, tables, bits, scales, minmax=None, stream=None):
        import torch

        self._check("dqrm_scale_refresh", self.lib.dqrm_scale_refresh(
            self._h, _ptr(tables, torch.float32), _ptr(bits, torch.int32), _ptr(scales, torch.float32),
            _ptr(minmax, torch.float32), self._scratch_ptr, self.scratch_bytes, _stream(stream)))

    def emb_fwd(self, tables, indices, offsets, scales, bits, out, codes_out=None, *, B, L, stream=None):
        import torch

        self._check("dqrm_emb_fwd", self.lib.dqrm_emb_fwd(
            self._h, _ptr(tables, torch.float32), _ptr(indices, torch.int32), _ptr(offsets, torch.int32),
            _ptr(scales, torch.float32), _ptr(bits, torch.int32), _ptr(out, torch.float32),
            _ptr(codes_out, torch.int8), int(B), int(L), _stream(stream)))

    def emb_bwd(self, grad_out, indices, offsets, unique_rows, uniq_off, grad_rows, *, B, L, stream=None):
        import torch

        self._check("dqrm_emb_bwd", self.lib.dqrm_emb_bwd(
            self._h, _ptr(grad_out, torch.float32), _ptr(indices, torch.int32), _ptr(offsets, torch.int32),
            _ptr(unique_rows, torch.int32), _ptr(uniq_off, torch.int32), _ptr(grad_rows, torch.float32),
            int(B), int(L), self._ws_ptr, self.workspace_bytes, _stream(stream)))

    def grad_quant_int8(self, grad_rows, uniq_off, codes, grad_scales, stream=None):
        import torch

        self._check("dqrm_grad_quant_int8", self.lib.dqrm_grad_quant_int8(
            self._h, _ptr(grad_rows, torch.float32), _ptr(uniq_off, torch.int32), _ptr(codes, torch.int8),
            _ptr(grad_scales, torch.float32), self._scratch_ptr, self.scratch_bytes, _stream(stream)))

    def row_update(self, tables, unique_rows, uniq_off, codes, grad_scales, lr, stream=None):
        import torch

        self._check("dqrm_row_update", self.lib.dqrm_row_update(
            self._h, _ptr(tables, torch.float32), _ptr(unique_rows, torch.int32), _ptr(uniq_off, torch.int32),
            _ptr(codes, torch.int8), _ptr(grad_scales, torch.float32), float(lr), _stream(stream)))

    def train_step(self, tables, indices, offsets, grad_out, scales, bits, out, unique_rows, uniq_off,
                   grad_rows, codes, grad_scales, lr, *, B, L, stream=None):
        import torch

        self._check("dqrm_train_step", self.lib.dqrm_train_step(
            self._h, _ptr(tables, torch.float32), _ptr(indices, torch.int32), _ptr(offsets, torch.int32),
            _ptr(grad_out, torch.float32), _ptr(scales, torch.float32), _ptr(bits, torch.int32),
            _ptr(out, torch.float32), _ptr(unique_rows, torch.int32), _ptr(uniq_off, torch.int32),
            _ptr(grad_rows, torch.float32), _ptr(codes, torch.int8), _ptr(grad_scales, torch.float32),
            float(lr), int(B), int(L), self._ws_ptr, self.workspace_bytes, _stream(stream)))

    # ---- the step in two calls; `ws` picks a workspace (number 0 exists, the others are made on first use) ----
    def _workspace(self, ws: int) -> int:
        import torch

        if ws == 0:
            return self._ws_ptr
        more = self.__dict__.setdefault("_more_workspaces", {})
        if ws not in more:
            buf = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device="cuda")
            more[ws] = (buf, (buf.data_ptr() + 255) // 256 * 256)
        return more[ws][1]

    def sort_batch(self, indices, offsets, unique_rows, uniq_off, *, B, L, ws=0, stream=None):
        import torch

        self._check("dqrm_sort_batch", self.lib.dqrm_sort_batch(
            self._h, _ptr(indices, torch.int32), _ptr(offsets, torch.int32), _ptr(unique_rows, torch.int32),
            _ptr(uniq_off, torch.int32), int(B), int(L), self._workspace(ws), self.workspace_bytes, _stream(stream)))

    def train_step_sorted(self, tables, indices, offsets, grad_out, scales, bits, out, unique_rows, uniq_off,
                          grad_rows, codes, grad_scales, lr, *, B, L, ws=0, stream=None):
        import torch

        self._check("dqrm_train_step_sorted", self.lib.dqrm_train_step_sorted(
            self._h, _ptr(tables, torch.float32), _ptr(indices, torch.int32), _ptr(offsets, torch.int32),
            _ptr(grad_out, torch.float32), _ptr(scales, torch.float32), _ptr(bits, torch.int32),
            _ptr(out, torch.float32), _ptr(unique_rows, torch.int32), _ptr(uniq_off, torch.int32),
            _ptr(grad_rows, torch.float32), _ptr(codes, torch.int8), _ptr(grad_scales, torch.float32),
            float(lr), int(B), int(L), self._workspace(ws), self.workspace_bytes, _stream(stream)))

    def stream_wait_forward(self, stream):
        self._check("dqrm_stream_wait_forward", self.lib.dqrm_stream_wait_forward(self._h, _stream(stream)))

    def row_summary_attach(self, tables, stream=None):
        """Allocates the per-row (min, max) buffer, fills it from `tables` and attaches it."""
        import torch

        n = int(self.lib.dqrm_row_summary_bytes(self._h))
        self.row_summary = torch.empty(max(n, 8) // 4, dtype=torch.float32, device=tables.device)
        self._check("dqrm_row_summary_attach", self.lib.dqrm_row_summary_attach(
            self._h, _ptr(tables), _ptr(self.row_summary), n, _stream(stream)))
        return self.row_summary

    def row_summary_detach(self):
        self._check("dqrm_row_summary_detach", self.lib.dqrm_row_summary_detach(self._h))
        self.row_summary = None

    def train_step_host(self, tables, h_indices, h_offsets, h_grad_out, scales, bits, h_out, lr, *, B, L,
                        stream=None):
        import torch

        assert self.host_workspace is not None, "create the Context with host_step=True"
        self._check("dqrm_train_step_host", self.lib.dqrm_train_step_host(
            self._h, _ptr(tables, torch.float32), _ptr(h_indices, torch.int32, "cpu"),
            _ptr(h_offsets, torch.int32, "cpu"), _ptr(h_grad_out, torch.float32, "cpu"),
            _ptr(scales, torch.float32), _ptr(bits, torch.int32), _ptr(h_out, torch.float32, "cpu"),
            float(lr), int(B), int(L), self._hws_ptr, self.host_workspace_bytes, _stream(stream)))


def grad_quant_int8_static(T, D, grad_rows, uniq_off, codes, grad_scales, stream=None) -> int:
    """``dqrm_grad_quant_int8_static``: the gradient quantiser for callers that must not
    allocate device memory (no context, no workspace; scratch is a fixed array inside the
    library).  Returns the status code instead of raising, so that the size limit can be
    handled by the caller."""
    import torch

    lib = load_library()
    return int(lib.dqrm_grad_quant_int8_static(
        int(T), int(D), _ptr(grad_rows, torch.float32), _ptr(uniq_off, torch.int32), _ptr(codes, torch.int8),
        _ptr(grad_scales, torch.float32), _stream(stream)))
