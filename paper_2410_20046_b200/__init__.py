"""B200 (sm_100a) CUDA library for the embedding half of a DQRM training step
(quantisation-aware training of DLRM embedding tables, arXiv 2410.20046), and a thin
ctypes binding with the same names as the C ABI in ``include/dqrm.h``.

The binding only marshals arguments (torch tensors -> device pointers, the current
torch stream -> cudaStream_t); every step of the path runs in the library's kernels.
There is no CPU fallback: importing the binding without the built library raises.
"""
from .binding import (  # noqa: F401
    DqrmError, Context, load_library, LIB_PATH,
    OK, ERR_INVALID_ARG, ERR_WORKSPACE, ERR_CUDA, ERR_INDEX_RANGE, ERR_TIMEOUT, ERR_STATIC_LIMIT,
    STATIC_MAX_TABLES, grad_quant_int8_static,
)
