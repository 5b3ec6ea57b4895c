"""Python binding of the LLVQ CUDA library (``include/llvq.h``).

Argument marshalling only: every step of the dequantization path runs in the
CUDA kernels of ``libllvq.so``.  PyTorch is used for device memory and streams.
There is no CPU fallback: if the library is missing or the device is not a CUDA
device, calls raise.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .build import LIB

__all__ = [
    "Context", "llvq_decode_blocks", "llvq_dequant_matrix", "llvq_gemv", "llvq_gemm_small_batch", "llvq_gemm_small_batch_noalloc",
    "llvq_dequant_matrix_sg", "llvq_gemv_sg",
    "llvq_encode_blocks", "llvq_rank_blocks", "llvq_pack_fields", "LLVQ_EUCLIDEAN", "LLVQ_ANGULAR",
    "llvq_sort_blocks", "llvq_gemv_sorted", "llvq_sort_blocks_gemm", "llvq_gemm_small_batch_sorted",
    "llvq_sort_blocks_sg", "llvq_gemv_sorted_sg", "llvq_gemm_small_batch_sg",
    "llvq_gemv_rowshard", "llvq_gemv_sorted_rowshard", "llvq_exchange_create", "llvq_exchange_destroy", "llvq_exchange_open",
    "llvq_exchange_close", "llvq_signal_ranks", "llvq_wait_ranks", "LLVQ_EXCHANGE_HANDLE_BYTES",
    "llvq_gemm_small_batch_rowshard", "llvq_gemm_small_batch_sorted_rowshard",
    "llvq_sort_blocks_gemm_sg", "llvq_gemm_small_batch_sorted_sg",
    "llvq_last_error", "LlvqError", "EXPORTS", "load_library", "llvq_gemv_multi", "llvq_gemv_sorted_multi", "GemvDesc",
    "LLVQ_LAYOUT_FLAT", "LLVQ_LAYOUT_ROWWISE", "LLVQ_F32", "LLVQ_BF16",
]

LLVQ_LAYOUT_FLAT, LLVQ_LAYOUT_ROWWISE = 0, 1
LLVQ_F32, LLVQ_BF16 = 0, 1
LLVQ_EUCLIDEAN, LLVQ_ANGULAR = 0, 1
LLVQ_FLAG_WAIT_TIMEOUT, LLVQ_FLAG_SEARCH_GAVE_UP = 1, 4
LLVQ_EXCHANGE_HANDLE_BYTES = 64
_STATUS = {0: "LLVQ_OK", 1: "LLVQ_EINVAL", 2: "LLVQ_EALIGN", 3: "LLVQ_EUNSUPPORTED", 4: "LLVQ_ECUDA",
           5: "LLVQ_EINDEX", 6: "LLVQ_ETIMEOUT"}

# every symbol include/llvq.h declares
EXPORTS = [
    "llvq_create", "llvq_destroy", "llvq_index_bits", "llvq_num_points", "llvq_num_classes", "llvq_index_bytes",
    "llvq_decode_blocks", "llvq_dequant_matrix", "llvq_gemv", "llvq_gemm_small_batch", "llvq_gemm_small_batch_noalloc",
    "llvq_selftest_wait_timeout", "llvq_last_error",
    "llvq_field_bytes", "llvq_dequant_matrix_sg", "llvq_gemv_sg", "llvq_class_info", "llvq_golay_table",
    "llvq_encode_blocks", "llvq_rank_blocks", "llvq_pack_fields",
    "llvq_sorted_bytes", "llvq_sort_blocks", "llvq_gemv_sorted", "llvq_sort_blocks_sg", "llvq_gemv_sorted_sg",
    "llvq_sorted_gemm_bytes", "llvq_sort_blocks_gemm", "llvq_gemm_small_batch_sorted", "llvq_gemm_small_batch_sg",
    "llvq_gemv_rowshard", "llvq_gemv_sorted_rowshard", "llvq_exchange_create", "llvq_exchange_destroy", "llvq_exchange_open",
    "llvq_exchange_close", "llvq_signal_ranks", "llvq_wait_ranks",
    "llvq_gemm_small_batch_rowshard", "llvq_gemm_small_batch_sorted_rowshard",
    "llvq_sort_blocks_gemm_sg", "llvq_gemm_small_batch_sorted_sg",
    "llvq_gemv_multi", "llvq_gemv_sorted_multi",
]


class LlvqError(RuntimeError):
    def __init__(self, call: str, status: int):
        super().__init__(f"{call} failed: {_STATUS.get(status, status)}")
        self.status = status


_lib = None


class GemvDesc(ctypes.Structure):
    """llvq_gemv_desc of include/llvq.h: one matrix of a multi-matrix GEMV call."""
    _fields_ = [("d_weights", ctypes.c_void_p), ("d_gain_f16", ctypes.c_void_p), ("n_out", ctypes.c_int64), ("k_in", ctypes.c_int64),
                ("d_x_bf16", ctypes.c_void_p), ("d_y", ctypes.c_void_p)]


def load_library() -> ctypes.CDLL:
    """Load libllvq.so (built in-tree by ``paper_2603_11021_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB):
        raise ImportError(f"{LIB} not found: run `python -m paper_2603_11021_b200.build` (needs nvcc); there is no fallback path")
    lib = ctypes.CDLL(LIB)
    vp, i64, u64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64
    lib.llvq_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, ctypes.c_int]
    lib.llvq_destroy.argtypes = [vp]
    lib.llvq_destroy.restype = None
    lib.llvq_index_bits.argtypes = [vp]
    lib.llvq_num_points.argtypes = [vp, ctypes.POINTER(u64)]
    lib.llvq_num_classes.argtypes = [vp]
    lib.llvq_index_bytes.argtypes = [vp, u64]
    lib.llvq_index_bytes.restype = ctypes.c_size_t
    lib.llvq_decode_blocks.argtypes = [vp, vp, u64, vp, vp]
    lib.llvq_dequant_matrix.argtypes = [vp, vp, vp, i64, i64, ctypes.c_int, vp, i64, vp]
    lib.llvq_gemv.argtypes = [vp, vp, vp, i64, i64, vp, vp, ctypes.c_int, vp]
    lib.llvq_gemm_small_batch.argtypes = [vp, vp, vp, i64, i64, vp, ctypes.c_int, vp, vp]
    lib.llvq_gemm_small_batch_noalloc.argtypes = [vp, vp, vp, i64, i64, vp, ctypes.c_int, vp, vp]
    lib.llvq_selftest_wait_timeout.argtypes = [vp, vp]
    lib.llvq_field_bytes.argtypes = [vp, u64, ctypes.c_int]
    lib.llvq_field_bytes.restype = ctypes.c_size_t
    lib.llvq_dequant_matrix_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp, i64, vp]
    lib.llvq_gemv_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp, vp, ctypes.c_int, vp]
    lib.llvq_sorted_bytes.argtypes = [vp, i64, i64]
    lib.llvq_sorted_bytes.restype = ctypes.c_size_t
    lib.llvq_sort_blocks.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.llvq_gemv_sorted.argtypes = [vp, vp, vp, i64, i64, vp, vp, ctypes.c_int, vp]
    lib.llvq_gemv_multi.argtypes = [vp, ctypes.POINTER(GemvDesc), ctypes.c_int, ctypes.c_int, vp]
    lib.llvq_gemv_sorted_multi.argtypes = [vp, ctypes.POINTER(GemvDesc), ctypes.c_int, ctypes.c_int, vp]
    lib.llvq_gemm_small_batch_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp, ctypes.c_int, vp, vp]
    lib.llvq_sort_blocks_gemm_sg.argtypes = [vp, vp, ctypes.c_int, i64, i64, vp, vp]
    lib.llvq_gemm_small_batch_sorted_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp, ctypes.c_int, vp, vp]
    lib.llvq_sort_blocks_sg.argtypes = [vp, vp, ctypes.c_int, i64, i64, vp, vp]
    lib.llvq_gemv_sorted_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp, vp, ctypes.c_int, vp]
    lib.llvq_sorted_gemm_bytes.argtypes = [vp, i64, i64]
    lib.llvq_sorted_gemm_bytes.restype = ctypes.c_size_t
    lib.llvq_sort_blocks_gemm.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.llvq_gemm_small_batch_sorted.argtypes = [vp, vp, vp, i64, i64, vp, ctypes.c_int, vp, vp]
    lib.llvq_encode_blocks.argtypes = [vp, vp, u64, ctypes.c_int, vp, vp, vp]
    lib.llvq_rank_blocks.argtypes = [vp, vp, u64, vp, vp]
    lib.llvq_pack_fields.argtypes = [vp, vp, vp, ctypes.c_int, u64, vp, vp]
    lib.llvq_last_error.argtypes = [vp, vp, ctypes.POINTER(u64), ctypes.POINTER(ctypes.c_uint32)]
    lib.llvq_class_info.argtypes = [vp, ctypes.c_int, vp, vp, vp, vp, vp, vp]
    lib.llvq_golay_table.argtypes = [vp, vp]
    shard = [vp, vp, vp, i64, i64, vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, i64, ctypes.c_int, ctypes.POINTER(vp),
             ctypes.c_uint32, vp]
    lib.llvq_gemv_rowshard.argtypes = shard
    lib.llvq_gemv_sorted_rowshard.argtypes = shard
    gshard = [vp, vp, vp, i64, i64, vp, ctypes.c_int, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, i64, i64, ctypes.POINTER(vp),
              ctypes.c_uint32, vp]
    lib.llvq_gemm_small_batch_rowshard.argtypes = gshard
    lib.llvq_gemm_small_batch_sorted_rowshard.argtypes = gshard
    lib.llvq_exchange_create.argtypes = [vp, ctypes.c_size_t, ctypes.POINTER(vp), ctypes.c_char_p]
    lib.llvq_exchange_destroy.argtypes = [vp, vp]
    lib.llvq_exchange_open.argtypes = [vp, ctypes.c_char_p, ctypes.POINTER(vp)]
    lib.llvq_exchange_close.argtypes = [vp, vp]
    lib.llvq_signal_ranks.argtypes = [vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_uint32, vp]
    lib.llvq_wait_ranks.argtypes = [vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_uint32, ctypes.c_uint32, vp]
    _lib = lib
    return lib


def _check(call: str, status: int) -> None:
    if status != 0:
        raise LlvqError(call, status)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev(t: torch.Tensor, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor")
    return t.data_ptr()


class Context:
    """Tables of the code  union of Shell(m), m_lo <= m <= m_hi,  on one CUDA device."""

    def __init__(self, m_lo: int, m_hi: int, device: int = 0):
        self._lib = load_library()
        h = ctypes.c_void_p()
        _check("llvq_create", self._lib.llvq_create(ctypes.byref(h), m_lo, m_hi, device))
        self._h = h
        self.device = device
        self.m_lo, self.m_hi = m_lo, m_hi
        self.index_bits = int(self._lib.llvq_index_bits(h))
        out = (ctypes.c_uint64 * 2)()
        _check("llvq_num_points", self._lib.llvq_num_points(h, out))
        self.num_points = (int(out[1]) << 64) | int(out[0])
        self.num_classes = int(self._lib.llvq_num_classes(h))

    def index_bytes(self, nblocks: int) -> int:
        return int(self._lib.llvq_index_bytes(self._h, nblocks))

    def class_info(self, j: int) -> dict:
        """Host-side description of class j as the library's own table generator built it."""
        import numpy as np
        info = np.zeros(5, dtype=np.int32)
        A = np.zeros(1, dtype=np.uint64)
        card = np.zeros(2, dtype=np.uint64)
        off = np.zeros(2, dtype=np.uint64)
        vals = np.zeros(24, dtype=np.int32)
        mults = np.zeros(24, dtype=np.int32)
        p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
        _check("llvq_class_info", self._lib.llvq_class_info(self._h, j, p(info), p(A), p(card), p(off), p(vals), p(mults)))
        nv = int(info[4])
        return {"m": int(info[0]), "parity": int(info[1]), "w": int(info[2]), "B": int(info[3]), "A": int(A[0]),
                "card": (int(card[1]) << 64) | int(card[0]), "offset": (int(off[1]) << 64) | int(off[0]),
                "values": [int(v) for v in vals[:nv]], "mults": [int(v) for v in mults[:nv]]}

    def golay_table(self):
        import numpy as np
        out = np.zeros(4096, dtype=np.uint32)
        _check("llvq_golay_table", self._lib.llvq_golay_table(self._h, out.ctypes.data_as(ctypes.c_void_p)))
        return out

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.llvq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def llvq_decode_blocks(ctx: Context, d_idx: torch.Tensor, nblocks: int, d_points: torch.Tensor | None = None, stream=None):
    """int8 [nblocks, 24] lattice points of the fields of the index stream ``d_idx`` (uint8, CUDA)."""
    if d_points is None:
        d_points = torch.empty((nblocks, 24), dtype=torch.int8, device=d_idx.device)
    assert d_points.dtype == torch.int8 and d_points.numel() >= nblocks * 24
    assert d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(nblocks)
    _check("llvq_decode_blocks", ctx._lib.llvq_decode_blocks(ctx._h, _dev(d_idx, "d_idx"), nblocks, _dev(d_points, "d_points"), _stream_ptr(stream)))
    return d_points


def llvq_dequant_matrix(ctx: Context, d_idx: torch.Tensor, d_gain: torch.Tensor, rows: int, cols: int, layout: int,
                        d_w: torch.Tensor | None = None, ld: int | None = None, stream=None):
    """bf16 [rows, cols] dequantized weights; ``d_gain`` is float16 [nblocks]."""
    ld = cols if ld is None else ld
    if d_w is None:
        d_w = torch.empty((rows, ld), dtype=torch.bfloat16, device=d_idx.device)
    assert d_w.dtype == torch.bfloat16 and d_gain.dtype == torch.float16
    nblocks = (rows * cols + 23) // 24 if layout == LLVQ_LAYOUT_FLAT else rows * ((cols + 23) // 24)
    assert d_gain.numel() >= nblocks and d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(nblocks)
    assert d_w.numel() >= (rows - 1) * ld + cols if rows else True
    _check("llvq_dequant_matrix", ctx._lib.llvq_dequant_matrix(
        ctx._h, _dev(d_idx, "d_idx"), _dev(d_gain, "d_gain"), rows, cols, layout, _dev(d_w, "d_w"), ld, _stream_ptr(stream)))
    return d_w


def llvq_gemv(ctx: Context, d_idx: torch.Tensor, d_gain: torch.Tensor, n_out: int, k_in: int, d_x: torch.Tensor,
              d_y: torch.Tensor | None = None, y_dtype: torch.dtype = torch.float32, stream=None):
    """y = W x with W given by (index stream, gains), ROWWISE blocks; x bf16 [k_in]; y float32 or bf16 [n_out]."""
    if d_y is None:
        d_y = torch.empty(n_out, dtype=y_dtype, device=d_idx.device)
    assert d_x.dtype == torch.bfloat16 and d_x.numel() >= k_in and d_gain.dtype == torch.float16
    assert d_y.dtype in (torch.float32, torch.bfloat16) and d_y.numel() >= n_out
    nblocks = n_out * ((k_in + 23) // 24)
    assert d_gain.numel() >= nblocks and d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(nblocks)
    code = LLVQ_F32 if d_y.dtype == torch.float32 else LLVQ_BF16
    _check("llvq_gemv", ctx._lib.llvq_gemv(ctx._h, _dev(d_idx, "d_idx"), _dev(d_gain, "d_gain"), n_out, k_in,
                                           _dev(d_x, "d_x"), _dev(d_y, "d_y"), code, _stream_ptr(stream)))
    return d_y


def _sg_args(ctx: Context, d_fields, gain_bits: int, d_codebook, d_row_scale, rows: int, nblocks: int):
    assert d_codebook.dtype == torch.float32 and d_codebook.numel() >= (1 << gain_bits)
    assert d_row_scale is None or (d_row_scale.dtype == torch.float32 and d_row_scale.numel() >= rows)
    assert d_fields.numel() * d_fields.element_size() >= int(ctx._lib.llvq_field_bytes(ctx._h, nblocks, gain_bits))
    return _dev(d_codebook, "d_codebook"), (None if d_row_scale is None else _dev(d_row_scale, "d_row_scale"))


def llvq_dequant_matrix_sg(ctx: Context, d_fields: torch.Tensor, gain_bits: int, d_codebook: torch.Tensor,
                           d_row_scale: torch.Tensor | None, rows: int, cols: int,
                           d_w: torch.Tensor | None = None, ld: int | None = None, stream=None):
    """bf16 [rows, cols] weights of the shape-gain form: (row_scale * codebook[k]) * x / |x|, ROWWISE fields
    (shape index | gain index << index_bits); ``d_row_scale`` may be None."""
    ld = cols if ld is None else ld
    if d_w is None:
        d_w = torch.empty((rows, ld), dtype=torch.bfloat16, device=d_fields.device)
    assert d_w.dtype == torch.bfloat16
    assert d_w.numel() >= (rows - 1) * ld + cols if rows else True
    cb, rs = _sg_args(ctx, d_fields, gain_bits, d_codebook, d_row_scale, rows, rows * ((cols + 23) // 24))
    _check("llvq_dequant_matrix_sg", ctx._lib.llvq_dequant_matrix_sg(
        ctx._h, _dev(d_fields, "d_fields"), gain_bits, cb, rs, rows, cols, _dev(d_w, "d_w"), ld, _stream_ptr(stream)))
    return d_w


def llvq_gemv_sg(ctx: Context, d_fields: torch.Tensor, gain_bits: int, d_codebook: torch.Tensor,
                 d_row_scale: torch.Tensor | None, n_out: int, k_in: int, d_x: torch.Tensor,
                 d_y: torch.Tensor | None = None, y_dtype: torch.dtype = torch.float32, stream=None):
    """y = W x with W in the shape-gain form of ``llvq_dequant_matrix_sg``."""
    if d_y is None:
        d_y = torch.empty(n_out, dtype=y_dtype, device=d_fields.device)
    assert d_x.dtype == torch.bfloat16 and d_x.numel() >= k_in
    assert d_y.dtype in (torch.float32, torch.bfloat16) and d_y.numel() >= n_out
    cb, rs = _sg_args(ctx, d_fields, gain_bits, d_codebook, d_row_scale, n_out, n_out * ((k_in + 23) // 24))
    code = LLVQ_F32 if d_y.dtype == torch.float32 else LLVQ_BF16
    _check("llvq_gemv_sg", ctx._lib.llvq_gemv_sg(ctx._h, _dev(d_fields, "d_fields"), gain_bits, cb, rs, n_out, k_in,
                                                 _dev(d_x, "d_x"), _dev(d_y, "d_y"), code, _stream_ptr(stream)))
    return d_y


def llvq_gemm_small_batch_sg(ctx: Context, d_fields: torch.Tensor, gain_bits: int, d_codebook: torch.Tensor,
                             d_row_scale: torch.Tensor | None, n_out: int, k_in: int, d_x: torch.Tensor,
                             d_y: torch.Tensor | None = None, stream=None):
    """Y[b, i] = sum_k X[b, k] W[i, k] with W in the shape-gain form of ``llvq_dequant_matrix_sg``; batch <= 64."""
    assert d_x.dtype == torch.bfloat16 and d_x.dim() == 2 and d_x.shape[1] == k_in
    batch = d_x.shape[0]
    if d_y is None:
        d_y = torch.empty((batch, n_out), dtype=torch.bfloat16, device=d_fields.device)
    assert d_y.dtype == torch.bfloat16 and d_y.numel() >= batch * n_out
    cb, rs = _sg_args(ctx, d_fields, gain_bits, d_codebook, d_row_scale, n_out, n_out * ((k_in + 23) // 24))
    _check("llvq_gemm_small_batch_sg", ctx._lib.llvq_gemm_small_batch_sg(
        ctx._h, _dev(d_fields, "d_fields"), gain_bits, cb, rs, n_out, k_in, _dev(d_x, "d_x"), batch, _dev(d_y, "d_y"), _stream_ptr(stream)))
    return d_y


def llvq_gemm_small_batch(ctx: Context, d_idx: torch.Tensor, d_gain: torch.Tensor, n_out: int, k_in: int,
                          d_x: torch.Tensor, d_y: torch.Tensor | None = None, stream=None):
    """Y[b, i] = sum_k X[b, k] W[i, k]; X bf16 [batch, k_in], Y bf16 [batch, n_out], batch <= 64."""
    assert d_x.dtype == torch.bfloat16 and d_x.dim() == 2 and d_x.shape[1] == k_in and d_gain.dtype == torch.float16
    batch = d_x.shape[0]
    if d_y is None:
        d_y = torch.empty((batch, n_out), dtype=torch.bfloat16, device=d_idx.device)
    assert d_y.dtype == torch.bfloat16 and d_y.numel() >= batch * n_out
    nblocks = n_out * ((k_in + 23) // 24)
    assert d_gain.numel() >= nblocks and d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(nblocks)
    _check("llvq_gemm_small_batch", ctx._lib.llvq_gemm_small_batch(
        ctx._h, _dev(d_idx, "d_idx"), _dev(d_gain, "d_gain"), n_out, k_in, _dev(d_x, "d_x"), batch, _dev(d_y, "d_y"), _stream_ptr(stream)))
    return d_y


def llvq_gemm_small_batch_noalloc(ctx: Context, d_idx: torch.Tensor, d_gain: torch.Tensor, n_out: int, k_in: int,
                                  d_x: torch.Tensor, d_y: torch.Tensor, stream=None):
    """Same product as ``llvq_gemm_small_batch`` for callers that must not allocate device memory: the
    library uses a fixed built-in scratch array instead of allocated memory, and this wrapper does not allocate
    either, so the output tensor ``d_y`` (bf16 [batch, n_out]) has to be passed in.  Sizes beyond the built-in
    array (see ``include/llvq.h``) raise ``LlvqError`` with LLVQ_EUNSUPPORTED.  Calls must not overlap on the GPU."""
    assert d_x.dtype == torch.bfloat16 and d_x.dim() == 2 and d_x.shape[1] == k_in and d_gain.dtype == torch.float16
    batch = d_x.shape[0]
    assert d_y.dtype == torch.bfloat16 and d_y.numel() >= batch * n_out
    _check("llvq_gemm_small_batch_noalloc", ctx._lib.llvq_gemm_small_batch_noalloc(
        ctx._h, _dev(d_idx, "d_idx"), _dev(d_gain, "d_gain"), n_out, k_in, _dev(d_x, "d_x"), batch, _dev(d_y, "d_y"), _stream_ptr(stream)))
    return d_y


def llvq_sort_blocks(ctx: Context, d_idx: torch.Tensor, n_out: int, k_in: int, d_sorted: torch.Tensor | None = None, stream=None):
    """Rewrite a ROWWISE index stream into the sorted layout of ``llvq_gemv_sorted`` (done once per matrix, per device)."""
    nbytes = int(ctx._lib.llvq_sorted_bytes(ctx._h, n_out, k_in))
    if nbytes == 0:
        raise LlvqError("llvq_sorted_bytes", 3)
    if d_sorted is None:
        d_sorted = torch.empty(nbytes, dtype=torch.uint8, device=d_idx.device)
    assert d_sorted.numel() * d_sorted.element_size() >= nbytes
    assert d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(n_out * ((k_in + 23) // 24))
    _check("llvq_sort_blocks", ctx._lib.llvq_sort_blocks(ctx._h, _dev(d_idx, "d_idx"), n_out, k_in, _dev(d_sorted, "d_sorted"), _stream_ptr(stream)))
    return d_sorted


def llvq_gemv_sorted(ctx: Context, d_sorted: torch.Tensor, d_gain: torch.Tensor, n_out: int, k_in: int, d_x: torch.Tensor,
                     d_y: torch.Tensor | None = None, y_dtype: torch.dtype = torch.float32, stream=None):
    """y = W x from the sorted stream of ``llvq_sort_blocks`` and the ROWWISE gains; same result as ``llvq_gemv``."""
    if d_y is None:
        d_y = torch.empty(n_out, dtype=y_dtype, device=d_sorted.device)
    assert d_x.dtype == torch.bfloat16 and d_x.numel() >= k_in and d_gain.dtype == torch.float16
    assert d_y.dtype in (torch.float32, torch.bfloat16) and d_y.numel() >= n_out
    assert d_gain.numel() >= n_out * ((k_in + 23) // 24)
    assert d_sorted.numel() * d_sorted.element_size() >= int(ctx._lib.llvq_sorted_bytes(ctx._h, n_out, k_in))
    code = LLVQ_F32 if d_y.dtype == torch.float32 else LLVQ_BF16
    _check("llvq_gemv_sorted", ctx._lib.llvq_gemv_sorted(ctx._h, _dev(d_sorted, "d_sorted"), _dev(d_gain, "d_gain"), n_out, k_in,
                                                         _dev(d_x, "d_x"), _dev(d_y, "d_y"), code, _stream_ptr(stream)))
    return d_y


def _gemv_multi(call: str, ctx: Context, mats, y_dtype, stream):
    descs = (GemvDesc * len(mats))()
    for d, (d_w, d_gain, n_out, k_in, d_x, d_y) in zip(descs, mats):
        assert d_x.dtype == torch.bfloat16 and d_x.numel() >= k_in and d_gain.dtype == torch.float16
        assert d_y.dtype == y_dtype and d_y.numel() >= n_out and d_gain.numel() >= n_out * ((k_in + 23) // 24)
        d.d_weights, d.d_gain_f16, d.n_out, d.k_in = _dev(d_w, "d_weights"), _dev(d_gain, "d_gain"), n_out, k_in
        d.d_x_bf16, d.d_y = _dev(d_x, "d_x"), _dev(d_y, "d_y")
    _check(call, getattr(ctx._lib, call)(ctx._h, descs, len(mats), LLVQ_F32 if y_dtype == torch.float32 else LLVQ_BF16, _stream_ptr(stream)))


def llvq_gemv_multi(ctx: Context, mats, y_dtype: torch.dtype = torch.float32, stream=None) -> None:
    """Up to 8 independent products in one launch.  mats: (d_idx, d_gain, n_out, k_in, d_x, d_y) per matrix, all device tensors
    owned by the caller (outputs included); no d_y may be a d_x of the same call."""
    _gemv_multi("llvq_gemv_multi", ctx, mats, y_dtype, stream)


def llvq_gemv_sorted_multi(ctx: Context, mats, y_dtype: torch.dtype = torch.float32, stream=None) -> None:
    """The same on streams made by ``llvq_sort_blocks``: (d_sorted, d_gain, n_out, k_in, d_x, d_y) per matrix."""
    _gemv_multi("llvq_gemv_sorted_multi", ctx, mats, y_dtype, stream)


def llvq_sort_blocks_sg(ctx: Context, d_fields: torch.Tensor, gain_bits: int, n_out: int, k_in: int,
                        d_sorted: torch.Tensor | None = None, stream=None):
    """``llvq_sort_blocks`` for a stream of shape-gain fields (index_bits + gain_bits <= 48 bits each)."""
    nbytes = int(ctx._lib.llvq_sorted_bytes(ctx._h, n_out, k_in))
    if nbytes == 0:
        raise LlvqError("llvq_sorted_bytes", 3)
    if d_sorted is None:
        d_sorted = torch.empty(nbytes, dtype=torch.uint8, device=d_fields.device)
    assert d_sorted.numel() * d_sorted.element_size() >= nbytes
    assert d_fields.numel() * d_fields.element_size() >= int(ctx._lib.llvq_field_bytes(ctx._h, n_out * ((k_in + 23) // 24), gain_bits))
    _check("llvq_sort_blocks_sg", ctx._lib.llvq_sort_blocks_sg(ctx._h, _dev(d_fields, "d_fields"), gain_bits, n_out, k_in,
                                                               _dev(d_sorted, "d_sorted"), _stream_ptr(stream)))
    return d_sorted


def llvq_gemv_sorted_sg(ctx: Context, d_sorted: torch.Tensor, gain_bits: int, d_codebook: torch.Tensor,
                        d_row_scale: torch.Tensor | None, n_out: int, k_in: int, d_x: torch.Tensor,
                        d_y: torch.Tensor | None = None, y_dtype: torch.dtype = torch.float32, stream=None):
    """y = W x with W in the shape-gain form, from the sorted stream of ``llvq_sort_blocks_sg``; same result as ``llvq_gemv_sg``."""
    if d_y is None:
        d_y = torch.empty(n_out, dtype=y_dtype, device=d_sorted.device)
    assert d_x.dtype == torch.bfloat16 and d_x.numel() >= k_in
    assert d_y.dtype in (torch.float32, torch.bfloat16) and d_y.numel() >= n_out
    assert d_codebook.dtype == torch.float32 and d_codebook.numel() >= (1 << gain_bits)
    assert d_row_scale is None or (d_row_scale.dtype == torch.float32 and d_row_scale.numel() >= n_out)
    assert d_sorted.numel() * d_sorted.element_size() >= int(ctx._lib.llvq_sorted_bytes(ctx._h, n_out, k_in))
    code = LLVQ_F32 if d_y.dtype == torch.float32 else LLVQ_BF16
    _check("llvq_gemv_sorted_sg", ctx._lib.llvq_gemv_sorted_sg(
        ctx._h, _dev(d_sorted, "d_sorted"), gain_bits, _dev(d_codebook, "d_codebook"),
        None if d_row_scale is None else _dev(d_row_scale, "d_row_scale"), n_out, k_in, _dev(d_x, "d_x"), _dev(d_y, "d_y"), code, _stream_ptr(stream)))
    return d_y


def llvq_sort_blocks_gemm(ctx: Context, d_idx: torch.Tensor, n_out: int, k_in: int, d_sorted: torch.Tensor | None = None, stream=None):
    """Rewrite a ROWWISE index stream into the sorted layout of ``llvq_gemm_small_batch_sorted`` (done once per matrix)."""
    nbytes = int(ctx._lib.llvq_sorted_gemm_bytes(ctx._h, n_out, k_in))
    if nbytes == 0:
        raise LlvqError("llvq_sorted_gemm_bytes", 3)
    if d_sorted is None:
        d_sorted = torch.empty(nbytes, dtype=torch.uint8, device=d_idx.device)
    assert d_sorted.numel() * d_sorted.element_size() >= nbytes
    assert d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(n_out * ((k_in + 23) // 24))
    _check("llvq_sort_blocks_gemm", ctx._lib.llvq_sort_blocks_gemm(ctx._h, _dev(d_idx, "d_idx"), n_out, k_in, _dev(d_sorted, "d_sorted"),
                                                                   _stream_ptr(stream)))
    return d_sorted


def llvq_gemm_small_batch_sorted(ctx: Context, d_sorted: torch.Tensor, d_gain: torch.Tensor, n_out: int, k_in: int,
                                 d_x: torch.Tensor, d_y: torch.Tensor | None = None, stream=None):
    """Y[b, i] = sum_k X[b, k] W[i, k] from the sorted stream of ``llvq_sort_blocks_gemm``; same result as ``llvq_gemm_small_batch``."""
    assert d_x.dtype == torch.bfloat16 and d_x.dim() == 2 and d_x.shape[1] == k_in and d_gain.dtype == torch.float16
    batch = d_x.shape[0]
    if d_y is None:
        d_y = torch.empty((batch, n_out), dtype=torch.bfloat16, device=d_sorted.device)
    assert d_y.dtype == torch.bfloat16 and d_y.numel() >= batch * n_out
    assert d_gain.numel() >= n_out * ((k_in + 23) // 24)
    assert d_sorted.numel() * d_sorted.element_size() >= int(ctx._lib.llvq_sorted_gemm_bytes(ctx._h, n_out, k_in))
    _check("llvq_gemm_small_batch_sorted", ctx._lib.llvq_gemm_small_batch_sorted(
        ctx._h, _dev(d_sorted, "d_sorted"), _dev(d_gain, "d_gain"), n_out, k_in, _dev(d_x, "d_x"), batch, _dev(d_y, "d_y"), _stream_ptr(stream)))
    return d_y


def llvq_sort_blocks_gemm_sg(ctx: Context, d_fields: torch.Tensor, gain_bits: int, n_out: int, k_in: int,
                             d_sorted: torch.Tensor | None = None, stream=None):
    """``llvq_sort_blocks_gemm`` for a stream of shape-gain fields (index_bits + gain_bits <= 48 bits each)."""
    nbytes = int(ctx._lib.llvq_sorted_gemm_bytes(ctx._h, n_out, k_in))
    if nbytes == 0:
        raise LlvqError("llvq_sorted_gemm_bytes", 3)
    if d_sorted is None:
        d_sorted = torch.empty(nbytes, dtype=torch.uint8, device=d_fields.device)
    assert d_sorted.numel() * d_sorted.element_size() >= nbytes
    _check("llvq_sort_blocks_gemm_sg", ctx._lib.llvq_sort_blocks_gemm_sg(ctx._h, _dev(d_fields, "d_fields"), gain_bits, n_out, k_in,
                                                                         _dev(d_sorted, "d_sorted"), _stream_ptr(stream)))
    return d_sorted


def llvq_gemm_small_batch_sorted_sg(ctx: Context, d_sorted: torch.Tensor, gain_bits: int, d_codebook: torch.Tensor,
                                    d_row_scale: torch.Tensor | None, n_out: int, k_in: int, d_x: torch.Tensor,
                                    d_y: torch.Tensor | None = None, stream=None):
    """``llvq_gemm_small_batch_sg`` from the sorted stream of ``llvq_sort_blocks_gemm_sg``."""
    assert d_x.dtype == torch.bfloat16 and d_x.dim() == 2 and d_x.shape[1] == k_in
    batch = d_x.shape[0]
    if d_y is None:
        d_y = torch.empty((batch, n_out), dtype=torch.bfloat16, device=d_sorted.device)
    assert d_y.dtype == torch.bfloat16 and d_y.numel() >= batch * n_out
    assert d_sorted.numel() * d_sorted.element_size() >= int(ctx._lib.llvq_sorted_gemm_bytes(ctx._h, n_out, k_in))
    assert d_codebook.dtype == torch.float32 and d_codebook.numel() >= (1 << gain_bits)
    assert d_row_scale is None or (d_row_scale.dtype == torch.float32 and d_row_scale.numel() >= n_out)
    _check("llvq_gemm_small_batch_sorted_sg", ctx._lib.llvq_gemm_small_batch_sorted_sg(
        ctx._h, _dev(d_sorted, "d_sorted"), gain_bits, _dev(d_codebook, "d_codebook"),
        None if d_row_scale is None else _dev(d_row_scale, "d_row_scale"), n_out, k_in, _dev(d_x, "d_x"), batch, _dev(d_y, "d_y"),
        _stream_ptr(stream)))
    return d_y


def llvq_encode_blocks(ctx: Context, d_v: torch.Tensor, metric: int, d_points: torch.Tensor | None = None,
                       d_index: torch.Tensor | None = None, stream=None):
    """(points int8 [n, 24], indices int64 [n]) of the code points nearest to the rows of ``d_v`` (float32 [n, 24],
    integer-coordinate units) under LLVQ_EUCLIDEAN or LLVQ_ANGULAR scoring."""
    assert d_v.dtype == torch.float32 and d_v.dim() == 2 and d_v.shape[1] == 24
    n = d_v.shape[0]
    if d_points is None:
        d_points = torch.empty((n, 24), dtype=torch.int8, device=d_v.device)
    if d_index is None:
        d_index = torch.empty(n, dtype=torch.int64, device=d_v.device)
    assert d_points.dtype == torch.int8 and d_points.numel() >= n * 24 and d_index.dtype == torch.int64 and d_index.numel() >= n
    _check("llvq_encode_blocks", ctx._lib.llvq_encode_blocks(ctx._h, _dev(d_v, "d_v"), n, metric, _dev(d_points, "d_points"),
                                                             _dev(d_index, "d_index"), _stream_ptr(stream)))
    return d_points, d_index


def llvq_rank_blocks(ctx: Context, d_points: torch.Tensor, d_index: torch.Tensor | None = None, stream=None):
    """Indices (int64 [n]) of the lattice points ``d_points`` (int8 [n, 24]); the inverse of ``llvq_decode_blocks``."""
    assert d_points.dtype == torch.int8 and d_points.dim() == 2 and d_points.shape[1] == 24
    n = d_points.shape[0]
    if d_index is None:
        d_index = torch.empty(n, dtype=torch.int64, device=d_points.device)
    assert d_index.dtype == torch.int64 and d_index.numel() >= n
    _check("llvq_rank_blocks", ctx._lib.llvq_rank_blocks(ctx._h, _dev(d_points, "d_points"), n, _dev(d_index, "d_index"), _stream_ptr(stream)))
    return d_index


def llvq_pack_fields(ctx: Context, d_index: torch.Tensor, d_gain_index: torch.Tensor | None = None, gain_bits: int = 0,
                     d_fields: torch.Tensor | None = None, stream=None):
    """The stored stream (uint8) of the fields index | gain index << index_bits."""
    assert d_index.dtype == torch.int64
    n = d_index.numel()
    nbytes = int(ctx._lib.llvq_field_bytes(ctx._h, n, gain_bits))
    if d_fields is None:
        d_fields = torch.empty(nbytes, dtype=torch.uint8, device=d_index.device)
    assert d_fields.numel() * d_fields.element_size() >= nbytes
    assert gain_bits == 0 or (d_gain_index is not None and d_gain_index.dtype == torch.uint8 and d_gain_index.numel() >= n)
    _check("llvq_pack_fields", ctx._lib.llvq_pack_fields(
        ctx._h, _dev(d_index, "d_index"), None if d_gain_index is None or gain_bits == 0 else _dev(d_gain_index, "d_gain_index"),
        gain_bits, n, _dev(d_fields, "d_fields"), _stream_ptr(stream)))
    return d_fields


def _ptr(p, name: str) -> int:
    """A device address given as an int or as a CUDA tensor."""
    return _dev(p, name) if isinstance(p, torch.Tensor) else int(p)


def _gemv_rowshard(call: str, ctx: Context, d_stream, d_gain, n_rows, k_in, d_x, y_all, own_slot, row0, y_dtype, flag_words, epoch, stream):
    assert d_x.dtype == torch.bfloat16 and d_x.numel() >= k_in and d_gain.dtype == torch.float16
    assert y_dtype in (torch.float32, torch.bfloat16) and 1 <= len(y_all) <= 8
    assert d_gain.numel() >= n_rows * ((k_in + 23) // 24)
    ptrs = (ctypes.c_void_p * len(y_all))(*[_ptr(y, "y_all") for y in y_all])
    code = LLVQ_F32 if y_dtype == torch.float32 else LLVQ_BF16
    flags = None
    if flag_words is not None:
        assert len(flag_words) == len(y_all)
        flags = (ctypes.c_void_p * len(y_all))(*[_ptr(w, "flag_words") for w in flag_words])
    _check(call, getattr(ctx._lib, call)(ctx._h, _dev(d_stream, "d_stream"), _dev(d_gain, "d_gain"), n_rows, k_in, _dev(d_x, "d_x"),
                                         ptrs, len(y_all), own_slot, row0, code, flags, epoch & 0xffffffff, _stream_ptr(stream)))


def llvq_gemv_rowshard(ctx: Context, d_idx: torch.Tensor, d_gain: torch.Tensor, n_rows: int, k_in: int, d_x: torch.Tensor,
                       y_all, own_slot: int, row0: int, y_dtype: torch.dtype = torch.float32, flag_words=None, epoch: int = 0,
                       stream=None) -> None:
    """``llvq_gemv`` of one rank's band of rows, written at row ``row0`` of every full-length y in ``y_all``
    (tensors or device addresses; ``y_all[own_slot]`` is this rank's own copy).  With ``flag_words`` (one device
    address per destination) the kernel also stores ``epoch`` to every peer's word when the band is in place."""
    assert d_idx.numel() * d_idx.element_size() >= ctx.index_bytes(n_rows * ((k_in + 23) // 24))
    _gemv_rowshard("llvq_gemv_rowshard", ctx, d_idx, d_gain, n_rows, k_in, d_x, y_all, own_slot, row0, y_dtype, flag_words, epoch, stream)


def llvq_gemv_sorted_rowshard(ctx: Context, d_sorted: torch.Tensor, d_gain: torch.Tensor, n_rows: int, k_in: int, d_x: torch.Tensor,
                              y_all, own_slot: int, row0: int, y_dtype: torch.dtype = torch.float32, flag_words=None,
                              epoch: int = 0, stream=None) -> None:
    """``llvq_gemv_rowshard`` from the band's sorted stream (``llvq_sort_blocks`` with n_out = n_rows)."""
    assert d_sorted.numel() * d_sorted.element_size() >= int(ctx._lib.llvq_sorted_bytes(ctx._h, n_rows, k_in))
    _gemv_rowshard("llvq_gemv_sorted_rowshard", ctx, d_sorted, d_gain, n_rows, k_in, d_x, y_all, own_slot, row0, y_dtype, flag_words,
                   epoch, stream)


def llvq_gemm_small_batch_rowshard(ctx: Context, d_stream: torch.Tensor, d_gain: torch.Tensor, n_rows: int, k_in: int, d_x: torch.Tensor,
                                   y_all, own_slot: int, row0: int, n_out_total: int, flag_words=None, epoch: int = 0,
                                   sorted_layout: bool = False, stream=None) -> None:
    """Small-batch product of one rank's band of rows, written into columns ``row0..`` of every Y [batch][n_out_total]
    (bf16) in ``y_all``; ``sorted_layout`` = the stream comes from ``llvq_sort_blocks_gemm`` (called with n_out = n_rows)."""
    assert d_x.dtype == torch.bfloat16 and d_x.dim() == 2 and d_x.shape[1] == k_in and d_gain.dtype == torch.float16
    assert 1 <= len(y_all) <= 8 and d_gain.numel() >= n_rows * ((k_in + 23) // 24)
    ptrs = (ctypes.c_void_p * len(y_all))(*[_ptr(y, "y_all") for y in y_all])
    flags = None
    if flag_words is not None:
        assert len(flag_words) == len(y_all)
        flags = (ctypes.c_void_p * len(y_all))(*[_ptr(w, "flag_words") for w in flag_words])
    call = "llvq_gemm_small_batch_sorted_rowshard" if sorted_layout else "llvq_gemm_small_batch_rowshard"
    _check(call, getattr(ctx._lib, call)(ctx._h, _dev(d_stream, "d_stream"), _dev(d_gain, "d_gain"), n_rows, k_in, _dev(d_x, "d_x"),
                                         d_x.shape[0], ptrs, len(y_all), own_slot, row0, n_out_total, flags, epoch & 0xffffffff,
                                         _stream_ptr(stream)))


def llvq_gemm_small_batch_sorted_rowshard(ctx: Context, d_sorted, d_gain, n_rows, k_in, d_x, y_all, own_slot, row0, n_out_total,
                                          flag_words=None, epoch: int = 0, stream=None) -> None:
    """``llvq_gemm_small_batch_rowshard`` from the band's sorted stream."""
    llvq_gemm_small_batch_rowshard(ctx, d_sorted, d_gain, n_rows, k_in, d_x, y_all, own_slot, row0, n_out_total, flag_words, epoch,
                                   sorted_layout=True, stream=stream)


def llvq_exchange_create(ctx: Context, nbytes: int) -> tuple[int, bytes]:
    """(device address of a new zeroed exchange buffer, its 64-byte inter-process handle)."""
    buf = ctypes.c_void_p()
    handle = ctypes.create_string_buffer(LLVQ_EXCHANGE_HANDLE_BYTES)
    _check("llvq_exchange_create", ctx._lib.llvq_exchange_create(ctx._h, nbytes, ctypes.byref(buf), handle))
    return int(buf.value), handle.raw


def llvq_exchange_destroy(ctx: Context, d_buf: int) -> None:
    _check("llvq_exchange_destroy", ctx._lib.llvq_exchange_destroy(ctx._h, d_buf))


def llvq_exchange_open(ctx: Context, handle: bytes) -> int:
    """Device address, in this process, of another process's exchange buffer."""
    assert len(handle) == LLVQ_EXCHANGE_HANDLE_BYTES
    buf = ctypes.c_void_p()
    _check("llvq_exchange_open", ctx._lib.llvq_exchange_open(ctx._h, handle, ctypes.byref(buf)))
    return int(buf.value)


def llvq_exchange_close(ctx: Context, d_peer_buf: int) -> None:
    _check("llvq_exchange_close", ctx._lib.llvq_exchange_close(ctx._h, d_peer_buf))


def llvq_signal_ranks(ctx: Context, flag_words, epoch: int, stream=None) -> None:
    """After the work already on the stream, store ``epoch`` to each device word in ``flag_words`` (addresses)."""
    ptrs = (ctypes.c_void_p * max(len(flag_words), 1))(*[_ptr(w, "flag_words") for w in flag_words])
    _check("llvq_signal_ranks", ctx._lib.llvq_signal_ranks(ctx._h, ptrs, len(flag_words), epoch & 0xffffffff, _stream_ptr(stream)))


def llvq_wait_ranks(ctx: Context, d_flags, world: int, skip: int, epoch: int, max_spins: int = 0, stream=None) -> None:
    """Bounded device-side wait until the words d_flags[p], p != skip, reach ``epoch``; expiry sets LLVQ_FLAG_WAIT_TIMEOUT."""
    _check("llvq_wait_ranks", ctx._lib.llvq_wait_ranks(ctx._h, _ptr(d_flags, "d_flags"), world, skip, epoch & 0xffffffff, max_spins,
                                                       _stream_ptr(stream)))


def llvq_selftest_wait_timeout(ctx: Context, stream=None) -> None:
    """Run the bounded-wait self-test kernel: afterwards ``llvq_last_error`` reports LLVQ_FLAG_WAIT_TIMEOUT."""
    _check("llvq_selftest_wait_timeout", ctx._lib.llvq_selftest_wait_timeout(ctx._h, _stream_ptr(stream)))


def llvq_last_error(ctx: Context, stream=None) -> tuple[int, int]:
    """(number of out-of-range fields since the last call, error flags); synchronises the stream."""
    n = ctypes.c_uint64(0)
    f = ctypes.c_uint32(0)
    _check("llvq_last_error", ctx._lib.llvq_last_error(ctx._h, _stream_ptr(stream), ctypes.byref(n), ctypes.byref(f)))
    return int(n.value), int(f.value)
