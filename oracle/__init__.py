"""ctypes front end of the CPU oracle (``llvq_oracle.c``).

TEST INFRASTRUCTURE.  Only ``tests/``, the smoke check and the CPU-baseline leg
of the benchmark may import this package; the CUDA library and its Python
binding never do, and nothing here imports them.

Indices are Python integers at this level (a 72-bit code does not fit a machine
word); arrays of indices travel to C as two uint64 arrays (low and high half).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "llvq_oracle.c")
_LIB = os.path.join(_HERE, "build", "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C11, no dependencies)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            vp, i64, u64p = ctypes.c_void_p, ctypes.c_int64, ctypes.POINTER(ctypes.c_uint64)
            lib.oc_code_create.restype = vp
            lib.oc_code_create.argtypes = [ctypes.c_int, ctypes.c_int]
            lib.oc_code_destroy.argtypes = [vp]
            lib.oc_code_num_classes.argtypes = [vp]
            lib.oc_code_index_bits.argtypes = [vp]
            lib.oc_code_num_points.argtypes = [vp, u64p]
            lib.oc_class_info.argtypes = [vp, ctypes.c_int, vp, vp, vp, vp, vp, vp]
            lib.oc_unrank.argtypes = [vp, vp, vp, i64, vp]
            lib.oc_rank.argtypes = [vp, vp, i64, vp, vp]
            lib.oc_check_range.restype = i64
            lib.oc_check_range.argtypes = [vp, ctypes.c_uint64, ctypes.c_uint64, i64]
            lib.oc_unpack_stream.argtypes = [vp, ctypes.c_int, i64, vp, vp]
            lib.oc_decode_stream.restype = i64
            lib.oc_decode_stream.argtypes = [vp, vp, i64, vp]
            lib.oc_dequant_scalar.restype = ctypes.c_uint16
            lib.oc_dequant_scalar.argtypes = [ctypes.c_uint16, ctypes.c_int]
            lib.oc_dequant_matrix.restype = i64
            lib.oc_dequant_matrix.argtypes = [vp, vp, vp, i64, i64, ctypes.c_int, vp]
            lib.oc_gemm_rows.restype = i64
            lib.oc_gemm_rows.argtypes = [vp, vp, vp, i64, i64, vp, ctypes.c_int, i64, i64, vp]
            lib.oc_dequant_matrix_sg.restype = i64
            lib.oc_dequant_matrix_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp]
            lib.oc_gemm_rows_sg.restype = i64
            lib.oc_gemm_rows_sg.argtypes = [vp, vp, ctypes.c_int, vp, vp, i64, i64, vp, ctypes.c_int, i64, i64, vp]
            lib.oc_nearest_angular.argtypes = [vp, vp, vp]
            lib.oc_encode.restype = i64
            lib.oc_encode.argtypes = [vp, vp, i64, ctypes.c_int, vp, vp, vp]
            lib.oc_nearest_lattice_point.argtypes = [vp, i64, vp, vp]
            lib.oc_is_member.argtypes = [vp]
            lib.oc_shell_size.argtypes = [ctypes.c_int, u64p]
            lib.oc_golay_table.argtypes = [vp]
            _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _split(indices) -> tuple[np.ndarray, np.ndarray]:
    lo = np.fromiter(((int(i) & 0xFFFFFFFFFFFFFFFF) for i in indices), dtype=np.uint64)
    hi = np.fromiter(((int(i) >> 64) for i in indices), dtype=np.uint64)
    return lo, hi


def _join(lo: np.ndarray, hi: np.ndarray) -> list[int]:
    return [(int(h) << 64) | int(l) for l, h in zip(lo.tolist(), hi.tolist())]


def golay_table() -> np.ndarray:
    """The 4096 codewords, sorted by (weight, value); bit i <-> coordinate i."""
    out = np.zeros(4096, dtype=np.uint32)
    _load().oc_golay_table(_ptr(out))
    return out


def shell_size(m: int) -> int:
    """n(m) from the theta series (independent of the class enumeration)."""
    out = (ctypes.c_uint64 * 2)()
    _load().oc_shell_size(m, out)
    return (int(out[1]) << 64) | int(out[0])


def is_member(x) -> int:
    """0 = even coset, 1 = odd coset, -1 = not in the lattice (integer coordinates)."""
    a = np.ascontiguousarray(np.asarray(x, dtype=np.int8))
    assert a.shape == (24,)
    return int(_load().oc_is_member(_ptr(a)))


def dequant_scalar(gain_f16_bits: int, x: int) -> int:
    return int(_load().oc_dequant_scalar(int(gain_f16_bits), int(x)))


def nearest_lattice_point(v) -> tuple[np.ndarray, np.ndarray]:
    """Nearest point of the unbounded lattice (integer coordinates) to each row of v, and the squared distances."""
    a = np.ascontiguousarray(np.asarray(v, dtype=np.float64)).reshape(-1, 24)
    pts = np.zeros((len(a), 24), dtype=np.int32)
    d2 = np.zeros(len(a), dtype=np.float64)
    _load().oc_nearest_lattice_point(_ptr(a), len(a), _ptr(pts), _ptr(d2))
    return pts, d2


EUCLIDEAN, ANGULAR = 0, 1


class Code:
    """Union of Shell(m), m_lo <= m <= m_hi, with its class table and index range."""

    def __init__(self, m_lo: int, m_hi: int):
        self._lib = _load()
        self._h = self._lib.oc_code_create(m_lo, m_hi)
        if not self._h:
            raise ValueError(f"unsupported code ({m_lo}, {m_hi})")
        self.m_lo, self.m_hi = m_lo, m_hi
        out = (ctypes.c_uint64 * 2)()
        self._lib.oc_code_num_points(self._h, out)
        self.N = (int(out[1]) << 64) | int(out[0])
        self.W = int(self._lib.oc_code_index_bits(self._h))
        self.num_classes = int(self._lib.oc_code_num_classes(self._h))

    def __del__(self):
        if getattr(self, "_h", None):
            self._lib.oc_code_destroy(self._h)
            self._h = None

    def class_info(self, j: int) -> dict:
        info = np.zeros(5, dtype=np.int32)
        A = np.zeros(1, dtype=np.uint64)
        card = np.zeros(2, dtype=np.uint64)
        off = np.zeros(2, dtype=np.uint64)
        vals = np.zeros(24, dtype=np.int32)
        mults = np.zeros(24, dtype=np.int32)
        self._lib.oc_class_info(self._h, j, _ptr(info), _ptr(A), _ptr(card), _ptr(off), _ptr(vals), _ptr(mults))
        nv = int(info[3])
        return {
            "m": int(info[0]), "parity": int(info[1]), "w": int(info[2]), "B": int(info[4]),
            "A": int(A[0]),
            "card": (int(card[1]) << 64) | int(card[0]),
            "offset": (int(off[1]) << 64) | int(off[0]),
            "values": [int(v) for v in vals[:nv]],
            "mults": [int(v) for v in mults[:nv]],
        }

    def classes(self) -> list[dict]:
        return [self.class_info(j) for j in range(self.num_classes)]

    # -- index <-> point ---------------------------------------------------
    def unrank(self, indices) -> np.ndarray:
        lo, hi = _split(indices)
        pts = np.zeros((len(lo), 24), dtype=np.int8)
        self._lib.oc_unrank(self._h, _ptr(lo), _ptr(hi), len(lo), _ptr(pts))
        return pts

    def unrank_arrays(self, lo: np.ndarray, hi: np.ndarray) -> np.ndarray:
        lo = np.ascontiguousarray(lo, dtype=np.uint64)
        hi = np.ascontiguousarray(hi, dtype=np.uint64)
        pts = np.zeros((len(lo), 24), dtype=np.int8)
        self._lib.oc_unrank(self._h, _ptr(lo), _ptr(hi), len(lo), _ptr(pts))
        return pts

    def rank(self, points) -> list[int]:
        pts = np.ascontiguousarray(np.asarray(points, dtype=np.int8)).reshape(-1, 24)
        lo = np.zeros(len(pts), dtype=np.uint64)
        hi = np.zeros(len(pts), dtype=np.uint64)
        bad = self._lib.oc_rank(self._h, _ptr(pts), len(pts), _ptr(lo), _ptr(hi))
        if bad:
            raise ValueError(f"{bad} points are not in the code")
        return _join(lo, hi)

    def check_range(self, first: int, count: int, threads: int = 1) -> int:
        """Failures of {member, norm, rank(unrank(I)) == I} over [first, first+count)."""
        if threads <= 1 or count < 4 * threads:
            return int(self._lib.oc_check_range(self._h, first & (2**64 - 1), first >> 64, count))
        step = -(-count // threads)
        jobs = [(first + s, min(step, count - s)) for s in range(0, count, step)]
        with ThreadPoolExecutor(threads) as ex:
            return sum(ex.map(lambda j: int(self._lib.oc_check_range(self._h, j[0] & (2**64 - 1), j[0] >> 64, j[1])), jobs))

    # -- stored format -----------------------------------------------------
    def unpack(self, stream: np.ndarray, nblocks: int) -> list[int]:
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        assert stream.size * 8 >= nblocks * self.W
        lo = np.zeros(nblocks, dtype=np.uint64)
        hi = np.zeros(nblocks, dtype=np.uint64)
        self._lib.oc_unpack_stream(_ptr(stream), self.W, nblocks, _ptr(lo), _ptr(hi))
        return _join(lo, hi)

    def decode_stream(self, stream: np.ndarray, nblocks: int) -> tuple[np.ndarray, int]:
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        assert stream.size * 8 >= nblocks * self.W
        pts = np.zeros((nblocks, 24), dtype=np.int8)
        bad = self._lib.oc_decode_stream(self._h, _ptr(stream), nblocks, _ptr(pts))
        return pts, int(bad)

    def dequant_matrix(self, stream, gain_f16, rows: int, cols: int, layout: int) -> np.ndarray:
        """bf16 bit patterns (uint16), rows x cols.  layout 0 = FLAT, 1 = ROWWISE."""
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        gain = np.ascontiguousarray(gain_f16, dtype=np.uint16)
        out = np.zeros((rows, cols), dtype=np.uint16)
        self._lib.oc_dequant_matrix(self._h, _ptr(stream), _ptr(gain), rows, cols, layout, _ptr(out))
        return out

    def gemm(self, stream, gain_f16, n_out: int, k_in: int, x_bf16, rows=None, threads: int = 1) -> np.ndarray:
        """Y[b][i] = sum_k X[b][k] w[i][k] in float64; x_bf16 is [batch, k_in] (or [k_in]) bf16 bits.

        ``rows = (first, count)`` restricts the computation to those output rows
        (the others stay zero)."""
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        gain = np.ascontiguousarray(gain_f16, dtype=np.uint16)
        x = np.ascontiguousarray(x_bf16, dtype=np.uint16)
        vec = x.ndim == 1
        x2 = x.reshape(1, -1) if vec else x
        batch = x2.shape[0]
        assert x2.shape[1] == k_in
        y = np.zeros((batch, n_out), dtype=np.float64)
        first, count = rows if rows is not None else (0, n_out)

        def run(job):
            self._lib.oc_gemm_rows(self._h, _ptr(stream), _ptr(gain), n_out, k_in, _ptr(x2), batch, job[0], job[1], _ptr(y))

        if threads <= 1:
            run((first, count))
        else:
            step = -(-count // threads)
            jobs = [(first + s, min(step, count - s)) for s in range(0, count, step)]
            with ThreadPoolExecutor(threads) as ex:
                list(ex.map(run, jobs))
        return y[0] if vec else y

    def gemv(self, stream, gain_f16, n_out: int, k_in: int, x_bf16, **kw) -> np.ndarray:
        return self.gemm(stream, gain_f16, n_out, k_in, np.asarray(x_bf16).reshape(-1), **kw)

    # -- shape-gain with a gain codebook and an optional scale per row ------
    def dequant_matrix_sg(self, stream, gain_bits: int, codebook, row_scale, rows: int, cols: int) -> np.ndarray:
        """bf16 bit patterns of gain * x / |x| (ROWWISE fields of W + gain_bits bits); row_scale may be None."""
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        cb = np.ascontiguousarray(codebook, dtype=np.float32)
        assert cb.size == 1 << gain_bits
        rs = None if row_scale is None else np.ascontiguousarray(row_scale, dtype=np.float32)
        out = np.zeros((rows, cols), dtype=np.uint16)
        self._lib.oc_dequant_matrix_sg(self._h, _ptr(stream), gain_bits, _ptr(cb), None if rs is None else _ptr(rs),
                                       rows, cols, _ptr(out))
        return out

    def gemm_sg(self, stream, gain_bits: int, codebook, row_scale, n_out: int, k_in: int, x_bf16, rows=None,
                threads: int = 1) -> np.ndarray:
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        cb = np.ascontiguousarray(codebook, dtype=np.float32)
        assert cb.size == 1 << gain_bits
        rs = None if row_scale is None else np.ascontiguousarray(row_scale, dtype=np.float32)
        x = np.ascontiguousarray(x_bf16, dtype=np.uint16)
        vec = x.ndim == 1
        x2 = x.reshape(1, -1) if vec else x
        batch = x2.shape[0]
        assert x2.shape[1] == k_in
        y = np.zeros((batch, n_out), dtype=np.float64)
        first, count = rows if rows is not None else (0, n_out)

        def run(job):
            self._lib.oc_gemm_rows_sg(self._h, _ptr(stream), gain_bits, _ptr(cb), None if rs is None else _ptr(rs),
                                      n_out, k_in, _ptr(x2), batch, job[0], job[1], _ptr(y))

        if threads <= 1:
            run((first, count))
        else:
            step = -(-count // threads)
            jobs = [(first + s, min(step, count - s)) for s in range(0, count, step)]
            with ThreadPoolExecutor(threads) as ex:
                list(ex.map(run, jobs))
        return y[0] if vec else y

    def encode(self, v, metric: int, threads: int = 1) -> tuple[np.ndarray, list[int]]:
        """Nearest points of the code to the rows of v (integer-coordinate units) and their indices."""
        a = np.ascontiguousarray(np.asarray(v, dtype=np.float64)).reshape(-1, 24)
        n = len(a)
        pts = np.zeros((n, 24), dtype=np.int8)
        lo = np.zeros(n, dtype=np.uint64)
        hi = np.zeros(n, dtype=np.uint64)

        def run(job):
            f, c = job
            return int(self._lib.oc_encode(self._h, _ptr(a[f:f + c]), c, metric, _ptr(pts[f:f + c]), _ptr(lo[f:f + c]), _ptr(hi[f:f + c])))

        if threads <= 1 or n < 2 * threads:
            bad = run((0, n))
        else:
            step = -(-n // threads)
            with ThreadPoolExecutor(threads) as ex:
                bad = sum(ex.map(run, [(s, min(step, n - s)) for s in range(0, n, step)]))
        if bad:
            raise ValueError(f"the search gave up on {bad} vectors (unsupported code?)")
        return pts, _join(lo, hi)

    def nearest_angular(self, x) -> int:
        v = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
        assert v.shape == (24,)
        out = np.zeros(2, dtype=np.uint64)
        self._lib.oc_nearest_angular(self._h, _ptr(v), _ptr(out))
        return (int(out[1]) << 64) | int(out[0])
