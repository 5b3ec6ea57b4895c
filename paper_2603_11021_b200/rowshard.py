"""Row-sharded fused GEMV over several GPUs, one process per GPU.

Blocks are independent (App. A step 5), so W splits by output rows without any change to the arithmetic: every rank
holds the index and gain streams of its own band of rows, x is the same on all ranks, and the only exchange is
y itself (2 or 4 bytes per row).  The GEMV kernel writes a band straight into every rank's copy of y over NVLink
(``llvq_gemv_rowshard``); a flag word per writer tells the readers when a step's y is complete.

Host logic only: planning the bands, slicing a ROWWISE stream, carrying the exchange handles between the processes
through ``torch.distributed`` (any backend that moves Python objects), and the order of the calls of one step.
"""
from __future__ import annotations

import numpy as np
import torch

from . import (Context, llvq_exchange_close, llvq_exchange_create, llvq_exchange_destroy, llvq_exchange_open,
               llvq_gemv_rowshard, llvq_gemv_sorted_rowshard, llvq_signal_ranks, llvq_sort_blocks, llvq_wait_ranks)

__all__ = ["row_bands", "band_of_stream", "exchange_handles", "RowShardedGemv", "MAX_RANKS"]

MAX_RANKS = 8
_FLAG_BYTES = 256          # one 32-bit word per writer, padded so that the vectors behind start 256-byte aligned


def row_bands(n_out: int, world: int, align: int = 8) -> list[tuple[int, int]]:
    """Contiguous bands (row0, n_rows), one per rank, covering [0, n_out).

    Band boundaries fall on multiples of ``align`` rows (8 = the row group of the GEMV kernels, which also keeps a
    band's slice of a ROWWISE stream on a byte boundary for every index width); the groups of ``align`` rows are dealt
    as evenly as they go, earlier ranks taking the extra ones.  A rank may get an empty band when there are fewer
    groups than ranks.
    """
    if n_out < 0 or world < 1 or align < 1:
        raise ValueError("row_bands: n_out >= 0, world >= 1, align >= 1")
    groups = (n_out + align - 1) // align
    base, extra = divmod(groups, world)
    bands, g0 = [], 0
    for r in range(world):
        g1 = g0 + base + (1 if r < extra else 0)
        row0, row1 = min(g0 * align, n_out), min(g1 * align, n_out)
        bands.append((row0, row1 - row0))
        g0 = g1
    return bands


def band_of_stream(stream: np.ndarray, gains: np.ndarray, k_in: int, index_bits: int, row0: int, n_rows: int):
    """The part of a ROWWISE index stream (uint8) and gain array that belongs to rows [row0, row0 + n_rows).

    The band must start on a byte boundary of the bit stream (row0 a multiple of 8 always does).  The index bytes come
    back padded to a multiple of 16, as the device calls expect.
    """
    bpr = (k_in + 23) // 24
    if n_rows == 0:                                # an empty band (more ranks than row groups) may sit anywhere
        return np.zeros(0, dtype=np.uint8), np.asarray(gains)[:0].copy()
    b0, b1 = row0 * bpr * index_bits, (row0 + n_rows) * bpr * index_bits
    if b0 % 8:
        raise ValueError("band_of_stream: the band does not start on a byte boundary")
    raw = np.asarray(stream, dtype=np.uint8)[b0 // 8:(b1 + 7) // 8]
    if b1 % 8:                                     # bits of the next band share the last byte: clear them
        raw = raw.copy()
        raw[-1] &= (1 << (b1 % 8)) - 1
    out = np.zeros((raw.size + 15) // 16 * 16, dtype=np.uint8)
    out[:raw.size] = raw
    return out, np.ascontiguousarray(np.asarray(gains)[row0 * bpr:(row0 + n_rows) * bpr])


def exchange_handles(handle: bytes, group=None) -> list[bytes]:
    """All ranks' handles, in rank order (an object all-gather over the process group)."""
    import torch.distributed as dist
    out = [None] * dist.get_world_size(group)
    dist.all_gather_object(out, bytes(handle), group=group)
    return [bytes(h) for h in out]


class _RawDeviceArray:
    """Lets torch view device memory that the library allocated."""

    def __init__(self, ptr: int, n: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}


class RowShardedGemv:
    """y = W x with the rows of W spread over the ranks of a process group; every rank ends up with all of y.

    Each rank passes its own band (``row_bands(n_out, world)[rank]``) as device tensors.  One step is
    ``launch(x)`` (one kernel: the band's fused GEMV, writing into every rank's y and then the epoch flag of every peer) followed by
    ``wait()`` (bounded device-side wait for the other ranks' flags) — ``__call__`` does both and returns this
    rank's y.  Two y buffers alternate between steps: a rank that is one step ahead writes the other buffer, and it
    cannot be two steps ahead because each step waits for every rank's previous flag.
    """

    def __init__(self, ctx: Context, n_out: int, k_in: int, d_stream: torch.Tensor, d_gain: torch.Tensor,
                 y_dtype: torch.dtype = torch.bfloat16, sorted_layout: bool = False, group=None, align: int = 8):
        import torch.distributed as dist
        self.ctx, self.group = ctx, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        if self.world > MAX_RANKS:
            raise ValueError(f"at most {MAX_RANKS} ranks")
        assert y_dtype in (torch.float32, torch.bfloat16)
        self.n_out, self.k_in, self.y_dtype = n_out, k_in, y_dtype
        self.row0, self.n_rows = row_bands(n_out, self.world, align)[self.rank]
        self.d_gain = d_gain
        self.sorted_layout = sorted_layout
        self.d_stream = llvq_sort_blocks(ctx, d_stream, self.n_rows, k_in) if sorted_layout and self.n_rows else d_stream
        es = 4 if y_dtype == torch.float32 else 2
        self._y_bytes = (n_out * es + 255) // 256 * 256
        self._own, handle = llvq_exchange_create(ctx, _FLAG_BYTES + 2 * self._y_bytes)
        handles = exchange_handles(handle, group)
        self._bufs = [self._own if r == self.rank else llvq_exchange_open(ctx, handles[r]) for r in range(self.world)]
        self._views = [self._wrap(self._own + _FLAG_BYTES + parity * self._y_bytes) for parity in range(2)]
        self.epoch = 0
        dist.barrier(group)                         # every buffer is mapped everywhere before anybody writes

    def _wrap(self, ptr: int) -> torch.Tensor:
        """A tensor over one of the own y buffers (device memory that the library allocated)."""
        typestr = "<f4" if self.y_dtype == torch.float32 else "<i2"
        raw = torch.as_tensor(_RawDeviceArray(ptr, self.n_out, typestr), device=torch.device("cuda", self.ctx.device))
        return raw if self.y_dtype == torch.float32 else raw.view(torch.bfloat16)

    def _y_all(self, parity: int) -> list[int]:
        return [b + _FLAG_BYTES + parity * self._y_bytes for b in self._bufs]

    def launch(self, d_x: torch.Tensor, stream=None) -> None:
        """Enqueue this rank's part of the next step."""
        self.epoch += 1
        call = llvq_gemv_sorted_rowshard if self.sorted_layout else llvq_gemv_rowshard
        words = [b + 4 * self.rank for b in self._bufs]                  # this rank's word in every buffer
        if self.n_rows:
            call(self.ctx, self.d_stream, self.d_gain, self.n_rows, self.k_in, d_x, self._y_all(self.epoch & 1), self.rank, self.row0,
                 self.y_dtype, words, self.epoch, stream)
        else:
            llvq_signal_ranks(self.ctx, [w for r, w in enumerate(words) if r != self.rank], self.epoch, stream)

    def wait(self, stream=None, max_spins: int = 0) -> torch.Tensor:
        """Enqueue the wait for the other ranks' parts of the step launched last; returns this rank's y (valid in
        stream order once the wait has run; ``llvq_last_error`` tells whether it ran out)."""
        llvq_wait_ranks(self.ctx, self._own, self.world, self.rank, self.epoch, max_spins, stream)
        return self._views[self.epoch & 1]

    def __call__(self, d_x: torch.Tensor, stream=None) -> torch.Tensor:
        self.launch(d_x, stream)
        return self.wait(stream)

    def _synchronize(self) -> None:
        torch.cuda.synchronize(self.ctx.device)

    def close(self) -> None:
        """Collective: unmap the peers' buffers, then free the own one."""
        import torch.distributed as dist
        if self._bufs is None:
            return
        self._synchronize()
        for r, b in enumerate(self._bufs):
            if r != self.rank:
                llvq_exchange_close(self.ctx, b)
        dist.barrier(self.group)
        self._views = []
        llvq_exchange_destroy(self.ctx, self._own)
        self._bufs = None
