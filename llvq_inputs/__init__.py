"""Seeded synthetic inputs shared by the CPU oracle and the CUDA library.

This module holds none of the method's arithmetic (no lattice, no Golay code,
no unranking): it draws random integers, packs them into the stored bit-stream
format, and draws gains and activations.  Both sides receive exactly the same
bytes.  The code size N and index width W are passed in by the caller.

Recipe (stands in for quantized LLM linear layers):
  * indices: i.i.d. uniform on [0, N), by rejection from W random bits of a
    counter-based generator: splitmix64 finaliser of a linear combination of
    (seed, block number, attempt, word);
  * gains: fp16(|z| * 0.02), z ~ N(0, 1);
  * activations: N(0, 1) rounded to bf16 (round to nearest even).
"""
from __future__ import annotations

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_K_SEED = 0x9E3779B97F4A7C15
_K_BLOCK = 0xD1B54A32D192ED03
_K_TRY = 0x8CB92BA72F3D8DD7
_K_WORD = 0xABC98388FB8FAC03


def splitmix64(z: np.ndarray) -> np.ndarray:
    """The splitmix64 output function applied to each uint64 of z."""
    z = z.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        z ^= z >> np.uint64(30)
        z *= np.uint64(0xBF58476D1CE4E5B9)
        z ^= z >> np.uint64(27)
        z *= np.uint64(0x94D049BB133111EB)
        z ^= z >> np.uint64(31)
    return z


def _draw(seed: int, blocks: np.ndarray, attempt: int, word: int) -> np.ndarray:
    base = (seed * _K_SEED + attempt * _K_TRY + word * _K_WORD + 0x632BE59BD9B4E019) & 0xFFFFFFFFFFFFFFFF
    with np.errstate(over="ignore"):
        ctr = blocks.astype(np.uint64) * np.uint64(_K_BLOCK) + np.uint64(base)
    return splitmix64(ctr)


def random_indices(N: int, W: int, nblocks: int, seed: int = 0, first_block: int = 0):
    """Uniform indices on [0, N) as (lo, hi) uint64 arrays; W = index width in bits."""
    assert 1 <= W <= 128 and 0 < N <= (1 << W)
    blocks = np.arange(first_block, first_block + nblocks, dtype=np.uint64)
    lo = np.zeros(nblocks, dtype=np.uint64)
    hi = np.zeros(nblocks, dtype=np.uint64)
    todo = np.arange(nblocks)
    n_lo, n_hi = np.uint64(N & 0xFFFFFFFFFFFFFFFF), np.uint64(N >> 64)
    mask_lo = np.uint64((1 << min(W, 64)) - 1)
    mask_hi = np.uint64((1 << max(W - 64, 0)) - 1)
    attempt = 0
    while todo.size:
        c_lo = _draw(seed, blocks[todo], attempt, 0) & mask_lo
        c_hi = (_draw(seed, blocks[todo], attempt, 1) & mask_hi) if W > 64 else np.zeros(todo.size, dtype=np.uint64)
        ok = (c_hi < n_hi) | ((c_hi == n_hi) & (c_lo < n_lo))
        lo[todo[ok]] = c_lo[ok]
        hi[todo[ok]] = c_hi[ok]
        todo = todo[~ok]
        attempt += 1
    return lo, hi


def index_stream_bytes(nblocks: int, W: int) -> int:
    """Length of the packed stream: ceil(nblocks * W / 8) rounded up to 16 bytes."""
    n = (nblocks * W + 7) // 8
    return (n + 15) // 16 * 16


def pack_indices(lo: np.ndarray, hi: np.ndarray, W: int) -> np.ndarray:
    """Pack W-bit fields into the stored stream: field b occupies stream bits
    [b*W, (b+1)*W), stream bit t being bit (t % 8) of byte (t // 8); zero padded
    to a multiple of 16 bytes."""
    n = len(lo)
    out = np.zeros(index_stream_bytes(n, W), dtype=np.uint8)
    if n == 0:
        return out
    raw = np.empty((n, 16), dtype=np.uint8)
    raw[:, :8] = lo.astype("<u8").view(np.uint8).reshape(n, 8)
    raw[:, 8:] = hi.astype("<u8").view(np.uint8).reshape(n, 8)
    if W % 8 == 0:
        out[: n * (W // 8)] = raw[:, : W // 8].reshape(-1)
    else:
        bits = np.unpackbits(raw, axis=1, bitorder="little")[:, :W].reshape(-1)
        packed = np.packbits(bits, bitorder="little")
        out[: packed.size] = packed
    return out


def indices_to_arrays(indices) -> tuple[np.ndarray, np.ndarray]:
    """Python integers -> (lo, hi) uint64 arrays."""
    lo = np.array([int(i) & 0xFFFFFFFFFFFFFFFF for i in indices], dtype=np.uint64)
    hi = np.array([int(i) >> 64 for i in indices], dtype=np.uint64)
    return lo, hi


def gains_f16(nblocks: int, seed: int = 0, scale: float = 0.02) -> np.ndarray:
    """fp16(|z| * scale), z ~ N(0,1), as uint16 bit patterns."""
    rng = np.random.Generator(np.random.PCG64([seed, 0x6761696E]))
    z = np.abs(rng.standard_normal(nblocks, dtype=np.float32)) * np.float32(scale)
    return z.astype(np.float16).view(np.uint16)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 bit patterns (nearest even); finite inputs."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, seed: int = 0) -> np.ndarray:
    """N(0,1) activations rounded to bf16, as uint16 bit patterns."""
    rng = np.random.Generator(np.random.PCG64([seed, 0x61637476]))
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


def make_layer(N: int, W: int, rows: int, cols: int, layout: int, seed: int = 0):
    """(stream, gains, nblocks) for one weight matrix.  layout 0 = FLAT (blocks
    over the flattened matrix), 1 = ROWWISE (each row has ceil(cols/24) blocks)."""
    nblocks = (rows * cols + 23) // 24 if layout == 0 else rows * ((cols + 23) // 24)
    lo, hi = random_indices(N, W, nblocks, seed)
    return pack_indices(lo, hi, W), gains_f16(nblocks, seed), nblocks


def gain_indices(nblocks: int, gain_bits: int, seed: int = 0) -> np.ndarray:
    """Uniform gain-codebook indices in [0, 2**gain_bits), one per block (uint64)."""
    if gain_bits == 0:
        return np.zeros(nblocks, dtype=np.uint64)
    blocks = np.arange(nblocks, dtype=np.uint64)
    return _draw(seed ^ 0x6A09E667, blocks, 0, 7) >> np.uint64(64 - gain_bits)


def row_scales_f32(rows: int, seed: int = 0, scale: float = 0.02) -> np.ndarray:
    """One positive binary32 scale per output row: scale * (1 + 0.1 z), z ~ N(0,1) clipped to +-3."""
    rng = np.random.default_rng(seed + 0x5CA1E)
    z = np.clip(rng.standard_normal(rows), -3.0, 3.0)
    return (scale * (1.0 + 0.1 * z)).astype(np.float32)


def make_layer_sg(N: int, W: int, gain_bits: int, rows: int, cols: int, seed: int = 0):
    """(stream, nblocks) of a ROWWISE layer whose fields are W + gain_bits wide: shape index | gain index << W."""
    assert W + gain_bits <= 64
    nblocks = rows * ((cols + 23) // 24)
    lo, hi = random_indices(N, W, nblocks, seed)
    lo = lo | (gain_indices(nblocks, gain_bits, seed) << np.uint64(W)) if gain_bits else lo
    return pack_indices(lo, hi, W + gain_bits), nblocks
