"""Parity of the CUDA library against the CPU oracle, through the C ABI.

Integer work (lattice points, bf16 weights) must be bit-exact.  Fused products
accumulate in binary32 and are compared with the oracle's binary64 result:
max relative error <= 1e-3 with the denominator floored at 1e-3 * max|y|; bf16
outputs are additionally allowed the half-ulp of their own rounding (2^-9).
"""
import numpy as np
import pytest
import torch

import llvq_inputs as gen
from gpu_util import bf16_bits, gemm_error, gemv_error, to_dev_bf16, to_dev_f16, to_dev_u8

pytestmark = pytest.mark.gpu

TOL = 1e-3
TOL_BF16_OUT = 1e-3 + 2.0 ** -8


@pytest.fixture(scope="module")
def lib():
    import paper_2603_11021_b200 as P
    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU path"
    return P


@pytest.fixture(scope="module")
def ctxs(lib):
    return {code: lib.Context(*code, device=0) for code in [(2, 2), (3, 3), (2, 13), (2, 53)]}


def _oracle(oracle_mod, cache={}):
    def get(code):
        if code not in cache:
            cache[code] = oracle_mod.Code(*code)
        return cache[code]
    return get


def _threads():
    import os
    return os.cpu_count() or 1


def _decode_gpu(lib, ctx, lo, hi):
    stream = gen.pack_indices(lo, hi, ctx.index_bits)
    assert stream.size == ctx.index_bytes(len(lo))
    pts = lib.llvq_decode_blocks(ctx, to_dev_u8(stream), len(lo))
    torch.cuda.synchronize()
    return pts.cpu().numpy()


def test_context_matches_oracle_tables(lib, ctxs, oracle_mod):
    for code, ctx in ctxs.items():
        o = _oracle(oracle_mod)(code)
        assert (ctx.index_bits, ctx.num_points, ctx.num_classes) == (o.W, o.N, o.num_classes)


def test_decode_exhaustive_minimal_shell(lib, ctxs, oracle_mod):
    o = _oracle(oracle_mod)((2, 2))
    lo = np.arange(o.N, dtype=np.uint64)
    got = _decode_gpu(lib, ctxs[(2, 2)], lo, np.zeros_like(lo))
    assert np.array_equal(got, o.unrank_arrays(lo, np.zeros_like(lo)))
    assert lib.llvq_last_error(ctxs[(2, 2)]) == (0, 0)


@pytest.mark.parametrize("code,nrand", [((2, 2), 8192), ((3, 3), 200003), ((2, 13), 300007), ((2, 53), 100001)])
def test_decode_random_and_class_edges(lib, ctxs, oracle_mod, code, nrand):
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    lo, hi = gen.random_indices(o.N, o.W, nrand, seed=0)
    edges = []
    for k in o.classes():
        edges += [k["offset"], k["offset"] + k["card"] - 1, k["offset"] + k["card"] // 2]
    elo, ehi = gen.indices_to_arrays(edges)
    lo, hi = np.concatenate([lo, elo]), np.concatenate([hi, ehi])
    got = _decode_gpu(lib, ctx, lo, hi)
    want = o.unrank_arrays(lo, hi)
    bad = np.nonzero((got != want).any(axis=1))[0]
    assert bad.size == 0, (bad[:5], got[bad[:2]], want[bad[:2]])
    assert lib.llvq_last_error(ctx) == (0, 0)


@pytest.mark.parametrize("code", [(2, 2), (2, 13), (2, 53)])
def test_decode_out_of_range_fields_are_zero_and_counted(lib, ctxs, oracle_mod, code):
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    idx = [0, o.N, o.N - 1, (1 << o.W) - 1, o.N + 12345, 5]
    lo, hi = gen.indices_to_arrays(idx)
    got = _decode_gpu(lib, ctx, lo, hi)
    want = o.unrank(idx)
    assert np.array_equal(got, want)
    assert not got[1].any() and not got[3].any() and got[2].any()
    assert lib.llvq_last_error(ctx) == (3, 0)
    assert lib.llvq_last_error(ctx) == (0, 0)          # cleared by the read


def test_decode_empty_and_single(lib, ctxs, oracle_mod):
    ctx = ctxs[(2, 13)]
    o = _oracle(oracle_mod)((2, 13))
    out = lib.llvq_decode_blocks(ctx, torch.zeros(16, dtype=torch.uint8, device="cuda"), 0)
    assert out.shape == (0, 24)
    lo, hi = gen.indices_to_arrays([o.N - 1])
    assert np.array_equal(_decode_gpu(lib, ctx, lo, hi), o.unrank([o.N - 1]))


@pytest.mark.parametrize("code,rows,cols,layout", [
    ((2, 2), 256, 768, 1),           # config 1 shape
    ((2, 13), 37, 1000, 0),          # FLAT, 37000 elements = 1541 blocks + 16 elements
    ((2, 13), 301, 4096, 1),         # ROWWISE, 171 blocks per row, 8 pad lanes per row
    ((2, 13), 64, 24, 1),
    ((2, 13), 1, 7, 0),
    ((2, 53), 129, 520, 1),
    ((2, 53), 100, 333, 0),
    ((3, 3), 50, 4104, 1),           # the shape of the paper's own kernel timing
])
def test_dequant_matrix_bit_exact(lib, ctxs, oracle_mod, code, rows, cols, layout):
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    stream, gain, nblocks = gen.make_layer(o.N, o.W, rows, cols, layout, seed=1)
    want = o.dequant_matrix(stream, gain, rows, cols, layout)
    got = lib.llvq_dequant_matrix(ctx, to_dev_u8(stream), to_dev_f16(gain), rows, cols, layout)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(got), want)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_dequant_matrix_leading_dimension_and_unaligned_rows(lib, ctxs, oracle_mod):
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    rows, cols, ld = 33, 100, 107                       # odd ld: rows start at 2-byte aligned addresses only
    stream, gain, _ = gen.make_layer(o.N, o.W, rows, cols, 1, seed=2)
    want = o.dequant_matrix(stream, gain, rows, cols, 1)
    buf = torch.full((rows, ld), -7.0, dtype=torch.bfloat16, device="cuda")
    lib.llvq_dequant_matrix(ctx, to_dev_u8(stream), to_dev_f16(gain), rows, cols, 1, d_w=buf, ld=ld)
    torch.cuda.synchronize()
    out = bf16_bits(buf)
    assert np.array_equal(out[:, :cols], want)
    assert (buf[:, cols:].float().cpu().numpy() == -7.0).all()      # padding untouched


def test_dequant_signed_zero_and_special_gains(lib, ctxs, oracle_mod):
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    rows, cols = 16, 240
    stream, gain, nblocks = gen.make_layer(o.N, o.W, rows, cols, 1, seed=3)
    special = np.array([0x0000, 0x8000, 0x0001, 0x03FF, 0x0400, 0x7BFF, 0xFBFF, 0x3C00, 0xBC00, 0x3555], dtype=np.uint16)
    gain[: special.size * 4] = np.tile(special, 4)
    want = o.dequant_matrix(stream, gain, rows, cols, 1)
    got = lib.llvq_dequant_matrix(ctx, to_dev_u8(stream), to_dev_f16(gain), rows, cols, 1)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(got), want)


def test_gemv_config1_tiny(lib, ctxs, oracle_mod):
    # 256 x 768, minimal shell only, 18-bit fields, fp32 output
    o = _oracle(oracle_mod)((2, 2))
    ctx = ctxs[(2, 2)]
    n_out, k_in = 256, 768
    stream, gain, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=0)
    assert nblocks == 8192
    x = gen.normal_bf16(k_in, seed=0)
    want = o.gemv(stream, gain, n_out, k_in, x)
    got = lib.llvq_gemv(ctx, to_dev_u8(stream), to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    assert gemv_error(got.cpu().numpy(), want) <= TOL


@pytest.mark.parametrize("code,n_out,k_in", [((2, 13), 67, 4096), ((2, 13), 8, 24), ((2, 13), 129, 1000),
                                             ((2, 53), 40, 2048), ((3, 3), 33, 4104)])
def test_gemv_small_shapes_both_output_types(lib, ctxs, oracle_mod, code, n_out, k_in):
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=4)
    x = gen.normal_bf16(k_in, seed=4)
    want = o.gemv(stream, gain, n_out, k_in, x)
    d = (to_dev_u8(stream), to_dev_f16(gain))
    y32 = lib.llvq_gemv(ctx, *d, n_out, k_in, to_dev_bf16(x))
    y16 = lib.llvq_gemv(ctx, *d, n_out, k_in, to_dev_bf16(x), y_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert gemv_error(y32.cpu().numpy(), want) <= TOL
    assert gemv_error(y16.float().cpu().numpy(), want) <= TOL_BF16_OUT
    # the bf16 output is the rounding of the fp32 one; the two launches may add their partial sums in a different
    # order (shared-memory atomics), so a value next to a rounding boundary may land on either side of it
    a, b = y32.to(torch.bfloat16).float(), y16.float()
    assert float(((a - b).abs() / a.abs().clamp_min(1e-30)).max()) <= 2.0 ** -7


def test_gemv_exact_integer_cases(lib, ctxs, oracle_mod):
    # gains = 1 and x = e_k / all-ones: results are small integers, exact in binary32
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n_out, k_in = 50, 500
    stream, _, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=5)
    ones = np.full(nblocks, 0x3C00, dtype=np.uint16)
    pts, _ = o.decode_stream(stream, nblocks)
    Wint = pts.reshape(n_out, -1)[:, :k_in].astype(np.int64)
    for xv in (np.ones(k_in, dtype=np.float32), np.eye(k_in, dtype=np.float32)[499], np.eye(k_in, dtype=np.float32)[24]):
        y = lib.llvq_gemv(ctx, to_dev_u8(stream), to_dev_f16(ones), n_out, k_in, to_dev_bf16(gen.f32_to_bf16_bits(xv)))
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy().astype(np.int64), (Wint * xv.astype(np.int64)).sum(axis=1))


@pytest.mark.parametrize("n_out,k_in", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_gemv_full_size_layers_all_rows(lib, ctxs, oracle_mod, n_out, k_in):
    # the 7B-shaped layers the benchmark times, in the same launch configuration; the oracle recomputes every output row
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=0)
    x = gen.normal_bf16(k_in, seed=0)
    y = lib.llvq_gemv(ctx, to_dev_u8(stream), to_dev_f16(gain), n_out, k_in, to_dev_bf16(x), y_dtype=torch.bfloat16)
    y32 = lib.llvq_gemv(ctx, to_dev_u8(stream), to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    ref = o.gemv(stream, gain, n_out, k_in, x, threads=_threads())
    assert gemv_error(y.float().cpu().numpy(), ref) <= TOL_BF16_OUT
    assert gemv_error(y32.cpu().numpy(), ref) <= TOL
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_argument_checks(lib, ctxs):
    ctx = ctxs[(2, 13)]
    idx = torch.zeros(64, dtype=torch.uint8, device="cuda")
    pts = torch.zeros((4, 24), dtype=torch.int8, device="cuda")
    L = ctx._lib
    assert L.llvq_decode_blocks(ctx._h, None, 4, pts.data_ptr(), None) == 1           # EINVAL
    assert L.llvq_decode_blocks(ctx._h, idx.data_ptr() + 4, 4, pts.data_ptr(), None) == 2   # EALIGN
    assert L.llvq_decode_blocks(ctx._h, idx.data_ptr(), 4, pts.data_ptr() + 1, None) == 2
    g = torch.zeros(8, dtype=torch.float16, device="cuda")
    w = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    assert L.llvq_dequant_matrix(ctx._h, idx.data_ptr(), g.data_ptr(), 2, 24, 7, w.data_ptr(), 24, None) == 1
    assert L.llvq_dequant_matrix(ctx._h, idx.data_ptr(), g.data_ptr(), 2, 24, 1, w.data_ptr(), 8, None) == 1
    assert L.llvq_gemv(ctx._h, idx.data_ptr(), g.data_ptr(), 2, 24, w.data_ptr(), w.data_ptr(), 9, None) == 1
    assert L.llvq_gemv(ctx._h, idx.data_ptr(), g.data_ptr(), 2, 10_000_000, w.data_ptr(), w.data_ptr(), 0, None) == 3   # x does not fit shared memory
    torch.cuda.synchronize()


# --------------------------------------------------------------------------
# small-batch GEMM on the tensor cores
# --------------------------------------------------------------------------
def _gemm_check(lib, ctx, o, n_out, k_in, batch, seed, repeat=1):
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=seed)
    X = gen.normal_bf16((batch, k_in), seed=seed)
    want = o.gemm(stream, gain, n_out, k_in, X, threads=8)
    d_idx, d_gain, d_x = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(X)
    for _ in range(repeat):
        y = lib.llvq_gemm_small_batch(ctx, d_idx, d_gain, n_out, k_in, d_x)
        torch.cuda.synchronize()
        assert lib.llvq_last_error(ctx) == (0, 0)
        got = y.float().cpu().numpy()
        assert got.shape == (batch, n_out)
        scale = np.abs(want).max()
        err = np.abs(got - want) / np.maximum(np.abs(want), 1e-3 * scale)
        assert err.max() <= TOL_BF16_OUT, (err.max(), np.unravel_index(err.argmax(), err.shape))


@pytest.mark.parametrize("n_out,k_in,batch", [(128, 96, 16), (300, 1000, 16), (300, 1000, 64), (129, 192, 1),
                                              (257, 4104, 7), (640, 2048, 33), (100, 24, 64)])
def test_gemm_small_batch_2bit(lib, ctxs, oracle_mod, n_out, k_in, batch):
    _gemm_check(lib, ctxs[(2, 13)], _oracle(oracle_mod)((2, 13)), n_out, k_in, batch, seed=7, repeat=2)


@pytest.mark.parametrize("code,n_out,k_in,batch", [((2, 53), 200, 1000, 16), ((2, 53), 130, 480, 64), ((2, 2), 256, 768, 5)])
def test_gemm_small_batch_other_codes(lib, ctxs, oracle_mod, code, n_out, k_in, batch):
    _gemm_check(lib, ctxs[code], _oracle(oracle_mod)(code), n_out, k_in, batch, seed=8)


@pytest.mark.parametrize("batch", [16, 64])
def test_gemm_code_whose_tables_leave_no_room_for_two_buffer_sets(lib, oracle_mod, batch):
    # shells 2..16: 788 classes, tables still in shared memory but too large for the kernel without a block barrier,
    # so the product runs through the kernel with the two alternating thread groups
    ctx = lib.Context(2, 16, device=0)
    _gemm_check(lib, ctx, _oracle(oracle_mod)((2, 16)), 300, 1000, batch, seed=9)


@pytest.mark.parametrize("code", [(2, 13), (2, 53)])
def test_products_on_a_stream_with_out_of_range_fields(lib, ctxs, oracle_mod, code):
    # fields >= N decode to the zero block and are counted once per launch, whatever kernel serves the product
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    n_out, k_in = 300, 1000                                 # 42 blocks per row: ragged domains and units
    stream, gain, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=27)
    idx = o.unpack(stream, nblocks)
    for b in (0, 41, 42 * 128 + 5, 42 * 200 + 17, nblocks - 1):
        idx[b] = o.N + b                                     # still below 2^W
    lo, hi = gen.indices_to_arrays(idx)
    stream = gen.pack_indices(lo, hi, o.W)
    d_idx, d_gain = to_dev_u8(stream), to_dev_f16(gain)
    x = gen.normal_bf16(k_in, seed=27)
    y = lib.llvq_gemv(ctx, d_idx, d_gain, n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (5, 0)
    assert gemv_error(y.cpu().numpy(), o.gemv(stream, gain, n_out, k_in, x)) <= TOL
    for batch in (16, 64):
        X = gen.normal_bf16((batch, k_in), seed=batch)
        want = o.gemm(stream, gain, n_out, k_in, X, threads=8)
        Y = lib.llvq_gemm_small_batch(ctx, d_idx, d_gain, n_out, k_in, to_dev_bf16(X))
        torch.cuda.synchronize()
        assert lib.llvq_last_error(ctx) == (5, 0)
        err = np.abs(Y.float().cpu().numpy() - want) / np.maximum(np.abs(want), 1e-3 * np.abs(want).max())
        assert err.max() <= TOL_BF16_OUT


@pytest.mark.parametrize("code", [(2, 13), (2, 53)])
def test_gemm_stored_stream_and_sorted_layout_agree_on_random_shapes(lib, ctxs, code):
    # the kernels that serve the stored stream (domains ordered inside the kernel, one, two or four per round, or unordered
    # chunks) and the sorted layout unrank the same blocks: their products may differ by the accumulation order only.  Both
    # are compared with the oracle elsewhere; this sweep runs through many ragged shapes and every padded batch cheaply.
    ctx = ctxs[code]
    rng = np.random.default_rng(31)
    for case in range(14):
        n_out, k_in = int(rng.integers(1, 900)), int(rng.integers(1, 260)) * 8
        batch = [1, 16, 17, 32, 33, 48, 49, 64][case % 8]
        stream, gain, _ = gen.make_layer(ctx.num_points, ctx.index_bits, n_out, k_in, 1, seed=100 + case)
        X = to_dev_bf16(gen.normal_bf16((batch, k_in), seed=case))
        d_idx, d_gain = to_dev_u8(stream), to_dev_f16(gain)
        y1 = lib.llvq_gemm_small_batch(ctx, d_idx, d_gain, n_out, k_in, X).float()
        y2 = lib.llvq_gemm_small_batch_sorted(ctx, lib.llvq_sort_blocks_gemm(ctx, d_idx, n_out, k_in), d_gain, n_out, k_in, X).float()
        torch.cuda.synchronize()
        assert lib.llvq_last_error(ctx) == (0, 0)
        floor = 1e-3 * y2.abs().max().clamp_min(1e-30)
        err = ((y1 - y2).abs() / y2.abs().clamp_min(floor)).max().item()
        assert err <= 2.0 ** -7, (err, n_out, k_in, batch)          # one bf16 step at most


def test_gemm_exact_integer_case(lib, ctxs, oracle_mod):
    # gains = 1, X = 0/1 patterns: every partial sum is a small integer, exact in binary32 and in bf16
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n_out, k_in, batch = 200, 480, 16
    stream, _, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=9)
    ones = np.full(nblocks, 0x3C00, dtype=np.uint16)
    pts, _ = o.decode_stream(stream, nblocks)
    Wint = pts.reshape(n_out, -1)[:, :k_in].astype(np.int64)
    X = np.zeros((batch, k_in), dtype=np.float32)
    for b in range(batch):
        X[b, b * 30:(b + 1) * 30:3] = 1.0
    y = lib.llvq_gemm_small_batch(ctx, to_dev_u8(stream), to_dev_f16(ones), n_out, k_in, to_dev_bf16(gen.f32_to_bf16_bits(X)))
    torch.cuda.synchronize()
    assert np.array_equal(y.float().cpu().numpy().astype(np.int64), X.astype(np.int64) @ Wint.T)


def test_gemm_matches_gemv_rows(lib, ctxs, oracle_mod):
    # batch rows are independent: row b of the GEMM equals the GEMV with x = X[b] up to accumulation order
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n_out, k_in, batch = 384, 1536, 16
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=10)
    X = gen.normal_bf16((batch, k_in), seed=10)
    d = (to_dev_u8(stream), to_dev_f16(gain))
    Y = lib.llvq_gemm_small_batch(ctx, *d, n_out, k_in, to_dev_bf16(X)).float()
    for b in (0, 7, 15):
        y = lib.llvq_gemv(ctx, *d, n_out, k_in, to_dev_bf16(X[b]))
        torch.cuda.synchronize()
        ref = y.cpu().numpy().astype(np.float64)
        assert gemv_error(Y[b].cpu().numpy(), ref) <= 2.0 ** -8 + 1e-4


# --------------------------------------------------------------------------
# full benchmark sizes, in the launch configuration bench.py times
# --------------------------------------------------------------------------
def test_dequant_full_size_config2(lib, ctxs, oracle_mod):
    # 4096 x 4096 FLAT, 699051 blocks (the last one holds 16 real weights), 48-bit indices: every element compared
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    rows = cols = 4096
    stream, gain, nblocks = gen.make_layer(o.N, o.W, rows, cols, 0, seed=0)
    assert nblocks == 699051
    got = lib.llvq_dequant_matrix(ctx, to_dev_u8(stream), to_dev_f16(gain), rows, cols, 0)
    torch.cuda.synchronize()
    want = o.dequant_matrix(stream, gain, rows, cols, 0)
    assert np.array_equal(bf16_bits(got), want)
    assert lib.llvq_last_error(ctx) == (0, 0)


_CONFIG4_LAYER = {}


def _config4_rows(n_out, batch):
    """Output rows the oracle recomputes: all of them at batch 16; at batch 64 every row of eight whole 128-row tiles
    (the first two, the last, and five spread over the thread blocks' boundaries in between)."""
    if batch <= 16:
        return [(0, n_out)]
    tiles = n_out // 128
    picks = sorted({0, 1, tiles - 1} | {(tiles * j) // 6 + j for j in range(1, 6)})
    return [(t * 128, 128) for t in picks]


@pytest.mark.parametrize("batch", [16, 64])
@pytest.mark.parametrize("n_out,k_in", [(8192, 8192), (28672, 8192), (8192, 28672)])
@pytest.mark.parametrize("code", [(2, 13), (2, 53)])
def test_gemm_full_size_config4(lib, ctxs, oracle_mod, code, n_out, k_in, batch):
    # every cell of the 70B-shaped configuration: three shapes x two batch sizes x the ~2 and ~3 bits/weight codes, on the
    # stored stream and on the sorted layout, in the launch configuration bench.py times
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    key = (code, n_out, k_in)
    if _CONFIG4_LAYER.get("key") != key:                   # the two batch sizes of a cell share the generated layer
        _CONFIG4_LAYER.clear()
        _CONFIG4_LAYER.update(key=key, layer=gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=0))
    stream, gain, _ = _CONFIG4_LAYER["layer"]
    X = gen.normal_bf16((batch, k_in), seed=0)
    d_idx, d_gain, d_x = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(X)
    Y = lib.llvq_gemm_small_batch(ctx, d_idx, d_gain, n_out, k_in, d_x).float().cpu().numpy()
    srt = lib.llvq_sort_blocks_gemm(ctx, d_idx, n_out, k_in)
    Ys = lib.llvq_gemm_small_batch_sorted(ctx, srt, d_gain, n_out, k_in, d_x).float().cpu().numpy()
    del srt, d_idx
    assert np.isfinite(Y).all() and np.isfinite(Ys).all()
    spans = _config4_rows(n_out, batch)
    ref = np.concatenate([o.gemm(stream, gain, n_out, k_in, X, rows=sp, threads=_threads())[:, sp[0]:sp[0] + sp[1]] for sp in spans], axis=1)
    cols = np.concatenate([np.arange(a, a + c) for a, c in spans])
    assert len(cols) >= min(n_out, 1024)
    # over 10^5 outputs of 28672-term sums the tail of the tensor cores' truncating accumulation shows in the few
    # outputs that are a thousand times smaller than the largest: gemm_error allows for it (see gpu_util)
    for got in (Y, Ys):
        assert gemm_error(got[:, cols], ref, k_in) <= TOL_BF16_OUT
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_smallest_and_odd_shapes(lib, ctxs, oracle_mod):
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    for n_out, k_in, batch in [(1, 8, 1), (1, 24, 64), (17, 40, 3), (2049, 72, 2)]:
        stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=12)
        X = gen.normal_bf16((batch, k_in), seed=12)
        want = o.gemm(stream, gain, n_out, k_in, X)
        d = (to_dev_u8(stream), to_dev_f16(gain))
        Y = lib.llvq_gemm_small_batch(ctx, *d, n_out, k_in, to_dev_bf16(X)).float().cpu().numpy()
        y = lib.llvq_gemv(ctx, *d, n_out, k_in, to_dev_bf16(X[0])).cpu().numpy()
        torch.cuda.synchronize()
        scale = np.abs(want).max()
        assert (np.abs(Y - want) / np.maximum(np.abs(want), 1e-3 * scale)).max() <= TOL_BF16_OUT
        assert gemv_error(y, want[0]) <= TOL
    # zero-sized calls are accepted and touch nothing
    assert lib.llvq_dequant_matrix(ctx, torch.zeros(16, dtype=torch.uint8, device="cuda"), torch.zeros(1, dtype=torch.float16, device="cuda"),
                                   0, 24, 1).numel() == 0


def test_bounded_wait_reports_timeout_and_context_stays_usable(lib, ctxs, oracle_mod):
    # a wait nothing satisfies runs into its iteration limit: the kernel returns, the flag is set, later calls work
    ctx = ctxs[(2, 2)]
    assert lib.llvq_last_error(ctx) == (0, 0)
    lib.llvq_selftest_wait_timeout(ctx)
    assert lib.llvq_last_error(ctx) == (0, 1)            # LLVQ_FLAG_WAIT_TIMEOUT
    assert lib.llvq_last_error(ctx) == (0, 0)            # cleared by the read
    o = _oracle(oracle_mod)((2, 2))
    lo = np.arange(100, dtype=np.uint64)
    assert np.array_equal(_decode_gpu(lib, ctx, lo, np.zeros_like(lo)), o.unrank_arrays(lo, np.zeros_like(lo)))


# --------------------------------------------------------------------------
# sorted layout: rearrange once, then the fused GEMV on the sorted stream
# --------------------------------------------------------------------------
def _sm_count():
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("code,n_out,k_in", [((2, 13), 67, 4096), ((2, 13), 16, 384), ((2, 13), 129, 1000), ((2, 13), 1, 24),
                                             ((2, 13), 3000, 96), ((2, 2), 256, 768), ((3, 3), 33, 4104)])
def test_gemv_sorted_small_shapes(lib, ctxs, oracle_mod, code, n_out, k_in):
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=14)
    x = gen.normal_bf16(k_in, seed=14)
    want = o.gemv(stream, gain, n_out, k_in, x)
    srt = lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n_out, k_in)
    assert srt.numel() == 256 * ((n_out + 7) // 8) * (((k_in + 23) // 24 + 3) // 4)
    y32 = lib.llvq_gemv_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    y16 = lib.llvq_gemv_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x), y_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert gemv_error(y32.cpu().numpy(), want) <= TOL
    assert gemv_error(y16.float().cpu().numpy(), want) <= TOL_BF16_OUT
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_sort_blocks_is_a_permutation_of_the_blocks(lib, ctxs, oracle_mod):
    # every block of the matrix appears exactly once, with its stored index unchanged, inside the range of units of
    # the thread block that owns it; entries of one range are ordered by decoder form, unranking steps and class
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n_out, k_in = 523, 1000                                 # 42 blocks per row, 11 units per row group, ragged in both directions
    bpr, nq, groups = 42, 11, 66
    stream, _, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=15)
    idx = o.unpack(stream, nblocks)
    idx[7] = o.N                                            # one out-of-range field
    lo, hi = gen.indices_to_arrays(idx)
    stream = gen.pack_indices(lo, hi, o.W)
    srt = lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n_out, k_in)
    torch.cuda.synchronize()
    assert lib.llvq_last_error(ctx) == (1, 0)
    e = srt.cpu().numpy().view(np.uint64)
    U, G = groups * nq, min(groups * nq, _sm_count())
    assert e.size == U * 32
    cls = o.classes()
    offs = np.array([c["offset"] for c in cls] + [o.N], dtype=np.uint64)

    def form(c):
        k = cls[c]
        if k["parity"]:
            return (0, -(len(k["values"]) - 1), c)
        g1 = sum(1 for v in k["values"] if v % 4 == 2)
        g0 = len(k["values"]) - g1
        return (1 if k["w"] in (8, 12, 16) else 2, -(max(g1 - 1, 0) + max(g0 - 1, 0)), c)

    seen = set()
    for cta in range(G):
        u0, u1 = cta * U // G, (cta + 1) * U // G
        seg = e[u0 * 32:u1 * 32]                             # a single segment and a single pass at this size
        keys = []
        for ent in seg.tolist():
            I, pos = ent & ((1 << 48) - 1), ent >> 48
            u, lane = u0 + pos // 32, pos % 32
            rg, kq = divmod(u, nq)
            row, cb = rg * 8 + lane // 4, kq * 4 + lane % 4
            assert u < u1
            if I == (1 << 48) - 1:
                assert row >= n_out or cb >= bpr or row * bpr + cb == 7
                keys.append((3, 0, 0))
                continue
            b = row * bpr + cb
            assert idx[b] == I and b not in seen
            seen.add(b)
            keys.append(form(int(np.searchsorted(offs, np.uint64(I), side="right")) - 1))
        assert keys == sorted(keys)
    assert len(seen) == nblocks - 1


@pytest.mark.parametrize("n_out,k_in", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_gemv_sorted_full_size_layers_all_rows(lib, ctxs, oracle_mod, n_out, k_in):
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=0)
    x = gen.normal_bf16(k_in, seed=0)
    srt = lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n_out, k_in)
    y = lib.llvq_gemv_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x), y_dtype=torch.bfloat16)
    y32 = lib.llvq_gemv_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    ref = o.gemv(stream, gain, n_out, k_in, x, threads=_threads())          # every output row
    assert gemv_error(y.float().cpu().numpy(), ref) <= TOL_BF16_OUT
    assert gemv_error(y32.cpu().numpy(), ref) <= TOL
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_gemv_sorted_many_row_groups_per_thread_block(lib, ctxs, oracle_mod):
    # narrow and tall: every thread block owns more row groups than it keeps sums for at a time (several passes)
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n_out, k_in = 8 * 130 * _sm_count() + 5, 48
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=3)
    x = gen.normal_bf16(k_in, seed=3)
    srt = lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n_out, k_in)
    y = lib.llvq_gemv_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    y2 = lib.llvq_gemv(ctx, to_dev_u8(stream), to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    ref = o.gemv(stream, gain, n_out, k_in, x, threads=4)                     # all rows: two blocks each
    assert gemv_error(y.cpu().numpy(), ref) <= TOL
    assert gemv_error(y2.cpu().numpy(), ref) <= TOL                           # the kernel on the stored stream takes several passes too
    assert lib.llvq_last_error(ctx) == (0, 0)
    assert lib.llvq_last_error(ctx) == (0, 0)


@pytest.mark.parametrize("n_out,k_in", [(14336, 4096), (1024, 4096), (4096, 14336), (28672, 4096), (6144, 4096)])
def test_gemv_decoder_sweep_shapes_all_rows(lib, ctxs, oracle_mod, n_out, k_in):
    # the layer shapes of the 8B-decoder sweep the benchmark times (gate/up, k/v, down, and q|k|v, gate|up stored as one),
    # stored stream and sorted layout; the oracle recomputes every output row
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=50)
    x = gen.normal_bf16(k_in, seed=50)
    ds, dg, dx = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(x)
    y = lib.llvq_gemv(ctx, ds, dg, n_out, k_in, dx, y_dtype=torch.bfloat16).float().cpu().numpy()
    ys = lib.llvq_gemv_sorted(ctx, lib.llvq_sort_blocks(ctx, ds, n_out, k_in), dg, n_out, k_in, dx,
                              y_dtype=torch.bfloat16).float().cpu().numpy()
    ref = o.gemv(stream, gain, n_out, k_in, x, threads=_threads())
    for got in (y, ys):
        assert gemv_error(got, ref) <= TOL_BF16_OUT
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_gemv_at_the_largest_row_count(lib, ctxs, oracle_mod):
    # 64 * 65536 rows is the most the scratch rows, arrival counters and pair slots of a context are sized for
    o = _oracle(oracle_mod)((2, 2))
    ctx = ctxs[(2, 2)]
    n_out, k_in = 64 * 65536, 24
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=9)
    x = gen.normal_bf16(k_in, seed=9)
    ds, dg, dx = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(x)
    y = lib.llvq_gemv(ctx, ds, dg, n_out, k_in, dx)
    ys = lib.llvq_gemv_sorted(ctx, lib.llvq_sort_blocks(ctx, ds, n_out, k_in), dg, n_out, k_in, dx)
    torch.cuda.synchronize()
    assert torch.equal(y, ys)                                  # one block per row: no summation order to differ in
    ref = o.gemv(stream, gain, n_out, k_in, x, threads=_threads())            # every row
    assert gemv_error(y.cpu().numpy(), ref) <= TOL
    assert lib.llvq_last_error(ctx) == (0, 0)
    # one row group more is refused, not truncated (nothing is launched, so the short buffers do not matter)
    assert ctx._lib.llvq_gemv(ctx._h, ds.data_ptr(), dg.data_ptr(), n_out + 8, k_in, dx.data_ptr(), y.data_ptr(), 0, None) == 3


@pytest.mark.parametrize("n_out,k_in", [(4096, 4096), (200, 1000), (129, 24)])
def test_gemv_72bit_stored_and_sorted_all_rows(lib, ctxs, oracle_mod, n_out, k_in):
    # the ~3 bits/weight code: the fused product on the stored stream and on the sorted layout (for this code the layout
    # of the small-batch product serves both), both output types, every row against the oracle
    o = _oracle(oracle_mod)((2, 53))
    ctx = ctxs[(2, 53)]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=31)
    x = gen.normal_bf16(k_in, seed=31)
    ds, dg, dx = to_dev_u8(stream), to_dev_f16(gain), to_dev_bf16(x)
    ref = o.gemv(stream, gain, n_out, k_in, x, threads=_threads())
    assert ctx._lib.llvq_sorted_bytes(ctx._h, n_out, k_in) == ctx._lib.llvq_sorted_gemm_bytes(ctx._h, n_out, k_in) > 0
    srt = lib.llvq_sort_blocks(ctx, ds, n_out, k_in)
    assert torch.equal(srt, lib.llvq_sort_blocks_gemm(ctx, ds, n_out, k_in))
    for dt, tol in ((torch.float32, TOL), (torch.bfloat16, TOL_BF16_OUT)):
        y = lib.llvq_gemv(ctx, ds, dg, n_out, k_in, dx, y_dtype=dt)
        ys = lib.llvq_gemv_sorted(ctx, srt, dg, n_out, k_in, dx, y_dtype=dt)
        torch.cuda.synchronize()
        assert gemv_error(y.float().cpu().numpy(), ref) <= tol
        assert gemv_error(ys.float().cpu().numpy(), ref) <= tol
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_back_to_back_launches_see_the_previous_result(lib, ctxs, oracle_mod):
    # the kernels start before their predecessor in the stream has finished (programmatic dependent launch) and must
    # wait before reading its output: y1 = W1 x, y2 = W2 y1, y3 = W3 y2 queued without any synchronisation in between,
    # repeated so that stale data from the previous round would show
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n = 1536
    layers = [gen.make_layer(o.N, o.W, n, n, 1, seed=40 + j)[:2] for j in range(3)]
    dev = [(to_dev_u8(s), to_dev_f16(g)) for s, g in layers]
    srt = [lib.llvq_sort_blocks(ctx, d[0], n, n) for d in dev]
    ys = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    for use_sorted in (False, True):
        for rnd in range(3):
            x = gen.normal_bf16(n, seed=50 + rnd)
            d_x = to_dev_bf16(x)
            cur = d_x
            for j in range(3):
                if use_sorted:
                    lib.llvq_gemv_sorted(ctx, srt[j], dev[j][1], n, n, cur, d_y=ys[j])
                else:
                    lib.llvq_gemv(ctx, dev[j][0], dev[j][1], n, n, cur, d_y=ys[j])
                cur = ys[j]
            torch.cuda.synchronize()
            ref_in = x
            for j in range(3):
                ref = o.gemv(layers[j][0], layers[j][1], n, n, ref_in, threads=4)
                got = ys[j].float().cpu().numpy()
                assert gemv_error(got, ref) <= TOL_BF16_OUT, (use_sorted, rnd, j)
                ref_in = bf16_bits(ys[j])                    # the next layer's reference starts from what the device produced
    assert lib.llvq_last_error(ctx) == (0, 0)


# --------------------------------------------------------------------------
# sorted layout of the small-batch product
# --------------------------------------------------------------------------
@pytest.mark.parametrize("code,n_out,k_in,batch", [((2, 13), 200, 480, 3), ((2, 13), 129, 1000, 16), ((2, 13), 1000, 2000, 33),
                                                   ((2, 13), 64, 4096, 64), ((2, 13), 1, 24, 1), ((2, 2), 256, 768, 16),
                                                   ((3, 3), 130, 4104, 20), ((2, 53), 200, 480, 3), ((2, 53), 300, 2000, 33),
                                                   ((2, 53), 129, 1000, 64)])
def test_gemm_sorted_small_shapes(lib, ctxs, oracle_mod, code, n_out, k_in, batch):
    o = _oracle(oracle_mod)(code)
    ctx = ctxs[code]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=24)
    x = gen.normal_bf16((batch, k_in), seed=24)
    want = o.gemm(stream, gain, n_out, k_in, x, threads=4)
    srt = lib.llvq_sort_blocks_gemm(ctx, to_dev_u8(stream), n_out, k_in)
    entry_bytes = 12 if o.W > 48 else 8                      # the 72-bit code keeps index, class within its bucket and position in 96 bits
    assert srt.numel() == 1024 * entry_bytes * ((n_out + 127) // 128) * (((k_in + 23) // 24 + 7) // 8)
    y = lib.llvq_gemm_small_batch_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    y_plain = lib.llvq_gemm_small_batch(ctx, to_dev_u8(stream), to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    assert gemv_error(y.float().cpu().numpy(), want) <= TOL_BF16_OUT
    assert gemv_error(y.float().cpu().numpy(), y_plain.float().cpu().numpy().astype(np.float64)) <= 2.0 ** -7
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_sort_blocks_gemm_is_a_permutation_inside_every_domain(lib, ctxs, oracle_mod):
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n_out, k_in = 300, 1000                                 # 3 row tiles (the last ragged), 42 blocks per row -> 6 domains (the last ragged)
    bpr, nd = 42, 6
    stream, _, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=25)
    idx = o.unpack(stream, nblocks)
    e = lib.llvq_sort_blocks_gemm(ctx, to_dev_u8(stream), n_out, k_in).cpu().numpy().view(np.uint64).reshape(3 * nd, 1024)
    offs = np.array([c["offset"] for c in o.classes()] + [o.N], dtype=np.uint64)
    seen = set()
    for dom in range(3 * nd):
        rt, d = divmod(dom, nd)
        last_parity_rank = -1
        positions = set()
        for ent in e[dom].tolist():
            I, pos = ent & ((1 << 48) - 1), ent >> 48
            row, cb = rt * 128 + pos // 8, d * 8 + pos % 8
            assert pos < 1024 and pos not in positions
            positions.add(pos)
            if I == (1 << 48) - 1:
                assert row >= n_out or cb >= bpr
                last_parity_rank = 2
                continue
            b = row * bpr + cb
            assert idx[b] == I and b not in seen
            seen.add(b)
            parity_rank = 0 if o.class_info(int(np.searchsorted(offs, np.uint64(I), side="right")) - 1)["parity"] else 1
            assert parity_rank >= last_parity_rank          # odd classes first, then even, then the entries without a block
            last_parity_rank = parity_rank
    assert len(seen) == nblocks
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_sort_blocks_gemm_72bit_entries(lib, ctxs, oracle_mod):
    # 96-bit entries: the class-local index (bit 63 of its two words = no block), the class (17 bits) and the position; a
    # domain is ordered by the shape of the unranking (odd classes first, then by number of steps, most first); entries
    # without a block come last
    o = _oracle(oracle_mod)((2, 53))
    ctx = ctxs[(2, 53)]
    n_out, k_in = 200, 1000                                 # 2 row tiles, 42 blocks per row -> 6 domains per tile, ragged both ways
    bpr, nd = 42, 6
    stream, _, nblocks = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=26)
    idx = o.unpack(stream, nblocks)
    e = lib.llvq_sort_blocks_gemm(ctx, to_dev_u8(stream), n_out, k_in).cpu().numpy().view(np.uint32).reshape(2 * nd, 1024, 3)
    classes = o.classes()
    offs = [c["offset"] for c in classes] + [o.N]
    import bisect

    def steps(c):
        if c["parity"]:
            return len(c["values"]) - 1
        g1 = sum(1 for v in c["values"] if v % 4 == 2)
        g0 = len(c["values"]) - g1
        return max(g1 - 1, 0) + max(g0 - 1, 0)
    seen = set()
    for dom in range(2 * nd):
        rt, d = divmod(dom, nd)
        positions, last_key, ended = set(), (-1, -99), False
        for w0, w1, w2 in e[dom].tolist():
            pos = w2 >> 17
            row, cb = rt * 128 + pos // 8, d * 8 + pos % 8
            assert pos not in positions
            positions.add(pos)
            if w1 >> 31:
                assert row >= n_out or cb >= bpr
                ended = True                                # nothing with a block may follow
                continue
            assert not ended
            b = row * bpr + cb
            I = int(idx[b])
            assert b not in seen
            seen.add(b)
            cls = bisect.bisect_right(offs, I) - 1
            assert w2 & 0x1ffff == cls and (w0 | w1 << 32) == I - offs[cls]
            key = (1 - classes[cls]["parity"], -steps(classes[cls]))
            assert key >= last_key
            last_key = key
    assert len(seen) == nblocks
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_gemm_sorted_unsupported_and_arguments(lib, ctxs):
    buf = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    p = buf.data_ptr()
    big = ctxs[(2, 53)]
    assert big._lib.llvq_sorted_gemm_bytes(big._h, 64, 96) == 1024 * 12
    ctx = ctxs[(2, 13)]
    assert ctx._lib.llvq_sorted_gemm_bytes(ctx._h, 64, 96) == 1024 * 8
    assert ctx._lib.llvq_gemm_small_batch_sorted(ctx._h, p, p, 16, 96, p, 65, p, None) == 1       # batch out of range
    assert ctx._lib.llvq_gemm_small_batch_sorted(ctx._h, p, p, 16, 100, p, 4, p, None) == 2      # k_in not a multiple of 8
    assert ctx._lib.llvq_gemm_small_batch_sorted(ctx._h, None, None, 0, 96, None, 4, None, None) == 0


@pytest.mark.parametrize("n_out,k_in", [(72, 14336), (40, 20000), (24, 40008)])
def test_gemv_wide_rows(lib, ctxs, oracle_mod, n_out, k_in):
    # long rows: the x slice takes more shared memory, so the kernel bins smaller segments (or not at all)
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    stream, gain, _ = gen.make_layer(o.N, o.W, n_out, k_in, 1, seed=60)
    x = gen.normal_bf16(k_in, seed=60)
    want = o.gemv(stream, gain, n_out, k_in, x, threads=4)
    y = lib.llvq_gemv(ctx, to_dev_u8(stream), to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    srt = lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n_out, k_in)
    y2 = lib.llvq_gemv_sorted(ctx, srt, to_dev_f16(gain), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    assert gemv_error(y.cpu().numpy(), want) <= TOL
    assert gemv_error(y2.cpu().numpy(), want) <= TOL
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_chain_of_launches_replays_from_a_cuda_graph(lib, ctxs, oracle_mod):
    # the entry points only enqueue kernels: a three-layer chain captured once into a CUDA graph gives, on every replay
    # with new activations, what the directly launched chain gives
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    n = 1536
    layers = [gen.make_layer(o.N, o.W, n, n, 1, seed=70 + j)[:2] for j in range(3)]
    dev = [(to_dev_u8(s), to_dev_f16(g)) for s, g in layers]
    x = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    ys = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(3)]

    def chain():
        cur = x
        for j in range(3):
            lib.llvq_gemv(ctx, dev[j][0], dev[j][1], n, n, cur, d_y=ys[j])
            cur = ys[j]

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        chain()                                              # first use of the kernels outside the capture
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        chain()
    for rnd in range(3):
        xin = gen.normal_bf16(n, seed=80 + rnd)
        x.copy_(to_dev_bf16(xin))
        graph.replay()
        torch.cuda.synchronize()
        got = ys[2].float().cpu().numpy()
        ref_in = xin
        for j in range(3):
            ref = o.gemv(layers[j][0], layers[j][1], n, n, ref_in, threads=4)
            if j == 2:
                assert gemv_error(got, ref) <= TOL_BF16_OUT, rnd
            ref_in = bf16_bits(ys[j])
    assert lib.llvq_last_error(ctx) == (0, 0)


# --------------------------------------------------------------------------
# several matrices in one launch
# --------------------------------------------------------------------------
@pytest.mark.parametrize("sorted_layout", [False, True])
@pytest.mark.parametrize("y_dtype", [torch.float32, torch.bfloat16])
def test_gemv_multi_seven_ragged_matrices(lib, ctxs, oracle_mod, sorted_layout, y_dtype):
    # seven matrices of different, ragged shapes (row counts that are not multiples of 8, column counts that are not
    # multiples of 24 or 96, two different inputs shared by some matrices) in one call, every row against the oracle
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    shapes = [(1203, 1000), (517, 1000), (517, 1000), (1000, 2040), (2049, 1000), (1500, 4104), (999, 24 * 7)]
    xs = {k: gen.normal_bf16(k, seed=k) for k in sorted({k for _, k in shapes})}
    d_xs = {k: to_dev_bf16(v) for k, v in xs.items()}
    mats, refs, outs = [], [], []
    for i, (n, k) in enumerate(shapes):
        stream, gain, _ = gen.make_layer(o.N, o.W, n, k, 1, seed=80 + i)
        d_w = to_dev_u8(stream)
        if sorted_layout:
            d_w = lib.llvq_sort_blocks(ctx, d_w, n, k)
        d_y = torch.full((n,), float("nan"), dtype=y_dtype, device="cuda")
        mats.append((d_w, to_dev_f16(gain), n, k, d_xs[k], d_y))
        outs.append(d_y)
        refs.append(o.gemv(stream, gain, n, k, xs[k], threads=_threads()))
    call = lib.llvq_gemv_sorted_multi if sorted_layout else lib.llvq_gemv_multi
    for _ in range(2):                                        # twice: the shared scratch must come back clean
        for d_y in outs:
            d_y.fill_(float("nan"))
        call(ctx, mats, y_dtype=y_dtype)
        torch.cuda.synchronize()
        for d_y, ref in zip(outs, refs):
            assert gemv_error(d_y.float().cpu().numpy(), ref) <= (TOL if y_dtype == torch.float32 else TOL_BF16_OUT)
    assert lib.llvq_last_error(ctx) == (0, 0)
    # the single-matrix calls still work afterwards on the same context (scratch rows and counters are zero again)
    d_w, d_g, n, k, d_x, _ = mats[0]
    y1 = (lib.llvq_gemv_sorted if sorted_layout else lib.llvq_gemv)(ctx, d_w, d_g, n, k, d_x)
    assert gemv_error(y1.cpu().numpy(), refs[0]) <= TOL


def test_gemv_multi_full_size_step_and_limits(lib, ctxs, oracle_mod):
    # the three 7B-shaped layers of the benchmark step in one call, sorted layout, every row against the oracle
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    shapes = [(4096, 4096), (11008, 4096), (4096, 11008)]
    mats, refs = [], []
    for i, (n, k) in enumerate(shapes):
        stream, gain, _ = gen.make_layer(o.N, o.W, n, k, 1, seed=i)
        x = gen.normal_bf16(k, seed=i)
        d_y = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        mats.append((lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n, k), to_dev_f16(gain), n, k, to_dev_bf16(x), d_y))
        refs.append(o.gemv(stream, gain, n, k, x, threads=_threads()))
    lib.llvq_gemv_sorted_multi(ctx, mats, y_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    for m, ref in zip(mats, refs):
        assert gemv_error(m[5].float().cpu().numpy(), ref) <= TOL_BF16_OUT
    # nine matrices, and a matrix with fewer work units than the device has SMs, are refused
    with pytest.raises(lib.LlvqError):
        lib.llvq_gemv_sorted_multi(ctx, mats * 3, y_dtype=torch.bfloat16)
    tiny = (mats[0][0], mats[0][1], 8, 24, mats[0][4], mats[0][5])
    with pytest.raises(lib.LlvqError):
        lib.llvq_gemv_sorted_multi(ctx, [tiny], y_dtype=torch.bfloat16)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_gemv_sorted_multi_takes_the_kernel_with_barriers_where_a_share_needs_several_passes(lib, ctxs, oracle_mod):
    # tall, narrow matrices: a thread block's share covers more row groups than it keeps sums for at a time, so the
    # multi-matrix call cannot let its warps run ahead into the next matrix and uses the kernel with a block barrier
    # between the matrices; a call with a single matrix does too
    o = _oracle(oracle_mod)((2, 13))
    ctx = ctxs[(2, 13)]
    mats, refs = [], []
    for i, (n, k) in enumerate([(8 * 140 * _sm_count() + 3, 24), (8 * 131 * _sm_count(), 48)]):
        stream, gain, _ = gen.make_layer(o.N, o.W, n, k, 1, seed=90 + i)
        x = gen.normal_bf16(k, seed=90 + i)
        mats.append((lib.llvq_sort_blocks(ctx, to_dev_u8(stream), n, k), to_dev_f16(gain), n, k, to_dev_bf16(x),
                     torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")))
        refs.append(o.gemv(stream, gain, n, k, x, threads=_threads()))
    lib.llvq_gemv_sorted_multi(ctx, mats)
    torch.cuda.synchronize()
    for m, ref in zip(mats, refs):
        assert gemv_error(m[5].cpu().numpy(), ref) <= TOL
    mats[0][5].fill_(float("nan"))
    lib.llvq_gemv_sorted_multi(ctx, mats[:1])
    torch.cuda.synchronize()
    assert gemv_error(mats[0][5].cpu().numpy(), refs[0]) <= TOL
    assert lib.llvq_last_error(ctx) == (0, 0)
