"""Parity of the shape-gain entry points (gain codebook, optional row scale) against the CPU oracle, through
the C ABI.  Dequantized weights are bit-exact; fused products within the stated tolerance."""
import numpy as np
import pytest
import torch

import llvq_inputs as gen
from gpu_util import bf16_bits, gemv_error, to_dev_bf16, to_dev_u8

pytestmark = pytest.mark.gpu

TOL = 1e-3
TOL_BF16_OUT = 1e-3 + 2.0 ** -8

# (code, gain bits): the equal-rate allocations of the paper's shape-gain comparison (47+1, 46+2, 44+4 bits per block),
# the 0-bit form of the 2-bit code, and the single-shell code with a per-row scale
CASES = [((2, 12), 1), ((2, 11), 2), ((2, 10), 4), ((2, 13), 0), ((3, 3), 0)]


@pytest.fixture(scope="module")
def lib():
    import paper_2603_11021_b200 as P
    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU path"
    return P


@pytest.fixture(scope="module")
def ctxs(lib):
    return {code: lib.Context(*code, device=0) for code, _ in CASES}


@pytest.fixture(scope="module")
def codes(oracle_mod):
    return {code: oracle_mod.Code(*code) for code, _ in CASES}


def _codebook(oracle_bits):
    from oracle.gain_codebook import chi_codebook
    return chi_codebook(oracle_bits).astype(np.float32)


def _f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


@pytest.mark.parametrize("code,bits", CASES)
@pytest.mark.parametrize("scaled", [False, True])
def test_dequant_sg_bit_exact(lib, ctxs, codes, code, bits, scaled):
    o, ctx = codes[code], ctxs[code]
    assert ctx.index_bits == o.W
    rows, cols, ld = 37, 1003, 1016                        # ragged last block of every row, padded leading dimension
    stream, nblocks = gen.make_layer_sg(o.N, o.W, bits, rows, cols, seed=11)
    cb = _codebook(bits)
    rs = gen.row_scales_f32(rows, seed=4) if scaled else None
    want = o.dequant_matrix_sg(stream, bits, cb, rs, rows, cols)
    d_w = torch.zeros((rows, ld), dtype=torch.bfloat16, device="cuda")
    lib.llvq_dequant_matrix_sg(ctx, to_dev_u8(stream), bits, _f32(cb), None if rs is None else _f32(rs), rows, cols, d_w, ld)
    torch.cuda.synchronize()
    got = bf16_bits(d_w)
    assert np.array_equal(got[:, :cols], want)
    assert not got[:, cols:].any()                         # nothing written past the row
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_dequant_sg_special_scales_and_bad_fields(lib, ctxs, codes):
    code, bits = (2, 12), 1
    o, ctx = codes[code], ctxs[code]
    rows, cols = 6, 24 * 9
    lo, hi = gen.random_indices(o.N, o.W, rows * 9, seed=2)
    lo[5] = np.uint64(o.N)                                  # out of range: zeros, counted
    lo[17] = np.uint64((1 << o.W) - 1)
    k = gen.gain_indices(rows * 9, bits, seed=2)
    stream = gen.pack_indices(lo | (k << np.uint64(o.W)), hi, o.W + bits)
    cb = np.array([-4.25, 5.5], dtype=np.float32)           # a negative entry: signs flip, zeros become -0
    rs = np.array([1.0, 0.0, -0.5, 1e-30, 3e4, 0.02], dtype=np.float32)
    want = o.dequant_matrix_sg(stream, bits, cb, rs, rows, cols)
    got = bf16_bits(lib.llvq_dequant_matrix_sg(ctx, to_dev_u8(stream), bits, _f32(cb), _f32(rs), rows, cols))
    assert np.array_equal(got, want)
    assert lib.llvq_last_error(ctx) == (2, 0)


@pytest.mark.parametrize("code,bits", CASES)
def test_gemv_sg(lib, ctxs, codes, code, bits):
    o, ctx = codes[code], ctxs[code]
    n_out, k_in = 333, 2000
    stream, nblocks = gen.make_layer_sg(o.N, o.W, bits, n_out, k_in, seed=21)
    cb = _codebook(bits)
    rs = gen.row_scales_f32(n_out, seed=8)
    x = gen.normal_bf16(k_in, seed=5)
    ref = o.gemm_sg(stream, bits, cb, rs, n_out, k_in, x, threads=4)
    d_s, d_cb, d_rs, d_x = to_dev_u8(stream), _f32(cb), _f32(rs), to_dev_bf16(x)
    y = lib.llvq_gemv_sg(ctx, d_s, bits, d_cb, d_rs, n_out, k_in, d_x)
    yb = lib.llvq_gemv_sg(ctx, d_s, bits, d_cb, d_rs, n_out, k_in, d_x, y_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert gemv_error(y.cpu().numpy(), ref) <= TOL
    assert gemv_error(yb.float().cpu().numpy(), ref) <= TOL_BF16_OUT
    # the fused product uses exactly the weights the dequantizer writes
    w = lib.llvq_dequant_matrix_sg(ctx, d_s, bits, d_cb, d_rs, n_out, k_in)
    y2 = (w.double() @ d_x.double()).cpu().numpy()
    assert gemv_error(y.cpu().numpy(), y2) <= 5e-4          # binary32 accumulation only (its order varies from run to run)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_gemv_sg_exact_on_shell_four(lib, ctxs, codes):
    # Shell(4): |x| = 8, a gain of 8 gives back the integers; all-ones input -> exact integer row sums
    code = (2, 13)
    o, ctx = codes[code], ctxs[code]
    cls = o.classes()
    first = min(c["offset"] for c in cls if c["m"] == 4)
    n_out, bpr = 19, 13
    idx = [first + 7919 * i for i in range(n_out * bpr)]
    stream = gen.pack_indices(*gen.indices_to_arrays(idx), o.W)
    ones = gen.f32_to_bf16_bits(np.ones(bpr * 24, dtype=np.float32))
    y = lib.llvq_gemv_sg(ctx, to_dev_u8(stream), 0, _f32([8.0]), None, n_out, bpr * 24, to_dev_bf16(ones))
    pts = o.unrank(idx).reshape(n_out, bpr * 24)
    assert np.array_equal(y.cpu().numpy().astype(np.float64), pts.sum(axis=1).astype(np.float64))


def test_gemv_sg_full_size_sampled_rows(lib, ctxs, codes):
    code, bits = (2, 12), 1
    o, ctx = codes[code], ctxs[code]
    n_out, k_in = 4096, 4096
    stream, nblocks = gen.make_layer_sg(o.N, o.W, bits, n_out, k_in, seed=1)
    cb = _codebook(bits)
    rs = gen.row_scales_f32(n_out, seed=1)
    x = gen.normal_bf16(k_in, seed=1)
    y = lib.llvq_gemv_sg(ctx, to_dev_u8(stream), bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x)).cpu().numpy()
    import os
    ref = o.gemm_sg(stream, bits, cb, rs, n_out, k_in, x, threads=os.cpu_count() or 1)     # every output row
    assert gemv_error(y, ref) <= TOL
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_sg_argument_checks(lib, ctxs):
    ctx = ctxs[(2, 12)]
    L = ctx._lib
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    cb = torch.ones(256, dtype=torch.float32, device="cuda")
    w = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    p, c, o = buf.data_ptr(), cb.data_ptr(), w.data_ptr()
    assert L.llvq_dequant_matrix_sg(ctx._h, p, 9, c, None, 1, 24, o, 24, None) == 1          # gain bits out of range
    assert L.llvq_dequant_matrix_sg(ctx._h, p, -1, c, None, 1, 24, o, 24, None) == 1
    assert L.llvq_dequant_matrix_sg(ctx._h, p, 1, None, None, 1, 24, o, 24, None) == 1       # no codebook
    assert L.llvq_dequant_matrix_sg(ctx._h, p + 4, 1, c, None, 1, 24, o, 24, None) == 2      # misaligned stream
    assert L.llvq_dequant_matrix_sg(ctx._h, p, 1, c + 2, None, 1, 24, o, 24, None) == 2
    assert L.llvq_dequant_matrix_sg(ctx._h, p, 1, c, None, 1, 48, o, 24, None) == 1          # ld < cols
    assert L.llvq_dequant_matrix_sg(ctx._h, None, 1, None, None, 0, 24, None, 24, None) == 0 # empty: nothing to do
    assert L.llvq_gemv_sg(ctx._h, p, 1, c, None, 8, 24, None, o, 0, None) == 1
    assert int(L.llvq_field_bytes(ctx._h, 3, 1)) == 32 and int(L.llvq_field_bytes(ctx._h, 3, 9)) == 0
    big = lib.Context(2, 53, device=0)                                                       # class tables not in shared memory
    assert big._lib.llvq_dequant_matrix_sg(big._h, p, 0, c, None, 1, 24, o, 24, None) == 3
    assert lib.llvq_last_error(ctx) == (0, 0)


@pytest.mark.parametrize("code,bits", [((2, 12), 1), ((2, 11), 2), ((2, 10), 4), ((2, 13), 0)])
def test_gemv_sorted_sg(lib, ctxs, codes, code, bits):
    o, ctx = codes[code], ctxs[code]
    n_out, k_in = 333, 2000
    stream, nblocks = gen.make_layer_sg(o.N, o.W, bits, n_out, k_in, seed=31)
    cb = _codebook(bits)
    rs = gen.row_scales_f32(n_out, seed=9)
    x = gen.normal_bf16(k_in, seed=6)
    ref = o.gemm_sg(stream, bits, cb, rs, n_out, k_in, x, threads=4)
    d_cb, d_rs, d_x = _f32(cb), _f32(rs), to_dev_bf16(x)
    srt = lib.llvq_sort_blocks_sg(ctx, to_dev_u8(stream), bits, n_out, k_in)
    y = lib.llvq_gemv_sorted_sg(ctx, srt, bits, d_cb, d_rs, n_out, k_in, d_x)
    yb = lib.llvq_gemv_sorted_sg(ctx, srt, bits, d_cb, None, n_out, k_in, d_x, y_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert gemv_error(y.cpu().numpy(), ref) <= TOL
    ref_noscale = o.gemm_sg(stream, bits, cb, None, n_out, k_in, x, threads=4)
    assert gemv_error(yb.float().cpu().numpy(), ref_noscale) <= TOL_BF16_OUT
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_gemv_sorted_sg_full_size_and_limits(lib, ctxs, codes):
    code, bits = (2, 12), 1
    o, ctx = codes[code], ctxs[code]
    n_out, k_in = 4096, 4096
    stream, nblocks = gen.make_layer_sg(o.N, o.W, bits, n_out, k_in, seed=2)
    cb = _codebook(bits)
    rs = gen.row_scales_f32(n_out, seed=2)
    x = gen.normal_bf16(k_in, seed=2)
    d_s = to_dev_u8(stream)
    srt = lib.llvq_sort_blocks_sg(ctx, d_s, bits, n_out, k_in)
    y = lib.llvq_gemv_sorted_sg(ctx, srt, bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x)).cpu().numpy()
    y2 = lib.llvq_gemv_sg(ctx, d_s, bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x)).cpu().numpy()
    # two binary32 sums of the same 4096 products in different (and, through the shared-memory atomics, run-dependent)
    # orders; relative to the floor of 1e-3 of the largest output a small row's sum can move by about 1e-4
    assert gemv_error(y, y2.astype(np.float64)) <= 5e-4
    import os
    ref = o.gemm_sg(stream, bits, cb, rs, n_out, k_in, x, threads=os.cpu_count() or 1)     # every output row, both kernels
    assert gemv_error(y, ref) <= TOL
    assert gemv_error(y2, ref) <= TOL
    # 47 + 2 bits do not fit the 48-bit entry
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    assert ctx._lib.llvq_sort_blocks_sg(ctx._h, buf.data_ptr(), 2, 8, 24, buf.data_ptr(), None) == 3
    assert ctx._lib.llvq_gemv_sorted_sg(ctx._h, buf.data_ptr(), 2, buf.data_ptr(), None, 8, 24, buf.data_ptr(), buf.data_ptr(), 0, None) == 3
    assert lib.llvq_last_error(ctx) == (0, 0)


@pytest.mark.parametrize("code,bits,n_out,k_in,batch", [((2, 12), 1, 200, 480, 5), ((2, 10), 4, 129, 1000, 16), ((2, 13), 0, 300, 2000, 40),
                                                        ((3, 3), 0, 64, 4104, 64)])
def test_gemm_small_batch_sg(lib, ctxs, codes, code, bits, n_out, k_in, batch):
    o, ctx = codes[code], ctxs[code]
    stream, nblocks = gen.make_layer_sg(o.N, o.W, bits, n_out, k_in, seed=41)
    cb = _codebook(bits)
    rs = gen.row_scales_f32(n_out, seed=10)
    x = gen.normal_bf16((batch, k_in), seed=7)
    ref = o.gemm_sg(stream, bits, cb, rs, n_out, k_in, x, threads=4)
    y = lib.llvq_gemm_small_batch_sg(ctx, to_dev_u8(stream), bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    assert gemv_error(y.float().cpu().numpy(), ref) <= TOL_BF16_OUT
    # the same product from the sorted layout
    srt = lib.llvq_sort_blocks_gemm_sg(ctx, to_dev_u8(stream), bits, n_out, k_in)
    ys = lib.llvq_gemm_small_batch_sorted_sg(ctx, srt, bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x))
    torch.cuda.synchronize()
    assert gemv_error(ys.float().cpu().numpy(), ref) <= TOL_BF16_OUT
    # batch 1 agrees with the fused matrix-vector product
    y1 = lib.llvq_gemm_small_batch_sg(ctx, to_dev_u8(stream), bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x[:1]))
    yv = lib.llvq_gemv_sg(ctx, to_dev_u8(stream), bits, _f32(cb), _f32(rs), n_out, k_in, to_dev_bf16(x[0]), y_dtype=torch.bfloat16)
    assert gemv_error(y1[0].float().cpu().numpy(), yv.float().cpu().numpy().astype(np.float64)) <= 2.0 ** -7
    assert lib.llvq_last_error(ctx) == (0, 0)
