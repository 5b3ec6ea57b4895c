"""Parity of the encoder entry points (search, point -> index, field packing) against the CPU oracle, through the
C ABI, and the end-to-end distortion on a Gaussian source against the values the paper prints."""
import math

import numpy as np
import pytest
import torch

import llvq_inputs as gen
from gpu_util import bf16_bits, to_dev_u8

pytestmark = pytest.mark.gpu

CODES = [(2, 13), (2, 12), (2, 10)]


@pytest.fixture(scope="module")
def lib():
    import paper_2603_11021_b200 as P
    assert torch.cuda.is_available(), "these tests need a CUDA device; there is no CPU path"
    return P


@pytest.fixture(scope="module")
def ctxs(lib):
    return {code: lib.Context(*code, device=0) for code in CODES}


@pytest.fixture(scope="module")
def codes(oracle_mod):
    return {code: oracle_mod.Code(*code) for code in CODES}


def _idx_np(t):
    return t.cpu().numpy().view(np.uint64)


@pytest.mark.parametrize("code", CODES)
def test_rank_is_the_inverse_of_decode(lib, ctxs, codes, code):
    o, ctx = codes[code], ctxs[code]
    lo, hi = gen.random_indices(o.N, o.W, 20000, seed=31)
    edges = []
    for c in o.classes():
        edges += [c["offset"], c["offset"] + c["card"] - 1, c["offset"] + c["card"] // 2]
    lo = np.concatenate([lo, np.array(edges, dtype=np.uint64)])
    pts = o.unrank_arrays(lo, np.zeros_like(lo))
    got = _idx_np(lib.llvq_rank_blocks(ctx, torch.from_numpy(pts).cuda()))
    assert np.array_equal(got, lo)
    # and against the library's own decoder, on the device
    stream = gen.pack_indices(lo, np.zeros_like(lo), o.W)
    d_pts = lib.llvq_decode_blocks(ctx, to_dev_u8(stream), len(lo))
    assert np.array_equal(d_pts.cpu().numpy(), pts)
    assert np.array_equal(_idx_np(lib.llvq_rank_blocks(ctx, d_pts)), lo)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_rank_rejects_points_outside_the_code(lib, ctxs, codes, oracle_mod):
    o, ctx = codes[(2, 13)], ctxs[(2, 13)]
    good = o.unrank([5, 196560, 16969680, o.N - 1])
    bad = np.zeros((7, 24), dtype=np.int8)
    bad[0] = good[0]; bad[0, 0] += 1                      # mixed parities
    bad[1] = good[1]; bad[1, 3] += 2                      # even, but the bits are no codeword / wrong norm
    bad[2] = 2                                            # (2^24): lattice point of Shell(6)? no: sum = 48 = 0 mod 8, w = 24 -> it IS one
    bad[3] = good[3]; bad[3, 5] = -bad[3, 5]              # odd point with one sign flipped: leaves the lattice
    bad[4, 0] = 8                                         # (8, 0^23): Shell(4), in the code
    bad[5] = 4                                            # (4^24): norm 384 = 16 * 24, outside shells 2..13
    bad[6, 0] = 4                                         # (4, 0^23): norm 16, Shell(1) does not exist
    want_member = []
    for row in bad:
        norm = int((row.astype(np.int64) ** 2).sum())
        want_member.append(oracle_mod.is_member(row) >= 0 and norm % 16 == 0 and 2 <= norm // 16 <= 13)
    assert want_member == [False, False, True, False, True, False, False]
    got = _idx_np(lib.llvq_rank_blocks(ctx, torch.from_numpy(np.concatenate([good, bad])).cuda()))
    assert list(got[:4]) == [5, 196560, 16969680, o.N - 1]
    for j, member in enumerate(want_member):
        if member:
            assert o.rank([bad[j]]) == [int(got[4 + j])]
        else:
            assert got[4 + j] == 0
    assert lib.llvq_last_error(ctx) == (want_member.count(False), 0)


@pytest.mark.parametrize("W,bits", [(48, 0), (47, 1), (44, 4), (18, 0), (24, 3)])
def test_pack_fields_matches_the_stored_format(lib, oracle_mod, W, bits):
    code = {48: (2, 13), 47: (2, 12), 44: (2, 10), 18: (2, 2), 24: (3, 3)}[W]
    ctx = lib.Context(*code, device=0)
    assert ctx.index_bits == W
    n = 1237
    lo, hi = gen.random_indices(ctx.num_points, W, n, seed=77)
    k = gen.gain_indices(n, bits, seed=77)
    want = gen.pack_indices(lo | (k << np.uint64(W)), hi, W + bits)
    d_idx = torch.from_numpy(lo.view(np.int64)).cuda()
    d_k = torch.from_numpy(k.astype(np.uint8)).cuda()
    got = lib.llvq_pack_fields(ctx, d_idx, d_k, bits).cpu().numpy()
    assert np.array_equal(got, want)
    if bits == 0:
        assert got.size == ctx.index_bytes(n)


def _check_against_oracle(o, pts_gpu, idx_gpu, pts_ref, idx_ref):
    """The device search scores in binary64 in the oracle's operation order: points and indices must be identical."""
    assert np.array_equal(pts_gpu, pts_ref)
    assert np.array_equal(idx_gpu, np.array(idx_ref, dtype=np.uint64))
    assert np.array_equal(np.array(o.rank(pts_gpu), dtype=np.uint64), idx_gpu)       # valid points of the code, correctly indexed


@pytest.mark.parametrize("code", [(2, 13), (2, 10)])
def test_encode_euclidean(lib, ctxs, codes, oracle_mod, code):
    o, ctx = codes[code], ctxs[code]
    rng = np.random.default_rng(5)
    v = (rng.standard_normal((3000, 24)) * 2.5).astype(np.float32)
    v[0] = 0.0
    v[1] *= 40.0
    v[2] *= 0.004
    v[3:40] = o.unrank([o.N // 41 * j + 3 for j in range(1, 38)]).astype(np.float32)      # lattice points encode to themselves
    pts_ref, idx_ref = o.encode(v.astype(np.float64), oracle_mod.EUCLIDEAN, threads=4)
    d_pts, d_idx = lib.llvq_encode_blocks(ctx, torch.from_numpy(v).cuda(), lib.LLVQ_EUCLIDEAN)
    pts, idx = d_pts.cpu().numpy(), _idx_np(d_idx)
    assert idx[0] == 0 and np.array_equal(pts[3:40], pts_ref[3:40])
    _check_against_oracle(o, pts, idx, pts_ref, idx_ref)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_encode_angular(lib, ctxs, codes, oracle_mod):
    code = (2, 12)
    o, ctx = codes[code], ctxs[code]
    rng = np.random.default_rng(6)
    v = rng.standard_normal((700, 24)).astype(np.float32)
    v[0] = 0.0
    v[1] *= 1e4
    v[2] *= 1e-4
    pts_ref, idx_ref = o.encode(v.astype(np.float64), oracle_mod.ANGULAR, threads=4)
    d_pts, d_idx = lib.llvq_encode_blocks(ctx, torch.from_numpy(v).cuda(), lib.LLVQ_ANGULAR)
    _check_against_oracle(o, d_pts.cpu().numpy(), _idx_np(d_idx), pts_ref, idx_ref)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_encode_non_finite_input_is_flagged(lib, ctxs):
    ctx = ctxs[(2, 13)]
    v = torch.zeros((3, 24), dtype=torch.float32, device="cuda")
    v[1, 3] = float("nan")
    v[2, :] = 1.0
    d_pts, d_idx = lib.llvq_encode_blocks(ctx, v, lib.LLVQ_EUCLIDEAN)
    assert _idx_np(d_idx)[0] == 0 and _idx_np(d_idx)[1] == 0 and _idx_np(d_idx)[2] != 0
    assert lib.llvq_last_error(ctx) == (0, lib.LLVQ_FLAG_SEARCH_GAVE_UP)
    assert lib.llvq_last_error(ctx) == (0, 0)


def test_encode_unsupported_codes_and_arguments(lib):
    v = torch.zeros((2, 24), dtype=torch.float32, device="cuda")
    for code in [(2, 2), (3, 3), (2, 53)]:
        ctx = lib.Context(*code, device=0)
        with pytest.raises(lib.LlvqError) as e:
            lib.llvq_encode_blocks(ctx, v, lib.LLVQ_ANGULAR)
        assert e.value.status == 3
    ctx = lib.Context(2, 13, device=0)
    p = torch.zeros((2, 24), dtype=torch.int8, device="cuda")
    i = torch.zeros(2, dtype=torch.int64, device="cuda")
    L = ctx._lib
    assert L.llvq_encode_blocks(ctx._h, v.data_ptr(), 2, 2, p.data_ptr(), i.data_ptr(), None) == 1      # unknown metric
    assert L.llvq_encode_blocks(ctx._h, None, 2, 0, p.data_ptr(), i.data_ptr(), None) == 1
    assert L.llvq_encode_blocks(ctx._h, v.data_ptr(), 2, 0, p.data_ptr(), i.data_ptr() + 4, None) == 2
    assert L.llvq_encode_blocks(ctx._h, None, 0, 0, None, None, None) == 0
    assert L.llvq_pack_fields(ctx._h, i.data_ptr(), None, 3, 2, p.data_ptr(), None) == 1                # gain bits without gain indices


def test_gaussian_source_distortion_end_to_end(lib, ctxs):
    """Quantize and reconstruct a unit-variance Gaussian source entirely on the device.  The paper's table for
    2 bits/dim: ball cut up to shell 13 with Euclidean search 0.084; normalized points up to shell 12 with one
    chi-matched gain bit 0.078; normalized points up to shell 13 with no gain bits 0.085."""
    from oracle.gain_codebook import chi_codebook
    torch.manual_seed(1)
    n = 60000
    w = torch.randn((n, 24), device="cuda", dtype=torch.float32)
    # spherical shaping: scale, search, pack, dequantize with a constant gain 1/alpha
    ctx = ctxs[(2, 13)]
    alpha = 2.5
    d_pts, d_idx = lib.llvq_encode_blocks(ctx, w * alpha, lib.LLVQ_EUCLIDEAN)
    stream = lib.llvq_pack_fields(ctx, d_idx)
    gain = torch.full((n,), 1.0 / alpha, dtype=torch.float16, device="cuda")
    rec = lib.llvq_dequant_matrix(ctx, stream, gain, 1, n * 24, lib.LLVQ_LAYOUT_ROWWISE).float().view(n, 24)
    mse = float(((w - rec) ** 2).mean())
    assert mse == pytest.approx(0.084, abs=0.005)
    # shape-gain: angular search, nearest chi-matched gain level, one global scale folded into the codebook
    for code, bits, want in [((2, 12), 1, 0.078), ((2, 13), 0, 0.085)]:
        ctx = ctxs[code]
        m = 20000
        d_pts, d_idx = lib.llvq_encode_blocks(ctx, w[:m].contiguous(), lib.LLVQ_ANGULAR)
        cb = torch.tensor(chi_codebook(bits), dtype=torch.float32, device="cuda")
        r = w[:m].norm(dim=1)
        k = (r[:, None] - cb[None, :]).abs().argmin(dim=1).to(torch.uint8)
        s = d_pts.float() / d_pts.float().norm(dim=1, keepdim=True)
        rec0 = cb[k.long()][:, None] * s
        beta = float((w[:m] * rec0).sum() / (rec0 * rec0).sum())
        fields = lib.llvq_pack_fields(ctx, d_idx, k, bits)
        rec = lib.llvq_dequant_matrix_sg(ctx, fields, bits, (cb * beta).contiguous(), None, 1, m * 24).float().view(m, 24)
        assert float(((w[:m] - rec) ** 2).mean()) == pytest.approx(want, abs=0.005)
        assert float((rec - beta * rec0).abs().max()) < 0.02          # the dequantizer reconstructs what was encoded (bf16 rounding)
    for c in ctxs.values():
        assert lib.llvq_last_error(c) == (0, 0)


@pytest.mark.parametrize("code", [(2, 6), (2, 16), (2, 20), (2, 24)])
def test_other_ball_cuts_decode_and_rank(lib, oracle_mod, code):
    # cuts the benchmarks do not use: 36-, 52-, 56- and 59-bit indices; the last three keep their class tables in global memory
    ctx = lib.Context(*code, device=0)
    o = oracle_mod.Code(*code)
    assert (ctx.index_bits, ctx.num_points, ctx.num_classes) == (o.W, o.N, o.num_classes)
    n = 6000
    lo, hi = gen.random_indices(o.N, o.W, n, seed=5)
    cls = o.classes()
    edges = [c["offset"] for c in cls[::17]] + [c["offset"] + c["card"] - 1 for c in cls[::17]]
    lo = np.concatenate([lo, np.array(edges, dtype=np.uint64)])
    hi = np.zeros_like(lo)
    pts = lib.llvq_decode_blocks(ctx, to_dev_u8(gen.pack_indices(lo, hi, o.W)), len(lo))
    assert np.array_equal(pts.cpu().numpy(), o.unrank_arrays(lo, hi))
    assert np.array_equal(_idx_np(lib.llvq_rank_blocks(ctx, pts)), lo)
    v = torch.randn((500, 24), device="cuda") * 2.5
    p, i = lib.llvq_encode_blocks(ctx, v, lib.LLVQ_EUCLIDEAN)
    assert torch.equal(lib.llvq_decode_blocks(ctx, lib.llvq_pack_fields(ctx, i), 500), p)
    assert lib.llvq_last_error(ctx) == (0, 0)
