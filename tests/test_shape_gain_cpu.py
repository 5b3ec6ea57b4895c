"""Pins of the oracle's shape-gain reconstruction (gain codebook entry * x / |x|, optional row scale) and of
the chi-matched gain codebook, against facts that do not come from the oracle itself."""
import math

import numpy as np
import pytest

import llvq_inputs as gen


def _bf16(a):
    return gen.bf16_bits_to_f32(a).astype(np.float64)


@pytest.fixture(scope="module")
def code13(oracle_mod):
    return oracle_mod.Code(2, 13)


# ---- gain codebook ----------------------------------------------------------------------------------------------

def _chi_pdf(r, n=24):
    # density of the norm of n independent N(0,1): r^(n-1) exp(-r^2/2) / (2^(n/2-1) Gamma(n/2))
    return np.exp((n - 1) * np.log(r) - r * r / 2 - (n / 2 - 1) * math.log(2.0) - math.lgamma(n / 2))


def test_zero_bit_codebook_is_the_mean_of_chi24():
    from oracle.gain_codebook import chi_codebook
    want = math.sqrt(2.0) * math.gamma(12.5) / math.gamma(12.0)          # E chi_24
    assert chi_codebook(0)[0] == pytest.approx(want, rel=1e-12)


@pytest.mark.parametrize("bits", [1, 2, 4])
def test_codebook_levels_are_centroids_of_nearest_level_cells(bits):
    from oracle.gain_codebook import chi_codebook
    y = chi_codebook(bits)
    assert np.all(np.diff(y) > 0) and y.size == 1 << bits
    r = np.linspace(1e-6, 14.0, 1400001)
    f = _chi_pdf(r)
    assert np.trapezoid(f, r) == pytest.approx(1.0, abs=1e-9)
    edges = np.concatenate(([0.0], 0.5 * (y[1:] + y[:-1]), [np.inf]))
    for i in range(y.size):
        cell = (r >= edges[i]) & (r < edges[i + 1])
        centroid = np.trapezoid(r[cell] * f[cell], r[cell]) / np.trapezoid(f[cell], r[cell])
        assert y[i] == pytest.approx(centroid, rel=2e-5)


def test_codebook_distortion_follows_the_high_resolution_slope():
    from oracle.gain_codebook import chi_codebook, chi_distortion
    d = [chi_distortion(chi_codebook(b)) for b in range(0, 6)]
    var = 24.0 - (math.sqrt(2.0) * math.gamma(12.5) / math.gamma(12.0)) ** 2
    assert d[0] == pytest.approx(var, rel=1e-9)                          # one level at the mean: the variance
    for b in range(1, 6):
        assert 2.5 < d[b - 1] / d[b] < 4.2                               # -> 4 per bit (6.02 dB) at high resolution
    assert d[5] / d[4] < d[2] / d[1] * 1.5 and 3.3 < d[4] / d[5] < 4.05
    # chi_24 is close to N(sqrt(23.5), 1/2): Lloyd-Max of a Gaussian at 1 bit leaves (1 - 2/pi) of the variance
    assert d[1] / d[0] == pytest.approx(1.0 - 2.0 / math.pi, abs=0.01)


# ---- reconstruction ---------------------------------------------------------------------------------------------

def _fields(code, nblocks, gain_bits, seed, ks=None):
    lo, hi = gen.random_indices(code.N, code.W, nblocks, seed)
    k = gen.gain_indices(nblocks, gain_bits, seed) if ks is None else np.asarray(ks, dtype=np.uint64)
    f = lo | (k << np.uint64(code.W))
    return gen.pack_indices(f, hi, code.W + gain_bits), lo, k


def test_zero_bit_reconstruction_is_the_unit_vector_of_the_point(code13):
    rows, cols = 16, 24 * 40
    stream, lo, _ = _fields(code13, rows * 40, 0, seed=3)
    w = _bf16(code13.dequant_matrix_sg(stream, 0, [1.0], None, rows, cols)).reshape(-1, 24)
    x = code13.unrank_arrays(lo, np.zeros_like(lo)).astype(np.float64)
    shells = (x * x).sum(axis=1) / 16
    assert set(shells.astype(int)) >= {9, 10, 11, 12, 13}                # several radii present
    unit = x / np.sqrt((x * x).sum(axis=1, keepdims=True))
    assert np.max(np.abs(w - unit)) <= 2.0 ** -9 * 1.01 + 2.0 ** -24     # one bf16 rounding of a number < 1 (+ the binary32 steps)
    assert np.max(np.abs((w * w).sum(axis=1) - 1.0)) < 5e-3


def test_gain_index_and_row_scale_set_the_norm(code13):
    rows, bpr, bits = 8, 12, 2
    ks = (np.arange(rows * bpr) * 7 + 1) % 4
    stream, lo, k = _fields(code13, rows * bpr, bits, seed=5, ks=ks)
    cb = np.array([3.5, 4.25, 5.0, 6.5], dtype=np.float32)
    rs = (0.01 * (1 + np.arange(rows))).astype(np.float32)
    w = _bf16(code13.dequant_matrix_sg(stream, bits, cb, rs, rows, bpr * 24)).reshape(rows, bpr, 24)
    norms = np.sqrt((w * w).sum(axis=2))
    want = rs.astype(np.float64)[:, None] * cb.astype(np.float64)[k.astype(int)].reshape(rows, bpr)
    assert np.max(np.abs(norms / want - 1.0)) < 4e-3


def test_shell_four_is_exact(code13):
    # |x|^2 = 64 on Shell(4): 1/|x| = 1/8 exactly, so a gain of 8 returns the integer point itself, exactly
    cls = code13.classes()
    first = min(c["offset"] for c in cls if c["m"] == 4)
    last = max(c["offset"] + c["card"] for c in cls if c["m"] == 4)
    rng = np.random.default_rng(1)
    idx = [first, last - 1] + [int(first + int(rng.integers(0, last - first))) for _ in range(190)]
    bits = 3
    ks = np.arange(len(idx)) % 8
    f = [i | (int(k) << code13.W) for i, k in zip(idx, ks)]
    lo, hi = gen.indices_to_arrays(f)
    stream = gen.pack_indices(lo, hi, code13.W + bits)
    cb = np.array([8.0, 16.0, 4.0, 8.0, 2.0, 8.0, 1.0, 32.0], dtype=np.float32)
    w = _bf16(code13.dequant_matrix_sg(stream, bits, cb, None, 1, len(idx) * 24)).reshape(-1, 24)
    x = code13.unrank(idx).astype(np.float64)
    assert np.array_equal(w, x * (cb[ks] / 8.0).astype(np.float64)[:, None])
    # ... and with a binary16-representable gain the result equals the stored-gain form of the same blocks
    g16 = np.array([0.0123, 1.5, -0.75, 3.0e-4], dtype=np.float16)
    ks2 = np.arange(len(idx)) % 4
    f2 = [i | (int(k) << code13.W) for i, k in zip(idx, ks2)]
    lo2, hi2 = gen.indices_to_arrays(f2)
    s_sg = gen.pack_indices(lo2, hi2, code13.W + 2)
    s_plain = gen.pack_indices(*gen.indices_to_arrays(idx), code13.W)
    a = code13.dequant_matrix_sg(s_sg, 2, (g16.astype(np.float32) * 8.0), None, 1, len(idx) * 24)
    b = code13.dequant_matrix(s_plain, g16[ks2].view(np.uint16), 1, len(idx) * 24, 1)
    assert np.array_equal(a, b)


def test_out_of_range_field_decodes_to_zero(code13):
    f = [code13.N, code13.N - 1, (1 << code13.W) - 1]
    lo, hi = gen.indices_to_arrays(f)
    w = _bf16(code13.dequant_matrix_sg(gen.pack_indices(lo, hi, code13.W), 0, [2.0], None, 1, 72)).reshape(3, 24)
    assert not w[0].any() and not w[2].any() and w[1].any()


def test_gemm_sg_is_the_product_with_the_reconstructed_matrix(code13):
    n_out, k_in, bits = 24, 500, 1
    stream, nblocks = gen.make_layer_sg(code13.N, code13.W, bits, n_out, k_in, seed=9)
    cb = np.array([4.3, 5.4], dtype=np.float32)
    rs = gen.row_scales_f32(n_out, seed=9)
    x = gen.normal_bf16((3, k_in), seed=2)
    w = _bf16(code13.dequant_matrix_sg(stream, bits, cb, rs, n_out, k_in))
    y = code13.gemm_sg(stream, bits, cb, rs, n_out, k_in, x)
    assert np.allclose(y, _bf16(x) @ w.T, rtol=1e-12, atol=1e-12)
    # integer special case: Shell(4) blocks, gain 8, all-ones input -> the coordinate sums of the points, exactly
    cls = code13.classes()
    first = min(c["offset"] for c in cls if c["m"] == 4)
    idx = [first + 12345 * i for i in range(4 * 21)]
    s4 = gen.pack_indices(*gen.indices_to_arrays(idx), code13.W)
    ones = gen.f32_to_bf16_bits(np.ones(500, dtype=np.float32))
    y4 = code13.gemm_sg(s4, 0, [8.0], None, 4, 500, ones)
    pts = code13.unrank(idx).reshape(4, 21 * 24)[:, :500]
    assert np.array_equal(y4, pts.sum(axis=1).astype(np.float64))
