"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible mistake in the oracle (wrong sign rule, wrong radix order, transposed
table, dropped term) fails at least one of them.
"""
import math
import os
import random

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


# --------------------------------------------------------------------------
# Golay code: Sec. 2.3 (size 4096, nonzero weights 8/12/16/24), Sec. 2.5 (A values)
# --------------------------------------------------------------------------
def test_golay_weight_distribution_and_linearity(oracle_mod):
    T = oracle_mod.golay_table()
    assert len(set(T.tolist())) == 4096
    weights = np.array([bin(int(c)).count("1") for c in T])
    hist = {w: int((weights == w).sum()) for w in set(weights.tolist())}
    assert hist == {0: 1, 8: 759, 12: 2576, 16: 759, 24: 1}
    # sorted by (weight, value)
    keys = list(zip(weights.tolist(), T.tolist()))
    assert keys == sorted(keys)
    assert int(T[-1]) == 0xFFFFFF
    # closed under XOR (linear code) and self-orthogonal (all overlaps even)
    member = np.zeros(1 << 24, dtype=bool)
    member[T] = True
    for c in T[:: 37].tolist() + T[-3:].tolist():
        assert member[T ^ np.uint32(c)].all()
        overlaps = np.array([bin(int(v)).count("1") for v in (T & np.uint32(c))])
        assert (overlaps % 2 == 0).all()
    # linear + these weights => minimum distance 8


# --------------------------------------------------------------------------
# Shell sizes: Table 1
# --------------------------------------------------------------------------
def test_shell_sizes_match_table_1(oracle_mod):
    cum = 0
    have = {}
    for m in range(2, 20):
        cum += oracle_mod.shell_size(m)
        have[m] = (oracle_mod.shell_size(m), cum)
    for m, n, N, bits in _rows("table1_shell_sizes.txt"):
        m = int(m)
        if n != "-":
            assert have[m][0] == int(n)
        assert have[m][1] == int(N)
        W = math.ceil(math.log2(int(N)))
        assert abs(W / 24 - float(bits)) < 5e-4
    assert oracle_mod.shell_size(2) == 196560      # kissing number, App. D


def test_code_sizes_and_index_widths(code_2_2, code_3_3, code_2_13, code_2_53, oracle_mod):
    assert (code_2_2.N, code_2_2.W) == (196560, 18)
    assert (code_3_3.N, code_3_3.W) == (16773120, 24)
    assert (code_2_13.N, code_2_13.W) == (280974212784720, 48)
    assert code_2_53.W == 72 and code_2_53.N < 2 ** 72
    assert code_2_53.N + oracle_mod.shell_size(54) > 2 ** 72    # 53 is the largest cut that fits 72 bits


# --------------------------------------------------------------------------
# Classes: Table 2 (rows, order, counts), Sec. 2.5 (A values), theta series
# --------------------------------------------------------------------------
def test_classes_match_table_2(oracle_mod):
    code = oracle_mod.Code(2, 4)
    got = code.classes()
    want = _rows("table2_classes.txt")
    assert len(got) == len(want) == 15
    off = 0
    for k, row in zip(got, want):
        m, parity, count = int(row[0]), row[1], int(row[2])
        mult = {v: int(c) for v, c in zip(range(8, -1, -1), row[3:]) if int(c)}
        assert k["m"] == m
        assert k["parity"] == (1 if parity == "odd" else 0)
        assert k["card"] == count
        assert dict(zip(k["values"], k["mults"])) == mult
        assert k["offset"] == off
        off += count
        assert k["A"] in ((4096,) if k["parity"] else (1, 759, 2576))
    assert off == code.N == 415003680


def test_class_cardinalities_sum_to_theta_series(code_2_53, oracle_mod):
    # two independent computations: enumeration of classes vs modular-form coefficients
    per_shell = {}
    count = {}
    for k in code_2_53.classes():
        per_shell[k["m"]] = per_shell.get(k["m"], 0) + k["card"]
        count[k["m"]] = count.get(k["m"], 0) + 1
        assert sum(v * v * c for v, c in zip(k["values"], k["mults"])) == 16 * k["m"]
        assert sum(k["mults"]) == 24
    for m in range(2, 54):
        assert per_shell[m] == oracle_mod.shell_size(m), m
    assert [count[m] for m in range(2, 14)] == [3, 4, 8, 9, 17, 17, 30, 33, 47, 54, 79, 82]
    assert code_2_53.num_classes == sum(count.values())


# --------------------------------------------------------------------------
# Index <-> point
# --------------------------------------------------------------------------
def _textbook_minimal_vectors(T):
    """The 196560 minimal vectors in the classical description: (+-4, +-4, 0^22) on any
    two positions; (+-2^8, 0^16) on octads with an even number of minus signs;
    (-+3, +-1^23): all ones, negated on a codeword, one coordinate multiplied by -3."""
    pts = set()
    for i in range(24):
        for j in range(i + 1, 24):
            for si in (4, -4):
                for sj in (4, -4):
                    v = [0] * 24
                    v[i], v[j] = si, sj
                    pts.add(tuple(v))
    for c in T.tolist():
        if bin(c).count("1") != 8:
            continue
        pos = [i for i in range(24) if (c >> i) & 1]
        for s in range(256):
            if bin(s).count("1") % 2:
                continue
            v = [0] * 24
            for t, i in enumerate(pos):
                v[i] = -2 if (s >> t) & 1 else 2
            pts.add(tuple(v))
    for c in T.tolist():
        base = [-1 if (c >> i) & 1 else 1 for i in range(24)]
        for i in range(24):
            v = list(base)
            v[i] = -3 * v[i]
            pts.add(tuple(v))
    return pts


def test_shell2_is_exactly_the_minimal_vectors(code_2_2, oracle_mod):
    pts = code_2_2.unrank(range(code_2_2.N))
    decoded = set(map(tuple, pts.tolist()))
    assert len(decoded) == 196560                          # injective
    assert decoded == _textbook_minimal_vectors(oracle_mod.golay_table())
    # first class = the 1104 vectors (4^2, 0^22), Sec. 2.3
    head = np.abs(pts[:1104]).astype(int)
    assert (np.sort(head, axis=1)[:, -2:] == 4).all() and (head.sum(axis=1) == 8).all()
    assert not (np.abs(pts[1104]).max() == 4)
    # (24, 196560, 1/2) spherical code: <x,y> <= 16 = 32/2 for distinct points (sampled rows, all columns)
    sample = pts[:: 997].astype(np.int32)
    gram = sample @ pts.astype(np.int32).T
    assert gram.max() == 32 and ((gram == 32).sum(axis=1) == 1).all()
    assert np.partition(gram, -2, axis=1)[:, -2].max() <= 16


def test_exhaustive_bijection_shell2_and_shell3(code_2_2, code_3_3):
    # member + norm + rank(unrank(I)) == I for every index; with |Shell(m)| = n(m) this is a bijection
    assert code_2_2.check_range(0, code_2_2.N, threads=8) == 0
    assert code_3_3.check_range(0, code_3_3.N, threads=8) == 0


def test_hand_derived_examples(code_2_13):
    # class 0 = (4^2, 0^22): A = 1, B = 2, P = C(24,2).  I = r + A*(s + 4*p).
    def pt(I):
        return code_2_13.unrank([I])[0].tolist()
    assert pt(0) == [4, 4] + [0] * 22                       # p = 0 -> slots {0,1}
    assert pt(1) == [-4, 4] + [0] * 22                      # s = 1 -> first nonzero F0 position negative
    assert pt(2) == [4, -4] + [0] * 22
    assert pt(4) == [4, 0, 4] + [0] * 21                    # p = 1 -> colex {0,2}
    assert pt(1103) == [0] * 22 + [-4, -4]                  # p = 275 -> {22,23}, s = 3
    # first odd point of Shell(2): class (3, 1^23), r = 0 -> zero codeword, p = 0 -> 3 at slot 0,
    # 3 = 3 mod 4 on F0 must be negated, 1 = 1 mod 4 stays
    assert pt(1104 + 97152) == [-3] + [1] * 23
    # last point of Shell(2): r = 4095 -> all-ones codeword, p = 23 -> 3 at slot 23
    assert pt(196559) == [-1] * 23 + [3]
    # first point of Shell(4) inside the union: (4^4, 0^20)
    assert pt(16969680) == [4, 4, 4, 4] + [0] * 20
    # last index of the code: shell 13, last odd class in descending order = (3^23, 1), all-ones word
    assert pt(code_2_13.N - 1) == [-1] + [3] * 23


def test_first_and_last_index_of_every_class_and_random(code_2_13, code_2_53):
    rnd = random.Random(5)
    for code, nrand in ((code_2_13, 200000), (code_2_53, 100000)):
        edge = []
        for k in code.classes():
            edge += [k["offset"], k["offset"] + k["card"] - 1]
        for I in edge:
            assert code.check_range(I, 1) == 0, I
        # random single indices (full width) and a few contiguous runs
        singles = [rnd.randrange(code.N) for _ in range(nrand)]
        pts = code.unrank(singles)
        assert code.rank(pts) == singles
        for _ in range(4):
            assert code.check_range(rnd.randrange(code.N - 20000), 20000, threads=1) == 0
        assert np.abs(pts).max() <= (13 if code.m_hi == 13 else 28)


def test_out_of_range_index_decodes_to_zero(code_2_13):
    pts = code_2_13.unrank([code_2_13.N, 2 ** 48 - 1])
    assert not pts.any()


def test_lattice_structure_of_decoded_points(code_2_13, oracle_mod):
    rnd = random.Random(11)
    idx = [rnd.randrange(code_2_13.N) for _ in range(4000)] + [rnd.randrange(415003680) for _ in range(2000)]
    pts = code_2_13.unrank(idx).astype(np.int64)
    gram = pts[:3000] @ pts[3000:].T
    assert (gram % 8 == 0).all()                           # even unimodular at scale 1/sqrt(8)
    assert ((pts * pts).sum(axis=1) % 16 == 0).all()       # |x|^2 = 16 m: even lattice at scale 1/sqrt(8)
    classes = code_2_13.classes()
    offsets = [k["offset"] for k in classes]
    import bisect
    for a, b in zip(pts[:300], pts[300:600]):
        for v in (a + b, a - b):
            if np.abs(v).max() <= 127:
                assert oracle_mod.is_member(v.astype(np.int8)) >= 0 or not v.any()
    neg = code_2_13.rank((-pts[:500]).astype(np.int8))
    for I, J in zip(idx[:500], neg):
        assert bisect.bisect_right(offsets, I) == bisect.bisect_right(offsets, J)


def test_membership_rejects_non_lattice_points(oracle_mod):
    assert oracle_mod.is_member([4, 4] + [0] * 22) == 0
    assert oracle_mod.is_member([-3] + [1] * 23) == 1
    assert oracle_mod.is_member([4] + [0] * 23) == -1           # sum = 4 mod 8
    assert oracle_mod.is_member([2, 2] + [0] * 22) == -1        # (1,1,0..) is not a codeword
    assert oracle_mod.is_member([3] + [1] * 23) == -1           # wrong residue pattern
    assert oracle_mod.is_member([2] + [1] * 23) == -1           # mixed parity


# --------------------------------------------------------------------------
# Stored format
# --------------------------------------------------------------------------
def test_unpack_hand_made_stream(code_2_2, code_2_13):
    # W = 18: fields 1, 2, 0x3FFFF, 5 -> bit stream written out by hand
    # bits 0..17 = 1; 18..35 = 2 (bit 19 set); 36..53 all ones; 54.. = 5 (bits 54, 56)
    bits = [0] * 128
    bits[0] = 1
    bits[19] = 1
    for t in range(36, 54):
        bits[t] = 1
    bits[54] = 1
    bits[56] = 1
    stream = np.packbits(np.array(bits, dtype=np.uint8), bitorder="little")
    assert code_2_2.unpack(stream, 4) == [1, 2, 0x3FFFF, 5]
    # W = 48: six little-endian bytes per field
    stream = np.zeros(16, dtype=np.uint8)
    stream[:6] = [0x01, 0x02, 0x03, 0x04, 0x05, 0x06]
    stream[6:12] = [0xFF, 0, 0, 0, 0, 0x80]
    assert code_2_13.unpack(stream, 2) == [0x060504030201, 0x8000000000FF]


def test_pack_is_inverse_of_oracle_unpack(code_2_2, code_2_13, code_2_53):
    import llvq_inputs as gen
    for code in (code_2_2, code_2_13, code_2_53):
        lo, hi = gen.random_indices(code.N, code.W, 1001, seed=3)
        stream = gen.pack_indices(lo, hi, code.W)
        assert stream.size % 16 == 0 and stream.size == gen.index_stream_bytes(1001, code.W)
        got = code.unpack(stream, 1001)
        assert got == [(int(h) << 64) | int(l) for l, h in zip(lo, hi)]
        assert max(got) < code.N


# --------------------------------------------------------------------------
# Dequantization and fused products
# --------------------------------------------------------------------------
def test_dequant_scalar_against_library_conversion(oracle_mod):
    import torch
    gains = torch.arange(0, 1 << 16, dtype=torch.int32).to(torch.int16).view(torch.float16)
    finite = torch.isfinite(gains)
    for x in range(-28, 29):
        want = (gains.to(torch.float64) * x).to(torch.bfloat16).view(torch.int16).to(torch.int32) & 0xFFFF
        got = torch.tensor([oracle_mod.dequant_scalar(g, x) for g in range(0, 1 << 16, 1 if x in (-28, -1, 0, 1, 3, 13, 28) else 97)],
                           dtype=torch.int32)
        step = 1 if x in (-28, -1, 0, 1, 3, 13, 28) else 97
        sel = finite[::step]
        assert torch.equal(got[sel], want[::step][sel]), x
    # signed zeros follow IEEE multiplication
    assert oracle_mod.dequant_scalar(0x3C00, 0) == 0x0000
    assert oracle_mod.dequant_scalar(0xBC00, 0) == 0x8000
    assert oracle_mod.dequant_scalar(0x0000, -4) == 0x8000
    assert oracle_mod.dequant_scalar(0x3C00, -3) == 0xC040


def _layer(code, rows, cols, layout, seed):
    import llvq_inputs as gen
    return gen.make_layer(code.N, code.W, rows, cols, layout, seed)


def test_dequant_matrix_layouts(code_2_13):
    import llvq_inputs as gen
    rows, cols = 7, 100                                    # ROWWISE: 5 blocks per row, 20 pad lanes dropped
    stream, gain, nblocks = _layer(code_2_13, rows, cols, 1, seed=1)
    assert nblocks == 35
    pts, bad = code_2_13.decode_stream(stream, nblocks)
    assert bad == 0
    g = gain.view(np.float16).astype(np.float64)
    want = gen.f32_to_bf16_bits((pts.astype(np.float64) * g[:, None]).astype(np.float32))   # exact products
    got = code_2_13.dequant_matrix(stream, gain, rows, cols, 1)
    assert np.array_equal(got, want.reshape(rows, 120)[:, :100])
    # FLAT: 700 elements = 29 full blocks + 4 elements
    stream, gain, nblocks = _layer(code_2_13, rows, cols, 0, seed=2)
    assert nblocks == 30
    pts, _ = code_2_13.decode_stream(stream, nblocks)
    g = gain.view(np.float16).astype(np.float64)
    want = gen.f32_to_bf16_bits((pts.astype(np.float64) * g[:, None]).astype(np.float32)).reshape(-1)[:700]
    assert np.array_equal(code_2_13.dequant_matrix(stream, gain, rows, cols, 0).reshape(-1), want)


def test_gemv_exact_special_cases(code_2_13):
    import llvq_inputs as gen
    n_out, k_in = 9, 100
    stream, _, nblocks = _layer(code_2_13, n_out, k_in, 1, seed=4)
    ones = np.full(nblocks, 0x3C00, dtype=np.uint16)       # gain 1.0
    pts, _ = code_2_13.decode_stream(stream, nblocks)
    Wint = pts.reshape(n_out, -1)[:, :k_in].astype(np.int64)
    # x = e_k picks column k of the integer matrix exactly
    for k in (0, 23, 24, 99):
        x = np.zeros(k_in, dtype=np.float32)
        x[k] = 1
        y = code_2_13.gemv(stream, ones, n_out, k_in, gen.f32_to_bf16_bits(x))
        assert np.array_equal(y, Wint[:, k].astype(np.float64))
    # x = all ones gives integer row sums (pad lanes excluded)
    y = code_2_13.gemv(stream, ones, n_out, k_in, gen.f32_to_bf16_bits(np.ones(k_in, dtype=np.float32)))
    assert np.array_equal(y, Wint.sum(axis=1).astype(np.float64))


def test_gemm_against_numpy_matmul(code_2_13):
    import llvq_inputs as gen
    n_out, k_in, batch = 11, 200, 5
    stream, gain, _ = _layer(code_2_13, n_out, k_in, 1, seed=6)
    X = gen.normal_bf16((batch, k_in), seed=6)
    Wd = gen.bf16_bits_to_f32(code_2_13.dequant_matrix(stream, gain, n_out, k_in, 1)).astype(np.float64)
    want = gen.bf16_bits_to_f32(X).astype(np.float64) @ Wd.T
    got = code_2_13.gemm(stream, gain, n_out, k_in, X)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-15)
    got_t = code_2_13.gemm(stream, gain, n_out, k_in, X, threads=3)
    assert np.array_equal(got, got_t)
    part = code_2_13.gemm(stream, gain, n_out, k_in, X, rows=(3, 4))
    assert np.array_equal(part[:, 3:7], got[:, 3:7]) and not part[:, :3].any() and not part[:, 7:].any()


# --------------------------------------------------------------------------
# Angular nearest point (Sec. 3.1), brute force on the minimal shell
# --------------------------------------------------------------------------
def test_nearest_angular_on_shell2(code_2_2):
    pts = code_2_2.unrank(range(code_2_2.N)).astype(np.float64)
    rng = np.random.default_rng(0)
    for _ in range(3):
        v = rng.standard_normal(24)
        I = code_2_2.nearest_angular(v)
        scores = pts @ v                                    # one shell: constant norm
        assert I == int(np.argmax(scores))
        J = code_2_2.nearest_angular(-v)
        assert np.array_equal(pts[J], -pts[I])              # antipodal code
    for I in (0, 1104, 150000, 196559):
        assert code_2_2.nearest_angular(pts[I]) == I        # a code point is its own nearest point
