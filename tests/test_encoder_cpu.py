"""Pins of the oracle's encoder (nearest-point search + indexing): exactness of the lattice search against
brute force and textbook constants, and the distortions the paper prints for a Gaussian source."""
import math

import numpy as np
import pytest

import llvq_inputs as gen


@pytest.fixture(scope="module")
def shell2(oracle_mod):
    o = oracle_mod.Code(2, 2)
    lo = np.arange(o.N, dtype=np.uint64)
    return o.unrank_arrays(lo, np.zeros_like(lo)).astype(np.float64)


@pytest.fixture(scope="module")
def code13(oracle_mod):
    return oracle_mod.Code(2, 13)


def _brute_small(v, shell2):
    """Nearest lattice point of a vector of norm <= 3.4: only the origin and the 196560 minimal vectors can win
    (every other lattice point has norm >= sqrt(48) > 2 * 3.4)."""
    d2 = ((shell2 - v[None, :]) ** 2).sum(axis=1)
    k = int(np.argmin(d2))
    return (shell2[k], d2[k]) if d2[k] < (v * v).sum() else (np.zeros(24), float((v * v).sum()))


def test_lattice_search_is_exact_near_the_origin_and_after_translation(oracle_mod, shell2, code13):
    rng = np.random.default_rng(7)
    v = rng.standard_normal((40, 24))
    v[20:] = 0.15 * v[20:] + shell2[rng.integers(0, len(shell2), size=20)]     # half of them lean towards a minimal vector
    v *= (rng.uniform(2.0, 3.4, size=40) / np.linalg.norm(v, axis=1))[:, None]
    pts, d2 = oracle_mod.nearest_lattice_point(v)
    n_origin = 0
    for i in range(len(v)):
        want, wd = _brute_small(v[i], shell2)
        assert d2[i] == pytest.approx(wd, rel=1e-12)
        assert np.array_equal(pts[i], want.astype(np.int32)) or abs(wd - ((v[i] - pts[i]) ** 2).sum()) < 1e-12
        n_origin += not want.any()
    assert 0 < n_origin < len(v)                          # both outcomes occur
    # the lattice is a group: shifting the input by a lattice vector shifts the answer
    lam = code13.unrank([code13.N - 1 - 977 * i for i in range(len(v))]).astype(np.float64)
    pts2, d22 = oracle_mod.nearest_lattice_point(v + lam)
    assert np.allclose(d22, d2, rtol=1e-9)
    assert np.array_equal(pts2 - lam.astype(np.int32), pts)


def test_lattice_points_are_fixed_points(oracle_mod, code13):
    idx = [0, 1103, 1104, 196559, 196560, 16969680, code13.N - 1] + [code13.N // 7 * k + 5 for k in range(1, 7)]
    x = code13.unrank(idx)
    pts, d2 = oracle_mod.nearest_lattice_point(x.astype(np.float64))
    assert np.array_equal(pts, x.astype(np.int32)) and not d2.any()
    p2, i2 = code13.encode(x.astype(np.float64), oracle_mod.EUCLIDEAN)
    assert np.array_equal(p2, x) and i2 == idx
    p3, i3 = code13.encode(0.37 * x.astype(np.float64), oracle_mod.ANGULAR)        # direction only
    assert np.array_equal(p3, x) and i3 == idx


def test_second_moment_and_covering_radius_of_the_lattice(oracle_mod):
    # uniform inputs over a large box: mean squared error per dimension = G(Leech) * V^(2/24) with the normalized
    # second moment G = 0.065771 (Conway & Sloane) and V = 8^12 in integer coordinates; no input is farther than
    # the covering radius sqrt(2) * sqrt(8) = 4 from the lattice
    rng = np.random.default_rng(3)
    v = rng.uniform(-40.0, 40.0, size=(3000, 24))
    pts, d2 = oracle_mod.nearest_lattice_point(v)
    assert d2.max() <= 16.0 + 1e-9
    assert d2.mean() / 24 == pytest.approx(0.065771 * 8.0, rel=0.012)
    for p in pts[:200]:
        assert oracle_mod.is_member(p.astype(np.int8)) >= 0


def test_encoder_outputs_are_points_of_the_code(oracle_mod, code13):
    rng = np.random.default_rng(11)
    w = rng.standard_normal((150, 24))
    w[0] = 0.0                                                # zero input -> index 0
    w[1] *= 10.0                                              # far outside the ball: the best of the shell-radius decodes
    w[2] *= 0.01                                              # nearest lattice point is the origin: the same, it ends on a small shell
    for metric in (oracle_mod.EUCLIDEAN, oracle_mod.ANGULAR):
        pts, idx = code13.encode(2.5 * w, metric)
        assert idx[0] == 0
        assert all(0 <= i < code13.N for i in idx)
        assert np.array_equal(code13.unrank(idx), pts)
        m = (pts.astype(np.int64) ** 2).sum(axis=1) // 16
        assert m.min() >= 2 and m.max() <= 13
    pts, _ = code13.encode(2.5 * w, oracle_mod.EUCLIDEAN)
    assert ((pts[1].astype(np.int64) ** 2).sum()) // 16 >= 10  # the far vector lands on the outer shells
    assert ((pts[2].astype(np.int64) ** 2).sum()) // 16 <= 5
    with pytest.raises(ValueError):
        oracle_mod.Code(3, 3).encode(w[:2], oracle_mod.ANGULAR)


def test_gaussian_source_distortion_matches_the_paper(oracle_mod, code13):
    # Table "spherical shaping vs shape-gain" at 2 bits/dim, unit-variance Gaussian source:
    #   ball cut of the lattice up to shell 13, Euclidean search:   MSE 0.084
    #   normalized points up to shell 13 + 0 gain bits:             MSE 0.085
    #   normalized points up to shell 12 + 1 chi-matched gain bit:  MSE 0.078
    from oracle.gain_codebook import chi_codebook
    rng = np.random.default_rng(2024)
    w = rng.standard_normal((1600, 24))
    alpha = 2.5                                               # lattice scale: ball radius / alpha = 5.77 keeps ~89 % of the source inside
    pts, idx = code13.encode(alpha * w, oracle_mod.EUCLIDEAN, threads=4)
    mse = ((w - pts / alpha) ** 2).mean()
    assert mse == pytest.approx(0.084, abs=0.004)
    inside = (np.linalg.norm(w, axis=1) * alpha <= math.sqrt(16 * 13)).mean()
    assert inside == pytest.approx(0.8937, abs=0.03)          # the "Ret" column

    def shape_gain_mse(code, bits, n):
        p, _ = code.encode(w[:n], oracle_mod.ANGULAR, threads=4)
        s = p / np.linalg.norm(p.astype(np.float64), axis=1, keepdims=True)
        r = np.linalg.norm(w[:n], axis=1)
        cb = chi_codebook(bits)
        g = cb[np.argmin(np.abs(r[:, None] - cb[None, :]), axis=1)]
        rec = g[:, None] * s
        beta = (w[:n] * rec).sum() / (rec * rec).sum()         # one global scale (the closed-form optimal scale)
        return ((w[:n] - beta * rec) ** 2).mean()

    assert shape_gain_mse(code13, 0, 700) == pytest.approx(0.085, abs=0.004)
    assert shape_gain_mse(oracle_mod.Code(2, 12), 1, 700) == pytest.approx(0.078, abs=0.004)


def test_euclidean_search_on_the_cut_against_brute_force(oracle_mod):
    # the cut of the lattice at shell 3 has 16 969 680 points: small enough to try them all.  Inputs whose nearest lattice
    # point lies in the cut must get exactly the brute-force answer (the search is exact there); inputs outside the ball
    # or next to the origin get a point of the cut that is at least as near as the decode of their projection onto the
    # outermost shell, and the brute-force optimum is never farther than what the search returns.
    import os
    from concurrent.futures import ThreadPoolExecutor
    o = oracle_mod.Code(2, 3)
    lo = np.arange(o.N, dtype=np.uint64)
    parts = np.array_split(lo, 4 * (os.cpu_count() or 1))
    with ThreadPoolExecutor(os.cpu_count() or 1) as ex:          # the C decoder runs outside the interpreter lock
        allpts = np.concatenate(list(ex.map(lambda p: o.unrank_arrays(p, np.zeros_like(p)), parts)))
    rng = np.random.default_rng(12)
    v = rng.standard_normal((14, 24))
    v *= (np.array([1.5, 4.0, 5.0, 5.5, 6.0, 6.3, 6.6, 6.9, 7.2, 7.6, 8.5, 10.0, 14.0, 30.0]) / np.linalg.norm(v, axis=1))[:, None]
    v = v.astype(np.float32).astype(np.float64)                  # the encoder's inputs are binary32 values
    pts, idx = o.encode(v, oracle_mod.EUCLIDEAN)
    unconstrained, _ = oracle_mod.nearest_lattice_point(v)
    # brute force: 2 <v, x> - |x|^2 for all points at once in binary32 (one matrix product per chunk), then the few
    # points within rounding distance of each chunk's maximum again in binary64
    cands = [[] for _ in v]
    v32 = v.astype(np.float32)
    for c in range(0, len(allpts), 1 << 19):
        blk = allpts[c:c + (1 << 19)].astype(np.float32)
        score = 2.0 * (blk @ v32.T) - (blk * blk).sum(axis=1, keepdims=True)
        for i in range(len(v)):
            near = np.nonzero(score[:, i] >= score[:, i].max() - 0.05)[0]
            cands[i] += [c + int(j) for j in near]
    exact_cases = 0
    for i in range(len(v)):
        d2c = ((allpts[cands[i]].astype(np.float64) - v[i][None, :]) ** 2).sum(axis=1)
        best, best_at = float(d2c.min()), cands[i][int(np.argmin(d2c))]
        got = float(((pts[i] - v[i]) ** 2).sum())
        m = int((unconstrained[i].astype(np.int64) ** 2).sum()) // 16
        assert int(idx[i]) < o.N and np.array_equal(allpts[int(idx[i])], pts[i])
        assert got >= best - 1e-9
        if 2 <= m <= 3:                                          # the unconstrained answer is in the cut: exact
            assert got == pytest.approx(best, rel=1e-12)
            assert np.array_equal(pts[i], unconstrained[i].astype(np.int8)) and (best_at == int(idx[i]) or sum(d == best for d in d2c) > 1)
            exact_cases += 1
        else:
            proj, _ = oracle_mod.nearest_lattice_point((v[i] * (math.sqrt(48.0) / np.linalg.norm(v[i])))[None, :])
            if 2 <= int((proj[0].astype(np.int64) ** 2).sum()) // 16 <= 3:
                assert got <= float(((proj[0] - v[i]) ** 2).sum()) + 1e-9
            assert got <= best * 1.6 + 1e-9                      # the candidate search stays near the optimum (it is not exact)
    assert 3 <= exact_cases <= 11                                # both regimes occur
