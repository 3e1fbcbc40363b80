"""Pins of the clustering oracle (Section 2.2: pair-probe matrix -> SM resource groups):
planted partitions with noise, a null matrix, the A100-shaped case, label canonicity, and an
exact-rational brute force of the agglomeration on small matrices."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import rr_inputs


@pytest.mark.parametrize("drop", [0.06, 0.10, 0.15, 0.25])
def test_planted_partitions_recovered_exactly(drop):
    for s in range(100):
        sizes = rr_inputs.random_group_sizes(1000 + s)       # 8-16 groups of 8-20 SMs
        T, truth = rr_inputs.planted_matrix(sizes, drop, seed=s)  # sigma 2 %, TPC drop, background
        g, G, conf, _ = oracle.cluster(T)
        assert G == len(sizes), (drop, s)
        assert np.array_equal(g, truth), (drop, s)
        assert conf >= 4.0


def test_null_matrix_gives_one_group():
    for s in range(50):
        sizes = rr_inputs.random_group_sizes(2000 + s)
        T, _ = rr_inputs.planted_matrix(sizes, 0.0, seed=s)
        g, G, conf, _ = oracle.cluster(T)
        assert G == 1 and not g.any() and conf < 4.0


def test_a100_shaped_case():
    # 14 groups of 6 or 8 SMs (108 SMs), as the paper reports for its card
    sizes = [8] * 12 + [6] * 2
    for s in range(20):
        T, truth = rr_inputs.planted_matrix(sizes, 0.10, seed=s)
        g, G, _, _ = oracle.cluster(T)
        assert G == 14 and np.array_equal(g, truth)
        assert sorted(np.bincount(g).tolist()) == [6, 6] + [8] * 12


def test_asymmetric_input_is_symmetrised_and_labels_are_canonical():
    T, truth = rr_inputs.planted_matrix([8, 10, 12, 8, 16, 10], 0.2, seed=5)
    g1, G1, _, _ = oracle.cluster(T)
    g2, G2, _, _ = oracle.cluster(T.T.copy())
    assert G1 == G2 == 6 and np.array_equal(g1, g2) and np.array_equal(g1, truth)
    # canonical: first occurrences of labels appear in increasing order
    firsts = [int(np.argmax(g1 == k)) for k in range(G1)]
    assert firsts == sorted(firsts) and g1[0] == 0
    # diagonal (solo runs) is ignored
    T2 = T.copy()
    np.fill_diagonal(T2, 1e9)
    assert np.array_equal(oracle.cluster(T2)[0], g1)


def test_rejects_bad_matrices():
    T, _ = rr_inputs.planted_matrix([8, 8, 8], 0.2, seed=1)
    for bad in (np.nan, 0.0, -1.0, np.inf):
        B = T.copy()
        B[3, 7] = bad
        with pytest.raises(oracle.OracleError):
            oracle.cluster(B)
    with pytest.raises(oracle.OracleError):
        oracle.cluster(np.ones((1, 1), np.float32))


def _upgma_rational(T):
    """Average linkage written with exact fractions over the raw definition (mean of all member
    pair distances recomputed from scratch at every step)."""
    n = T.shape[0]
    t = (T.astype(np.float64) + T.astype(np.float64).T) * 0.5
    off = sorted(t[i, j] for i in range(n) for j in range(i + 1, n))
    med = off[(len(off) - 1) // 2]
    q = [[int(np.rint(t[i, j] * 1048576.0 / med)) if i != j else 0 for j in range(n)]
         for i in range(n)]
    clusters = {i: [i] for i in range(n)}
    heights, merges = [], []
    while len(clusters) > 1:
        best = None
        for a in sorted(clusters):
            for b in sorted(clusters):
                if b <= a:
                    continue
                mean = Fraction(sum(q[i][j] for i in clusters[a] for j in clusters[b]),
                                len(clusters[a]) * len(clusters[b]))
                if best is None or mean < best[0]:
                    best = (mean, a, b)
        mean, a, b = best
        heights.append(float(mean))
        merges.append((a, b))
        clusters[a] = clusters[a] + clusters.pop(b)
    return heights, merges


@pytest.mark.parametrize("seed", range(6))
def test_agglomeration_matches_exact_rational_brute_force(seed):
    sizes = [4, 6, 4, 2, 6][: 3 + seed % 3]
    T, truth = rr_inputs.planted_matrix(sizes, 0.15, seed=seed)
    g, G, conf, heights = oracle.cluster(T)
    ref_h, merges = _upgma_rational(T)
    assert np.allclose(heights, ref_h, rtol=0, atol=0)      # same divisions, same doubles
    assert all(a <= b for a, b in zip(ref_h, ref_h[1:]))     # average linkage is monotone
    # replay the brute-force merges down to G clusters and compare partitions
    n = T.shape[0]
    rep = list(range(n))
    for a, b in merges[: n - G]:
        rep = [a if r == b else r for r in rep]
    for i in range(n):
        for j in range(n):
            assert (rep[i] == rep[j]) == (g[i] == g[j])


def test_ties_break_towards_smallest_pair():
    # all entries equal: every step merges the lexicographically smallest alive pair -> (0,1),
    # (0,2), ...; no gap anywhere -> one group
    T = np.full((9, 9), 50.0, np.float32)
    g, G, conf, heights = oracle.cluster(T)
    assert G == 1 and conf == 0.0 and np.all(heights == 1048576.0)


def test_solo_normalisation_removes_per_sm_speed_differences():
    # SMs whose solo rates differ by +-15 % blur a 10 % contention drop in the raw matrix; dividing
    # each pair by its two solo rates (the diagonal) restores exact recovery
    raw_ok = norm_ok = 0
    for s in range(40):
        sizes = rr_inputs.random_group_sizes(3000 + s)
        T, truth = rr_inputs.planted_matrix(sizes, 0.10, seed=s, solo_spread=0.15)
        g, G, _, _ = oracle.cluster(T)
        raw_ok += G == len(sizes) and np.array_equal(g, truth)
        g, G, conf, _ = oracle.cluster(T, solo_normalise=True)
        norm_ok += G == len(sizes) and np.array_equal(g, truth)
    assert norm_ok == 40 and raw_ok < 40


def test_solo_normalisation_is_scale_free_and_checks_the_diagonal():
    T, truth = rr_inputs.planted_matrix([6, 8, 6, 8, 6], 0.3, seed=2, solo_spread=0.1)
    g1, G1, c1, h1 = oracle.cluster(T, solo_normalise=True)
    g2, G2, c2, h2 = oracle.cluster(T * 4.0, solo_normalise=True)   # power-of-two scale: exact
    assert G1 == G2 == 5 and np.array_equal(g1, g2) and np.array_equal(h1, h2)
    assert np.array_equal(g1, truth)
    B = T.copy()
    B[3, 3] = 0.0
    with pytest.raises(oracle.OracleError):
        oracle.cluster(B, solo_normalise=True)
    oracle.cluster(B)      # without the flag the diagonal is ignored


def test_faint_background_pattern_is_not_a_grouping():
    # an almost flat matrix (0.02 % structure, as measured inside the reach on B200) must give one
    # group however small its noise is: the paper ignores the faint pattern behind the boxes
    rng = np.random.default_rng(0)
    n = 148
    T = np.full((n, n), 150.0) * (1 + 2e-5 * rng.standard_normal((n, n)))
    T[:4, :] *= 0.9998
    T[:, :4] *= 0.9998
    np.fill_diagonal(T, 75.0)
    g, G, conf, _ = oracle.cluster(T.astype(np.float32), solo_normalise=True)
    assert G == 1 and not g.any()
    # a 3 % same-group drop with equally small noise is a grouping
    T2, truth = rr_inputs.planted_matrix([6] * 12 + [8] * 4, 0.03, seed=1, tpc_drop=0.0,
                                         background=0.0, sigma=2e-5)
    g, G, conf, _ = oracle.cluster(T2, solo_normalise=True)
    assert G == 16 and np.array_equal(g, truth)
