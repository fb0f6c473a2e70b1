"""Pins of the oracle's exact solver of the transport problem (Eq. 2-6): the linear program with the
dustbin marginals, whose optimum is a maximum-weight partial matching with pair gains S_ij - z.  None of
these retypes the solver: brute-force enumeration on tiny problems, a library assignment routine, the
small-eps limit of the oracle's own Sinkhorn iterations, and linear-programming duality (a feasible dual
of equal value proves optimality whatever produced the primal)."""
import itertools

import numpy as np
import pytest
from scipy.optimize import linear_sum_assignment


def _rng(seed):
    return np.random.default_rng(seed)


def _brute_force(S, z):
    """Best value of sum_ij S-bar P-bar over all partial matchings (every vertex of the LP)."""
    M, B = S.shape
    best, arg = -np.inf, None
    for m in range(0, min(M, B) + 1):
        for rows in itertools.combinations(range(M), m):
            for cols in itertools.permutations(range(B), m):
                val = sum(S[i, j] for i, j in zip(rows, cols)) + z * (M + B - m)
                if val > best + 1e-15:
                    best, arg = val, tuple(sorted(zip(rows, cols)))
    return best, arg


def _check_matching(match, M):
    used = [i for i in match if i >= 0]
    assert len(used) == len(set(used)) and all(0 <= i < M for i in used)


def test_brute_force_on_every_shape_up_to_eight_tokens(oracle):
    for seed in range(40):
        r = _rng(seed)
        N = int(r.integers(2, 9))
        M = int(r.integers(1, N))
        S = r.uniform(-1.0, 1.0, size=(M, N - M))
        z = float(r.choice([0.2, 0.0, -0.5, 0.7]))
        match, obj, _, _ = oracle.exact_matching(S, z=z)
        _check_matching(match, M)
        best, _ = _brute_force(S, z)
        assert obj == pytest.approx(best, abs=1e-12), (seed, S, match)
        # the reported objective is the value of the reported matching
        pairs = [(i, j) for j, i in enumerate(match) if i >= 0]
        assert obj == pytest.approx(sum(S[i, j] for i, j in pairs) + z * (N - len(pairs)), abs=1e-12)


def test_hand_cases(oracle):
    # one pair clearly worth it, one not: S - z = +0.5 and -0.1
    S = np.array([[0.7, 0.1]])
    match, obj, _, _ = oracle.exact_matching(S, z=0.2)
    assert match.tolist() == [0, -1] and obj == pytest.approx(0.7 + 0.2 * 2)
    # two kept tokens want the same pruned token: the better pair wins, the other stays unpaired
    S = np.array([[0.9], [0.8]])
    match, obj, _, _ = oracle.exact_matching(S, z=0.2)
    assert match.tolist() == [0] and obj == pytest.approx(0.9 + 0.2 * 2)
    # no score above z: nothing is paired and the value is z N
    S = np.full((3, 4), 0.1)
    match, obj, _, _ = oracle.exact_matching(S, z=0.2)
    assert match.tolist() == [-1] * 4 and obj == pytest.approx(0.2 * 7)
    # crossing assignment beats the greedy one: greedy takes 0.9 then 0.3, optimum 0.8 + 0.8
    S = np.array([[0.9, 0.8], [0.8, 0.3]])
    match, obj, _, _ = oracle.exact_matching(S, z=0.0)
    assert match.tolist() == [1, 0] and obj == pytest.approx(1.6)


@pytest.mark.parametrize("M,B", [(30, 20), (20, 30), (25, 25), (48, 16), (5, 60)])
def test_library_assignment_routine_agrees(oracle, M, B):
    S = _rng(M * 100 + B).uniform(-0.3, 1.0, size=(M, B))
    z = 0.2
    match, obj, _, _ = oracle.exact_matching(S, z=z)
    _check_matching(match, M)
    gain = np.maximum(S - z, 0.0)
    rows, cols = linear_sum_assignment(gain, maximize=True)
    assert obj == pytest.approx(gain[rows, cols].sum() + z * (M + B), abs=1e-10)


@pytest.mark.parametrize("seed", range(4))
def test_duality_certificate(oracle, seed):
    # N ~ 50: a dual (u, v) of the clipped assignment problem with u_i + v_j >= max(S_ij - z, 0) everywhere,
    # the duals of the side that may stay unassigned >= 0, and sum u + sum v equal to the gain the matching
    # collects, proves that no matching collects more (weak duality), whoever computed it.
    r = _rng(50 + seed)
    M, B = int(r.integers(25, 35)), int(r.integers(15, 25))
    S = r.uniform(-0.5, 1.0, size=(M, B))
    z = 0.2
    match, obj, du, dv = oracle.exact_matching(S, z=z)
    gain = np.maximum(S - z, 0.0)
    assert np.all(du[:, None] + dv[None, :] >= gain - 1e-12)
    assert np.all(du >= -1e-12)                       # B < M here: kept tokens are the side with free members
    collected = sum(gain[i, j] for j, i in enumerate(match) if i >= 0)
    assert du.sum() + dv.sum() == pytest.approx(collected, abs=1e-10)
    assert obj == pytest.approx(collected + z * (M + B), abs=1e-10)


def test_small_eps_sinkhorn_tends_to_the_exact_plan(oracle):
    # the entropic plan of Appendix C tends to the LP's vertex as eps -> 0 (when the optimum is unique with
    # a margin): the exact solver must name the same pairs, on problems larger than brute force reaches
    checked = 0
    for seed in range(30):
        r = _rng(300 + seed)
        M, B = int(r.integers(6, 14)), int(r.integers(3, 9))
        S = np.round(r.uniform(-1.0, 1.0, size=(M, B)), 1)
        match, obj, _, _ = oracle.exact_matching(S, z=0.25)
        _, _, P = oracle.sinkhorn(S, z=0.25, eps=0.005, iters=20000)
        hard = P[:M, :B]
        if not np.all((hard > 0.99) | (hard < 0.01)):
            continue                                    # optimum not unique: the entropic plan splits mass
        got = [-1] * B
        for i, j in zip(*np.nonzero(hard > 0.5)):
            got[j] = int(i)
        assert got == match.tolist(), (seed, S)
        checked += 1
    assert checked >= 8


def test_plan_of_a_matching_has_the_marginals_of_eq_5(oracle):
    S = _rng(9).uniform(-0.2, 1.0, size=(12, 7))
    match, obj, _, _ = oracle.exact_matching(S, z=0.2)
    Pbar = oracle.matching_plan(match, 12)
    np.testing.assert_allclose(Pbar.sum(axis=1), [1.0] * 12 + [7.0])
    np.testing.assert_allclose(Pbar.sum(axis=0), [1.0] * 7 + [12.0])
    Sbar = np.full((13, 8), 0.2)
    Sbar[:12, :7] = S
    assert (Sbar * Pbar).sum() == pytest.approx(obj, abs=1e-12)


def test_whole_image_in_exact_mode(oracle):
    from paper_2605_00392_b200 import synth
    w = synth.ragged([60], params=dict(r_fixed=0.3))
    p = oracle.Params(r_fixed=float(np.float32(0.3)), exact=True)
    im = oracle.run_image(w.image_f64(0), p)
    assert im.M == 42 and im.B == 18 and im.Pbar.shape == (43, 19)
    X = w.image_f64(0)
    expect = X[im.kept].copy()
    for j, i in enumerate(im.partner):
        if i >= 0:
            expect[i] += 0.1 * X[im.prop[j]]
    np.testing.assert_allclose(im.Y, expect, rtol=1e-12, atol=1e-12)
