"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these tests re-types an oracle formula: each compares the oracle with a printed value, a
closed form, a different formulation of the same object (scaling-form Sinkhorn, the Gram identity
for phi, brute-force enumeration), or an invariant.  A mistake planted in the oracle (dropped term,
sign, index, transposed operand) should fail at least one of them.
"""
import itertools
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rng(seed):
    return np.random.Generator(np.random.Philox(key=seed))


def _tokens(seed, n, d, spread=True):
    r = _rng(seed)
    x = r.standard_normal((n, d))
    if spread:
        x *= np.exp(0.5 * r.standard_normal(n))[:, None]
    return x


# ---------------------------------------------------------------------------- Eq. 1: norms
def test_norms_hand_values(oracle):
    T = np.array([[3.0, 4.0, 0.0], [0.0, 0.0, 0.0], [1.0, -2.0, 2.0], [-12.0, 0.0, 5.0]])
    np.testing.assert_array_equal(oracle.norms(T), [5.0, 0.0, 3.0, 13.0])


def test_norms_match_library(oracle):
    T = _tokens(1, 37, 53)
    np.testing.assert_allclose(oracle.norms(T), np.linalg.norm(T, axis=1), rtol=1e-14)


# ---------------------------------------------------------------------------- Eq. 8: phi
def test_phi_hand_value(oracle):
    # cosines: (e1,e2)=0, (e1,e1+e2)=1/sqrt2, (e2,e1+e2)=1/sqrt2 -> mean = sqrt2/3
    T = np.array([[2.0, 0.0], [0.0, 0.5], [3.0, 3.0]])
    assert oracle.phi(T) == pytest.approx(np.sqrt(2.0) / 3.0, abs=1e-15)


def test_phi_orthogonal_and_parallel(oracle):
    T = np.diag([1.0, 2.0, 3.0, 4.0, 0.5])
    assert oracle.phi(T) == pytest.approx(0.0, abs=1e-15)
    base = _tokens(2, 1, 9)[0]
    T = np.outer([0.3, 1.0, 2.5, 7.0], base)
    assert oracle.phi(T) == pytest.approx(1.0, abs=1e-14)
    T[2] *= -1.0      # one antiparallel token: pairs (3 of 6) flip sign -> phi = 0
    assert oracle.phi(T) == pytest.approx(0.0, abs=1e-14)


def test_phi_gram_identity(oracle):
    # sum_{i<j} xh_i.xh_j = (|sum_i xh_i|^2 - N) / 2: a different route to the same number
    for seed, n, d in [(3, 2, 5), (4, 17, 8), (5, 64, 40)]:
        T = _tokens(seed, n, d) + 0.7          # a common offset makes phi clearly non-zero
        xh = T / np.linalg.norm(T, axis=1, keepdims=True)
        s = xh.sum(axis=0)
        closed = (s @ s - n) / (n * (n - 1))
        assert oracle.phi(T) == pytest.approx(closed, abs=1e-13)
    assert oracle.phi(_tokens(6, 1, 4)) == 0.0   # a single token has no pair


def test_phi_scale_invariant(oracle):
    T = _tokens(7, 12, 6) + 0.3
    scaled = T * np.linspace(0.1, 9.0, 12)[:, None]
    assert oracle.phi(scaled) == pytest.approx(oracle.phi(T), abs=1e-14)


# ---------------------------------------------------------------------------- Eq. 10 and M = N(1-r)
def test_token_counts_printed_in_the_paper(oracle):
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "token_counts.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 6
    for n, r, m in rows:
        _, B, M = oracle.ratio(0.0, 0.0, int(n), dynamic=False, r_fixed=float(r))
        assert M == int(m) and B == int(n) - int(m)


def test_ratio_fp32_constant_rounds_to_nearest(oracle):
    # 0.35 stored in fp32 is 0.34999999404...; 400 tokens must still give B = 140
    r32 = float(np.float32(0.35))
    assert oracle.ratio(0.0, 0.0, 400, dynamic=False, r_fixed=r32)[1:] == (140, 260)


def test_ratio_dynamic_hand_cases(oracle):
    r, B, M = oracle.ratio(0.4, 0.5, 100, dynamic=True)                     # identity f_normalize
    assert (r, B, M) == (pytest.approx(0.2), 20, 80)
    r, B, M = oracle.ratio(0.4, 0.5, 100, dynamic=True, phi_lo=0.2, phi_hi=0.6)
    assert (r, B, M) == (pytest.approx(0.25), 25, 75)
    assert oracle.ratio(0.9, 0.0, 100, dynamic=True, phi_hi=0.5)[0] == pytest.approx(1.0)   # clamp hi
    assert oracle.ratio(-0.3, 0.0, 100, dynamic=True)[0] == 0.0                              # clamp lo
    assert oracle.ratio(0.9, 0.0, 100, dynamic=True, r_max=0.5)[1:] == (50, 50)              # cap
    assert oracle.ratio(0.9, 1.0, 100, dynamic=True)[1:] == (0, 100)     # rho = 1: nothing pruned
    assert oracle.ratio(1.0, 0.0, 10, dynamic=True)[1:] == (9, 1)        # at least one token kept


def test_ratio_monotone(oracle):
    phis = np.linspace(-0.2, 1.2, 29)
    rs = [oracle.ratio(p, 0.3, 400, dynamic=True, phi_lo=0.1, phi_hi=0.8)[0] for p in phis]
    assert all(b >= a for a, b in zip(rs, rs[1:])) and rs[0] == 0.0 and rs[-1] == pytest.approx(0.7)
    rhos = np.linspace(0.0, 1.0, 21)
    rs = [oracle.ratio(0.5, q, 400, dynamic=True)[0] for q in rhos]
    assert all(b <= a for a, b in zip(rs, rs[1:]))


# ---------------------------------------------------------------------------- stage 1: top-M
def test_select_matches_lexsort(oracle):
    r = _rng(11)
    for n, m in [(1, 1), (5, 2), (64, 48), (257, 100), (400, 400)]:
        C = np.exp(r.standard_normal(n))
        C[r.integers(0, n, size=n // 4)] = C[0]            # plant exact ties
        kept, prop = oracle.select(C, m)
        order = np.lexsort((np.arange(n), -C))             # C descending, then index ascending
        np.testing.assert_array_equal(kept, np.sort(order[:m]))
        np.testing.assert_array_equal(prop, np.sort(order[m:]))


def test_select_ties_keep_lower_index(oracle):
    kept, prop = oracle.select(np.array([1.0, 2.0, 2.0, 2.0, 0.5]), 2)
    np.testing.assert_array_equal(kept, [1, 2])
    np.testing.assert_array_equal(prop, [0, 3, 4])


# ---------------------------------------------------------------------------- scores
def test_scores_match_normalised_matmul(oracle):
    T = _tokens(21, 23, 11)
    C = np.linalg.norm(T, axis=1)
    kept = np.array([0, 3, 4, 9, 10, 15, 22], dtype=np.int32)
    prop = np.array([1, 2, 20], dtype=np.int32)
    S = oracle.scores(T, C, kept, prop)
    xh = T / C[:, None]
    np.testing.assert_allclose(S, xh[kept] @ xh[prop].T, atol=1e-14)
    assert S.shape == (7, 3)
    assert np.all(np.abs(S) <= 1.0 + 1e-14)
    # a token scored against a scaled copy of itself has cosine exactly 1 (up to rounding)
    T2 = np.vstack([T[:2], 3.0 * T[0]])
    S2 = oracle.scores(T2, np.linalg.norm(T2, axis=1), np.array([0, 1], np.int32),
                       np.array([2], np.int32))
    assert S2[0, 0] == pytest.approx(1.0, abs=1e-14)


def test_scores_zero_token_gives_zero(oracle):
    T = _tokens(22, 4, 6)
    T[2] = 0.0
    S = oracle.scores(T, oracle.norms(T), np.array([0, 1], np.int32), np.array([2, 3], np.int32))
    np.testing.assert_array_equal(S[:, 0], [0.0, 0.0])


# ---------------------------------------------------------------------------- Sinkhorn (Eq. 5, App. C)
def _random_scores(seed, M, B):
    return np.tanh(_rng(seed).standard_normal((M, B)))


@pytest.mark.parametrize("M,B", [(1, 1), (5, 3), (3, 5), (48, 16), (300, 100), (337, 63)])
def test_sinkhorn_marginals(oracle, M, B):
    S = _random_scores(31, M, B)
    u, v, P = oracle.sinkhorn(S, z=0.2, eps=1.0, iters=100)
    a = np.concatenate([np.ones(M), [B]])
    b = np.concatenate([np.ones(B), [M]])
    np.testing.assert_allclose(P.sum(axis=1), a, rtol=1e-10)
    np.testing.assert_allclose(P.sum(axis=0), b, rtol=1e-10)
    assert P.shape == (M + 1, B + 1) and np.all(P > 0)
    # the plan is diag(e^u) exp(S-bar) diag(e^v) cell by cell
    Sbar = np.full((M + 1, B + 1), 0.2)
    Sbar[:M, :B] = S
    np.testing.assert_allclose(P, np.exp(Sbar + u[:, None] + v[None, :]), rtol=1e-12)


def test_sinkhorn_last_update_is_v(oracle):
    # after ONE iteration (u then v) the column marginals are exact and the row marginals are not
    S = _random_scores(32, 6, 4)
    _, _, P = oracle.sinkhorn(S, iters=1)
    np.testing.assert_allclose(P.sum(axis=0), [1, 1, 1, 1, 6], rtol=1e-13)
    assert np.max(np.abs(P.sum(axis=1) - [1, 1, 1, 1, 1, 1, 4])) > 1e-4


def test_sinkhorn_first_half_iteration_by_hand(oracle):
    # with v = 0 the first u is log mu - log sum_j exp(Z_ij); check through iters=1 and the final v
    S = np.array([[0.5, -0.25]])
    z, eps = 0.2, 0.5
    u, v, _ = oracle.sinkhorn(S, z=z, eps=eps, iters=1)
    Z = np.array([[0.5, -0.25, z], [z, z, z]]) / eps
    u_hand = np.array([0.0, np.log(2.0)]) - np.log(np.exp(Z).sum(axis=1))
    v_hand = np.array([0.0, 0.0, np.log(1.0)]) - np.log(np.exp(Z + u_hand[:, None]).sum(axis=0))
    np.testing.assert_allclose(u, u_hand, atol=1e-14)
    np.testing.assert_allclose(v, v_hand, atol=1e-14)


@pytest.mark.parametrize("eps", [1.0, 0.3])
def test_sinkhorn_equals_scaling_form(oracle, eps):
    # textbook Sinkhorn-Knopp on the kernel K = exp(S-bar/eps): u <- a / (K v), v <- b / (K^T u)
    M, B = 40, 13
    S = _random_scores(33, M, B)
    Sbar = np.full((M + 1, B + 1), 0.2)
    Sbar[:M, :B] = S
    K = np.exp(Sbar / eps)
    a = np.concatenate([np.ones(M), [B]])
    b = np.concatenate([np.ones(B), [M]])
    su, sv = np.ones(M + 1), np.ones(B + 1)
    for _ in range(25):
        su = a / (K @ sv)
        sv = b / (K.T @ su)
    u, v, P = oracle.sinkhorn(S, z=0.2, eps=eps, iters=25)
    np.testing.assert_allclose(np.exp(u), su, rtol=1e-11)
    np.testing.assert_allclose(np.exp(v), sv, rtol=1e-11)
    np.testing.assert_allclose(P, su[:, None] * K * sv[None, :], rtol=1e-11)


@pytest.mark.parametrize("N,M,c,z,eps", [(64, 48, 0.0, 0.2, 1.0), (400, 300, 0.0, 0.2, 1.0),
                                         (400, 337, 1.0, 0.2, 1.0), (8, 5, 0.6, 0.2, 0.5),
                                         (12, 7, 0.2, 0.2, 1.0), (30, 20, -0.3, 0.5, 0.7)])
def test_sinkhorn_closed_form_for_equal_scores(oracle, N, M, c, z, eps):
    # All real scores equal c.  The four marginal equations plus the rank-one structure of
    # diag(e^u) K diag(e^v) give every real cell x as the root in (0, 1/max(M,B)) of
    #   M B (1-k) x^2 + k N x - k = 0,  k = exp((c - z)/eps)     (x = 1/N when k = 1)
    B = N - M
    k = np.exp((c - z) / eps)
    if abs(k - 1.0) < 1e-14:
        x = 1.0 / N
    else:
        qa, qb, qc = M * B * (1.0 - k), k * N, -k
        roots = [(-qb + s * np.sqrt(qb * qb - 4 * qa * qc)) / (2 * qa) for s in (1.0, -1.0)]
        x = [t for t in roots if 0.0 < t < 1.0 / max(M, B)][0]
    _, _, P = oracle.sinkhorn(np.full((M, B), c), z=z, eps=eps, iters=100)
    np.testing.assert_allclose(P[:M, :B], x, rtol=1e-10)
    np.testing.assert_allclose(P[:M, B], 1.0 - B * x, rtol=1e-9)
    np.testing.assert_allclose(P[M, :B], 1.0 - M * x, rtol=1e-9)
    assert P[M, B] == pytest.approx(M * B * x, rel=1e-9)


def test_sinkhorn_fixed_point_at_T100(oracle):
    S = _random_scores(34, 60, 21)
    _, _, P100 = oracle.sinkhorn(S, iters=100)
    _, _, P101 = oracle.sinkhorn(S, iters=101)
    np.testing.assert_allclose(P101, P100, rtol=1e-12)


def _best_partial_matchings(S, z):
    """Brute force over all partial matchings kept<->prop; value = sum of (S_ij - z) over pairs."""
    M, B = S.shape
    results = []
    for m in range(0, min(M, B) + 1):
        for rows in itertools.combinations(range(M), m):
            for cols in itertools.permutations(range(B), m):
                results.append((sum(S[i, j] - z for i, j in zip(rows, cols)),
                                tuple(sorted(zip(rows, cols)))))
    results.sort(key=lambda t: -t[0])
    return results


def test_small_eps_sinkhorn_rounds_to_brute_force_matching(oracle):
    # eps -> 0: the entropic plan tends to the vertex of the linear programme (Eq. 2 with the
    # dustbin marginals), i.e. the maximum-weight partial matching with pair gain S_ij - z.
    checked = 0
    for seed in range(60):
        r = _rng(1000 + seed)
        N = int(r.integers(3, 9))
        M = int(r.integers(1, N))
        B = N - M
        S = np.round(r.uniform(-1.0, 1.0, size=(M, B)), 2)
        z = 0.2
        ranked = _best_partial_matchings(S, z)
        if len(ranked) > 1 and ranked[0][0] - ranked[1][0] < 0.1:
            continue                                   # optimum not unique with margin
        _, _, P = oracle.sinkhorn(S, z=z, eps=0.01, iters=5000)
        got = tuple(sorted((int(i), int(j)) for i, j in zip(*np.nonzero(P[:M, :B] > 0.5))))
        assert got == ranked[0][1], (seed, S, got, ranked[0])
        assert np.all((P[:M, :B] > 0.99) | (P[:M, :B] < 0.01))
        checked += 1
    assert checked >= 15


# ---------------------------------------------------------------------------- merge (Eq. 7), partners
def _stage2(oracle, T, M, z=0.2, eps=1.0, iters=100):
    C = oracle.norms(T)
    kept, prop = oracle.select(C, M)
    S = oracle.scores(T, C, kept, prop)
    u, v, P = oracle.sinkhorn(S, z=z, eps=eps, iters=iters)
    return kept, prop, P


def test_merge_matches_matrix_product(oracle):
    T = _tokens(41, 30, 17)
    kept, prop, P = _stage2(oracle, T, 21)
    Y = oracle.merge(T, kept, prop, P, alpha=0.1)
    np.testing.assert_allclose(Y, T[kept] + 0.1 * P[:-1, :-1] @ T[prop], rtol=1e-13, atol=1e-13)
    assert Y.shape == (21, 17)


def test_merge_alpha_zero_is_plain_pruning(oracle):
    T = _tokens(42, 25, 9)
    kept, prop, P = _stage2(oracle, T, 18)
    np.testing.assert_array_equal(oracle.merge(T, kept, prop, P, alpha=0.0), T[kept])


def test_merge_linear_in_alpha(oracle):
    T = _tokens(43, 25, 9)
    kept, prop, P = _stage2(oracle, T, 18)
    y1 = oracle.merge(T, kept, prop, P, alpha=0.1) - T[kept]
    y5 = oracle.merge(T, kept, prop, P, alpha=0.5) - T[kept]
    np.testing.assert_allclose(y5, 5.0 * y1, rtol=1e-12, atol=1e-14)


def test_merge_closed_form_orthogonal_tokens(oracle):
    # distinct scaled basis vectors: every cosine is 0, the plan is the constant x of the closed form
    N, M, alpha, z = 12, 8, 0.1, 0.2
    T = np.diag(np.linspace(1.0, 4.0, N))
    res = oracle.run_image(T, oracle.Params(r_fixed=1.0 - M / N, z=z, alpha=alpha))
    B = N - M
    k = np.exp(0.0 - z)
    qa, qb, qc = M * B * (1.0 - k), k * N, -k
    x = (-qb + np.sqrt(qb * qb - 4 * qa * qc)) / (2 * qa)
    assert 0 < x < 1.0 / M
    np.testing.assert_array_equal(res.kept, np.arange(N - M, N))      # the largest norms
    expect = T[res.kept] + alpha * x * T[res.prop].sum(axis=0)[None, :]
    np.testing.assert_allclose(res.Y, expect, rtol=1e-10, atol=1e-12)


def test_scaling_a_pruned_token_only_scales_its_contribution(oracle):
    T = _tokens(44, 20, 7)
    C = oracle.norms(T)
    kept, prop = oracle.select(C, 14)
    T2 = T.copy()
    j = prop[np.argmax(C[prop])]
    T2[j] *= 0.5                    # still among the pruned: it had the largest pruned norm, now smaller
    kept2, prop2, P2 = _stage2(oracle, T2, 14)
    _, _, P = _stage2(oracle, T, 14)
    np.testing.assert_array_equal(kept2, kept)
    np.testing.assert_allclose(P2, P, rtol=1e-12)       # cosines do not see the scale


def test_scaling_an_image_scales_the_output(oracle):
    T = _tokens(45, 33, 12)
    p = oracle.Params(r_fixed=0.3)
    a = oracle.run_image(T, p)
    b = oracle.run_image(4.0 * T, p)                    # power of two: exact in fp64
    np.testing.assert_array_equal(a.kept, b.kept)
    np.testing.assert_array_equal(a.partner, b.partner)
    np.testing.assert_allclose(b.Y, 4.0 * a.Y, rtol=1e-13)


def test_partners_are_column_argmax(oracle):
    T = _tokens(46, 40, 10)
    res = oracle.run_image(T, oracle.Params(r_fixed=0.4), want_plan=True)
    P = res.Pbar[:-1, :-1]
    np.testing.assert_array_equal(res.partner, np.argmax(P, axis=0))
    np.testing.assert_allclose(res.weight, P.max(axis=0), rtol=0)
    top2 = np.sort(np.log(P), axis=0)[-2:]
    np.testing.assert_allclose(res.gap, top2[1] - top2[0], atol=1e-12)
    # argmax_i P_ij is argmax_i (Z_ij + u_i): v_j is common to the column
    S = oracle.scores(T, res.C, res.kept, res.prop)
    np.testing.assert_array_equal(res.partner, np.argmax(S + res.u[:-1, None], axis=0))


def test_partner_tie_goes_to_lower_kept_index(oracle):
    # two bit-identical kept tokens receive bit-identical plan rows: the pair goes to the first
    T = _tokens(47, 9, 5)
    T[4] = T[1] = 10.0 * T[1]
    res = oracle.run_image(T, oracle.Params(r_fixed=1.0 / 3.0), want_plan=True)
    pos1, pos4 = list(res.kept).index(1), list(res.kept).index(4)
    np.testing.assert_array_equal(res.Pbar[pos1], res.Pbar[pos4])
    assert pos4 not in set(res.partner)
    T[:, :] = T[1]                      # every token identical: all pairs go to kept position 0
    res = oracle.run_image(T, oracle.Params(r_fixed=1.0 / 3.0))
    np.testing.assert_array_equal(res.kept, np.arange(6))
    np.testing.assert_array_equal(res.partner, [0, 0, 0])


# ---------------------------------------------------------------------------- Algorithm 1 as a whole
def test_pipeline_matches_its_steps(oracle):
    T = _tokens(51, 50, 16) + 0.4
    p = oracle.Params(dynamic=True, phi_lo=0.0, phi_hi=0.6, r_max=0.5, z=0.3, alpha=0.2, eps=0.8,
                      iters=60)
    rho = 0.25
    res = oracle.run_image(T, p, rho, want_plan=True)
    C = oracle.norms(T)
    ph = oracle.phi(T, C)
    r, B, M = oracle.ratio(ph, rho, 50, dynamic=True, phi_lo=0.0, phi_hi=0.6, r_max=0.5)
    kept, prop = oracle.select(C, M)
    S = oracle.scores(T, C, kept, prop)
    u, v, P = oracle.sinkhorn(S, z=0.3, eps=0.8, iters=60)
    Y = oracle.merge(T, kept, prop, P, alpha=0.2)
    assert (res.M, res.B, res.phi, res.r) == (M, B, ph, r) and 0 < B < 50
    np.testing.assert_array_equal(res.kept, kept)
    np.testing.assert_array_equal(res.Y, Y)
    np.testing.assert_array_equal(res.Pbar, P)


def test_retention_one_is_identity(oracle):
    T = _tokens(52, 19, 8)
    for p, rho in [(oracle.Params(r_fixed=0.0), 0.0), (oracle.Params(dynamic=True), 1.0)]:
        res = oracle.run_image(T, p, rho)
        assert res.M == 19 and res.B == 0 and len(res.partner) == 0
        np.testing.assert_array_equal(res.kept, np.arange(19))
        np.testing.assert_array_equal(res.Y, T)


def test_permutation_equivariance(oracle):
    T = _tokens(53, 36, 14) + 0.2
    p = oracle.Params(dynamic=True, phi_hi=0.5, r_max=0.5)
    perm = _rng(54).permutation(36)
    a = oracle.run_image(T, p, 0.2)
    b = oracle.run_image(T[perm], p, 0.2)          # token perm[k] of a sits at position k of b
    assert a.M == b.M and a.phi == pytest.approx(b.phi, abs=1e-14)
    np.testing.assert_array_equal(np.sort(perm[b.kept]), a.kept)
    ya = {int(k): a.Y[i] for i, k in enumerate(a.kept)}
    for i, k in enumerate(b.kept):
        np.testing.assert_allclose(b.Y[i], ya[int(perm[k])], rtol=1e-12, atol=1e-13)
    pa = {int(a.prop[j]): int(a.kept[a.partner[j]]) for j in range(a.B)}
    for j in range(b.B):
        assert pa[int(perm[b.prop[j]])] == int(perm[b.kept[b.partner[j]]])


def test_counts_and_partition(oracle):
    lens = [5, 64, 1, 33]
    r = _rng(55)
    X = np.concatenate([_tokens(60 + i, n, 10) for i, n in enumerate(lens)])
    offsets = np.concatenate([[0], np.cumsum(lens)])
    res = oracle.run_batch(X, offsets, oracle.Params(r_fixed=0.3), threads=2)
    assert list(res.counts) == [n - int(np.floor(0.3 * n + 0.5)) if n > 1 else 1 for n in lens]
    assert res.out_offsets[-1] == res.counts.sum()
    for im, n in zip(res.images, lens):
        assert im.M + im.B == n and len(im.kept) == im.M and len(im.prop) == im.B
        both = np.concatenate([im.kept, im.prop])
        np.testing.assert_array_equal(np.sort(both), np.arange(n))
        assert np.all(np.diff(im.kept) > 0) and np.all(np.diff(im.prop) > 0)
        assert im.Y.shape == (im.M, 10)
        if im.B:
            assert np.all((im.partner >= 0) & (im.partner < im.M))
    # a threaded run is the same arithmetic
    res1 = oracle.run_batch(X, offsets, oracle.Params(r_fixed=0.3), threads=1)
    for a, b in zip(res.images, res1.images):
        np.testing.assert_array_equal(a.Y, b.Y)


# ------------------------------------------------- selection-metric ablation: variance, entropy
def test_variance_hand_values_and_library(oracle):
    T = np.array([[1.0, 1.0, 1.0, 1.0], [0.0, 2.0, 0.0, 2.0], [-3.0, 0.0, 3.0, 0.0], [1.0, 2.0, 3.0, 4.0]])
    np.testing.assert_allclose(oracle.variance(T), [0.0, 1.0, 4.5, 1.25], rtol=0, atol=1e-15)
    T = _tokens(31, 29, 47) + 0.3
    np.testing.assert_allclose(oracle.variance(T), np.var(T, axis=1), rtol=1e-13)


def test_variance_ignores_a_common_shift_and_scales_quadratically(oracle):
    # the paper's remark on this metric: a token whose norm grows by an overall feature shift is not
    # ranked higher by its variance
    T = _tokens(32, 11, 40)
    v = oracle.variance(T)
    np.testing.assert_allclose(oracle.variance(T + 5.0), v, rtol=1e-12)
    assert np.all(oracle.norms(T + 5.0) > oracle.norms(T))
    np.testing.assert_allclose(oracle.variance(-3.0 * T), 9.0 * v, rtol=1e-13)
    # and it is the mean square minus the squared mean
    np.testing.assert_allclose(v, (T * T).mean(axis=1) - T.mean(axis=1) ** 2, rtol=1e-12)


def test_entropy_closed_forms(oracle):
    d = 12
    # equal features: the uniform distribution, log d
    assert oracle.entropy(np.full((1, d), -2.5))[0] == pytest.approx(np.log(d), abs=1e-14)
    # one feature far above the rest: a point mass, 0
    T = np.zeros((1, d))
    T[0, 3] = 800.0
    assert oracle.entropy(T)[0] == pytest.approx(0.0, abs=1e-300)
    # two levels: k features at a, the rest at 0 -> p = e^a / (k e^a + d - k) on the k, 1 / (...) elsewhere
    a, k = 1.7, 5
    T = np.zeros((1, d))
    T[0, :k] = a
    zsum = k * np.exp(a) + (d - k)
    p1, p0 = np.exp(a) / zsum, 1.0 / zsum
    expect = -(k * p1 * np.log(p1) + (d - k) * p0 * np.log(p0))
    assert oracle.entropy(T)[0] == pytest.approx(expect, abs=1e-14)
    # large features must not overflow (max-shifted) and a common shift changes nothing
    T = _tokens(33, 6, 30)
    np.testing.assert_allclose(oracle.entropy(T + 700.0), oracle.entropy(T), rtol=1e-12)


def test_entropy_matches_library(oracle):
    from scipy.special import softmax
    from scipy.stats import entropy as scipy_entropy
    T = 2.0 * _tokens(34, 23, 61)
    np.testing.assert_allclose(oracle.entropy(T), scipy_entropy(softmax(T, axis=1), axis=1), rtol=1e-12)
    # a permutation of the features changes nothing; sharpening (scaling up) lowers the entropy
    np.testing.assert_allclose(oracle.entropy(T[:, ::-1]), oracle.entropy(T), rtol=1e-13)
    assert np.all(oracle.entropy(3.0 * T) < oracle.entropy(T))


@pytest.mark.parametrize("which", [1, 2])
def test_alternative_criterion_changes_only_the_ranking(oracle, which):
    # stage 1 keeps the M tokens of largest criterion (ties to the lower index); everything after the
    # selection is the unchanged pipeline applied to that split
    T = _tokens(35 + which, 24, 16) + np.linspace(-1.0, 1.0, 24)[:, None]   # shifts separate norm and variance rankings
    p = oracle.Params(r_fixed=0.375, criterion=which)
    res = oracle.run_image(T, p, want_plan=True)
    C = oracle.criterion(T, which)
    M = 15
    rank = sorted(range(24), key=lambda k: (-C[k], k))
    assert res.M == M and res.kept.tolist() == sorted(rank[:M]) and res.prop.tolist() == sorted(rank[M:])
    assert res.kept.tolist() != oracle.run_image(T, oracle.Params(r_fixed=0.375)).kept.tolist()
    np.testing.assert_array_equal(res.C, oracle.norms(T))          # cosines still use the l2 norms
    S = oracle.scores(T, res.C, res.kept, res.prop)
    _, _, Pbar = oracle.sinkhorn(S)
    np.testing.assert_allclose(res.Pbar, Pbar, rtol=1e-13)
    np.testing.assert_allclose(res.Y, oracle.merge(T, res.kept, res.prop, Pbar), rtol=1e-13)


def test_criterion_ties_keep_lower_index(oracle):
    T = _tokens(38, 10, 8)
    T[7] = T[2]
    T[9] = T[2] + 4.0              # same variance as tokens 2 and 7, another norm
    for which in (1, 2):
        C = oracle.criterion(T, which)
        assert C[7] == C[2]
    C = oracle.variance(T)
    assert C[9] == pytest.approx(C[2], rel=1e-12)
    order = sorted(range(10), key=lambda k: (-oracle.variance(T)[k], k))
    M = order.index(7)             # cut between token 2 (kept) and token 7
    if order.index(2) < M:
        res = oracle.run_image(T, oracle.Params(r_fixed=(10 - M) / 10.0, criterion=1))
        assert 2 in res.kept and 7 in res.prop


def test_echo_tokens_pair_with_their_anchors(oracle):
    """An input whose answer is known without running anything: the pruned tokens are noisy low-norm copies of
    kept tokens.  The oracle must keep exactly the anchors and pair every echo with its own anchor, by a wide
    margin (the generator's construction, not the oracle's arithmetic, is the reference here)."""
    import torch
    from paper_2605_00392_b200 import synth
    w, truth = synth.paired([64, 100, 37], 0.25, d=256, dtype=torch.float32)
    res = oracle.run_batch(w.X_f64(), w.offsets, oracle.Params(r_fixed=0.25), w.rho, want_plan=True)
    for i, (im, echo_of) in enumerate(zip(res.images, truth)):
        anchors = np.nonzero(echo_of < 0)[0]
        echoes = np.nonzero(echo_of >= 0)[0]
        np.testing.assert_array_equal(im.kept, anchors)
        np.testing.assert_array_equal(im.prop, echoes)
        np.testing.assert_array_equal(im.kept[im.partner], echo_of[echoes])
        assert im.gap.min() > 0.5            # log P of the anchor stands clear of every other kept token
        # the exact pairing is one to one: every anchor with echoes is paired with one of its own echoes (a
        # second echo of the same anchor may find a stranger worth more than the dustbin score, or nobody)
        ex = oracle.run_image_exact(w.image_f64(i), oracle.Params(r_fixed=0.25))
        taken = {int(ex.kept[p]): int(ex.prop[j]) for j, p in enumerate(ex.partner) if p >= 0}
        for a in np.unique(echo_of[echoes]):
            assert int(a) in taken and echo_of[taken[int(a)]] == a, (i, int(a))
