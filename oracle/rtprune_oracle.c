/*
 * RTPrune visual-token pruning -- plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
 * CUDA path must compute.  It shares no code with the CUDA path, is never called by the
 * product, and is only reached from the tests, the smoke check and the benchmark's CPU-baseline
 * leg.  Everything is scalar double-precision loops: no blocking, no fusion, no BLAS.
 *
 * Each function cites the passage of the paper (RTPrune) it follows.  Notation follows the
 * paper: T_v is the N x D token matrix, C_k the selection criterion, M the number of kept
 * tokens, S the cosine score matrix, S-bar / P-bar the dustbin-augmented score / plan, u and v
 * the Sinkhorn duals, alpha the merge strength, z the dustbin score, phi the mean inter-token
 * similarity, rho the textual density.
 *
 * Parity pins (tests that check this file against the paper and the mathematics, not against
 * itself): see tests/test_oracle_pins.py.  Parity UNPINNED against the paper (the paper is silent,
 * so only the reading chosen here can be checked): the form of f_normalize in Eq. 10, the
 * semantics of rho as a caller-supplied number, and the pruning unit of a multi-view image.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define RTP_ORACLE_NORM_FLOOR 1e-12 /* divisor floor for a zero-norm token (paper silent) */

/* Eq. 1: selection criterion C_k = || T_v^k ||_2 for every token k. */
void rtp_oracle_norms(const double *T, int N, int D, double *C)
{
    for (int k = 0; k < N; ++k) {
        double ss = 0.0;
        for (int c = 0; c < D; ++c)
            ss += T[(size_t)k * D + c] * T[(size_t)k * D + c];
        C[k] = sqrt(ss);
    }
}

/*
 * Selection-metric ablation (the table that ranks tokens by "variance" and by "entropy" instead of the
 * l2 norm): alternative criteria C_k for stage 1; everything after the selection is unchanged
 * (cosines still divide by the l2 norms).
 *   variance: C_k = (1/D) sum_c (T_kc - mean_k)^2, mean_k = (1/D) sum_c T_kc  (population variance
 *             over the D features of token k, the "dispersion" the ablation's discussion speaks of).
 *   entropy:  the paper gives no formula.  Reading taken: the token's features are turned into a
 *             distribution over the D channels by a softmax, p_c = exp(T_kc) / sum_c' exp(T_kc'),
 *             and C_k = - sum_c p_c log p_c (natural logarithm); the M tokens of LARGEST criterion
 *             are kept, as for the other two.  PARITY UNPINNED against the paper for this reading.
 */
void rtp_oracle_variance(const double *T, int N, int D, double *C)
{
    for (int k = 0; k < N; ++k) {
        double mean = 0.0;
        for (int c = 0; c < D; ++c)
            mean += T[(size_t)k * D + c];
        mean /= (double)D;
        double acc = 0.0;
        for (int c = 0; c < D; ++c) {
            double dv = T[(size_t)k * D + c] - mean;
            acc += dv * dv;
        }
        C[k] = acc / (double)D;
    }
}

void rtp_oracle_entropy(const double *T, int N, int D, double *C)
{
    for (int k = 0; k < N; ++k) {
        const double *t = T + (size_t)k * D;
        double mx = t[0];
        for (int c = 1; c < D; ++c)
            if (t[c] > mx) mx = t[c];
        double total = 0.0;
        for (int c = 0; c < D; ++c)
            total += exp(t[c] - mx);
        double h = 0.0;
        for (int c = 0; c < D; ++c) {
            double p = exp(t[c] - mx) / total;
            if (p > 0.0) h -= p * log(p);
        }
        C[k] = h;
    }
}

static double floor_norm(double n) { return n > RTP_ORACLE_NORM_FLOOR ? n : RTP_ORACLE_NORM_FLOOR; }

/* Eq. 8: phi = 2 / (N (N-1)) * sum_{i<j} (T_i . T_j) / (||T_i|| ||T_j||), by the double loop. */
double rtp_oracle_phi(const double *T, const double *C, int N, int D)
{
    if (N < 2)
        return 0.0;
    double total = 0.0;
    for (int i = 0; i < N; ++i) {
        for (int j = i + 1; j < N; ++j) {
            double dot = 0.0;
            for (int c = 0; c < D; ++c)
                dot += T[(size_t)i * D + c] * T[(size_t)j * D + c];
            total += dot / (floor_norm(C[i]) * floor_norm(C[j]));
        }
    }
    return 2.0 * total / ((double)N * (double)(N - 1));
}

/*
 * Eq. 10: r_dyn = f_normalize(phi) * (1 - rho), or a fixed target ratio r.
 * Reading taken where the paper is silent: f_normalize is the affine map of [phi_lo, phi_hi] onto
 * [0, 1], clamped; r is capped at r_max.  Section 3.3.1: M = N (1 - r); reading for non-integer
 * r N: B = floor(r N + 1/2) tokens are proposed for pruning, 0 <= B <= N-1, M = N - B.
 */
void rtp_oracle_ratio(double phi, double rho, int dynamic, double r_fixed, double phi_lo,
                      double phi_hi, double r_max, int N, double *r_out, int *B_out, int *M_out)
{
    double r;
    if (dynamic) {
        double f = (phi - phi_lo) / (phi_hi - phi_lo);
        if (f < 0.0) f = 0.0;
        if (f > 1.0) f = 1.0;
        r = f * (1.0 - rho);
        if (r > r_max) r = r_max;
    } else {
        r = r_fixed;
    }
    if (r < 0.0) r = 0.0;
    int B = (int)floor(r * (double)N + 0.5);
    if (B < 0) B = 0;
    if (B > N - 1) B = N - 1;
    *r_out = r;
    *B_out = B;
    *M_out = N - B;
}

/*
 * Section 3.3.1 / Algorithm 1, stage 1: T_kept = the top-M tokens ranked by C_k, T_prop = the rest.
 * Full sort of all tokens by (C descending, index ascending), so equal criteria keep the lower
 * index; both lists are then reported in ascending original index.
 */
void rtp_oracle_select(const double *C, int N, int M, int32_t *kept, int32_t *prop)
{
    int *order = (int *)malloc(sizeof(int) * (size_t)(N > 0 ? N : 1));
    for (int k = 0; k < N; ++k)
        order[k] = k;
    /* insertion sort: stable, so ties stay in ascending index */
    for (int a = 1; a < N; ++a) {
        int k = order[a];
        int b = a - 1;
        while (b >= 0 && C[order[b]] < C[k]) {
            order[b + 1] = order[b];
            --b;
        }
        order[b + 1] = k;
    }
    char *is_kept = (char *)calloc((size_t)(N > 0 ? N : 1), 1);
    for (int a = 0; a < M; ++a)
        is_kept[order[a]] = 1;
    int nk = 0, np = 0;
    for (int k = 0; k < N; ++k) {
        if (is_kept[k]) kept[nk++] = k;
        else prop[np++] = k;
    }
    free(is_kept);
    free(order);
}

/* Section 3.3.2 (score equation) / Appendix C: S_ij = T_i . T_j / (||T_i|| ||T_j||), i kept, j prop. */
void rtp_oracle_scores(const double *T, const double *C, int D, const int32_t *kept, int M,
                       const int32_t *prop, int B, double *S)
{
    for (int i = 0; i < M; ++i) {
        const double *ti = T + (size_t)kept[i] * D;
        for (int j = 0; j < B; ++j) {
            const double *tj = T + (size_t)prop[j] * D;
            double dot = 0.0;
            for (int c = 0; c < D; ++c)
                dot += ti[c] * tj[c];
            S[(size_t)i * B + j] = dot / (floor_norm(C[kept[i]]) * floor_norm(C[prop[j]]));
        }
    }
}

static double logsumexp(const double *x, int n, int stride)
{
    double m = x[0];
    for (int k = 1; k < n; ++k)
        if (x[(size_t)k * stride] > m) m = x[(size_t)k * stride];
    double s = 0.0;
    for (int k = 0; k < n; ++k)
        s += exp(x[(size_t)k * stride] - m);
    return m + log(s);
}

/*
 * Eq. 5 + Appendix C: dustbin augmentation and log-domain Sinkhorn.
 *   S-bar is (M+1) x (B+1): S in the top-left block, z in the last row and the last column.
 *   Z = S-bar / eps (the paper gives no eps; eps = 1 uses S-bar itself as the log-kernel).
 *   log mu = [0_M, log B], log nu = [0_B, log M].
 *   u, v start at 0; each of the `iters` iterations updates u from v, then v from the new u:
 *       u_i = log mu_i - LSE_j (Z_ij + v_j),   v_j = log nu_j - LSE_i (Z_ij + u_i).
 *   P-bar = exp(Z + u 1^T + 1 v^T); the plan P is its top-left M x B block.
 * Outputs: u[M+1], v[B+1], Pbar[(M+1)*(B+1)] row-major.  Requires M >= 1 and B >= 1.
 */
void rtp_oracle_sinkhorn(const double *S, int M, int B, double z, double eps, int iters,
                         double *u, double *v, double *Pbar)
{
    const int R = M + 1, Cc = B + 1;
    double *Z = (double *)malloc(sizeof(double) * (size_t)R * Cc);
    double *tmp = (double *)malloc(sizeof(double) * (size_t)(R > Cc ? R : Cc));
    for (int i = 0; i < R; ++i)
        for (int j = 0; j < Cc; ++j)
            Z[(size_t)i * Cc + j] = ((i < M && j < B) ? S[(size_t)i * B + j] : z) / eps;
    for (int i = 0; i < R; ++i) u[i] = 0.0;
    for (int j = 0; j < Cc; ++j) v[j] = 0.0;
    for (int t = 0; t < iters; ++t) {
        for (int i = 0; i < R; ++i) {
            for (int j = 0; j < Cc; ++j)
                tmp[j] = Z[(size_t)i * Cc + j] + v[j];
            double log_mu = (i < M) ? 0.0 : log((double)B);
            u[i] = log_mu - logsumexp(tmp, Cc, 1);
        }
        for (int j = 0; j < Cc; ++j) {
            for (int i = 0; i < R; ++i)
                tmp[i] = Z[(size_t)i * Cc + j] + u[i];
            double log_nu = (j < B) ? 0.0 : log((double)M);
            v[j] = log_nu - logsumexp(tmp, R, 1);
        }
    }
    for (int i = 0; i < R; ++i)
        for (int j = 0; j < Cc; ++j)
            Pbar[(size_t)i * Cc + j] = exp(Z[(size_t)i * Cc + j] + u[i] + v[j]);
    free(tmp);
    free(Z);
}

/*
 * Eq. 2-6 solved EXACTLY (no entropic regularisation): the linear program
 *     max sum_ij S-bar_ij P-bar_ij   s.t.  P-bar 1 = a = [1_M, B],  P-bar^T 1 = b = [1_B, M],  P-bar >= 0
 * over the dustbin-augmented (M+1) x (B+1) plan.  Its constraint matrix is that of a transportation
 * problem, so an optimal vertex is integral: every kept token i is either paired with one pruned token j
 * (P_ij = 1) or sent to the dustbin column, every pruned token is either paired or sent to the dustbin
 * row, and the dustbin-dustbin cell takes the rest.  With m pairs the objective is
 *     sum_{pairs} S_ij + z (M - m) + z (B - m) + z m = sum_{pairs} (S_ij - z) + z N,
 * so the optimum is a maximum-weight partial matching with gains g_ij = S_ij - z (pairs of non-positive
 * gain are never needed).  Solved as an assignment problem on the clipped gains max(g_ij, 0): the smaller
 * side is assigned, one by one, along shortest augmenting paths with dual potentials (the Hungarian
 * method, O(n^2 m)); an assignment of clipped gain 0 means "unpaired".
 *
 * Outputs: match_prop[j] = kept position paired with pruned token j, or -1; objective = the LP value
 * sum S-bar P-bar; dual_kept[M], dual_prop[B]: an optimal dual of the clipped assignment problem in
 * max form (dual_kept_i + dual_prop_j >= max(g_ij, 0), duals of the unassigned side >= 0, and their sum
 * equal to the clipped gain collected): a certificate of optimality a test can check by itself.
 * Returns the number of pairs.  Ties between optimal matchings are broken by the order of the search.
 */
int rtp_oracle_exact_matching(const double *S, int M, int B, double z, int32_t *match_prop,
                              double *objective, double *dual_kept, double *dual_prop)
{
    const int transposed = B > M;            /* rows of the assignment = the smaller side */
    const int n = transposed ? M : B, m = transposed ? B : M;
    /* cost[r][c] = -max(g, 0); 1-based arrays as in the classical formulation */
    double *u = (double *)calloc((size_t)n + 1, sizeof(double));
    double *v = (double *)calloc((size_t)m + 1, sizeof(double));
    double *minv = (double *)malloc(((size_t)m + 1) * sizeof(double));
    int *p = (int *)calloc((size_t)m + 1, sizeof(int));       /* p[c] = row assigned to column c (0: none) */
    int *way = (int *)calloc((size_t)m + 1, sizeof(int));
    char *used = (char *)malloc((size_t)m + 1);
#define RTP_GAIN(r, c)                                                                           \
    (transposed ? fmax(S[(size_t)((r) - 1) * B + ((c) - 1)] - z, 0.0)                            \
                : fmax(S[(size_t)((c) - 1) * B + ((r) - 1)] - z, 0.0))
    for (int i = 1; i <= n; ++i) {
        p[0] = i;
        int j0 = 0;
        for (int j = 0; j <= m; ++j) {
            minv[j] = INFINITY;
            used[j] = 0;
        }
        do {
            used[j0] = 1;
            const int i0 = p[j0];
            double delta = INFINITY;
            int j1 = 0;
            for (int j = 1; j <= m; ++j) {
                if (used[j]) continue;
                const double cur = -RTP_GAIN(i0, j) - u[i0] - v[j];
                if (cur < minv[j]) {
                    minv[j] = cur;
                    way[j] = j0;
                }
                if (minv[j] < delta) {
                    delta = minv[j];
                    j1 = j;
                }
            }
            for (int j = 0; j <= m; ++j) {
                if (used[j]) {
                    u[p[j]] += delta;
                    v[j] -= delta;
                } else {
                    minv[j] -= delta;
                }
            }
            j0 = j1;
        } while (p[j0] != 0);
        do {
            const int j1 = way[j0];
            p[j0] = p[j1];
            j0 = j1;
        } while (j0);
    }
    for (int j = 0; j < B; ++j) match_prop[j] = -1;
    int pairs = 0;
    double value = z * (double)(M + B);
    for (int c = 1; c <= m; ++c) {
        const int r = p[c];
        if (r == 0) continue;
        const int kept_i = transposed ? r - 1 : c - 1, prop_j = transposed ? c - 1 : r - 1;
        const double g = S[(size_t)kept_i * B + prop_j] - z;
        if (g > 0.0) {                       /* clipped gain 0: the two stay unpaired */
            match_prop[prop_j] = kept_i;
            value += g;
            ++pairs;
        }
    }
    *objective = value;
    if (dual_kept && dual_prop) {            /* max form: minus the potentials of the min-cost form */
        for (int r = 1; r <= n; ++r) (transposed ? dual_kept : dual_prop)[r - 1] = -u[r];
        for (int c = 1; c <= m; ++c) (transposed ? dual_prop : dual_kept)[c - 1] = -v[c];
    }
#undef RTP_GAIN
    free(u);
    free(v);
    free(minv);
    free(p);
    free(way);
    free(used);
    return pairs;
}

/*
 * Eq. 7 / Appendix C (merge equation): T_k^i <- T_k^i + alpha * sum_j P_ij T_p^j, with P the
 * non-dustbin block of P-bar (row stride B+1).  No renormalisation.  Y is M x D, rows in the order
 * of `kept`.
 */
void rtp_oracle_merge(const double *T, int D, const int32_t *kept, int M, const int32_t *prop,
                      int B, const double *Pbar, double alpha, double *Y)
{
    for (int i = 0; i < M; ++i) {
        const double *ti = T + (size_t)kept[i] * D;
        for (int c = 0; c < D; ++c) {
            double acc = 0.0;
            for (int j = 0; j < B; ++j)
                acc += Pbar[(size_t)i * (B + 1) + j] * T[(size_t)prop[j] * D + c];
            Y[(size_t)i * D + c] = ti[c] + alpha * acc;
        }
    }
}

/*
 * Discrete "merge pairs" (not in the paper, which only has the dense plan): proposed token j is
 * paired with the kept token that receives most of its mass, argmax_i P_ij (lower i on ties), and
 * the pair's weight is P at that cell.  gap[j] = the difference between the largest and the
 * second-largest log P_ij over i (infinity if M == 1), which tells a comparison how decisive the
 * argmax is.
 */
void rtp_oracle_partners(const double *Pbar, int M, int B, int32_t *partner, double *weight,
                         double *gap)
{
    for (int j = 0; j < B; ++j) {
        int best = 0;
        double pbest = Pbar[j], psecond = -1.0;
        for (int i = 1; i < M; ++i) {
            double p = Pbar[(size_t)i * (B + 1) + j];
            if (p > pbest) {
                psecond = pbest;
                pbest = p;
                best = i;
            } else if (p > psecond) {
                psecond = p;
            }
        }
        partner[j] = best;
        weight[j] = pbest;
        gap[j] = (psecond > 0.0) ? log(pbest) - log(psecond) : HUGE_VAL;
    }
}

/*
 * Algorithm 1 for one image: ratio (optional) -> stage 1 -> stage 2 -> merged kept tokens.
 *   T [N x D] fp64 (the exact input values), rho the caller's textual density.
 * Outputs (caller-allocated at worst-case size):
 *   C[N]; stats[4] = {phi, rho, r, M}; kept[N], prop[N] (first M / B entries valid, image-local,
 *   ascending); partner[N], weight[N], gap[N] (first B valid); Y[N x D] (first M rows valid);
 *   optional (may be NULL) u[N+1], v[N+1], Pbar[(M+1)(B+1)] -- Pbar needs (N/2+1)^2 doubles at most.
 * With B == 0 stage 2 is skipped and Y is the input, unchanged.  phi is evaluated in dynamic mode
 * only when compute_phi is zero, else always.  criterion: 0 ranks by the l2 norm (Eq. 1), 1 by
 * the variance, 2 by the entropy (see rtp_oracle_variance / rtp_oracle_entropy); C always
 * returns the l2 norms, which the cosines use whatever the ranking.
 * Returns M.
 */
int rtp_oracle_image(const double *T, int N, int D, double rho, int dynamic, double r_fixed,
                     double phi_lo, double phi_hi, double r_max, double z, double alpha,
                     double eps, int iters, int compute_phi, int criterion, double *C, double *stats,
                     int32_t *kept, int32_t *prop, int32_t *partner, double *weight, double *gap,
                     double *Y, double *u_out, double *v_out, double *Pbar_out)
{
    rtp_oracle_norms(T, N, D, C);
    double phi = 0.0;
    if (dynamic || compute_phi)
        phi = rtp_oracle_phi(T, C, N, D);
    double r;
    int B, M;
    rtp_oracle_ratio(phi, rho, dynamic, r_fixed, phi_lo, phi_hi, r_max, N, &r, &B, &M);
    stats[0] = phi;
    stats[1] = rho;
    stats[2] = r;
    stats[3] = (double)M;
    if (criterion == 0) {
        rtp_oracle_select(C, N, M, kept, prop);
    } else {
        double *Calt = (double *)malloc(sizeof(double) * (size_t)N);
        if (criterion == 1) rtp_oracle_variance(T, N, D, Calt);
        else rtp_oracle_entropy(T, N, D, Calt);
        rtp_oracle_select(Calt, N, M, kept, prop);
        free(Calt);
    }
    if (B == 0) {
        for (int i = 0; i < M; ++i)
            memcpy(Y + (size_t)i * D, T + (size_t)kept[i] * D, sizeof(double) * (size_t)D);
        return M;
    }
    double *S = (double *)malloc(sizeof(double) * (size_t)M * B);
    double *u = (double *)malloc(sizeof(double) * (size_t)(M + 1));
    double *v = (double *)malloc(sizeof(double) * (size_t)(B + 1));
    double *Pbar = (double *)malloc(sizeof(double) * (size_t)(M + 1) * (B + 1));
    rtp_oracle_scores(T, C, D, kept, M, prop, B, S);
    rtp_oracle_sinkhorn(S, M, B, z, eps, iters, u, v, Pbar);
    rtp_oracle_merge(T, D, kept, M, prop, B, Pbar, alpha, Y);
    rtp_oracle_partners(Pbar, M, B, partner, weight, gap);
    if (u_out) memcpy(u_out, u, sizeof(double) * (size_t)(M + 1));
    if (v_out) memcpy(v_out, v, sizeof(double) * (size_t)(B + 1));
    if (Pbar_out) memcpy(Pbar_out, Pbar, sizeof(double) * (size_t)(M + 1) * (B + 1));
    free(Pbar);
    free(v);
    free(u);
    free(S);
    return M;
}
