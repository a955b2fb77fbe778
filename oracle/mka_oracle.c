/*
 * CPU oracle for the FastMKA / MKA attention operator -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, obviously-correct fp64 C written from the paper's definitions.
 * It shares no code with the CUDA library and must never be linked, imported or
 * called by the product path: only the tests, the smoke check and the
 * benchmark's cpu-baseline leg may use it.
 *
 * What each routine restates:
 *   orc_router          Alg. 1 step "lambda <- softmax(MLP(q))" / Alg. 2 step 5, with the
 *                       router read as one linear layer; hard top-1 / top-2 and fixed 1/3
 *                       gates are the routing-ablation variants (Table 10).
 *   orc_visible         which rows of a level a query may see: L1 = causal window
 *                       (Motivation, "L1: local cache for current window tokens"), L2 = causal
 *                       prefix ("causal L2 summary", Alg. 1 steps 5-7), L3 = every recalled slot.
 *   orc_fwd_fast_head   Eq. 5, the gated mixture of exponentiated scores with ONE
 *                       normalisation, evaluated directly (three nested loops, one global
 *                       row maximum for stability, scale tau as in Eq. 3).
 *   orc_fwd_full_head   Alg. 1 steps 14-20: one softmax attention per level, outputs mixed by
 *                       the gate.
 *   orc_fwd_recursive_head  Eq. 6-8 accumulated level by level with the max shift of
 *                       Eq. 11-14, each level scanned in key blocks as in Alg. 3 (with the
 *                       rescale of Eq. 13-14, which Alg. 3 as printed leaves out).  Written
 *                       separately; used only to test Theorem 1 and block-wise == full.
 *   orc_bwd_head        gradients of <dO, O> for O of Eq. 5; derived by differentiating
 *                       Eq. 5 (the paper prints no backward).
 *   orc_sum_rows_f32, orc_srp_code, orc_l3_select   the L3 recall of Alg. 2 step 4 under the
 *                       sign-random-projection reading described above them (fp32 by definition,
 *                       because floating point decides the code bits).
 *
 * All arrays are row-major doubles.  One call handles one (batch, head) problem:
 *   Q[T][d], K_l[n_l][d], V_l[n_l][d], gate[T][3].
 * Parity: every routine here is pinned by the CPU tests (brute force, library softmax
 * attention, closed forms, finite differences); none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Rows [lo, hi) of level `level` (0,1,2) visible to the query at key-timeline position p.
 * decode != 0: every cached row is visible. */
void orc_visible(int level, int64_t p, int64_t W, int64_t n, int decode, int64_t *lo, int64_t *hi) {
    int64_t a = 0, b = n;
    if (!decode) {
        if (level == 0) {            /* W keys ending at and including position p */
            a = p - W + 1;
            b = p + 1;
        } else if (level == 1) {     /* causal prefix */
            a = 0;
            b = p + 1;
        }
        if (a < 0) a = 0;
        if (b > n) b = n;
    }
    if (b < a) b = a;
    *lo = a;
    *hi = b;
}

/* route: 0 soft, 1 uniform, 2 top-1, 3 top-2.  gate[rows][3]; idx[rows][2] (kept levels,
 * ascending; -1 = unused; all three kept in soft/uniform mode gives {-1,-1}). */
int orc_router(const double *R, const double *Wr, const double *br, int64_t rows, int64_t D, int route,
               double *gate, int8_t *idx) {
    if (route < 0 || route > 3) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double g[3], lam[3];
        for (int l = 0; l < 3; ++l) {
            double acc = br ? br[l] : 0.0;
            for (int64_t c = 0; c < D; ++c) acc += R[r * D + c] * Wr[c * 3 + l];
            g[l] = acc;
        }
        double mx = fmax(g[0], fmax(g[1], g[2]));
        double sum = 0.0;
        for (int l = 0; l < 3; ++l) { lam[l] = exp(g[l] - mx); sum += lam[l]; }
        for (int l = 0; l < 3; ++l) lam[l] /= sum;
        int8_t id0 = -1, id1 = -1;
        if (route == 1) {
            lam[0] = lam[1] = lam[2] = 1.0 / 3.0;
        } else if (route == 2 || route == 3) {
            int keep = route == 2 ? 1 : 2;
            int kept[3] = {0, 0, 0};
            for (int k = 0; k < keep; ++k) {        /* largest logit first; ties -> lower level */
                int best = -1;
                for (int l = 0; l < 3; ++l)
                    if (!kept[l] && (best < 0 || g[l] > g[best])) best = l;
                kept[best] = 1;
            }
            double ks = 0.0;
            for (int l = 0; l < 3; ++l) if (kept[l]) ks += lam[l];
            for (int l = 0; l < 3; ++l) lam[l] = kept[l] ? lam[l] / ks : 0.0;
            for (int l = 0; l < 3; ++l)
                if (kept[l]) { if (id0 < 0) id0 = (int8_t)l; else id1 = (int8_t)l; }
        }
        for (int l = 0; l < 3; ++l) gate[r * 3 + l] = lam[l];
        if (idx) { idx[r * 2] = id0; idx[r * 2 + 1] = id1; }
    }
    return 0;
}

static double dot(const double *a, const double *b, int64_t d) {
    double s = 0.0;
    for (int64_t c = 0; c < d; ++c) s += a[c] * b[c];
    return s;
}

/* Eq. 5 for the listed query rows (rows == NULL: all T rows, in order).
 * O[n_rows][d], lse[n_rows] = log of the gated partition sum (natural log). */
int orc_fwd_fast_head(const double *Q, int64_t T, int64_t d,
                      const double *K0, const double *V0, int64_t n0,
                      const double *K1, const double *V1, int64_t n1,
                      const double *K2, const double *V2, int64_t n2,
                      const double *gate, int64_t W, int64_t q_off, double tau, int decode,
                      const int64_t *rows, int64_t n_rows, double *O, double *lse) {
    const double *K[3] = {K0, K1, K2}, *V[3] = {V0, V1, V2};
    const int64_t n[3] = {n0, n1, n2};
    if (!rows) n_rows = T;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < n_rows; ++r) {
        int64_t t = rows ? rows[r] : r;
        const double *q = Q + t * d, *lam = gate + t * 3;
        int64_t lo[3], hi[3];
        for (int l = 0; l < 3; ++l) orc_visible(l, t + q_off, W, n[l], decode, &lo[l], &hi[l]);
        /* one global maximum over every visible score of a level with non-zero gate */
        double M = -INFINITY;
        for (int l = 0; l < 3; ++l) {
            if (!(lam[l] > 0.0)) continue;
            for (int64_t j = lo[l]; j < hi[l]; ++j) {
                double s = tau * dot(q, K[l] + j * d, d);
                if (s > M) M = s;
            }
        }
        double *o = O + r * d;
        for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
        double Z = 0.0;
        if (M == -INFINITY) { lse[r] = -INFINITY; continue; }
        for (int l = 0; l < 3; ++l) {
            if (!(lam[l] > 0.0)) continue;
            for (int64_t j = lo[l]; j < hi[l]; ++j) {
                double e = lam[l] * exp(tau * dot(q, K[l] + j * d, d) - M);
                Z += e;
                const double *v = V[l] + j * d;
                for (int64_t c = 0; c < d; ++c) o[c] += e * v[c];
            }
        }
        for (int64_t c = 0; c < d; ++c) o[c] /= Z;
        lse[r] = M + log(Z);
    }
    return 0;
}

/* Alg. 1: a_l = softmax(q k_l^T) v_l on each level's visible rows (0 if none), O = sum_l lambda_l a_l. */
int orc_fwd_full_head(const double *Q, int64_t T, int64_t d,
                      const double *K0, const double *V0, int64_t n0,
                      const double *K1, const double *V1, int64_t n1,
                      const double *K2, const double *V2, int64_t n2,
                      const double *gate, int64_t W, int64_t q_off, double tau, int decode,
                      const int64_t *rows, int64_t n_rows, double *O) {
    const double *K[3] = {K0, K1, K2}, *V[3] = {V0, V1, V2};
    const int64_t n[3] = {n0, n1, n2};
    if (!rows) n_rows = T;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < n_rows; ++r) {
        int64_t t = rows ? rows[r] : r;
        const double *q = Q + t * d, *lam = gate + t * 3;
        double *o = O + r * d;
        double *a = (double *)malloc(sizeof(double) * (size_t)d);
        for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
        for (int l = 0; l < 3; ++l) {
            int64_t lo, hi;
            orc_visible(l, t + q_off, W, n[l], decode, &lo, &hi);
            if (hi <= lo) continue;
            double m = -INFINITY;
            for (int64_t j = lo; j < hi; ++j) m = fmax(m, tau * dot(q, K[l] + j * d, d));
            double z = 0.0;
            for (int64_t c = 0; c < d; ++c) a[c] = 0.0;
            for (int64_t j = lo; j < hi; ++j) {
                double e = exp(tau * dot(q, K[l] + j * d, d) - m);
                z += e;
                for (int64_t c = 0; c < d; ++c) a[c] += e * V[l][j * d + c];
            }
            for (int64_t c = 0; c < d; ++c) o[c] += lam[l] * a[c] / z;
        }
        free(a);
    }
    return 0;
}

/* Eq. 6-8 with the max shift of Eq. 11-14, level by level, each level scanned in key blocks
 * of `block` rows (the inner loop of Alg. 3 with the missing rescale put back).  The running
 * maximum mu is taken over raw scores, as Eq. 11 writes it. */
int orc_fwd_recursive_head(const double *Q, int64_t T, int64_t d,
                           const double *K0, const double *V0, int64_t n0,
                           const double *K1, const double *V1, int64_t n1,
                           const double *K2, const double *V2, int64_t n2,
                           const double *gate, int64_t W, int64_t q_off, double tau, int decode,
                           int64_t block, double *O, double *lse) {
    const double *K[3] = {K0, K1, K2}, *V[3] = {V0, V1, V2};
    const int64_t n[3] = {n0, n1, n2};
    if (block < 1) return 1;
    for (int64_t t = 0; t < T; ++t) {
        const double *q = Q + t * d, *lam = gate + t * 3;
        double mu = -INFINITY, z = 0.0;
        double *alpha = O + t * d;
        for (int64_t c = 0; c < d; ++c) alpha[c] = 0.0;
        for (int l = 0; l < 3; ++l) {
            int64_t lo, hi;
            orc_visible(l, t + q_off, W, n[l], decode, &lo, &hi);
            if (!(lam[l] > 0.0)) continue;
            for (int64_t j0 = lo; j0 < hi; j0 += block) {
                int64_t j1 = j0 + block < hi ? j0 + block : hi;
                double bm = -INFINITY;
                for (int64_t j = j0; j < j1; ++j) bm = fmax(bm, tau * dot(q, K[l] + j * d, d));
                double mu_new = fmax(mu, bm);
                double resc = (mu == -INFINITY) ? 0.0 : exp(mu - mu_new);
                z *= resc;
                for (int64_t c = 0; c < d; ++c) alpha[c] *= resc;
                for (int64_t j = j0; j < j1; ++j) {
                    double s = exp(tau * dot(q, K[l] + j * d, d) - mu_new);
                    z += lam[l] * s;
                    for (int64_t c = 0; c < d; ++c) alpha[c] += lam[l] * s * V[l][j * d + c];
                }
                mu = mu_new;
            }
        }
        if (z > 0.0) {
            for (int64_t c = 0; c < d; ++c) alpha[c] /= z;
            lse[t] = mu + log(z);
        } else {
            lse[t] = -INFINITY;
        }
    }
    return 0;
}

/*
 * Backward of Eq. 5 for one head.  With p_{t,l,j} = lambda_{t,l} exp(s_{t,l,j} - LSE_t) on the
 * visible set (s = tau q.k), and D_t = dO_t . O_t:
 *   dV_{l,j} = sum_t p dO_t            dP = dO_t . v_{l,j}          dS = p (dP - D_t)
 *   dQ_t = tau sum_{l,j} dS k_{l,j}    dK_{l,j} = tau sum_t dS q_t  G_{t,l} = sum_j dS_{t,l,j}
 * G is this head's gradient with respect to the router logit of level l (the softmax Jacobian
 * reduces to the identity here because sum_l G_{t,l} = 0).  O and LSE are recomputed in fp64
 * from the inputs, not taken from the caller.
 * rows == NULL: all rows, and dK/dV (may be NULL to skip) are complete.  With a row list only
 * dQ[n_rows][d] and G[n_rows][3] are meaningful; dK/dV then hold the listed rows' share.
 */
int orc_bwd_head(const double *Q, int64_t T, int64_t d,
                 const double *K0, const double *V0, int64_t n0,
                 const double *K1, const double *V1, int64_t n1,
                 const double *K2, const double *V2, int64_t n2,
                 const double *gate, int64_t W, int64_t q_off, double tau, int decode,
                 const double *dO, const int64_t *rows, int64_t n_rows,
                 double *dQ, double *dK0, double *dV0, double *dK1, double *dV1, double *dK2, double *dV2,
                 double *G) {
    const double *K[3] = {K0, K1, K2}, *V[3] = {V0, V1, V2};
    double *dK[3] = {dK0, dK1, dK2}, *dV[3] = {dV0, dV1, dV2};
    const int64_t n[3] = {n0, n1, n2};
    if (!rows) n_rows = T;
    for (int l = 0; l < 3; ++l) {
        if (dK[l]) memset(dK[l], 0, sizeof(double) * (size_t)(n[l] * d));
        if (dV[l]) memset(dV[l], 0, sizeof(double) * (size_t)(n[l] * d));
    }
    int nthreads = orc_num_threads();
    /* per-thread dK/dV accumulators keep the parallel loop free of races */
    double **tK = NULL, **tV = NULL;
    int want_kv = 0;
    for (int l = 0; l < 3; ++l) if (dK[l] || dV[l]) want_kv = 1;
    if (want_kv) {
        tK = (double **)calloc((size_t)nthreads * 3, sizeof(double *));
        tV = (double **)calloc((size_t)nthreads * 3, sizeof(double *));
        for (int th = 0; th < nthreads; ++th)
            for (int l = 0; l < 3; ++l) {
                tK[th * 3 + l] = (double *)calloc((size_t)(n[l] * d) + 1, sizeof(double));
                tV[th * 3 + l] = (double *)calloc((size_t)(n[l] * d) + 1, sizeof(double));
            }
    }
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < n_rows; ++r) {
#ifdef _OPENMP
        int th = omp_get_thread_num();
#else
        int th = 0;
#endif
        int64_t t = rows ? rows[r] : r;
        const double *q = Q + t * d, *lam = gate + t * 3, *go = dO + t * d;
        int64_t lo[3], hi[3];
        for (int l = 0; l < 3; ++l) orc_visible(l, t + q_off, W, n[l], decode, &lo[l], &hi[l]);
        double *dq = dQ + r * d;
        for (int64_t c = 0; c < d; ++c) dq[c] = 0.0;
        for (int l = 0; l < 3; ++l) G[r * 3 + l] = 0.0;
        /* forward for this row: M, Z, O */
        double M = -INFINITY;
        for (int l = 0; l < 3; ++l) {
            if (!(lam[l] > 0.0)) continue;
            for (int64_t j = lo[l]; j < hi[l]; ++j) M = fmax(M, tau * dot(q, K[l] + j * d, d));
        }
        if (M == -INFINITY) continue;
        double Z = 0.0;
        double *o = (double *)calloc((size_t)d, sizeof(double));
        for (int l = 0; l < 3; ++l) {
            if (!(lam[l] > 0.0)) continue;
            for (int64_t j = lo[l]; j < hi[l]; ++j) {
                double e = lam[l] * exp(tau * dot(q, K[l] + j * d, d) - M);
                Z += e;
                for (int64_t c = 0; c < d; ++c) o[c] += e * V[l][j * d + c];
            }
        }
        for (int64_t c = 0; c < d; ++c) o[c] /= Z;
        double Dt = dot(go, o, d);
        free(o);
        for (int l = 0; l < 3; ++l) {
            if (!(lam[l] > 0.0)) continue;
            for (int64_t j = lo[l]; j < hi[l]; ++j) {
                const double *k = K[l] + j * d, *v = V[l] + j * d;
                double p = lam[l] * exp(tau * dot(q, k, d) - M) / Z;
                double dP = dot(go, v, d);
                double dS = p * (dP - Dt);
                G[r * 3 + l] += dS;
                for (int64_t c = 0; c < d; ++c) dq[c] += tau * dS * k[c];
                if (want_kv) {
                    double *ak = tK[th * 3 + l] + j * d, *av = tV[th * 3 + l] + j * d;
                    for (int64_t c = 0; c < d; ++c) { ak[c] += tau * dS * q[c]; av[c] += p * go[c]; }
                }
            }
        }
    }
    if (want_kv) {
        for (int l = 0; l < 3; ++l)
            for (int th = 0; th < nthreads; ++th) {
                if (dK[l]) for (int64_t i = 0; i < n[l] * d; ++i) dK[l][i] += tK[th * 3 + l][i];
                if (dV[l]) for (int64_t i = 0; i < n[l] * d; ++i) dV[l][i] += tV[th * 3 + l][i];
            }
        for (int i = 0; i < nthreads * 3; ++i) { free(tK[i]); free(tV[i]); }
        free(tK); free(tV);
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * L3 recall (Alg. 2 step 4, "L3 <- Retrieve(Q_h)"; the method section's "vectorized hashing" with
 * "chunk-based recall"; R = 8 recalled chunks in the passkey table).  The paper names the mechanism
 * but not the hash, so this is a READING: every chunk of the long-term bank carries a
 * sign-random-projection code of the sum of its keys, the query carries the code of the sum of the
 * query heads that share the KV head, and the R chunks whose codes agree with the query's in the
 * most bits are recalled (ties go to the earlier chunk), listed in bank order.
 * The code bits are decided by fp32 arithmetic, so the order of that arithmetic is part of the
 * definition: sums run row by row in fp32, projections are one fmaf chain over the columns.
 */
#include <stdint.h>

/* s[i] = ((x[0][i] + x[1][i]) + x[2][i]) + ... in fp32 */
int orc_sum_rows_f32(const float *x, int64_t n, int64_t d, float *s) {
    for (int64_t i = 0; i < d; ++i) {
        float acc = 0.0f;
        for (int64_t r = 0; r < n; ++r) acc = acc + x[r * d + i];
        s[i] = acc;
    }
    return 0;
}

/* bit j of the code = [ fmaf(P[j][d-1], x[d-1], ... fmaf(P[j][0], x[0], 0)) >= 0 ]; bits is a multiple of 32 */
int orc_srp_code(const float *x, const float *proj, int64_t d, int64_t bits, uint32_t *code) {
    if (bits % 32) return 1;
    for (int64_t w = 0; w < bits / 32; ++w) code[w] = 0u;
    for (int64_t j = 0; j < bits; ++j) {
        float acc = 0.0f;
        for (int64_t i = 0; i < d; ++i) acc = fmaf(proj[j * d + i], x[i], acc);
        if (acc >= 0.0f) code[j / 32] |= 1u << (j % 32);
    }
    return 0;
}

/* The R entries of codes[n][words] closest to qcode in Hamming distance, ties to the lower index; their indices
 * ascending in out[0..*n_out), *n_out = min(R, n).  Selection by repeated scan, as plain as it gets. */
int orc_l3_select(const uint32_t *qcode, const uint32_t *codes, int64_t n, int64_t words, int64_t R, int64_t *out,
                  int64_t *n_out) {
    int64_t k = R < n ? R : n;
    char *taken = (char *)calloc((size_t)(n > 0 ? n : 1), 1);
    if (!taken) return 1;
    for (int64_t s = 0; s < k; ++s) {
        int64_t best = -1, best_dist = 0;
        for (int64_t c = 0; c < n; ++c) {
            if (taken[c]) continue;
            int64_t dist = 0;
            for (int64_t w = 0; w < words; ++w) {
                uint32_t x = qcode[w] ^ codes[c * words + w];
                while (x) { dist += x & 1u; x >>= 1; }
            }
            if (best < 0 || dist < best_dist) { best = c; best_dist = dist; }
        }
        taken[best] = 1;
    }
    int64_t m = 0;
    for (int64_t c = 0; c < n; ++c) if (taken[c]) out[m++] = c;
    *n_out = m;
    free(taken);
    return 0;
}
