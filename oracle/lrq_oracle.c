/*
 * CPU oracle for the LRQ-DiT quantized-linear path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of what the path computes, written from the
 * paper's equations and taken in the paper's order.  Nothing here is shared with the CUDA
 * library (no common header, table, helper or constant), and the product never calls it: only
 * the tests, the smoke check and the bench's CPU-baseline leg load this file.
 *
 * Rounding |.| -> nearest uses rint() in the default IEEE mode (ties to even); the paper
 * does not fix the tie rule.  OpenMP is used over tokens / output rows only: no blocking,
 * no fusion, no reordering of any sum.
 *
 * Parity pins: every function below is checked in the CPU test-suite against closed forms,
 * library routines, brute force or exact rational arithmetic.  The readings of the paper that
 * no pin can reach (they are choices, not consequences) are "parity unpinned": the merge of
 * the two zero codes into one table entry, the clipping grid values, the search objective,
 * the block-diagonal Hadamard for sizes that are not a power of two, the symmetric
 * activation mode, and the shape in which the dual transformation's factors are taken
 * (block-diagonal rotations of one block size around an index map).  The smoothing vector of orc_smooth (Sec. 5.1) is an input here: how it is
 * calibrated (migration strength 0.5) is outside the path, so only its application is pinned.
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

/* ------------------------------------------------------------------------------------------
 * Sec. 3.2, Eq. 3 (Sylvester construction).  H_2 = [[1,1],[1,-1]]/sqrt(2) and
 * H_{2^n} = H_2 (x) H_{2^{n-1}}, built literally by the Kronecker recursion.
 * H is n x n row-major, n a power of two.  Returns 0, or -1 if n is not a power of two.
 * ---------------------------------------------------------------------------------------- */
int orc_hadamard_matrix(int n, double *H) {
    if (n < 1 || (n & (n - 1))) return -1;
    H[0] = 1.0;
    /* grow in place: size m -> 2m, entries (i,j) of the m-block replicated with signs */
    for (int m = 1; m < n; m *= 2) {
        /* use stride n for the final matrix from the start */
        for (int i = m - 1; i >= 0; --i)
            for (int j = m - 1; j >= 0; --j) {
                double v = H[(size_t)i * n + j] * M_SQRT1_2;
                H[(size_t)i * n + j] = v;             /* H2[0][0] * block */
                H[(size_t)i * n + (j + m)] = v;       /* H2[0][1] * block */
                H[(size_t)(i + m) * n + j] = v;       /* H2[1][0] * block */
                H[(size_t)(i + m) * n + (j + m)] = -v; /* H2[1][1] * block */
            }
    }
    return 0;
}

/* Sec. 4.2, Eq. 12 (first case) with the block-diagonal reading for K not a power of two:
 * y[m, jB:(j+1)B] = x[m, jB:(j+1)B] . H_B, as an explicit matrix product with the matrix of
 * Eq. 3.  X, Y are [M,K] row-major. */
int orc_rotate_hadamard_explicit(const double *X, int M, int K, int B, double *Y) {
    if (B < 1 || (B & (B - 1)) || K % B) return -1;
    double *H = (double *)malloc(sizeof(double) * (size_t)B * B);
    if (!H) return -2;
    orc_hadamard_matrix(B, H);
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int j = 0; j < K / B; ++j) {
            const double *x = X + (size_t)m * K + (size_t)j * B;
            double *y = Y + (size_t)m * K + (size_t)j * B;
            for (int i = 0; i < B; ++i) {
                double acc = 0.0;
                for (int l = 0; l < B; ++l) acc += x[l] * H[(size_t)l * B + i];
                y[i] = acc;
            }
        }
    free(H);
    return 0;
}

/* The same map by the butterfly factorisation of Eq. 3 (fast Walsh-Hadamard transform,
 * natural order), normalised by 1/sqrt(B) at the end. */
int orc_rotate_hadamard_fwht(const double *X, int M, int K, int B, double *Y) {
    if (B < 1 || (B & (B - 1)) || K % B) return -1;
    const double nrm = 1.0 / sqrt((double)B);
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int j = 0; j < K / B; ++j) {
            const double *x = X + (size_t)m * K + (size_t)j * B;
            double *y = Y + (size_t)m * K + (size_t)j * B;
            for (int i = 0; i < B; ++i) y[i] = x[i];
            for (int h = 1; h < B; h *= 2)
                for (int i = 0; i < B; i += 2 * h)
                    for (int l = i; l < i + h; ++l) {
                        double a = y[l], b = y[l + h];
                        y[l] = a + b;
                        y[l + h] = a - b;
                    }
            for (int i = 0; i < B; ++i) y[i] *= nrm;
        }
    return 0;
}

/* Sec. 4.2, Eq. 12 (second case): y = x . R with R the composed K x K rotation, row-major,
 * y_i = sum_l x_l R[l,i]. */
int orc_rotate_dense(const double *X, int M, int K, const double *R, double *Y) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double *x = X + (size_t)m * K;
        double *y = Y + (size_t)m * K;
        for (int i = 0; i < K; ++i) y[i] = 0.0;
        for (int l = 0; l < K; ++l) {
            const double xl = x[l];
            const double *r = R + (size_t)l * K;
            for (int i = 0; i < K; ++i) y[i] += xl * r[i];   /* sum over l in increasing order */
        }
    }
    return 0;
}

/* Sec. 4.2, the dual transformation behind the second case of Eq. 12, kept in its factors:
 *   y = x . R1hat . P . R2hat
 * R1hat, R2hat block-diagonal with K/Bd orthogonal blocks of Bd x Bd (block j row-major at R[j*Bd*Bd],
 * acting on channels j*Bd .. j*Bd+Bd-1: u_{jBd+i} = sum_l x_{jBd+l} R[j][l][i]); P the channel
 * reordering, given as an index map: (u . P)_i = u_{perm[i]}, i.e. P[l][i] = 1 exactly when l = perm[i].
 * The three maps are applied one after the other, each sum over l in increasing order.
 * Returns -1 when Bd does not divide K or perm is not a permutation of 0..K-1. */
int orc_rotate_dual(const double *X, int M, int K, int Bd, const double *R1, const int32_t *perm,
                    const double *R2, double *Y) {
    if (Bd < 1 || K % Bd) return -1;
    {
        char *seen = (char *)calloc((size_t)K, 1);
        int bad = 0;
        for (int i = 0; i < K; ++i) {
            if (perm[i] < 0 || perm[i] >= K || seen[perm[i]]) { bad = 1; break; }
            seen[perm[i]] = 1;
        }
        free(seen);
        if (bad) return -1;
    }
#pragma omp parallel
    {
        double *u = (double *)malloc((size_t)K * sizeof(double));
        double *v = (double *)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int m = 0; m < M; ++m) {
            const double *x = X + (size_t)m * K;
            double *y = Y + (size_t)m * K;
            for (int j = 0; j < K / Bd; ++j) {             /* u = x . R1hat */
                const double *Rj = R1 + (size_t)j * Bd * Bd;
                for (int i = 0; i < Bd; ++i) {
                    double acc = 0.0;
                    for (int l = 0; l < Bd; ++l) acc += x[j * Bd + l] * Rj[(size_t)l * Bd + i];
                    u[j * Bd + i] = acc;
                }
            }
            for (int i = 0; i < K; ++i) v[i] = u[perm[i]]; /* v = u . P */
            for (int j = 0; j < K / Bd; ++j) {             /* y = v . R2hat */
                const double *Rj = R2 + (size_t)j * Bd * Bd;
                for (int i = 0; i < Bd; ++i) {
                    double acc = 0.0;
                    for (int l = 0; l < Bd; ++l) acc += v[j * Bd + l] * Rj[(size_t)l * Bd + i];
                    y[j * Bd + i] = acc;
                }
            }
        }
        free(u);
        free(v);
    }
    return 0;
}

static double clampd(double v, double lo, double hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* ------------------------------------------------------------------------------------------
 * Sec. 3.1, Eq. 1, applied per token (Sec. 5.1: per-token dynamic activation quantization).
 *   mode 0 (asymmetric, Eq. 1 literally): s = (max-min)/(2^b-1), z = rint(min/s),
 *           q = clamp(rint(y/s) - z, 0, 2^b-1).
 *   mode 1 (symmetric variant): s = max|y|/(2^(b-1)-1), z = -2^(b-1), same q formula.
 * A token whose range is empty (max == min, or all zeros in mode 1) takes s = 1.
 * Outputs: Q [M,K] int32 codes, S [M] scales, Z [M] zero-points.
 * ---------------------------------------------------------------------------------------- */
int orc_quantize_act(const double *Y, int M, int K, int bits, int mode, int32_t *Q, double *S, int32_t *Z) {
    if (bits < 1 || bits > 16) return -1;
    const double qmax = (double)((1 << bits) - 1);
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double *y = Y + (size_t)m * K;
        double s, z;
        if (mode == 0) {
            double mn = y[0], mx = y[0];
            for (int k = 1; k < K; ++k) { if (y[k] < mn) mn = y[k]; if (y[k] > mx) mx = y[k]; }
            s = (mx - mn) / qmax;
            if (!(s > 0.0)) s = 1.0;
            z = rint(mn / s);
        } else {
            double am = 0.0;
            for (int k = 0; k < K; ++k) { double a = fabs(y[k]); if (a > am) am = a; }
            s = am / (double)((1 << (bits - 1)) - 1);
            if (!(s > 0.0)) s = 1.0;
            z = -(double)(1 << (bits - 1));
        }
        S[m] = s;
        Z[m] = (int32_t)z;
        for (int k = 0; k < K; ++k)
            Q[(size_t)m * K + k] = (int32_t)clampd(rint(y[k] / s) - z, 0.0, qmax);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Sec. 4.1, Eqs. 8-9: value of the level with log-domain exponent e.
 *   f = floor(e), r = e - f, II = rint(2^r * 2^I), value = II * 2^(f-I).
 * I < 0 selects Eq. 7 itself: value = 2^e.
 * ---------------------------------------------------------------------------------------- */
double orc_level_value(double e, int I) {
    if (I < 0) return exp2(e);
    double f = floor(e);
    double r = e - f;
    double II = rint(exp2(r) * ldexp(1.0, I));
    return ldexp(II, (int)f - I);
}

/* One side (positive or negative part) of one group.  l[0..n) are log2|w| of the side's
 * elements, a[0..n) their magnitudes |w|.  nq = index of the highest code on this side
 * (2^(b-1)-1 on the positive side, 2^(b-1) on the negative side); it is also the denominator
 * of Eq. 6.  Searches the clipping factor over grid[0..ng) (Eq. 6), squared error of the
 * de-quantized magnitudes (Eq. 7 / Eqs. 8-9) in the linear domain, first minimum wins.
 * Returns s, z, the chosen factor, codes q[0..n), the smallest relative gap between the best
 * and the second-best candidate. */
typedef struct { double s, z, factor, best_err, second_err; int n_valid; } side_result;

static void side_codes(const double *l, int n, double s, double z, int nq, int *q) {
    for (int i = 0; i < n; ++i) q[i] = (int)clampd(rint(l[i] / s) - z, 0.0, (double)nq);
}

static side_result tlq_side(const double *l, const double *a, int n, int nq, int I,
                            const double *grid, int ng, int *q) {
    side_result R;
    R.s = 1.0; R.z = 0.0; R.factor = 1.0; R.best_err = INFINITY; R.second_err = INFINITY; R.n_valid = 0;
    if (n == 0) return R;
    double lmax = l[0], lmin = l[0];
    for (int i = 1; i < n; ++i) { if (l[i] > lmax) lmax = l[i]; if (l[i] < lmin) lmin = l[i]; }
    int *qt = (int *)malloc(sizeof(int) * (size_t)n);
    int found = 0;
    if (nq > 0) {
        for (int g = 0; g < ng; ++g) {
            double top = grid[g] * lmax, bot = lmin;
            if (!(top > bot)) continue;
            double s = (top - bot) / (double)nq;
            double z = rint(bot / s);
            side_codes(l, n, s, z, nq, qt);
            double err = 0.0;
            for (int i = 0; i < n; ++i) {
                double d = a[i] - orc_level_value(s * ((double)qt[i] + z), I);
                err += d * d;
            }
            R.n_valid++;
            if (err < R.best_err) {
                R.second_err = R.best_err;
                R.best_err = err; R.s = s; R.z = z; R.factor = grid[g];
                memcpy(q, qt, sizeof(int) * (size_t)n);
                found = 1;
            } else if (err < R.second_err) {
                R.second_err = err;
            }
        }
    }
    if (!found) {           /* no usable range: unit step anchored at the smallest element */
        R.s = 1.0; R.z = rint(lmin); R.factor = 1.0;
        side_codes(l, n, R.s, R.z, nq, q);
    }
    free(qt);
    return R;
}

/* ------------------------------------------------------------------------------------------
 * Sec. 4.1, Eqs. 4-9: twin-log quantization of W [N,K] (row-major), per output row n and per
 * group of G consecutive input channels (G = K: per output channel).
 *   positive side: codes 0..2^(b-1)-1, step (alpha*max - min)/(2^(b-1)-1)
 *   negative side: codes 0..2^(b-1),   step (beta*max - min)/2^(b-1)
 *   signed code c = q+ for w>0, -q- for w<0, 0 for w==0            (Eq. 5, last line)
 * The masks of Eq. 4 select: min/max and quantization of a side run over that side's elements.
 * Level table T[n,g,u], u = c + 2^(b-1) in 0..2^b-1:
 *   c > 0: +lev(s+(c+z+));  c < 0: -lev(s-(|c|+z-));  c = 0: +lev(s+ z+) (0 if no positive element).
 * Outputs: codes int8 [N,K] (signed c), levels double [N,K/G,2^b], meta double [N,K/G,6] =
 * (s+, z+, s-, z-, alpha, beta), wsum double [N] = sum_k T[c_nk], margin double [N,K/G] = smallest
 * relative gap (second-best)/(best) - 1 of the two searches (INF if fewer than two candidates).
 * ---------------------------------------------------------------------------------------- */
int orc_tlq_quantize(const double *W, int N, int K, int bits, int G, int I,
                     const double *alpha, int n_alpha, const double *beta, int n_beta,
                     int8_t *codes, double *levels, double *meta, double *wsum, double *margin) {
    if (bits < 2 || bits > 8) return -1;
    if (G <= 0) G = K;
    if (K % G) return -1;
    const int ngrp = K / G, half = 1 << (bits - 1), nlev = 1 << bits;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 4)
    for (int n = 0; n < N; ++n) {
        double *lp = (double *)malloc(sizeof(double) * (size_t)G * 4);
        int *qp = (int *)malloc(sizeof(int) * (size_t)G * 2);
        int *ip = (int *)malloc(sizeof(int) * (size_t)G * 2);
        double *ap = lp + G, *ln = lp + 2 * G, *an = lp + 3 * G;
        int *qn = qp + G, *in = ip + G;
        double ws = 0.0;
        for (int g = 0; g < ngrp; ++g) {
            const double *w = W + (size_t)n * K + (size_t)g * G;
            int8_t *c = codes + (size_t)n * K + (size_t)g * G;
            int np = 0, nn = 0;
            for (int k = 0; k < G; ++k) {
                if (w[k] > 0.0) { lp[np] = log2(w[k]); ap[np] = w[k]; ip[np++] = k; }
                else if (w[k] < 0.0) { ln[nn] = log2(-w[k]); an[nn] = -w[k]; in[nn++] = k; }
            }
            side_result P = tlq_side(lp, ap, np, half - 1, I, alpha, n_alpha, qp);
            side_result Q = tlq_side(ln, an, nn, half, I, beta, n_beta, qn);
            for (int k = 0; k < G; ++k) c[k] = 0;
            for (int i = 0; i < np; ++i) c[ip[i]] = (int8_t)qp[i];
            for (int i = 0; i < nn; ++i) c[in[i]] = (int8_t)(-qn[i]);
            double *T = levels + ((size_t)n * ngrp + g) * nlev;
            for (int u = 0; u < nlev; ++u) {
                int cc = u - half;
                if (cc > 0) T[u] = np ? orc_level_value(P.s * ((double)cc + P.z), I) : 0.0;
                else if (cc < 0) T[u] = nn ? -orc_level_value(Q.s * ((double)(-cc) + Q.z), I) : 0.0;
                else T[u] = np ? orc_level_value(P.s * P.z, I) : 0.0;
            }
            double *mt = meta + ((size_t)n * ngrp + g) * 6;
            mt[0] = P.s; mt[1] = P.z; mt[2] = Q.s; mt[3] = Q.z; mt[4] = P.factor; mt[5] = Q.factor;
            if (margin) {
                double mg = INFINITY;
                if (P.n_valid >= 2 && P.best_err > 0) { double v = P.second_err / P.best_err - 1.0; if (v < mg) mg = v; }
                if (Q.n_valid >= 2 && Q.best_err > 0) { double v = Q.second_err / Q.best_err - 1.0; if (v < mg) mg = v; }
                margin[(size_t)n * ngrp + g] = mg;
            }
            for (int k = 0; k < G; ++k) ws += T[(int)c[k] + half];
        }
        wsum[n] = ws;
        free(lp); free(qp); free(ip);
    }
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * Sec. 4.1, Eq. 10 evaluated exactly: Y = X_f . W_f^T with X_f = s (q + z) (Eq. 1) and W_f the
 * level table entries (Eq. 7 / Eqs. 8-9).
 *   acc[m,n] = sum_k q[m,k] * T[n, k/G, c[n,k]]
 *   y[m,n]   = s_m * (acc + z_m * sum_k T[n, k/G, c[n,k]]) * wscale_n + bias_n
 * wscale, bias may be NULL (1 and 0).  Y is [M,N] row-major double.
 * ---------------------------------------------------------------------------------------- */
int orc_qmatmul(const int32_t *Q, const double *S, const int32_t *Z, int M, int K,
                const int8_t *codes, const double *levels, int N, int G, int bits,
                const double *wscale, const double *bias, double *Y) {
    if (G <= 0) G = K;
    if (K % G) return -1;
    const int ngrp = K / G, half = 1 << (bits - 1), nlev = 1 << bits;
    /* de-quantized weights, one row at a time per thread */
#pragma omp parallel
    {
        double *wf = (double *)malloc(sizeof(double) * (size_t)K);
#pragma omp for schedule(static)
        for (int n = 0; n < N; ++n) {
            double tsum = 0.0;
            for (int k = 0; k < K; ++k) {
                wf[k] = levels[((size_t)n * ngrp + k / G) * nlev + ((int)codes[(size_t)n * K + k] + half)];
                tsum += wf[k];
            }
            for (int m = 0; m < M; ++m) {
                const int32_t *q = Q + (size_t)m * K;
                double acc = 0.0;
                for (int k = 0; k < K; ++k) acc += (double)q[k] * wf[k];
                double y = S[m] * (acc + (double)Z[m] * tsum);
                if (wscale) y *= wscale[n];
                if (bias) y += bias[n];
                Y[(size_t)m * N + n] = y;
            }
        }
        free(wf);
    }
    return 0;
}

/* De-quantized activations of Eq. 1, x_f = s (q + z): used by the tests only. */
int orc_dequantize_act(const int32_t *Q, const double *S, const int32_t *Z, int M, int K, double *Xf) {
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k)
            Xf[(size_t)m * K + k] = S[m] * ((double)Q[(size_t)m * K + k] + (double)Z[m]);
    return 0;
}


/* ------------------------------------------------------------------------------------------
 * Sec. 5.1 (smoothing, after SmoothQuant): activations are divided channel-wise by a smoothing
 * factor that the weights absorb, X' = X diag(p), W' = W diag(1/p), so that X' W'^T = X W^T.
 * p (length K) holds the multipliers 1/lambda_k applied to the activations.  Y = X diag(p).
 * ---------------------------------------------------------------------------------------- */
int orc_smooth(const double *X, int M, int K, const double *p, double *Y) {
    if (M <= 0 || K <= 0) return -1;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) Y[(size_t)m * K + k] = X[(size_t)m * K + k] * p[k];
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Sec. 4.2, Eq. 11: fluctuation metric of a layer's activations X (B x N x C values, here a
 * matrix of M = B*N tokens by K = C channels):  J = ||X||_F / sqrt(B N C).
 * Eq. 12: the layer takes the Hadamard rotation when J < Thr, the outlier-aware one otherwise.
 * Returns J; *kind gets 1 (Hadamard) or 2 (outlier-aware dense rotation).
 * ---------------------------------------------------------------------------------------- */
double orc_fluctuation_metric(const double *X, int M, int K, double thr, int *kind) {
    double ss = 0.0;
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) ss += X[(size_t)m * K + k] * X[(size_t)m * K + k];
    const double J = sqrt(ss) / sqrt((double)M * (double)K);
    if (kind) *kind = J < thr ? 1 : 2;
    return J;
}
