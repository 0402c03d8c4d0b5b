/*
 * CPU oracle for the FLARE token mixer -- TEST INFRASTRUCTURE, not the product.
 *
 * Plain double-precision loops that write out the definitions of the paper:
 *   encode  z_m = sum_n softmax_n(s * q_m . k_n) v_n        (Section 3.2 encode equation;
 *                                                            per-latent form in the design-principles appendix)
 *   decode  y_n = sum_m softmax_m(s * k_n . q_m) z_m        (Section 3.2 decode equation;
 *                                                            per-token form in the same appendix)
 * with the score scale s = 1 in the paper (exposed here as `scale`).  Every score is recomputed from
 * q and k where it is needed, so memory stays O(M*D) per head and nothing is blocked, fused or reordered
 * beyond "for each row: max, sum of exponentials, weighted sum".
 *
 * Layouts: Q [H, M, D];  K, V, Y, dY, dK, dV [B, N, H, D];  Z, dZ [B, H, M, D];  lse_enc [B, H, M];
 * lse_dec [B, N, H];  key_mask [B, N] bytes (1 = valid, 0 = padding; may be NULL).
 *
 * Padding (the paper is silent; reading used by this build): a masked token takes no part in the encode
 * softmax (weight exactly 0).  Decode evaluates every token as written.  A batch item with no valid token
 * has Z = 0 and lse_enc = -inf.
 *
 * This file shares no code with the CUDA path.  OpenMP only parallelises independent rows; every sum runs
 * in index order inside one thread, so results do not depend on the thread count.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define IDX_Q(h, m) ((((size_t)(h)) * M + (m)) * D)
#define IDX_T(b, n, h) (((((size_t)(b)) * N + (n)) * H + (h)) * D)
#define IDX_Z(b, h, m) (((((size_t)(b)) * H + (h)) * M + (m)) * D)

static double dot(const double *a, const double *b, int D) {
    double s = 0.0;
    for (int d = 0; d < D; ++d) s += a[d] * b[d];
    return s;
}

/* Encode: Z[b,h,m,:] and lse_enc[b,h,m] = log sum_n exp(score) over valid tokens. */
void flare_oracle_encode(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                         const double *V, const uint8_t *key_mask, double *Z, double *lse_enc) {
#pragma omp parallel for collapse(3) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int m = 0; m < M; ++m) {
                const double *q = Q + IDX_Q(h, m);
                double *z = Z + IDX_Z(b, h, m);
                double smax = -INFINITY;
                for (int n = 0; n < N; ++n) {
                    if (key_mask && !key_mask[(size_t)b * N + n]) continue;
                    double s = scale * dot(q, K + IDX_T(b, n, h), D);
                    if (s > smax) smax = s;
                }
                for (int d = 0; d < D; ++d) z[d] = 0.0;
                if (smax == -INFINITY) { /* no valid token */
                    if (lse_enc) lse_enc[((size_t)b * H + h) * M + m] = -INFINITY;
                    continue;
                }
                double den = 0.0;
                for (int n = 0; n < N; ++n) {
                    if (key_mask && !key_mask[(size_t)b * N + n]) continue;
                    double e = exp(scale * dot(q, K + IDX_T(b, n, h), D) - smax);
                    den += e;
                    const double *v = V + IDX_T(b, n, h);
                    for (int d = 0; d < D; ++d) z[d] += e * v[d];
                }
                for (int d = 0; d < D; ++d) z[d] /= den;
                if (lse_enc) lse_enc[((size_t)b * H + h) * M + m] = smax + log(den);
            }
}

/* Decode rows n in [n0, n1) of every (b, h): Y[b,n,h,:] and lse_dec[b,n,h] = log sum_m exp(score). */
void flare_oracle_decode_range(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                               const double *Z, int n0, int n1, double *Y, double *lse_dec) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = n0; n < n1; ++n)
            for (int h = 0; h < H; ++h) {
                const double *k = K + IDX_T(b, n, h);
                double *y = Y + IDX_T(b, n, h);
                double smax = -INFINITY;
                for (int m = 0; m < M; ++m) {
                    double s = scale * dot(k, Q + IDX_Q(h, m), D);
                    if (s > smax) smax = s;
                }
                double den = 0.0;
                for (int d = 0; d < D; ++d) y[d] = 0.0;
                for (int m = 0; m < M; ++m) {
                    double e = exp(scale * dot(k, Q + IDX_Q(h, m), D) - smax);
                    den += e;
                    const double *z = Z + IDX_Z(b, h, m);
                    for (int d = 0; d < D; ++d) y[d] += e * z[d];
                }
                for (int d = 0; d < D; ++d) y[d] /= den;
                if (lse_dec) lse_dec[((size_t)b * N + n) * H + h] = smax + log(den);
            }
}

void flare_oracle_decode(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                         const double *Z, double *Y, double *lse_dec) {
    flare_oracle_decode_range(B, H, N, M, D, scale, Q, K, Z, 0, N, Y, lse_dec);
}

/* Decode a list of sampled token rows: rows[i] = b*N + n; outputs Y_rows [nrows, H, D]. */
void flare_oracle_decode_rows(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                              const double *Z, const int64_t *rows, int nrows, double *Y_rows) {
    (void)B;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < nrows; ++i) {
        int b = (int)(rows[i] / N), n = (int)(rows[i] % N);
        for (int h = 0; h < H; ++h) {
            const double *k = K + IDX_T(b, n, h);
            double *y = Y_rows + ((size_t)i * H + h) * D;
            double smax = -INFINITY;
            for (int m = 0; m < M; ++m) {
                double s = scale * dot(k, Q + IDX_Q(h, m), D);
                if (s > smax) smax = s;
            }
            double den = 0.0;
            for (int d = 0; d < D; ++d) y[d] = 0.0;
            for (int m = 0; m < M; ++m) {
                double e = exp(scale * dot(k, Q + IDX_Q(h, m), D) - smax);
                den += e;
                const double *z = Z + IDX_Z(b, h, m);
                for (int d = 0; d < D; ++d) y[d] += e * z[d];
            }
            for (int d = 0; d < D; ++d) y[d] /= den;
        }
    }
}

/* Whole mixer: encode, then decode. */
void flare_oracle_forward(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                          const double *V, const uint8_t *key_mask, double *Z, double *lse_enc, double *Y,
                          double *lse_dec) {
    flare_oracle_encode(B, H, N, M, D, scale, Q, K, V, key_mask, Z, lse_enc);
    flare_oracle_decode(B, H, N, M, D, scale, Q, K, Z, Y, lse_dec);
}

/*
 * The two projection matrices and the induced mixing matrix of one (b, h) (Section 3.2, "Low-rank
 * communication"):  W_enc [M, N] = row softmax of the scores, W_dec [N, M] = row softmax of the transposed
 * scores, W [N, N] = W_dec . W_enc.  Dense; for small N only.  Any output pointer may be NULL.
 */
void flare_oracle_mixing_matrices(int B, int H, int N, int M, int D, double scale, const double *Q,
                                  const double *K, const uint8_t *key_mask, int b, int h, double *W_enc,
                                  double *W_dec, double *W) {
    (void)B;
    double *we = (double *)malloc(sizeof(double) * (size_t)M * N);
    double *wd = (double *)malloc(sizeof(double) * (size_t)N * M);
    for (int m = 0; m < M; ++m) {
        double smax = -INFINITY, den = 0.0;
        for (int n = 0; n < N; ++n) {
            int valid = !(key_mask && !key_mask[(size_t)b * N + n]);
            double s = scale * dot(Q + IDX_Q(h, m), K + IDX_T(b, n, h), D);
            if (valid && s > smax) smax = s;
        }
        for (int n = 0; n < N; ++n) {
            int valid = !(key_mask && !key_mask[(size_t)b * N + n]);
            double e = valid ? exp(scale * dot(Q + IDX_Q(h, m), K + IDX_T(b, n, h), D) - smax) : 0.0;
            we[(size_t)m * N + n] = e;
            den += e;
        }
        for (int n = 0; n < N; ++n) we[(size_t)m * N + n] = den > 0.0 ? we[(size_t)m * N + n] / den : 0.0;
    }
    for (int n = 0; n < N; ++n) {
        double smax = -INFINITY, den = 0.0;
        for (int m = 0; m < M; ++m) {
            double s = scale * dot(K + IDX_T(b, n, h), Q + IDX_Q(h, m), D);
            if (s > smax) smax = s;
        }
        for (int m = 0; m < M; ++m) {
            double e = exp(scale * dot(K + IDX_T(b, n, h), Q + IDX_Q(h, m), D) - smax);
            wd[(size_t)n * M + m] = e;
            den += e;
        }
        for (int m = 0; m < M; ++m) wd[(size_t)n * M + m] /= den;
    }
    if (W)
        for (int i = 0; i < N; ++i)
            for (int j = 0; j < N; ++j) {
                double s = 0.0;
                for (int m = 0; m < M; ++m) s += wd[(size_t)i * M + m] * we[(size_t)m * N + j];
                W[(size_t)i * N + j] = s;
            }
    if (W_enc) memcpy(W_enc, we, sizeof(double) * (size_t)M * N);
    if (W_dec) memcpy(W_dec, wd, sizeof(double) * (size_t)N * M);
    free(we);
    free(wd);
}

/*
 * Backward of the mixer.  The paper only says that a backward pass is timed; these are the chain-rule
 * derivatives of the forward definition above, with W_enc and W_dec the two softmax matrices:
 *   delta_d[n] = dY_n . Y_n                 dZ_m = sum_n W_dec[n,m] dY_n
 *   dSd[m,n]   = W_dec[n,m] (dY_n . Z_m - delta_d[n])
 *   delta_e[m] = dZ_m . Z_m                 dV_n = sum_m W_enc[m,n] dZ_m
 *   dSe[m,n]   = W_enc[m,n] (dZ_m . V_n - delta_e[m])
 *   dS = dSd + dSe;   dQ[h,m] = scale * sum_b sum_n dS[m,n] K_n;   dK_n = scale * sum_m dS[m,n] Q_m.
 * Z, Y, lse_enc, lse_dec are recomputed here from the inputs (the oracle keeps no state).
 * Outputs: dQ [H, M, D] (summed over the batch), dK, dV [B, N, H, D]; dZ_out [B, H, M, D] may be NULL.
 */
static void backward_impl(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                          const double *V, const uint8_t *key_mask, const double *dY, const int64_t *rows,
                          int64_t nrows, double *dQ, double *dK, double *dV, double *dZ_out) {
    size_t nZ = (size_t)B * H * M * D, nT = (size_t)B * N * H * D;
    double *Z = (double *)malloc(sizeof(double) * nZ);
    double *dZ = (double *)calloc(nZ, sizeof(double));
    double *Y = (double *)malloc(sizeof(double) * nT);
    double *le = (double *)malloc(sizeof(double) * (size_t)B * H * M);
    double *ld = (double *)malloc(sizeof(double) * (size_t)B * N * H);
    double *dQb = (double *)calloc((size_t)B * H * M * D, sizeof(double)); /* per batch item, summed at the end */
    flare_oracle_forward(B, H, N, M, D, scale, Q, K, V, key_mask, Z, le, Y, ld);

    /* dZ: a reduction over tokens, one (b,h,m) row per task so each sum runs in token order */
#pragma omp parallel for collapse(3) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int m = 0; m < M; ++m) {
                double *dz = dZ + IDX_Z(b, h, m);
                for (int n = 0; n < N; ++n) {
                    double s = scale * dot(K + IDX_T(b, n, h), Q + IDX_Q(h, m), D);
                    double wdec = exp(s - ld[((size_t)b * N + n) * H + h]);
                    const double *dy = dY + IDX_T(b, n, h);
                    for (int d = 0; d < D; ++d) dz[d] += wdec * dy[d];
                }
            }

    /* per token: dV_n, dK_n.  Token i of the list is rows[i] = b*N + n, or token i itself without a list; its
       gradient rows go to row i of dK and dV. */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t flat = rows ? rows[i] : i;
        int b = (int)(flat / N), n = (int)(flat % N);
        for (int h = 0; h < H; ++h) {
            const double *k = K + IDX_T(b, n, h), *v = V + IDX_T(b, n, h);
            const double *dy = dY + IDX_T(b, n, h), *y = Y + IDX_T(b, n, h);
            double *dk = dK + ((size_t)i * H + h) * D, *dv = dV + ((size_t)i * H + h) * D;
            int valid = !(key_mask && !key_mask[(size_t)b * N + n]);
            double delta_d = dot(dy, y, D);
            for (int d = 0; d < D; ++d) dk[d] = 0.0, dv[d] = 0.0;
            for (int m = 0; m < M; ++m) {
                const double *q = Q + IDX_Q(h, m);
                const double *z = Z + IDX_Z(b, h, m), *dz = dZ + IDX_Z(b, h, m);
                double s = scale * dot(k, q, D);
                double wdec = exp(s - ld[((size_t)b * N + n) * H + h]);
                double lem = le[((size_t)b * H + h) * M + m];
                double wenc = (valid && lem != -INFINITY) ? exp(s - lem) : 0.0;
                double dS = wdec * (dot(dy, z, D) - delta_d) + wenc * (dot(dz, v, D) - dot(dz, z, D));
                for (int d = 0; d < D; ++d) {
                    dv[d] += wenc * dz[d];
                    dk[d] += scale * dS * q[d];
                }
            }
        }
    }

    /* dQ: a reduction over tokens per (b,h,m), then over the batch in index order */
#pragma omp parallel for collapse(3) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int m = 0; m < M; ++m) {
                const double *q = Q + IDX_Q(h, m);
                const double *z = Z + IDX_Z(b, h, m), *dz = dZ + IDX_Z(b, h, m);
                double lem = le[((size_t)b * H + h) * M + m];
                double delta_e = dot(dz, z, D);
                double *acc = dQb + IDX_Z(b, h, m);
                for (int n = 0; n < N; ++n) {
                    const double *k = K + IDX_T(b, n, h);
                    int valid = !(key_mask && !key_mask[(size_t)b * N + n]);
                    double s = scale * dot(k, q, D);
                    double wdec = exp(s - ld[((size_t)b * N + n) * H + h]);
                    double wenc = (valid && lem != -INFINITY) ? exp(s - lem) : 0.0;
                    const double *dy = dY + IDX_T(b, n, h);
                    double delta_d = dot(dy, Y + IDX_T(b, n, h), D);
                    double dS = wdec * (dot(dy, z, D) - delta_d) + wenc * (dot(dz, V + IDX_T(b, n, h), D) - delta_e);
                    for (int d = 0; d < D; ++d) acc[d] += scale * dS * k[d];
                }
            }
    for (size_t i = 0; i < (size_t)H * M * D; ++i) dQ[i] = 0.0;
    for (int b = 0; b < B; ++b)
        for (size_t i = 0; i < (size_t)H * M * D; ++i) dQ[i] += dQb[(size_t)b * H * M * D + i];
    if (dZ_out) memcpy(dZ_out, dZ, sizeof(double) * nZ);
    free(Z); free(dZ); free(Y); free(le); free(ld); free(dQb);
}

void flare_oracle_backward(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                           const double *V, const uint8_t *key_mask, const double *dY, double *dQ, double *dK,
                           double *dV, double *dZ_out) {
    backward_impl(B, H, N, M, D, scale, Q, K, V, key_mask, dY, NULL, (int64_t)B * N, dQ, dK, dV, dZ_out);
}

/*
 * The same backward with the per-token gradients evaluated only for a list of sampled tokens (rows[i] = b*N + n;
 * dK_rows, dV_rows [nrows, H, D]).  The reductions over all tokens (Z, Y, the log-sum-exp rows, dZ, dQ) still run
 * in full: a token's dK_n and dV_n depend on the other tokens only through them.  For problem sizes at which the
 * per-token loop over every token would dominate the run time.
 */
void flare_oracle_backward_rows(int B, int H, int N, int M, int D, double scale, const double *Q, const double *K,
                                const double *V, const uint8_t *key_mask, const double *dY, const int64_t *rows,
                                int nrows, double *dQ, double *dK_rows, double *dV_rows, double *dZ_out) {
    backward_impl(B, H, N, M, D, scale, Q, K, V, key_mask, dY, rows, nrows, dQ, dK_rows, dV_rows, dZ_out);
}

/*
 * Backward of the mixer with separate latent queries for the two stages (the "asymmetric" variant the paper's
 * design-principles appendix mentions and sets aside): encode scores q^e_m . k_n, decode scores k_n . q^d_m,
 *   Z = softmax(s Qe K^T) V,   Y = softmax(s K Qd^T) Z.
 * The chain rule as above, with each stage's weights and score gradient on its own queries:
 *   dSd[m,n] = W_dec[n,m] (dY_n . Z_m - dY_n . Y_n),      dSe[m,n] = W_enc[m,n] (dZ_m . V_n - dZ_m . Z_m),
 *   dQd_m = s sum_n dSd[m,n] K_n,   dQe_m = s sum_n dSe[m,n] K_n,   dK_n = s sum_m (dSd[m,n] Qd_m + dSe[m,n] Qe_m).
 * Outputs: dQe, dQd [H, M, D] (summed over the batch), dK, dV [B, N, H, D].  Dense loops; small cases.
 */
void flare_oracle_backward_asym(int B, int H, int N, int M, int D, double scale, const double *Qe, const double *Qd,
                                const double *K, const double *V, const uint8_t *key_mask, const double *dY, double *dQe,
                                double *dQd, double *dK, double *dV) {
    size_t nZ = (size_t)B * H * M * D, nT = (size_t)B * N * H * D;
    double *Z = (double *)malloc(sizeof(double) * nZ);
    double *dZ = (double *)calloc(nZ, sizeof(double));
    double *Y = (double *)malloc(sizeof(double) * nT);
    double *le = (double *)malloc(sizeof(double) * (size_t)B * H * M);
    double *ld = (double *)malloc(sizeof(double) * (size_t)B * N * H);
    flare_oracle_encode(B, H, N, M, D, scale, Qe, K, V, key_mask, Z, le);
    flare_oracle_decode(B, H, N, M, D, scale, Qd, K, Z, Y, ld);
    for (size_t i = 0; i < (size_t)H * M * D; ++i) dQe[i] = 0.0, dQd[i] = 0.0;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            for (int m = 0; m < M; ++m) {                       /* dZ_m = sum_n W_dec[n,m] dY_n */
                double *dz = dZ + IDX_Z(b, h, m);
                for (int n = 0; n < N; ++n) {
                    double wdec = exp(scale * dot(K + IDX_T(b, n, h), Qd + IDX_Q(h, m), D) - ld[((size_t)b * N + n) * H + h]);
                    for (int d = 0; d < D; ++d) dz[d] += wdec * dY[IDX_T(b, n, h) + d];
                }
            }
            for (int n = 0; n < N; ++n) {
                const double *k = K + IDX_T(b, n, h), *v = V + IDX_T(b, n, h), *dy = dY + IDX_T(b, n, h);
                double *dk = dK + IDX_T(b, n, h), *dv = dV + IDX_T(b, n, h);
                int valid = !(key_mask && !key_mask[(size_t)b * N + n]);
                double delta_d = dot(dy, Y + IDX_T(b, n, h), D);
                for (int d = 0; d < D; ++d) dk[d] = 0.0, dv[d] = 0.0;
                for (int m = 0; m < M; ++m) {
                    const double *qe = Qe + IDX_Q(h, m), *qd = Qd + IDX_Q(h, m);
                    const double *z = Z + IDX_Z(b, h, m), *dz = dZ + IDX_Z(b, h, m);
                    double lem = le[((size_t)b * H + h) * M + m];
                    double wdec = exp(scale * dot(k, qd, D) - ld[((size_t)b * N + n) * H + h]);
                    double wenc = (valid && lem != -INFINITY) ? exp(scale * dot(k, qe, D) - lem) : 0.0;
                    double dSd = wdec * (dot(dy, z, D) - delta_d);
                    double dSe = wenc * (dot(dz, v, D) - dot(dz, z, D));
                    for (int d = 0; d < D; ++d) {
                        dv[d] += wenc * dz[d];
                        dk[d] += scale * (dSd * qd[d] + dSe * qe[d]);
                        dQd[IDX_Q(h, m) + d] += scale * dSd * k[d];
                        dQe[IDX_Q(h, m) + d] += scale * dSe * k[d];
                    }
                }
            }
        }
    free(Z); free(dZ); free(Y); free(le); free(ld);
}

int flare_oracle_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
