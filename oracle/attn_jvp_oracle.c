/*
 * attn_jvp_oracle.c -- TEST INFRASTRUCTURE, not part of the product path.
 *
 * Plain fp64 CPU oracle for the forward-mode Jacobian-vector product (JVP) of
 * non-causal softmax attention (Appendix C.1, "FlashAttention-2 JVP").
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference
 * leg may build, load or call this file.  It shares no code with the CUDA path.
 *
 * Two independent routes to the same numbers live here:
 *
 *   attn_jvp_def_*   the definition written out row by row (the unnumbered
 *                    equations of Appendix C.1: S, P = softmax(S), O = P V,
 *                    tS = tQ K^T + Q tK^T, tP = P.tS - P.(rowsum(P.tS) 1 1^T),
 *                    tO = tP V + P tV), two passes over one row of scores.
 *
 *   attn_jvp_fold_*  the same quantities reached block by block: the definition
 *                    on each block of B_c keys, the block results folded into a
 *                    running (O, tO, LSE, mu) with the chunk-merge identity that
 *                    follows from the aggregated form of Appendix C.1.  It pins
 *                    the streaming property (any block size gives the result of
 *                    the definition) without restating the paper's listing.
 *
 * Readings where the paper is silent:
 *   - the paper writes S = Q K^T with no softmax scale; here S = s Q K^T and
 *     tS = s (tQ K^T + Q tK^T) with a constant s ("scale");
 *   - L (the log-sum-exp) is the natural log of sum_j exp(S_ij);
 *   - the (P.tS) 1 1^T term is the per-row scalar mu_i = sum_j P_ij tS_ij
 *     broadcast along the row; mu is returned as an extra output because
 *     d(LSE_i) = mu_i, which gives a second finite-difference pin.
 *
 * Pins (tests/, "not gpu"): central finite differences of O and LSE, linearity
 * in the tangent, zero tangent, Lk = 1, Q = 0 closed form, constant-V,
 * hand-derived golden values, torch.func.jvp, and definition == block-fold on
 * brute-force tiny shapes.
 *
 * All matrices handed to the *_f64 entry points are dense row-major doubles:
 * Q,tQ [Lq][D]; K,tK,V,tV [Lk][D]; O,tO [Lq][D]; LSE,mu [Lq].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* One query row, by the definition.  s_buf and ts_buf hold Lk doubles each. */
static void def_row(const double *q, const double *tq,
                    const double *K, const double *tK,
                    const double *V, const double *tV,
                    long Lk, long D, long ldk, double scale,
                    double *o, double *to, double *lse, double *mu,
                    double *s_buf, double *ts_buf)
{
    /* S_ij = s * sum_d Q_id K_jd ;  tS_ij = s * sum_d (tQ_id K_jd + Q_id tK_jd) */
    double m = -INFINITY;
    for (long j = 0; j < Lk; ++j) {
        const double *kj = K + j * ldk;
        double s = 0.0, ts = 0.0;
        for (long d = 0; d < D; ++d) {
            s += q[d] * kj[d];
            ts += tq[d] * kj[d];
        }
        if (tK) {
            const double *tkj = tK + j * ldk;
            for (long d = 0; d < D; ++d) ts += q[d] * tkj[d];
        }
        s_buf[j] = scale * s;
        ts_buf[j] = scale * ts;
        if (s_buf[j] > m) m = s_buf[j];
    }
    /* P_ij = exp(S_ij - m_i) / sum_j exp(S_ij - m_i) */
    double denom = 0.0;
    for (long j = 0; j < Lk; ++j) {
        s_buf[j] = exp(s_buf[j] - m);
        denom += s_buf[j];
    }
    for (long j = 0; j < Lk; ++j) s_buf[j] /= denom;
    /* mu_i = sum_j P_ij tS_ij  (the rowsum(P.tS) term) */
    double mu_i = 0.0;
    for (long j = 0; j < Lk; ++j) mu_i += s_buf[j] * ts_buf[j];
    /* O_i = sum_j P_ij V_j ; tO_i = sum_j tP_ij V_j + sum_j P_ij tV_j,
       tP_ij = P_ij tS_ij - P_ij mu_i */
    for (long d = 0; d < D; ++d) { o[d] = 0.0; to[d] = 0.0; }
    for (long j = 0; j < Lk; ++j) {
        const double p = s_buf[j];
        const double tp = p * ts_buf[j] - p * mu_i;
        const double *vj = V + j * ldk;
        for (long d = 0; d < D; ++d) {
            o[d] += p * vj[d];
            to[d] += tp * vj[d];
        }
        if (tV) {
            const double *tvj = tV + j * ldk;
            for (long d = 0; d < D; ++d) to[d] += p * tvj[d];
        }
    }
    *lse = m + log(denom);
    *mu = mu_i;
}

/* Definition route, fp64 in / fp64 out.  tK and tV may be NULL (zero tangent). */
int attn_jvp_def_f64(const double *Q, const double *K, const double *V,
                     const double *tQ, const double *tK, const double *tV,
                     long Lq, long Lk, long D, double scale,
                     double *O, double *tO, double *LSE, double *MU)
{
    if (Lq < 1 || Lk < 1 || D < 1) return 1;
    int fail = 0;
#pragma omp parallel
    {
        double *s_buf = (double *)malloc(sizeof(double) * (size_t)Lk);
        double *ts_buf = (double *)malloc(sizeof(double) * (size_t)Lk);
        if (!s_buf || !ts_buf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 4)
            for (long i = 0; i < Lq; ++i)
                def_row(Q + i * D, tQ + i * D, K, tK, V, tV, Lk, D, D, scale,
                        O + i * D, tO + i * D, LSE + i, MU + i, s_buf, ts_buf);
        }
        free(s_buf);
        free(ts_buf);
    }
    return fail ? 2 : 0;
}

/* ------------------------------------------------------------------------- */
/*
 * Second route: the keys are cut into consecutive blocks of B_c; each block is
 * evaluated on its own by the definition above (softmax within the block), and
 * the block results are folded into a running result one after the other.
 *
 * Folding two disjoint key sets a and b, each normalised within itself: the
 * softmax weights over the union are P_j = w_a P^a_j on a and w_b P^b_j on b,
 * with w_x = exp(LSE_x - LSE) and LSE = log(exp(LSE_a) + exp(LSE_b)).  Putting
 * that into the aggregated form of Appendix C.1,
 *     tO = (P.tS) V + P tV - diag(mu) O,   mu = rowsum(P.tS),
 * and using (P^x.tS) V + P^x tV = tO_x + mu_x O_x on each set gives
 *     O  = w_a O_a + w_b O_b,        mu = w_a mu_a + w_b mu_b,
 *     tO = w_a (tO_a + mu_a O_a) + w_b (tO_b + mu_b O_b) - mu O.
 * In exact arithmetic this is what a single streaming pass over key blocks
 * (Algorithm 2) arrives at for any block size; only the order of the sums
 * differs from the definition.
 */
static void fold_row(const double *q, const double *tq,
                     const double *K, const double *tK,
                     const double *V, const double *tV,
                     long Lk, long D, long Bc, double scale,
                     double *o, double *to, double *lse, double *mu,
                     double *work /* 2*D + 2*Bc doubles */)
{
    double *o_b = work, *to_b = work + D;
    double *s_buf = work + 2 * D, *ts_buf = s_buf + Bc;
    for (long j0 = 0; j0 < Lk; j0 += Bc) {
        const long nb = (Lk - j0 < Bc) ? (Lk - j0) : Bc;
        double lse_b, mu_b;
        def_row(q, tq, K + j0 * D, tK ? tK + j0 * D : NULL, V + j0 * D, tV ? tV + j0 * D : NULL,
                nb, D, D, scale, o_b, to_b, &lse_b, &mu_b, s_buf, ts_buf);
        if (j0 == 0) {
            memcpy(o, o_b, sizeof(double) * (size_t)D);
            memcpy(to, to_b, sizeof(double) * (size_t)D);
            *lse = lse_b;
            *mu = mu_b;
            continue;
        }
        const double top = (*lse > lse_b) ? *lse : lse_b;
        const double lse_ab = top + log(exp(*lse - top) + exp(lse_b - top));
        const double w_a = exp(*lse - lse_ab), w_b = exp(lse_b - lse_ab);
        const double mu_a = *mu;
        const double mu_ab = w_a * mu_a + w_b * mu_b;
        for (long d = 0; d < D; ++d) {
            const double o_ab = w_a * o[d] + w_b * o_b[d];
            to[d] = w_a * (to[d] + mu_a * o[d]) + w_b * (to_b[d] + mu_b * o_b[d]) - mu_ab * o_ab;
            o[d] = o_ab;
        }
        *lse = lse_ab;
        *mu = mu_ab;
    }
}

int attn_jvp_fold_f64(const double *Q, const double *K, const double *V,
                      const double *tQ, const double *tK, const double *tV,
                      long Lq, long Lk, long D, long Bc, double scale,
                      double *O, double *tO, double *LSE, double *MU)
{
    if (Lq < 1 || Lk < 1 || D < 1 || Bc < 1) return 1;
    int fail = 0;
#pragma omp parallel
    {
        double *work = (double *)malloc(sizeof(double) * (size_t)(2 * D + 2 * Bc));
        if (!work) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 4)
            for (long i = 0; i < Lq; ++i)
                fold_row(Q + i * D, tQ + i * D, K, tK, V, tV, Lk, D, Bc, scale,
                         O + i * D, tO + i * D, LSE + i, MU + i, work);
        }
        free(work);
    }
    return fail ? 2 : 0;
}

/* ------------------------------------------------------------------------- */
/* bf16 bit patterns, [B][L][H][D] ("BLHD") layout, selected rows.           */

static double bf16_to_f64(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16; /* bf16 is the top half of an fp32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Widen one head's [L][D] slice out of a BLHD bf16 tensor. */
static void widen_head(const uint16_t *x, long b, long h, long L, long H, long D, double *dst)
{
    for (long l = 0; l < L; ++l) {
        const uint16_t *src = x + ((b * L + l) * H + h) * D;
        for (long d = 0; d < D; ++d) dst[l * D + d] = bf16_to_f64(src[d]);
    }
}

/*
 * Definition route on bf16 BLHD inputs for a list of query rows.
 * rows[n] is a flat index (b*H + h)*Lq + i, sorted so that equal (b,h) are
 * adjacent (the head's K/V are widened once per run of equal heads).
 * Outputs: O,tO [nrows][D]; LSE,MU [nrows] in fp64.
 * tk / tv may be NULL (cross-attention with a constant context: tK = tV = 0).
 */
int attn_jvp_def_bf16_blhd_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                const uint16_t *tq, const uint16_t *tk, const uint16_t *tv,
                                long B, long H, long Lq, long Lk, long D, double scale,
                                const int64_t *rows, long nrows,
                                double *O, double *tO, double *LSE, double *MU)
{
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1 || D < 1 || nrows < 0) return 1;
    const size_t kv = (size_t)Lk * (size_t)D;
    double *Kd = (double *)malloc(sizeof(double) * kv);
    double *Vd = (double *)malloc(sizeof(double) * kv);
    double *tKd = tk ? (double *)malloc(sizeof(double) * kv) : NULL;
    double *tVd = tv ? (double *)malloc(sizeof(double) * kv) : NULL;
    int rc = 0;
    if (!Kd || !Vd || (tk && !tKd) || (tv && !tVd)) rc = 2;

    long n0 = 0;
    while (rc == 0 && n0 < nrows) {
        const long bh = (long)(rows[n0] / Lq);
        long n1 = n0;
        while (n1 < nrows && (long)(rows[n1] / Lq) == bh) ++n1;
        if (bh < 0 || bh >= B * H) { rc = 3; break; }
        const long b = bh / H, h = bh % H;
        widen_head(k, b, h, Lk, H, D, Kd);
        widen_head(v, b, h, Lk, H, D, Vd);
        if (tk) widen_head(tk, b, h, Lk, H, D, tKd);
        if (tv) widen_head(tv, b, h, Lk, H, D, tVd);
#pragma omp parallel
        {
            double *s_buf = (double *)malloc(sizeof(double) * (size_t)Lk);
            double *ts_buf = (double *)malloc(sizeof(double) * (size_t)Lk);
            double *qd = (double *)malloc(sizeof(double) * (size_t)D * 2);
            if (!s_buf || !ts_buf || !qd) {
#pragma omp atomic write
                rc = 2;
            }
#pragma omp barrier
            if (rc == 0) {
#pragma omp for schedule(dynamic, 4)
                for (long n = n0; n < n1; ++n) {
                    const long i = (long)(rows[n] % Lq);
                    const uint16_t *qs = q + ((b * Lq + i) * H + h) * D;
                    const uint16_t *tqs = tq + ((b * Lq + i) * H + h) * D;
                    for (long d = 0; d < D; ++d) {
                        qd[d] = bf16_to_f64(qs[d]);
                        qd[D + d] = bf16_to_f64(tqs[d]);
                    }
                    def_row(qd, qd + D, Kd, tKd, Vd, tVd, Lk, D, D, scale,
                            O + n * D, tO + n * D, LSE + n, MU + n, s_buf, ts_buf);
                }
            }
            free(s_buf); free(ts_buf); free(qd);
        }
        n0 = n1;
    }
    free(Kd); free(Vd); free(tKd); free(tVd);
    return rc;
}

int attn_jvp_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/*
 * RMS normalisation over the last dimension and its forward-mode tangent (the QK normalisation of the DiT
 * attention block, Sec. 3.1, in the JVP-mode layer form of Appendix C.2), written out from the definition:
 *     n = sqrt(mean_d x_d^2 + eps),  y_d = w_d x_d / n,
 *     ty_d = d/d(eps') y_d(x + eps' tx) at 0 = w_d (tx_d / n - x_d (sum_e x_e tx_e) / (D n^3)).
 * x, tx, y, ty: [rows][D] doubles; w: [D].  tx / ty may be NULL.
 */
int rmsnorm_jvp_f64(const double *x, const double *tx, const double *w, long rows, long D, double eps,
                    double *y, double *ty)
{
    if (rows < 1 || D < 1) return 1;
    for (long r = 0; r < rows; ++r) {
        const double *xr = x + r * D;
        double ss = 0.0;
        for (long d = 0; d < D; ++d) ss += xr[d] * xr[d];
        const double n = sqrt(ss / (double)D + eps);
        for (long d = 0; d < D; ++d) y[r * D + d] = w[d] * xr[d] / n;
        if (tx && ty) {
            const double *tr = tx + r * D;
            double dot = 0.0;
            for (long d = 0; d < D; ++d) dot += xr[d] * tr[d];
            /* dn = dot / (D n) ; d(x/n) = tx/n - x dn / n^2 */
            const double dn = dot / ((double)D * n);
            for (long d = 0; d < D; ++d) ty[r * D + d] = w[d] * (tr[d] / n - xr[d] * dn / (n * n));
        }
    }
    return 0;
}
