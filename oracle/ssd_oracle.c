/*
 * TEST INFRASTRUCTURE — fp64 CPU oracle for the SSD selective-scan layer.
 *
 * This file is the slow, plain definition that the CUDA library is checked against.
 * Only the test-suite, the smoke check and the bench's CPU-baseline leg may call it;
 * the product path never does.  It shares no code with the CUDA kernels.
 *
 * What it computes (Eq. 1 of the paper, specialised the way Mamba-2 uses it:
 * a scalar decay per head, the input scaled by the step size dt, and a skip term D):
 *
 *     h_t = exp(dt_t * A) * h_{t-1} + dt_t * x_t B_t^T          h_t in R^{P x N}
 *     y_t = C_t h_t + D * x_t
 *
 * one time step at a time, per (batch b, head h); head h reads the B/C vectors of
 * group g = h / (H/G).  The backward is the exact reverse-mode derivative of that
 * loop, run the way Algorithm 2 prescribes along the sequence axis: the forward
 * keeps only the state at the start of every block of `blk` steps (the S_ckpt of
 * Algorithm 1), the backward walks the blocks in reverse, recomputes the states of
 * one block from its checkpoint, back-propagates through it and hands the state
 * gradient to the block on its left.
 *
 * Layouts (row-major, innermost contiguous):
 *   x, y, dy, dx : [B, L, H, P]        dt, ddt : [B, L, H]
 *   Bm, Cm, dB, dC : [B, L, G, N]      A, D, dA, dD : [H]
 *   h0, h_final, dh_final, dh0 : [B, H, P, N]
 *   boundary : [B, nseg, H, P, N], boundary[:,k] = state entering segment k.
 *
 * Pins (tests/test_oracle_pins.py): linear-attention closed form for A=0, dt=1; the
 * H=P=N=1 hand case; the geometric-series case; the unrolled sum on tiny inputs;
 * central finite differences for all seven gradients; block-length invariance.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int ssd_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* one forward step of Eq. 1 on the P x N state `h` (in place). */
static void step_state(double *h, int P, int N, double alpha, double dtv,
                       const double *xt, const double *Bt) {
    for (int p = 0; p < P; ++p) {
        const double dx = dtv * xt[p];
        double *hp = h + (size_t)p * N;
        for (int n = 0; n < N; ++n) hp[n] = alpha * hp[n] + dx * Bt[n];
    }
}

/*
 * Forward.  seg > 0 with boundary != NULL also stores the state entering every
 * segment of `seg` steps (Algorithm 1, the sequence-axis checkpoint).
 * h0 == NULL means a zero initial state; h_final and boundary may be NULL.
 */
int ssd_oracle_fwd(int B, int L, int H, int P, int N, int G, int seg,
                   const double *x, const double *dt, const double *A,
                   const double *Bm, const double *Cm, const double *D,
                   const double *h0, double *y, double *h_final, double *boundary) {
    if (B <= 0 || L < 0 || H <= 0 || P <= 0 || N <= 0 || G <= 0 || H % G) return -1;
    const int hpg = H / G;
    const int nseg = (seg > 0) ? (L + seg - 1) / seg : 0;
    const size_t PN = (size_t)P * N;
    int fail = 0;
#pragma omp parallel for schedule(static)
    for (int bh = 0; bh < B * H; ++bh) {
        const int b = bh / H, hd = bh % H, g = hd / hpg;
        double *h = (double *)malloc(PN * sizeof(double));
        if (!h) { fail = 1; continue; }
        if (h0) memcpy(h, h0 + (size_t)bh * PN, PN * sizeof(double));
        else memset(h, 0, PN * sizeof(double));
        for (int t = 0; t < L; ++t) {
            if (boundary && seg > 0 && t % seg == 0)
                memcpy(boundary + (((size_t)b * nseg + t / seg) * H + hd) * PN, h, PN * sizeof(double));
            const size_t bt = (size_t)b * L + t;
            const double dtv = dt[bt * H + hd];
            const double alpha = exp(dtv * A[hd]);
            const double *xt = x + (bt * H + hd) * P;
            const double *Bt = Bm + (bt * G + g) * N;
            const double *Ct = Cm + (bt * G + g) * N;
            step_state(h, P, N, alpha, dtv, xt, Bt);
            double *yt = y + (bt * H + hd) * P;
            for (int p = 0; p < P; ++p) {
                const double *hp = h + (size_t)p * N;
                double acc = 0.0;
                for (int n = 0; n < N; ++n) acc += Ct[n] * hp[n];
                yt[p] = acc + D[hd] * xt[p];
            }
        }
        if (h_final) memcpy(h_final + (size_t)bh * PN, h, PN * sizeof(double));
        free(h);
    }
    return fail ? -2 : 0;
}

/*
 * Backward (Algorithm 2 along the sequence axis, one layer).
 * Loss = sum(y * dy) + sum(h_final * dh_final);  dh_final == NULL means zero.
 * blk  = the oracle's own checkpoint interval (any value >= 1; results do not
 *        depend on it).  Outputs dA[H], dD[H] are summed over batch and time,
 *        dB/dC over the heads of a group in ascending head order.  dh0 may be NULL.
 */
int ssd_oracle_bwd(int B, int L, int H, int P, int N, int G, int blk,
                   const double *x, const double *dt, const double *A,
                   const double *Bm, const double *Cm, const double *D,
                   const double *h0, const double *dy, const double *dh_final,
                   double *dx, double *ddt, double *dA, double *dB, double *dC,
                   double *dD, double *dh0) {
    if (B <= 0 || L <= 0 || H <= 0 || P <= 0 || N <= 0 || G <= 0 || H % G || blk <= 0) return -1;
    const int hpg = H / G;
    const int nblk = (L + blk - 1) / blk;
    const size_t PN = (size_t)P * N;
    const int BH = B * H;
    int fail = 0;

    /* S_ckpt: state entering every block, per (b, head). */
    double *ck = (double *)malloc((size_t)BH * nblk * PN * sizeof(double));
    /* state gradient carried leftwards across blocks, per (b, head): the nabla_h of Alg. 2 */
    double *carry = (double *)malloc((size_t)BH * PN * sizeof(double));
    /* per-head contributions to dB / dC inside the current block */
    double *dBh = (double *)malloc((size_t)BH * blk * N * sizeof(double));
    double *dCh = (double *)malloc((size_t)BH * blk * N * sizeof(double));
    double *dAbh = (double *)calloc((size_t)BH, sizeof(double));
    double *dDbh = (double *)calloc((size_t)BH, sizeof(double));
    if (!ck || !carry || !dBh || !dCh || !dAbh || !dDbh) {
        free(ck); free(carry); free(dBh); free(dCh); free(dAbh); free(dDbh);
        return -2;
    }

    /* forward sweep: keep only the block-entry states */
#pragma omp parallel for schedule(static)
    for (int bh = 0; bh < BH; ++bh) {
        const int b = bh / H, hd = bh % H, g = hd / hpg;
        double *h = (double *)malloc(PN * sizeof(double));
        if (!h) { fail = 1; continue; }
        if (h0) memcpy(h, h0 + (size_t)bh * PN, PN * sizeof(double));
        else memset(h, 0, PN * sizeof(double));
        for (int t = 0; t < L; ++t) {
            if (t % blk == 0) memcpy(ck + ((size_t)bh * nblk + t / blk) * PN, h, PN * sizeof(double));
            const size_t bt = (size_t)b * L + t;
            const double dtv = dt[bt * H + hd];
            step_state(h, P, N, exp(dtv * A[hd]), dtv, x + (bt * H + hd) * P, Bm + (bt * G + g) * N);
        }
        if (dh_final) memcpy(carry + (size_t)bh * PN, dh_final + (size_t)bh * PN, PN * sizeof(double));
        else memset(carry + (size_t)bh * PN, 0, PN * sizeof(double));
        free(h);
    }
    if (fail) goto done;

    for (int kb = nblk - 1; kb >= 0; --kb) {
        const int t0 = kb * blk;
        const int t1 = (t0 + blk < L) ? t0 + blk : L;
        const int len = t1 - t0;
#pragma omp parallel for schedule(static)
        for (int bh = 0; bh < BH; ++bh) {
            const int b = bh / H, hd = bh % H, g = hd / hpg;
            /* Recompute_Forward: hs[i] = state after token t0+i-1; hs[0] = checkpoint */
            double *hs = (double *)malloc((size_t)(len + 1) * PN * sizeof(double));
            double *gs = (double *)malloc(PN * sizeof(double));
            if (!hs || !gs) { fail = 1; free(hs); free(gs); continue; }
            memcpy(hs, ck + ((size_t)bh * nblk + kb) * PN, PN * sizeof(double));
            for (int i = 0; i < len; ++i) {
                const size_t bt = (size_t)b * L + t0 + i;
                const double dtv = dt[bt * H + hd];
                memcpy(hs + (size_t)(i + 1) * PN, hs + (size_t)i * PN, PN * sizeof(double));
                step_state(hs + (size_t)(i + 1) * PN, P, N, exp(dtv * A[hd]), dtv,
                           x + (bt * H + hd) * P, Bm + (bt * G + g) * N);
            }
            /* Backward through the block, newest step first. c = dLoss/dh_t from the future. */
            double *c = carry + (size_t)bh * PN;
            double accA = 0.0, accD = 0.0;
            for (int i = len - 1; i >= 0; --i) {
                const size_t bt = (size_t)b * L + t0 + i;
                const double dtv = dt[bt * H + hd];
                const double alpha = exp(dtv * A[hd]);
                const double *xt = x + (bt * H + hd) * P;
                const double *dyt = dy + (bt * H + hd) * P;
                const double *Bt = Bm + (bt * G + g) * N;
                const double *Ct = Cm + (bt * G + g) * N;
                const double *hcur = hs + (size_t)(i + 1) * PN;   /* h_t     */
                const double *hprev = hs + (size_t)i * PN;        /* h_{t-1} */
                double *dBt = dBh + ((size_t)bh * blk + i) * N;
                double *dCt = dCh + ((size_t)bh * blk + i) * N;
                double *dxt = dx + (bt * H + hd) * P;
                for (int n = 0; n < N; ++n) { dBt[n] = 0.0; dCt[n] = 0.0; }
                double ddt_direct = 0.0, da = 0.0;
                for (int p = 0; p < P; ++p) {
                    double *cp = c + (size_t)p * N;
                    const double *hp = hcur + (size_t)p * N;
                    const double *hq = hprev + (size_t)p * N;
                    double u = 0.0;
                    for (int n = 0; n < N; ++n) {
                        const double gpn = dyt[p] * Ct[n] + cp[n];   /* total dLoss/dh_t[p,n] */
                        gs[(size_t)p * N + n] = gpn;
                        dCt[n] += dyt[p] * hp[n];
                        u += gpn * Bt[n];
                        dBt[n] += dtv * gpn * xt[p];
                        da += gpn * hq[n];
                    }
                    dxt[p] = D[hd] * dyt[p] + dtv * u;
                    ddt_direct += xt[p] * u;
                    accD += dyt[p] * xt[p];
                }
                da *= alpha;                      /* dLoss/d(dt_t * A) */
                ddt[bt * H + hd] = ddt_direct + A[hd] * da;
                accA += dtv * da;
                for (size_t e = 0; e < PN; ++e) c[e] = alpha * gs[e];
            }
            dAbh[bh] += accA;
            dDbh[bh] += accD;
            free(hs); free(gs);
        }
        if (fail) goto done;
        /* sum the heads of each group, ascending head order */
#pragma omp parallel for schedule(static)
        for (int i = 0; i < len; ++i) {
            for (int b = 0; b < B; ++b)
                for (int g = 0; g < G; ++g) {
                    double *dBt = dB + (((size_t)b * L + t0 + i) * G + g) * N;
                    double *dCt = dC + (((size_t)b * L + t0 + i) * G + g) * N;
                    for (int n = 0; n < N; ++n) { dBt[n] = 0.0; dCt[n] = 0.0; }
                    for (int hd = g * hpg; hd < (g + 1) * hpg; ++hd) {
                        const double *sB = dBh + (((size_t)b * H + hd) * blk + i) * N;
                        const double *sC = dCh + (((size_t)b * H + hd) * blk + i) * N;
                        for (int n = 0; n < N; ++n) { dBt[n] += sB[n]; dCt[n] += sC[n]; }
                    }
                }
        }
    }
    for (int hd = 0; hd < H; ++hd) {
        double sA = 0.0, sD = 0.0;
        for (int b = 0; b < B; ++b) { sA += dAbh[(size_t)b * H + hd]; sD += dDbh[(size_t)b * H + hd]; }
        dA[hd] = sA; dD[hd] = sD;
    }
    if (dh0) memcpy(dh0, carry, (size_t)BH * PN * sizeof(double));
done:
    free(ck); free(carry); free(dBh); free(dCh); free(dAbh); free(dDbh);
    return fail ? -2 : 0;
}
