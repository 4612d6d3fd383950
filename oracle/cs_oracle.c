/*
 * CPU oracle for the measure -> recover -> execute step of a SwiGLU FFN layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
 * what the CUDA library computes.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the library never does, and the
 * two share no code.
 *
 * Every function follows the paper's pipeline in its own order:
 *   sensor    (Sec. 8 "Measurement Design": z_t = A_t u_t, written here y = S h),
 *   estimator (Sec. 7 "Hardware-Aware Structured Recovery": least squares
 *              subject to supp in H, solved by the "projected proximal method
 *              with a small fixed number of iterations" of Sec. 8 -- with
 *              lambda = 0 and H = all k-subsets of G groups that is iterative
 *              hard thresholding, z <- H_k(z + mu Phi^T (y - Phi z))),
 *   support   (Sec. 3: s_t = supp_tau(alpha_t), here the k kept indices),
 *   actuator  (Sec. 3: F(x; theta, s_t), execution only on the support -- here
 *              the SwiGLU FFN restricted to the active channel groups),
 *   prompt-level support (Sec. 4 "Task-Conditioned Measurements": one support
 *              s*(p) per prompt, from the mean of the prompt's sketches).
 *
 * Parameters are read in their storage type (float32, or bfloat16 as uint16)
 * and widened exactly to double; all arithmetic is double.  Loops are in
 * definition order; OpenMP only spreads independent output elements over
 * threads (no blocking, no reassociation inside a sum).
 *
 * Pins (tests/test_oracle_*.py): closed forms for T=1, orthonormal Phi and
 * Phi = I; fixed-point, monotone-residual and homogeneity invariants; planted
 * recovery and brute-force agreement on easy shapes; k = G equals a dense FFN
 * written with numpy matmuls; additivity over disjoint supports; hand cases
 * for H_k ties, RMSNorm and single channels.
 * Parity unpinned: nothing fixes that the support IHT returns is the *best*
 * k-subset at the benchmark shapes (IHT is a heuristic there); only
 * resid_IHT >= resid_bruteforce is asserted.
 *
 * Further estimators and sensors the paper names (each pinned in
 * tests/test_oracle_solvers.py):
 *   temporal term   (Sec. 5: Omega_temp = gamma ||alpha_t - alpha_{t-1}||^2 added to the
 *                    recovery objective; here the projected-gradient iteration on it),
 *   normalised step (Sec. 8 "projected proximal methods with a small fixed number of
 *                    iterations", with the step chosen per iteration from the current
 *                    support instead of a constant),
 *   OMP             (Sec. 8 / Sec. 9 proposition: orthogonal matching pursuit restricted to
 *                    the feasible supports, here any k of the G groups),
 *   SRHT sensor     (Sec. 8: a subsampled randomized Hadamard operator as A_t).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F32 0
#define ORACLE_BF16 1

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* bfloat16 is the upper half of a float32: widening is exact. */
static double bf16_to_double(uint16_t v) {
    uint32_t u = ((uint32_t)v) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double weight_at(const void *W, int dtype, size_t idx) {
    if (dtype == ORACLE_BF16) return bf16_to_double(((const uint16_t *)W)[idx]);
    return (double)((const float *)W)[idx];
}

/* n = x / sqrt(mean(x^2) + eps) * gamma  (RMSNorm ahead of the FFN in the stacked workload). */
void oracle_rmsnorm(const double *x, const float *gamma, int d, double eps, double *n) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / (double)d + eps);
    for (int i = 0; i < d; ++i) n[i] = x[i] * r * (double)gamma[i];
}

/* Sensor: y = S h, S [m,d] row-major float32. */
void oracle_sketch(const float *S, const double *h, int m, int d, double *y) {
    for (int r = 0; r < m; ++r) {
        double acc = 0.0;
        for (int i = 0; i < d; ++i) acc += (double)S[(size_t)r * d + i] * h[i];
        y[r] = acc;
    }
}

/* 1 if entry (a, ia) comes before (b, ib) in the order |v| descending, index ascending. */
static int precedes(double a, int ia, double b, int ib) {
    double fa = fabs(a), fb = fabs(b);
    if (fa != fb) return fa > fb;
    return ia < ib;
}

/*
 * H_k: keep the k entries that come first in the order above, zero the rest.
 * keep[g] = 1 for kept entries.  *gap = (|v|_(k) - |v|_(k+1)) / |v|_(k), the
 * relative margin between the last kept and first dropped magnitude
 * (INFINITY when k == G or |v|_(k) == 0 == |v|_(k+1) gives 0/0 -> reported 0).
 */
void oracle_hard_threshold(const double *v, int G, int k, int *keep, double *gap) {
    double kth = 0.0, next = 0.0;
    for (int g = 0; g < G; ++g) {
        int rank = 0;
        for (int j = 0; j < G; ++j)
            if (j != g && precedes(v[j], j, v[g], g)) ++rank;
        keep[g] = rank < k;
        if (rank == k - 1) kth = fabs(v[g]);
        if (rank == k) next = fabs(v[g]);
    }
    if (gap) {
        if (k >= G) *gap = INFINITY;
        else if (kth == 0.0) *gap = 0.0;
        else *gap = (kth - next) / kth;
    }
}

static double residual_norm(const float *Phi, const double *y, const double *z, int m, int G, double *r) {
    double ss = 0.0;
    for (int i = 0; i < m; ++i) {
        double acc = 0.0;
        for (int g = 0; g < G; ++g) acc += (double)Phi[(size_t)i * G + g] * z[g];
        r[i] = y[i] - acc;
        ss += r[i] * r[i];
    }
    return sqrt(ss);
}

/*
 * Estimator: z_0 given (or 0); T times  r = y - Phi z;  v = z + mu Phi^T r;  z = H_k(v).
 * Outputs: z [G] (k-sparse), support [k] ascending = the indices kept by the
 * last H_k (for T == 0: the first k indices of the order applied to z_0),
 * resid_hist [T+1] = ||y - Phi z_t|| for t = 0..T, gap_hist [T] = margin of each H_k.
 */
void oracle_iht(const float *Phi, const double *y, int m, int G, int k, int T, double mu,
                const double *z0, double *z, int32_t *support, double *resid_hist, double *gap_hist) {
    double *r = (double *)malloc(sizeof(double) * (size_t)m);
    double *v = (double *)malloc(sizeof(double) * (size_t)G);
    int *keep = (int *)malloc(sizeof(int) * (size_t)G);
    for (int g = 0; g < G; ++g) z[g] = z0 ? z0[g] : 0.0;
    oracle_hard_threshold(z, G, k, keep, NULL);
    double rn = residual_norm(Phi, y, z, m, G, r);
    if (resid_hist) resid_hist[0] = rn;
    for (int t = 0; t < T; ++t) {
        for (int g = 0; g < G; ++g) {
            double acc = 0.0;
            for (int i = 0; i < m; ++i) acc += (double)Phi[(size_t)i * G + g] * r[i];
            v[g] = z[g] + mu * acc;
        }
        double gap;
        oracle_hard_threshold(v, G, k, keep, &gap);
        for (int g = 0; g < G; ++g) z[g] = keep[g] ? v[g] : 0.0;
        rn = residual_norm(Phi, y, z, m, G, r);
        if (resid_hist) resid_hist[t + 1] = rn;
        if (gap_hist) gap_hist[t] = gap;
    }
    int c = 0;
    for (int g = 0; g < G; ++g)
        if (keep[g]) support[c++] = g;
    free(r); free(v); free(keep);
}

/*
 * The same estimator with the temporal regulariser of Sec. 5,
 *     minimise  1/2 ||y - Phi z||^2 + gamma ||z - z_prev||^2   subject to  ||z||_0 <= k,
 * by the projected-gradient step of the iteration above on this objective:
 *     v = z + mu (Phi^T (y - Phi z) - 2 gamma (z - z_prev));   z = H_k(v).
 * z_prev [G] is the previous decoding step's (k-sparse) estimate; gamma = 0 gives oracle_iht exactly.
 * resid_hist records ||y - Phi z_t|| (the data term alone), as oracle_iht does.
 */
void oracle_iht_temporal(const float *Phi, const double *y, int m, int G, int k, int T, double mu, double gamma,
                         const double *z_prev, const double *z0, double *z, int32_t *support,
                         double *resid_hist, double *gap_hist) {
    double *r = (double *)malloc(sizeof(double) * (size_t)m);
    double *v = (double *)malloc(sizeof(double) * (size_t)G);
    int *keep = (int *)malloc(sizeof(int) * (size_t)G);
    for (int g = 0; g < G; ++g) z[g] = z0 ? z0[g] : 0.0;
    oracle_hard_threshold(z, G, k, keep, NULL);
    double rn = residual_norm(Phi, y, z, m, G, r);
    if (resid_hist) resid_hist[0] = rn;
    for (int t = 0; t < T; ++t) {
        for (int g = 0; g < G; ++g) {
            double acc = 0.0;
            for (int i = 0; i < m; ++i) acc += (double)Phi[(size_t)i * G + g] * r[i];
            v[g] = z[g] + mu * (acc - 2.0 * gamma * (z[g] - (z_prev ? z_prev[g] : 0.0)));
        }
        double gap;
        oracle_hard_threshold(v, G, k, keep, &gap);
        for (int g = 0; g < G; ++g) z[g] = keep[g] ? v[g] : 0.0;
        rn = residual_norm(Phi, y, z, m, G, r);
        if (resid_hist) resid_hist[t + 1] = rn;
        if (gap_hist) gap_hist[t] = gap;
    }
    int c = 0;
    for (int g = 0; g < G; ++g)
        if (keep[g]) support[c++] = g;
    free(r); free(v); free(keep);
}

/*
 * Iterative hard thresholding with a normalised step: in every iteration the step is the one that
 * minimises the residual along the gradient restricted to the current support S,
 *     g = Phi^T (y - Phi z);   S = supp(z)  (for z = 0: the k entries H_k keeps of g);
 *     mu_t = ||g_S||^2 / ||Phi g_S||^2   (mu_fallback when the denominator is 0);
 *     z = H_k(z + mu_t g).
 * No line search follows the step (the published method adds one for the iterations that change the
 * support); with it left out the residual need not fall in such an iteration.
 * step_hist [T] receives mu_t; other outputs as oracle_iht.
 */
void oracle_niht(const float *Phi, const double *y, int m, int G, int k, int T, double mu_fallback,
                 double *z, int32_t *support, double *resid_hist, double *gap_hist, double *step_hist) {
    double *r = (double *)malloc(sizeof(double) * (size_t)m);
    double *g = (double *)malloc(sizeof(double) * (size_t)G);
    double *v = (double *)malloc(sizeof(double) * (size_t)G);
    int *keep = (int *)malloc(sizeof(int) * (size_t)G);
    for (int j = 0; j < G; ++j) z[j] = 0.0;
    oracle_hard_threshold(z, G, k, keep, NULL);
    double rn = residual_norm(Phi, y, z, m, G, r);
    if (resid_hist) resid_hist[0] = rn;
    for (int t = 0; t < T; ++t) {
        for (int j = 0; j < G; ++j) {
            double acc = 0.0;
            for (int i = 0; i < m; ++i) acc += (double)Phi[(size_t)i * G + j] * r[i];
            g[j] = acc;
        }
        if (t == 0) oracle_hard_threshold(g, G, k, keep, NULL);   /* z = 0 has no support of its own yet */
        double num = 0.0, den = 0.0;
        for (int j = 0; j < G; ++j) if (keep[j]) num += g[j] * g[j];
        for (int i = 0; i < m; ++i) {
            double acc = 0.0;
            for (int j = 0; j < G; ++j) if (keep[j]) acc += (double)Phi[(size_t)i * G + j] * g[j];
            den += acc * acc;
        }
        double mu_t = den > 0.0 ? num / den : mu_fallback;
        if (step_hist) step_hist[t] = mu_t;
        for (int j = 0; j < G; ++j) v[j] = z[j] + mu_t * g[j];
        double gap;
        oracle_hard_threshold(v, G, k, keep, &gap);
        for (int j = 0; j < G; ++j) z[j] = keep[j] ? v[j] : 0.0;
        rn = residual_norm(Phi, y, z, m, G, r);
        if (resid_hist) resid_hist[t + 1] = rn;
        if (gap_hist) gap_hist[t] = gap;
    }
    int c = 0;
    for (int j = 0; j < G; ++j)
        if (keep[j]) support[c++] = j;
    free(r); free(g); free(v); free(keep);
}

/*
 * Orthogonal matching pursuit over the feasible supports (any k of the G groups): k times, pick the
 * group whose normalised column correlates most with the residual,
 *     j = argmax_{g not in S} |phi_g^T r| / ||phi_g||    (ties: lowest index; zero columns never),
 * add it to S and refit  z_S = argmin ||y - Phi_S z||,  r = y - Phi_S z_S.
 * The refit keeps an orthonormal basis Q of the chosen columns (Gram-Schmidt, applied twice) and the
 * triangular factor R with Phi_S = Q R, so z_S = R^{-1} Q^T y by back substitution.  A column that
 * lies in the span of those already chosen (norm after orthogonalisation <= 1e-12 of its own) adds
 * nothing: it enters the support with coefficient 0.  If no column is left to pick (all correlations
 * zero) the support is completed with the lowest unused indices, coefficient 0, so that exactly k
 * indices are returned.
 * Outputs: z [G], support [k] ascending, order [k] the groups in the order picked (-1 for
 * completions), *resid = ||y - Phi z||, gap_hist [k] = (best - second best) / best of the normalised
 * correlations at each pick (INFINITY when only one candidate is left, 0 for completions).
 */
void oracle_omp(const float *Phi, const double *y, int m, int G, int k, double *z, int32_t *support,
                int32_t *order, double *resid, double *gap_hist) {
    double *r = (double *)malloc(sizeof(double) * (size_t)m);
    double *Q = (double *)calloc((size_t)m * (size_t)k, sizeof(double));      /* column s at Q[s*m ..] */
    double *R = (double *)calloc((size_t)k * (size_t)k, sizeof(double));      /* R[a*k + s], a <= s */
    double *qty = (double *)calloc((size_t)k, sizeof(double));
    double *col = (double *)malloc(sizeof(double) * (size_t)m);
    double *cn = (double *)malloc(sizeof(double) * (size_t)G);
    int *in = (int *)calloc((size_t)G, sizeof(int));
    int *picked = (int *)malloc(sizeof(int) * (size_t)k);
    int *live = (int *)calloc((size_t)k, sizeof(int));                        /* basis vector exists for pick s */
    for (int i = 0; i < m; ++i) r[i] = y[i];
    for (int g = 0; g < G; ++g) {
        double ss = 0.0;
        for (int i = 0; i < m; ++i) ss += (double)Phi[(size_t)i * G + g] * (double)Phi[(size_t)i * G + g];
        cn[g] = sqrt(ss);
        z[g] = 0.0;
    }
    int ns = 0;
    for (int s = 0; s < k; ++s) {
        int best = -1, cand = 0;
        double bv = 0.0, second = 0.0;
        for (int g = 0; g < G; ++g) {
            if (in[g] || cn[g] == 0.0) continue;
            double acc = 0.0;
            for (int i = 0; i < m; ++i) acc += (double)Phi[(size_t)i * G + g] * r[i];
            double c = fabs(acc) / cn[g];
            ++cand;
            if (c > bv) { second = bv; bv = c; best = g; }
            else if (c > second) second = c;
        }
        if (best < 0 || bv == 0.0) {          /* nothing correlates: complete with the lowest unused indices */
            int g = 0;
            while (in[g]) ++g;
            in[g] = 1; picked[s] = g; order[s] = -1;
            if (gap_hist) gap_hist[s] = 0.0;
            ++ns;
            continue;
        }
        if (gap_hist) gap_hist[s] = cand > 1 ? (bv - second) / bv : INFINITY;
        in[best] = 1; picked[s] = best; order[s] = best; ++ns;
        for (int i = 0; i < m; ++i) col[i] = (double)Phi[(size_t)i * G + best];
        for (int pass = 0; pass < 2; ++pass)          /* Gram-Schmidt, twice */
            for (int a = 0; a < s; ++a) {
                if (!live[a]) continue;
                double dot = 0.0;
                for (int i = 0; i < m; ++i) dot += Q[(size_t)a * m + i] * col[i];
                for (int i = 0; i < m; ++i) col[i] -= dot * Q[(size_t)a * m + i];
                R[(size_t)a * k + s] += dot;
            }
        double nn = 0.0;
        for (int i = 0; i < m; ++i) nn += col[i] * col[i];
        nn = sqrt(nn);
        if (nn <= 1e-12 * cn[best]) continue;          /* in the span already: coefficient stays 0 */
        live[s] = 1;
        R[(size_t)s * k + s] = nn;
        double qy = 0.0;
        for (int i = 0; i < m; ++i) { Q[(size_t)s * m + i] = col[i] / nn; qy += Q[(size_t)s * m + i] * y[i]; }
        qty[s] = qy;
        /* r = y - Q Q^T y over the live basis vectors */
        for (int i = 0; i < m; ++i) r[i] = y[i];
        for (int a = 0; a <= s; ++a) {
            if (!live[a]) continue;
            for (int i = 0; i < m; ++i) r[i] -= qty[a] * Q[(size_t)a * m + i];
        }
    }
    /* z_S = R^{-1} Q^T y by back substitution over the live picks */
    double *coef = (double *)calloc((size_t)k, sizeof(double));
    for (int s = ns - 1; s >= 0; --s) {
        if (!live[s]) continue;
        double acc = qty[s];
        for (int b = s + 1; b < ns; ++b)
            if (live[b]) acc -= R[(size_t)s * k + b] * coef[b];
        coef[s] = acc / R[(size_t)s * k + s];
    }
    for (int s = 0; s < ns; ++s) z[picked[s]] = coef[s];
    int c = 0;
    for (int g = 0; g < G; ++g)
        if (in[g]) support[c++] = g;
    double ss = 0.0;
    for (int i = 0; i < m; ++i) {
        double acc = 0.0;
        for (int g = 0; g < G; ++g) acc += (double)Phi[(size_t)i * G + g] * z[g];
        ss += (y[i] - acc) * (y[i] - acc);
    }
    if (resid) *resid = sqrt(ss);
    free(r); free(Q); free(R); free(qty); free(col); free(cn); free(in); free(picked); free(live); free(coef);
}

/*
 * Sensor, structured: a subsampled randomized Hadamard operator (Sec. 8),
 *     y_r = (1 / sqrt(m)) sum_i H[rows[r], i] sign[i] h[i],   H[a, i] = (-1)^popcount(a & i),
 * with d a power of two, sign[i] in {+1, -1} and rows [m] distinct indices in [0, d).  Written out
 * term by term (no fast transform): m * d multiply-adds.
 */
void oracle_srht(const int8_t *sign, const int32_t *rows, const double *h, int m, int d, double *y) {
    double scale = 1.0 / sqrt((double)m);
    for (int r = 0; r < m; ++r) {
        double acc = 0.0;
        unsigned a = (unsigned)rows[r];
        for (int i = 0; i < d; ++i) {
            unsigned bits = a & (unsigned)i, par = 0;
            while (bits) { par ^= 1u; bits &= bits - 1u; }
            double term = (double)sign[i] * h[i];
            acc += par ? -term : term;
        }
        y[r] = scale * acc;
    }
}

static double silu(double x) { return x / (1.0 + exp(-x)); }

/*
 * Actuator: out = sum_{g in support} sum_{j<b} silu(W_gate[gb+j,:] h) (W_up[gb+j,:] h) Wd_t[gb+j,:]
 * W_gate, W_up, Wd_t: [d_ff, d] row-major in `dtype`; Wd_t is W_down transposed, so row
 * gb+j of Wd_t is column gb+j of W_down.  out [d] is overwritten.  act (may be NULL)
 * receives the k*b intermediate values in support order.
 */
void oracle_ffn(const void *Wg, const void *Wu, const void *Wdt, int dtype, int d, int b,
                const double *h, const int32_t *support, int k, double *out, double *act) {
    int n = k * b;
    double *a = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
#pragma omp parallel for schedule(static)
    for (int c = 0; c < n; ++c) {
        size_t row = (size_t)support[c / b] * b + (size_t)(c % b);
        double g = 0.0, u = 0.0;
        for (int i = 0; i < d; ++i) {
            g += weight_at(Wg, dtype, row * d + i) * h[i];
            u += weight_at(Wu, dtype, row * d + i) * h[i];
        }
        a[c] = silu(g) * u;
    }
    /* out[i] = sum_c a[c] Wd_t[row(c), i], c ascending; threads own disjoint ranges of i. */
#pragma omp parallel for schedule(static)
    for (int i0 = 0; i0 < d; i0 += 256) {
        int i1 = i0 + 256 < d ? i0 + 256 : d;
        for (int i = i0; i < i1; ++i) out[i] = 0.0;
        for (int c = 0; c < n; ++c) {
            size_t row = (size_t)support[c / b] * b + (size_t)(c % b);
            for (int i = i0; i < i1; ++i) out[i] += a[c] * weight_at(Wdt, dtype, row * d + i);
        }
    }
    if (act) memcpy(act, a, sizeof(double) * (size_t)n);
    free(a);
}

/*
 * One layer for B tokens, each with its own support (Sec. 5 "Token-Adaptive Recovery":
 * sketch, recover, execute at every step).
 *   n   = rms_gamma ? RMSNorm(x) : x
 *   y   = S n ;  (z, support) = IHT(Phi, y) ;  f = FFN(n, support)
 *   out = add_residual ? x + f : f
 * forced_support (may be NULL): if given, [B,k] supports used for the FFN in place of the
 * recovered ones (recovery outputs are still produced).
 * Outputs (any may be NULL except x_out): y [B,m], z_full [B,G], support [B,k], z_sup [B,k]
 * (z on the support), resid [B] (final ||y - Phi z_T||), min_gap [B] (min over iterations).
 */
void oracle_layer_step(const float *S, const float *Phi, const void *Wg, const void *Wu, const void *Wdt,
                       int dtype, const float *rms_gamma, double rms_eps, int add_residual,
                       int d, int d_ff, int b, int m, int k, int T, double mu,
                       const double *x, int B, const int32_t *forced_support,
                       double *x_out, double *y_out, double *z_full, int32_t *support_out,
                       double *z_sup, double *resid, double *min_gap) {
    int G = d_ff / b;
    double *n = (double *)malloc(sizeof(double) * (size_t)d);
    double *y = (double *)malloc(sizeof(double) * (size_t)m);
    double *z = (double *)malloc(sizeof(double) * (size_t)G);
    double *f = (double *)malloc(sizeof(double) * (size_t)d);
    double *rh = (double *)malloc(sizeof(double) * (size_t)(T + 1));
    double *gh = (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    int32_t *sup = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
    for (int t = 0; t < B; ++t) {
        const double *xt = x + (size_t)t * d;
        if (rms_gamma) oracle_rmsnorm(xt, rms_gamma, d, rms_eps, n);
        else memcpy(n, xt, sizeof(double) * (size_t)d);
        oracle_sketch(S, n, m, d, y);
        oracle_iht(Phi, y, m, G, k, T, mu, NULL, z, sup, rh, gh);
        if (y_out) memcpy(y_out + (size_t)t * m, y, sizeof(double) * (size_t)m);
        if (z_full) memcpy(z_full + (size_t)t * G, z, sizeof(double) * (size_t)G);
        if (support_out) memcpy(support_out + (size_t)t * k, sup, sizeof(int32_t) * (size_t)k);
        if (z_sup) for (int c = 0; c < k; ++c) z_sup[(size_t)t * k + c] = z[sup[c]];
        if (resid) resid[t] = rh[T];
        if (min_gap) {
            double mg = INFINITY;
            for (int it = 0; it < T; ++it) if (gh[it] < mg) mg = gh[it];
            min_gap[t] = mg;
        }
        const int32_t *use = forced_support ? forced_support + (size_t)t * k : sup;
        oracle_ffn(Wg, Wu, Wdt, dtype, d, b, n, use, k, f, NULL);
        for (int i = 0; i < d; ++i) x_out[(size_t)t * d + i] = (add_residual ? xt[i] : 0.0) + f[i];
    }
    free(n); free(y); free(z); free(f); free(rh); free(gh); free(sup);
}

/*
 * Prompt-level support (Sec. 4): ybar = (1/n) sum_i S h_i, then one IHT.
 * H [n,d] double.  Outputs as oracle_iht plus ybar [m].
 */
void oracle_prompt_support(const float *S, const float *Phi, const double *H, int n, int d, int m, int G,
                           int k, int T, double mu, double *ybar, double *z, int32_t *support,
                           double *resid_hist, double *gap_hist) {
    double *y = (double *)malloc(sizeof(double) * (size_t)m);
    for (int r = 0; r < m; ++r) ybar[r] = 0.0;
    for (int i = 0; i < n; ++i) {
        oracle_sketch(S, H + (size_t)i * d, m, d, y);
        for (int r = 0; r < m; ++r) ybar[r] += y[r];
    }
    for (int r = 0; r < m; ++r) ybar[r] /= (double)n;
    oracle_iht(Phi, ybar, m, G, k, T, mu, NULL, z, support, resid_hist, gap_hist);
    free(y);
}
