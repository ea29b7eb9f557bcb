/*
 * DES-LOC reference oracle  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded restatement of the DES-LOC update rules, used
 * only to check the CUDA library and to give a host-core timing baseline.  It
 * shares no code with the CUDA path and the CUDA path never calls it.
 *
 * What it computes (paper notation):
 *   - Algorithm 1 (generic DES-LOC): M workers; at step t each worker clips its
 *     own gradient coordinate-wise, updates every optimizer state s^j from
 *     either its own previous state or -- when t mod K_j = 0 -- the mean over
 *     workers of the previous states, then updates x from its own x_t or --
 *     when t mod K_x = 0 -- the worker-mean of x_t.
 *   - Algorithm 2 (DES-LOC-Adam), Algorithm 3 (DES-LOC-ADOPT), and Algorithm 1
 *     with the single-state SGDM rule  u = beta u + (1-beta) g,  x = x - eta u
 *     (the update rule stated at the start of the SGDM convergence appendix).
 *   - Coordinate-wise clipping, Section 3.1:  clip(X,rho)_i = sgn(X_i) min(|X_i|,rho).
 *   - Post-average ordering of Algorithms 4 and 5 (average taken after the
 *     local update instead of before it), selected by DESLOC_ORACLE_POST_AVERAGE.
 *
 * Precision: state is stored as fp32 (the workload fixes x,u,v as fp32); every
 * step is computed in fp64 from those fp32 values and rounded to nearest-even
 * once when stored.  Sums over workers run in the fixed order m = 0..M-1.
 *
 * Readings where the paper is silent (each is listed in the design notes too):
 *   - "never sync" (K = infinity, the FAVG+OPT baseline of Section 5.1) is K = 0.
 *   - ADOPT divides by max(sqrt(v_{t-1}^m), eps) with the worker's own,
 *     un-averaged previous v even on a v-sync step, exactly as Algorithm 3 is
 *     written; DESLOC_ORACLE_ADOPT_AVG_NORMALISER switches to the averaged one
 *     (used only to measure how much the reading matters).
 *   - weight decay (absent from the paper's algorithms) is decoupled:
 *     x_{t+1} = x* (1 - eta_t wd) - d_t, x* being the possibly averaged base.
 *   - the optional ADOPT clip of the normalised gradient to +-c_t takes c_t
 *     from the caller each step.
 *   - no bias-correction factor is applied: none appears in Algorithm 2's
 *     formulas.  A caller folds it into eta_t.
 *
 *   - norm-based clipping (used by the paper's language-model runs, absent from the
 *     algorithm listings) scales each worker's whole gradient by min(1, rho_norm/||g||_2)
 *     BEFORE the coordinate clip; no epsilon is added to the norm.
 *
 *   - norms reported as diagnostics: the gradient norm is taken over the gradient as it is
 *     read (before any clipping), the parameter norm over x_{t+1} as stored, the update norm
 *     over d_t; each per worker and per tensor.
 *
 * Pins (tests/test_oracle_pins.py): M=1 against torch.optim.Adam / AdamW / SGD
 * in fp64; identical gradients keep replicas equal to the single-worker run;
 * the worker-mean of u, v (and of x for SGDM) does not depend on the schedule;
 * three hand-worked examples in exact rationals; the clipping bounds of
 * Eqs. 5-6; the printed communication ratios (170x, 85x, 256x, 2x); full
 * agreement of the workers' inputs at multiples of lcm(K_x,K_u,K_v); d_t against
 * the hand examples (both as eta u / sqrt(v) and as the difference of consecutive x), against
 * the parameter change torch.optim makes at M = 1, and one-step closed forms; tensor norms
 * against 3-4-5 style closed forms and numpy.linalg.norm.
 * Parity unpinned: the ADOPT normalised-gradient clip bound and the
 * weight-decay form are readings, not facts the paper fixes; the ADOPT rule
 * itself is pinned only by the hand example and brute force (no library has it).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_ADAM = 0, ORACLE_ADOPT = 1, ORACLE_SGDM = 2 };
enum { ORACLE_SYNC_X = 1, ORACLE_SYNC_U = 2, ORACLE_SYNC_V = 4 };
enum {
    DESLOC_ORACLE_ADOPT_NORM_CLIP = 1u,
    DESLOC_ORACLE_POST_AVERAGE = 2u,
    DESLOC_ORACLE_ADOPT_AVG_NORMALISER = 4u
};

typedef struct {
    int32_t M;
    int32_t opt;
    double beta1, beta2;
    double eps;          /* Adam: lambda (enters as lambda^2); ADOPT: epsilon */
    double weight_decay;
    double clip_rho;     /* <= 0: clipping off */
    int32_t Kx, Ku, Kv;  /* 0: never */
    uint32_t flags;
} desloc_oracle_cfg;

/* Algorithm 1, the three "t mod K = 0" tests; t counts from 0. */
uint32_t desloc_oracle_sync_mask(int32_t opt, int32_t Kx, int32_t Ku, int32_t Kv, int64_t t) {
    uint32_t mask = 0;
    if (Kx > 0 && t % Kx == 0) mask |= ORACLE_SYNC_X;
    if (Ku > 0 && t % Ku == 0) mask |= ORACLE_SYNC_U;
    if (opt != ORACLE_SGDM && Kv > 0 && t % Kv == 0) mask |= ORACLE_SYNC_V;
    return mask;
}

/* Section 3.1: clip(X, rho)_i = sgn(X_i) * min(|X_i|, rho). */
static double clip_coord(double g, double rho) {
    if (!(rho > 0.0)) return g;
    double a = fabs(g);
    if (a > rho) a = rho;
    return g < 0.0 ? -a : a;
}

/* E_m[.] over one coordinate: fixed order m = 0..M-1, fp64. */
static double worker_mean(const float *s, int64_t stride, int64_t i, int M) {
    double acc = 0.0;
    for (int m = 0; m < M; ++m) acc += (double)s[(int64_t)m * stride + i];
    return acc / (double)M;
}

/*
 * One DES-LOC step over n coordinates.  x, u, v, g are [M][stride] arrays
 * (worker-major), g already widened to fp32 (bf16 widens exactly).  v may be
 * NULL for SGDM.  Updates x, u, v in place; returns the sync mask used.
 * gscale (may be NULL): per-worker factors applied to g before the coordinate clip.
 * d_out (may be NULL): [M][stride] doubles, receives every worker's update d_t -- the quantity
 * Algorithm 2 names d_t = eta_t u_t / sqrt(v_t + lambda^2) (eta_t u_t for ADOPT and SGDM),
 * i.e. the step taken from the (possibly averaged) base, without the weight-decay term.
 */
uint32_t desloc_oracle_step_full(const desloc_oracle_cfg *c, int64_t t, double lr,
                                 double clip_bound, int64_t n, int64_t stride, float *x, float *u,
                                 float *v, const float *g, const double *gscale, double *d_out) {
    const int M = c->M;
    const uint32_t mask = desloc_oracle_sync_mask(c->opt, c->Kx, c->Ku, c->Kv, t);
    const int post = (c->flags & DESLOC_ORACLE_POST_AVERAGE) != 0;
    double *xn = (double *)malloc(sizeof(double) * (size_t)M);
    double *un = (double *)malloc(sizeof(double) * (size_t)M);
    double *vn = (double *)malloc(sizeof(double) * (size_t)M);

    for (int64_t i = 0; i < n; ++i) {
        double xbar = 0.0, ubar = 0.0, vbar = 0.0;
        if (!post) {
            /* Algorithms 1-3: the PREVIOUS values are averaged, then updated. */
            if (mask & ORACLE_SYNC_X) xbar = worker_mean(x, stride, i, M);
            if (mask & ORACLE_SYNC_U) ubar = worker_mean(u, stride, i, M);
            if (mask & ORACLE_SYNC_V) vbar = worker_mean(v, stride, i, M);
        }
        /* ---- optimizer states ------------------------------------------- */
        for (int m = 0; m < M; ++m) {
            const int64_t k = (int64_t)m * stride + i;
            const double gs = gscale ? gscale[m] : 1.0; /* norm-based clip factor, if any */
            const double gh = clip_coord((double)g[k] * gs, c->clip_rho);
            const double up = (!post && (mask & ORACLE_SYNC_U)) ? ubar : (double)u[k];
            double vp = 0.0;
            if (c->opt != ORACLE_SGDM)
                vp = (!post && (mask & ORACLE_SYNC_V)) ? vbar : (double)v[k];
            if (c->opt == ORACLE_ADAM) {
                /* Algorithm 2 (Eqs. 1-2): both moments from the clipped gradient. */
                un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;
                vn[m] = c->beta2 * vp + (1.0 - c->beta2) * gh * gh;
            } else if (c->opt == ORACLE_ADOPT) {
                /* Algorithm 3: v first; the momentum takes the gradient divided
                   by max(sqrt(v_{t-1}), eps) -- the value from BEFORE this step. */
                vn[m] = c->beta2 * vp + (1.0 - c->beta2) * gh * gh;
                double vold = (double)v[k];
                if ((c->flags & DESLOC_ORACLE_ADOPT_AVG_NORMALISER) && !post &&
                    (mask & ORACLE_SYNC_V))
                    vold = vbar;
                double den = sqrt(vold);
                if (den < c->eps) den = c->eps;
                double r = gh / den;
                if (c->flags & DESLOC_ORACLE_ADOPT_NORM_CLIP) {
                    if (r > clip_bound) r = clip_bound;
                    if (r < -clip_bound) r = -clip_bound;
                }
                un[m] = c->beta1 * up + (1.0 - c->beta1) * r;
            } else {
                /* SGDM: u = beta u + (1 - beta) g. */
                un[m] = c->beta1 * up + (1.0 - c->beta1) * gh;
                vn[m] = 0.0;
            }
        }
        if (post) {
            /* Algorithms 4-5: the freshly updated states are averaged, and the
               parameter step below uses the averaged ones. */
            if (mask & ORACLE_SYNC_U) {
                double acc = 0.0;
                for (int m = 0; m < M; ++m) acc += un[m];
                acc /= (double)M;
                for (int m = 0; m < M; ++m) un[m] = acc;
            }
            if (mask & ORACLE_SYNC_V) {
                double acc = 0.0;
                for (int m = 0; m < M; ++m) acc += vn[m];
                acc /= (double)M;
                for (int m = 0; m < M; ++m) vn[m] = acc;
            }
        }
        /* ---- direction and parameter update ----------------------------- */
        for (int m = 0; m < M; ++m) {
            const int64_t k = (int64_t)m * stride + i;
            const double xp = (!post && (mask & ORACLE_SYNC_X)) ? xbar : (double)x[k];
            double d;
            if (c->opt == ORACLE_ADAM)
                d = lr / sqrt(vn[m] + c->eps * c->eps) * un[m]; /* Algorithm 2 */
            else
                d = lr * un[m]; /* Algorithm 3 / SGDM */
            xn[m] = xp * (1.0 - lr * c->weight_decay) - d;
            if (d_out) d_out[k] = d; /* the update d_t of Algorithms 2-3, kept in fp64 */
        }
        if (post && (mask & ORACLE_SYNC_X)) {
            double acc = 0.0;
            for (int m = 0; m < M; ++m) acc += xn[m];
            acc /= (double)M;
            for (int m = 0; m < M; ++m) xn[m] = acc;
        }
        for (int m = 0; m < M; ++m) {
            const int64_t k = (int64_t)m * stride + i;
            x[k] = (float)xn[m];
            u[k] = (float)un[m];
            if (c->opt != ORACLE_SGDM) v[k] = (float)vn[m];
        }
    }
    free(xn);
    free(un);
    free(vn);
    return mask;
}

/* The same step with per-worker gradient factors (norm-based clipping) and no report of d. */
uint32_t desloc_oracle_step_scaled(const desloc_oracle_cfg *c, int64_t t, double lr,
                                   double clip_bound, int64_t n, int64_t stride, float *x, float *u,
                                   float *v, const float *g, const double *gscale) {
    return desloc_oracle_step_full(c, t, lr, clip_bound, n, stride, x, u, v, g, gscale, NULL);
}

uint32_t desloc_oracle_step(const desloc_oracle_cfg *c, int64_t t, double lr, double clip_bound,
                            int64_t n, int64_t stride, float *x, float *u, float *v,
                            const float *g) {
    return desloc_oracle_step_scaled(c, t, lr, clip_bound, n, stride, x, u, v, g, NULL);
}

/*
 * Clipping by the gradient's norm, the form the paper's language-model runs used (the model
 * table of the experimental-details appendix lists it with the bound rho): worker m's whole
 * gradient (all tensors, here one [M][stride] array) is scaled by min(1, max_norm / ||g^m||_2).  Writes the norms and
 * the factors; a zero gradient keeps factor 1.
 */
void desloc_oracle_norm_scales(int32_t M, int64_t n, int64_t stride, const float *g, double max_norm,
                               double *norms_out, double *scales_out) {
    for (int m = 0; m < M; ++m) {
        double acc = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            const double a = (double)g[(int64_t)m * stride + i];
            acc += a * a;
        }
        const double nrm = sqrt(acc);
        norms_out[m] = nrm;
        scales_out[m] = (nrm > max_norm) ? max_norm / nrm : 1.0;
    }
}

/*
 * Adding workers (Section 6, RQ3: the worker count is doubled mid-run; new workers start from
 * the synchronised state): out[i] = E_m[s^m_i] over the M current workers, fp64 sum in the
 * order m = 0..M-1, rounded to fp32 once.  The caller copies `out` into each new replica.
 */
void desloc_oracle_worker_mean(int32_t M, int64_t n, int64_t stride, const float *s, float *out) {
    for (int64_t i = 0; i < n; ++i) out[i] = (float)worker_mean(s, stride, i, M);
}

/*
 * Relative change of a state over an interval, ||s_now - s_then||_2 / ||s_then||_2 per worker
 * (the rate-of-change measure of Section 5.1, "Metrics").
 */
void desloc_oracle_rel_change(int32_t M, int64_t n, int64_t stride, const float *now,
                              const float *then, double *out) {
    for (int m = 0; m < M; ++m) {
        double num = 0.0, den = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            const double a = (double)now[(int64_t)m * stride + i];
            const double b = (double)then[(int64_t)m * stride + i];
            num += (a - b) * (a - b);
            den += b * b;
        }
        out[m] = sqrt(num) / sqrt(den);
    }
}

/*
 * Per-worker, per-tensor L2 norms (the parameter, update and gradient norms the paper plots
 * for its billion-scale runs: additional-results appendix, figure on update and parameter
 * norms; Section 6, RQ3, gradient norms after doubling the workers).  a is [M][stride] in
 * fp64; tensor k of worker m occupies a[m*stride + offs[k] .. + numel[k]).  Writes
 * out[m*num_tensors + k] = sqrt(sum of squares) and, if total_out is not NULL,
 * total_out[m] = the norm over all tensors of worker m (elements between tensors are not read).
 */
void desloc_oracle_tensor_norms(int32_t M, int64_t stride, int32_t num_tensors, const int64_t *offs,
                                const int64_t *numel, const double *a, double *out,
                                double *total_out) {
    for (int m = 0; m < M; ++m) {
        double all = 0.0;
        for (int32_t k = 0; k < num_tensors; ++k) {
            double acc = 0.0;
            for (int64_t i = 0; i < numel[k]; ++i) {
                const double e = a[(int64_t)m * stride + offs[k] + i];
                acc += e * e;
            }
            out[(int64_t)m * num_tensors + k] = sqrt(acc);
            all += acc;
        }
        if (total_out) total_out[m] = sqrt(all);
    }
}

/*
 * T steps in a row: g is [T][M][stride]; lr and clip_bound are [T].
 * masks_out (may be NULL) receives the sync mask of every step.
 */
void desloc_oracle_run(const desloc_oracle_cfg *c, int64_t t0, int64_t T, const double *lr,
                       const double *clip_bound, int64_t n, int64_t stride, float *x, float *u,
                       float *v, const float *g, uint32_t *masks_out) {
    for (int64_t s = 0; s < T; ++s) {
        const float *gs = g + (size_t)s * (size_t)c->M * (size_t)stride;
        uint32_t mk = desloc_oracle_step(c, t0 + s, lr[s], clip_bound ? clip_bound[s] : 0.0, n,
                                         stride, x, u, v, gs);
        if (masks_out) masks_out[s] = mk;
    }
}
