/*
 * ssm_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * Plain, slow, sequential fp64 CPU definition of the selective state-space scan (S6): only tests, the smoke
 * check and the benchmark's cpu_baseline / reference arm may call it.  It shares no code with the CUDA path.
 *
 * What it computes, per batch b and channel d independently (Section 2 "Structure and Dimensions": the SSM is
 * applied independently to each channel, A is diagonal and stored as N numbers per channel):
 *
 *   discretization (Eq. 4, Algorithm 2 step 5)   a[t,n]    = exp(delta[t] * A[d,n])
 *                                                bbar[t,n] = delta[t] * B[b,t,n]                     (default rule)
 *                                      or (ZOH)  bbar[t,n] = (exp(delta[t]*A[d,n]) - 1) / A[d,n] * B[b,t,n]
 *   recurrence (Eq. 2a, Algorithm 2 step 6)      h[t,n]    = a[t,n] * h[t-1,n] + bbar[t,n] * x[t],  h[0,n] = h0 or 0
 *   readout (Eq. 2b) plus skip term              s[t]      = sum_n C[b,t,n] * h[t,n] + D_skip[d] * x[t]
 *   gate (Section 3.4, the SiLU branch of the block multiplies the SSM output)
 *                                                out[t]    = s[t] * z[t] / (1 + exp(-z[t]))
 *
 * The method is an exact reorganisation of this definition, so the oracle is the definition itself: one time
 * step after another, states ascending in n, no blocking, no fusion, no reordering.
 *
 * The backward functions are the analytic adjoint of the same definition for loss = sum(dout * out) (the paper
 * prints no backward formulas; these follow from the chain rule through the four lines above):
 *   ds[t]   = dout[t] * silu(z[t]);        dz[t] = dout[t] * s[t] * silu'(z[t]),  silu'(z) = sig(z) (1 + z (1 - sig(z)))
 *   lam[t,n] = C[t,n] ds[t] + a[t+1,n] lam[t+1,n],  lam[L+1] = 0
 *   dC[t,n] += ds[t] h[t,n];   dD += ds[t] x[t];   dB[t,n] += lam[t,n] delta[t] x[t]
 *   dx[t]   = ds[t] D_skip + delta[t] sum_n lam[t,n] B[t,n]
 *   w[t,n]  = lam[t,n] h[t-1,n] a[t,n];   ddelta[t] = sum_n w[t,n] A[n] + x[t] sum_n lam[t,n] B[t,n];   dA[n] += w[t,n] delta[t]
 * With the ZOH rule write bbar = E B with the input gain E(delta, A) = (exp(delta A) - 1) / A (E = delta at A = 0),
 * whose partial derivatives are dE/ddelta = a and dE/dA = (delta a - E) / A (delta^2 / 2 at A = 0).  Then
 *   dB[t,n] += lam E x;   dx[t] = ds D_skip + sum_n lam E B;
 *   ddelta[t] = sum_n w A + x sum_n lam a B;   dA[n] += w delta + lam (dE/dA) B x.
 * With an initial state h0 and an adjoint dh_last flowing into the last state from outside (a later piece of the
 * same sequence), h[0] = h0, the reverse recurrence starts from a[L+1] lam[L+1] := dh_last, and the gradient of h0 is
 * dh0[n] = a[1,n] lam[1,n].
 * With the softplus switch the input is the pre-activation v, delta = softplus(v + delta_bias[d]), ddelta is the
 * gradient of v (the line above times sigmoid(v + delta_bias[d])) and dbias[d] = sum over batch and time of ddelta.
 * Sums over channels (dB, dC) and over batch (dA, dD) are taken in a fixed order that does not depend on the
 * number of threads: channels are grouped in blocks of ORACLE_CH_BLOCK, each block accumulates in ascending channel
 * order into its own buffer, and the buffers are added in ascending block order.
 *
 * All pins (LTI convolution, lower-triangular matrix form, cumulative sum at A = 0, the gating theorem, finite
 * differences, invariants, chunk splitting, operator folding) live in tests/test_oracle_pins.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_CH_BLOCK 64

typedef struct {
  int32_t batch, L, D, N;
  int32_t has_z;      /* 0: out = s (no gate) */
  int32_t has_dskip;  /* 0: skip term absent */
  int32_t zoh_bbar;   /* 1: zero-order-hold B-bar of Eq. 4 instead of delta * B */
  int32_t softplus;   /* 1: `delta` holds the pre-activation v and the step size is softplus(v + delta_bias[d])
                         (Algorithm 2 step 4: Delta = tau_Delta(Parameter + s_Delta(x)), tau_Delta = softplus) */
  int32_t nthreads;   /* <= 0: all available */
} oracle_dims_t;

static int pick_threads(const oracle_dims_t* p) {
#ifdef _OPENMP
  return p->nthreads > 0 ? p->nthreads : omp_get_max_threads();
#else
  (void)p;
  return 1;
#endif
}

int ssm_oracle_threads_available(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static inline double silu(double z) { return z / (1.0 + exp(-z)); }
static inline double sigmoid(double z) { return 1.0 / (1.0 + exp(-z)); }
/* softplus(v) = log(1 + e^v), written so that neither large nor very negative v loses accuracy */
static inline double softplus(double v) { return (v > 0.0 ? v : 0.0) + log1p(exp(-fabs(v))); }
/* input gain of the ZOH rule (Eq. 4 for diagonal A): E = (exp(dt A) - 1) / A, and its derivative in A */
static inline double zoh_gain(double dt, double An) { return An != 0.0 ? expm1(dt * An) / An : dt; }
static inline double zoh_gain_dA(double dt, double An) {
  const double xx = dt * An;
  if (fabs(xx) < 1e-3) /* (x e^x - e^x + 1) / x^2 = 1/2 + x/3 + x^2/8 + x^3/30 + ... : no cancellation near 0 */
    return dt * dt * (0.5 + xx * (1.0 / 3.0 + xx * (0.125 + xx * (1.0 / 30.0 + xx / 144.0))));
  return (dt * exp(xx) - expm1(xx) / An) / An;
}

/* ------------------------------------------------------------------------------------------------------------
 * The two entry-point families differ only in the storage type of the (batch, L, *) inputs.
 * ---------------------------------------------------------------------------------------------------------- */
#define DEFINE_ORACLE(SUFFIX, REAL)                                                                              \
  /* forward: out (batch,L,D); optional s_pre (pre-gate readout, batch,L,D); optional h_last (batch,D,N) */      \
  int ssm_oracle_fwd_##SUFFIX(const oracle_dims_t* p, const REAL* x, const REAL* delta, const double* A,         \
                              const REAL* B, const REAL* C, const double* D_skip, const REAL* z,                 \
                              const double* h0, const double* delta_bias, double* out, double* s_pre,            \
                              double* h_last) {                                                                  \
    if (!p || p->batch < 1 || p->L < 1 || p->D < 1 || p->N < 1) return 1;                                         \
    const int64_t L = p->L, D = p->D, N = p->N;                                                                  \
    const int64_t items = (int64_t)p->batch * D;                                                                 \
    const int nt = pick_threads(p);                                                                              \
    (void)nt;                                                                                                    \
    _Pragma("omp parallel for schedule(dynamic, 8) num_threads(nt)")                                             \
    for (int64_t it = 0; it < items; ++it) {                                                                     \
      const int64_t b = it / D, d = it % D;                                                                      \
      double h[p->N];                                                                                            \
      for (int64_t n = 0; n < N; ++n) h[n] = h0 ? h0[(b * D + d) * N + n] : 0.0;                                 \
      for (int64_t t = 0; t < L; ++t) {                                                                          \
        const int64_t e = (b * L + t) * D + d;                                                                   \
        const double dv = (double)delta[e] + (delta_bias ? delta_bias[d] : 0.0);                                 \
        const double dt = p->softplus ? softplus(dv) : dv, u = (double)x[e];                                     \
        const REAL* Bt = B + (b * L + t) * N;                                                                    \
        const REAL* Ct = C + (b * L + t) * N;                                                                    \
        double s = 0.0;                                                                                          \
        for (int64_t n = 0; n < N; ++n) {                                                                        \
          const double An = A[d * N + n];                                                                        \
          const double a = exp(dt * An);                                                                         \
          double bbar;                                                                                           \
          if (p->zoh_bbar) bbar = zoh_gain(dt, An) * (double)Bt[n];                                              \
          else             bbar = dt * (double)Bt[n];                                                            \
          h[n] = a * h[n] + bbar * u;                                                                            \
          s += (double)Ct[n] * h[n];                                                                             \
        }                                                                                                        \
        if (p->has_dskip) s += D_skip[d] * u;                                                                    \
        if (s_pre) s_pre[e] = s;                                                                                 \
        out[e] = p->has_z ? s * silu((double)z[e]) : s;                                                          \
      }                                                                                                          \
      if (h_last) for (int64_t n = 0; n < N; ++n) h_last[(b * D + d) * N + n] = h[n];                            \
    }                                                                                                            \
    return 0;                                                                                                    \
  }                                                                                                              \
                                                                                                                 \
  /* backward: every output is overwritten; dD and dz may be NULL */                                             \
  int ssm_oracle_bwd_##SUFFIX(const oracle_dims_t* p, const REAL* x, const REAL* delta, const double* A,         \
                              const REAL* B, const REAL* C, const double* D_skip, const REAL* z,                 \
                              const REAL* dout, const double* delta_bias, const double* h0,                    \
                              const double* dh_last, double* dx, double* ddelta, double* dA, double* dB,       \
                              double* dC, double* dD, double* dz, double* dbias, double* dh0) {                  \
    if (!p || p->batch < 1 || p->L < 1 || p->D < 1 || p->N < 1) return 1;                                         \
    const int64_t L = p->L, D = p->D, N = p->N, NB = p->batch;                                                   \
    const int64_t nblk = (D + ORACLE_CH_BLOCK - 1) / ORACLE_CH_BLOCK;                                            \
    const int64_t items = NB * nblk;                                                                             \
    const int nt = pick_threads(p);                                                                              \
    (void)nt;                                                                                                    \
    double* dA_part = (double*)calloc((size_t)(NB * D * N), sizeof(double));     /* [b][d][n] */                 \
    double* dD_part = (double*)calloc((size_t)(NB * D), sizeof(double));         /* [b][d]    */                 \
    double* dbias_part = (double*)calloc((size_t)(NB * D), sizeof(double));      /* [b][d]    */                 \
    double* dBC_part = (double*)calloc((size_t)(items * L * N * 2), sizeof(double)); /* [b][blk][2][t][n] */     \
    int fail = (!dA_part || !dD_part || !dBC_part || !dbias_part);                                                              \
    if (!fail) {                                                                                                 \
      _Pragma("omp parallel for schedule(dynamic, 1) num_threads(nt)")                                           \
      for (int64_t it = 0; it < items; ++it) {                                                                   \
        const int64_t b = it / nblk, blk = it % nblk;                                                            \
        const int64_t d0 = blk * ORACLE_CH_BLOCK, d1 = (d0 + ORACLE_CH_BLOCK < D) ? d0 + ORACLE_CH_BLOCK : D;    \
        double* dBp = dBC_part + it * L * N * 2;                                                                 \
        double* dCp = dBp + L * N;                                                                               \
        double* hs = (double*)malloc((size_t)((L + 1) * N) * sizeof(double));  /* h[0..L][n] */                  \
        double* as = (double*)malloc((size_t)((L + 1) * N) * sizeof(double));  /* a[1..L][n] */                  \
        double* ss = (double*)malloc((size_t)(L + 1) * sizeof(double));        /* s[1..L] */                     \
        double lam[p->N];                                                                                        \
        for (int64_t d = d0; d < d1; ++d) {                                                                      \
          for (int64_t n = 0; n < N; ++n) hs[n] = h0 ? h0[(b * D + d) * N + n] : 0.0;                            \
          for (int64_t t = 1; t <= L; ++t) {                                                                     \
            const int64_t e = (b * L + (t - 1)) * D + d;                                                         \
            const double dv = (double)delta[e] + (delta_bias ? delta_bias[d] : 0.0);                             \
            const double dt = p->softplus ? softplus(dv) : dv, u = (double)x[e];                                 \
            const REAL* Bt = B + (b * L + (t - 1)) * N;                                                          \
            const REAL* Ct = C + (b * L + (t - 1)) * N;                                                          \
            double s = 0.0;                                                                                      \
            for (int64_t n = 0; n < N; ++n) {                                                                    \
              const double a = exp(dt * A[d * N + n]);                                                           \
              as[t * N + n] = a;                                                                                 \
              const double E = p->zoh_bbar ? zoh_gain(dt, A[d * N + n]) : dt;                                    \
              hs[t * N + n] = a * hs[(t - 1) * N + n] + E * (double)Bt[n] * u;                                   \
              s += (double)Ct[n] * hs[t * N + n];                                                                \
            }                                                                                                    \
            if (p->has_dskip) s += D_skip[d] * u;                                                                \
            ss[t] = s;                                                                                           \
          }                                                                                                      \
          for (int64_t n = 0; n < N; ++n) lam[n] = dh_last ? dh_last[(b * D + d) * N + n] : 0.0;                 \
          double dD_acc = 0.0, dbias_acc = 0.0;                                                                  \
          for (int64_t t = L; t >= 1; --t) {                                                                     \
            const int64_t e = (b * L + (t - 1)) * D + d;                                                         \
            const double dv = (double)delta[e] + (delta_bias ? delta_bias[d] : 0.0);                             \
            const double dt = p->softplus ? softplus(dv) : dv, u = (double)x[e], g = (double)dout[e];            \
            const REAL* Bt = B + (b * L + (t - 1)) * N;                                                          \
            const REAL* Ct = C + (b * L + (t - 1)) * N;                                                          \
            double ds;                                                                                           \
            if (p->has_z) {                                                                                      \
              const double zz = (double)z[e], sg = sigmoid(zz);                                                  \
              ds = g * zz * sg;                                                                                  \
              if (dz) dz[e] = g * ss[t] * sg * (1.0 + zz * (1.0 - sg));                                          \
            } else {                                                                                             \
              ds = g;                                                                                            \
              if (dz) dz[e] = 0.0;                                                                               \
            }                                                                                                    \
            /* lamEB = sum lam E B (input gradient), lamGB = sum lam (dE/ddelta) B (step-size gradient) */     \
            double lamEB = 0.0, lamGB = 0.0, wA = 0.0;                                                           \
            for (int64_t n = 0; n < N; ++n) {                                                                    \
              /* lam currently holds a[t+1] * lam[t+1] (zero for t = L) */                                       \
              const double l = (double)Ct[n] * ds + lam[n];                                                      \
              const double An = A[d * N + n], a = as[t * N + n];                                                 \
              const double E = p->zoh_bbar ? zoh_gain(dt, An) : dt;                                              \
              const double dE_ddt = p->zoh_bbar ? a : 1.0;                                                       \
              const double dE_dA = p->zoh_bbar ? zoh_gain_dA(dt, An) : 0.0;                                      \
              dCp[(t - 1) * N + n] += ds * hs[t * N + n];                                                        \
              dBp[(t - 1) * N + n] += l * E * u;                                                                 \
              lamEB += l * E * (double)Bt[n];                                                                    \
              lamGB += l * dE_ddt * (double)Bt[n];                                                               \
              const double w = l * hs[(t - 1) * N + n] * a;                                                      \
              wA += w * An;                                                                                      \
              dA_part[(b * D + d) * N + n] += w * dt + l * dE_dA * (double)Bt[n] * u;                            \
              lam[n] = a * l;                                                                                    \
            }                                                                                                    \
            dx[e] = (p->has_dskip ? ds * D_skip[d] : 0.0) + lamEB;                                               \
            /* with the softplus, ddelta is the gradient of the pre-activation: d softplus(v)/dv = sigmoid(v) */ \
            ddelta[e] = (wA + u * lamGB) * (p->softplus ? sigmoid(dv) : 1.0);                                    \
            dbias_acc += ddelta[e];                                                                              \
            dD_acc += ds * u;                                                                                    \
          }                                                                                                      \
          if (dh0) for (int64_t n = 0; n < N; ++n) dh0[(b * D + d) * N + n] = lam[n];                            \
          dD_part[b * D + d] = dD_acc;                                                                           \
          dbias_part[b * D + d] = dbias_acc;                                                                     \
        }                                                                                                        \
        free(hs); free(as); free(ss);                                                                            \
      }                                                                                                          \
      /* fixed-order second stage */                                                                             \
      _Pragma("omp parallel for schedule(static) num_threads(nt)")                                               \
      for (int64_t bt = 0; bt < NB * L; ++bt) {                                                                  \
        const int64_t b = bt / L, t = bt % L;                                                                    \
        for (int64_t n = 0; n < N; ++n) {                                                                        \
          double sb = 0.0, sc = 0.0;                                                                             \
          for (int64_t blk = 0; blk < nblk; ++blk) {                                                             \
            const double* q = dBC_part + (b * nblk + blk) * L * N * 2;                                           \
            sb += q[t * N + n];                                                                                  \
            sc += q[L * N + t * N + n];                                                                          \
          }                                                                                                      \
          dB[bt * N + n] = sb;                                                                                   \
          dC[bt * N + n] = sc;                                                                                   \
        }                                                                                                        \
      }                                                                                                          \
      for (int64_t d = 0; d < D; ++d) {                                                                          \
        for (int64_t n = 0; n < N; ++n) {                                                                        \
          double sa = 0.0;                                                                                       \
          for (int64_t b = 0; b < NB; ++b) sa += dA_part[(b * D + d) * N + n];                                   \
          dA[d * N + n] = sa;                                                                                    \
        }                                                                                                        \
        if (dD) {                                                                                                \
          double sd = 0.0;                                                                                       \
          for (int64_t b = 0; b < NB; ++b) sd += dD_part[b * D + d];                                             \
          dD[d] = p->has_dskip ? sd : 0.0;                                                                       \
        }                                                                                                        \
        if (dbias) {                                                                                             \
          double sb = 0.0;                                                                                       \
          for (int64_t b = 0; b < NB; ++b) sb += dbias_part[b * D + d];                                          \
          dbias[d] = sb;                                                                                         \
        }                                                                                                        \
      }                                                                                                          \
    }                                                                                                            \
    free(dA_part); free(dD_part); free(dBC_part); free(dbias_part);                                                                \
    return fail ? 2 : 0;                                                                                         \
  }

DEFINE_ORACLE(f64, double)
DEFINE_ORACLE(f32, float)
