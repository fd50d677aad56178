// Batched fitting of the throughput-model parameters theta_sys (Sec. 4.1, "online model
// fitting"): for every job, minimise the root mean squared logarithmic error between
// Eq. 11 and the observed (a, m, s, T_iter) tuples, with alpha, beta >= 0 and gamma in
// [1, 10].  The paper uses L-BFGS-B on one CPU core per job; here one warp fits one job with a
// projected Levenberg-Marquardt iteration in double precision (lanes split the observations,
// the 7 x 7 normal equations are reduced by shuffles and solved by lane 0).
#include "common.cuh"

namespace {

constexpr int NP = 7;   // alpha_grad, beta_grad, alpha_local, beta_local, alpha_node, beta_node, gamma

struct FitArgs {
  const int32_t *offset;   // [J + 1] observations of job j are offset[j] .. offset[j + 1]
  const int32_t *k, *n, *m, *s;
  const float *t;
  const float *theta0;     // [J][7]
  const uint8_t *frozen;   // [J] bit i set: parameter i is held at its starting value, or NULL
  int J, max_iters;
  float *theta_out;        // [J][7]
  float *loss_out;         // [J]
};

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// T_iter of Eq. 11 and, optionally, its gradient with respect to the seven parameters.
__device__ double t_iter_model(const double th[NP], int K, int N, int m, int s, double *grad) {
  const double tg = th[0] + th[1] * (double)m;
  double ts = 0.0;
  int cls = -1;   // 0: local pair, 1: node pair
  if (K >= 2) {
    cls = (N == 1) ? 0 : 1;
    ts = th[2 + 2 * cls] + th[3 + 2 * cls] * (double)(K - 2);
  }
  const double g = th[6];
  double ov = tg, dov_dtg = 1.0, dov_dts = 0.0, dov_dg = 0.0;
  if (ts > 0.0 && tg > 0.0) {
    const double a = pow(tg, g), b = pow(ts, g), sum = a + b;
    ov = pow(sum, 1.0 / g);
    dov_dtg = pow(tg / ov, g - 1.0);
    dov_dts = pow(ts / ov, g - 1.0);
    dov_dg = ov * (-log(sum) / (g * g) + (a * log(tg) + b * log(ts)) / (g * sum));
  } else if (ts > 0.0) {   // tg == 0
    ov = ts; dov_dtg = 0.0; dov_dts = 1.0;
  }
  if (grad) {
    for (int i = 0; i < NP; ++i) grad[i] = 0.0;
    const double dp_dtg = (double)s + dov_dtg;
    grad[0] = dp_dtg;
    grad[1] = dp_dtg * (double)m;
    if (cls >= 0) {
      grad[2 + 2 * cls] = dov_dts;
      grad[3 + 2 * cls] = dov_dts * (double)(K - 2);
    }
    grad[6] = dov_dg;
  }
  return (double)s * tg + ov;
}

// sum of squared log residuals over the job's observations (all lanes get the total)
__device__ double sum_sq(const FitArgs &a, int lo, int hi, const double th[NP], int lane) {
  double acc = 0.0;
  for (int i = lo + lane; i < hi; i += 32) {
    const double p = t_iter_model(th, a.k[i], a.n[i], a.m[i], a.s[i], nullptr);
    const double r = log1p(p) - log1p((double)a.t[i]);
    acc += r * r;
  }
  return warp_sum_d(acc);
}

__global__ void __launch_bounds__(128) fit_kernel(FitArgs a) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (j >= a.J) return;
  const int lo = a.offset[j], hi = a.offset[j + 1];
  const int n = hi - lo;
  const unsigned frozen = a.frozen ? a.frozen[j] : 0u;
  double th[NP], lb[NP], ub[NP];
  for (int i = 0; i < NP; ++i) {
    lb[i] = (i == 6) ? 1.0 : 0.0;
    ub[i] = (i == 6) ? 10.0 : 1e300;
    th[i] = fmin(fmax((double)a.theta0[(size_t)j * NP + i], lb[i]), ub[i]);
    if ((frozen >> i) & 1u) { th[i] = (double)a.theta0[(size_t)j * NP + i]; lb[i] = ub[i] = th[i]; }
  }
  if (n <= 0) {
    if (lane == 0) {
      for (int i = 0; i < NP; ++i) a.theta_out[(size_t)j * NP + i] = (float)th[i];
      a.loss_out[j] = 0.f;
    }
    return;
  }
  double S = sum_sq(a, lo, hi, th, lane);
  double lambda = 1e-3;
  for (int it = 0; it < a.max_iters; ++it) {
    // normal equations A = J^T J (upper triangle), g = J^T r
    double A[NP * (NP + 1) / 2], gv[NP];
    for (int i = 0; i < NP * (NP + 1) / 2; ++i) A[i] = 0.0;
    for (int i = 0; i < NP; ++i) gv[i] = 0.0;
    for (int o = lo + lane; o < hi; o += 32) {
      double grad[NP];
      const double p = t_iter_model(th, a.k[o], a.n[o], a.m[o], a.s[o], grad);
      const double r = log1p(p) - log1p((double)a.t[o]);
      const double w = 1.0 / (1.0 + p);
      int idx = 0;
      for (int x = 0; x < NP; ++x) {
        const double jx = grad[x] * w;
        gv[x] += jx * r;
        for (int y = x; y < NP; ++y) A[idx++] += jx * grad[y] * w;
      }
    }
    for (int i = 0; i < NP * (NP + 1) / 2; ++i) A[i] = warp_sum_d(A[i]);
    for (int i = 0; i < NP; ++i) gv[i] = warp_sum_d(gv[i]);

    bool accepted = false;
    for (int tries = 0; tries < 8 && !accepted; ++tries) {
      double cand[NP];
      if (lane == 0) {
        // free parameters: not frozen, and not sitting on a bound with the gradient pushing out
        bool free_[NP];
        for (int i = 0; i < NP; ++i)
          free_[i] = lb[i] < ub[i] && !((th[i] <= lb[i] && gv[i] > 0.0) || (th[i] >= ub[i] && gv[i] < 0.0));
        // damped system (A + lambda diag(A) + eps) d = -g on the free set, by Cholesky
        double Mx[NP][NP], d[NP];
        int idx = 0;
        for (int x = 0; x < NP; ++x)
          for (int y = x; y < NP; ++y) { Mx[x][y] = Mx[y][x] = A[idx++]; }
        for (int x = 0; x < NP; ++x) {
          if (!free_[x]) {
            for (int y = 0; y < NP; ++y) Mx[x][y] = Mx[y][x] = 0.0;
            Mx[x][x] = 1.0;
            d[x] = 0.0;
          } else {
            Mx[x][x] = Mx[x][x] * (1.0 + lambda) + 1e-30;
            d[x] = -gv[x];
          }
        }
        bool ok = true;
        for (int x = 0; x < NP && ok; ++x) {         // in-place Cholesky, lower triangle
          for (int y = 0; y <= x; ++y) {
            double sum = Mx[x][y];
            for (int z = 0; z < y; ++z) sum -= Mx[x][z] * Mx[y][z];
            if (x == y) {
              if (sum <= 0.0) { ok = false; break; }
              Mx[x][x] = sqrt(sum);
            } else {
              Mx[x][y] = sum / Mx[y][y];
            }
          }
        }
        if (ok) {
          for (int x = 0; x < NP; ++x) {             // forward, then backward substitution
            double sum = d[x];
            for (int z = 0; z < x; ++z) sum -= Mx[x][z] * d[z];
            d[x] = sum / Mx[x][x];
          }
          for (int x = NP - 1; x >= 0; --x) {
            double sum = d[x];
            for (int z = x + 1; z < NP; ++z) sum -= Mx[z][x] * d[z];
            d[x] = sum / Mx[x][x];
          }
        }
        for (int i = 0; i < NP; ++i) cand[i] = ok ? fmin(fmax(th[i] + d[i], lb[i]), ub[i]) : th[i];
      }
      for (int i = 0; i < NP; ++i) cand[i] = __shfl_sync(0xffffffffu, cand[i], 0);
      const double Sc = sum_sq(a, lo, hi, cand, lane);
      if (Sc < S) {
        const double gain = (S - Sc) / fmax(S, 1e-300);
        for (int i = 0; i < NP; ++i) th[i] = cand[i];
        S = Sc;
        lambda = fmax(lambda / 3.0, 1e-12);
        accepted = true;
        if (gain < 1e-12) it = a.max_iters;           // converged
      } else {
        lambda *= 4.0;
      }
    }
    if (!accepted) break;
  }
  if (lane == 0) {
    for (int i = 0; i < NP; ++i) a.theta_out[(size_t)j * NP + i] = (float)th[i];
    a.loss_out[j] = (float)sqrt(S / (double)n);
  }
}

}  // namespace

int launch_fit(sched_ctx *ctx, int32_t num_jobs, const int32_t *d_offset, const int32_t *d_k, const int32_t *d_n,
               const int32_t *d_m, const int32_t *d_s, const float *d_t, const float *d_theta0,
               const uint8_t *d_frozen, int32_t max_iters, float *d_theta_out, float *d_loss_out) {
  if (num_jobs == 0) return SCHED_OK;
  FitArgs a;
  a.offset = d_offset; a.k = d_k; a.n = d_n; a.m = d_m; a.s = d_s; a.t = d_t;
  a.theta0 = d_theta0; a.frozen = d_frozen; a.J = num_jobs; a.max_iters = max_iters;
  a.theta_out = d_theta_out; a.loss_out = d_loss_out;
  {
    TimedLaunch tl_(ctx, KK_FIT);
    fit_kernel<<<(num_jobs + 3) / 4, 128, 0, ctx->stream>>>(a);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}
