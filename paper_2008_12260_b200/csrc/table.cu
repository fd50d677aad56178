// Speedup-table builder: goodput sweep over the (m, s) grid (Eq. 4-11, 13) and
// normalisation by the fair-share goodput (Eq. 15).
//
// The goodput of an allocation depends on the allocation only through K = SUM(a) and
// whether one or several nodes are occupied (Eq. 9), so the sweep runs once per
// (job, K, class) with class in {local, node}; a second kernel broadcasts the class
// results along the N axis of the [J][K][N] tables and divides by the fair-share entry.
#include <algorithm>

#include "common.cuh"

namespace {

struct JobPtrs {
  const float *alpha_grad, *beta_grad, *alpha_local, *beta_local, *alpha_node, *beta_node;
  const float *gamma, *phi, *m0, *m_max_total;
};

__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// (T_grad^g + T_sync^g)^(1/g) in ratio form: hi * (1 + (lo/hi)^g)^(1/g).  Both exponent
// arguments stay in [-inf, 1], so the approximate lg2/ex2 keep ~1e-7 relative accuracy.
__device__ __forceinline__ float overlap_time(float tg, float ts, float gamma, float inv_gamma) {
  if (ts <= 0.f) return tg;
  const float hi = fmaxf(tg, ts), lo = fminf(tg, ts);
  const float r = __fdividef(lo, hi);
  const float x = ex2_approx(gamma * lg2_approx(r));
  return hi * ex2_approx(lg2_approx(1.f + x) * inv_gamma);
}

// A candidate optimum: goodput = num / den; tie = (s << 16) | grid index (smaller wins).
struct Best {
  float num, den;
  uint32_t tie;
};

__device__ __forceinline__ bool beats(const Best &a, const Best &b) {
  const float l = a.num * b.den, r = b.num * a.den;
  return (l > r) || (l == r && a.num > 0.f && a.tie < b.tie);
}

// One warp per (job, K, class).  Lane l owns grid indices l, l+32, ... (MQ of them per
// pass), held in registers while the warp sweeps s.  Goodput is kept as num/den and
// compared by cross-multiplication:
//   num = M = K m (s+1),  den = T_iter * (phi + M) / (phi + M0)  =>  num/den = THROUGHPUT * EFFICIENCY.
template <int MQ>
__global__ void __launch_bounds__(256)
goodput_sweep_kernel(JobPtrs jp, const int32_t *__restrict__ m_grid,
                     const int32_t *__restrict__ pairs, int npairs, int k_max, int Gm, int Gs,
                     float one, float zero, float *__restrict__ gmax, uint16_t *__restrict__ amax) {
  const int lane = threadIdx.x & 31;
  // blockIdx.x = job; the block's warps walk the list of (K, class) pairs that exist on
  // this cluster (pairs[] = K * 2 + class, built on the host)
  const int j = blockIdx.x;
  const int pi = blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pi >= npairs) return;
  const int pr = pairs[pi];
  const int cls = pr & 1, K = pr >> 1;
  const int KD = k_max + 1;
  const size_t out = ((size_t)j * KD + K) * 2 + cls;

  const float a_g = jp.alpha_grad[j], b_g = jp.beta_grad[j];
  const float gamma = jp.gamma[j], inv_gamma = 1.f / gamma;
  const float phi = jp.phi[j], M0 = jp.m0[j], Mmax = jp.m_max_total[j];
  float ts = 0.f;
  if (K >= 2) {
    const float a = cls ? jp.alpha_node[j] : jp.alpha_local[j];
    const float b = cls ? jp.beta_node[j] : jp.beta_local[j];
    ts = fmaf(b, (float)(K - 2), a);
  }
  const float rinv = 1.f / (phi + M0);   // (phi + M) * rinv = 1 / EFFICIENCY
  const float c0 = phi * rinv;
  const float Kf = (float)K;

  Best best = {0.f, 1.f, 0xFFFFFFFFu};
  for (int base = 0; base < Gm; base += 32 * MQ) {
    // Per grid point m of this lane, with u = s + 1:
    //   T_iter = ta + u tg,  1/EFFICIENCY = c0 + u kr  (kr = K m / (phi + M0)),
    //   goodput = K m * u / den(u),  den(u) = (ta + u tg)(c0 + u kr).
    // den(u)/u is convex in u, so goodput is unimodal in s for a fixed m.  The loop therefore
    // tracks, per m, the maximiser over ALL s (a chain of its own, no masking); the window
    // M0 <= K m u <= Mmax is a contiguous range of u, and the masked maximum is at the
    // unmasked maximiser clamped into that range.
    float tg[MQ], ta[MQ], kr[MQ], bu[MQ], bd[MQ];
#pragma unroll
    for (int q = 0; q < MQ; ++q) {
      const int i = base + lane + 32 * q;
      const float mf = (i < Gm) ? (float)m_grid[(size_t)j * Gm + i] : 1.f;
      tg[q] = fmaf(b_g, mf, a_g);
      ta[q] = overlap_time(tg[q], ts, gamma, inv_gamma) - tg[q];
      kr[q] = Kf * mf * rinv;
      bu[q] = 0.f;
      bd[q] = 1.f;
    }
    float u = 1.f;
    if (MQ >= 2) {
      // two grid points per instruction: sm_100's packed fp32 FMA / MUL work on register
      // pairs and halve the issue slots of the arithmetic (same roundings as the scalar ops)
      constexpr int H = MQ >= 2 ? MQ / 2 : 1;
      float2 tg2[H], ta2[H], kr2[H], bu2[H], bd2[H];
#pragma unroll
      for (int h = 0; h < H; ++h) {
        tg2[h] = make_float2(tg[2 * h], tg[2 * h + (MQ >= 2)]);
        ta2[h] = make_float2(ta[2 * h], ta[2 * h + (MQ >= 2)]);
        kr2[h] = make_float2(kr[2 * h], kr[2 * h + (MQ >= 2)]);
        bu2[h] = make_float2(0.f, 0.f);
        bd2[h] = make_float2(1.f, 1.f);
      }
      const float2 c02 = make_float2(c0, c0);
#pragma unroll 4
      for (int s = 0; s < Gs; ++s, u += 1.f) {
        const float2 u2 = make_float2(u, u);
#pragma unroll
        for (int h = 0; h < H; ++h) {
          const float2 den2 = __fmul2_rn(__ffma2_rn(u2, tg2[h], ta2[h]), __ffma2_rn(u2, kr2[h], c02));
          const float2 l2 = __fmul2_rn(u2, bd2[h]);
          const float2 r2 = __fmul2_rn(bu2[h], den2);
          // per half: if (l > r) { bu = u; bd = den; } with the moves as predicated FMAs
          // (x * 1 + 0, run-time 1 and 0): compares and selects share the half-rate integer
          // pipe, and this form measured faster than plain selects
          asm("{\n"
              " .reg .pred pa, pb;\n"
              " setp.gt.f32 pa, %4, %6;\n"
              " setp.gt.f32 pb, %5, %7;\n"
              " @pa fma.rn.f32 %0, %8, %11, %12;\n"
              " @pa fma.rn.f32 %2, %9, %11, %12;\n"
              " @pb fma.rn.f32 %1, %8, %11, %12;\n"
              " @pb fma.rn.f32 %3, %10, %11, %12;\n"
              "}"
              : "+f"(bu2[h].x), "+f"(bu2[h].y), "+f"(bd2[h].x), "+f"(bd2[h].y)
              : "f"(l2.x), "f"(l2.y), "f"(r2.x), "f"(r2.y), "f"(u), "f"(den2.x), "f"(den2.y), "f"(one), "f"(zero));
        }
      }
#pragma unroll
      for (int h = 0; h < H; ++h) {
        bu[2 * h] = bu2[h].x; bd[2 * h] = bd2[h].x;
        bu[2 * h + (MQ >= 2)] = bu2[h].y; bd[2 * h + (MQ >= 2)] = bd2[h].y;
      }
    } else {
#pragma unroll 4
      for (int s = 0; s < Gs; ++s, u += 1.f) {
        const float den = fmaf(u, tg[0], ta[0]) * fmaf(u, kr[0], c0);
        // if (u * bd > bu * den) { bu = u; bd = den; }   -- u/den > bu/bd
        asm("{\n"
            " .reg .pred pb;\n"
            " .reg .f32 l, r;\n"
            " mul.f32 l, %2, %1;\n"
            " mul.f32 r, %0, %3;\n"
            " setp.gt.f32 pb, l, r;\n"
            " @pb fma.rn.f32 %0, %2, %4, %5;\n"
            " @pb fma.rn.f32 %1, %3, %4, %5;\n"
            "}"
            : "+f"(bu[0]), "+f"(bd[0])
            : "f"(u), "f"(den), "f"(one), "f"(zero));
      }
    }
#pragma unroll
    for (int q = 0; q < MQ; ++q) {
      const int i = base + lane + 32 * q;
      if (i >= Gm) continue;
      const float km = Kf * (float)m_grid[(size_t)j * Gm + i];
      // integer range of u with M0 <= km u <= Mmax (products are exact integers below 2^24)
      // approximate quotients are enough: the four exact product tests below correct an
      // off-by-one in either direction
      const float rkm = __frcp_rn(km);
      float ulo = ceilf(M0 * rkm), uhi = floorf(Mmax * rkm);
      if (km * (ulo - 1.f) >= M0) ulo -= 1.f;
      if (km * ulo < M0) ulo += 1.f;
      if (km * (uhi + 1.f) <= Mmax) uhi += 1.f;
      if (km * uhi > Mmax) uhi -= 1.f;
      ulo = fmaxf(ulo, 1.f);
      uhi = fminf(uhi, (float)Gs);
      if (ulo > uhi) continue;
      const float us = fminf(fmaxf(bu[q], ulo), uhi);
      Best b;
      b.num = km * us;
      b.den = (us == bu[q]) ? bd[q] : fmaf(us, tg[q], ta[q]) * fmaf(us, kr[q], c0);
      b.tie = ((uint32_t)(us - 1.f) << 16) | (uint32_t)i;
      if (beats(b, best)) best = b;
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    Best o;
    o.num = __shfl_xor_sync(0xffffffffu, best.num, off);
    o.den = __shfl_xor_sync(0xffffffffu, best.den, off);
    o.tie = __shfl_xor_sync(0xffffffffu, best.tie, off);
    if (beats(o, best)) best = o;
  }
  if (lane == 0) {
    const bool found = best.num > 0.f;
    gmax[out] = found ? best.num / best.den : 0.f;
    amax[out] = found ? (uint16_t)((best.tie & 0xFFFFu) * Gs + (best.tie >> 16)) : (uint16_t)0xFFFFu;
  }
}

// The (m, s) search as the paper words it (Sec. 4.3): candidate total batch sizes M are given;
// per candidate, per_gpu = ceil(M / K), s = ceil(per_gpu / m_max) - 1 (the fewest accumulation
// steps that fit the per-GPU limit), m = ceil(per_gpu / (s + 1)), and the batch actually run
// is M' = K m (s + 1), feasible when M0 <= M' <= M_max.  A non-adaptive job has the single
// candidate M0 and EFFICIENCY fixed to 1 (Sec. 4.2).  One warp per (job, K, class), lanes over
// the candidates; all feasibility decisions are integer.
__global__ void __launch_bounds__(256)
msample_sweep_kernel(JobPtrs jp, const int32_t *__restrict__ m_samples, const int32_t *__restrict__ m_max_gpu,
                     const uint8_t *__restrict__ adaptive, const int32_t *__restrict__ pairs, int npairs,
                     int k_max, int G, float *__restrict__ gmax, uint16_t *__restrict__ amax) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x;
  const int pi = blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (pi >= npairs) return;
  const int pr = pairs[pi];
  const int cls = pr & 1, K = pr >> 1;
  const size_t out = ((size_t)j * (k_max + 1) + K) * 2 + cls;
  const float a_g = jp.alpha_grad[j], b_g = jp.beta_grad[j];
  const float gamma = jp.gamma[j], inv_gamma = 1.f / gamma;
  const float phi = jp.phi[j], M0 = jp.m0[j], Mmax = jp.m_max_total[j];
  const bool adapt = !adaptive || adaptive[j];
  const int mmax = m_max_gpu[j];
  float ts = 0.f;
  if (K >= 2) {
    const float a = cls ? jp.alpha_node[j] : jp.alpha_local[j];
    const float b = cls ? jp.beta_node[j] : jp.beta_local[j];
    ts = fmaf(b, (float)(K - 2), a);
  }
  const float rinv = adapt ? 1.f / (phi + M0) : 0.f;   // (c0 + M rinv) = 1 / EFFICIENCY; 1 when fixed
  const float c0 = adapt ? phi * rinv : 1.f;
  Best best = {0.f, 1.f, 0xFFFFFFFFu};
  const int ns = adapt ? G : 1;
  if (mmax >= 1) {
    for (int i = lane; i < ns; i += 32) {
      const long long M = adapt ? (long long)m_samples[(size_t)j * G + i] : (long long)M0;
      if (M < 1) continue;
      long long s, m;
      if (M <= (1ll << 30)) {          // 32-bit divisions (the usual case) are several times cheaper
        const unsigned Mu = (unsigned)M, Ku = (unsigned)K, mu = (unsigned)mmax;
        const unsigned per_gpu = (Mu + Ku - 1u) / Ku;
        const unsigned su = (per_gpu + mu - 1u) / mu - 1u;
        s = su;
        m = (per_gpu + su) / (su + 1u);
      } else {
        const long long per_gpu = (M + K - 1) / K;
        s = (per_gpu + mmax - 1) / mmax - 1;
        m = (per_gpu + s) / (s + 1);
      }
      const float Mrun = (float)((long long)K * m * (s + 1));
      if (Mrun < M0 || Mrun > Mmax) continue;
      const float tg = fmaf(b_g, (float)m, a_g);
      const float tit = fmaf((float)s, tg, overlap_time(tg, ts, gamma, inv_gamma));
      Best b;
      b.num = Mrun;
      b.den = tit * fmaf(Mrun, rinv, c0);
      b.tie = (uint32_t)i;
      if (beats(b, best)) best = b;
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    Best o;
    o.num = __shfl_xor_sync(0xffffffffu, best.num, off);
    o.den = __shfl_xor_sync(0xffffffffu, best.den, off);
    o.tie = __shfl_xor_sync(0xffffffffu, best.tie, off);
    if (beats(o, best)) best = o;
  }
  if (lane == 0) {
    const bool found = best.num > 0.f;
    gmax[out] = found ? best.num / best.den : 0.f;
    amax[out] = found ? (uint16_t)best.tie : (uint16_t)0xFFFFu;
  }
}

__device__ __forceinline__ bool kn_valid(int K, int N, int k_max, int n_max,
                                         const int32_t *__restrict__ kfit) {
  return N >= 1 && N <= n_max && K >= N && K <= k_max && K <= kfit[N];
}

// Broadcast the class results along N and divide by the fair-share goodput (Eq. 15).
// Block = one job's slab of (k_max + 1) x (n_max + 1) entries, walked in memory order (thread
// t takes entries t, t + 256, ...; its (K, N) advance without divisions), so every store is
// coalesced whatever the slab's width.
// gden: the class results that hold the fair-share goodput (the two-class sweep's; the table of
// the rack class is normalised by the same goodput); min_n: entries with fewer nodes stay empty
// (1 for the two-class table, 2 for the rack class, which always takes the second class of gmax).
__global__ void __launch_bounds__(256)
speedup_expand_kernel(const float *__restrict__ gmax, const uint16_t *__restrict__ amax,
                      const float *__restrict__ gden, int min_n,
                      const int32_t *__restrict__ kfit, const int32_t *__restrict__ fair_k,
                      const int32_t *__restrict__ fair_n, int j_first, int k_max, int n_max,
                      float *__restrict__ goodput, float *__restrict__ speedup,
                      uint16_t *__restrict__ argmax) {
  const int KD = k_max + 1, ND = n_max + 1;
  const int j = j_first + blockIdx.x;
  const int kf = fair_k[j], nf = fair_n[j];
  float denom = 0.f;
  if (kn_valid(kf, nf, k_max, n_max, kfit)) denom = gden[((size_t)j * KD + kf) * 2 + (nf >= 2 ? 1 : 0)];
  const int entries = KD * ND;
  const int step_k = (int)blockDim.x / ND, step_n = (int)blockDim.x % ND;
  int K = (int)threadIdx.x / ND, N = (int)threadIdx.x % ND;
  // the job's own pieces of every array, so that the loop indexes with 32-bit offsets
  const float *gj = gmax + (size_t)j * KD * 2;
  const uint16_t *aj = amax + (size_t)j * KD * 2;
  float *gout = goodput ? goodput + (size_t)j * entries : nullptr;
  uint16_t *aout = argmax ? argmax + (size_t)j * entries : nullptr;
  float *sout = speedup + (size_t)j * entries;
  for (int e = threadIdx.x; e < entries; e += blockDim.x) {
    float g = 0.f, sp = 0.f;
    uint16_t a = 0xFFFFu;
    if (N >= min_n && K >= N && K <= __ldg(kfit + N)) {
      const int src = K * 2 + (N >= 2 ? 1 : 0);
      g = gj[src];
      a = aj[src];
      if (denom > 0.f) sp = g / denom;   // empty entries stay 0 without a division
    }
    if (gout) gout[e] = g;
    if (aout) aout[e] = a;
    sout[e] = sp;
    K += step_k;
    N += step_n;
    if (N >= ND) { N -= ND; ++K; }
  }
}

// REALLOC_FACTOR_j(delta) = (T_j - R_j delta) / (T_j + delta), clamped to [0, 1].
__global__ void realloc_factor_kernel(const float *__restrict__ age, const int32_t *__restrict__ restarts,
                                      float delta, int J, float *__restrict__ out) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= J) return;
  const float T = age[j], R = (float)restarts[j];
  float f = (T - R * delta) / (T + delta);
  if (!(f >= 0.f)) f = 0.f;
  out[j] = fminf(f, 1.f);
}

// Goodput-driven auto-scaling rule (Sec. 5.3): one thread per job.  All products are
// rounded one by one (no contraction): the comparisons decide integers.
__global__ void autoscale_kernel(const float *__restrict__ goodput, const int32_t *__restrict__ cur_nodes,
                                 int J, int k_max, int n_max, int gpn, float U, float L,
                                 int32_t *__restrict__ target_nodes) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= J) return;
  const int KD = k_max + 1, ND = n_max + 1;
  const float *g = goodput + (size_t)j * KD * ND;
  const float g1 = g[ND + 1];
  const int n = cur_nodes[j];
  const int limit = min(n_max, k_max / gpn);
  int target = n;
  if (n >= 1 && n <= limit && g1 > 0.f) {
    const float ideal_u = __fmul_rn(__fmul_rn(U, (float)(n * gpn)), g1);
    if (g[(size_t)(n * gpn) * ND + n] > ideal_u) {
      for (int t = n + 1; t <= limit; ++t) {
        const float ideal_l = __fmul_rn(__fmul_rn(L, (float)(t * gpn)), g1);
        if (g[(size_t)(t * gpn) * ND + t] >= ideal_l) target = t;
      }
    }
  }
  target_nodes[j] = target;
}

}  // namespace

int launch_autoscale(sched_ctx *ctx, const float *d_goodput, const int32_t *d_cur_nodes, int gpn, float U, float L,
                     int32_t *d_target_nodes) {
  const int J = ctx->cfg.num_jobs;
  if (J == 0) return SCHED_OK;
  autoscale_kernel<<<(J + 127) / 128, 128, 0, ctx->stream>>>(d_goodput, d_cur_nodes, J, ctx->cfg.k_max,
                                                             ctx->cfg.n_max, gpn, U, L, d_target_nodes);
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

static int launch_expand(sched_ctx *ctx, const sched_jobs *jobs, float *d_goodput, float *d_speedup,
                         uint16_t *d_argmax, bool rack_class = false) {
  const sched_config &c = ctx->cfg;
  const int J = c.num_jobs;
  for (int j0 = 0; j0 < J; j0 += 65535) {      // at most 65535 jobs per launch
    const unsigned grid = (unsigned)std::min(65535, J - j0);
    {
      TimedLaunch tl_(ctx, KK_EXPAND);
      speedup_expand_kernel<<<grid, 256, 0, ctx->stream>>>(rack_class ? ctx->d_gmax_rack : ctx->d_gmax,
                                                           rack_class ? ctx->d_amax_rack : ctx->d_amax, ctx->d_gmax,
                                                           rack_class ? 2 : 1, ctx->d_kfit, jobs->fair_k, jobs->fair_n,
                                                           j0, c.k_max, c.n_max, d_goodput, d_speedup, d_argmax);
    }
    SCHED_LAUNCH_CHECK(ctx);
  }
  return SCHED_OK;
}

int launch_speedup_table(sched_ctx *ctx, const sched_jobs *jobs, float *d_goodput, float *d_speedup,
                         uint16_t *d_argmax) {
  const sched_config &c = ctx->cfg;
  const int J = c.num_jobs;
  if (J == 0) return SCHED_OK;
  JobPtrs jp = {jobs->alpha_grad, jobs->beta_grad, jobs->alpha_local, jobs->beta_local,
                jobs->alpha_node, jobs->beta_node, jobs->gamma, jobs->phi, jobs->m0,
                jobs->m_max_total};
  const int mq = (c.grid_m + 31) / 32;
  if (ctx->num_pairs > 0) {
    dim3 grid((unsigned)J, (unsigned)((ctx->num_pairs + 7) / 8));
#define SWEEP(MQ)                                                                              \
  TimedLaunch tl_(ctx, KK_SWEEP);                                                              \
  goodput_sweep_kernel<MQ><<<grid, 256, 0, ctx->stream>>>(                                     \
      jp, jobs->m_grid, ctx->d_pairs, ctx->num_pairs, c.k_max, c.grid_m, c.grid_s, 1.f, 0.f,   \
      ctx->d_gmax, ctx->d_amax)
    if (mq <= 1) { SWEEP(1); }
    else if (mq == 2) { SWEEP(2); }
    else { SWEEP(4); }
#undef SWEEP
    SCHED_LAUNCH_CHECK(ctx);
  }
  return launch_expand(ctx, jobs, d_goodput, d_speedup, d_argmax);
}

// Tables of the rack class (allocations whose nodes lie in two or more racks): the sweep of the
// node class with the rack pair in the node pair's place; needs the two-class sweep's results in
// d_gmax for the fair-share goodput, so that sweep runs first.
int launch_speedup_table_rack(sched_ctx *ctx, const sched_jobs *jobs, const float *d_alpha_rack,
                              const float *d_beta_rack, float *d_goodput, float *d_speedup, uint16_t *d_argmax) {
  const sched_config &c = ctx->cfg;
  const int J = c.num_jobs;
  if (J == 0) return SCHED_OK;
  const size_t n = (size_t)J * ctx->KD * 2;
  if (!ctx->d_gmax_rack) {
    SCHED_CUDA_CHECK(ctx, cudaMalloc((void **)&ctx->d_gmax_rack, sizeof(float) * n));
    SCHED_CUDA_CHECK(ctx, cudaMalloc((void **)&ctx->d_amax_rack, sizeof(uint16_t) * n));
    ctx->scratch_epoch++;
  }
  SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->d_gmax_rack, 0, sizeof(float) * n, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->d_amax_rack, 0xFF, sizeof(uint16_t) * n, ctx->stream));
  const int mq = (c.grid_m + 31) / 32;
  if (ctx->num_pairs > 0) {
    dim3 grid((unsigned)J, (unsigned)((ctx->num_pairs + 7) / 8));
    for (int pass = 0; pass < 2; ++pass) {
      JobPtrs jp = {jobs->alpha_grad, jobs->beta_grad, jobs->alpha_local, jobs->beta_local,
                    pass ? d_alpha_rack : jobs->alpha_node, pass ? d_beta_rack : jobs->beta_node, jobs->gamma,
                    jobs->phi, jobs->m0, jobs->m_max_total};
      float *gm = pass ? ctx->d_gmax_rack : ctx->d_gmax;
      uint16_t *am = pass ? ctx->d_amax_rack : ctx->d_amax;
#define SWEEP(MQ)                                                                              \
  TimedLaunch tl_(ctx, KK_SWEEP);                                                              \
  goodput_sweep_kernel<MQ><<<grid, 256, 0, ctx->stream>>>(                                     \
      jp, jobs->m_grid, ctx->d_pairs, ctx->num_pairs, c.k_max, c.grid_m, c.grid_s, 1.f, 0.f, gm, am)
      if (mq <= 1) { SWEEP(1); }
      else if (mq == 2) { SWEEP(2); }
      else { SWEEP(4); }
#undef SWEEP
      SCHED_LAUNCH_CHECK(ctx);
    }
  }
  return launch_expand(ctx, jobs, d_goodput, d_speedup, d_argmax, true);
}

int launch_speedup_table_msample(sched_ctx *ctx, const sched_jobs *jobs, const int32_t *d_m_samples, int G,
                                 const int32_t *d_m_max_gpu, const uint8_t *d_adaptive, float *d_goodput,
                                 float *d_speedup, uint16_t *d_argmax) {
  const sched_config &c = ctx->cfg;
  const int J = c.num_jobs;
  if (J == 0) return SCHED_OK;
  JobPtrs jp = {jobs->alpha_grad, jobs->beta_grad, jobs->alpha_local, jobs->beta_local,
                jobs->alpha_node, jobs->beta_node, jobs->gamma, jobs->phi, jobs->m0,
                jobs->m_max_total};
  if (ctx->num_pairs > 0) {
    dim3 grid((unsigned)J, (unsigned)((ctx->num_pairs + 7) / 8));
    {
      TimedLaunch tl_(ctx, KK_SWEEP);
      msample_sweep_kernel<<<grid, 256, 0, ctx->stream>>>(jp, d_m_samples, d_m_max_gpu, d_adaptive, ctx->d_pairs,
                                                          ctx->num_pairs, c.k_max, G, ctx->d_gmax, ctx->d_amax);
    }
    SCHED_LAUNCH_CHECK(ctx);
  }
  return launch_expand(ctx, jobs, d_goodput, d_speedup, d_argmax);
}

int launch_realloc_factor(sched_ctx *ctx, const sched_jobs *jobs, float *d_out) {
  const int J = ctx->cfg.num_jobs;
  if (J == 0) return SCHED_OK;
  {
  TimedLaunch tl_(ctx, KK_REALLOC);
  realloc_factor_kernel<<<(J + 127) / 128, 128, 0, ctx->stream>>>(jobs->age_sec, jobs->num_restarts,
                                                                   ctx->cfg.delta_sec, J, d_out);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}
