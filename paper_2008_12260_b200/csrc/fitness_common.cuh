// Pieces of the fitness evaluation (Eq. 14) shared by the dense fitness kernel and the
// fused small-problem generation kernel, so that both produce identical bits: the term of
// one row, the reduction of a block's terms in a fixed order, and the final power mean.
#pragma once

#include "common.cuh"

enum { MODE_POW = 0, MODE_ARITH = 1, MODE_HARM = 2, MODE_GEO = 3, MODE_SQRT = 4 };

inline int fitness_mode(float p) {
  return (p == 1.f) ? MODE_ARITH : (p == -1.f) ? MODE_HARM : (p == 0.f) ? MODE_GEO
         : (p == 0.5f) ? MODE_SQRT : MODE_POW;
}

struct TermParams {
  const float *table;     // speedup [J][k_max+1][n_max+1]
  const float *pen;       // [J] factor applied to rows that differ from the current one, or NULL
  const uint8_t *active;  // [J] or NULL
  int k_max, n_max, mode;
  float p, floor_;
};

// Table position of SPEEDUP_j at (K, N), both clamped into the table.
__device__ __forceinline__ size_t fitness_table_index(const TermParams &tp, int j, int K, int N) {
  K = min(K, tp.k_max);
  N = min(N, tp.n_max);
  return ((size_t)j * (tp.k_max + 1) + K) * (tp.n_max + 1) + N;
}

// x_j^p from the looked-up speedup x and the job's penalty factor (used when the row changed):
// re-allocation penalty, floor, and the form that the mode sums (x, 1/x, ln x, sqrt x or x^p).
__device__ __forceinline__ float fitness_term_with(const TermParams &tp, float x, float pen, bool changed) {
  if (tp.pen && changed) x *= pen;
  x = fmaxf(x, tp.floor_);
  switch (tp.mode) {
    case MODE_ARITH: return x;
    case MODE_HARM: return 1.f / x;
    case MODE_GEO: return logf(x);
    case MODE_SQRT: return sqrtf(x);
    default: return powf(x, tp.p);
  }
}

__device__ __forceinline__ float fitness_term_of(const TermParams &tp, int j, float x, bool changed) {
  return fitness_term_with(tp, x, (tp.pen && changed) ? tp.pen[j] : 1.f, changed);
}

// x_j^p of one row (SPEEDUP looked up at (K, N), re-allocation penalty, floor).
__device__ __forceinline__ float fitness_term(const TermParams &tp, int j, int K, int N, bool changed) {
  return fitness_term_of(tp, j, __ldg(tp.table + fitness_table_index(tp, j, K, N)), changed);
}

// Sum and count of the terms s_term[0 .. nrows) of the active rows j_first + i, in a fixed
// order that depends only on nrows and the block size: thread t adds rows t, t + blockDim,
// ... in double, then a shuffle tree per warp and the warps in index order.  Result valid
// in thread 0.  Must be called by the whole block (256 threads), after a __syncthreads()
// that made s_term visible.
__device__ __forceinline__ void block_term_sum(const float *s_term, int nrows, int j_first,
                                               const uint8_t *active, double &sum, double &count) {
  __shared__ double s_acc[8];
  __shared__ int s_cnt[8];
  double acc = 0.0;
  int cnt = 0;
  for (int i = threadIdx.x; i < nrows; i += blockDim.x) {
    if (!active || active[j_first + i]) {
      acc += (double)s_term[i];
      cnt += 1;
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    acc += __shfl_xor_sync(0xffffffffu, acc, off);
    cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { s_acc[warp] = acc; s_cnt[warp] = cnt; }
  __syncthreads();
  sum = 0.0;
  count = 0.0;
  if (threadIdx.x == 0) {
    int n = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { sum += s_acc[w]; n += s_cnt[w]; }
    count = (double)n;
  }
}

// ((1/J) sum x^p)^(1/p) from the summed terms; 0 when no job is active.
__device__ __forceinline__ float fitness_finalise(int mode, float p, double sum, double count) {
  if (count == 0.0) return 0.f;
  const double mean = sum / count;
  double f;
  switch (mode) {
    case MODE_ARITH: f = mean; break;
    case MODE_HARM: f = 1.0 / mean; break;
    case MODE_GEO: f = exp(mean); break;
    case MODE_SQRT: f = mean * mean; break;
    default: f = pow(mean, 1.0 / (double)p); break;
  }
  return (float)f;
}

constexpr int FITNESS_MAX_ROWS_PER_BLOCK = 2048;
