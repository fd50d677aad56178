// Population-search operators (Sec. 4.3): ranking, parent selection + row-wise crossover
// + row perturbation, and the repair that enforces node capacity and interference
// avoidance (Sec. 4.2).  Integer work only; all randomness comes from the counter-based
// stream, so every output is a pure function of the inputs.
//
// Three implementations of the same operators on dense matrices, chosen by shape:
//  * rows_kernel + cols_kernel (+ rank_kernel): the general pair - a warp per (candidate, job)
//    row through shared memory, then a thread per (candidate, node) column;
//  * rows2_kernel + colrepair_kernel: rows of whole 16-byte vectors and at most 512 nodes -
//    batched rows with fused column sums and occupant lists, a work list of violating nodes;
//    for at most 256 jobs the row kernel also does the column pass and the fitness (FUSE);
//  * generation_small_kernel: at most 256 jobs and 32 nodes inside a round - a thread per row.
// Rounds of more than 256 jobs do not use dense matrices for their generations at all (rowstore.cu).
#include "common.cuh"
#include "fitness_common.cuh"

namespace {

enum { ROWS_GENERATION = 0, ROWS_INIT = 1, ROWS_REPAIR = 2 };

// rank[i] = number of candidates ordered before i (fitness descending, index ascending)
__global__ void __launch_bounds__(128)
rank_kernel(const uint32_t *__restrict__ fitness_bits, int P, int32_t *__restrict__ rank,
            int32_t *__restrict__ order) {
  __shared__ uint32_t tile[128];
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t ki = (i < P) ? order_key(fitness_bits[i]) : 0u;
  int r = 0;
  for (int base = 0; base < P; base += 128) {
    const int o = base + threadIdx.x;
    tile[threadIdx.x] = (o < P) ? order_key(fitness_bits[o]) : 0u;
    __syncthreads();
    const int lim = min(128, P - base);
    for (int t = 0; t < lim; ++t) {
      const uint32_t ko = tile[t];
      r += (ko > ki || (ko == ki && base + t < i)) ? 1 : 0;
    }
    __syncthreads();
  }
  if (i < P) {
    rank[i] = r;
    order[r] = i;
  }
}

struct RowsArgs {
  const int16_t *src;       // parents [P][J][N], or the current allocation [J][N] (may be NULL), or dst
  int16_t *dst;             // children [count][J][N]
  const int16_t *cap;       // [N]
  const int32_t *k_cap;     // [J] or NULL
  const uint8_t *active;    // [J] or NULL
  const int32_t *rank;      // [P]   (generation mode)
  const int32_t *order;     // [P]
  const uint32_t *fitness_bits;  // [P] parents' fitness (generation mode)
  uint8_t *dflag;           // [count][J]
  const int16_t *cur;       // [J][N] current allocation for the summaries' "changed" bit, or NULL
  uint32_t *summ;           // [count][J] row summaries (batched kernels only), or NULL
  const uint32_t *summ_in;  // [P][J] summaries of the parents (generation mode), or NULL
  int mode, P, J, num_nodes, k_max, n_max, num_elite, count;
  uint32_t thr, gen, first_cand;
  RngKey key;
};

__global__ void __launch_bounds__(256) rows_kernel(RowsArgs a) {
  extern __shared__ __align__(16) int16_t s_rows[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long gw = (long long)blockIdx.x * (blockDim.x >> 5) + warp;
  if (gw >= (long long)a.count * a.J) return;
  const int cl = (int)(gw / a.J), j = (int)(gw % a.J);
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int NN = a.num_nodes;
  const int row_stride = (NN + 7) & ~7;
  int16_t *row = s_rows + (size_t)warp * row_stride;
  int16_t *out = a.dst + ((size_t)cl * a.J + j) * NN;
  const bool vec = ((NN & 7) == 0) && ((((uintptr_t)a.dst | (uintptr_t)a.src) & 15) == 0);

  if (a.active && !a.active[j]) {
    if (vec) for (int v = lane; v < NN / 8; v += 32) ((uint4 *)out)[v] = make_uint4(0, 0, 0, 0);
    else for (int n = lane; n < NN; n += 32) out[n] = 0;
    if (lane == 0) a.dflag[(size_t)cl * a.J + j] = 0;
    return;
  }

  // which row feeds this child row, and the perturbation draw
  const int16_t *src = nullptr;
  bool mutate = false;
  u32x4 mw = {0, 0, 0, 0};
  if (a.mode == ROWS_GENERATION) {
    int parent;
    if ((int)c < a.num_elite) {
      parent = a.order[c];
    } else {
      const u32x4 s = draw(a.key, 0u, c, a.gen, SLOT_SELECT);
      const int i0 = bounded(s.x, a.P), i1 = bounded(s.y, a.P);
      const int i2 = bounded(s.z, a.P), i3 = bounded(s.w, a.P);
      const int pa = a.rank[i0] <= a.rank[i1] ? i0 : i1;
      const int pb = a.rank[i2] <= a.rank[i3] ? i2 : i3;
      const u32x4 x = draw(a.key, (uint32_t)j, c, a.gen, SLOT_XOVER);
      parent = (x.x >> 31) ? pb : pa;
      mw = draw(a.key, (uint32_t)j, c, a.gen, SLOT_MUTATE);
      mutate = mw.x < a.thr;
    }
    src = a.src + ((size_t)parent * a.J + j) * NN;
  } else if (a.mode == ROWS_INIT) {
    src = a.src ? a.src + (size_t)j * NN : nullptr;
    if (c > 0) {
      mw = draw(a.key, (uint32_t)j, c, GEN_INIT, SLOT_INIT);
      mutate = mw.x < a.thr;
    }
  } else {
    src = out;
  }

  // load into shared memory, every entry forced into [0, capacity of its node]
  int K = 0, N = 0;
  if (!src) {
    for (int n = lane; n < row_stride; n += 32) row[n] = 0;
  } else if (vec) {
    for (int v = lane; v < NN / 8; v += 32) {
      uint4 x = __ldg((const uint4 *)src + v);
      const uint4 cp = __ldg((const uint4 *)a.cap + v);
      x.x = __vimin_s16x2_relu(x.x, __vimax_s16x2_relu(cp.x, 0u));
      x.y = __vimin_s16x2_relu(x.y, __vimax_s16x2_relu(cp.y, 0u));
      x.z = __vimin_s16x2_relu(x.z, __vimax_s16x2_relu(cp.z, 0u));
      x.w = __vimin_s16x2_relu(x.w, __vimax_s16x2_relu(cp.w, 0u));
      ((uint4 *)row)[v] = x;
      const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        K += (int)(w[q] & 0xFFFFu) + (int)(w[q] >> 16);
        N += ((w[q] & 0xFFFFu) != 0u) + ((w[q] >> 16) != 0u);
      }
    }
  } else {
    for (int n = lane; n < NN; n += 32) {
      const int cp = max((int)a.cap[n], 0);
      const int v = min(max((int)src[n], 0), cp);
      row[n] = (int16_t)v;
      K += v;
      N += v > 0;
    }
  }
  K = warp_sum(K);
  N = warp_sum(N);
  __syncwarp();

  if (mutate) {
    const uint32_t op = bounded(mw.y, 3u);
    if (op == 0u) {
      const int n = (int)bounded(mw.w, (uint32_t)NN);
      if (lane == 0) row[n] = (int16_t)min((int)row[n] + 1, max((int)a.cap[n], 0));
    } else if (N > 0) {
      const int ns = nth_occupied(row, NN, bounded(mw.z, (uint32_t)N), lane);
      if (op == 1u) {
        if (lane == 0) row[ns] = (int16_t)(row[ns] - 1);
      } else {
        const int nd = (int)bounded(mw.w, (uint32_t)NN);
        if (nd != ns && lane == 0) {
          row[nd] = (int16_t)min((int)row[nd] + (int)row[ns], max((int)a.cap[nd], 0));
          row[ns] = 0;
        }
      }
    }
    __syncwarp();
    K = 0; N = 0;
    for (int n = lane; n < NN; n += 32) { K += row[n]; N += row[n] > 0; }
    K = warp_sum(K);
    N = warp_sum(N);
  }

  // per-row caps: replicas above the job's cap leave from the highest node index down,
  // then occupied nodes beyond n_max are cleared from the highest index down
  int kc = a.k_cap ? a.k_cap[j] : a.k_max;
  kc = max(0, min(kc, a.k_max));
  if (K > kc || N > a.n_max) {
    if (lane == 0) {
      int excess = K - kc;
      for (int n = NN - 1; n >= 0 && excess > 0; --n) {
        const int take = min((int)row[n], excess);
        row[n] = (int16_t)(row[n] - take);
        excess -= take;
      }
      int occ = 0;
      for (int n = 0; n < NN; ++n) {
        if (row[n] > 0) {
          ++occ;
          if (occ > a.n_max) row[n] = 0;
        }
      }
      N = min(occ, a.n_max);
    }
    N = __shfl_sync(0xffffffffu, N, 0);
    __syncwarp();
  }

  if (vec) for (int v = lane; v < NN / 8; v += 32) ((uint4 *)out)[v] = ((const uint4 *)row)[v];
  else for (int n = lane; n < NN; n += 32) out[n] = row[n];
  if (lane == 0) a.dflag[(size_t)cl * a.J + j] = (N >= 2) ? 1 : 0;
}

struct ColsArgs {
  int16_t *pop;             // [count][J][N], repaired in place
  const uint8_t *dflag;     // [count][J]
  const int16_t *cap;
  int J, num_nodes, count;
  uint32_t gen, first_cand;
  RngKey key;
};

// One thread per (candidate, node).  Interference avoidance: of the jobs flagged as
// distributed that occupy the node, only the first in job order rotated by the node's
// draw stays.  Capacity: GPUs above the node's size are taken from its jobs in job order
// rotated by a second draw.
__global__ void __launch_bounds__(128) cols_kernel(ColsArgs a) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int cl = blockIdx.y;
  if (n >= a.num_nodes) return;
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int J = a.J, NN = a.num_nodes;
  int16_t *col = a.pop + (size_t)cl * J * NN + n;
  const uint8_t *df = a.dflag + (size_t)cl * J;
  int total = 0, nelig = 0;
#pragma unroll 8
  for (int j = 0; j < J; ++j) {
    const int v = col[(size_t)j * NN];
    total += v;
    nelig += (v > 0 && df[j]) ? 1 : 0;
  }
  const int cp = max((int)a.cap[n], 0);
  if (nelig <= 1 && total <= cp) return;
  if (nelig >= 2) {
    const int o = (int)bounded(draw(a.key, (uint32_t)n, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
    int keep = -1, best = J;
    for (int j = 0; j < J; ++j) {
      if (df[j] && col[(size_t)j * NN] > 0) {
        int t = j - o;
        if (t < 0) t += J;
        if (t < best) { best = t; keep = j; }
      }
    }
    for (int j = 0; j < J; ++j) {
      if (j != keep && df[j]) {
        const int v = col[(size_t)j * NN];
        if (v > 0) { total -= v; col[(size_t)j * NN] = 0; }
      }
    }
  }
  int excess = total - cp;
  if (excess > 0) {
    const int o = (int)bounded(draw(a.key, (uint32_t)n, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J);
    for (int t = 0; t < J && excess > 0; ++t) {
      int j = o + t;
      if (j >= J) j -= J;
      const int v = col[(size_t)j * NN];
      if (v > 0) {
        const int take = min(v, excess);
        col[(size_t)j * NN] = (int16_t)(v - take);
        excess -= take;
      }
    }
  }
}

// index of the best candidate (largest key, lowest index on ties) and its fitness
__global__ void __launch_bounds__(256)
best_index_kernel(const uint32_t *__restrict__ fitness_bits, int P, int32_t *__restrict__ best_idx,
                  float *__restrict__ best_fitness) {
  __shared__ unsigned long long s[256];
  unsigned long long best = 0ull;   // (key << 32) | (0xFFFFFFFF - index): larger is better
  for (int i = threadIdx.x; i < P; i += blockDim.x) {
    const unsigned long long v = ((unsigned long long)order_key(fitness_bits[i]) << 32) |
                                 (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
    best = v > best ? v : best;
  }
  s[threadIdx.x] = best;
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if ((int)threadIdx.x < off) s[threadIdx.x] = s[threadIdx.x] > s[threadIdx.x + off] ? s[threadIdx.x] : s[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const int idx = (int)(0xFFFFFFFFu - (uint32_t)(s[0] & 0xFFFFFFFFull));
    *best_idx = idx;
    if (best_fitness) *best_fitness = __uint_as_float(fitness_bits[idx]);
  }
}

__global__ void copy_best_kernel(const int16_t *__restrict__ pop, const int32_t *__restrict__ best_idx,
                                 size_t elems, int16_t *__restrict__ out) {
  const int16_t *src = pop + (size_t)(*best_idx) * elems;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < elems;
       i += (size_t)gridDim.x * blockDim.x)
    out[i] = src[i];
}


// ---------------------------------------------------------------------------------------
// Batched row kernel with fused column sums (rows of at most 64 16-byte vectors).
//
// A block owns 256 consecutive rows of one candidate, a warp 32 of them.  Each lane draws
// the crossover / perturbation words of "its" row once (32 Philox calls run side by side
// instead of one per warp), then the warp walks the 32 rows: one 16-byte load per lane and
// vector, clamp, row totals by shuffle, store.  Rows that are perturbed or break a row cap
// detour through shared memory.  While walking, every lane accumulates, for its own
// columns, the GPUs placed and the number of distributed jobs; the block's column partials
// go to scratch, so the column pass never re-reads the population.
// ---------------------------------------------------------------------------------------
// Occupants of a node recorded per (candidate, row batch, node); a node with more occupants in
// one batch than this falls back to scanning the column.
constexpr int OCC_SLOTS = 8;

struct Rows2Args {
  RowsArgs r;
  int32_t *colsum;   // [count][nbatch][num_nodes] GPUs placed on the node by the batch's rows
  int32_t *colelig;  // same shape: rows of the batch that are distributed and occupy the node
  unsigned int *list_count;  // length of the column work list (zeroed before this kernel)
  uint32_t *list;            // the work list: (candidate << 13 | node) of nodes that need repair
  unsigned int *cand_ticket; // [count] blocks of the candidate that have finished (self-resetting)
  int32_t *occ_count;        // [count][nbatch][num_nodes] rows of the batch that occupy the node
  uint32_t *occ_list;        // [count][nbatch][num_nodes][OCC_SLOTS] job | GPUs << 20 | distributed << 31
  int nbatch, lpr_log2;
  // Single-batch candidates (J <= 256): the block also does the column pass and the fitness of
  // its candidate, so a whole generation is one kernel.
  int fuse;
  TermParams tp;
  float *fitness_out;        // [count]
};

__device__ __forceinline__ uint4 clamp_vec(uint4 x, uint4 cp) {
  x.x = __vimin_s16x2_relu(x.x, cp.x);
  x.y = __vimin_s16x2_relu(x.y, cp.y);
  x.z = __vimin_s16x2_relu(x.z, cp.z);
  x.w = __vimin_s16x2_relu(x.w, cp.w);
  return x;
}

// K in the low 22 bits, occupied-node count in the high 10 (entries are >= 0 here)
__device__ __forceinline__ uint32_t row_partial(uint4 x) {
  int k = __dp2a_lo((int)x.x, 0x0101, 0);
  k = __dp2a_lo((int)x.y, 0x0101, k);
  k = __dp2a_lo((int)x.z, 0x0101, k);
  k = __dp2a_lo((int)x.w, 0x0101, k);
  const uint32_t o = __vimin_s16x2_relu(x.x, 0x00010001u) + __vimin_s16x2_relu(x.y, 0x00010001u) +
                     __vimin_s16x2_relu(x.z, 0x00010001u) + __vimin_s16x2_relu(x.w, 0x00010001u);
  return (uint32_t)k | (((o & 0xFFFFu) + (o >> 16)) << 22);
}

struct ColfixArgs {
  int16_t *pop;
  const uint8_t *dflag;
  const int16_t *cap;
  const int32_t *colsum, *colelig;
  uint32_t *summ;           // [count][J] row summaries to keep in step with the removals, or NULL
  const int16_t *cur;       // current allocation (for the summaries' differing-entries count), or NULL
  const int32_t *occ_count; // per (candidate, row batch, node) occupants recorded by the row kernel
  const uint32_t *occ_list;
  uint32_t *list;           // work list of (candidate << 13 | node) entries
  unsigned int *list_count;
  int J, num_nodes, nbatch;
  uint32_t gen, first_cand;
  RngKey key;
};

// A column-pass write A[j][n]: v_old -> v_new keeps row j's summary in step:
// K += v_new - v_old, N -= 1 if the entry became empty, and the count of entries that
// differ from the current allocation is adjusted.  The three fields never leave their
// ranges, so one wrapped 32-bit add does all three.
__device__ __forceinline__ void summ_update(const ColfixArgs &a, uint32_t *summ_c, int j, int n, int v_old, int v_new) {
  if (!summ_c) return;
  int d_diff = 0;
  if (a.cur) {
    const int cv = a.cur[(size_t)j * a.num_nodes + n];
    d_diff = (int)(v_new != cv) - (int)(v_old != cv);
  }
  const uint32_t delta = (uint32_t)(v_new - v_old) + ((uint32_t)((v_new == 0 && v_old > 0) ? -1 : 0) << 11) +
                         ((uint32_t)d_diff << 22);
  atomicAdd(summ_c + j, delta);
}

// Repair of one column by a whole warp (any J): interference, then capacity, each with a
// few passes over the column; loads are issued in batches so that they overlap.
__device__ __noinline__ void repair_column_any(const ColfixArgs &a, uint32_t *summ_c, int cl, int nn, int tot, int ne,
                                               int cap_n, int lane) {
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int J = a.J, NN = a.num_nodes;
  const uint8_t *df = a.dflag + (size_t)cl * J;
  {
    int16_t *col = a.pop + (size_t)cl * J * NN + nn;
    // the loops below first issue a batch of independent column loads, then work on them
    constexpr int U = 8;
    if (ne >= 2) {
      const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
      int best = J;
      for (int jb = 0; jb < J; jb += 32 * U) {
        int v[U], d[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
          const int j = jb + 32 * k + lane;
          v[k] = (j < J) ? (int)col[(size_t)j * NN] : 0;
          d[k] = (j < J) ? (int)df[j] : 0;
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
          if (d[k] && v[k] > 0) {
            int t = jb + 32 * k + lane - o;
            if (t < 0) t += J;
            best = min(best, t);
          }
        }
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, off));
      int keep = o + best;
      if (keep >= J) keep -= J;
      int removed = 0;
      for (int jb = 0; jb < J; jb += 32 * U) {
        int v[U], d[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
          const int j = jb + 32 * k + lane;
          v[k] = (j < J) ? (int)col[(size_t)j * NN] : 0;
          d[k] = (j < J) ? (int)df[j] : 0;
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
          const int j = jb + 32 * k + lane;
          if (d[k] && v[k] > 0 && j != keep) {
            col[(size_t)j * NN] = 0;
            removed += v[k];
            summ_update(a, summ_c, j, nn, v[k], 0);
          }
        }
      }
      tot -= warp_sum(removed);
    }
    int excess = tot - cap_n;
    if (excess > 0) {
      const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J);
      constexpr int C = 4;   // chunks of 32 jobs loaded together
      for (int t0 = 0; t0 < J && excess > 0; t0 += 32 * C) {
        int v[C], jj[C];
#pragma unroll
        for (int k = 0; k < C; ++k) {
          const int t = t0 + 32 * k + lane;
          int j = o + t;
          if (j >= J) j -= J;
          jj[k] = j;
          v[k] = (t < J) ? (int)col[(size_t)j * NN] : 0;
        }
#pragma unroll
        for (int k = 0; k < C; ++k) {
          if (excess <= 0) break;
          int s = v[k];                                // inclusive prefix over the 32 jobs
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, s, off);
            if (lane >= off) s += u;
          }
          const int take = min(v[k], max(excess - (s - v[k]), 0));
          if (take > 0) {
            col[(size_t)jj[k] * NN] = (int16_t)(v[k] - take);
            summ_update(a, summ_c, jj[k], nn, v[k], v[k] - take);
          }
          excess -= __shfl_sync(0xffffffffu, s, 31);
        }
      }
    }
  }
}

// Repair of one column from its occupants, one occupant per lane (entry = job | GPUs << 20 |
// distributed << 31 in the first have_n lanes): no pass over the column.
__device__ void repair_column_entries(const ColfixArgs &a, uint32_t *summ_c, int cl, int nn, int tot, int ne,
                                      int cap_n, int lane, uint32_t entry, int have_n) {
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int J = a.J, NN = a.num_nodes;
  const bool have = lane < have_n;
  const int j = (int)(entry & 0xFFFFFu);
  int v = have ? (int)((entry >> 20) & 0x7FFu) : 0;
  const bool dist = have && (entry >> 31);
  int16_t *col = a.pop + (size_t)cl * J * NN + nn;
  if (ne >= 2) {
    const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
    int t = J;
    if (dist && v > 0) { t = j - o; if (t < 0) t += J; }
    int best = t;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, off));
    int removed = 0;
    if (dist && v > 0 && t != best) {
      col[(size_t)j * NN] = 0;
      summ_update(a, summ_c, j, nn, v, 0);
      removed = v;
      v = 0;
    }
    tot -= warp_sum(removed);
  }
  const int excess = tot - cap_n;
  if (excess > 0) {
    const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J);
    int rot = 0x7fffffff;
    if (have) { rot = j - o; if (rot < 0) rot += J; }
    int ahead = 0;                       // GPUs of the occupants that come first in rotated order
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      const int rk = __shfl_sync(0xffffffffu, rot, k);
      const int vk = __shfl_sync(0xffffffffu, v, k);
      if (rk < rot) ahead += vk;
    }
    const int take = have ? min(v, max(excess - ahead, 0)) : 0;
    if (take > 0) {
      col[(size_t)j * NN] = (int16_t)(v - take);
      summ_update(a, summ_c, j, nn, v, v - take);
    }
  }
}

// Occupants gathered from the per-batch lists the row kernel left in global memory.  Falls
// back to the column scan when a batch overflowed its slots or the node has more than 32
// occupants.
__device__ void repair_column_list(const ColfixArgs &a, int cl, int nn, int tot, int ne, int cap_n, int lane) {
  const int NN = a.num_nodes;
  uint32_t *summ_c = a.summ ? a.summ + (size_t)cl * a.J : nullptr;
  uint32_t entry = 0;
  int have_n = 0;
  bool overflow = false;
  for (int b = 0; b < a.nbatch; ++b) {
    const size_t at = ((size_t)cl * a.nbatch + b) * NN + nn;
    const int cb = a.occ_count[at];
    overflow |= cb > OCC_SLOTS;
    const int take_n = min(cb, OCC_SLOTS);
    if (lane >= have_n && lane < have_n + take_n) entry = a.occ_list[at * OCC_SLOTS + (lane - have_n)];
    have_n += take_n;
  }
  if (overflow || have_n > 32) repair_column_any(a, summ_c, cl, nn, tot, ne, cap_n, lane);
  else repair_column_entries(a, summ_c, cl, nn, tot, ne, cap_n, lane, entry, have_n);
}

// VPL = 16-byte vectors per lane; a row is split over LPR = 1 << LPR_LOG2 lanes
// (LPR * VPL >= row_vecs, FULL when equal), so a warp works on 32 / LPR rows at a time.
template <int LPR_LOG2, int VPL, bool FULL, bool FUSE>
__global__ void __launch_bounds__(256, 4) rows2_kernel(Rows2Args aa) {
  const RowsArgs &a = aa.r;
  constexpr int MAXN = 8 * (1 << LPR_LOG2) * VPL;   // nodes this instantiation can hold
  constexpr int QCAP = 64;                          // vectors in a warp's occupant queue
  __shared__ __align__(16) int16_t s_row[8][MAXN];  // per-warp detour buffer
  __shared__ __align__(16) int16_t s_cap[MAXN];     // node sizes floored at 0
  __shared__ int32_t s_tot[MAXN], s_el[MAXN], s_cnt[MAXN];
  __shared__ uint32_t s_occ[MAXN * OCC_SLOTS];
  __shared__ int s_parent[2];
  __shared__ uint32_t s_summ[256];   // row summaries of the block's rows
  __shared__ float s_term[256];
  // per-warp queue of non-empty vectors waiting to be expanded into occupants
  __shared__ __align__(16) uint4 s_qvec[8][QCAP];
  __shared__ uint32_t s_qmeta[8][QCAP];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cl = blockIdx.y, batch = blockIdx.x;
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int NN = a.num_nodes, J = a.J;
  const int row_vecs = NN >> 3;
  constexpr int LPR = 1 << LPR_LOG2, RPI = 32 >> LPR_LOG2;        // lanes per row, rows per iteration
  const int grp = lane >> LPR_LOG2, sub = lane & (LPR - 1);
  const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << (grp * LPR));
  for (int i = threadIdx.x; i < NN; i += blockDim.x) {
    s_tot[i] = 0; s_el[i] = 0; s_cnt[i] = 0;
    s_cap[i] = (int16_t)max((int)a.cap[i], 0);
  }

  // ---- parents of this candidate (generation mode), found by the block itself -------------
  // rank(i) = number of candidates ordered before i (fitness descending, index ascending).
  // An elite child needs the candidate of rank c; any other child the better-ranked of two
  // random pairs, which the two candidates' own keys and indices decide.
  if (a.mode == ROWS_GENERATION) {
    const int P = a.P;
    if ((int)c < a.num_elite) {
      for (int i = threadIdx.x; i < P; i += blockDim.x) {
        const uint32_t ki = order_key(a.fitness_bits[i]);
        int rk = 0;
        for (int o = 0; o < P; ++o) {
          const uint32_t ko = order_key(__ldg(a.fitness_bits + o));
          rk += (ko > ki || (ko == ki && o < i)) ? 1 : 0;
        }
        if (rk == (int)c) s_parent[0] = s_parent[1] = i;
      }
    } else {
      const u32x4 sel = draw(a.key, 0u, c, a.gen, SLOT_SELECT);
      const int idx[4] = {(int)bounded(sel.x, P), (int)bounded(sel.y, P), (int)bounded(sel.z, P),
                          (int)bounded(sel.w, P)};
      if (threadIdx.x == 0) {
        uint32_t k4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) k4[q] = order_key(__ldg(a.fitness_bits + idx[q]));
        s_parent[0] = tournament_winner(k4[0], idx[0], k4[1], idx[1]);
        s_parent[1] = tournament_winner(k4[2], idx[2], k4[3], idx[3]);
      }
    }
  }
  __syncthreads();

  const int j0 = batch * 256 + warp * 32;
  const int nrows = min(32, J - j0);          // may be <= 0 for trailing warps
  // ---- per-lane set-up for row j0 + lane: 32 draws side by side -----------------------------
  uint32_t flags_l = 0;   // bit 0 perturb, bit 1 active, bit 2 row comes from the second parent, bits 3.. replica cap
  u32x4 mw = {0, 0, 0, 0};
  if (lane < nrows) {
    const int j = j0 + lane;
    const bool act = !a.active || a.active[j];
    int kc = a.k_cap ? a.k_cap[j] : a.k_max;
    kc = max(0, min(kc, a.k_max));
    bool mut = false, second = false;
    if (a.mode == ROWS_GENERATION) {
      if ((int)c >= a.num_elite) {
        const u32x4 x = draw(a.key, (uint32_t)j, c, a.gen, SLOT_XOVER);
        second = (x.x >> 31) != 0u;
        mw = draw(a.key, (uint32_t)j, c, a.gen, SLOT_MUTATE);
        mut = mw.x < a.thr;
      }
    } else if (a.mode == ROWS_INIT && c > 0) {
      mw = draw(a.key, (uint32_t)j, c, GEN_INIT, SLOT_INIT);
      mut = mw.x < a.thr;
    }
    flags_l = (mut ? 1u : 0u) | (act ? 2u : 0u) | (second ? 4u : 0u) | ((uint32_t)kc << 3);
  }

  // row j0 of the possible sources; per row only the offset r * NN is added
  const size_t roff0 = (size_t)j0 * NN;
  const int16_t *src_a = nullptr, *src_b = nullptr;
  if (a.mode == ROWS_GENERATION) {
    src_a = a.src + (size_t)s_parent[0] * J * NN + roff0;
    src_b = a.src + (size_t)s_parent[1] * J * NN + roff0;
  } else if (a.mode == ROWS_INIT) {
    src_a = src_b = a.src ? a.src + roff0 : nullptr;
  } else {
    src_a = src_b = a.dst + (size_t)cl * J * NN + roff0;
  }
  const int16_t *cur0 = a.cur ? a.cur + roff0 : nullptr;
  int16_t *dst0 = a.dst + (size_t)cl * J * NN + roff0;
  int16_t *row = s_row[warp];

  // Iterations are software-pipelined: the loads of the next RPI rows are issued before the
  // current ones are processed.
  // An unperturbed child row is a verbatim copy of a parent's row, whose summary (K, N, entries
  // differing from the current allocation; kept exact by the column pass) is already known:
  // such rows skip the row totals and the comparison with the current allocation.
  const bool inherit = !FUSE && a.mode == ROWS_GENERATION && a.summ_in != nullptr;
  const uint32_t *sin_a = inherit ? a.summ_in + (size_t)s_parent[0] * J + j0 : nullptr;
  const uint32_t *sin_b = inherit ? a.summ_in + (size_t)s_parent[1] * J + j0 : nullptr;
  uint4 raw[VPL];
  uint32_t pword = 0;
  auto fetch = [&](int r) {   // r = this lane's row within the warp's 32 (may be >= nrows)
    const uint32_t fl = __shfl_sync(0xffffffffu, flags_l, r & 31);
    const int16_t *src = (fl & 4u) ? src_b : src_a;
    const bool on = r < nrows && (fl & 2u) && src;
    const bool copy = inherit && !(fl & 1u);
    if (copy && on && sub == 0) pword = __ldg(((fl & 4u) ? sin_b : sin_a) + r);
#pragma unroll
    for (int q = 0; q < VPL; ++q) {
      const int v = sub + LPR * q;
      raw[q] = make_uint4(0, 0, 0, 0);
      if (on && (FULL || v < row_vecs)) raw[q] = __ldg((const uint4 *)(src + (size_t)r * NN) + v);
      // the matching piece of the current allocation is read late in the iteration: pull it
      // towards L1 now, without tying up registers
      if (cur0 && !copy && r < nrows && (FULL || v < row_vecs))
        asm volatile("prefetch.global.L1 [%0];" ::"l"((const uint4 *)(cur0 + (size_t)r * NN) + v));
    }
  };
  if (nrows > 0) fetch(grp);
  // Expands the queued vectors: entry e = (vector e / 8, half e % 8), one lane per entry.  Per
  // occupant: add to the node's GPU total and distributed-job count, record it in the
  // node's occupant list.
  auto flush_queue = [&](int count) {
    __syncwarp();
    for (int e = lane; e < count * 8; e += 32) {
      const uint32_t val = ((const uint16_t *)s_qvec[warp])[e];
      if (val) {
        const uint32_t meta = s_qmeta[warp][e >> 3];
        const int n = (int)((meta >> 20) & 0x7FFu) * 8 + (e & 7);
        atomicAdd(&s_tot[n], (int)val);
        if (meta >> 31) atomicAdd(&s_el[n], 1);
        const int slot = atomicAdd(&s_cnt[n], 1);
        if (slot < OCC_SLOTS) s_occ[n * OCC_SLOTS + slot] = (meta & 0xFFFFFu) | (val << 20) | (meta & 0x80000000u);
      }
    }
    __syncwarp();
  };

  for (int r0 = 0; r0 < nrows; r0 += RPI) {
    const int r = r0 + grp;                       // this lane's row
    const bool live = r < nrows;
    const uint32_t flags = __shfl_sync(0xffffffffu, flags_l, r & 31);
    const bool act = live && (flags & 2u);
    uint4 x[VPL];
#pragma unroll
    for (int q = 0; q < VPL; ++q) {
      const int v = sub + LPR * q;
      x[q] = make_uint4(0, 0, 0, 0);
      if (FULL || v < row_vecs) x[q] = clamp_vec(raw[q], ((const uint4 *)s_cap)[v]);
    }
    const bool copy = inherit && act && !(flags & 1u);       // uniform within the row's lanes
    const uint32_t pw = __shfl_sync(0xffffffffu, pword, grp << LPR_LOG2);
    if (r0 + RPI < nrows) fetch(r0 + RPI + grp);

    const bool compute = __any_sync(0xffffffffu, live && !copy);   // some row of this iteration needs totals
    int K = 0, N = 0;
    if (compute) {
      uint32_t part = 0;
#pragma unroll
      for (int q = 0; q < VPL; ++q) part += row_partial(x[q]);
      part = __reduce_add_sync(gmask, part);
      K = (int)(part & 0x3FFFFFu);
      N = (int)(part >> 22);
    }
    if (copy) { K = (int)(pw & 0x7FFu); N = (int)((pw >> 11) & 0x7FFu); }
    const int kc = (int)(flags >> 3);

    // rows that are perturbed or break a row cap take a detour through shared memory, one
    // row at a time with the whole warp
    unsigned need = __ballot_sync(0xffffffffu, act && !copy && sub == 0 && ((flags & 1u) || K > kc || N > a.n_max));
    while (need) {
      const int leader = __ffs(need) - 1;         // lane `leader` is sub 0 of the row's group
      need &= need - 1;
      const int g = leader >> LPR_LOG2;
      const int rr = r0 + g;
      const uint32_t rflags = __shfl_sync(0xffffffffu, flags, leader);
      int rK = __shfl_sync(0xffffffffu, K, leader), rN = __shfl_sync(0xffffffffu, N, leader);
      const int rkc = (int)(rflags >> 3);
      if (grp == g) {
#pragma unroll
        for (int q = 0; q < VPL; ++q)
          if (FULL || sub + LPR * q < row_vecs) ((uint4 *)row)[sub + LPR * q] = x[q];
      }
      __syncwarp();
      if (rflags & 1u) {
        const uint32_t m1 = __shfl_sync(0xffffffffu, mw.y, rr), m2 = __shfl_sync(0xffffffffu, mw.z, rr),
                       m3 = __shfl_sync(0xffffffffu, mw.w, rr);
        const uint32_t op = bounded(m1, 3u);
        if (op == 0u) {
          const int n = (int)bounded(m3, (uint32_t)NN);
          if (lane == 0) row[n] = (int16_t)min((int)row[n] + 1, (int)s_cap[n]);
        } else if (rN > 0) {
          const int ns = nth_occupied(row, NN, bounded(m2, (uint32_t)rN), lane);
          if (op == 1u) {
            if (lane == 0) row[ns] = (int16_t)(row[ns] - 1);
          } else {
            const int nd = (int)bounded(m3, (uint32_t)NN);
            if (nd != ns && lane == 0) {
              row[nd] = (int16_t)min((int)row[nd] + (int)row[ns], (int)s_cap[nd]);
              row[ns] = 0;
            }
          }
        }
        __syncwarp();
        rK = 0; rN = 0;
        for (int n = lane; n < NN; n += 32) { rK += row[n]; rN += row[n] > 0; }
        rK = __reduce_add_sync(0xffffffffu, rK);
        rN = __reduce_add_sync(0xffffffffu, rN);
      }
      if (rK > rkc || rN > a.n_max) {
        if (lane == 0) {
          int excess = rK - rkc;
          rK = min(rK, rkc);
          for (int n = NN - 1; n >= 0 && excess > 0; --n) {
            const int take = min((int)row[n], excess);
            row[n] = (int16_t)(row[n] - take);
            excess -= take;
          }
          int occ = 0;
          for (int n = 0; n < NN; ++n) {
            if (row[n] > 0) {
              ++occ;
              if (occ > a.n_max) { rK -= row[n]; row[n] = 0; }
            }
          }
          rN = min(occ, a.n_max);
        }
        rN = __shfl_sync(0xffffffffu, rN, 0);
        rK = __shfl_sync(0xffffffffu, rK, 0);
      }
      __syncwarp();
      if (grp == g) {
#pragma unroll
        for (int q = 0; q < VPL; ++q)
          if (FULL || sub + LPR * q < row_vecs) x[q] = ((const uint4 *)row)[sub + LPR * q];
        K = rK;
        N = rN;
      }
      __syncwarp();
    }

    // ---- store, column bookkeeping, row summary ---------------------------------------------
    const bool dist = N >= 2;
    int ndiff = 0;   // entries of this lane that differ from the current allocation
    int qn = 0;      // vectors queued by the warp in this iteration
    const int j = j0 + r;
#pragma unroll
    for (int q = 0; q < VPL; ++q) {
      const int v = sub + LPR * q;
      const bool in = live && (FULL || v < row_vecs);
      if (in) ((uint4 *)(dst0 + (size_t)r * NN))[v] = x[q];
      // Occupied nodes are few.  Vectors with any occupant are compacted into a per-warp
      // queue (ballot + popc, no atomics) and expanded below with one lane per entry.
      if (qn > QCAP - 32) { flush_queue(qn); qn = 0; }
      const bool nz = in && (x[q].x | x[q].y | x[q].z | x[q].w) != 0u;
      const unsigned bal = __ballot_sync(0xffffffffu, nz);
      if (nz) {
        const int pos = qn + __popc(bal & ((1u << lane) - 1u));
        s_qvec[warp][pos] = x[q];
        s_qmeta[warp][pos] = (uint32_t)j | ((uint32_t)v << 20) | (dist ? 0x80000000u : 0u);   // v < 64
      }
      qn += __popc(bal);
      if (cur0 && in && !copy) {
        const uint4 cx = __ldg((const uint4 *)(cur0 + (size_t)r * NN) + v);
        const uint4 d = make_uint4(x[q].x ^ cx.x, x[q].y ^ cx.y, x[q].z ^ cx.z, x[q].w ^ cx.w);
        if ((d.x | d.y | d.z | d.w) != 0u) {
          // entries on both sides are in [0, 32767], so each half of the xor is a non-negative
          // int16 and min(half, 1) counts the halves that differ
          const uint32_t dc = __vimin_s16x2_relu(d.x, 0x00010001u) + __vimin_s16x2_relu(d.y, 0x00010001u) +
                              __vimin_s16x2_relu(d.z, 0x00010001u) + __vimin_s16x2_relu(d.w, 0x00010001u);
          ndiff += (int)((dc & 0xFFFFu) + (dc >> 16));
        }
      }
    }
    flush_queue(qn);
    qn = 0;
    if (cur0 && compute) ndiff = __reduce_add_sync(gmask, ndiff);
    if (copy) ndiff = (int)(pw >> 22);
    if (live && sub == 0) {
      const bool on = (flags & 2u) != 0u;
      a.dflag[(size_t)cl * J + j] = (on && dist) ? 1 : 0;
      // row summary for the fitness: K | N << 11 | (entries that differ from current) << 22
      const uint32_t word = on ? ((uint32_t)K | ((uint32_t)N << 11) | ((uint32_t)ndiff << 22)) : 0u;
      if (FUSE) s_summ[warp * 32 + r] = word;
      if (!FUSE && a.summ) a.summ[(size_t)cl * J + j] = word;
    }
  }

  __syncthreads();
  if (FUSE) {
    // ---- the whole candidate lives in this block: column pass and fitness right here ---------
    ColfixArgs f;
    f.pop = a.dst; f.dflag = a.dflag; f.cap = a.cap; f.cur = a.cur;
    f.colsum = nullptr; f.colelig = nullptr; f.summ = nullptr; f.occ_count = nullptr; f.occ_list = nullptr;
    f.list = nullptr; f.list_count = nullptr;
    f.J = J; f.num_nodes = NN; f.nbatch = 1; f.gen = a.gen; f.first_cand = a.first_cand; f.key = a.key;
    for (int nb = warp * 32; nb < NN; nb += 256) {
      const int n = nb + lane;
      const int total = (n < NN) ? s_tot[n] : 0, nelig = (n < NN) ? s_el[n] : 0;
      const int cp = (n < NN) ? (int)s_cap[n] : 0;
      unsigned todo = __ballot_sync(0xffffffffu, n < NN && (nelig >= 2 || total > cp));
      while (todo) {
        const int srcl = __ffs(todo) - 1;
        todo &= todo - 1;
        const int nn = nb + srcl;
        const int tot_n = __shfl_sync(0xffffffffu, total, srcl), ne_n = __shfl_sync(0xffffffffu, nelig, srcl);
        const int cap_n = __shfl_sync(0xffffffffu, cp, srcl);
        const int have_n = s_cnt[nn];
        if (have_n > OCC_SLOTS) {
          repair_column_any(f, s_summ, cl, nn, tot_n, ne_n, cap_n, lane);
        } else {
          const uint32_t entry = (lane < have_n) ? s_occ[nn * OCC_SLOTS + lane] : 0u;
          repair_column_entries(f, s_summ, cl, nn, tot_n, ne_n, cap_n, lane, entry, have_n);
        }
        __syncwarp();
      }
    }
    __syncthreads();
    for (int j = threadIdx.x; j < J; j += blockDim.x) {
      if (!aa.tp.active || aa.tp.active[j]) {
        const uint32_t w = s_summ[j];
        s_term[j] = fitness_term(aa.tp, j, (int)(w & 0x7FFu), (int)((w >> 11) & 0x7FFu), (w >> 22) != 0u);
      }
    }
    __syncthreads();
    double tsum, tcount;
    block_term_sum(s_term, J, 0, aa.tp.active, tsum, tcount);
    if (threadIdx.x == 0) aa.fitness_out[cl] = fitness_finalise(aa.tp.mode, aa.tp.p, tsum, tcount);
    return;
  }
  // ---- column partials and occupant lists of the block -------------------------------------
  const size_t base = ((size_t)cl * aa.nbatch + batch) * NN;
  for (int i = threadIdx.x; i < NN; i += blockDim.x) {
    aa.colsum[base + i] = s_tot[i];
    aa.colelig[base + i] = s_el[i];
    aa.occ_count[base + i] = s_cnt[i];
    const int cnt = min(s_cnt[i], OCC_SLOTS);
    for (int k = 0; k < cnt; ++k) aa.occ_list[(base + i) * OCC_SLOTS + k] = s_occ[i * OCC_SLOTS + k];
  }
  // The last block of the candidate to get here adds the batch partials per node and appends
  // the nodes that hold two distributed jobs or exceed their size to the work list.
  __shared__ bool s_last_block;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned prev = atomicAdd(aa.cand_ticket + cl, 1u);
    s_last_block = (prev == (unsigned)aa.nbatch - 1u);
    if (s_last_block) aa.cand_ticket[cl] = 0u;
  }
  __syncthreads();
  if (s_last_block) {
    __threadfence();
    for (int n = threadIdx.x; n < NN; n += blockDim.x) {
      int total = 0, nelig = 0;
      for (int b = 0; b < aa.nbatch; ++b) {
        total += __ldcg(aa.colsum + ((size_t)cl * aa.nbatch + b) * NN + n);
        nelig += __ldcg(aa.colelig + ((size_t)cl * aa.nbatch + b) * NN + n);
      }
      if (nelig >= 2 || total > (int)s_cap[n]) {
        const unsigned slot = atomicAdd(aa.list_count, 1u);
        aa.list[slot] = ((uint32_t)cl << 13) | (uint32_t)n;      // n < 8192, cl < 65536
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Streaming row kernel: the row pass when no per-row summaries are wanted (the dense entry
// points called on their own) and a row is a power-of-two number of 16-byte vectors.
//
// Almost every entry of a population is zero and almost every row is copied unchanged, so the
// rows are moved as a stream - a warp reads its 32 rows as one flat run of vectors, four loads
// per lane in flight, and stores them straight back out - and only the vectors that hold
// something are looked at: they are compacted into a per-warp queue (ballot + popc) and
// expanded one lane per entry, once to get each row's K, N and whether any entry leaves
// [0, node size], and once more for the column totals and occupant lists.  A row that is
// perturbed, has an entry out of range or breaks a row cap is rebuilt in shared memory by the
// whole warp, written again, and its queue entries are replaced.  Same operators, draws and
// results as rows2_kernel; block and grid shapes, column partials and the work list are shared
// with it.
// ---------------------------------------------------------------------------------------
constexpr int STREAM_QCAP = 128;        // vectors a warp queues per tile

// dynamic shared memory of the streaming kernel: per-node arrays sized by the cluster
__host__ __device__ inline size_t stream_smem_bytes(int NN) {
  return (size_t)8 * NN * 2          // a row per warp (rebuilt rows)
         + (size_t)NN * 2            // node sizes
         + (size_t)NN * 4 * 3        // GPUs placed, distributed jobs, occupants per node
         + (size_t)NN * OCC_SLOTS * 4;
}

__global__ void __launch_bounds__(256, 4) rows_stream_kernel(Rows2Args aa) {
  const RowsArgs &a = aa.r;
  extern __shared__ __align__(16) unsigned char stream_smem[];
  const int NN = a.num_nodes, J = a.J;
  int16_t *s_rows = (int16_t *)stream_smem;                       // [8][NN] per-warp buffer for a row that is rebuilt
  int16_t *s_cap = s_rows + (size_t)8 * NN;                       // node sizes floored at 0
  int32_t *s_tot = (int32_t *)(s_cap + NN), *s_el = s_tot + NN, *s_cnt = s_el + NN;
  uint32_t *s_occ = (uint32_t *)(s_cnt + NN);
  __shared__ int s_parent[2];
  __shared__ __align__(16) uint4 s_qvec[8][STREAM_QCAP];
  __shared__ uint32_t s_qmeta[8][STREAM_QCAP];       // row (bits 0..4) | vector of the row (8..13) | alive (31)
  __shared__ int s_rowK[8][32], s_rowN[8][32], s_rowbad[8][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cl = blockIdx.y, batch = blockIdx.x;
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int row_vecs = NN >> 3;                      // a power of two, 1 .. 64
  const int rv_log2 = 31 - __clz(row_vecs);
  for (int i = threadIdx.x; i < NN; i += blockDim.x) {
    s_tot[i] = 0; s_el[i] = 0; s_cnt[i] = 0;
    s_cap[i] = (int16_t)max((int)a.cap[i], 0);
  }
  // ---- parents of this candidate (generation mode), found by the block itself (as rows2_kernel) ----
  if (a.mode == ROWS_GENERATION) {
    const int P = a.P;
    if ((int)c < a.num_elite) {
      for (int i = threadIdx.x; i < P; i += blockDim.x) {
        const uint32_t ki = order_key(a.fitness_bits[i]);
        int rk = 0;
        for (int o = 0; o < P; ++o) {
          const uint32_t ko = order_key(__ldg(a.fitness_bits + o));
          rk += (ko > ki || (ko == ki && o < i)) ? 1 : 0;
        }
        if (rk == (int)c) s_parent[0] = s_parent[1] = i;
      }
    } else {
      const u32x4 sel = draw(a.key, 0u, c, a.gen, SLOT_SELECT);
      const int idx[4] = {(int)bounded(sel.x, P), (int)bounded(sel.y, P), (int)bounded(sel.z, P),
                          (int)bounded(sel.w, P)};
      if (threadIdx.x == 0) {
        uint32_t k4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) k4[q] = order_key(__ldg(a.fitness_bits + idx[q]));
        s_parent[0] = tournament_winner(k4[0], idx[0], k4[1], idx[1]);
        s_parent[1] = tournament_winner(k4[2], idx[2], k4[3], idx[3]);
      }
    }
  }
  __syncthreads();

  const int j0 = batch * 256 + warp * 32;
  const int nrows = min(32, J - j0);          // may be <= 0 for trailing warps
  // ---- per-lane set-up for row j0 + lane: the row's draws, 32 side by side ---------------------
  bool act_l = false, mut_l = false, sec_l = false;
  int kc_l = 0;
  u32x4 mw = {0, 0, 0, 0};
  if (lane < nrows) {
    const int j = j0 + lane;
    act_l = !a.active || a.active[j];
    kc_l = max(0, min(a.k_cap ? a.k_cap[j] : a.k_max, a.k_max));
    if (a.mode == ROWS_GENERATION) {
      if ((int)c >= a.num_elite) {
        sec_l = (draw(a.key, (uint32_t)j, c, a.gen, SLOT_XOVER).x >> 31) != 0u;
        mw = draw(a.key, (uint32_t)j, c, a.gen, SLOT_MUTATE);
        mut_l = mw.x < a.thr;
      }
    } else if (a.mode == ROWS_INIT && c > 0) {
      mw = draw(a.key, (uint32_t)j, c, GEN_INIT, SLOT_INIT);
      mut_l = mw.x < a.thr;
    }
  }
  const unsigned act_mask = __ballot_sync(0xffffffffu, act_l);
  const unsigned sec_mask = __ballot_sync(0xffffffffu, sec_l);
  const unsigned mut_mask = __ballot_sync(0xffffffffu, mut_l && act_l);

  // row j0 of the possible sources; per row only the offset r * NN is added
  const size_t roff0 = (size_t)j0 * NN;
  const int16_t *src_a = nullptr, *src_b = nullptr;
  if (a.mode == ROWS_GENERATION) {
    src_a = a.src + (size_t)s_parent[0] * J * NN + roff0;
    src_b = a.src + (size_t)s_parent[1] * J * NN + roff0;
  } else if (a.mode == ROWS_INIT) {
    src_a = src_b = a.src ? a.src + roff0 : nullptr;
  } else {
    src_a = src_b = a.dst + (size_t)cl * J * NN + roff0;
  }
  int16_t *dst0 = a.dst + (size_t)cl * J * NN + roff0;
  int16_t *row = s_rows + (size_t)warp * NN;
  uint4 *qvec = s_qvec[warp];
  uint32_t *qmeta = s_qmeta[warp];

  const int total_vecs = max(nrows, 0) << rv_log2;      // the warp's rows as one run of vectors
  // Rows are contiguous, so the warp's rows are one flat array of vectors in each source and in the
  // destination: vector t of the run is element t of all three.  What depends on the lane and the
  // slot q only (a tile never splits a row) is worked out once: the vector's row within the tile and
  // its place in that row.
  const uint4 *flat_a = (const uint4 *)src_a, *flat_b = (const uint4 *)src_b;
  uint4 *flat_d = (uint4 *)dst0;
  uint32_t meta_q[4];
  int rel_row[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int u = q * 32 + lane;
    rel_row[q] = u >> rv_log2;
    meta_q[q] = (uint32_t)rel_row[q] | ((uint32_t)(u & (row_vecs - 1)) << 8) | 0x80000000u;
  }
  for (int t0 = 0; t0 < total_vecs; t0 += 128) {
    // rows of this tile: [r_first, r_first + rows_here)
    const int r_first = t0 >> rv_log2;
    const int rows_here = min(nrows - r_first, max(128 >> rv_log2, 1));
    s_rowK[warp][lane] = 0; s_rowN[warp][lane] = 0; s_rowbad[warp][lane] = 0;
    // ---- the stream: four vectors per lane in, queued if they hold anything, out ---------------
    // (rows that are inactive or have no source read as empty)
    uint4 x[4];
    bool in[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int t = t0 + q * 32 + lane;
      const int r = r_first + rel_row[q];
      in[q] = t < total_vecs;
      x[q] = make_uint4(0u, 0u, 0u, 0u);
      if (in[q] && ((act_mask >> (r & 31)) & 1u) && flat_a) x[q] = __ldg((((sec_mask >> (r & 31)) & 1u) ? flat_b : flat_a) + t);
    }
    int qn = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const bool nz = (x[q].x | x[q].y | x[q].z | x[q].w) != 0u;      // vectors outside the run are empty
      const unsigned bal = __ballot_sync(0xffffffffu, nz);
      if (nz) {
        const int pos = qn + __popc(bal & ((1u << lane) - 1u));
        qvec[pos] = x[q];
        qmeta[pos] = meta_q[q];
      }
      qn += __popc(bal);
      if (in[q]) flat_d[t0 + q * 32 + lane] = x[q];       // final for every row that is not rebuilt below
    }
    __syncwarp();
    // ---- first look at the queued entries: each row's K and N, entries outside [0, node size] ----
    for (int e = lane; e < qn * 8; e += 32) {
      const int val = (int)((const int16_t *)qvec)[e];
      if (val != 0) {
        const uint32_t meta = qmeta[e >> 3];
        const int rr = (int)(meta & 31u), n = (int)((meta >> 8) & 63u) * 8 + (e & 7);
        const int cv = min(max(val, 0), (int)s_cap[n]);
        if (cv != val) s_rowbad[warp][rr] = 1;
        if (cv > 0) { atomicAdd(&s_rowK[warp][rr], cv); atomicAdd(&s_rowN[warp][rr], 1); }
      }
    }
    __syncwarp();
    // ---- rows that have to be rebuilt: perturbed, an entry out of range, or a row cap broken ----
    bool need_l = false;
    const int kc_r = __shfl_sync(0xffffffffu, kc_l, (r_first + lane) & 31);   // the cap of the tile's lane-th row
    if (lane < rows_here) {
      const int r = r_first + lane;
      need_l = ((act_mask >> r) & 1u) &&
               (((mut_mask >> r) & 1u) || s_rowbad[warp][lane] || s_rowK[warp][lane] > kc_r || s_rowN[warp][lane] > a.n_max);
    }
    unsigned need = __ballot_sync(0xffffffffu, need_l);
    while (need) {
      const int rl = __ffs(need) - 1;           // row within the tile
      need &= need - 1;
      const int rr = r_first + rl;
      const int16_t *src = ((sec_mask >> rr) & 1u) ? src_b : src_a;
      // the row, every entry forced into [0, node size]
      for (int v = lane; v < row_vecs; v += 32) {
        uint4 y = make_uint4(0u, 0u, 0u, 0u);
        if (src) y = clamp_vec(__ldg((const uint4 *)(src + (size_t)rr * NN) + v), ((const uint4 *)s_cap)[v]);
        ((uint4 *)row)[v] = y;
      }
      __syncwarp();
      int rK = 0, rN = 0;
      for (int n = lane; n < NN; n += 32) { rK += row[n]; rN += row[n] > 0; }
      rK = __reduce_add_sync(0xffffffffu, rK);
      rN = __reduce_add_sync(0xffffffffu, rN);
      if ((mut_mask >> rr) & 1u) {
        const uint32_t m1 = __shfl_sync(0xffffffffu, mw.y, rr), m2 = __shfl_sync(0xffffffffu, mw.z, rr),
                       m3 = __shfl_sync(0xffffffffu, mw.w, rr);
        const uint32_t op = bounded(m1, 3u);
        if (op == 0u) {
          const int n = (int)bounded(m3, (uint32_t)NN);
          if (lane == 0) row[n] = (int16_t)min((int)row[n] + 1, (int)s_cap[n]);
        } else if (rN > 0) {
          const int ns = nth_occupied(row, NN, bounded(m2, (uint32_t)rN), lane);
          if (op == 1u) {
            if (lane == 0) row[ns] = (int16_t)(row[ns] - 1);
          } else {
            const int nd = (int)bounded(m3, (uint32_t)NN);
            if (nd != ns && lane == 0) {
              row[nd] = (int16_t)min((int)row[nd] + (int)row[ns], (int)s_cap[nd]);
              row[ns] = 0;
            }
          }
        }
        __syncwarp();
        rK = 0; rN = 0;
        for (int n = lane; n < NN; n += 32) { rK += row[n]; rN += row[n] > 0; }
        rK = __reduce_add_sync(0xffffffffu, rK);
        rN = __reduce_add_sync(0xffffffffu, rN);
      }
      const int rkc = __shfl_sync(0xffffffffu, kc_l, rr);
      if (rK > rkc || rN > a.n_max) {
        if (lane == 0) {
          int excess = rK - rkc;
          rK = min(rK, rkc);
          for (int n = NN - 1; n >= 0 && excess > 0; --n) {
            const int take = min((int)row[n], excess);
            row[n] = (int16_t)(row[n] - take);
            excess -= take;
          }
          int occ = 0;
          for (int n = 0; n < NN; ++n) {
            if (row[n] > 0) {
              ++occ;
              if (occ > a.n_max) { rK -= row[n]; row[n] = 0; }
            }
          }
          rN = min(occ, a.n_max);
        }
        rN = __shfl_sync(0xffffffffu, rN, 0);
        rK = __shfl_sync(0xffffffffu, rK, 0);
        __syncwarp();
      }
      if (lane == 0) { s_rowK[warp][rl] = rK; s_rowN[warp][rl] = rN; }
      // the row's queued vectors are dropped; the row is written again and its occupants go
      // straight into the column totals and lists
      for (int e = lane; e < qn; e += 32)
        if ((qmeta[e] & 31u) == (uint32_t)rl) qmeta[e] &= 0x7FFFFFFFu;
      for (int v = lane; v < row_vecs; v += 32) ((uint4 *)(dst0 + (size_t)rr * NN))[v] = ((const uint4 *)row)[v];
      for (int n = lane; n < NN; n += 32) {
        const int val = row[n];
        if (val > 0) {
          atomicAdd(&s_tot[n], val);
          if (rN >= 2) atomicAdd(&s_el[n], 1);
          const int slot = atomicAdd(&s_cnt[n], 1);
          if (slot < OCC_SLOTS)
            s_occ[n * OCC_SLOTS + slot] = (uint32_t)(j0 + rr) | ((uint32_t)val << 20) | (rN >= 2 ? 0x80000000u : 0u);
        }
      }
      __syncwarp();
    }
    // ---- second look: column totals, distributed-job counts and occupant lists --------------------
    for (int e = lane; e < qn * 8; e += 32) {
      const uint32_t meta = qmeta[e >> 3];
      const int val = (int)((const int16_t *)qvec)[e];
      if ((meta >> 31) && val > 0) {
        const int rl = (int)(meta & 31u), n = (int)((meta >> 8) & 63u) * 8 + (e & 7);
        const bool dist = s_rowN[warp][rl] >= 2;
        atomicAdd(&s_tot[n], val);
        if (dist) atomicAdd(&s_el[n], 1);
        const int slot = atomicAdd(&s_cnt[n], 1);
        if (slot < OCC_SLOTS)
          s_occ[n * OCC_SLOTS + slot] = (uint32_t)(j0 + r_first + rl) | ((uint32_t)val << 20) | (dist ? 0x80000000u : 0u);
      }
    }
    if (lane < rows_here) {
      const int r = r_first + lane;
      a.dflag[(size_t)cl * J + j0 + r] = (((act_mask >> r) & 1u) && s_rowN[warp][lane] >= 2) ? 1 : 0;
    }
    __syncwarp();
  }

  __syncthreads();
  // ---- column partials and occupant lists of the block (as rows2_kernel) ----------------------
  const size_t base = ((size_t)cl * aa.nbatch + batch) * NN;
  for (int i = threadIdx.x; i < NN; i += blockDim.x) {
    aa.colsum[base + i] = s_tot[i];
    aa.colelig[base + i] = s_el[i];
    aa.occ_count[base + i] = s_cnt[i];
    const int cnt = min(s_cnt[i], OCC_SLOTS);
    for (int k = 0; k < cnt; ++k) aa.occ_list[(base + i) * OCC_SLOTS + k] = s_occ[i * OCC_SLOTS + k];
  }
  __shared__ bool s_last_block;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned prev = atomicAdd(aa.cand_ticket + cl, 1u);
    s_last_block = (prev == (unsigned)aa.nbatch - 1u);
    if (s_last_block) aa.cand_ticket[cl] = 0u;
  }
  __syncthreads();
  if (s_last_block) {
    __threadfence();
    for (int n = threadIdx.x; n < NN; n += blockDim.x) {
      int total = 0, nelig = 0;
      for (int b = 0; b < aa.nbatch; ++b) {
        total += __ldcg(aa.colsum + ((size_t)cl * aa.nbatch + b) * NN + n);
        nelig += __ldcg(aa.colelig + ((size_t)cl * aa.nbatch + b) * NN + n);
      }
      if (nelig >= 2 || total > (int)s_cap[n]) {
        const unsigned slot = atomicAdd(aa.list_count, 1u);
        aa.list[slot] = ((uint32_t)cl << 13) | (uint32_t)n;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Small problems (at most 256 jobs, at most 32 nodes): one block per candidate, one THREAD
// per row.  A row is 16 to 64 bytes, so a thread reads its parent's row with one to four
// vector loads, keeps it in its own line of shared memory, perturbs and caps it there, and
// adds its occupants to per-node lists; warps then repair the violating nodes from the
// lists (or from the rows in shared memory when a list overflows), the threads write their
// rows out and the block sums the fitness.  Same operators, draws and sums as the kernels
// above: identical populations and fitness bits, with far fewer dependent steps.
// ---------------------------------------------------------------------------------------
constexpr int SMALL_MAX_NODES = 32;
constexpr int SMALL_OCC = 32;   // occupants listed per node: one lane each in the repair

__global__ void __launch_bounds__(256) generation_small_kernel(Rows2Args aa) {
  const RowsArgs &a = aa.r;
  __shared__ __align__(16) int16_t s_rows[256][SMALL_MAX_NODES];   // child rows, a line per job
  __shared__ __align__(16) int16_t s_cap[SMALL_MAX_NODES];
  __shared__ uint32_t s_tot[SMALL_MAX_NODES], s_cnt[SMALL_MAX_NODES];  // GPUs placed; distributed jobs | occupants << 16
  __shared__ uint32_t s_occ[SMALL_MAX_NODES][SMALL_OCC];               // job | GPUs << 13 | distributed << 31
  __shared__ uint32_t s_summ[256];
  __shared__ uint8_t s_dirty[256];
  __shared__ float s_term[256];
  __shared__ int s_parent[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cl = blockIdx.x;
  const uint32_t c = a.first_cand + (uint32_t)cl;
  const int NN = a.num_nodes, J = a.J, P = a.P;
  const int row_vecs = NN >> 3;
  const bool elite = (int)c < a.num_elite;

  // The next generation's grid may be set up while this one runs (programmatic dependent launch):
  // its blocks do their own parent-independent prologue and then wait, below, for this grid to
  // finish.  Nothing this kernel writes to global memory is written before its own wait.
  asm volatile("griddepcontrol.launch_dependents;");
  // Everything that does not depend on the parents is asked for first, so that the waits overlap:
  // the job's flags and caps, the fitness keys (staged in shared memory), and the row's draws.
  const int j = tid;
  bool on = false;
  int kc = a.k_max;
  if (j < J) {
    on = !a.active || a.active[j];
    if (a.k_cap) kc = a.k_cap[j];
  }
  __shared__ __align__(16) uint32_t s_keys[256];
  const bool staged = P <= 256;
  if (tid < NN) {
    s_cap[tid] = (int16_t)max((int)a.cap[tid], 0);
    s_tot[tid] = 0u;
    s_cnt[tid] = 0u;
  }
  bool second = false, mut = false;
  u32x4 mw = {0, 0, 0, 0};
  if (on && !elite) {
    second = (draw(a.key, (uint32_t)j, c, a.gen, SLOT_XOVER).x >> 31) != 0u;
    mw = draw(a.key, (uint32_t)j, c, a.gen, SLOT_MUTATE);
    mut = mw.x < a.thr;
  }
  uint4 cur4[SMALL_MAX_NODES / 8];
#pragma unroll
  for (int v = 0; v < SMALL_MAX_NODES / 8; ++v) {
    cur4[v] = make_uint4(0u, 0u, 0u, 0u);
    if (a.cur && j < J && v < row_vecs) cur4[v] = __ldg((const uint4 *)(a.cur + (size_t)j * NN) + v);
  }
  // from here on the parents' population and fitness are read: the grid that wrote them must be done
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (elite) {
    if (staged && tid < P) s_keys[tid] = order_key(__ldcg(a.fitness_bits + tid));
    __syncthreads();
  }
  const bool early = !elite && row_vecs <= 2;
  uint4 cand[2][2] = {{make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)},
                      {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)}};
  int pair0 = -1;
  // ---- parents (rank = candidates ordered before, fitness descending, index ascending) --------
  if (elite) {
    for (int i = tid; i < P; i += blockDim.x) {
      const uint32_t ki = staged ? s_keys[i] : order_key(__ldcg(a.fitness_bits + i));
      int rk = 0, o = 0;
      if (staged) {
        for (; o + 4 <= P; o += 4) {   // four staged keys per step
          const uint4 k4 = *(const uint4 *)(s_keys + o);
          rk += (k4.x > ki || (k4.x == ki && o < i)) ? 1 : 0;
          rk += (k4.y > ki || (k4.y == ki && o + 1 < i)) ? 1 : 0;
          rk += (k4.z > ki || (k4.z == ki && o + 2 < i)) ? 1 : 0;
          rk += (k4.w > ki || (k4.w == ki && o + 3 < i)) ? 1 : 0;
        }
      }
      for (; o < P; ++o) {
        const uint32_t ko = staged ? s_keys[o] : order_key(__ldcg(a.fitness_bits + o));
        rk += (ko > ki || (ko == ki && o < i)) ? 1 : 0;
      }
      if (rk == (int)c) s_parent[0] = s_parent[1] = i;
    }
  } else {
    const u32x4 sel = draw(a.key, 0u, c, a.gen, SLOT_SELECT);
    const int idx[4] = {(int)bounded(sel.x, P), (int)bounded(sel.y, P), (int)bounded(sel.z, P), (int)bounded(sel.w, P)};
    // short rows: this thread's row of both candidates of its pair is fetched together with the
    // candidates' keys
    if (early && j < J && on) {
      pair0 = idx[second ? 2 : 0];
      const uint4 *r0 = (const uint4 *)(a.src + ((size_t)pair0 * J + j) * NN);
      const uint4 *r1 = (const uint4 *)(a.src + ((size_t)idx[second ? 3 : 1] * J + j) * NN);
      cand[0][0] = __ldcg(r0);
      cand[1][0] = __ldcg(r1);
      if (row_vecs > 1) { cand[0][1] = __ldcg(r0 + 1); cand[1][1] = __ldcg(r1 + 1); }
    }
    if (tid == 0) {
      uint32_t k4[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) k4[q] = order_key(__ldcg(a.fitness_bits + idx[q]));
      s_parent[0] = tournament_winner(k4[0], idx[0], k4[1], idx[1]);
      s_parent[1] = tournament_winner(k4[2], idx[2], k4[3], idx[3]);
    }
  }
  __syncthreads();

  // ---- rows: thread j builds row j of the child ----------------------------------------------
  // K and N of the row in this thread's line of shared memory, from its 16-byte pieces
  auto row_totals = [&](const int16_t *r, int &k_out, int &n_out) {
    uint32_t part = 0;
    for (int v = 0; v < row_vecs; ++v) part += row_partial(((const uint4 *)r)[v]);
    k_out = (int)(part & 0x3FFFFFu);
    n_out = (int)(part >> 22);
  };
  int16_t *row = s_rows[tid];
  int K = 0, N = 0, ndiff = 0;
  if (j < J) {
    const int parent = s_parent[second ? 1 : 0];
    const uint4 *src = (const uint4 *)(a.src + ((size_t)parent * J + j) * NN);
    const int which = (parent == pair0) ? 0 : 1;   // when the row was fetched early
#pragma unroll
    for (int v = 0; v < SMALL_MAX_NODES / 8; ++v) {
      uint4 x = make_uint4(0u, 0u, 0u, 0u);
      if (v < row_vecs) {
        if (on) {
          const uint4 raw = (early && v < 2) ? (which == 0 ? cand[0][v] : cand[1][v]) : __ldcg(src + v);
          x = clamp_vec(raw, ((const uint4 *)s_cap)[v]);   // entries into [0, node size]
        }
        ((uint4 *)row)[v] = x;
      }
    }
    if (on) {
      row_totals(row, K, N);
      if (mut) {
        const uint32_t op = bounded(mw.y, 3u);
        if (op == 0u) {
          const int n = (int)bounded(mw.w, (uint32_t)NN);
          row[n] = (int16_t)min((int)row[n] + 1, (int)s_cap[n]);
        } else if (N > 0) {
          int t = (int)bounded(mw.z, (uint32_t)N), ns = 0;
          for (int n = 0; n < NN; ++n) {
            if (row[n] > 0 && t-- == 0) { ns = n; break; }
          }
          if (op == 1u) {
            row[ns] = (int16_t)(row[ns] - 1);
          } else {
            const int nd = (int)bounded(mw.w, (uint32_t)NN);
            if (nd != ns) {
              row[nd] = (int16_t)min((int)row[nd] + (int)row[ns], (int)s_cap[nd]);
              row[ns] = 0;
            }
          }
        }
        row_totals(row, K, N);
      }
      // per-row caps: replicas above the job's cap leave from the highest node index down, then
      // occupied nodes beyond n_max are cleared from the highest index down
      kc = max(0, min(kc, a.k_max));
      if (K > kc || N > a.n_max) {
        int excess = K - kc;
        for (int n = NN - 1; n >= 0 && excess > 0; --n) {
          const int take = min((int)row[n], excess);
          row[n] = (int16_t)(row[n] - take);
          excess -= take;
        }
        int occ = 0;
        K = 0;
        for (int n = 0; n < NN; ++n) {
          if (row[n] > 0) {
            ++occ;
            if (occ > a.n_max) row[n] = 0;
          }
          K += row[n];
        }
        N = min(occ, a.n_max);
      }
      // occupants into the nodes' totals and lists; entries differing from the current allocation
      const bool dist = N >= 2;
#pragma unroll
      for (int v = 0; v < SMALL_MAX_NODES / 8; ++v) {
        if (v >= row_vecs) break;
        const uint4 x = ((const uint4 *)row)[v];
        if (a.cur) {
          // each half of the xor is a non-negative int16, so min(half, 1) counts the halves that differ
          const uint32_t d = __vimin_s16x2_relu(x.x ^ cur4[v].x, 0x00010001u) + __vimin_s16x2_relu(x.y ^ cur4[v].y, 0x00010001u) +
                             __vimin_s16x2_relu(x.z ^ cur4[v].z, 0x00010001u) + __vimin_s16x2_relu(x.w ^ cur4[v].w, 0x00010001u);
          ndiff += (int)((d & 0xFFFFu) + (d >> 16));
        }
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          const int g = (int)((w[h >> 1] >> ((h & 1) * 16)) & 0xFFFFu);
          if (g > 0) {
            const int n = 8 * v + h;
            atomicAdd(&s_tot[n], (uint32_t)g);
            const uint32_t k = atomicAdd(&s_cnt[n], (dist ? 1u : 0u) | (1u << 16)) >> 16;
            if (k < SMALL_OCC) s_occ[n][k] = (uint32_t)j | ((uint32_t)g << 13) | (dist ? 0x80000000u : 0u);
          }
        }
      }
    }
    s_summ[j] = on ? ((uint32_t)K | ((uint32_t)N << 11) | ((uint32_t)ndiff << 22)) : 0u;
    s_dirty[j] = 0;
  }
  __syncthreads();

  // ---- repair, a warp per violating node -------------------------------------------------------
  for (int nn = warp; nn < NN; nn += 8) {
    int tot = (int)s_tot[nn];
    const int ne = (int)(s_cnt[nn] & 0xFFFFu), have_n = (int)(s_cnt[nn] >> 16), cap_n = (int)s_cap[nn];
    if (ne < 2 && tot <= cap_n) continue;
    if (have_n <= SMALL_OCC) {
      // one occupant per lane
      const bool have = lane < have_n;
      const uint32_t entry = have ? s_occ[nn][lane] : 0u;
      const int jj = (int)(entry & 0x1FFFu);
      const int v_old = have ? (int)((entry >> 13) & 0x7FFu) : 0;
      int v = v_old;
      const bool dist = have && (entry >> 31);
      if (ne >= 2) {
        const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
        int t = J;
        if (dist && v > 0) { t = jj - o; if (t < 0) t += J; }
        int best = t;
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, off));
        int removed = 0;
        if (dist && v > 0 && t != best) { removed = v; v = 0; }
        tot -= warp_sum(removed);
      }
      const int excess = tot - cap_n;
      if (excess > 0) {
        const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J);
        int rot = 0x7fffffff;
        if (have) { rot = jj - o; if (rot < 0) rot += J; }
        int ahead = 0;                       // GPUs of the occupants that come first in rotated order
        for (int k = 0; k < have_n; ++k) {
          const int rk = __shfl_sync(0xffffffffu, rot, k);
          const int vk = __shfl_sync(0xffffffffu, v, k);
          if (rk < rot) ahead += vk;
        }
        if (have) v -= min(v, max(excess - ahead, 0));
      }
      if (have && v != v_old) {
        s_rows[jj][nn] = (int16_t)v;
        s_dirty[jj] = 1;
      }
    } else {
      // more occupants than the list holds: the column of the rows in shared memory
      int keep = -1;
      const bool intf = ne >= 2;
      if (intf) {
        const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
        int best = J;
        for (int jj = lane; jj < J; jj += 32) {
          if (s_rows[jj][nn] > 0 && ((s_summ[jj] >> 11) & 0x7FFu) >= 2u) {
            int t = jj - o;
            if (t < 0) t += J;
            best = min(best, t);
          }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, off));
        keep = o + best;
        if (keep >= J) keep -= J;
        int removed = 0;
        for (int jj = lane; jj < J; jj += 32) {
          const int v = s_rows[jj][nn];
          if (v > 0 && ((s_summ[jj] >> 11) & 0x7FFu) >= 2u && jj != keep) removed += v;
        }
        tot -= warp_sum(removed);
      }
      int excess = tot - cap_n;
      const int o = (excess > 0) ? (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J) : 0;
      for (int t0 = 0; t0 < J; t0 += 32) {
        const int t = t0 + lane;
        int jj = o + t;
        if (jj >= J) jj -= J;
        int v_old = 0, v_eff = 0;
        if (t < J) {
          v_old = s_rows[jj][nn];
          const bool dist = ((s_summ[jj] >> 11) & 0x7FFu) >= 2u;
          v_eff = (intf && dist && v_old > 0 && jj != keep) ? 0 : v_old;
        }
        int sfx = v_eff;                              // inclusive prefix over the 32 jobs
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int u = __shfl_up_sync(0xffffffffu, sfx, off);
          if (lane >= off) sfx += u;
        }
        const int take = (excess > 0) ? min(v_eff, max(excess - (sfx - v_eff), 0)) : 0;
        const int v_new = v_eff - take;
        if (t < J && v_new != v_old) {
          s_rows[jj][nn] = (int16_t)v_new;
          s_dirty[jj] = 1;
        }
        excess -= __shfl_sync(0xffffffffu, sfx, 31);
      }
    }
  }
  __syncthreads();

  // ---- rows out, fitness -----------------------------------------------------------------------
  if (j < J) {
    if (s_dirty[j]) {
      row_totals(row, K, N);
      ndiff = 0;
      if (a.cur) {
#pragma unroll
        for (int v = 0; v < SMALL_MAX_NODES / 8; ++v) {
          if (v >= row_vecs) break;
          const uint4 x = ((const uint4 *)row)[v];
          const uint32_t d = __vimin_s16x2_relu(x.x ^ cur4[v].x, 0x00010001u) + __vimin_s16x2_relu(x.y ^ cur4[v].y, 0x00010001u) +
                             __vimin_s16x2_relu(x.z ^ cur4[v].z, 0x00010001u) + __vimin_s16x2_relu(x.w ^ cur4[v].w, 0x00010001u);
          ndiff += (int)((d & 0xFFFFu) + (d >> 16));
        }
      }
    }
    uint4 *dst = (uint4 *)(a.dst + ((size_t)cl * J + j) * NN);
    for (int v = 0; v < row_vecs; ++v) dst[v] = ((const uint4 *)row)[v];
    if (on && (!aa.tp.active || aa.tp.active[j])) s_term[j] = fitness_term(aa.tp, j, K, N, ndiff != 0);
  }
  __syncthreads();
  double tsum, tcount;
  block_term_sum(s_term, J, 0, aa.tp.active, tsum, tcount);
  if (tid == 0) aa.fitness_out[cl] = fitness_finalise(aa.tp.mode, aa.tp.p, tsum, tcount);
}

// Column pass: warps take nodes from the work list the row kernel built (any order: columns are
// independent) and repair them.
__global__ void __launch_bounds__(128, 4) colrepair_kernel(ColfixArgs a) {
  const int lane = threadIdx.x & 31;
  const unsigned nwarps = gridDim.x * (blockDim.x >> 5);
  const unsigned count = *a.list_count;
  const int NN = a.num_nodes;
  for (unsigned i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < count; i += nwarps) {
    const uint32_t e = a.list[i];
    const int cl = (int)(e >> 13), n = (int)(e & 0x1FFFu);
    int total = 0, nelig = 0;
    for (int b = 0; b < a.nbatch; ++b) {
      total += a.colsum[((size_t)cl * a.nbatch + b) * NN + n];
      nelig += a.colelig[((size_t)cl * a.nbatch + b) * NN + n];
    }
    const int cp = max((int)a.cap[n], 0);
    repair_column_list(a, cl, n, total, nelig, cp, lane);
    __syncwarp();
  }
}

int launch_rows(sched_ctx *ctx, RowsArgs &a) {
  const long long warps = (long long)a.count * a.J;
  if (warps == 0) return SCHED_OK;
  const int wpb = 8;
  const size_t smem = (size_t)wpb * ((a.num_nodes + 7) & ~7) * sizeof(int16_t);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
      set_error(ctx, "cudaFuncSetAttribute failed: %s", cudaGetErrorString(e));
      return SCHED_ERR_CUDA;
    }
  }
  const long long blocks = (warps + wpb - 1) / wpb;
  {
  TimedLaunch tl_(ctx, KK_ROWS);
  rows_kernel<<<(unsigned)blocks, wpb * 32, smem, ctx->stream>>>(a);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

int launch_cols(sched_ctx *ctx, int16_t *pop, int count, uint32_t first_cand, uint32_t gen) {
  if (count == 0 || ctx->cfg.num_jobs == 0) return SCHED_OK;
  ColsArgs a;
  a.pop = pop; a.dflag = ctx->d_dflag; a.cap = ctx->d_cap;
  a.J = ctx->cfg.num_jobs; a.num_nodes = ctx->cfg.num_nodes;
  a.gen = gen; a.key = make_key(ctx->cfg.seed, ctx->d_round);
  for (int first = 0; first < count; first += 65535) {
    const int n = min(65535, count - first);
    a.count = n;
    a.first_cand = first_cand + (uint32_t)first;
    a.pop = pop + (size_t)first * a.J * a.num_nodes;
    a.dflag = ctx->d_dflag + (size_t)first * a.J;
    dim3 grid((unsigned)((a.num_nodes + 127) / 128), (unsigned)n);
    { TimedLaunch tl_(ctx, KK_COLS); cols_kernel<<<grid, 128, 0, ctx->stream>>>(a); }
    SCHED_LAUNCH_CHECK(ctx);
  }
  return SCHED_OK;
}

// Row pass + column pass of `count` candidates.  Rows of a multiple of 8 and at most 512
// nodes (16-byte vectors, <= 2 per lane) with node sizes <= 2047 take the batched kernels
// with fused column sums; everything else the general warp-per-row / thread-per-column pair.
int launch_rows_cols(sched_ctx *ctx, RowsArgs &a, int16_t *pop, int count, uint32_t first_cand, uint32_t gen) {
  if (count == 0 || a.J == 0) return SCHED_OK;
  const int NN = a.num_nodes;
  const bool aligned = ((((uintptr_t)a.dst | (uintptr_t)a.src | (uintptr_t)a.cur) & 15) == 0);
  const bool fused = (NN % 8 == 0) && NN <= 512 && aligned && ctx->cap_max <= 2047 && count <= 65535 &&
                     a.J <= (1 << 20);
  ctx->summ_valid = fused && a.summ != nullptr;
  ctx->fit_done = false;
  if (!fused) {
    if (a.mode == ROWS_GENERATION) {
      {
        TimedLaunch tl_(ctx, KK_RANK);
        rank_kernel<<<(a.P + 127) / 128, 128, 0, ctx->stream>>>(a.fitness_bits, a.P, ctx->d_rank, ctx->d_order);
      }
      SCHED_LAUNCH_CHECK(ctx);
    }
    int rc = launch_rows(ctx, a);
    if (rc != SCHED_OK) return rc;
    return launch_cols(ctx, pop, count, first_cand, gen);
  }
  const int nbatch = (a.J + 255) / 256;
  int rc = ensure_colscratch(ctx, (size_t)count * nbatch * NN);
  if (rc != SCHED_OK) return rc;
  Rows2Args aa;
  aa.r = a;
  aa.colsum = ctx->d_colsum; aa.colelig = ctx->d_colelig; aa.nbatch = nbatch;
  aa.list_count = ctx->d_colcount; aa.list = ctx->d_collist; aa.cand_ticket = ctx->d_rowticket;
  aa.occ_count = ctx->d_occcount; aa.occ_list = ctx->d_occlist;
  aa.fuse = (nbatch == 1 && ctx->ff_on) ? 1 : 0;
  aa.tp.table = ctx->ff_table; aa.tp.pen = ctx->ff_pen; aa.tp.active = ctx->ff_active;
  aa.tp.k_max = ctx->cfg.k_max; aa.tp.n_max = ctx->cfg.n_max; aa.tp.mode = fitness_mode(ctx->ff_p);
  aa.tp.p = ctx->ff_p; aa.tp.floor_ = ctx->cfg.speedup_floor;
  aa.fitness_out = ctx->ff_out;
  ctx->fit_done = aa.fuse != 0;
  dim3 grid((unsigned)nbatch, (unsigned)count);
  const int row_vecs_all = NN / 8;
  if (!aa.fuse && a.summ == nullptr && (row_vecs_all & (row_vecs_all - 1)) == 0) {
    // no per-row summaries wanted (the entry points called on their own): the streaming kernel
    const size_t smem = stream_smem_bytes(NN);
    if (smem > 24 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(rows_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) {
        set_error(ctx, "cudaFuncSetAttribute failed: %s", cudaGetErrorString(e));
        return SCHED_ERR_CUDA;
      }
    }
    SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->d_colcount, 0, sizeof(unsigned int), ctx->stream));
    {
      TimedLaunch tl_(ctx, KK_ROWS);
      rows_stream_kernel<<<grid, 256, smem, ctx->stream>>>(aa);
    }
    SCHED_LAUNCH_CHECK(ctx);
    ColfixArgs f;
    f.pop = pop; f.dflag = ctx->d_dflag; f.cap = ctx->d_cap;
    f.colsum = ctx->d_colsum; f.colelig = ctx->d_colelig; f.summ = nullptr;
    f.J = a.J; f.num_nodes = NN; f.nbatch = nbatch;
    f.gen = gen; f.first_cand = first_cand; f.key = make_key(ctx->cfg.seed, ctx->d_round);
    f.list = ctx->d_collist; f.list_count = ctx->d_colcount;
    f.cur = nullptr; f.occ_count = ctx->d_occcount; f.occ_list = ctx->d_occlist;
    { TimedLaunch tl_(ctx, KK_COLS); colrepair_kernel<<<ctx->num_sms * 4, 128, 0, ctx->stream>>>(f); }
    SCHED_LAUNCH_CHECK(ctx);
    return SCHED_OK;
  }
  if (aa.fuse && a.mode == ROWS_GENERATION && NN <= SMALL_MAX_NODES && a.J <= 8192) {
    // small problem inside a round: thread-per-row kernel, fitness included
    {
      TimedLaunch tl_(ctx, KK_ROWS);
      // launched so that it may overlap the tail of the kernel before it (see the kernel's top)
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3((unsigned)count);
      lc.blockDim = dim3(256);
      lc.dynamicSmemBytes = 0;
      lc.stream = ctx->stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      lc.attrs = attr;
      lc.numAttrs = 1;
      if (cudaLaunchKernelEx(&lc, generation_small_kernel, aa) != cudaSuccess) {
        cudaGetLastError();
        generation_small_kernel<<<(unsigned)count, 256, 0, ctx->stream>>>(aa);
      }
    }
    SCHED_LAUNCH_CHECK(ctx);
    return SCHED_OK;
  }
  if (!aa.fuse) SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->d_colcount, 0, sizeof(unsigned int), ctx->stream));
  {
    TimedLaunch tl_(ctx, KK_ROWS);
    // about four vectors per lane: several loads in flight and the per-row overhead shared
    const int row_vecs = NN / 8;
    int lpr_log2 = 0;
    while ((4 << lpr_log2) < row_vecs && lpr_log2 < 5) ++lpr_log2;
    aa.lpr_log2 = lpr_log2;
    const int vpl = (row_vecs + (1 << lpr_log2) - 1) >> lpr_log2;
    const bool full = (vpl << lpr_log2) == row_vecs && (vpl == 1 || vpl == 2 || vpl == 4);
#define ROWS2(L, V)                                                            \
  do {                                                                         \
    if (aa.fuse) {                                                             \
      if (full) rows2_kernel<L, V, true, true><<<grid, 256, 0, ctx->stream>>>(aa);    \
      else rows2_kernel<L, V, false, true><<<grid, 256, 0, ctx->stream>>>(aa);        \
    } else {                                                                   \
      if (full) rows2_kernel<L, V, true, false><<<grid, 256, 0, ctx->stream>>>(aa);   \
      else rows2_kernel<L, V, false, false><<<grid, 256, 0, ctx->stream>>>(aa);       \
    }                                                                          \
  } while (0)
    if (lpr_log2 == 0) {
      if (vpl <= 1) ROWS2(0, 1);
      else if (vpl == 2) ROWS2(0, 2);
      else ROWS2(0, 4);
    } else if (lpr_log2 == 1) ROWS2(1, 4);
    else if (lpr_log2 == 2) ROWS2(2, 4);
    else if (lpr_log2 == 3) ROWS2(3, 4);
    else ROWS2(4, 4);
#undef ROWS2
  }
  SCHED_LAUNCH_CHECK(ctx);
  if (aa.fuse) return SCHED_OK;   // the block did the column pass and the fitness itself
  ColfixArgs f;
  f.pop = pop; f.dflag = ctx->d_dflag; f.cap = ctx->d_cap;
  f.colsum = ctx->d_colsum; f.colelig = ctx->d_colelig; f.summ = a.summ;
  f.J = a.J; f.num_nodes = NN; f.nbatch = nbatch;
  f.gen = gen; f.first_cand = first_cand; f.key = make_key(ctx->cfg.seed, ctx->d_round);
  f.list = ctx->d_collist; f.list_count = ctx->d_colcount;
  f.cur = a.cur; f.occ_count = ctx->d_occcount; f.occ_list = ctx->d_occlist;
  { TimedLaunch tl_(ctx, KK_COLS); colrepair_kernel<<<ctx->num_sms * 4, 128, 0, ctx->stream>>>(f); }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

RowsArgs base_rows_args(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, int count) {
  RowsArgs a;
  const sched_config &c = ctx->cfg;
  a.cap = ctx->d_cap; a.k_cap = d_k_cap; a.active = d_active;
  a.rank = ctx->d_rank; a.order = ctx->d_order; a.dflag = ctx->d_dflag;
  a.P = c.population; a.J = c.num_jobs; a.num_nodes = c.num_nodes;
  a.k_max = c.k_max; a.n_max = c.n_max; a.num_elite = c.num_elite; a.count = count;
  a.thr = 0; a.gen = 0; a.first_cand = 0;
  a.key = make_key(c.seed, ctx->d_round);
  a.src = nullptr; a.dst = nullptr; a.mode = ROWS_REPAIR; a.fitness_bits = nullptr;
  a.cur = nullptr; a.summ = nullptr; a.summ_in = nullptr;
  return a;
}

}  // namespace

int launch_repair(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, int16_t *d_pop,
                  int32_t count, uint32_t first_candidate, uint32_t generation) {
  int rc = ensure_dflag(ctx, count);
  if (rc != SCHED_OK) return rc;
  RowsArgs a = base_rows_args(ctx, d_k_cap, d_active, count);
  a.mode = ROWS_REPAIR; a.src = d_pop; a.dst = d_pop;
  a.first_cand = first_candidate; a.gen = generation; a.key = make_key(ctx->cfg.seed, ctx->d_round);
  return launch_rows_cols(ctx, a, d_pop, count, first_candidate, generation);
}

int launch_init_population(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active,
                           const int16_t *d_cur, int16_t *d_pop_out) {
  const int P = ctx->cfg.population;
  int rc = ensure_dflag(ctx, P);
  if (rc != SCHED_OK) return rc;
  RowsArgs a = base_rows_args(ctx, d_k_cap, d_active, P);
  a.mode = ROWS_INIT; a.src = d_cur; a.dst = d_pop_out;
  a.thr = ctx->cfg.thr_init; a.gen = GEN_INIT; a.key = make_key(ctx->cfg.seed, ctx->d_round);
  a.cur = ctx->round_cur; a.summ = ctx->round_summ;
  return launch_rows_cols(ctx, a, d_pop_out, P, 0u, GEN_INIT);
}

// children first_child .. first_child + num_children - 1 (num_children < 0: all of them)
int launch_generation(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active,
                      const int16_t *d_pop_in, const float *d_fitness_in, int16_t *d_pop_out,
                      uint32_t generation, int first_child, int num_children) {
  const int P = num_children < 0 ? ctx->cfg.population : num_children;
  if (P == 0) return SCHED_OK;
  int rc = ensure_dflag(ctx, P);
  if (rc != SCHED_OK) return rc;
  RowsArgs a = base_rows_args(ctx, d_k_cap, d_active, P);
  a.first_cand = (uint32_t)first_child;
  a.mode = ROWS_GENERATION; a.src = d_pop_in; a.dst = d_pop_out;
  a.fitness_bits = (const uint32_t *)d_fitness_in;
  a.thr = ctx->cfg.thr_mutate; a.gen = generation; a.key = make_key(ctx->cfg.seed, ctx->d_round);
  a.cur = ctx->round_cur; a.summ = ctx->round_summ; a.summ_in = ctx->round_summ_in;
  return launch_rows_cols(ctx, a, d_pop_out, P, (uint32_t)first_child, generation);
}

__global__ void set_round_kernel(uint32_t *dst, uint32_t value) { *dst = value; }

int launch_set_round(sched_ctx *ctx, uint32_t round) {
  set_round_kernel<<<1, 1, 0, ctx->stream>>>(ctx->d_round, round);
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

int launch_select_best(sched_ctx *ctx, const int16_t *d_pop, const float *d_fitness,
                       int16_t *d_best, float *d_best_fitness) {
  const int P = ctx->cfg.population;
  {
  TimedLaunch tl_(ctx, KK_BEST);
  best_index_kernel<<<1, 256, 0, ctx->stream>>>((const uint32_t *)d_fitness, P, ctx->d_best_idx,
                                                d_best_fitness);
  }
  SCHED_LAUNCH_CHECK(ctx);
  const size_t elems = (size_t)ctx->cfg.num_jobs * ctx->cfg.num_nodes;
  if (elems == 0 || !d_pop) return SCHED_OK;   // no dense population: the caller gathers the rows
  const int blocks = (int)((elems + 256 * 8 - 1) / (256 * 8));
  {
  TimedLaunch tl_(ctx, KK_COPY);
  copy_best_kernel<<<blocks > 1024 ? 1024 : blocks, 256, 0, ctx->stream>>>(d_pop, ctx->d_best_idx,
                                                                           elems, d_best);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}
