// Population fitness (Eq. 14): per (candidate, job) row summary (K = SUM(a), N = occupied
// nodes, "row differs from the current allocation"), speedup gather, re-allocation
// penalty, floor, and the power-mean reduction over the active jobs.
//
// The kernel streams the dense int16 population once with wide loads.  Rows are split
// over LPR lanes (a power of two <= 32); a warp summarises 32 rows, parks each row's
// packed (K, N, changed) in one lane, and then all 32 lanes do the gather / penalty /
// power term for their row at once.  A block covers a contiguous chunk of one
// candidate's rows; chunk sums go to a scratch array and the last block to arrive adds
// them in index order, so results are bitwise reproducible.
#include "common.cuh"
#include "fitness_common.cuh"

namespace {

template <int W>
struct VecLoad;
template <>
struct VecLoad<16> {
  static __device__ __forceinline__ uint4 ld(const void *p) {
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
  }
  static __device__ __forceinline__ uint4 ld_cached(const void *p) { return __ldg((const uint4 *)p); }
};
template <>
struct VecLoad<8> {
  static __device__ __forceinline__ uint4 ld(const void *p) {
    const uint2 t = __ldg((const uint2 *)p);
    return make_uint4(t.x, t.y, 0u, 0u);
  }
  static __device__ __forceinline__ uint4 ld_cached(const void *p) { return ld(p); }
};
template <>
struct VecLoad<4> {
  static __device__ __forceinline__ uint4 ld(const void *p) {
    return make_uint4(__ldg((const uint32_t *)p), 0u, 0u, 0u);
  }
  static __device__ __forceinline__ uint4 ld_cached(const void *p) { return ld(p); }
};
template <>
struct VecLoad<2> {
  static __device__ __forceinline__ uint4 ld(const void *p) {
    return make_uint4((uint32_t)__ldg((const uint16_t *)p), 0u, 0u, 0u);
  }
  static __device__ __forceinline__ uint4 ld_cached(const void *p) { return ld(p); }
};

// per 32-bit word (two int16 entries): signed sum, and count of entries > 0
__device__ __forceinline__ void summarise_word(uint32_t w, int &ksum, uint32_t &npos) {
  ksum = __dp2a_lo((int)w, 0x0101, ksum);
  npos += __vimin_s16x2_relu(w, 0x00010001u);   // min(v, 1) floored at 0, per half
}

struct FitnessArgs {
  const int16_t *pop;
  const int16_t *cur;
  const float *table;
  const float *pen;       // [J] factor applied to changed rows, or NULL
  const uint8_t *active;  // or NULL
  const uint32_t *summ;   // [count][J] row summaries from the row/column kernels (SUMMARY mode)
  int J, num_nodes, k_max, n_max;
  int lpr_log2;           // lanes per row = 1 << lpr_log2
  int rows_per_block, chunks;
  int mode;
  float p, floor_;
  double *partial;        // [count][chunks][2]: sum of terms, number of active rows
  unsigned int *ticket;   // [count]
  float *fitness;
};

// End of a block's work: its terms are added in a fixed order, the chunk sum goes to scratch,
// and the last block of the candidate to arrive adds the chunk sums in index order and
// writes the power mean.
__device__ __forceinline__ void block_finish(const FitnessArgs &a, int cand, int chunk, int j0, int j1,
                                             const float *s_term) {
  __syncthreads();
  double t, n;
  block_term_sum(s_term, j1 - j0, j0, a.active, t, n);
  __shared__ bool s_last;
  if (threadIdx.x == 0) {
    double *dst = a.partial + ((size_t)cand * a.chunks + chunk) * 2;
    dst[0] = t;
    dst[1] = n;
    __threadfence();
    const unsigned prev = atomicAdd(a.ticket + cand, 1u);
    s_last = (prev == (unsigned)a.chunks - 1u);
  }
  __syncthreads();
  if (s_last && threadIdx.x == 0) {
    __threadfence();
    const volatile double *src = a.partial + (size_t)cand * a.chunks * 2;
    double ts = 0.0, ns = 0.0;
    for (int c = 0; c < a.chunks; ++c) { ts += src[2 * c]; ns += src[2 * c + 1]; }
    a.fitness[cand] = fitness_finalise(a.mode, a.p, ts, ns);
    a.ticket[cand] = 0u;   // ready for the next call on this stream
  }
}

template <int W>
__global__ void __launch_bounds__(256) fitness_kernel(FitnessArgs a) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int cand = blockIdx.y, chunk = blockIdx.x;
  const int LPR = 1 << a.lpr_log2, RPW = 32 >> a.lpr_log2;
  const int group = lane >> a.lpr_log2, sub = lane & (LPR - 1);
  const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << (group * LPR));
  const int row_vecs = (a.num_nodes * 2) / W;
  const int j0 = chunk * a.rows_per_block;
  const int j1 = min(a.J, j0 + a.rows_per_block);
  const int KD = a.k_max + 1, ND = a.n_max + 1;
  const char *cand_base = (const char *)(a.pop + (size_t)cand * a.J * a.num_nodes);
  const char *cur_base = (const char *)a.cur;
  const size_t row_bytes = (size_t)a.num_nodes * 2;

  __shared__ float s_term[FITNESS_MAX_ROWS_PER_BLOCK];
  TermParams tp;
  tp.table = a.table; tp.pen = a.pen; tp.active = a.active;
  tp.k_max = a.k_max; tp.n_max = a.n_max; tp.mode = a.mode; tp.p = a.p; tp.floor_ = a.floor_;
  uint32_t mine = 0;
  int myrow = -1;
  int it = 0;
  const int slots_per_fill = LPR;        // iterations that fill all 32 lanes

  // warp-uniform loop: every lane takes part in the shuffles of every iteration
  for (int jb = j0 + warp * RPW; jb < j1; jb += nwarps * RPW, ++it) {
    const int j = jb + group;
    const bool live = j < j1;
    int ksum = 0;
    uint32_t npos = 0, diff = 0;
    if (live) {
      const char *row = cand_base + (size_t)j * row_bytes;
      const char *crow = cur_base ? cur_base + (size_t)j * row_bytes : nullptr;
      // batches of vectors per lane: all loads of a batch are issued before any is used
      if (!crow) {
        constexpr int B = 8;
        for (int v0 = sub; v0 < row_vecs; v0 += LPR * B) {
          uint4 x[B];
#pragma unroll
          for (int k = 0; k < B; ++k) {
            const int v = v0 + k * LPR;
            x[k] = make_uint4(0u, 0u, 0u, 0u);
            if (v < row_vecs) x[k] = VecLoad<W>::ld(row + (size_t)v * W);
          }
#pragma unroll
          for (int k = 0; k < B; ++k) {
            if ((x[k].x | x[k].y | x[k].z | x[k].w) != 0u) {
              summarise_word(x[k].x, ksum, npos);
              if (W >= 8) summarise_word(x[k].y, ksum, npos);
              if (W >= 16) { summarise_word(x[k].z, ksum, npos); summarise_word(x[k].w, ksum, npos); }
            }
          }
        }
      } else {
        constexpr int B = 4;   // the current allocation's vectors travel with the candidate's
        for (int v0 = sub; v0 < row_vecs; v0 += LPR * B) {
          uint4 x[B], c[B];
#pragma unroll
          for (int k = 0; k < B; ++k) {
            const int v = v0 + k * LPR;
            x[k] = make_uint4(0u, 0u, 0u, 0u);
            c[k] = make_uint4(0u, 0u, 0u, 0u);
            if (v < row_vecs) {
              x[k] = VecLoad<W>::ld(row + (size_t)v * W);
              c[k] = VecLoad<W>::ld_cached(crow + (size_t)v * W);
            }
          }
#pragma unroll
          for (int k = 0; k < B; ++k) {
            if ((x[k].x | x[k].y | x[k].z | x[k].w) != 0u) {
              summarise_word(x[k].x, ksum, npos);
              if (W >= 8) summarise_word(x[k].y, ksum, npos);
              if (W >= 16) { summarise_word(x[k].z, ksum, npos); summarise_word(x[k].w, ksum, npos); }
            }
            diff |= (x[k].x ^ c[k].x) | (x[k].y ^ c[k].y) | (x[k].z ^ c[k].z) | (x[k].w ^ c[k].w);
          }
        }
      }
    }
    // saturate the lane-local counts so that the packed fields cannot overflow when
    // 32 lanes are added: K in bits 0..15 (<= 32 * 2047), N in bits 16..31
    int nl = (int)((npos & 0xFFFFu) + (npos >> 16));
    ksum = max(0, min(ksum, 2047));
    nl = min(nl, 2047);
    uint32_t packed = (uint32_t)ksum | ((uint32_t)nl << 16);
    for (int off = LPR >> 1; off >= 1; off >>= 1) packed += __shfl_xor_sync(0xffffffffu, packed, off);
    const unsigned changed = __ballot_sync(0xffffffffu, diff != 0u) & gmask;
    // lane `sub` of each group parks the row its group summarised in iteration `sub`
    if (live && sub == (it & (LPR - 1))) {
      // K <= 32*2047 < 2^16, N likewise; keep "changed" in the top bit of the N field
      mine = (packed & 0x7FFFFFFFu) | (changed ? 0x80000000u : 0u);
      myrow = j;
    }
    const bool flush = ((it + 1) % slots_per_fill == 0) || (jb + nwarps * RPW >= j1);
    if (flush) {
      if (myrow >= 0 && (!a.active || a.active[myrow]))
        s_term[myrow - j0] = fitness_term(tp, myrow, (int)(mine & 0xFFFFu), (int)((mine >> 16) & 0x7FFFu),
                                          (mine >> 31) != 0u);
      myrow = -1;
    }
  }

  block_finish(a, cand, chunk, j0, j1, s_term);
}

// Fitness from the row summaries the row / column kernels keep (K | N << 11 | entries
// differing from the current allocation << 22): no pass over the matrices.  Same chunks, same
// terms and the same fixed-order sums as fitness_kernel, hence identical bits.
__global__ void __launch_bounds__(256) fitness_summary_kernel(FitnessArgs a) {
  __shared__ float s_term[FITNESS_MAX_ROWS_PER_BLOCK];
  const int cand = blockIdx.y, chunk = blockIdx.x;
  const int j0 = chunk * a.rows_per_block;
  const int j1 = min(a.J, j0 + a.rows_per_block);
  TermParams tp;
  tp.table = a.table; tp.pen = a.pen; tp.active = a.active;
  tp.k_max = a.k_max; tp.n_max = a.n_max; tp.mode = a.mode; tp.p = a.p; tp.floor_ = a.floor_;
  for (int j = j0 + threadIdx.x; j < j1; j += blockDim.x) {
    if (!a.active || a.active[j]) {
      const uint32_t w = a.summ[(size_t)cand * a.J + j];
      s_term[j - j0] = fitness_term(tp, j, (int)(w & 0x7FFu), (int)((w >> 11) & 0x7FFu), (w >> 22) != 0u);
    }
  }
  block_finish(a, cand, chunk, j0, j1, s_term);
}

// Eq. 14 with rack-level locality: a row whose occupied nodes lie in two or more racks takes its
// speedup from the rack-class table.  A plain warp-per-row pass (this variant is not the
// streaming kernel above); same chunks and the same fixed-order sums.
__global__ void __launch_bounds__(256)
fitness_racks_kernel(FitnessArgs a, const float *__restrict__ table_rack, const int16_t *__restrict__ rack) {
  __shared__ float s_term[FITNESS_MAX_ROWS_PER_BLOCK];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int cand = blockIdx.y, chunk = blockIdx.x;
  const int j0 = chunk * a.rows_per_block;
  const int j1 = min(a.J, j0 + a.rows_per_block);
  TermParams tp;
  tp.table = a.table; tp.pen = a.pen; tp.active = a.active;
  tp.k_max = a.k_max; tp.n_max = a.n_max; tp.mode = a.mode; tp.p = a.p; tp.floor_ = a.floor_;
  for (int j = j0 + warp; j < j1; j += nwarps) {
    if (a.active && !a.active[j]) continue;
    const int16_t *row = a.pop + ((size_t)cand * a.J + j) * a.num_nodes;
    const int16_t *crow = a.cur ? a.cur + (size_t)j * a.num_nodes : nullptr;
    long long K = 0;
    int N = 0, rmin = 0x7fffffff, rmax = -1, diff = 0;
    for (int n = lane; n < a.num_nodes; n += 32) {
      const int v = row[n];
      K += v;
      if (v > 0) {
        ++N;
        const int r = rack[n];
        rmin = min(rmin, r);
        rmax = max(rmax, r);
      }
      if (crow) diff |= (v != (int)crow[n]) ? 1 : 0;
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      K += __shfl_xor_sync(0xffffffffu, K, off);
      N += __shfl_xor_sync(0xffffffffu, N, off);
      rmin = min(rmin, __shfl_xor_sync(0xffffffffu, rmin, off));
      rmax = max(rmax, __shfl_xor_sync(0xffffffffu, rmax, off));
      diff |= __shfl_xor_sync(0xffffffffu, diff, off);
    }
    if (lane == 0) {
      const int Kc = (int)max(0ll, min(K, (long long)a.k_max));
      const bool several = N >= 1 && rmin != rmax;
      const float x = __ldg((several ? table_rack : a.table) + fitness_table_index(tp, j, Kc, N));
      s_term[j - j0] = fitness_term_of(tp, j, x, diff != 0);
    }
  }
  block_finish(a, cand, chunk, j0, j1, s_term);
}

// Effective penalty per job: the re-allocation factor when the job currently holds GPUs,
// else 1 (pending jobs are never penalised).  One warp per job.
__global__ void penalty_prep_kernel(const int16_t *__restrict__ cur, const float *__restrict__ rf,
                                    int J, int num_nodes, float *__restrict__ pen) {
  const int lane = threadIdx.x & 31;
  const int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (j >= J) return;
  long long k = 0;
  for (int n = lane; n < num_nodes; n += 32) k += cur[(size_t)j * num_nodes + n];
  for (int off = 16; off >= 1; off >>= 1) k += __shfl_xor_sync(0xffffffffu, k, off);
  if (lane == 0) pen[j] = (k > 0) ? rf[j] : 1.f;
}

// Launch geometry shared by the entry points: the widest vector that divides a row and
// keeps every row aligned; lanes per row so that a lane owns about four vectors (several
// loads in flight, few shuffle steps); rows per block of about 1 MB of population, shrunk
// while the grid would leave SMs idle.
void fitness_geometry(size_t row_bytes, uintptr_t align_bits, int J, int count, int num_sms, int &W,
                      int &lpr_log2, int &rows_per_block, int &chunks) {
  W = 2;
  if (row_bytes % 16 == 0 && align_bits % 16 == 0) W = 16;
  else if (row_bytes % 8 == 0 && align_bits % 8 == 0) W = 8;
  else if (row_bytes % 4 == 0 && align_bits % 4 == 0) W = 4;
  const int row_vecs = (int)(row_bytes / W);
  lpr_log2 = 0;
  while ((4 << lpr_log2) < row_vecs && lpr_log2 < 5) ++lpr_log2;
  rows_per_block = (int)((1u << 20) / row_bytes);
  if (rows_per_block < 256) rows_per_block = 256;
  if (rows_per_block > FITNESS_MAX_ROWS_PER_BLOCK) rows_per_block = FITNESS_MAX_ROWS_PER_BLOCK;
  if (rows_per_block > J) rows_per_block = J > 0 ? J : 1;
  while (rows_per_block > 256 &&
         (long long)count * ((J + rows_per_block - 1) / rows_per_block) < 4LL * num_sms)
    rows_per_block = (rows_per_block + 1) / 2;
  chunks = J > 0 ? (J + rows_per_block - 1) / rows_per_block : 1;
}

}  // namespace

// Rows per block and blocks per candidate that launch_fitness uses for `count` candidates.
void fitness_chunking(const sched_ctx *ctx, int32_t count, int &rows_per_block, int &chunks) {
  int W, lpr_log2;
  fitness_geometry((size_t)ctx->cfg.num_nodes * 2, 0, ctx->cfg.num_jobs, count, ctx->num_sms, W, lpr_log2,
                   rows_per_block, chunks);
}

int launch_penalty_prep(sched_ctx *ctx, const int16_t *d_cur, const float *d_rf) {
  const int J = ctx->cfg.num_jobs;
  if (J == 0) return SCHED_OK;
  {
    TimedLaunch tl_(ctx, KK_PENPREP);
    penalty_prep_kernel<<<(J * 32 + 255) / 256, 256, 0, ctx->stream>>>(d_cur, d_rf, J, ctx->cfg.num_nodes, ctx->d_pen);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

int launch_fitness(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                   const int16_t *d_cur, const float *d_rf, const uint8_t *d_active, float p,
                   float *d_fitness, const uint32_t *d_summ) {
  const sched_config &c = ctx->cfg;
  const int J = c.num_jobs;
  if (count == 0) return SCHED_OK;
  if (J == 0) {     // the mean over no jobs: 0 by definition
    SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(d_fitness, 0, (size_t)count * sizeof(float), ctx->stream));
    return SCHED_OK;
  }

  const bool penalise = d_cur && d_rf;
  if (penalise && J > 0 && !ctx->pen_ready) {
    {
    TimedLaunch tl_(ctx, KK_PENPREP);
    penalty_prep_kernel<<<(J * 32 + 255) / 256, 256, 0, ctx->stream>>>(d_cur, d_rf, J, c.num_nodes,
                                                                       ctx->d_pen);
    }
    SCHED_LAUNCH_CHECK(ctx);
  }

  int W, lpr_log2, rows_per_block, chunks;
  fitness_geometry((size_t)c.num_nodes * 2, (uintptr_t)d_pop | (penalise ? (uintptr_t)d_cur : 0), J, count,
                   ctx->num_sms, W, lpr_log2, rows_per_block, chunks);
  int rc = ensure_fitness_scratch(ctx, count, chunks);
  if (rc != SCHED_OK) return rc;

  FitnessArgs a;
  a.pop = d_pop;
  a.cur = penalise ? d_cur : nullptr;
  a.table = d_speedup;
  a.pen = penalise ? ctx->d_pen : nullptr;
  a.active = d_active;
  a.summ = d_summ;
  a.J = J; a.num_nodes = c.num_nodes; a.k_max = c.k_max; a.n_max = c.n_max;
  a.lpr_log2 = lpr_log2;
  a.rows_per_block = rows_per_block; a.chunks = chunks;
  a.p = p; a.floor_ = c.speedup_floor;
  a.mode = fitness_mode(p);
  a.partial = ctx->d_partial;
  a.ticket = ctx->d_ticket;
  a.fitness = d_fitness;

  // grid.y is limited to 65535 candidates per launch
  for (int32_t first = 0; first < count; first += 65535) {
    const int32_t n = (count - first < 65535) ? (count - first) : 65535;
    FitnessArgs b = a;
    b.pop = d_pop + (size_t)first * J * c.num_nodes;
    b.partial = ctx->d_partial + (size_t)first * chunks * 2;
    b.ticket = ctx->d_ticket + first;
    b.fitness = d_fitness + first;
    if (d_summ) b.summ = d_summ + (size_t)first * J;
    dim3 grid((unsigned)chunks, (unsigned)n);
    {
    TimedLaunch tl_(ctx, KK_FITNESS);
    if (d_summ) fitness_summary_kernel<<<grid, 256, 0, ctx->stream>>>(b);
    else
    switch (W) {
      case 16: fitness_kernel<16><<<grid, 256, 0, ctx->stream>>>(b); break;
      case 8: fitness_kernel<8><<<grid, 256, 0, ctx->stream>>>(b); break;
      case 4: fitness_kernel<4><<<grid, 256, 0, ctx->stream>>>(b); break;
      default: fitness_kernel<2><<<grid, 256, 0, ctx->stream>>>(b); break;
    }
    }
    SCHED_LAUNCH_CHECK(ctx);
  }
  return SCHED_OK;
}

int launch_fitness_racks(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                         const float *d_speedup_rack, const int16_t *d_cur, const float *d_rf,
                         const uint8_t *d_active, float p, float *d_fitness) {
  const sched_config &c = ctx->cfg;
  const int J = c.num_jobs;
  if (count == 0) return SCHED_OK;
  if (J == 0) {     // the mean over no jobs: 0 by definition
    SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(d_fitness, 0, (size_t)count * sizeof(float), ctx->stream));
    return SCHED_OK;
  }
  const bool penalise = d_cur && d_rf;
  if (penalise && J > 0 && !ctx->pen_ready) {
    int rc = launch_penalty_prep(ctx, d_cur, d_rf);
    if (rc != SCHED_OK) return rc;
  }
  int W, lpr_log2, rows_per_block, chunks;
  fitness_geometry((size_t)c.num_nodes * 2, 0, J, count, ctx->num_sms, W, lpr_log2, rows_per_block, chunks);
  int rc = ensure_fitness_scratch(ctx, count, chunks);
  if (rc != SCHED_OK) return rc;
  FitnessArgs a;
  a.pop = d_pop;
  a.cur = penalise ? d_cur : nullptr;
  a.table = d_speedup;
  a.pen = penalise ? ctx->d_pen : nullptr;
  a.active = d_active;
  a.summ = nullptr;
  a.J = J; a.num_nodes = c.num_nodes; a.k_max = c.k_max; a.n_max = c.n_max;
  a.lpr_log2 = 0;
  a.rows_per_block = rows_per_block; a.chunks = chunks;
  a.p = p; a.floor_ = c.speedup_floor;
  a.mode = fitness_mode(p);
  a.partial = ctx->d_partial;
  a.ticket = ctx->d_ticket;
  a.fitness = d_fitness;
  for (int32_t first = 0; first < count; first += 65535) {
    const int32_t n = (count - first < 65535) ? (count - first) : 65535;
    FitnessArgs b = a;
    b.pop = d_pop + (size_t)first * J * c.num_nodes;
    b.partial = ctx->d_partial + (size_t)first * chunks * 2;
    b.ticket = ctx->d_ticket + first;
    b.fitness = d_fitness + first;
    dim3 grid((unsigned)chunks, (unsigned)n);
    {
      TimedLaunch tl_(ctx, KK_FITNESS);
      fitness_racks_kernel<<<grid, 256, 0, ctx->stream>>>(b, d_speedup_rack, ctx->d_rack);
    }
    SCHED_LAUNCH_CHECK(ctx);
  }
  return SCHED_OK;
}

// ---------------------------------------------------------------------------------------
// Fitness without any allocation: same kernels, scratch in a fixed file-scope device array.
// ---------------------------------------------------------------------------------------
#include <mutex>

namespace {

constexpr int NOALLOC_MAX_COUNT = SCHED_NOALLOC_MAX_COUNT;
constexpr int NOALLOC_MAX_JOBS = SCHED_NOALLOC_MAX_JOBS;
// Chunk sums are stored flat, candidate-major: (candidate * chunks + chunk) * 2.  The geometry
// gives at most NOALLOC_MAX_JOBS / 256 chunks per candidate unless it halves the rows of a block
// to fill the GPU, which it only does while count * chunks < 4 * SMs: a halving at most doubles
// the chunks, so count * chunks then stays below 8 * SMs.  Either way count * chunks fits
// NOALLOC_MAX_PARTIALS for every size within the documented limits (checked again per call).
constexpr size_t NOALLOC_MAX_PARTIALS = (size_t)NOALLOC_MAX_COUNT * (NOALLOC_MAX_JOBS / 256);

struct NoAllocScratch {
  double partial[NOALLOC_MAX_PARTIALS * 2];
  unsigned int ticket[NOALLOC_MAX_COUNT];
  float pen[NOALLOC_MAX_JOBS];
};

// Lives in every GPU that loads the library, from load to exit (about 2.2 MB).  In host code
// this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
NoAllocScratch *g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};
int g_noalloc_sms[NOALLOC_MAX_DEVICES] = {};
char g_noalloc_error[256] = "";

int noalloc_fail(int code, const char *msg, cudaError_t e = cudaSuccess) {
  if (e != cudaSuccess) snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s: %s", msg, cudaGetErrorString(e));
  else snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", msg);
  return code;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

const char *eval_fitness_noalloc_last_error(void) { return g_noalloc_error; }

int eval_fitness_noalloc(const int16_t *d_pop, int32_t count, int32_t num_jobs, int32_t num_nodes,
                         int32_t k_max, int32_t n_max, const float *d_speedup, const int16_t *d_cur,
                         const float *d_realloc_factor, const uint8_t *d_active, float p,
                         float speedup_floor, float *d_fitness, void *cuda_stream) {
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (count < 0 || num_jobs < 1 || num_nodes < 1 || k_max < 1 || n_max < 1)
    return noalloc_fail(SCHED_ERR_INVALID_ARG, "eval_fitness_noalloc: sizes must be positive");
  if (count == 0) return SCHED_OK;
  if (!d_pop || !d_speedup || !d_fitness)
    return noalloc_fail(SCHED_ERR_INVALID_ARG, "eval_fitness_noalloc: d_pop, d_speedup and d_fitness must be non-NULL");
  if (count > NOALLOC_MAX_COUNT || num_jobs > NOALLOC_MAX_JOBS || num_nodes > SCHED_MAX_NODES ||
      k_max > SCHED_MAX_K || n_max > SCHED_MAX_N)
    return noalloc_fail(SCHED_ERR_TOO_LARGE,
                        "eval_fitness_noalloc: count <= 2048, num_jobs <= 16384, num_nodes <= 8192, "
                        "k_max, n_max <= 1024 (the scratch array is fixed; use eval_fitness beyond that)");
  if (!(p == p) || !(speedup_floor >= 0.f))
    return noalloc_fail(SCHED_ERR_INVALID_ARG, "eval_fitness_noalloc: p is NaN or speedup_floor negative");
  if (((uintptr_t)d_pop & 1) || ((uintptr_t)d_cur & 1) || ((uintptr_t)d_speedup & 3) || ((uintptr_t)d_fitness & 3))
    return noalloc_fail(SCHED_ERR_INVALID_ARG, "eval_fitness_noalloc: a buffer is not aligned to its element size");

  // set-up, once per device, with that device current: resolve the scratch array's address
  int device = -1;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) return noalloc_fail(SCHED_ERR_CUDA, "cudaGetDevice", e);
  if (device < 0 || device >= NOALLOC_MAX_DEVICES)
    return noalloc_fail(SCHED_ERR_TOO_LARGE, "eval_fitness_noalloc: device ordinal beyond 63");
  if (!g_noalloc_ptr[device]) {
    void *ptr = nullptr;
    e = cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || !ptr) return noalloc_fail(SCHED_ERR_CUDA, "cudaGetSymbolAddress(scratch)", e);
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return noalloc_fail(SCHED_ERR_CUDA, "cudaDeviceGetAttribute", e);
    g_noalloc_sms[device] = sms;
    g_noalloc_ptr[device] = (NoAllocScratch *)ptr;
  }
  NoAllocScratch *scratch = g_noalloc_ptr[device];
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const int J = num_jobs;

  // the arrival counters must start at zero; the array keeps whatever the last call left
  e = cudaMemsetAsync(scratch->ticket, 0, sizeof(unsigned int) * (size_t)count, stream);
  if (e != cudaSuccess) return noalloc_fail(SCHED_ERR_CUDA, "cudaMemsetAsync(ticket)", e);

  const bool penalise = d_cur && d_realloc_factor;
  if (penalise) {
    penalty_prep_kernel<<<(J * 32 + 255) / 256, 256, 0, stream>>>(d_cur, d_realloc_factor, J, num_nodes,
                                                                 scratch->pen);
    e = cudaGetLastError();
    if (e != cudaSuccess) return noalloc_fail(SCHED_ERR_CUDA, "penalty_prep_kernel launch", e);
  }

  int W, lpr_log2, rows_per_block, chunks;
  fitness_geometry((size_t)num_nodes * 2, (uintptr_t)d_pop | (penalise ? (uintptr_t)d_cur : 0), J, count,
                   g_noalloc_sms[device], W, lpr_log2, rows_per_block, chunks);
  if ((size_t)count * (size_t)chunks > NOALLOC_MAX_PARTIALS)   // cannot happen within the limits above
    return noalloc_fail(SCHED_ERR_TOO_LARGE, "eval_fitness_noalloc: chunk sums exceed the scratch array");

  FitnessArgs a;
  a.pop = d_pop;
  a.cur = penalise ? d_cur : nullptr;
  a.table = d_speedup;
  a.pen = penalise ? scratch->pen : nullptr;
  a.active = d_active;
  a.summ = nullptr;
  a.J = J; a.num_nodes = num_nodes; a.k_max = k_max; a.n_max = n_max;
  a.lpr_log2 = lpr_log2;
  a.rows_per_block = rows_per_block; a.chunks = chunks;
  a.p = p; a.floor_ = speedup_floor;
  a.mode = fitness_mode(p);
  a.partial = scratch->partial;
  a.ticket = scratch->ticket;
  a.fitness = d_fitness;
  dim3 grid((unsigned)chunks, (unsigned)count);
  switch (W) {
    case 16: fitness_kernel<16><<<grid, 256, 0, stream>>>(a); break;
    case 8: fitness_kernel<8><<<grid, 256, 0, stream>>>(a); break;
    case 4: fitness_kernel<4><<<grid, 256, 0, stream>>>(a); break;
    default: fitness_kernel<2><<<grid, 256, 0, stream>>>(a); break;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return noalloc_fail(SCHED_ERR_CUDA, "fitness_kernel launch", e);
  return SCHED_OK;
}

#pragma GCC visibility pop
}  // extern "C"
