// Shared declarations of the PolluxSched CUDA library: context, error plumbing,
// the counter-based random stream, small device helpers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <vector>

#include "polluxsched.h"

#define SLOT_SELECT 0u
#define SLOT_XOVER 1u
#define SLOT_MUTATE 2u
#define SLOT_REPAIR_INTF 3u
#define SLOT_REPAIR_CAP 4u
#define SLOT_INIT 5u
#define GEN_INIT 0xFFFFFFFFu

// kernel classes, for launch accounting and optional per-kernel timing
enum KernelKind {
  KK_SWEEP = 0, KK_EXPAND, KK_REALLOC, KK_PENPREP, KK_FITNESS, KK_RANK, KK_ROWS, KK_COLS, KK_BEST,
  KK_COPY, KK_COLSCAN, KK_FIT, KK_GENSTORE, KK_STORE_BUILD, KK_STORE_COMPACT, KK_STORE_GATHER, KK_COUNT
};

struct TimedSpan {
  cudaEvent_t start, stop;
  int kind;
};

// What identifies a round for graph reuse: every pointer it is given and its length.
struct RoundKey {
  sched_jobs jobs;
  const int16_t *cur;
  int16_t *best;
  float *best_fitness;
  int32_t generations;
};

struct sched_ctx {
  sched_config cfg;
  cudaStream_t stream;
  int device;
  int num_sms;
  int KD, ND;
  int64_t launches;
  char err[256];

  // device scratch owned by the context
  int16_t *d_cap;        // [num_nodes]
  int32_t *d_kfit;       // [ND] replicas that fit on the N largest nodes
  int32_t *d_pairs;      // [num_pairs] K * 2 + class of every (K, class) that exists on this cluster
  int num_pairs;
  float *d_gmax;         // [J][KD][2] compact goodput maxima (class local / node)
  uint16_t *d_amax;      // [J][KD][2]
  float *d_gmax_rack;    // [J][KD][2] the same with the rack pair in the node pair's place (allocated on first use)
  uint16_t *d_amax_rack;
  // rack-level locality (sched_set_racks): rack of every node, the third synchronisation pair
  int16_t *d_rack;       // [num_nodes] or NULL when the cluster is not split into racks
  const float *d_alpha_rack, *d_beta_rack;   // caller-owned device arrays [J]
  float *d_tab_speedup_rack;                 // [J][KD][ND] rack-class table of a running round
  int32_t *d_rank;       // [P]
  int32_t *d_order;      // [P] inverse of rank
  uint8_t *d_dflag;      // [P][J] "row spans >= 2 nodes" after the row pass
  float *d_pen;          // [J] effective penalty factor (1 when none applies)
  double *d_partial;     // [count][chunks] partial sums of the fitness reduction
  unsigned int *d_ticket;  // [count] arrival counters of the fitness reduction
  uint32_t *d_collist;   // [count * num_nodes] columns that need repair
  unsigned int *d_colcount;  // [1]
  unsigned int *d_rowticket; // [count] finished row blocks per candidate (kept at zero between kernels)
  size_t rowticket_cap;
  int32_t *d_occcount;   // [count][row batches][num_nodes] occupants recorded per node
  uint32_t *d_occlist;   // [count][row batches][num_nodes][8]
  int32_t *d_colsum, *d_colelig;  // [count][row batches][num_nodes] column partials of the row pass
  size_t partial_cap, ticket_cap, dflag_cap, col_cap;
  int cap_max;           // largest node size
  // state of a running schedule_round: the batched row kernel also emits per-row summaries
  // (K, N, differs-from-current) so that the in-round fitness need not re-read the population
  const int16_t *round_cur;  // current allocation of the round (NULL outside a round)
  uint32_t *round_summ;      // where the running round's row pass writes its summaries, else NULL
  const uint32_t *round_summ_in;  // summaries of the parent population (the other half), or NULL
  uint32_t *d_summ;          // [2][P][J]: parents' and children's summaries alternate
  bool summ_valid;           // the last row/column pass filled d_summ
  // fitness fused into the generation kernel (single-batch problems): inputs set by
  // schedule_round, fit_done reports that the last row/column pass also wrote the fitness
  const float *ff_table, *ff_pen;
  const uint8_t *ff_active;
  float ff_p;
  float *ff_out;
  bool ff_on, fit_done;
  bool pen_ready;        // d_pen already holds this round's factors (set by schedule_round)
  int *d_status;         // device status word
  uint32_t *d_round;     // round number read by the operator kernels

  // scratch of schedule_round (allocated on first use)
  int16_t *d_popA, *d_popB;
  float *d_fit;          // [P] fitness of the current population (points into d_fit_buf)
  float *d_fit_buf;      // [2][P]: parents' and children's fitness alternate between the halves
  float *d_tab_goodput, *d_tab_speedup;
  float *d_rf;           // [J]
  int32_t *d_best_idx;
  int16_t *d_pop_last;   // points at d_popA or d_popB after a round
  bool round_ready;

  // Row store of a running round (large problems): rows live once in a pool and candidates
  // hold row indices, so a child row that equals its parent's costs one index.
  int16_t *rs_pool;        // [2 * rs_half_cap + 1][num_nodes] row contents (last slot: the empty row)
  uint32_t *rs_rec;        // [slots][8] up to 7 occupied nodes of the row (node | GPUs << 12, or an overflow
                           // mark), then K | N << 11 | (entries differing from the current allocation) << 22
  uint32_t *rs_ptr;        // [2][P][J] row index per (candidate, job): parents and children alternate
  unsigned int *rs_state;  // [2][2] {next free slot, half in use}; the two copies alternate at each compaction check;
                           // [4]: times the rows have moved to the other half
  unsigned long long rs_budget;  // bytes the pool (rows + records) may take
  size_t rs_half_cap;      // slots per half of the pool
  int rs_check_every;      // generations between compaction checks
  bool rs_ready;           // the buffers above exist
  bool rs_off;             // the store could not be allocated: rounds run on dense matrices
  const uint32_t *rs_ptr_last;  // indices of the last round's final population, or NULL when it is dense

  // staging for the *_host entry points (allocated on first use)
  void *d_stage;         // job arrays + cur + best
  size_t stage_bytes;
  void *h_stage;         // pinned mirror of the inputs' part of d_stage (small problems: one copy instead of 18)
  size_t h_stage_bytes;
  void *d_stage_fit;     // eval_fitness_host staging
  size_t stage_fit_bytes;

  // CUDA graph of a whole round (see schedule_round)
  bool graphs_enabled, seen_valid;
  uint64_t scratch_epoch;   // bumped whenever a scratch buffer is reallocated: a captured graph
  uint64_t graph_epoch;     // holds raw pointers and is only valid for the epoch it was captured in
  RoundKey seen_key, graph_key;
  cudaGraphExec_t graph_exec;
  int64_t graph_launches;
  float *graph_fit;
  int16_t *graph_pop_last;
  const uint32_t *graph_ptr_last;

  // optional per-kernel timing with CUDA events on the context's stream
  bool timing_on;
  std::vector<TimedSpan> spans;      // recorded since the last read-out
  std::vector<TimedSpan> free_spans; // event pairs ready for reuse
  int64_t spans_dropped;
  int64_t kind_launches[KK_COUNT];
};

// Brackets one kernel launch with a pair of events when timing is enabled.
struct TimedLaunch {
  sched_ctx *ctx;
  TimedSpan span;
  bool on;
  TimedLaunch(sched_ctx *c, int kind);
  ~TimedLaunch();
};

const char *set_error(sched_ctx *ctx, const char *fmt, ...);
extern char g_init_error[256];

#define SCHED_CUDA_CHECK(ctx, call)                                                        \
  do {                                                                                     \
    cudaError_t e__ = (call);                                                              \
    if (e__ != cudaSuccess) {                                                              \
      set_error(ctx, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e__), __FILE__,    \
                __LINE__);                                                                 \
      return SCHED_ERR_CUDA;                                                               \
    }                                                                                      \
  } while (0)

#define SCHED_LAUNCH_CHECK(ctx)                                                            \
  do {                                                                                     \
    (ctx)->launches++;                                                                     \
    cudaError_t e__ = cudaGetLastError();                                                  \
    if (e__ != cudaSuccess) {                                                              \
      set_error(ctx, "kernel launch failed: %s (%s:%d)", cudaGetErrorString(e__),          \
                __FILE__, __LINE__);                                                       \
      return SCHED_ERR_CUDA;                                                               \
    }                                                                                      \
  } while (0)

// ---------------------------------------------------------------------------------------
// Checked build (-DSCHED_CHECKED, `python -m paper_2008_12260_b200.build --checked`): indices
// that kernels compute from data (row slots, node numbers, list positions) are range-tested
// before they are used; a violation records one of the codes below in the context's status word
// (first one wins, read by sched_sync_status) and the access is skipped.  Nothing traps.  In the
// normal build the test compiles away.
// ---------------------------------------------------------------------------------------
#define SCHED_CHK_SLOT (-101)     /* a row slot beyond the pool                           */
#define SCHED_CHK_NODE (-102)     /* a node (or job) number beyond the cluster (the jobs)  */
#define SCHED_CHK_LIST (-103)     /* a position beyond a block's work list                 */
#define SCHED_CHK_ENTRY (-104)    /* a position beyond a row's list of occupied nodes      */

__device__ __forceinline__ bool sched_index_ok(int *status, bool ok, int code) {
#ifdef SCHED_CHECKED
  if (!ok) atomicCAS(status, 0, code);
  return ok;
#else
  (void)status; (void)code; (void)ok;
  return true;
#endif
}

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies; the key is
// advanced by the Weyl constants before every round except the first.
// ---------------------------------------------------------------------------------------
struct u32x4 {
  uint32_t x, y, z, w;
};

__host__ __device__ __forceinline__ u32x4 philox4x32_10(u32x4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // one 32 x 32 -> 64 bit multiply per product (a single wide multiply-add on the device)
    const uint64_t p0 = (uint64_t)0xD2511F53u * c.x, p1 = (uint64_t)0xCD9E8D57u * c.z;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    u32x4 n;
    n.x = hi1 ^ c.y ^ k0;
    n.y = lo1;
    n.z = hi0 ^ c.w ^ k1;
    n.w = lo0;
    c = n;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

// Random stream of the operators: key = (seed_lo ^ seed_hi, round),
// counter = (idx, candidate, generation, slot).  The round number is read from device
// memory so that a captured CUDA graph of a round can be replayed for any round.
struct RngKey {
  uint32_t k0;
  const uint32_t *round_ptr;
};

inline RngKey make_key(uint64_t seed, const uint32_t *d_round) {
  RngKey k;
  k.k0 = (uint32_t)seed ^ (uint32_t)(seed >> 32);
  k.round_ptr = d_round;
  return k;
}

__device__ __forceinline__ u32x4 draw(RngKey k, uint32_t idx, uint32_t cand, uint32_t gen,
                                      uint32_t slot) {
  u32x4 c = {idx, cand, gen, slot};
  return philox4x32_10(c, k.k0, __ldg(k.round_ptr));
}

// floor(w * n / 2^32): an integer in [0, n)
__device__ __forceinline__ uint32_t bounded(uint32_t w, uint32_t n) { return __umulhi(w, n); }

// order-preserving integer image of an fp32 bit pattern
__device__ __forceinline__ uint32_t order_key(uint32_t bits) {
  return bits ^ ((bits >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}

// The better-ranked of two candidates.  A rank is a candidate's position when the population is
// ordered by fitness key descending, index ascending: a permutation, so comparing the two (key,
// index) pairs answers the same question as comparing the two ranks, without counting either.
__device__ __forceinline__ int tournament_winner(uint32_t key_i, int i, uint32_t key_j, int j) {
  return (key_i > key_j || (key_i == key_j && i <= j)) ? i : j;
}

__device__ __forceinline__ int warp_sum(int v) { return __reduce_add_sync(0xffffffffu, v); }

// node index of the t-th occupied entry (ascending) of a row held in shared memory
__device__ __forceinline__ int nth_occupied(const int16_t *row, int num_nodes, uint32_t t, int lane) {
  for (int base = 0; base < num_nodes; base += 32) {
    const int n = base + lane;
    const unsigned m = __ballot_sync(0xffffffffu, n < num_nodes && row[n] > 0);
    const uint32_t c = __popc(m);
    if (t < c) return base + (int)__fns(m, 0, (int)t + 1);
    t -= c;
  }
  return -1;
}

// kernels' launchers (defined in table.cu / fitness.cu / ga.cu / rowstore.cu)
int launch_speedup_table(sched_ctx *ctx, const sched_jobs *jobs, float *d_goodput, float *d_speedup,
                         uint16_t *d_argmax);
int launch_speedup_table_rack(sched_ctx *ctx, const sched_jobs *jobs, const float *d_alpha_rack,
                              const float *d_beta_rack, float *d_goodput, float *d_speedup, uint16_t *d_argmax);
int launch_fitness_racks(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                         const float *d_speedup_rack, const int16_t *d_cur, const float *d_rf,
                         const uint8_t *d_active, float p, float *d_fitness);
int launch_speedup_table_msample(sched_ctx *ctx, const sched_jobs *jobs, const int32_t *d_m_samples, int G,
                                 const int32_t *d_m_max_gpu, const uint8_t *d_adaptive, float *d_goodput,
                                 float *d_speedup, uint16_t *d_argmax);
int launch_realloc_factor(sched_ctx *ctx, const sched_jobs *jobs, float *d_out);
int launch_autoscale(sched_ctx *ctx, const float *d_goodput, const int32_t *d_cur_nodes, int gpn, float U, float L,
                     int32_t *d_target_nodes);
int launch_fitness(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                   const int16_t *d_cur, const float *d_rf, const uint8_t *d_active, float p,
                   float *d_fitness, const uint32_t *d_summ = nullptr);
int launch_repair(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, int16_t *d_pop,
                  int32_t count, uint32_t first_candidate, uint32_t generation);
int launch_init_population(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active,
                           const int16_t *d_cur, int16_t *d_pop_out);
int launch_generation(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active,
                      const int16_t *d_pop_in, const float *d_fitness_in, int16_t *d_pop_out,
                      uint32_t generation, int first_child = 0, int num_children = -1);
int launch_set_round(sched_ctx *ctx, uint32_t round);
int launch_fit(sched_ctx *ctx, int32_t num_jobs, const int32_t *d_offset, const int32_t *d_k, const int32_t *d_n,
               const int32_t *d_m, const int32_t *d_s, const float *d_t, const float *d_theta0,
               const uint8_t *d_frozen, int32_t max_iters, float *d_theta_out, float *d_loss_out);
int launch_select_best(sched_ctx *ctx, const int16_t *d_pop, const float *d_fitness,
                       int16_t *d_best, float *d_best_fitness);
int ensure_fitness_scratch(sched_ctx *ctx, int32_t count, int chunks);
int ensure_dflag(sched_ctx *ctx, int32_t count);
int launch_penalty_prep(sched_ctx *ctx, const int16_t *d_cur, const float *d_rf);
int ensure_colscratch(sched_ctx *ctx, size_t ints);
void fitness_chunking(const sched_ctx *ctx, int32_t count, int &rows_per_block, int &chunks);
// row store (rowstore.cu)
bool rowstore_eligible(const sched_ctx *ctx, const int16_t *d_cur);
int rowstore_ensure(sched_ctx *ctx);
int rowstore_build_current(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, const int16_t *d_seed,
                           const int16_t *d_cur, const float *d_pen);
int rowstore_generation(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, const int16_t *d_cur,
                        const float *d_pen, const float *d_fitness_in, float *d_fitness_out, int parity,
                        int state_phase, uint32_t generation);
int rowstore_compact(sched_ctx *ctx, int parity, int state_phase);
int rowstore_gather(sched_ctx *ctx, const uint32_t *d_ptr, int first_candidate, int count, const int32_t *d_index,
                    int16_t *d_out);
