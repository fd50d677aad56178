/*
 * polluxsched.h - C ABI of the B200-native PolluxSched optimizer core.
 *
 * The library evaluates, on one GPU, the data-parallel part of the cluster-wide
 * optimisation of Pollux (Qiao et al., OSDI'21, Sec. 4.2-4.3): per-job speedup tables
 * from the goodput model (Eq. 4-11, 13, 15), the fitness of a population of allocation
 * matrices (Eq. 14 with the re-allocation penalty), and the population search
 * ("perturbs and combines candidate allocation matrices ... and finally modifies them
 * to satisfy node resource constraints and interference avoidance", Sec. 4.3).
 *
 * Conventions
 *  - Every function returns SCHED_OK (0) or a negative SCHED_ERR_* code; nothing throws,
 *    aborts or traps.  sched_last_error() gives a human-readable reason.
 *  - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  All buffers passed in
 *    are owned by the caller; the library never frees or resizes them.  The context owns
 *    only its internal scratch (allocated in sched_init / on first use, freed in
 *    sched_destroy).
 *  - All work is enqueued on the CUDA stream given to sched_init; calls with device
 *    buffers are asynchronous with respect to the host, calls with host buffers
 *    (`*_host`) return after their results are in the host buffers.
 *  - Matrices are row-major.  An allocation matrix A is int16 [J][num_nodes] (node index
 *    fastest, A[j][n] = GPUs of node n given to job j, Sec. 4.2); a population is
 *    int16 [P][J][num_nodes].  Tables are fp32 [J][k_max+1][n_max+1] indexed by
 *    (job, replicas K, occupied nodes N).
 *  - Entries of allocation matrices are expected in [0, 32767].  Out-of-range values never
 *    cause out-of-bounds accesses: the fitness clamps (K, N) into the table, the
 *    operators first clamp every entry into [0, capacity of its node].
 *  - One context must not be used from two host threads at once.
 */
#ifndef POLLUXSCHED_H_
#define POLLUXSCHED_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SCHED_OK 0
#define SCHED_ERR_INVALID_ARG (-1) /* null pointer, negative size, misaligned buffer   */
#define SCHED_ERR_BAD_CONFIG (-2)  /* a sched_config field outside its documented range */
#define SCHED_ERR_CUDA (-3)        /* a CUDA runtime call failed                        */
#define SCHED_ERR_TIMEOUT (-4)     /* a bounded device-side wait ran out (reserved: no
                                      kernel of this version waits on another)          */
#define SCHED_ERR_NOT_FINITE (-5)  /* a host input array holds a NaN or an infinity     */
#define SCHED_ERR_TOO_LARGE (-6)   /* a size exceeds a documented fixed maximum         */

/* Limits checked by sched_init. */
#define SCHED_MAX_NODES 8192
#define SCHED_MAX_K 1024
#define SCHED_MAX_N 1024

typedef struct sched_ctx sched_ctx; /* opaque, library-owned */

typedef struct {
  int32_t num_nodes;   /* nodes in the cluster, 1..SCHED_MAX_NODES                       */
  int32_t num_jobs;    /* J: rows of every allocation matrix (running + pending jobs)     */
  int32_t k_max;       /* largest replica count tabulated, 1..SCHED_MAX_K                 */
  int32_t n_max;       /* largest node count tabulated, 1..SCHED_MAX_N                    */
  int32_t grid_m;      /* per-GPU batch sizes per job in the (m, s) grid, >= 1            */
  int32_t grid_s;      /* accumulation steps s = 0..grid_s-1; grid_m*grid_s <= 65535      */
  int32_t population;  /* P: candidates evolved by ga_generation / schedule_round, >= 1   */
  float p;             /* exponent of the power mean in Eq. 14 (schedule_round)           */
  float delta_sec;     /* re-allocation delay estimate delta (Sec. 4.2), >= 0             */
  float speedup_floor; /* lower bound applied to every penalised speedup, >= 0            */
  uint32_t thr_mutate; /* a row is perturbed when a 32-bit draw is below this value       */
  uint32_t thr_init;   /* same, for the initial population of a round                     */
  int32_t num_elite;   /* best candidates copied unchanged into the next generation, 0..P */
  uint64_t seed;       /* seed of the counter-based random stream                         */
} sched_config;

/* Per-job inputs, structure of arrays.  The struct lives on the host; for the device
 * entry points every member is a DEVICE pointer to J elements (m_grid: J*grid_m), for
 * the *_host entry points every member is a HOST pointer.  (theta_sys, phi, M0) of
 * Eq. 12 specify each job's goodput function. */
typedef struct {
  const float *alpha_grad, *beta_grad;   /* T_grad(m) = alpha + beta m           (Eq. 8) */
  const float *alpha_local, *beta_local; /* T_sync, all replicas on one node     (Eq. 9) */
  const float *alpha_node, *beta_node;   /* T_sync, replicas on several nodes    (Eq. 9) */
  const float *gamma;                    /* overlap exponent, >= 1               (Eq. 10) */
  const float *phi;                      /* gradient noise scale                 (Eq. 6) */
  const float *m0;                       /* initial batch size M0 (an exact integer)      */
  const float *m_max_total;              /* upper limit of the total batch size M         */
  const int32_t *m_grid;                 /* [J][grid_m] ascending per-GPU batch sizes     */
  const int32_t *k_cap;                  /* max replicas per job (Sec. 4.1 exploration cap);
                                            nullable = k_max                              */
  const int32_t *fair_k, *fair_n;        /* (K, N) of the fair allocation a_f    (Eq. 15) */
  const float *age_sec;                  /* T_j, nullable when no penalty is needed       */
  const int32_t *num_restarts;           /* R_j, nullable likewise                        */
  const uint8_t *active;                 /* nullable = all jobs active; inactive jobs are
                                            left out of Eq. 14 and get empty rows         */
} sched_jobs;

/* Creates a context.  h_node_capacity: HOST array [num_nodes] of GPUs per node (>= 0).
 * cuda_stream: a cudaStream_t (may be NULL for the default stream).  Allocates the
 * context's device scratch (cudaMalloc); the device current at this call is the
 * device the context lives on.  Errors: INVALID_ARG, BAD_CONFIG, TOO_LARGE, CUDA. */
int sched_init(const sched_config *cfg, const int16_t *h_node_capacity, void *cuda_stream,
               sched_ctx **out);

/* The fair allocation a_f of Eq. 15, "an exclusive 1/J share of the cluster", as a (K, N)
 * pair: fair_k = clamp(total GPUs / num_active, 1, k_max) (integer division; the whole
 * cluster when num_active <= 0), placed on as few nodes as possible, fair_n =
 * ceil(fair_k / largest node).  The paper leaves open what the share is when the quotient
 * is fractional or below one GPU; this is the reading the tables are normalised with.
 * Host-only helper, needs no context and no GPU: h_node_capacity is a HOST array
 * [num_nodes] (negative entries count as 0); the results are what sched_jobs.fair_k /
 * fair_n expect for every job.  Errors: INVALID_ARG (NULL pointer, num_nodes < 1,
 * k_max < 1), BAD_CONFIG (the cluster has no GPU). */
int sched_fair_share(const int16_t *h_node_capacity, int32_t num_nodes, int32_t num_active, int32_t k_max,
                     int32_t *fair_k, int32_t *fair_n);

/* Frees the context and its scratch.  NULL is accepted. */
int sched_destroy(sched_ctx *ctx);

/* Reason of the last failure on this context (or of the last failed sched_init when ctx
 * is NULL).  The string is owned by the library and valid until the next call. */
const char *sched_last_error(const sched_ctx *ctx);

/* Waits for the stream and returns the device-side status word (SCHED_OK unless a
 * kernel recorded an error, e.g. SCHED_ERR_TOO_LARGE when the row pool of a round ran
 * out).  A recorded error is reported once: reading it clears the word. */
int sched_sync_status(sched_ctx *ctx);

/* Number of kernels this context has launched so far (for accounting in benchmarks). */
int64_t sched_launch_count(const sched_ctx *ctx);

/* Optional per-kernel timing.  While enabled, every kernel the context launches is
 * bracketed by a pair of CUDA events on the context's stream (at most 131072 pairs between
 * read-outs; further launches are not timed).  sched_read_kernel_timing waits for the
 * stream and writes, per kernel class k in [0, sched_num_kernel_kinds()), the summed
 * device time in milliseconds and the number of timed launches since the previous
 * read-out into HOST arrays of that length.  The paper has no counterpart; this exists so
 * that a benchmark can attribute a round's time to kernels without a profiler. */
int sched_set_kernel_timing(sched_ctx *ctx, int enable);
int sched_num_kernel_kinds(void);
const char *sched_kernel_kind_name(int kind);
int sched_read_kernel_timing(sched_ctx *ctx, float *h_ms_total, int64_t *h_launches);

/* Machine peaks measured in place (the paper has no counterpart; for benchmarks, so that a
 * roofline fraction is taken against the clocks of the moment): the rate of independent fp32
 * FMA chains in lane-operations per second (an FMA counts once; bounds the goodput sweep), the
 * rate of special-function operations (lg2 / ex2 chains; the sweep's co-limit), and the
 * bandwidth of a read-only stream of 16-byte loads over d_buffer (DEVICE, 16-byte aligned,
 * `bytes` long, only read; NULL skips it and reports 0; bounds the dense fitness kernel).
 * Each figure is the mean of `reps` launches after one warm-up, timed with CUDA events on the
 * context's stream; the call waits.  Outputs are HOST doubles. */
int sched_measure_peaks(sched_ctx *ctx, const void *d_buffer, uint64_t bytes, int32_t reps,
                        double *h_fp32_lane_ops_per_s, double *h_mufu_ops_per_s, double *h_read_bytes_per_s);

/* Speedup tables (Eq. 13 and 15).  For every job and every (K, N) with 1 <= N <= n_max,
 * N <= K <= k_max and K no larger than the N largest nodes together:
 *   goodput[j][K][N] = max over the grid {m_grid[j][i]} x {s} of GOODPUT(a, m, s) (Eq. 4)
 *                      subject to M0 <= K m (s+1) <= m_max_total,
 *   argmax[j][K][N]  = i * grid_s + s of a maximiser,
 *   speedup[j][K][N] = goodput[j][K][N] / goodput[j][fair_k][fair_n].
 * All other entries are 0 (argmax 0xFFFF); so are entries with no feasible grid point,
 * and a job's whole speedup slab when its fair-share goodput is 0.  Outputs are
 * fp32/uint16 [J][k_max+1][n_max+1]; d_goodput and d_argmax may be NULL.  Batch sizes
 * must satisfy K m (s+1) < 2^24 for the feasibility test to be exact.
 * Uses: all fp32 members of jobs, m_grid, fair_k, fair_n. */
int build_speedup_table(sched_ctx *ctx, const sched_jobs *d_jobs, float *d_goodput,
                        float *d_speedup, uint16_t *d_argmax);

/* Speedup tables with the (m, s) sub-procedure as the paper words it (Sec. 4.3) instead of a
 * fixed grid: d_m_samples (int32 [J][num_samples]) holds candidate total batch sizes M; for
 * each, per_gpu = ceil(M / K), s = ceil(per_gpu / m_max_gpu[j]) - 1 is the smallest number of
 * accumulation steps whose per-GPU batch m = ceil(per_gpu / (s + 1)) fits the limit, the
 * batch run is M' = K m (s + 1) and must satisfy M0 <= M' <= m_max_total; the best goodput
 * over the candidates is tabulated (ties: smallest candidate index; argmax = candidate
 * index).  Jobs with d_adaptive[j] == 0 (d_adaptive nullable = all adaptive) are the
 * non-adaptive jobs of Sec. 4.2: the single candidate M = M0 with EFFICIENCY fixed to 1.
 * Outputs, validity of (K, N) and normalisation as build_speedup_table; m_grid is not used. */
int build_speedup_table_msample(sched_ctx *ctx, const sched_jobs *d_jobs, const int32_t *d_m_samples,
                                int32_t num_samples, const int32_t *d_m_max_gpu, const uint8_t *d_adaptive,
                                float *d_goodput, float *d_speedup, uint16_t *d_argmax);

/* Rack-level locality: "our model for T_sync can be extended to account for rack-level locality
 * by adding a third pair of parameters" (the sentence after Eq. 9).  Read as three placement
 * classes: all replicas on one node -> local pair; several nodes of one rack -> node pair;
 * nodes of two or more racks -> rack pair, T_sync = alpha_rack + beta_rack (K - 2).
 *
 * sched_set_racks gives the context the rack of every node (h_node_rack: HOST int16
 * [num_nodes], rack ids >= 0; NULL: one rack again) and the rack pair (DEVICE fp32 [J] each,
 * caller-owned, must stay valid while the context uses them; NULL = the node pair).  To be
 * called before the first schedule_round.  With racks set, schedule_round builds the
 * third-class table as well and evaluates every candidate with eval_fitness_racks; such rounds
 * run on dense matrices (the shared-row representation is not used).
 *
 * build_speedup_table_rack: tables of the third class.  Entry (K, N) with N >= 2 (valid as in
 * build_speedup_table) is the best goodput over the grid with the rack pair, and its ratio to
 * the SAME fair-share goodput as the two-class table (the fair share is packed on as few nodes
 * as possible, so inside one rack); entries with N < 2 are 0 / 0xFFFF.  Outputs as
 * build_speedup_table; d_goodput and d_argmax may be NULL.
 *
 * eval_fitness_racks: eval_fitness, but a row whose occupied nodes lie in two or more racks
 * reads d_speedup_rack instead of d_speedup.  Needs sched_set_racks. */
int sched_set_racks(sched_ctx *ctx, const int16_t *h_node_rack, const float *d_alpha_rack, const float *d_beta_rack);
int build_speedup_table_rack(sched_ctx *ctx, const sched_jobs *d_jobs, const float *d_alpha_rack,
                             const float *d_beta_rack, float *d_goodput, float *d_speedup, uint16_t *d_argmax);
int eval_fitness_racks(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                       const float *d_speedup_rack, const int16_t *d_cur, const float *d_realloc_factor,
                       const uint8_t *d_active, float p, float *d_fitness);

/* Batched fit of the throughput-model parameters (Sec. 4.1, online model fitting).  For each
 * of num_jobs jobs (independent of cfg.num_jobs) the observations offset[j] .. offset[j+1] of
 * (K, N, m, s, T_iter) are fitted by theta = (alpha_grad, beta_grad, alpha_local, beta_local,
 * alpha_node, beta_node, gamma) minimising the root mean squared logarithmic error
 * sqrt(mean((ln(1 + T_pred) - ln(1 + T_obs))^2)) with T_pred from Eq. 11, subject to
 * alpha, beta >= 0 and 1 <= gamma <= 10, starting from d_theta0 (fp32 [num_jobs][7], clamped
 * into the bounds).  Bit i of d_frozen[j] (nullable) holds parameter i at its starting value:
 * the paper's prior-driven exploration keeps unexplored synchronisation parameters at 0
 * this way.  At most max_iters damped Gauss-Newton steps per job.  Outputs: d_theta_out fp32
 * [num_jobs][7], d_loss_out fp32 [num_jobs] (the error reached; 0 for a job without
 * observations, whose theta is returned unchanged).  The minimiser found is a local one. */
int fit_throughput_model(sched_ctx *ctx, int32_t num_jobs, const int32_t *d_obs_offset, const int32_t *d_obs_k,
                         const int32_t *d_obs_n, const int32_t *d_obs_m, const int32_t *d_obs_s,
                         const float *d_obs_t, const float *d_theta0, const uint8_t *d_frozen, int32_t max_iters,
                         float *d_theta_out, float *d_loss_out);

/* REALLOC_FACTOR_j(delta) = (T_j - R_j delta) / (T_j + delta) clamped to [0, 1]
 * (Sec. 4.2), with delta = cfg.delta_sec.  d_out: fp32 [J].  Uses age_sec, num_restarts. */
int compute_realloc_factor(sched_ctx *ctx, const sched_jobs *d_jobs, float *d_out);

/* Goodput-driven auto-scaling rule (Sec. 5.3, "Cloud auto-scaling").  For a job that holds
 * d_cur_nodes[j] whole nodes of gpus_per_node GPUs, with g(n) = goodput[j][n G][n] and the
 * ideal n G goodput[j][1][1] of perfect scalability: if g(cur) > U * ideal(cur) the target is
 * the largest n > cur (n <= n_max, n G <= k_max) with g(n) >= L * ideal(n), or cur if there
 * is none; otherwise the target is cur (the rule never scales down).  The paper uses
 * U = 2/3, L = 1/2.  d_goodput: fp32 [J][k_max+1][n_max+1] from build_speedup_table;
 * d_cur_nodes, d_target_nodes: int32 [J].  Jobs with cur < 1 or beyond the table keep cur. */
int autoscale_targets(sched_ctx *ctx, const float *d_goodput, const int32_t *d_cur_nodes, int32_t gpus_per_node,
                      float U, float L, int32_t *d_target_nodes);

/* Fitness of `count` candidates (Eq. 14).  d_pop: int16 [count][J][num_nodes].  For each
 * active job the speedup is read at (K, N) = (sum of the row, entries > 0), clamped to
 * the table; if d_cur (int16 [J][num_nodes]) and d_realloc_factor (fp32 [J]) are both
 * given, a row that differs from a non-empty current row is multiplied by the job's
 * factor; the result is raised to cfg.speedup_floor; the power mean with exponent p
 * over the active jobs is written to d_fitness[count] (p = 0: geometric mean; no active
 * job: 0; with num_jobs = 0 the matrices and the table are empty and d_pop, d_speedup may be
 * NULL).  d_active: uint8 [J], nullable.  `count` may differ from cfg.population. */
int eval_fitness(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                 const int16_t *d_cur, const float *d_realloc_factor, const uint8_t *d_active,
                 float p, float *d_fitness);

/* The repair step alone, in place, on `count` matrices: entries into [0, node size], per-job
 * replica cap (k_cap, highest node index first) and n_max, then at most one distributed
 * job per node (interference avoidance, Sec. 4.2) and node capacity, the last two with
 * job order rotated by draws of the random stream addressed by (round, first_candidate
 * + c, generation).  Removal only; feasible matrices are left unchanged.
 * Uses k_cap, active (jobs may be NULL: no cap beyond k_max, all active). */
int repair_population(sched_ctx *ctx, const sched_jobs *d_jobs, int16_t *d_pop, int32_t count,
                      uint32_t first_candidate, uint32_t round, uint32_t generation);

/* Initial population of a round: candidate 0 is d_cur (NULL = empty cluster), candidates
 * 1..P-1 are d_cur with rows perturbed with threshold thr_init; all repaired.
 * d_pop_out: int16 [P][J][num_nodes]. */
int init_population(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_cur,
                    uint32_t round, int16_t *d_pop_out);

/* One generation of the population search (Sec. 4.3).  Children 0..num_elite-1 are the
 * best-ranked parents (fitness descending, index ascending, compared by bit pattern);
 * every other child takes each job's row from one of two parents (each the better of two
 * random candidates), perturbs it with threshold thr_mutate (grow / shrink / relocate)
 * and is repaired.  d_pop_in, d_pop_out: int16 [P][J][num_nodes], must not overlap;
 * d_fitness_in: fp32 [P].  The result is a pure function of the inputs, cfg.seed, round
 * and generation.  Uses k_cap, active (jobs may be NULL). */
int ga_generation(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_pop_in,
                  const float *d_fitness_in, int16_t *d_pop_out, uint32_t round,
                  uint32_t generation);

/* A slice of ga_generation: children first_child .. first_child + num_children - 1, bit for bit
 * the children that ga_generation puts at those positions (a child depends on its own index,
 * the parents and their fitness only).  This is how the population search of Sec. 4.3 shards
 * by candidate over several GPUs: every GPU holds all parents and their fitness, makes its
 * share of the children and evaluates them (eval_fitness with count = num_children), and the
 * caller gathers children and fitness between generations (see dist.evolve_sharded in the
 * Python package).  d_pop_in: int16 [P][J][num_nodes] and d_fitness_in: fp32 [P], all parents;
 * d_children: int16 [num_children][J][num_nodes], must not overlap the parents.
 * Errors: INVALID_ARG when the slice leaves [0, P). */
int ga_generation_shard(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_pop_in, const float *d_fitness_in,
                        int32_t first_child, int32_t num_children, int16_t *d_children, uint32_t round,
                        uint32_t generation);

/* A whole scheduling round: tables, re-allocation factors, initial population and its
 * fitness, `generations` x (ga_generation, eval_fitness), then the best candidate of the
 * last population.  d_cur: int16 [J][num_nodes] or NULL.  d_best: int16 [J][num_nodes],
 * d_best_fitness: fp32 [1].  Population and table buffers are context scratch allocated
 * on the first call.  Problems with more than 256 jobs (rows of whole 16-byte pieces, at
 * most 512 nodes and 8192 jobs) keep the population of the round as shared rows - row
 * indices per candidate into a pool of rows, copy on write - instead of dense matrices;
 * the results are the same bit for bit, the scratch is larger (see sched_set_store_budget),
 * and a pool overflow
 * (not expected: the pool is compacted before it can run out) would be reported as device
 * status SCHED_ERR_TOO_LARGE by sched_sync_status.  If the pool cannot be allocated the
 * round runs on dense matrices. */
int schedule_round(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_cur, uint32_t round,
                   int32_t generations, int16_t *d_best, float *d_best_fitness);

/* Memory the shared-row pool of schedule_round may take (rows + records; default 12 GiB), to be
 * set before the first schedule_round of the context.  The pool is sized at twice (the
 * population + as many worst-case generations as the budget allows, at most 24); with less
 * room the live rows move between the halves more often (same results, more time), and when
 * not even two worst-case generations fit, rounds run on dense matrices.  The paper has no
 * counterpart: a deployment knob.  sched_store_moves: how often the rows have moved since the
 * context was made (waits for the stream; 0 when rounds run on dense matrices, -1 on a CUDA
 * error). */
int sched_set_store_budget(sched_ctx *ctx, uint64_t bytes);
int64_t sched_store_moves(sched_ctx *ctx);

/* schedule_round replays a CUDA graph of the whole round from the third call on that passes
 * the same pointers and generation count (the second such call captures it); this removes
 * the per-kernel launch cost that dominates small problems.  Results are identical with
 * and without graphs.  On by default; not used on the NULL stream or while per-kernel
 * timing is enabled.  sched_set_graphs(ctx, 0) turns it off. */
int sched_set_graphs(sched_ctx *ctx, int enable);

/* Same with HOST buffers: copies the job arrays and h_cur to the device, runs the round,
 * copies the result back and waits for it.  Every member of h_jobs is a host pointer.
 * Because the arrays are on the host they are validated first: SCHED_ERR_NOT_FINITE when a
 * goodput-model parameter or age_sec is NaN or infinite;
 * SCHED_ERR_INVALID_ARG when alpha or beta is negative, gamma < 1, phi < 0, M0 < 1,
 * m_max_total < M0, a batch size of m_grid is < 1, age_sec or num_restarts is negative, or
 * an entry of h_cur is negative (Eq. 8-11 and Sec. 4.2 give these ranges).  The device
 * status word is read back with the result: a device-side error of the round (see
 * schedule_round) is this call's return value. */
int schedule_round_host(sched_ctx *ctx, const sched_jobs *h_jobs, const int16_t *h_cur,
                        uint32_t round, int32_t generations, int16_t *h_best,
                        float *h_best_fitness);

/* Copies the population and fitness left by the last schedule_round into caller buffers
 * (either may be NULL).  d_pop_out: int16 [P][J][num_nodes], d_fitness_out: fp32 [P]. */
int sched_get_population(sched_ctx *ctx, int16_t *d_pop_out, float *d_fitness_out);

/* Copies the goodput and speedup tables built by the last schedule_round (Eq. 13, 15) into
 * caller buffers, fp32 [J][k_max+1][n_max+1] each, either may be NULL.  goodput[j][K][N] is
 * the predicted goodput of job j at its best (m, s) on that allocation: what a simulator
 * needs to advance the job's training progress. */
int sched_get_round_tables(sched_ctx *ctx, float *d_goodput_out, float *d_speedup_out);

/* Pointer to the fp32 [J][k_max+1][n_max+1] speedup table built by the last schedule_round
 * (context scratch, device memory), or NULL before the first round. */
const float *sched_round_speedup_table(const sched_ctx *ctx);

/* Fitness with HOST buffers (population, table, optional cur / factors / active mask are
 * copied in, fitness copied out, the call waits).  Staging buffers are context scratch.
 * Validated first: SCHED_ERR_NOT_FINITE when h_speedup or h_realloc_factor holds a NaN or an
 * infinity; SCHED_ERR_INVALID_ARG when a speedup is negative or a factor lies outside [0, 1]. */
int eval_fitness_host(sched_ctx *ctx, const int16_t *h_pop, int32_t count, const float *h_speedup,
                      const int16_t *h_cur, const float *h_realloc_factor,
                      const uint8_t *h_active, float p, float *h_fitness);

/* Limits of eval_fitness_noalloc (its scratch array is sized for exactly these). */
#define SCHED_NOALLOC_MAX_COUNT 2048
#define SCHED_NOALLOC_MAX_JOBS 16384

/* eval_fitness for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of the Eq. 14 evaluation above, same kernels,
 * same results.)
 *
 * Who needs it: a scheduler embedded in a process whose GPU memory is handed out in full
 * to a caching allocator at start-up, where a later cudaMalloc can simply fail; and
 * latency-critical control loops that cannot accept the device-wide synchronisation a
 * cudaMalloc / cudaFree implies.  sched_init and the first eval_fitness call of a context
 * allocate their scratch; this entry point never calls cudaMalloc, cudaFree or any
 * allocating library routine.  It needs no context: sizes and the floor are passed
 * directly, and all work is enqueued on `cuda_stream` (a cudaStream_t, NULL = default
 * stream) of the current device.
 *
 * Its scratch (per-chunk partial sums, arrival counters, per-job penalty factors) is one
 * fixed file-scope device array of about 2.2 MB that every GPU holding the library keeps
 * from load to exit.  Hence fixed maxima: count <= SCHED_NOALLOC_MAX_COUNT, num_jobs <=
 * SCHED_NOALLOC_MAX_JOBS, num_nodes <= SCHED_MAX_NODES, k_max <= SCHED_MAX_K, n_max <=
 * SCHED_MAX_N; anything larger returns SCHED_ERR_TOO_LARGE (use eval_fitness, in chunks if
 * need be).  The first call on each device resolves the array's device address (one
 * cudaGetSymbolAddress, with that device current) and reads the SM count; make that first
 * call before any stream capture.  All calls share the one array: the part a call relies
 * on being zero is cleared on the stream at the start of each call, the rest is
 * overwritten before it is read, but two calls whose kernels overlap on the GPU (different
 * streams, or different host threads on different streams) race on it - serialise them.
 * Host-side the call is guarded by a mutex.
 *
 * Arguments as eval_fitness: d_pop int16 [count][num_jobs][num_nodes], d_speedup fp32
 * [num_jobs][k_max+1][n_max+1], optional d_cur / d_realloc_factor / d_active, exponent p,
 * floor, d_fitness fp32 [count].  Errors: INVALID_ARG, TOO_LARGE, CUDA; the reason is in
 * eval_fitness_noalloc_last_error(). */
int eval_fitness_noalloc(const int16_t *d_pop, int32_t count, int32_t num_jobs, int32_t num_nodes,
                         int32_t k_max, int32_t n_max, const float *d_speedup, const int16_t *d_cur,
                         const float *d_realloc_factor, const uint8_t *d_active, float p,
                         float speedup_floor, float *d_fitness, void *cuda_stream);
const char *eval_fitness_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* POLLUXSCHED_H_ */
