// C-ABI entry points: argument validation, context and scratch management, and the
// scheduling-round driver.  All arithmetic of the method lives in the kernels.
#include <stdarg.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "common.cuh"

char g_init_error[256] = "";

const char *set_error(sched_ctx *ctx, const char *fmt, ...) {
  char *dst = ctx ? ctx->err : g_init_error;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 256, fmt, ap);
  va_end(ap);
  return dst;
}

TimedLaunch::TimedLaunch(sched_ctx *c, int kind) : ctx(c), on(false) {
  span.kind = kind;
  c->kind_launches[kind]++;
  if (!c->timing_on) return;
  if (!c->free_spans.empty()) {
    span.start = c->free_spans.back().start;
    span.stop = c->free_spans.back().stop;
    c->free_spans.pop_back();
  } else {
    if (c->spans.size() >= (1u << 17)) { c->spans_dropped++; return; }
    if (cudaEventCreate(&span.start) != cudaSuccess) return;
    if (cudaEventCreate(&span.stop) != cudaSuccess) { cudaEventDestroy(span.start); return; }
  }
  on = true;
  cudaEventRecord(span.start, c->stream);
}

TimedLaunch::~TimedLaunch() {
  if (!on) return;
  cudaEventRecord(span.stop, ctx->stream);
  ctx->spans.push_back(span);
}

namespace {

template <typename T>
int dev_alloc(sched_ctx *ctx, T **p, size_t n) {
  *p = nullptr;
  if (n == 0) n = 1;
  SCHED_CUDA_CHECK(ctx, cudaMalloc((void **)p, n * sizeof(T)));
  ctx->scratch_epoch++;
  return SCHED_OK;
}

#define REQUIRE(ctx, cond, code, ...)   \
  do {                                  \
    if (!(cond)) {                      \
      set_error(ctx, __VA_ARGS__);      \
      return code;                      \
    }                                   \
  } while (0)

int check_table_jobs(sched_ctx *ctx, const sched_jobs *j) {
  REQUIRE(ctx, j, SCHED_ERR_INVALID_ARG, "jobs is NULL");
  REQUIRE(ctx, j->alpha_grad && j->beta_grad && j->alpha_local && j->beta_local && j->alpha_node &&
                   j->beta_node && j->gamma && j->phi && j->m0 && j->m_max_total && j->m_grid &&
                   j->fair_k && j->fair_n,
          SCHED_ERR_INVALID_ARG, "jobs: a goodput-model array, m_grid, fair_k or fair_n is NULL");
  return SCHED_OK;
}

int ensure_round_scratch(sched_ctx *ctx) {
  if (ctx->round_ready) return SCHED_OK;
  const sched_config &c = ctx->cfg;
  const size_t pop = (size_t)c.population * c.num_jobs * c.num_nodes;
  const size_t tab = (size_t)c.num_jobs * ctx->KD * ctx->ND;
  int rc;
  // Large problems keep the round's population in the row store, whose pool starts with the
  // dense initial population; if it cannot be allocated the round runs on dense matrices.
  if (rowstore_eligible(ctx, nullptr) && !ctx->rs_off && !ctx->d_rack) {
    if (rowstore_ensure(ctx) != SCHED_OK) ctx->rs_off = true;
  }
  if (!ctx->rs_ready) {
    if ((rc = dev_alloc(ctx, &ctx->d_popA, pop)) != SCHED_OK) return rc;
    if ((rc = dev_alloc(ctx, &ctx->d_popB, pop)) != SCHED_OK) return rc;
  }
  if ((rc = dev_alloc(ctx, &ctx->d_fit_buf, 2 * (size_t)c.population)) != SCHED_OK) return rc;
  ctx->d_fit = ctx->d_fit_buf;
  if ((rc = dev_alloc(ctx, &ctx->d_tab_goodput, tab)) != SCHED_OK) return rc;
  if ((rc = dev_alloc(ctx, &ctx->d_tab_speedup, tab)) != SCHED_OK) return rc;
  if (ctx->d_rack && (rc = dev_alloc(ctx, &ctx->d_tab_speedup_rack, tab)) != SCHED_OK) return rc;
  if ((rc = dev_alloc(ctx, &ctx->d_rf, (size_t)c.num_jobs)) != SCHED_OK) return rc;
  if ((rc = dev_alloc(ctx, &ctx->d_summ, 2 * (size_t)c.population * c.num_jobs)) != SCHED_OK) return rc;
  ctx->round_ready = true;
  return SCHED_OK;
}

}  // namespace

int ensure_fitness_scratch(sched_ctx *ctx, int32_t count, int chunks) {
  const size_t need_p = (size_t)count * chunks * 2;
  if (need_p > ctx->partial_cap) {
    if (ctx->d_partial) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_partial));
    }
    int rc = dev_alloc(ctx, &ctx->d_partial, need_p);
    if (rc != SCHED_OK) { ctx->partial_cap = 0; return rc; }
    ctx->partial_cap = need_p;
  }
  if ((size_t)count > ctx->ticket_cap) {
    if (ctx->d_ticket) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_ticket));
    }
    int rc = dev_alloc(ctx, &ctx->d_ticket, (size_t)count);
    if (rc != SCHED_OK) { ctx->ticket_cap = 0; return rc; }
    ctx->ticket_cap = (size_t)count;
    SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->d_ticket, 0, (size_t)count * sizeof(unsigned int), ctx->stream));
  }
  return SCHED_OK;
}

int ensure_dflag(sched_ctx *ctx, int32_t count) {
  const size_t need = (size_t)count * ctx->cfg.num_jobs;
  if (need > ctx->dflag_cap) {
    if (ctx->d_dflag) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_dflag));
    }
    int rc = dev_alloc(ctx, &ctx->d_dflag, need);
    if (rc != SCHED_OK) { ctx->dflag_cap = 0; return rc; }
    ctx->dflag_cap = need;
  }
  return SCHED_OK;
}

int ensure_colscratch(sched_ctx *ctx, size_t ints) {
  const size_t tickets = (size_t)65536;   // one per candidate of a launch
  if (!ctx->d_rowticket) {
    int rc = dev_alloc(ctx, &ctx->d_rowticket, tickets);
    if (rc != SCHED_OK) return rc;
    SCHED_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->d_rowticket, 0, tickets * sizeof(unsigned int), ctx->stream));
    ctx->rowticket_cap = tickets;
  }
  if (ints > ctx->col_cap) {
    if (ctx->d_colsum || ctx->d_colelig) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      if (ctx->d_colsum) SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_colsum));
      if (ctx->d_colelig) SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_colelig));
      ctx->d_colsum = ctx->d_colelig = nullptr;
    }
    ctx->col_cap = 0;
    int rc = dev_alloc(ctx, &ctx->d_colsum, ints);
    if (rc != SCHED_OK) return rc;
    rc = dev_alloc(ctx, &ctx->d_colelig, ints);
    if (rc != SCHED_OK) return rc;
    if (ctx->d_collist) SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_collist));
    rc = dev_alloc(ctx, &ctx->d_collist, ints);
    if (rc != SCHED_OK) return rc;
    if (ctx->d_occcount) SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_occcount));
    if (ctx->d_occlist) SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_occlist));
    rc = dev_alloc(ctx, &ctx->d_occcount, ints);
    if (rc != SCHED_OK) return rc;
    rc = dev_alloc(ctx, &ctx->d_occlist, ints * 8);
    if (rc != SCHED_OK) return rc;
    ctx->col_cap = ints;
  }
  return SCHED_OK;
}

extern "C" {
#pragma GCC visibility push(default)

int sched_init(const sched_config *cfg, const int16_t *h_node_capacity, void *cuda_stream,
               sched_ctx **out) {
  if (out) *out = nullptr;
  REQUIRE(nullptr, cfg && h_node_capacity && out, SCHED_ERR_INVALID_ARG,
          "sched_init: cfg, h_node_capacity and out must be non-NULL");
  REQUIRE(nullptr, cfg->num_nodes >= 1 && cfg->num_jobs >= 0 && cfg->k_max >= 1 && cfg->n_max >= 1 &&
                       cfg->grid_m >= 1 && cfg->grid_s >= 1 && cfg->population >= 1,
          SCHED_ERR_BAD_CONFIG, "sched_init: sizes must be positive (num_jobs may be 0)");
  REQUIRE(nullptr, cfg->num_nodes <= SCHED_MAX_NODES && cfg->k_max <= SCHED_MAX_K &&
                       cfg->n_max <= SCHED_MAX_N,
          SCHED_ERR_TOO_LARGE, "sched_init: num_nodes <= %d, k_max <= %d, n_max <= %d",
          SCHED_MAX_NODES, SCHED_MAX_K, SCHED_MAX_N);
  REQUIRE(nullptr, (long long)cfg->grid_m * cfg->grid_s <= 65535, SCHED_ERR_TOO_LARGE,
          "sched_init: grid_m * grid_s must be <= 65535");
  REQUIRE(nullptr, cfg->num_elite >= 0 && cfg->num_elite <= cfg->population, SCHED_ERR_BAD_CONFIG,
          "sched_init: num_elite must be in [0, population]");
  REQUIRE(nullptr, cfg->delta_sec >= 0.f && cfg->speedup_floor >= 0.f && cfg->p == cfg->p,
          SCHED_ERR_BAD_CONFIG, "sched_init: delta_sec and speedup_floor must be >= 0, p not NaN");
  REQUIRE(nullptr, (long long)cfg->population * cfg->num_jobs < (1LL << 31), SCHED_ERR_TOO_LARGE,
          "sched_init: population * num_jobs must be below 2^31");

  sched_ctx *ctx = new (std::nothrow) sched_ctx();
  REQUIRE(nullptr, ctx, SCHED_ERR_CUDA, "sched_init: out of host memory");
  ctx->cfg = *cfg;
  ctx->stream = (cudaStream_t)cuda_stream;
  ctx->KD = cfg->k_max + 1;
  ctx->ND = cfg->n_max + 1;

  auto fail = [&](int rc) {
    strncpy(g_init_error, ctx->err, sizeof(g_init_error) - 1);
    sched_destroy(ctx);
    return rc;
  };
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e != cudaSuccess) {
    set_error(ctx, "sched_init: no usable CUDA device: %s", cudaGetErrorString(e));
    return fail(SCHED_ERR_CUDA);
  }

  // replicas that fit on the N largest nodes, N = 0..n_max
  std::vector<int16_t> sorted(h_node_capacity, h_node_capacity + cfg->num_nodes);
  std::sort(sorted.begin(), sorted.end(), [](int16_t a, int16_t b) { return a > b; });
  ctx->cap_max = std::max<int>(sorted[0], 0);
  std::vector<int32_t> kfit(ctx->ND, 0);
  for (int n = 1; n < ctx->ND; ++n) {
    const int add = (n <= cfg->num_nodes && sorted[n - 1] > 0) ? sorted[n - 1] : 0;
    kfit[n] = kfit[n - 1] + add;
  }

  const size_t J = (size_t)cfg->num_jobs, P = (size_t)cfg->population;
  int rc;
  if ((rc = dev_alloc(ctx, &ctx->d_cap, ((size_t)cfg->num_nodes + 7) & ~(size_t)7)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_kfit, (size_t)ctx->ND)) != SCHED_OK) return fail(rc);
  // (K, class) pairs that exist: class 0 (one node) needs K <= largest node; class 1 (several
  // nodes) needs K >= 2 and K <= the min(K, n_max) largest nodes together
  std::vector<int32_t> pairs;
  for (int K = 1; K <= cfg->k_max; ++K) {
    if (K <= kfit[1]) pairs.push_back(K * 2);
    if (cfg->n_max >= 2 && K >= 2 && K <= kfit[std::min(K, cfg->n_max)]) pairs.push_back(K * 2 + 1);
  }
  ctx->num_pairs = (int)pairs.size();
  if ((rc = dev_alloc(ctx, &ctx->d_pairs, pairs.size())) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_gmax, J * ctx->KD * 2)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_amax, J * ctx->KD * 2)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_rank, P)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_order, P)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_pen, J)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_status, 1)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_best_idx, 1)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_colcount, 1)) != SCHED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_round, 1)) != SCHED_OK) return fail(rc);
  ctx->graphs_enabled = true;
  ctx->rs_budget = 12ull << 30;
  e = cudaMemcpyAsync(ctx->d_cap, h_node_capacity, sizeof(int16_t) * cfg->num_nodes,
                      cudaMemcpyHostToDevice, ctx->stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(ctx->d_kfit, kfit.data(), sizeof(int32_t) * ctx->ND, cudaMemcpyHostToDevice, ctx->stream);
  if (e == cudaSuccess && !pairs.empty())
    e = cudaMemcpyAsync(ctx->d_pairs, pairs.data(), sizeof(int32_t) * pairs.size(), cudaMemcpyHostToDevice, ctx->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_gmax, 0, sizeof(float) * std::max<size_t>(J * ctx->KD * 2, 1), ctx->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_amax, 0xFF, sizeof(uint16_t) * std::max<size_t>(J * ctx->KD * 2, 1), ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);   // host vectors go out of scope
  if (e != cudaSuccess) {
    set_error(ctx, "sched_init: upload failed: %s", cudaGetErrorString(e));
    return fail(SCHED_ERR_CUDA);
  }
  *out = ctx;
  return SCHED_OK;
}

int sched_fair_share(const int16_t *h_node_capacity, int32_t num_nodes, int32_t num_active, int32_t k_max,
                     int32_t *fair_k, int32_t *fair_n) {
  REQUIRE(nullptr, h_node_capacity && fair_k && fair_n, SCHED_ERR_INVALID_ARG,
          "sched_fair_share: h_node_capacity, fair_k and fair_n must be non-NULL");
  REQUIRE(nullptr, num_nodes >= 1 && k_max >= 1, SCHED_ERR_INVALID_ARG,
          "sched_fair_share: num_nodes and k_max must be positive");
  long long total = 0, largest = 0;
  for (int32_t n = 0; n < num_nodes; ++n) {
    const long long g = h_node_capacity[n] > 0 ? h_node_capacity[n] : 0;
    total += g;
    largest = std::max(largest, g);
  }
  REQUIRE(nullptr, largest > 0, SCHED_ERR_BAD_CONFIG, "sched_fair_share: the cluster has no GPU");
  long long k = num_active > 0 ? total / num_active : total;
  k = std::min<long long>(std::max<long long>(k, 1), k_max);
  *fair_k = (int32_t)k;
  *fair_n = (int32_t)((k + largest - 1) / largest);
  return SCHED_OK;
}

int sched_destroy(sched_ctx *ctx) {
  if (!ctx) return SCHED_OK;
  cudaStreamSynchronize(ctx->stream);
  void *ptrs[] = {ctx->d_cap, ctx->d_kfit, ctx->d_pairs, ctx->d_gmax, ctx->d_amax, ctx->d_rank, ctx->d_order,
                  ctx->d_dflag, ctx->d_pen, ctx->d_partial, ctx->d_ticket, ctx->d_status,
                  ctx->d_popA, ctx->d_popB, ctx->d_fit_buf, ctx->d_tab_goodput, ctx->d_tab_speedup,
                  ctx->d_rf, ctx->d_best_idx, ctx->d_stage, ctx->d_stage_fit, ctx->d_colsum, ctx->d_summ, ctx->d_collist, ctx->d_colcount, ctx->d_rowticket, ctx->d_round, ctx->d_occcount, ctx->d_occlist,
                  ctx->d_colelig, ctx->rs_pool, ctx->rs_rec, ctx->rs_ptr, ctx->rs_state, ctx->d_gmax_rack,
                  ctx->d_amax_rack, ctx->d_rack, ctx->d_tab_speedup_rack};
  for (void *p : ptrs)
    if (p) cudaFree(p);
  if (ctx->h_stage) cudaFreeHost(ctx->h_stage);
  if (ctx->graph_exec) cudaGraphExecDestroy(ctx->graph_exec);
  for (auto *v : {&ctx->spans, &ctx->free_spans})
    for (TimedSpan &t : *v) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
  delete ctx;
  return SCHED_OK;
}

const char *sched_last_error(const sched_ctx *ctx) { return ctx ? ctx->err : g_init_error; }

int sched_sync_status(sched_ctx *ctx) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_sync_status: ctx is NULL");
  int status = 0;
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(&status, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  if (status != SCHED_OK) {
    set_error(ctx, "a kernel recorded device status %d", status);
    cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream);   // reported once; the context stays usable
  }
  return status;
}

int64_t sched_launch_count(const sched_ctx *ctx) { return ctx ? ctx->launches : 0; }

int sched_set_kernel_timing(sched_ctx *ctx, int enable) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_set_kernel_timing: ctx is NULL");
  ctx->timing_on = enable != 0;
  return SCHED_OK;
}

int sched_set_graphs(sched_ctx *ctx, int enable) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_set_graphs: ctx is NULL");
  ctx->graphs_enabled = enable != 0;
  return SCHED_OK;
}

int sched_set_store_budget(sched_ctx *ctx, uint64_t bytes) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_set_store_budget: ctx is NULL");
  REQUIRE(ctx, !ctx->round_ready, SCHED_ERR_INVALID_ARG,
          "sched_set_store_budget: the round scratch exists already (call before the first schedule_round)");
  ctx->rs_budget = bytes;
  return SCHED_OK;
}

int64_t sched_store_moves(sched_ctx *ctx) {
  if (!ctx || !ctx->rs_ready) return 0;
  unsigned int moves = 0;
  if (cudaMemcpyAsync(&moves, ctx->rs_state + 4, sizeof(moves), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess ||
      cudaStreamSynchronize(ctx->stream) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return (int64_t)moves;
}

int sched_set_racks(sched_ctx *ctx, const int16_t *h_node_rack, const float *d_alpha_rack, const float *d_beta_rack) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_set_racks: ctx is NULL");
  REQUIRE(ctx, !ctx->round_ready, SCHED_ERR_INVALID_ARG,
          "sched_set_racks: the round scratch exists already (call before the first schedule_round)");
  if (!h_node_rack) {
    if (ctx->d_rack) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_rack));
    }
    ctx->d_rack = nullptr;
    ctx->d_alpha_rack = ctx->d_beta_rack = nullptr;
    return SCHED_OK;
  }
  for (int n = 0; n < ctx->cfg.num_nodes; ++n)
    REQUIRE(ctx, h_node_rack[n] >= 0, SCHED_ERR_INVALID_ARG, "sched_set_racks: node %d has a negative rack", n);
  if (!ctx->d_rack) {
    int rc = dev_alloc(ctx, &ctx->d_rack, (size_t)ctx->cfg.num_nodes);
    if (rc != SCHED_OK) return rc;
  }
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(ctx->d_rack, h_node_rack, sizeof(int16_t) * ctx->cfg.num_nodes,
                                        cudaMemcpyHostToDevice, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));   // the host array may go away
  ctx->d_alpha_rack = d_alpha_rack;
  ctx->d_beta_rack = d_beta_rack;
  return SCHED_OK;
}

int build_speedup_table_rack(sched_ctx *ctx, const sched_jobs *d_jobs, const float *d_alpha_rack,
                             const float *d_beta_rack, float *d_goodput, float *d_speedup, uint16_t *d_argmax) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "build_speedup_table_rack: ctx is NULL");
  int rc = check_table_jobs(ctx, d_jobs);
  if (rc != SCHED_OK) return rc;
  REQUIRE(ctx, d_alpha_rack && d_beta_rack && d_speedup, SCHED_ERR_INVALID_ARG,
          "build_speedup_table_rack: d_alpha_rack, d_beta_rack and d_speedup must be non-NULL");
  return launch_speedup_table_rack(ctx, d_jobs, d_alpha_rack, d_beta_rack, d_goodput, d_speedup, d_argmax);
}

int eval_fitness_racks(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                       const float *d_speedup_rack, const int16_t *d_cur, const float *d_realloc_factor,
                       const uint8_t *d_active, float p, float *d_fitness) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "eval_fitness_racks: ctx is NULL");
  REQUIRE(ctx, ctx->d_rack, SCHED_ERR_INVALID_ARG, "eval_fitness_racks: no racks set (sched_set_racks)");
  REQUIRE(ctx, count >= 0, SCHED_ERR_INVALID_ARG, "eval_fitness_racks: count is negative");
  REQUIRE(ctx, count == 0 || (d_fitness && (ctx->cfg.num_jobs == 0 || (d_pop && d_speedup && d_speedup_rack))),
          SCHED_ERR_INVALID_ARG, "eval_fitness_racks: d_pop, d_speedup, d_speedup_rack and d_fitness must be non-NULL");
  REQUIRE(ctx, p == p, SCHED_ERR_INVALID_ARG, "eval_fitness_racks: p is NaN");
  REQUIRE(ctx, ((uintptr_t)d_pop & 1) == 0 && ((uintptr_t)d_cur & 1) == 0 && ((uintptr_t)d_speedup & 3) == 0 &&
                   ((uintptr_t)d_speedup_rack & 3) == 0 && ((uintptr_t)d_fitness & 3) == 0,
          SCHED_ERR_INVALID_ARG, "eval_fitness_racks: a buffer is not aligned to its element size");
  REQUIRE(ctx, (long long)count * ctx->cfg.num_jobs < (1LL << 31), SCHED_ERR_TOO_LARGE,
          "eval_fitness_racks: count * num_jobs must be below 2^31");
  return launch_fitness_racks(ctx, d_pop, count, d_speedup, d_speedup_rack, d_cur, d_realloc_factor, d_active, p,
                              d_fitness);
}

int sched_num_kernel_kinds(void) { return KK_COUNT; }

const char *sched_kernel_kind_name(int kind) {
  static const char *names[KK_COUNT] = {"goodput_sweep", "speedup_expand", "realloc_factor",
                                        "penalty_prep", "fitness", "rank", "rows", "cols",
                                        "best_index", "copy_best", "colscan", "fit_theta",
                                        "generation_store", "store_build", "store_compact", "store_gather"};
  return (kind >= 0 && kind < KK_COUNT) ? names[kind] : "";
}

int sched_read_kernel_timing(sched_ctx *ctx, float *h_ms_total, int64_t *h_launches) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_read_kernel_timing: ctx is NULL");
  REQUIRE(ctx, h_ms_total && h_launches, SCHED_ERR_INVALID_ARG, "sched_read_kernel_timing: NULL output");
  SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  for (int k = 0; k < KK_COUNT; ++k) { h_ms_total[k] = 0.f; h_launches[k] = 0; }
  for (TimedSpan &t : ctx->spans) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, t.start, t.stop) == cudaSuccess) {
      h_ms_total[t.kind] += ms;
      h_launches[t.kind] += 1;
    }
    ctx->free_spans.push_back(t);
  }
  ctx->spans.clear();
  return SCHED_OK;
}

int build_speedup_table(sched_ctx *ctx, const sched_jobs *d_jobs, float *d_goodput,
                        float *d_speedup, uint16_t *d_argmax) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "build_speedup_table: ctx is NULL");
  int rc = check_table_jobs(ctx, d_jobs);
  if (rc != SCHED_OK) return rc;
  REQUIRE(ctx, d_speedup, SCHED_ERR_INVALID_ARG, "build_speedup_table: d_speedup is NULL");
  return launch_speedup_table(ctx, d_jobs, d_goodput, d_speedup, d_argmax);
}

int build_speedup_table_msample(sched_ctx *ctx, const sched_jobs *d_jobs, const int32_t *d_m_samples,
                                int32_t num_samples, const int32_t *d_m_max_gpu, const uint8_t *d_adaptive,
                                float *d_goodput, float *d_speedup, uint16_t *d_argmax) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "build_speedup_table_msample: ctx is NULL");
  REQUIRE(ctx, d_jobs && d_jobs->alpha_grad && d_jobs->beta_grad && d_jobs->alpha_local && d_jobs->beta_local &&
                   d_jobs->alpha_node && d_jobs->beta_node && d_jobs->gamma && d_jobs->phi && d_jobs->m0 &&
                   d_jobs->m_max_total && d_jobs->fair_k && d_jobs->fair_n,
          SCHED_ERR_INVALID_ARG, "build_speedup_table_msample: a goodput-model array, fair_k or fair_n is NULL");
  REQUIRE(ctx, d_m_samples && d_m_max_gpu && d_speedup, SCHED_ERR_INVALID_ARG,
          "build_speedup_table_msample: d_m_samples, d_m_max_gpu and d_speedup must be non-NULL");
  REQUIRE(ctx, num_samples >= 1 && num_samples <= 65535, SCHED_ERR_INVALID_ARG,
          "build_speedup_table_msample: num_samples must be in [1, 65535]");
  return launch_speedup_table_msample(ctx, d_jobs, d_m_samples, num_samples, d_m_max_gpu, d_adaptive, d_goodput,
                                      d_speedup, d_argmax);
}

int fit_throughput_model(sched_ctx *ctx, int32_t num_jobs, const int32_t *d_obs_offset, const int32_t *d_obs_k,
                         const int32_t *d_obs_n, const int32_t *d_obs_m, const int32_t *d_obs_s,
                         const float *d_obs_t, const float *d_theta0, const uint8_t *d_frozen, int32_t max_iters,
                         float *d_theta_out, float *d_loss_out) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "fit_throughput_model: ctx is NULL");
  REQUIRE(ctx, num_jobs >= 0 && max_iters >= 0, SCHED_ERR_INVALID_ARG,
          "fit_throughput_model: num_jobs and max_iters must be >= 0");
  REQUIRE(ctx, num_jobs == 0 || (d_obs_offset && d_obs_k && d_obs_n && d_obs_m && d_obs_s && d_obs_t && d_theta0 &&
                                 d_theta_out && d_loss_out),
          SCHED_ERR_INVALID_ARG, "fit_throughput_model: an observation array, d_theta0 or an output is NULL");
  return launch_fit(ctx, num_jobs, d_obs_offset, d_obs_k, d_obs_n, d_obs_m, d_obs_s, d_obs_t, d_theta0, d_frozen,
                    max_iters, d_theta_out, d_loss_out);
}

int compute_realloc_factor(sched_ctx *ctx, const sched_jobs *d_jobs, float *d_out) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "compute_realloc_factor: ctx is NULL");
  REQUIRE(ctx, d_jobs && d_jobs->age_sec && d_jobs->num_restarts && d_out, SCHED_ERR_INVALID_ARG,
          "compute_realloc_factor: jobs.age_sec, jobs.num_restarts and d_out must be non-NULL");
  return launch_realloc_factor(ctx, d_jobs, d_out);
}

int autoscale_targets(sched_ctx *ctx, const float *d_goodput, const int32_t *d_cur_nodes, int32_t gpus_per_node,
                      float U, float L, int32_t *d_target_nodes) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "autoscale_targets: ctx is NULL");
  REQUIRE(ctx, d_goodput && d_cur_nodes && d_target_nodes, SCHED_ERR_INVALID_ARG,
          "autoscale_targets: d_goodput, d_cur_nodes and d_target_nodes must be non-NULL");
  REQUIRE(ctx, gpus_per_node >= 1 && U == U && L == L, SCHED_ERR_INVALID_ARG,
          "autoscale_targets: gpus_per_node must be >= 1, U and L not NaN");
  return launch_autoscale(ctx, d_goodput, d_cur_nodes, gpus_per_node, U, L, d_target_nodes);
}

int eval_fitness(sched_ctx *ctx, const int16_t *d_pop, int32_t count, const float *d_speedup,
                 const int16_t *d_cur, const float *d_realloc_factor, const uint8_t *d_active,
                 float p, float *d_fitness) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "eval_fitness: ctx is NULL");
  REQUIRE(ctx, count >= 0, SCHED_ERR_INVALID_ARG, "eval_fitness: count is negative");
  REQUIRE(ctx, count == 0 || (d_fitness && (ctx->cfg.num_jobs == 0 || (d_pop && d_speedup))), SCHED_ERR_INVALID_ARG,
          "eval_fitness: d_pop, d_speedup and d_fitness must be non-NULL");
  REQUIRE(ctx, p == p, SCHED_ERR_INVALID_ARG, "eval_fitness: p is NaN");
  REQUIRE(ctx, ((uintptr_t)d_pop & 1) == 0 && ((uintptr_t)d_cur & 1) == 0 &&
                   ((uintptr_t)d_speedup & 3) == 0 && ((uintptr_t)d_fitness & 3) == 0,
          SCHED_ERR_INVALID_ARG, "eval_fitness: a buffer is not aligned to its element size");
  REQUIRE(ctx, (long long)count * ctx->cfg.num_jobs < (1LL << 31), SCHED_ERR_TOO_LARGE,
          "eval_fitness: count * num_jobs must be below 2^31");
  return launch_fitness(ctx, d_pop, count, d_speedup, d_cur, d_realloc_factor, d_active, p, d_fitness);
}

int repair_population(sched_ctx *ctx, const sched_jobs *d_jobs, int16_t *d_pop, int32_t count,
                      uint32_t first_candidate, uint32_t round, uint32_t generation) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "repair_population: ctx is NULL");
  REQUIRE(ctx, count >= 0 && (count == 0 || d_pop || ctx->cfg.num_jobs == 0), SCHED_ERR_INVALID_ARG,
          "repair_population: d_pop is NULL or count negative");
  REQUIRE(ctx, ((uintptr_t)d_pop & 1) == 0, SCHED_ERR_INVALID_ARG, "repair_population: d_pop misaligned");
  REQUIRE(ctx, (long long)count * ctx->cfg.num_jobs < (1LL << 31), SCHED_ERR_TOO_LARGE,
          "repair_population: count * num_jobs must be below 2^31");
  if (ctx->cfg.num_jobs == 0) return SCHED_OK;
  int rc = launch_set_round(ctx, round);
  if (rc != SCHED_OK) return rc;
  return launch_repair(ctx, d_jobs ? d_jobs->k_cap : nullptr, d_jobs ? d_jobs->active : nullptr, d_pop,
                       count, first_candidate, generation);
}

int init_population(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_cur, uint32_t round,
                    int16_t *d_pop_out) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "init_population: ctx is NULL");
  REQUIRE(ctx, d_pop_out, SCHED_ERR_INVALID_ARG, "init_population: d_pop_out is NULL");
  REQUIRE(ctx, ((uintptr_t)d_pop_out & 1) == 0 && ((uintptr_t)d_cur & 1) == 0, SCHED_ERR_INVALID_ARG,
          "init_population: a buffer is misaligned");
  if (ctx->cfg.num_jobs == 0) return SCHED_OK;
  int rc = launch_set_round(ctx, round);
  if (rc != SCHED_OK) return rc;
  return launch_init_population(ctx, d_jobs ? d_jobs->k_cap : nullptr,
                                d_jobs ? d_jobs->active : nullptr, d_cur, d_pop_out);
}

int ga_generation(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_pop_in,
                  const float *d_fitness_in, int16_t *d_pop_out, uint32_t round, uint32_t generation) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "ga_generation: ctx is NULL");
  REQUIRE(ctx, d_pop_in && d_fitness_in && d_pop_out, SCHED_ERR_INVALID_ARG,
          "ga_generation: d_pop_in, d_fitness_in and d_pop_out must be non-NULL");
  REQUIRE(ctx, d_pop_in != d_pop_out, SCHED_ERR_INVALID_ARG, "ga_generation: in and out must not overlap");
  REQUIRE(ctx, (((uintptr_t)d_pop_in | (uintptr_t)d_pop_out) & 1) == 0 && ((uintptr_t)d_fitness_in & 3) == 0,
          SCHED_ERR_INVALID_ARG, "ga_generation: a buffer is misaligned");
  if (ctx->cfg.num_jobs == 0) return SCHED_OK;
  int rc = launch_set_round(ctx, round);
  if (rc != SCHED_OK) return rc;
  return launch_generation(ctx, d_jobs ? d_jobs->k_cap : nullptr, d_jobs ? d_jobs->active : nullptr,
                           d_pop_in, d_fitness_in, d_pop_out, generation);
}

int ga_generation_shard(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_pop_in, const float *d_fitness_in,
                        int32_t first_child, int32_t num_children, int16_t *d_children, uint32_t round,
                        uint32_t generation) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "ga_generation_shard: ctx is NULL");
  REQUIRE(ctx, d_pop_in && d_fitness_in, SCHED_ERR_INVALID_ARG,
          "ga_generation_shard: d_pop_in and d_fitness_in must be non-NULL");
  REQUIRE(ctx, first_child >= 0 && num_children >= 0 && (long long)first_child + num_children <= ctx->cfg.population,
          SCHED_ERR_INVALID_ARG, "ga_generation_shard: children %d .. %d are not within the population of %d",
          first_child, first_child + num_children, ctx->cfg.population);
  if (num_children == 0 || ctx->cfg.num_jobs == 0) return SCHED_OK;
  REQUIRE(ctx, d_children, SCHED_ERR_INVALID_ARG, "ga_generation_shard: d_children is NULL");
  const size_t mat = (size_t)ctx->cfg.num_jobs * ctx->cfg.num_nodes;
  REQUIRE(ctx, d_children + mat * num_children <= d_pop_in || d_pop_in + mat * ctx->cfg.population <= d_children,
          SCHED_ERR_INVALID_ARG, "ga_generation_shard: parents and children must not overlap");
  REQUIRE(ctx, (((uintptr_t)d_pop_in | (uintptr_t)d_children) & 1) == 0 && ((uintptr_t)d_fitness_in & 3) == 0,
          SCHED_ERR_INVALID_ARG, "ga_generation_shard: a buffer is misaligned");
  int rc = launch_set_round(ctx, round);
  if (rc != SCHED_OK) return rc;
  return launch_generation(ctx, d_jobs ? d_jobs->k_cap : nullptr, d_jobs ? d_jobs->active : nullptr, d_pop_in,
                           d_fitness_in, d_children, generation, first_child, num_children);
}

// Everything a round enqueues on the stream (the round number is already in d_round).
static int round_body(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_cur, int32_t generations,
                      int16_t *d_best, float *d_best_fitness) {
  int rc;
  const bool penalise = d_cur && d_jobs->age_sec && d_jobs->num_restarts;
  if ((rc = launch_speedup_table(ctx, d_jobs, ctx->d_tab_goodput, ctx->d_tab_speedup, nullptr)) != SCHED_OK) return rc;
  // Rack-level locality: a second table for allocations that span racks; the round then runs on
  // dense matrices with the fitness read from them (the row summaries carry no rack count).
  const bool racks = ctx->d_rack != nullptr;
  if (racks) {
    const float *ar = ctx->d_alpha_rack ? ctx->d_alpha_rack : d_jobs->alpha_node;
    const float *br = ctx->d_beta_rack ? ctx->d_beta_rack : d_jobs->beta_node;
    if ((rc = launch_speedup_table_rack(ctx, d_jobs, ar, br, nullptr, ctx->d_tab_speedup_rack, nullptr)) != SCHED_OK)
      return rc;
  }
  if (penalise && (rc = launch_realloc_factor(ctx, d_jobs, ctx->d_rf)) != SCHED_OK) return rc;
  const float *rf = penalise ? ctx->d_rf : nullptr;
  int16_t *pa = ctx->d_popA, *pb = ctx->d_popB;
  // While the round runs, the row/column kernels also keep per-row summaries (K, N, differs
  // from the current allocation); the in-round fitness reads those instead of the matrices
  // whenever the batched kernels were used, with bit-identical results.
  ctx->round_cur = rf ? d_cur : nullptr;
  ctx->round_summ = racks ? nullptr : ctx->d_summ;
  ctx->round_summ_in = nullptr;
  uint32_t *summ_other = ctx->d_summ + (size_t)ctx->cfg.population * ctx->cfg.num_jobs;
  // the per-job penalty factors depend only on the current allocation: prepared once
  ctx->pen_ready = false;
  rc = SCHED_OK;
  if (rf) rc = launch_penalty_prep(ctx, d_cur, rf);
  ctx->pen_ready = (rc == SCHED_OK) && rf;
  // problems whose candidates fit one block get row pass, column pass and fitness in one kernel
  ctx->ff_on = !racks;
  ctx->ff_table = ctx->d_tab_speedup;
  ctx->ff_pen = rf ? ctx->d_pen : nullptr;
  ctx->ff_active = d_jobs->active;
  ctx->ff_p = ctx->cfg.p;
  // parents' fitness is read while children's is written: the two alternate between buffers
  float *fit_cur = ctx->d_fit_buf, *fit_next = ctx->d_fit_buf + ctx->cfg.population;
  ctx->ff_out = fit_cur;
  auto fitness_of = [&](const int16_t *pop, float *out) {
    if (ctx->fit_done) return (int)SCHED_OK;
    if (racks)
      return launch_fitness_racks(ctx, pop, ctx->cfg.population, ctx->d_tab_speedup, ctx->d_tab_speedup_rack, d_cur, rf,
                                  d_jobs->active, ctx->cfg.p, out);
    return launch_fitness(ctx, pop, ctx->cfg.population, ctx->d_tab_speedup, d_cur, rf, d_jobs->active,
                          ctx->cfg.p, out, ctx->summ_valid ? ctx->round_summ : nullptr);
  };
  const bool store = ctx->rs_ready && generations > 0;
  int parity = 0;
  if (store) {
    // The round runs on the row store: candidates are arrays of row indices.  The current
    // allocation's rows go in first; the initial population is then made like any generation (its
    // single parent is the current allocation), by the kernel that also does the operators, the
    // repair and the fitness; every few generations a check moves the live rows to the other half
    // of the pool if the half in use could run out.
    pa = ctx->rs_pool;
    if (rc == SCHED_OK) rc = rowstore_build_current(ctx, d_jobs->k_cap, d_jobs->active, d_cur, ctx->round_cur,
                                                    rf ? ctx->d_pen : nullptr);
    int phase = 0;
    if (rc == SCHED_OK)
      rc = rowstore_generation(ctx, d_jobs->k_cap, d_jobs->active, ctx->round_cur, rf ? ctx->d_pen : nullptr, fit_next,
                               fit_cur, 0, phase, GEN_INIT);
    parity = 1;
    for (int g = 0; g < generations && rc == SCHED_OK; ++g) {
      if (g > 0 && g % ctx->rs_check_every == 0) {
        rc = rowstore_compact(ctx, parity, phase);
        phase ^= 1;
        if (rc != SCHED_OK) break;
      }
      rc = rowstore_generation(ctx, d_jobs->k_cap, d_jobs->active, ctx->round_cur, rf ? ctx->d_pen : nullptr,
                               fit_cur, fit_next, parity, phase, (uint32_t)g);
      parity ^= 1;
      std::swap(fit_cur, fit_next);
    }
  } else {
    if (ctx->rs_ready) pa = ctx->rs_pool;   // no generations: the dense initial population sits at the start of the pool
    if (rc == SCHED_OK) rc = launch_init_population(ctx, d_jobs->k_cap, d_jobs->active, d_cur, pa);
    if (rc == SCHED_OK) rc = fitness_of(pa, fit_cur);
  }
  for (int g = 0; g < generations && rc == SCHED_OK && !store; ++g) {
    ctx->ff_out = fit_next;
    // children's summaries go to the other half; the parents' feed the unperturbed rows
    ctx->round_summ_in = ctx->summ_valid ? ctx->round_summ : nullptr;
    if (!racks) std::swap(ctx->round_summ, summ_other);
    rc = launch_generation(ctx, d_jobs->k_cap, d_jobs->active, pa, fit_cur, pb, (uint32_t)g);
    if (rc != SCHED_OK) break;
    std::swap(pa, pb);
    rc = fitness_of(pa, fit_next);
    std::swap(fit_cur, fit_next);
  }
  ctx->d_fit = fit_cur;
  ctx->pen_ready = false;
  ctx->ff_on = false;
  ctx->fit_done = false;
  ctx->round_cur = nullptr;
  ctx->round_summ = nullptr;
  ctx->round_summ_in = nullptr;
  ctx->summ_valid = false;
  if (rc != SCHED_OK) return rc;
  ctx->d_pop_last = pa;
  ctx->rs_ptr_last = nullptr;
  if (store) {
    ctx->rs_ptr_last = ctx->rs_ptr + (size_t)parity * ctx->cfg.population * ctx->cfg.num_jobs;
    if ((rc = launch_select_best(ctx, nullptr, ctx->d_fit, nullptr, d_best_fitness)) != SCHED_OK) return rc;
    return rowstore_gather(ctx, ctx->rs_ptr_last, 0, 1, ctx->d_best_idx, d_best);
  }
  return launch_select_best(ctx, pa, ctx->d_fit, d_best, d_best_fitness);
}


// A round is a fixed sequence of kernels whose arguments do not change from round to round
// when the caller reuses its buffers (the round number lives in device memory).  The second
// time a round is requested with the same pointers and generation count it is captured
// into a CUDA graph; later rounds replay the graph, which removes the per-kernel launch
// cost that dominates small problems.  Graphs are not used while per-kernel timing is on,
// on the legacy default stream, or after a capture failed.
static bool same_round_key(const RoundKey &a, const RoundKey &b) { return memcmp(&a, &b, sizeof(RoundKey)) == 0; }

int schedule_round(sched_ctx *ctx, const sched_jobs *d_jobs, const int16_t *d_cur, uint32_t round,
                   int32_t generations, int16_t *d_best, float *d_best_fitness) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "schedule_round: ctx is NULL");
  int rc = check_table_jobs(ctx, d_jobs);
  if (rc != SCHED_OK) return rc;
  REQUIRE(ctx, generations >= 0, SCHED_ERR_INVALID_ARG, "schedule_round: generations is negative");
  REQUIRE(ctx, d_best && d_best_fitness, SCHED_ERR_INVALID_ARG,
          "schedule_round: d_best and d_best_fitness must be non-NULL");
  REQUIRE(ctx, ctx->cfg.num_jobs >= 1, SCHED_ERR_BAD_CONFIG, "schedule_round: needs at least one job");
  if ((rc = ensure_round_scratch(ctx)) != SCHED_OK) return rc;
  if ((rc = launch_set_round(ctx, round)) != SCHED_OK) return rc;

  RoundKey key;
  memset(&key, 0, sizeof(key));
  key.jobs = *d_jobs;
  key.cur = d_cur; key.best = d_best; key.best_fitness = d_best_fitness; key.generations = generations;
  const bool graphs_ok = ctx->graphs_enabled && !ctx->timing_on && ctx->stream != nullptr;
  if (ctx->graph_exec && ctx->graph_epoch != ctx->scratch_epoch) {   // scratch moved: pointers in the graph are stale
    cudaGraphExecDestroy(ctx->graph_exec);
    ctx->graph_exec = nullptr;
  }
  if (graphs_ok && ctx->graph_exec && same_round_key(key, ctx->graph_key)) {
    SCHED_CUDA_CHECK(ctx, cudaGraphLaunch(ctx->graph_exec, ctx->stream));
    ctx->launches += ctx->graph_launches;
    ctx->d_fit = ctx->graph_fit;
    ctx->d_pop_last = ctx->graph_pop_last;
    ctx->rs_ptr_last = ctx->graph_ptr_last;
    return SCHED_OK;
  }
  const bool capture = graphs_ok && ctx->seen_valid && same_round_key(key, ctx->seen_key);
  memcpy(&ctx->seen_key, &key, sizeof(key));
  ctx->seen_valid = true;
  if (!capture) return round_body(ctx, d_jobs, d_cur, generations, d_best, d_best_fitness);

  // second request with the same arguments: all scratch exists already, so the body makes no
  // allocation and can be captured
  if (ctx->graph_exec) { cudaGraphExecDestroy(ctx->graph_exec); ctx->graph_exec = nullptr; }
  const int64_t launches_before = ctx->launches;
  const uint64_t epoch_before = ctx->scratch_epoch;
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    ctx->graphs_enabled = false;
    return round_body(ctx, d_jobs, d_cur, generations, d_best, d_best_fitness);
  }
  rc = round_body(ctx, d_jobs, d_cur, generations, d_best, d_best_fitness);
  const cudaError_t ce = cudaStreamEndCapture(ctx->stream, &graph);
  const int64_t captured = ctx->launches - launches_before;
  ctx->launches = launches_before;
  if (rc != SCHED_OK || ce != cudaSuccess || !graph || ctx->scratch_epoch != epoch_before ||
      cudaGraphInstantiate(&ctx->graph_exec, graph, 0) != cudaSuccess) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    ctx->graph_exec = nullptr;
    ctx->graphs_enabled = false;   // run plainly from now on
    return round_body(ctx, d_jobs, d_cur, generations, d_best, d_best_fitness);
  }
  cudaGraphDestroy(graph);
  memcpy(&ctx->graph_key, &key, sizeof(key));
  ctx->graph_epoch = ctx->scratch_epoch;
  ctx->graph_launches = captured;
  ctx->graph_fit = ctx->d_fit;
  ctx->graph_pop_last = ctx->d_pop_last;
  ctx->graph_ptr_last = ctx->rs_ptr_last;
  SCHED_CUDA_CHECK(ctx, cudaGraphLaunch(ctx->graph_exec, ctx->stream));
  ctx->launches += captured;
  return SCHED_OK;
}

int sched_get_population(sched_ctx *ctx, int16_t *d_pop_out, float *d_fitness_out) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_get_population: ctx is NULL");
  REQUIRE(ctx, ctx->d_pop_last, SCHED_ERR_INVALID_ARG, "sched_get_population: no round has run yet");
  const sched_config &c = ctx->cfg;
  if (d_pop_out && ctx->rs_ptr_last) {
    int rc = rowstore_gather(ctx, ctx->rs_ptr_last, 0, c.population, nullptr, d_pop_out);
    if (rc != SCHED_OK) return rc;
  } else if (d_pop_out)
    SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_pop_out, ctx->d_pop_last,
                                          sizeof(int16_t) * (size_t)c.population * c.num_jobs * c.num_nodes,
                                          cudaMemcpyDeviceToDevice, ctx->stream));
  if (d_fitness_out)
    SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_fitness_out, ctx->d_fit, sizeof(float) * c.population,
                                          cudaMemcpyDeviceToDevice, ctx->stream));
  return SCHED_OK;
}

int sched_get_round_tables(sched_ctx *ctx, float *d_goodput_out, float *d_speedup_out) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "sched_get_round_tables: ctx is NULL");
  REQUIRE(ctx, ctx->round_ready && ctx->d_pop_last, SCHED_ERR_INVALID_ARG, "sched_get_round_tables: no round has run yet");
  const size_t bytes = sizeof(float) * (size_t)ctx->cfg.num_jobs * ctx->KD * ctx->ND;
  if (d_goodput_out)
    SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_goodput_out, ctx->d_tab_goodput, bytes, cudaMemcpyDeviceToDevice, ctx->stream));
  if (d_speedup_out)
    SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_speedup_out, ctx->d_tab_speedup, bytes, cudaMemcpyDeviceToDevice, ctx->stream));
  return SCHED_OK;
}

const float *sched_round_speedup_table(const sched_ctx *ctx) {
  return (ctx && ctx->round_ready) ? ctx->d_tab_speedup : nullptr;
}

// ---- host-buffer entry points ------------------------------------------------------------

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Host-side checks of arrays that arrive in host memory.  first_bad: index of the first entry
// that is NaN / infinite (kind 1) or below `lo` / above `hi` (kind 2), or -1.
static long long first_bad(const float *a, size_t n, float lo, float hi, int &kind) {
  for (size_t i = 0; i < n; ++i) {
    const float v = a[i];
    if (!(v - v == 0.f)) { kind = 1; return (long long)i; }       // NaN or +-inf
    if (v < lo || v > hi) { kind = 2; return (long long)i; }
  }
  return -1;
}

#define CHECK_HOST_F32(ctx, who, name, ptr, n, lo, hi)                                              \
  do {                                                                                              \
    int kind__ = 0;                                                                                 \
    const long long at__ = (ptr) ? first_bad((ptr), (n), (lo), (hi), kind__) : -1;                  \
    if (at__ >= 0) {                                                                                \
      set_error(ctx, "%s: %s[%lld] = %g is %s", who, name, at__, (double)(ptr)[at__],               \
                kind__ == 1 ? "not finite" : "outside its range");                                  \
      return kind__ == 1 ? SCHED_ERR_NOT_FINITE : SCHED_ERR_INVALID_ARG;                            \
    }                                                                                               \
  } while (0)

static int validate_host_jobs(sched_ctx *ctx, const sched_jobs *h, const int16_t *h_cur) {
  const sched_config &c = ctx->cfg;
  const size_t J = (size_t)c.num_jobs;
  const float big = 3.0e38f;
  const char *who = "schedule_round_host";
  CHECK_HOST_F32(ctx, who, "alpha_grad", h->alpha_grad, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "beta_grad", h->beta_grad, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "alpha_local", h->alpha_local, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "beta_local", h->beta_local, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "alpha_node", h->alpha_node, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "beta_node", h->beta_node, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "gamma", h->gamma, J, 1.f, big);
  CHECK_HOST_F32(ctx, who, "phi", h->phi, J, 0.f, big);
  CHECK_HOST_F32(ctx, who, "m0", h->m0, J, 1.f, big);
  CHECK_HOST_F32(ctx, who, "m_max_total", h->m_max_total, J, 1.f, big);
  CHECK_HOST_F32(ctx, who, "age_sec", h->age_sec, J, 0.f, big);
  for (size_t j = 0; j < J; ++j) {
    REQUIRE(ctx, h->m_max_total[j] >= h->m0[j], SCHED_ERR_INVALID_ARG,
            "schedule_round_host: m_max_total[%zu] = %g is below m0 = %g", j, (double)h->m_max_total[j], (double)h->m0[j]);
    REQUIRE(ctx, !h->num_restarts || h->num_restarts[j] >= 0, SCHED_ERR_INVALID_ARG,
            "schedule_round_host: num_restarts[%zu] is negative", j);
  }
  for (size_t i = 0; i < J * (size_t)c.grid_m; ++i)
    REQUIRE(ctx, h->m_grid[i] >= 1, SCHED_ERR_INVALID_ARG, "schedule_round_host: m_grid[%zu] = %d is below 1", i,
            (int)h->m_grid[i]);
  if (h_cur)
    for (size_t i = 0; i < J * (size_t)c.num_nodes; ++i)
      REQUIRE(ctx, h_cur[i] >= 0, SCHED_ERR_INVALID_ARG, "schedule_round_host: h_cur[%zu] is negative", i);
  return SCHED_OK;
}

int schedule_round_host(sched_ctx *ctx, const sched_jobs *h_jobs, const int16_t *h_cur, uint32_t round,
                        int32_t generations, int16_t *h_best, float *h_best_fitness) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "schedule_round_host: ctx is NULL");
  int rc = check_table_jobs(ctx, h_jobs);
  if (rc != SCHED_OK) return rc;
  REQUIRE(ctx, h_best && h_best_fitness, SCHED_ERR_INVALID_ARG,
          "schedule_round_host: h_best and h_best_fitness must be non-NULL");
  if ((rc = validate_host_jobs(ctx, h_jobs, h_cur)) != SCHED_OK) return rc;
  const sched_config &c = ctx->cfg;
  const size_t J = (size_t)c.num_jobs, mat = J * c.num_nodes * sizeof(int16_t);
  // layout of the staging buffer: 10 fp32 arrays, m_grid, k_cap, fair_k, fair_n, age,
  // restarts, active, cur, best, best_fitness - each 256-byte aligned
  const size_t f32 = align256(J * 4), grid = align256(J * c.grid_m * 4), u8 = align256(J);
  const size_t need = 10 * f32 + grid + 5 * f32 + u8 + 2 * align256(mat) + 256;
  if (need > ctx->stage_bytes) {
    if (ctx->d_stage) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_stage));
      ctx->d_stage = nullptr;
      ctx->stage_bytes = 0;
    }
    SCHED_CUDA_CHECK(ctx, cudaMalloc(&ctx->d_stage, need));
    ctx->stage_bytes = need;
  }
  char *base = (char *)ctx->d_stage;
  size_t off = 0;
  // Small problems: the inputs are first gathered in a pinned buffer laid out like the device
  // one and go up in a single copy (launching 18 small copies costs more than the bytes do).
  const size_t input_bytes = need - 2 * align256(mat) - 256 + align256(mat);   // everything up to and including cur
  const bool gather = input_bytes <= (256u << 10);
  if (gather && input_bytes > ctx->h_stage_bytes) {
    if (ctx->h_stage) { cudaFreeHost(ctx->h_stage); ctx->h_stage = nullptr; ctx->h_stage_bytes = 0; }
    if (cudaMallocHost(&ctx->h_stage, input_bytes) == cudaSuccess) ctx->h_stage_bytes = input_bytes;
    else { cudaGetLastError(); ctx->h_stage = nullptr; }
  }
  char *hbase = (gather && ctx->h_stage) ? (char *)ctx->h_stage : nullptr;
  auto up = [&](const void *h, size_t bytes, size_t slot) -> const void * {
    void *d = base + off;
    char *hs = hbase ? hbase + off : nullptr;
    off += slot;
    if (!h) return nullptr;
    if (hs) { memcpy(hs, h, bytes); return d; }
    if (cudaMemcpyAsync(d, h, bytes, cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess) return (const void *)-1;
    return d;
  };
  sched_jobs dj;
  const float *const hf[10] = {h_jobs->alpha_grad, h_jobs->beta_grad, h_jobs->alpha_local, h_jobs->beta_local,
                               h_jobs->alpha_node, h_jobs->beta_node, h_jobs->gamma, h_jobs->phi,
                               h_jobs->m0, h_jobs->m_max_total};
  const float **df[10] = {&dj.alpha_grad, &dj.beta_grad, &dj.alpha_local, &dj.beta_local, &dj.alpha_node,
                          &dj.beta_node, &dj.gamma, &dj.phi, &dj.m0, &dj.m_max_total};
  bool bad = false;
  for (int i = 0; i < 10; ++i) {
    *df[i] = (const float *)up(hf[i], J * 4, f32);
    bad |= (*df[i] == (const float *)-1);
  }
  dj.m_grid = (const int32_t *)up(h_jobs->m_grid, J * c.grid_m * 4, grid);
  dj.k_cap = (const int32_t *)up(h_jobs->k_cap, J * 4, f32);
  dj.fair_k = (const int32_t *)up(h_jobs->fair_k, J * 4, f32);
  dj.fair_n = (const int32_t *)up(h_jobs->fair_n, J * 4, f32);
  dj.age_sec = (const float *)up(h_jobs->age_sec, J * 4, f32);
  dj.num_restarts = (const int32_t *)up(h_jobs->num_restarts, J * 4, f32);
  dj.active = (const uint8_t *)up(h_jobs->active, J, u8);
  const int16_t *d_cur = (const int16_t *)up(h_cur, mat, align256(mat));
  bad |= dj.m_grid == (const void *)-1 || dj.k_cap == (const void *)-1 || dj.fair_k == (const void *)-1 ||
         dj.fair_n == (const void *)-1 || dj.age_sec == (const void *)-1 ||
         dj.num_restarts == (const void *)-1 || dj.active == (const void *)-1 || d_cur == (const void *)-1;
  if (hbase && cudaMemcpyAsync(base, hbase, off, cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess) bad = true;
  REQUIRE(ctx, !bad, SCHED_ERR_CUDA, "schedule_round_host: a host-to-device copy failed: %s",
          cudaGetErrorString(cudaGetLastError()));
  int16_t *d_best = (int16_t *)(base + off);
  off += align256(mat);
  float *d_bf = (float *)(base + off);
  rc = schedule_round(ctx, &dj, d_cur, round, generations, d_best, d_bf);
  if (rc != SCHED_OK) return rc;
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(h_best, d_best, mat, cudaMemcpyDeviceToHost, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(h_best_fitness, d_bf, sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  int status = SCHED_OK;   // the call waits anyway: a device-side error of the round is its result
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(&status, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  if (status != SCHED_OK) {
    set_error(ctx, "schedule_round_host: a kernel recorded device status %d", status);
    cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream);
  }
  return status;
}

int eval_fitness_host(sched_ctx *ctx, const int16_t *h_pop, int32_t count, const float *h_speedup,
                      const int16_t *h_cur, const float *h_realloc_factor, const uint8_t *h_active,
                      float p, float *h_fitness) {
  REQUIRE(nullptr, ctx, SCHED_ERR_INVALID_ARG, "eval_fitness_host: ctx is NULL");
  REQUIRE(ctx, count >= 0 && (count == 0 || (h_pop && h_speedup && h_fitness)), SCHED_ERR_INVALID_ARG,
          "eval_fitness_host: h_pop, h_speedup and h_fitness must be non-NULL");
  if (count == 0) return SCHED_OK;
  const sched_config &c = ctx->cfg;
  const size_t J = (size_t)c.num_jobs, mat = J * c.num_nodes * sizeof(int16_t);
  CHECK_HOST_F32(ctx, "eval_fitness_host", "h_speedup", h_speedup, J * ctx->KD * ctx->ND, 0.f, 3.0e38f);
  CHECK_HOST_F32(ctx, "eval_fitness_host", "h_realloc_factor", h_realloc_factor, J, 0.f, 1.f);
  const size_t pop_b = align256(mat * count), tab_b = align256(J * ctx->KD * ctx->ND * 4);
  const size_t need = pop_b + tab_b + align256(mat) + align256(J * 4) + align256(J) + align256((size_t)count * 4);
  if (need > ctx->stage_fit_bytes) {
    if (ctx->d_stage_fit) {
      SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
      SCHED_CUDA_CHECK(ctx, cudaFree(ctx->d_stage_fit));
      ctx->d_stage_fit = nullptr;
      ctx->stage_fit_bytes = 0;
    }
    SCHED_CUDA_CHECK(ctx, cudaMalloc(&ctx->d_stage_fit, need));
    ctx->stage_fit_bytes = need;
  }
  char *base = (char *)ctx->d_stage_fit;
  int16_t *d_pop = (int16_t *)base;
  float *d_tab = (float *)(base + pop_b);
  int16_t *d_cur = (int16_t *)(base + pop_b + tab_b);
  float *d_rf = (float *)(base + pop_b + tab_b + align256(mat));
  uint8_t *d_act = (uint8_t *)(base + pop_b + tab_b + align256(mat) + align256(J * 4));
  float *d_fit = (float *)(base + pop_b + tab_b + align256(mat) + align256(J * 4) + align256(J));
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_pop, h_pop, mat * count, cudaMemcpyHostToDevice, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_tab, h_speedup, J * ctx->KD * ctx->ND * 4, cudaMemcpyHostToDevice, ctx->stream));
  if (h_cur) SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_cur, h_cur, mat, cudaMemcpyHostToDevice, ctx->stream));
  if (h_realloc_factor) SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_rf, h_realloc_factor, J * 4, cudaMemcpyHostToDevice, ctx->stream));
  if (h_active) SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(d_act, h_active, J, cudaMemcpyHostToDevice, ctx->stream));
  int rc = eval_fitness(ctx, d_pop, count, d_tab, h_cur ? d_cur : nullptr, h_realloc_factor ? d_rf : nullptr,
                        h_active ? d_act : nullptr, p, d_fit);
  if (rc != SCHED_OK) return rc;
  SCHED_CUDA_CHECK(ctx, cudaMemcpyAsync(h_fitness, d_fit, (size_t)count * 4, cudaMemcpyDeviceToHost, ctx->stream));
  SCHED_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  return SCHED_OK;
}

#pragma GCC visibility pop
}  // extern "C"
