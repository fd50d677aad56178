/*
 * CPU oracle for the PolluxSched optimizer core.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of what the scheduling hot path
 * computes, written from the paper's equations and, for the genetic operators the
 * paper describes in one sentence (Sec. 4.3), from the operator definitions this
 * project fixes in its design notes.  It shares no code with the CUDA library and is
 * only ever loaded by the tests, the smoke check and the benchmark's CPU-baseline leg.
 * Nothing in the product path may call it.
 *
 * Pins (see tests/test_oracle_*.py): hand-worked goodput values, closed forms of
 * Eq. 6/9/10/11/14/15, library power means, brute force on tiny clusters, an
 * independent library Philox, numpy sorting.  No function here is unpinned.
 *
 * All matrices are row-major.  An allocation matrix A is int16 [J][num_nodes]
 * (node index fastest); a population is [P][J][num_nodes].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)

#define SLOT_SELECT 0u
#define SLOT_XOVER 1u
#define SLOT_MUTATE 2u
#define SLOT_REPAIR_INTF 3u
#define SLOT_REPAIR_CAP 4u
#define SLOT_INIT 5u
#define GEN_INIT 0xFFFFFFFFu

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as    */
/* easy as 1, 2, 3", SC'11).  Ten rounds; the key is bumped before every      */
/* round but the first.                                                       */
/* ------------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        if (r > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The stream used by the operators: key = (seed_lo ^ seed_hi, round),
 * counter = (idx, candidate, generation, slot). */
static void draw(uint64_t seed, uint32_t round, uint32_t idx, uint32_t cand, uint32_t gen,
                 uint32_t slot, uint32_t w[4]) {
    uint32_t key[2] = {(uint32_t)seed ^ (uint32_t)(seed >> 32), round};
    uint32_t ctr[4] = {idx, cand, gen, slot};
    oracle_philox4x32_10(ctr, key, w);
}

void oracle_draw(uint64_t seed, uint32_t round, uint32_t idx, uint32_t cand, uint32_t gen,
                 uint32_t slot, uint32_t w[4]) {
    draw(seed, round, idx, cand, gen, slot, w);
}

/* floor(w * n / 2^32): a bounded integer in [0, n) without rejection. */
static uint32_t mulhi(uint32_t w, uint32_t n) { return (uint32_t)(((uint64_t)w * n) >> 32); }

/* ------------------------------------------------------------------------- */
/* Goodput model                                                              */
/* ------------------------------------------------------------------------- */

/* EFFICIENCY_t(M) = (phi + M0) / (phi + M)                       (Eq. 6) */
double oracle_efficiency(double phi, double m0, double M) { return (phi + m0) / (phi + M); }

/* T_grad(m) = alpha_grad + beta_grad * m                          (Eq. 8) */
double oracle_t_grad(double alpha_grad, double beta_grad, double m) { return alpha_grad + beta_grad * m; }

/* T_sync: 0 for one replica; the local pair when all replicas share a node; the
 * node pair otherwise; linear in K - 2                              (Eq. 9) */
double oracle_t_sync(double alpha_local, double beta_local, double alpha_node, double beta_node,
                     int K, int N) {
    if (K <= 1) return 0.0;
    if (N == 1) return alpha_local + beta_local * (double)(K - 2);
    return alpha_node + beta_node * (double)(K - 2);
}

/* T_iter(a, m, s) = s * T_grad + (T_grad^gamma + T_sync^gamma)^(1/gamma)   (Eq. 10, 11) */
double oracle_t_iter(double t_grad, double t_sync, double gamma, int s) {
    double overlap = (t_sync == 0.0) ? t_grad
                                     : pow(pow(t_grad, gamma) + pow(t_sync, gamma), 1.0 / gamma);
    return (double)s * t_grad + overlap;
}

/* GOODPUT = THROUGHPUT * EFFICIENCY with THROUGHPUT = M / T_iter and
 * M = K * m * (s + 1)  (Eq. 4, 7 and the batch-size definition of Sec. 3).  Returns 0
 * and clears *feasible when M falls outside [M0, M_max] (Sec. 3: only M >= M0 is
 * considered; Sec. 3.1: application-defined upper limit). */
double oracle_goodput(double alpha_grad, double beta_grad, double alpha_local, double beta_local,
                      double alpha_node, double beta_node, double gamma, double phi, double m0,
                      double m_max_total, int K, int N, int m, int s, int *feasible) {
    double M = (double)K * (double)m * (double)(s + 1);
    int ok = (K >= 1 && N >= 1 && N <= K && M >= m0 && M <= m_max_total);
    if (feasible) *feasible = ok;
    if (!ok) return 0.0;
    double tg = oracle_t_grad(alpha_grad, beta_grad, (double)m);
    double ts = oracle_t_sync(alpha_local, beta_local, alpha_node, beta_node, K, N);
    double ti = oracle_t_iter(tg, ts, gamma, s);
    return (M / ti) * oracle_efficiency(phi, m0, M);
}

static int cmp_desc_i16(const void *a, const void *b) {
    return (int)*(const int16_t *)b - (int)*(const int16_t *)a;
}

/* Largest replica count that N nodes can host: the sum of the N largest capacities. */
static void max_k_per_n(int num_nodes, const int16_t *cap, int n_max, int64_t *out /*[n_max+1]*/) {
    int16_t *sorted = (int16_t *)malloc(sizeof(int16_t) * (size_t)num_nodes);
    memcpy(sorted, cap, sizeof(int16_t) * (size_t)num_nodes);
    qsort(sorted, (size_t)num_nodes, sizeof(int16_t), cmp_desc_i16);
    out[0] = 0;
    for (int n = 1; n <= n_max; ++n)
        out[n] = out[n - 1] + (n <= num_nodes ? (sorted[n - 1] > 0 ? sorted[n - 1] : 0) : 0);
    free(sorted);
}

/* Fair share: an exclusive 1/J share of the cluster (Eq. 15), read as
 * K_f = clamp(floor(total GPUs / active jobs), 1, k_max) packed on as few nodes as
 * possible, N_f = ceil(K_f / largest node). */
int oracle_fair_share(int num_nodes, const int16_t *cap, int num_active, int k_max, int32_t *fair_k,
                      int32_t *fair_n) {
    if (num_nodes <= 0 || !cap) return ORACLE_ERR_ARG;
    int64_t total = 0;
    int big = 0;
    for (int n = 0; n < num_nodes; ++n) {
        if (cap[n] > 0) total += cap[n];
        if (cap[n] > big) big = cap[n];
    }
    if (big <= 0) return ORACLE_ERR_ARG;
    int64_t k = num_active > 0 ? total / num_active : total;
    if (k < 1) k = 1;
    if (k > k_max) k = k_max;
    *fair_k = (int32_t)k;
    *fair_n = (int32_t)((k + big - 1) / big);
    return ORACLE_OK;
}

/* Speedup table of one job set (Eq. 13: max over the (m, s) grid; Eq. 15: divided by the
 * fair-share goodput).  Entry (K, N) is populated when 1 <= N <= n_max, N <= K <= k_max
 * and K fits on the N largest nodes; every other entry is 0 with argmax 0xFFFF.  Ties
 * in the maximum go to the smaller s, then the smaller grid index.  argmax = i_m * Gs + s. */
int oracle_build_speedup_table(int J, int num_nodes, const int16_t *cap, int k_max, int n_max,
                               int grid_m, int grid_s, const float *alpha_grad,
                               const float *beta_grad, const float *alpha_local,
                               const float *beta_local, const float *alpha_node,
                               const float *beta_node, const float *gamma, const float *phi,
                               const float *m0, const float *m_max_total, const int32_t *m_grid,
                               const int32_t *fair_k, const int32_t *fair_n, double *goodput,
                               double *speedup, uint16_t *argmax) {
    if (J < 0 || k_max < 1 || n_max < 1 || grid_m < 1 || grid_s < 1) return ORACLE_ERR_ARG;
    const int KD = k_max + 1, ND = n_max + 1;
    int64_t *kfit = (int64_t *)malloc(sizeof(int64_t) * (size_t)ND);
    max_k_per_n(num_nodes, cap, n_max, kfit);
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < J; ++j) {
        double *gj = goodput + (size_t)j * KD * ND;
        double *sj = speedup + (size_t)j * KD * ND;
        uint16_t *aj = argmax ? argmax + (size_t)j * KD * ND : NULL;
        for (int K = 0; K < KD; ++K) {
            for (int N = 0; N < ND; ++N) {
                double best = 0.0;
                int best_s = -1, best_i = -1;
                int valid = (N >= 1 && K >= N && (int64_t)K <= kfit[N]);
                if (valid) {
                    for (int i = 0; i < grid_m; ++i) {
                        for (int s = 0; s < grid_s; ++s) {
                            int ok = 0;
                            double g = oracle_goodput(alpha_grad[j], beta_grad[j], alpha_local[j],
                                                      beta_local[j], alpha_node[j], beta_node[j],
                                                      gamma[j], phi[j], m0[j], m_max_total[j], K, N,
                                                      m_grid[(size_t)j * grid_m + i], s, &ok);
                            if (!ok) continue;
                            int better = (best_i < 0) || (g > best) ||
                                         (g == best && (s < best_s || (s == best_s && i < best_i)));
                            if (better) { best = g; best_s = s; best_i = i; }
                        }
                    }
                }
                gj[K * ND + N] = (best_i >= 0) ? best : 0.0;
                if (aj) aj[K * ND + N] = (best_i >= 0) ? (uint16_t)(best_i * grid_s + best_s) : 0xFFFFu;
            }
        }
        int kf = fair_k[j], nf = fair_n[j];
        double denom = (kf >= 0 && kf < KD && nf >= 0 && nf < ND) ? gj[kf * ND + nf] : 0.0;
        for (int e = 0; e < KD * ND; ++e) sj[e] = (denom > 0.0) ? gj[e] / denom : 0.0;
    }
    free(kfit);
    return ORACLE_OK;
}

/* The (m, s) sub-procedure as the paper words it (Sec. 4.3): sample candidate total batch
 * sizes M, for each take the smallest s such that the per-GPU batch fits the limit m_max,
 * and keep the configuration with the highest goodput.  Read here (the printed
 * "m = ceil(M / s)" cannot hold for s = 0) as: per_gpu = ceil(M / K);
 * s = ceil(per_gpu / m_max) - 1; m = ceil(per_gpu / (s + 1)); the batch actually run is
 * M' = K m (s + 1) >= M and must satisfy M0 <= M' <= M_max.  A non-adaptive job (Sec. 4.2,
 * "supporting non-adaptive jobs") has the single candidate M = M0 and EFFICIENCY fixed to 1.
 * Table layout, validity of (K, N), normalisation and ties (smallest sample index) as in
 * oracle_build_speedup_table; argmax = sample index. */
int oracle_build_speedup_table_msample(int J, int num_nodes, const int16_t *cap, int k_max, int n_max,
                                       int num_samples, const float *alpha_grad, const float *beta_grad,
                                       const float *alpha_local, const float *beta_local,
                                       const float *alpha_node, const float *beta_node, const float *gamma,
                                       const float *phi, const float *m0, const float *m_max_total,
                                       const int32_t *m_samples, const int32_t *m_max_gpu,
                                       const uint8_t *adaptive, const int32_t *fair_k, const int32_t *fair_n,
                                       double *goodput, double *speedup, uint16_t *argmax) {
  if (J < 0 || k_max < 1 || n_max < 1 || num_samples < 1) return ORACLE_ERR_ARG;
  const int KD = k_max + 1, ND = n_max + 1;
  int64_t *kfit = (int64_t *)malloc(sizeof(int64_t) * (size_t)ND);
  max_k_per_n(num_nodes, cap, n_max, kfit);
#pragma omp parallel for schedule(dynamic, 1)
  for (int j = 0; j < J; ++j) {
    double *gj = goodput + (size_t)j * KD * ND;
    double *sj = speedup + (size_t)j * KD * ND;
    uint16_t *aj = argmax ? argmax + (size_t)j * KD * ND : NULL;
    const int adapt = adaptive ? adaptive[j] != 0 : 1;
    const int ns = adapt ? num_samples : 1;
    for (int K = 0; K < KD; ++K) {
      for (int N = 0; N < ND; ++N) {
        double best = 0.0;
        int best_i = -1;
        if (N >= 1 && K >= N && (int64_t)K <= kfit[N] && m_max_gpu[j] >= 1) {
          for (int i = 0; i < ns; ++i) {
            const int64_t M = adapt ? (int64_t)m_samples[(size_t)j * num_samples + i] : (int64_t)m0[j];
            if (M < 1) continue;
            const int64_t per_gpu = (M + K - 1) / K;
            const int64_t s = (per_gpu + m_max_gpu[j] - 1) / m_max_gpu[j] - 1;
            const int64_t m = (per_gpu + s) / (s + 1);
            const double Mrun = (double)K * (double)m * (double)(s + 1);
            if (Mrun < m0[j] || Mrun > m_max_total[j]) continue;
            const double tg = oracle_t_grad(alpha_grad[j], beta_grad[j], (double)m);
            const double ts = oracle_t_sync(alpha_local[j], beta_local[j], alpha_node[j], beta_node[j], K, N);
            const double ti = oracle_t_iter(tg, ts, gamma[j], (int)s);
            const double eff = adapt ? oracle_efficiency(phi[j], m0[j], Mrun) : 1.0;
            const double g = (Mrun / ti) * eff;
            if (best_i < 0 || g > best) { best = g; best_i = i; }
          }
        }
        gj[K * ND + N] = best_i >= 0 ? best : 0.0;
        if (aj) aj[K * ND + N] = best_i >= 0 ? (uint16_t)best_i : 0xFFFFu;
      }
    }
    const int kf = fair_k[j], nf = fair_n[j];
    const double denom = (kf >= 0 && kf < KD && nf >= 0 && nf < ND) ? gj[kf * ND + nf] : 0.0;
    for (int e = 0; e < KD * ND; ++e) sj[e] = denom > 0.0 ? gj[e] / denom : 0.0;
  }
  free(kfit);
  return ORACLE_OK;
}

/* REALLOC_FACTOR_j(delta) = (T_j - R_j delta) / (T_j + delta), kept inside [0, 1]
 * (Sec. 4.2, re-allocation penalty). */
void oracle_realloc_factor(int J, const float *age_sec, const int32_t *num_restarts, double delta,
                           double *out) {
    for (int j = 0; j < J; ++j) {
        double T = age_sec[j], R = num_restarts[j];
        double f = (T - R * delta) / (T + delta);
        if (!(f >= 0.0)) f = 0.0;
        if (f > 1.0) f = 1.0;
        out[j] = f;
    }
}

/* FITNESS_p(A) = ((1/J) sum_j SPEEDUP_j(A_j)^p)^(1/p) over the active jobs (Eq. 14), with
 * SPEEDUP_j looked up at (K, N) of row j, multiplied by REALLOC_FACTOR_j when the row
 * differs from a running job's current row, then raised to the floor.  p = 0 is the
 * geometric mean (the limit of Eq. 14). */
int oracle_eval_fitness(int P, int J, int num_nodes, int k_max, int n_max, const int16_t *pop,
                        const double *speedup, const int16_t *cur, const double *realloc_factor,
                        const uint8_t *active, double p, double floor_, double *fitness) {
    if (P < 0 || J < 0 || num_nodes < 1 || !pop || !speedup || !fitness) return ORACLE_ERR_ARG;
    const int KD = k_max + 1, ND = n_max + 1;
#pragma omp parallel for schedule(static)
    for (int c = 0; c < P; ++c) {
        double acc = 0.0;
        int64_t count = 0;
        for (int j = 0; j < J; ++j) {
            if (active && !active[j]) continue;
            const int16_t *row = pop + ((size_t)c * J + j) * num_nodes;
            int64_t K = 0, N = 0, Kcur = 0;
            int changed = 0;
            for (int n = 0; n < num_nodes; ++n) {
                K += row[n];
                N += (row[n] > 0);
                if (cur) {
                    Kcur += cur[(size_t)j * num_nodes + n];
                    changed |= (row[n] != cur[(size_t)j * num_nodes + n]);
                }
            }
            if (K < 0) K = 0;
            if (K > k_max) K = k_max;
            if (N > n_max) N = n_max;
            double x = speedup[((size_t)j * KD + K) * ND + N];
            if (cur && realloc_factor && changed && Kcur > 0) x *= realloc_factor[j];
            if (x < floor_) x = floor_;
            if (p == 0.0) acc += log(x);
            else if (p == 1.0) acc += x;
            else if (p == -1.0) acc += 1.0 / x;
            else acc += pow(x, p);
            ++count;
        }
        double f;
        if (count == 0) f = 0.0;
        else if (p == 0.0) f = exp(acc / (double)count);
        else if (p == 1.0) f = acc / (double)count;
        else if (p == -1.0) f = (double)count / acc;
        else f = pow(acc / (double)count, 1.0 / p);
        fitness[c] = f;
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------- */
/* Genetic operators                                                          */
/* ------------------------------------------------------------------------- */

/* Order-preserving integer image of an fp32 bit pattern (larger float -> larger key). */
static uint32_t order_key(uint32_t bits) { return bits ^ ((bits >> 31) ? 0xFFFFFFFFu : 0x80000000u); }

/* rank[i] = number of candidates that sort before i under (fitness descending, index
 * ascending). */
void oracle_rank(int P, const uint32_t *fitness_bits, int32_t *rank) {
    for (int i = 0; i < P; ++i) {
        uint32_t ki = order_key(fitness_bits[i]);
        int32_t r = 0;
        for (int o = 0; o < P; ++o) {
            uint32_t ko = order_key(fitness_bits[o]);
            if (ko > ki || (ko == ki && o < i)) ++r;
        }
        rank[i] = r;
    }
}

/* Copy a row, forcing every entry into [0, capacity of its node]. */
static void sanitise_row(const int16_t *src, const int16_t *cap, int num_nodes, int16_t *dst) {
    for (int n = 0; n < num_nodes; ++n) {
        int v = src ? src[n] : 0;
        int c = cap[n] > 0 ? cap[n] : 0;
        if (v < 0) v = 0;
        if (v > c) v = c;
        dst[n] = (int16_t)v;
    }
}

/* index of the t-th (0-based) occupied node in ascending order, or -1 */
static int nth_occupied(const int16_t *row, int num_nodes, uint32_t t) {
    for (int n = 0; n < num_nodes; ++n)
        if (row[n] > 0) {
            if (t == 0) return n;
            --t;
        }
    return -1;
}

/* The "perturb" operator on one row: with probability thr / 2^32 apply one of
 * grow (one more GPU on a random node), shrink (one GPU less on a random occupied
 * node), relocate (move a random occupied node's GPUs onto a random node). */
void oracle_mutate_row(int16_t *row, int num_nodes, const uint32_t w[4], uint32_t thr) {
    if (!(w[0] < thr)) return;
    uint32_t op = mulhi(w[1], 3u);
    int occ = 0;
    for (int n = 0; n < num_nodes; ++n) occ += (row[n] > 0);
    if (op == 0u) {
        int n = (int)mulhi(w[3], (uint32_t)num_nodes);
        if (row[n] < 32767) row[n] = (int16_t)(row[n] + 1);
    } else if (op == 1u) {
        if (occ > 0) {
            int n = nth_occupied(row, num_nodes, mulhi(w[2], (uint32_t)occ));
            row[n] = (int16_t)(row[n] - 1);
        }
    } else {
        if (occ > 0) {
            int ns = nth_occupied(row, num_nodes, mulhi(w[2], (uint32_t)occ));
            int nd = (int)mulhi(w[3], (uint32_t)num_nodes);
            if (nd != ns) {
                int v = (int)row[nd] + (int)row[ns];
                row[nd] = (int16_t)(v > 32767 ? 32767 : v);
                row[ns] = 0;
            }
        }
    }
}

/* Row pass of repair: entries into [0, cap_n]; replicas above the job's cap removed from
 * the highest-index occupied node downward; occupied nodes beyond n_max cleared from
 * the highest index downward.  Returns whether the row still spans >= 2 nodes. */
static int repair_row(int16_t *row, const int16_t *cap, int num_nodes, int k_cap, int n_max) {
    int64_t K = 0;
    for (int n = 0; n < num_nodes; ++n) {
        int c = cap[n] > 0 ? cap[n] : 0;
        if (row[n] < 0) row[n] = 0;
        if (row[n] > c) row[n] = (int16_t)c;
        K += row[n];
    }
    int64_t excess = K - k_cap;
    for (int n = num_nodes - 1; n >= 0 && excess > 0; --n) {
        int64_t take = row[n] < excess ? row[n] : excess;
        row[n] = (int16_t)(row[n] - take);
        excess -= take;
    }
    int occ = 0;
    for (int n = 0; n < num_nodes; ++n) {
        if (row[n] > 0) {
            ++occ;
            if (occ > n_max) row[n] = 0;
        }
    }
    if (occ > n_max) occ = n_max;
    return occ >= 2;
}

/* Column passes of repair with explicit rotation offsets (one per node).
 * Interference avoidance (Sec. 4.2): on every node, of the jobs that were distributed
 * after the row pass and occupy the node, only the first in job order rotated to start
 * at intf_offset[n] stays.  Capacity: while a node is over capacity, GPUs are taken
 * from its jobs in job order rotated to start at cap_offset[n]. */
static void repair_columns(int16_t *A, int J, int num_nodes, const int16_t *cap,
                           const uint8_t *distributed, const uint32_t *intf_offset,
                           const uint32_t *cap_offset) {
    for (int n = 0; n < num_nodes; ++n) {
        int kept = 0;
        for (int t = 0; t < J; ++t) {
            int j = (int)(((uint64_t)intf_offset[n] + (uint64_t)t) % (uint64_t)J);
            if (distributed[j] && A[(size_t)j * num_nodes + n] > 0) {
                if (kept) A[(size_t)j * num_nodes + n] = 0;
                kept = 1;
            }
        }
    }
    for (int n = 0; n < num_nodes; ++n) {
        int64_t total = 0;
        for (int j = 0; j < J; ++j) total += A[(size_t)j * num_nodes + n];
        int64_t excess = total - (cap[n] > 0 ? cap[n] : 0);
        for (int t = 0; t < J && excess > 0; ++t) {
            int j = (int)(((uint64_t)cap_offset[n] + (uint64_t)t) % (uint64_t)J);
            int64_t v = A[(size_t)j * num_nodes + n];
            int64_t take = v < excess ? v : excess;
            A[(size_t)j * num_nodes + n] = (int16_t)(v - take);
            excess -= take;
        }
    }
}

static int clamp_k_cap(const int32_t *k_cap, int j, int k_max) {
    int kc = k_cap ? k_cap[j] : k_max;
    if (kc > k_max) kc = k_max;
    if (kc < 0) kc = 0;
    return kc;
}

/* Repair of one matrix in place with the rotation offsets given by the caller. */
int oracle_repair_with_offsets(int J, int num_nodes, const int16_t *cap, const int32_t *k_cap,
                               int k_max, int n_max, const uint8_t *active, int16_t *A,
                               const uint32_t *intf_offset, const uint32_t *cap_offset) {
    if (J < 1 || num_nodes < 1 || !cap || !A) return ORACLE_ERR_ARG;
    uint8_t *dist = (uint8_t *)malloc((size_t)J);
    for (int j = 0; j < J; ++j) {
        int16_t *row = A + (size_t)j * num_nodes;
        if (active && !active[j]) memset(row, 0, sizeof(int16_t) * (size_t)num_nodes);
        dist[j] = (uint8_t)repair_row(row, cap, num_nodes, clamp_k_cap(k_cap, j, k_max), n_max);
    }
    repair_columns(A, J, num_nodes, cap, dist, intf_offset, cap_offset);
    free(dist);
    return ORACLE_OK;
}

/* Repair with the offsets drawn from the operator stream: node n of candidate `cand`
 * uses floor(w0 * J / 2^32) of the REPAIR_INTF and REPAIR_CAP slots. */
int oracle_repair(int J, int num_nodes, const int16_t *cap, const int32_t *k_cap, int k_max,
                  int n_max, const uint8_t *active, int16_t *A, uint64_t seed, uint32_t round,
                  uint32_t cand, uint32_t generation) {
    if (J < 1 || num_nodes < 1) return ORACLE_ERR_ARG;
    uint32_t *oi = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)num_nodes * 2);
    uint32_t *oc = oi + num_nodes;
    for (int n = 0; n < num_nodes; ++n) {
        uint32_t w[4];
        draw(seed, round, (uint32_t)n, cand, generation, SLOT_REPAIR_INTF, w);
        oi[n] = mulhi(w[0], (uint32_t)J);
        draw(seed, round, (uint32_t)n, cand, generation, SLOT_REPAIR_CAP, w);
        oc[n] = mulhi(w[0], (uint32_t)J);
    }
    int rc = oracle_repair_with_offsets(J, num_nodes, cap, k_cap, k_max, n_max, active, A, oi, oc);
    free(oi);
    return rc;
}

/* One generation: elites are copies of the best-ranked parents; every other child takes
 * each job's row from one of two parents, each the better of a random pair (binary
 * tournament on rank), perturbs it, and the whole child is repaired. */
int oracle_ga_generation(int P, int J, int num_nodes, const int16_t *cap, const int32_t *k_cap,
                         int k_max, int n_max, const uint8_t *active, int num_elite,
                         uint32_t thr_mutate, uint64_t seed, uint32_t round, uint32_t generation,
                         const int16_t *pop_in, const uint32_t *fitness_bits, int16_t *pop_out) {
    if (P < 1 || J < 1 || num_nodes < 1 || num_elite < 0 || num_elite > P) return ORACLE_ERR_ARG;
    int32_t *rank = (int32_t *)malloc(sizeof(int32_t) * (size_t)P * 2);
    int32_t *order = rank + P;
    oracle_rank(P, fitness_bits, rank);
    for (int i = 0; i < P; ++i) order[rank[i]] = i;
    const size_t msz = (size_t)J * num_nodes;
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < P; ++c) {
        int16_t *child = pop_out + (size_t)c * msz;
        if (c < num_elite) {
            const int16_t *par = pop_in + (size_t)order[c] * msz;
            for (int j = 0; j < J; ++j)
                sanitise_row(par + (size_t)j * num_nodes, cap, num_nodes, child + (size_t)j * num_nodes);
        } else {
            uint32_t w[4];
            draw(seed, round, 0u, (uint32_t)c, generation, SLOT_SELECT, w);
            int i0 = (int)mulhi(w[0], (uint32_t)P), i1 = (int)mulhi(w[1], (uint32_t)P);
            int i2 = (int)mulhi(w[2], (uint32_t)P), i3 = (int)mulhi(w[3], (uint32_t)P);
            int pa = rank[i0] <= rank[i1] ? i0 : i1;
            int pb = rank[i2] <= rank[i3] ? i2 : i3;
            for (int j = 0; j < J; ++j) {
                int16_t *row = child + (size_t)j * num_nodes;
                draw(seed, round, (uint32_t)j, (uint32_t)c, generation, SLOT_XOVER, w);
                int src = (w[0] >> 31) ? pb : pa;
                sanitise_row(pop_in + (size_t)src * msz + (size_t)j * num_nodes, cap, num_nodes, row);
                draw(seed, round, (uint32_t)j, (uint32_t)c, generation, SLOT_MUTATE, w);
                oracle_mutate_row(row, num_nodes, w, thr_mutate);
            }
        }
        oracle_repair(J, num_nodes, cap, k_cap, k_max, n_max, active, child, seed, round,
                      (uint32_t)c, generation);
    }
    free(rank);
    return ORACLE_OK;
}

/* Initial population of a round: candidate 0 is the current allocation, the others are
 * the current allocation perturbed row by row with threshold thr_init; all repaired. */
int oracle_init_population(int P, int J, int num_nodes, const int16_t *cap, const int32_t *k_cap,
                           int k_max, int n_max, const uint8_t *active, uint32_t thr_init,
                           uint64_t seed, uint32_t round, const int16_t *cur, int16_t *pop_out) {
    if (P < 1 || J < 1 || num_nodes < 1) return ORACLE_ERR_ARG;
    const size_t msz = (size_t)J * num_nodes;
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < P; ++c) {
        int16_t *child = pop_out + (size_t)c * msz;
        for (int j = 0; j < J; ++j) {
            int16_t *row = child + (size_t)j * num_nodes;
            sanitise_row(cur ? cur + (size_t)j * num_nodes : NULL, cap, num_nodes, row);
            if (c > 0) {
                uint32_t w[4];
                draw(seed, round, (uint32_t)j, (uint32_t)c, GEN_INIT, SLOT_INIT, w);
                oracle_mutate_row(row, num_nodes, w, thr_init);
            }
        }
        oracle_repair(J, num_nodes, cap, k_cap, k_max, n_max, active, child, seed, round,
                      (uint32_t)c, GEN_INIT);
    }
    return ORACLE_OK;
}

static uint32_t f32_bits(double v) {
    float f = (float)v;
    uint32_t b;
    memcpy(&b, &f, 4);
    return b;
}

/* A whole scheduling round (Sec. 4.3): table, initial population, `generations` times
 * (operators, fitness), and the best matrix of the last population.  The selection
 * consumes the double fitness rounded to fp32. */
int oracle_schedule_round(int P, int J, int num_nodes, const int16_t *cap, int k_max, int n_max,
                          int grid_m, int grid_s, const float *alpha_grad, const float *beta_grad,
                          const float *alpha_local, const float *beta_local,
                          const float *alpha_node, const float *beta_node, const float *gamma,
                          const float *phi, const float *m0, const float *m_max_total,
                          const int32_t *m_grid, const int32_t *k_cap, const int32_t *fair_k,
                          const int32_t *fair_n, const float *age_sec, const int32_t *num_restarts,
                          const uint8_t *active, double p, double delta, double floor_,
                          int num_elite, uint32_t thr_mutate, uint32_t thr_init, uint64_t seed,
                          uint32_t round, int generations, const int16_t *cur, int16_t *best,
                          double *best_fitness) {
    if (P < 1 || J < 1 || num_nodes < 1 || generations < 0) return ORACLE_ERR_ARG;
    const int KD = k_max + 1, ND = n_max + 1;
    const size_t tsz = (size_t)J * KD * ND, msz = (size_t)J * num_nodes;
    double *goodput = (double *)malloc(sizeof(double) * tsz * 2);
    double *speedup = goodput + tsz;
    double *rf = (double *)malloc(sizeof(double) * (size_t)J);
    double *fit = (double *)malloc(sizeof(double) * (size_t)P);
    uint32_t *bits = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)P);
    int16_t *pa = (int16_t *)malloc(sizeof(int16_t) * msz * (size_t)P);
    int16_t *pb = (int16_t *)malloc(sizeof(int16_t) * msz * (size_t)P);
    oracle_build_speedup_table(J, num_nodes, cap, k_max, n_max, grid_m, grid_s, alpha_grad,
                               beta_grad, alpha_local, beta_local, alpha_node, beta_node, gamma,
                               phi, m0, m_max_total, m_grid, fair_k, fair_n, goodput, speedup, NULL);
    oracle_realloc_factor(J, age_sec, num_restarts, delta, rf);
    oracle_init_population(P, J, num_nodes, cap, k_cap, k_max, n_max, active, thr_init, seed, round,
                           cur, pa);
    oracle_eval_fitness(P, J, num_nodes, k_max, n_max, pa, speedup, cur, rf, active, p, floor_, fit);
    for (int g = 0; g < generations; ++g) {
        for (int c = 0; c < P; ++c) bits[c] = f32_bits(fit[c]);
        oracle_ga_generation(P, J, num_nodes, cap, k_cap, k_max, n_max, active, num_elite,
                             thr_mutate, seed, round, (uint32_t)g, pa, bits, pb);
        int16_t *t = pa; pa = pb; pb = t;
        oracle_eval_fitness(P, J, num_nodes, k_max, n_max, pa, speedup, cur, rf, active, p, floor_, fit);
    }
    int bi = 0;
    for (int c = 0; c < P; ++c) bits[c] = f32_bits(fit[c]);
    for (int c = 1; c < P; ++c)
        if (order_key(bits[c]) > order_key(bits[bi])) bi = c;
    memcpy(best, pa + (size_t)bi * msz, sizeof(int16_t) * msz);
    *best_fitness = fit[bi];
    free(goodput); free(rf); free(fit); free(bits); free(pa); free(pb);
    return ORACLE_OK;
}

/* Goodput-driven auto-scaling (Sec. 5.3, cloud auto-scaling): a job on n whole nodes of G GPUs
 * is scaled up when its goodput per GPU exceeds the fraction U of the single-GPU goodput
 * ("ideal" = perfect scalability), to the largest node count whose goodput is still at
 * least the fraction L of ideal; otherwise it keeps its nodes.  The comparisons are made in
 * fp32, in this order of operations, on the fp32 table: they decide integers. */
int oracle_autoscale_targets(int J, int k_max, int n_max, int gpus_per_node, const float *goodput,
                             const int32_t *cur_nodes, float U, float L, int32_t *target_nodes) {
  if (J < 0 || gpus_per_node < 1 || !goodput || !cur_nodes || !target_nodes) return ORACLE_ERR_ARG;
  const int KD = k_max + 1, ND = n_max + 1;
  for (int j = 0; j < J; ++j) {
    const float *g = goodput + (size_t)j * KD * ND;
    const float g1 = g[1 * ND + 1];
    int n = cur_nodes[j];
    int limit = n_max;
    if (limit * gpus_per_node > k_max) limit = k_max / gpus_per_node;
    int target = n;
    if (n >= 1 && n <= limit && g1 > 0.0f) {
      const float k = (float)(n * gpus_per_node);
      const float ideal_u = (float)((float)(U * k) * g1);
      if (g[(n * gpus_per_node) * ND + n] > ideal_u) {
        for (int t = n + 1; t <= limit; ++t) {
          const float kt = (float)(t * gpus_per_node);
          const float ideal_l = (float)((float)(L * kt) * g1);
          if (g[(t * gpus_per_node) * ND + t] >= ideal_l) target = t;
        }
      }
    }
    target_nodes[j] = target;
  }
  return ORACLE_OK;
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* ------------------------------------------------------------------------- */
/* Rack-level locality                                                        */
/* ------------------------------------------------------------------------- */

/* T_sync with the extension the paper names right after Eq. 9 ("a third pair of
 * parameters" for rack-level locality).  Read as three placement classes: all replicas on
 * one node -> local pair; several nodes of one rack -> node pair; nodes of two or more racks
 * (R >= 2 racks occupied) -> rack pair.  Linear in K - 2 like the other two. */
double oracle_t_sync_rack(double alpha_local, double beta_local, double alpha_node, double beta_node,
                          double alpha_rack, double beta_rack, int K, int N, int R) {
    if (K <= 1) return 0.0;
    if (N == 1) return alpha_local + beta_local * (double)(K - 2);
    if (R <= 1) return alpha_node + beta_node * (double)(K - 2);
    return alpha_rack + beta_rack * (double)(K - 2);
}

/* GOODPUT of Eq. 4/7 with the three-class T_sync. */
double oracle_goodput_rack(double alpha_grad, double beta_grad, double alpha_local, double beta_local,
                           double alpha_node, double beta_node, double alpha_rack, double beta_rack,
                           double gamma, double phi, double m0, double m_max_total, int K, int N, int R,
                           int m, int s, int *feasible) {
    double M = (double)K * (double)m * (double)(s + 1);
    int ok = (K >= 1 && N >= 1 && N <= K && R >= 1 && R <= N && M >= m0 && M <= m_max_total);
    if (feasible) *feasible = ok;
    if (!ok) return 0.0;
    double tg = oracle_t_grad(alpha_grad, beta_grad, (double)m);
    double ts = oracle_t_sync_rack(alpha_local, beta_local, alpha_node, beta_node, alpha_rack, beta_rack, K, N, R);
    double ti = oracle_t_iter(tg, ts, gamma, s);
    return (M / ti) * oracle_efficiency(phi, m0, M);
}

/* The table of the third class: entry (K, N), N >= 2, is the best goodput over the grid of an
 * allocation of K replicas on N nodes that lie in two or more racks, and its ratio to the same
 * fair-share goodput as the two-class table uses (Eq. 15; the fair share is packed on as few
 * nodes as possible, hence inside one rack).  Validity of (K, N) and ties as in
 * oracle_build_speedup_table; entries with N < 2 are 0 / 0xFFFF. */
int oracle_build_speedup_table_rack(int J, int num_nodes, const int16_t *cap, int k_max, int n_max,
                                    int grid_m, int grid_s, const float *alpha_grad,
                                    const float *beta_grad, const float *alpha_local,
                                    const float *beta_local, const float *alpha_node,
                                    const float *beta_node, const float *alpha_rack,
                                    const float *beta_rack, const float *gamma, const float *phi,
                                    const float *m0, const float *m_max_total, const int32_t *m_grid,
                                    const int32_t *fair_k, const int32_t *fair_n, double *goodput,
                                    double *speedup, uint16_t *argmax) {
    if (J < 0 || k_max < 1 || n_max < 1 || grid_m < 1 || grid_s < 1) return ORACLE_ERR_ARG;
    const int KD = k_max + 1, ND = n_max + 1;
    int64_t *kfit = (int64_t *)malloc(sizeof(int64_t) * (size_t)ND);
    max_k_per_n(num_nodes, cap, n_max, kfit);
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < J; ++j) {
        double *gj = goodput + (size_t)j * KD * ND;
        double *sj = speedup + (size_t)j * KD * ND;
        uint16_t *aj = argmax ? argmax + (size_t)j * KD * ND : NULL;
        for (int K = 0; K < KD; ++K) {
            for (int N = 0; N < ND; ++N) {
                double best = 0.0;
                int best_s = -1, best_i = -1;
                int valid = (N >= 2 && K >= N && (int64_t)K <= kfit[N]);
                if (valid) {
                    for (int i = 0; i < grid_m; ++i) {
                        for (int s = 0; s < grid_s; ++s) {
                            int ok = 0;
                            double g = oracle_goodput_rack(alpha_grad[j], beta_grad[j], alpha_local[j], beta_local[j],
                                                           alpha_node[j], beta_node[j], alpha_rack[j], beta_rack[j],
                                                           gamma[j], phi[j], m0[j], m_max_total[j], K, N, 2,
                                                           m_grid[(size_t)j * grid_m + i], s, &ok);
                            if (!ok) continue;
                            int better = (best_i < 0) || (g > best) ||
                                         (g == best && (s < best_s || (s == best_s && i < best_i)));
                            if (better) { best = g; best_s = s; best_i = i; }
                        }
                    }
                }
                gj[K * ND + N] = (best_i >= 0) ? best : 0.0;
                if (aj) aj[K * ND + N] = (best_i >= 0) ? (uint16_t)(best_i * grid_s + best_s) : 0xFFFFu;
            }
        }
        /* the fair-share goodput: one rack, so the local or the node pair */
        int kf = fair_k[j], nf = fair_n[j];
        double denom = 0.0;
        if (nf >= 1 && nf <= n_max && kf >= nf && kf <= k_max && (int64_t)kf <= kfit[nf]) {
            for (int i = 0; i < grid_m; ++i) {
                for (int s = 0; s < grid_s; ++s) {
                    int ok = 0;
                    double g = oracle_goodput_rack(alpha_grad[j], beta_grad[j], alpha_local[j], beta_local[j],
                                                   alpha_node[j], beta_node[j], alpha_rack[j], beta_rack[j], gamma[j],
                                                   phi[j], m0[j], m_max_total[j], kf, nf, 1,
                                                   m_grid[(size_t)j * grid_m + i], s, &ok);
                    if (ok && g > denom) denom = g;
                }
            }
        }
        for (int e = 0; e < KD * ND; ++e) sj[e] = (denom > 0.0) ? gj[e] / denom : 0.0;
    }
    free(kfit);
    return ORACLE_OK;
}

/* Eq. 14 with rack-level locality: as oracle_eval_fitness, but a row whose occupied nodes lie in
 * two or more racks (node_rack[n] = rack of node n) takes its speedup from the third-class
 * table. */
int oracle_eval_fitness_racks(int P, int J, int num_nodes, int k_max, int n_max, const int16_t *pop,
                              const double *speedup, const double *speedup_rack, const int16_t *node_rack,
                              const int16_t *cur, const double *realloc_factor, const uint8_t *active, double p,
                              double floor_, double *fitness) {
    if (P < 0 || J < 0 || num_nodes < 1 || !pop || !speedup || !speedup_rack || !node_rack || !fitness)
        return ORACLE_ERR_ARG;
    const int KD = k_max + 1, ND = n_max + 1;
#pragma omp parallel for schedule(static)
    for (int c = 0; c < P; ++c) {
        double acc = 0.0;
        int64_t count = 0;
        for (int j = 0; j < J; ++j) {
            if (active && !active[j]) continue;
            const int16_t *row = pop + ((size_t)c * J + j) * num_nodes;
            int64_t K = 0, N = 0, Kcur = 0;
            int changed = 0, first_rack = -1, several_racks = 0;
            for (int n = 0; n < num_nodes; ++n) {
                K += row[n];
                N += (row[n] > 0);
                if (row[n] > 0) {
                    if (first_rack < 0) first_rack = node_rack[n];
                    else if (node_rack[n] != first_rack) several_racks = 1;
                }
                if (cur) {
                    Kcur += cur[(size_t)j * num_nodes + n];
                    changed |= (row[n] != cur[(size_t)j * num_nodes + n]);
                }
            }
            if (K < 0) K = 0;
            if (K > k_max) K = k_max;
            if (N > n_max) N = n_max;
            const double *table = several_racks ? speedup_rack : speedup;
            double x = table[((size_t)j * KD + K) * ND + N];
            if (cur && realloc_factor && changed && Kcur > 0) x *= realloc_factor[j];
            if (x < floor_) x = floor_;
            if (p == 0.0) acc += log(x);
            else if (p == 1.0) acc += x;
            else if (p == -1.0) acc += 1.0 / x;
            else acc += pow(x, p);
            ++count;
        }
        double f;
        if (count == 0) f = 0.0;
        else if (p == 0.0) f = exp(acc / (double)count);
        else if (p == 1.0) f = acc / (double)count;
        else if (p == -1.0) f = (double)count / acc;
        else f = pow(acc / (double)count, 1.0 / p);
        fitness[c] = f;
    }
    return ORACLE_OK;
}

/* Threads the parallel loops above use from now on (1: the single-core figure the paper's
 * scheduler is quoted on); 0 restores the default. */
void oracle_set_threads(int n) {
#ifdef _OPENMP
    omp_set_num_threads(n > 0 ? n : omp_get_num_procs());
#else
    (void)n;
#endif
}
