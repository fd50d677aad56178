// Row store: the population of a running scheduling round kept as shared rows (Sec. 4.3).
//
// A generation copies almost every child row verbatim from one of two parents; only the
// perturbed rows and the few rows the repair touches are new.  Here a row's contents live
// once in a pool and a candidate is an array of row indices.  Next to each stored row sit
// a 32-byte record: up to six occupied nodes, the row's summary (K, N, entries that differ
// from the current allocation) and its term of the fitness sum (a stored row always serves
// the same job, so the term is fixed for the round).  A generation reads 36 bytes per
// unchanged row instead of the row, and writes 4.  New rows are appended to the pool (copy
// on write); when a half of the pool runs low the live rows are copied to the other half.
//
// One block evolves one candidate per generation: parent selection, row-wise crossover,
// perturbation, per-row caps, interference and capacity repair, and the candidate's fitness.
// The operators, their random draws and the order of the fitness sums are the same as in
// the dense kernels, so both paths produce identical populations and fitness bits.
#include "common.cuh"
#include "fitness_common.cuh"

namespace {

constexpr int REC_WORDS = 8;                  // words of a record: REC_ENTRIES occupants, the row's fitness term, its summary
constexpr int REC_ENTRIES = 6;                // occupied nodes a record can hold
constexpr int REC_TERM = 6, REC_SUMM = 7;     // positions of the term (float bits) and the summary
constexpr uint32_t REC_OVERFLOW = 0xFFFFFFFFu;  // first word of a record whose row has more
constexpr int OCC = 16;                       // occupants listed per node inside a block
constexpr int GEN_THREADS = 256;
constexpr int GEN_WARPS = GEN_THREADS / 32;
constexpr int GEN_GROUPS = GEN_THREADS / 16;  // rows worked on at a time by a block
constexpr int STORE_MAX_JOBS = 8192;          // job index must fit 13 bits of an occupant entry
constexpr int COW_RESERVE = 16;               // slots a block takes up front for rows the column pass changes

struct StoreView {
  int16_t *pool;
  uint32_t *rec;
  unsigned long long half_cap;
  uint32_t zero_slot;
};

// ---- a row as 16-byte pieces of 8 entries (entries of stored rows are in [0, 2047]) -----------
__device__ __forceinline__ uint32_t piece_mask(uint4 x) {   // bit h: entry h of the piece is occupied
  // per word: min(half, 1) for both halves (entries are non-negative), folded to two bits
  const uint32_t a = __vimin_s16x2_relu(x.x, 0x00010001u), b = __vimin_s16x2_relu(x.y, 0x00010001u);
  const uint32_t c = __vimin_s16x2_relu(x.z, 0x00010001u), d = __vimin_s16x2_relu(x.w, 0x00010001u);
  const uint32_t lo = a | (b << 2) | (c << 4) | (d << 6);   // bits 0,2,4,6: low halves; 16,18,20,22: high halves
  return (lo | (lo >> 15)) & 0xFFu;
}
__device__ __forceinline__ int piece_sum(uint4 x) {
  int k = __dp2a_lo((int)x.x, 0x0101, 0);
  k = __dp2a_lo((int)x.y, 0x0101, k);
  k = __dp2a_lo((int)x.z, 0x0101, k);
  return __dp2a_lo((int)x.w, 0x0101, k);
}
__device__ __forceinline__ int piece_entry(uint4 x, int h) {
  const uint32_t w = (h < 2) ? x.x : (h < 4) ? x.y : (h < 6) ? x.z : x.w;
  return (int)((w >> ((h & 1) * 16)) & 0xFFFFu);
}
__device__ __forceinline__ int piece_diff(uint4 x, uint4 c) {   // entries that differ
  // each half of the xor is a non-negative int16, so min(half, 1) counts the halves that differ
  const uint32_t d = __vimin_s16x2_relu(x.x ^ c.x, 0x00010001u) + __vimin_s16x2_relu(x.y ^ c.y, 0x00010001u) +
                     __vimin_s16x2_relu(x.z ^ c.z, 0x00010001u) + __vimin_s16x2_relu(x.w ^ c.w, 0x00010001u);
  return (int)((d & 0xFFFFu) + (d >> 16));
}

// Rows are worked on by groups of 16 lanes (two rows per warp at a time).  A lane looks after
// the PPL consecutive pieces [sub * PPL, sub * PPL + PPL) of its group's row, so lane order is
// node order.  PPL (1, 2 or 4: rows have at most 64 pieces) is a template parameter of
// everything that walks a row, so that short rows do not pay for the pieces they lack.
constexpr int GROUP = 16;

struct Grp {
  int sub;         // lane within the group
  unsigned mask;   // the group's lanes
  int row_vecs;    // pieces of a row
};

__device__ __forceinline__ Grp make_group(int lane, int NN) {
  Grp g;
  g.sub = lane & (GROUP - 1);
  g.mask = 0xFFFFu << (lane & GROUP);
  g.row_vecs = NN >> 3;
  return g;
}

__device__ __forceinline__ int group_sum(const Grp &g, int v) { return __reduce_add_sync(g.mask, v); }

// 16 bytes of a row in global memory (any alignment of the row's start); `cg` reads through to
// L2, for rows written earlier in the same kernel
template <bool CG>
__device__ __forceinline__ uint4 load_piece(const int16_t *src, int v) {
  if (((uintptr_t)src & 15) == 0) return CG ? __ldcg((const uint4 *)src + v) : *((const uint4 *)src + v);
  uint32_t w[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t lo = (uint16_t)(CG ? __ldcg(src + 8 * v + 2 * k) : src[8 * v + 2 * k]);
    const uint32_t hi = (uint16_t)(CG ? __ldcg(src + 8 * v + 2 * k + 1) : src[8 * v + 2 * k + 1]);
    w[k] = lo | (hi << 16);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// a row from global to shared memory by one group (coalesced: piece sub, sub + 16, ...)
template <bool CG>
__device__ __forceinline__ void load_row(const Grp &g, int16_t *dst, const int16_t *src) {
  for (int v = g.sub; v < g.row_vecs; v += GROUP) ((uint4 *)dst)[v] = load_piece<CG>(src, v);
}

__device__ __forceinline__ void store_row(const Grp &g, int16_t *dst, const int16_t *src_shared) {
  for (int v = g.sub; v < g.row_vecs; v += GROUP) ((uint4 *)dst)[v] = ((const uint4 *)src_shared)[v];
}

// This lane's pieces of a row in shared memory, their occupancy masks, and where the lane's
// occupants come in node order: `first` = occupants in lower lanes, `total` = the row's N.
template <int PPL>
struct RowPieces {
  uint4 x[PPL];
  uint32_t mask[PPL];
  int first, total;
};

template <int PPL>
__device__ __forceinline__ RowPieces<PPL> row_pieces(const Grp &g, const int16_t *row) {
  RowPieces<PPL> p;
  int cnt = 0;
#pragma unroll
  for (int q = 0; q < PPL; ++q) {
    const int v = g.sub * PPL + q;
    p.x[q] = make_uint4(0u, 0u, 0u, 0u);
    if (v < g.row_vecs) p.x[q] = ((const uint4 *)row)[v];
    p.mask[q] = piece_mask(p.x[q]);
    cnt += __popc(p.mask[q]);
  }
  int incl = cnt;
#pragma unroll
  for (int off = 1; off < GROUP; off <<= 1) {
    const int u = __shfl_up_sync(g.mask, incl, off, GROUP);
    if (g.sub >= off) incl += u;
  }
  p.total = __shfl_sync(g.mask, incl, GROUP - 1, GROUP);
  p.first = incl - cnt;
  return p;
}

// this lane's pieces of the matching row of the current allocation, if there is one
template <int PPL>
struct CurPieces {
  uint4 x[PPL];
  bool have;
};

// this lane's pieces of the current allocation's row (NULL: none), fetched ahead of their use
template <int PPL>
__device__ __forceinline__ CurPieces<PPL> cur_pieces(const Grp &g, const int16_t *cur_row) {
  CurPieces<PPL> c;
  c.have = cur_row != nullptr;
#pragma unroll
  for (int q = 0; q < PPL; ++q) {
    const int v = g.sub * PPL + q;
    c.x[q] = make_uint4(0u, 0u, 0u, 0u);
    if (c.have && v < g.row_vecs) c.x[q] = load_piece<false>(cur_row, v);
  }
  return c;
}

// K, N, entries differing from the current allocation's row (`cur`: its pieces, if any) and the
// occupant entries of a row held in shared memory.  All lanes of the group return the same K, N,
// ndiff; rec_out (shared, REC_WORDS: the entries, the other words are the caller's) is complete
// after the trailing __syncwarp(group).
template <int PPL>
__device__ __forceinline__ RowPieces<PPL> summarise_row(const Grp &g, const int16_t *row, const CurPieces<PPL> &cur,
                                                        int &K, int &N, int &ndiff, uint32_t *rec_out) {
  const RowPieces<PPL> p = row_pieces<PPL>(g, row);
  int k = 0, nd = 0, pos = p.first;
#pragma unroll
  for (int q = 0; q < PPL; ++q) {
    const int v = g.sub * PPL + q;
    k += piece_sum(p.x[q]);
    if (cur.have && v < g.row_vecs) nd += piece_diff(p.x[q], cur.x[q]);
    uint32_t m = p.mask[q];
    while (m && pos < REC_ENTRIES) {
      const int h = __ffs(m) - 1;
      m &= m - 1;
      rec_out[pos++] = (uint32_t)(8 * v + h) | ((uint32_t)piece_entry(p.x[q], h) << 12);
    }
  }
  K = group_sum(g, k);
  ndiff = group_sum(g, nd);
  N = p.total;
  __syncwarp(g.mask);
  if (N > REC_ENTRIES) {
    if (g.sub == 0) rec_out[0] = REC_OVERFLOW;
  } else if (g.sub >= N && g.sub < REC_ENTRIES) {
    rec_out[g.sub] = 0u;
  }
  __syncwarp(g.mask);
  return p;
}

// node index of the t-th occupied entry (ascending) of a row held in shared memory; t < N
template <int PPL>
__device__ __forceinline__ int nth_occupied_row(const Grp &g, const int16_t *row, uint32_t t) {
  const RowPieces<PPL> p = row_pieces<PPL>(g, row);
  int node = -1, before = p.first;
#pragma unroll
  for (int q = 0; q < PPL; ++q) {
    const int c = __popc(p.mask[q]);
    if ((int)t >= before && (int)t < before + c)
      node = 8 * (g.sub * PPL + q) + (int)__fns(p.mask[q], 0, (int)t - before + 1);
    before += c;
  }
  const unsigned who = __ballot_sync(g.mask, node >= 0);
  return __shfl_sync(g.mask, node, who ? __ffs(who) - 1 : (__ffs(g.mask) - 1));
}

// one 32-byte record with a single request
__device__ __forceinline__ void load_record(uint32_t (&r)[REC_WORDS], const uint32_t *p) {
  asm volatile("ld.global.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "l"(p) : "memory");
}

__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ uint32_t pack_summary(int K, int N, int ndiff) {
  return (uint32_t)K | ((uint32_t)N << 11) | ((uint32_t)ndiff << 22);
}

// ---------------------------------------------------------------------------------------
// Build: the dense initial population (rows c * J + j at the start of the pool) gets its
// records and summaries; candidate c, job j points at slot c * J + j.
// ---------------------------------------------------------------------------------------
struct BuildArgs {
  StoreView st;
  uint32_t *ptr;            // [P][J]
  unsigned int *state;      // {next free slot, half}
  const uint8_t *active;
  const int16_t *cur;       // or NULL
  TermParams tp;
  int P, J, NN;
};

template <int PPL>
__global__ void __launch_bounds__(256) rowstore_build_kernel(BuildArgs a) {
  __shared__ __align__(16) int16_t s_row[16][512];
  __shared__ uint32_t s_rec[16][REC_WORDS];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 4;   // 16 groups of 16 lanes, a row each
  const Grp g = make_group(lane, a.NN);
  const long long rows = (long long)a.P * a.J;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    a.state[0] = (unsigned int)rows;
    a.state[1] = 0u;
  }
  // the empty row: contents and record all zero
  if (blockIdx.x == 0) {
    for (int n = threadIdx.x; n < a.NN; n += blockDim.x) a.st.pool[(size_t)a.st.zero_slot * a.NN + n] = 0;
    if (threadIdx.x < REC_WORDS) a.st.rec[(size_t)a.st.zero_slot * REC_WORDS + threadIdx.x] = 0u;
  }
  for (long long r = (long long)blockIdx.x * 16 + grp; r < rows; r += (long long)gridDim.x * 16) {
    const int j = (int)(r % a.J);
    load_row<false>(g, s_row[grp], a.st.pool + (size_t)r * a.NN);
    const CurPieces<PPL> cur = cur_pieces<PPL>(g, a.cur ? a.cur + (size_t)j * a.NN : nullptr);
    __syncwarp(g.mask);
    int K, N, nd;
    summarise_row<PPL>(g, s_row[grp], cur, K, N, nd, s_rec[grp]);
    const bool on = !a.active || a.active[j];
    if (g.sub == 0) {
      s_rec[grp][REC_SUMM] = on ? pack_summary(K, N, nd) : 0u;
      s_rec[grp][REC_TERM] = on ? __float_as_uint(fitness_term(a.tp, j, K, N, nd != 0)) : 0u;
      a.ptr[r] = (uint32_t)r;
    }
    __syncwarp(g.mask);
    if (g.sub < REC_WORDS) a.st.rec[(size_t)r * REC_WORDS + g.sub] = s_rec[grp][g.sub];
    __syncwarp(g.mask);
  }
}

// most slots one generation can take: every row new, plus every block's reserve
__host__ __device__ inline unsigned long long store_worst_case(int P, int J) {
  return (unsigned long long)P * J + (unsigned long long)P * COW_RESERVE;
}

// ---------------------------------------------------------------------------------------
// Compaction check: when the half in use could run out within the next `gens_ahead`
// generations (each may take up to store_worst_case slots), every live row moves to the other half,
// in candidate order, and the indices are rewritten.  The state is read from one copy and
// written to the other, so no block sees it change under it.
// ---------------------------------------------------------------------------------------
struct CompactArgs {
  StoreView st;
  uint32_t *ptr;            // [P][J] indices of the current population (rewritten)
  const unsigned int *state_in;
  unsigned int *state_out;
  int P, J, NN, gens_ahead;
};

__global__ void __launch_bounds__(256) rowstore_compact_kernel(CompactArgs a) {
  const unsigned long long rows = (unsigned long long)a.P * a.J;
  const unsigned int used = a.state_in[0], half = a.state_in[1];
  const unsigned long long limit = (unsigned long long)(half + 1u) * a.st.half_cap;
  const bool move = (unsigned long long)used + (unsigned long long)a.gens_ahead * store_worst_case(a.P, a.J) > limit;
  if (!move) {
    if (blockIdx.x == 0 && threadIdx.x == 0) { a.state_out[0] = used; a.state_out[1] = half; }
    return;
  }
  const unsigned int new_half = 1u - half;
  const unsigned long long base = (unsigned long long)new_half * a.st.half_cap;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    a.state_out[0] = (unsigned int)(base + rows);
    a.state_out[1] = new_half;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row_vecs = a.NN >> 3;
  for (unsigned long long r = (unsigned long long)blockIdx.x * 8 + warp; r < rows; r += (unsigned long long)gridDim.x * 8) {
    const uint32_t slot = a.ptr[r];
    if (slot == a.st.zero_slot) continue;
    const size_t dst = (size_t)(base + r);
    const uint4 *s4 = (const uint4 *)(a.st.pool + (size_t)slot * a.NN);
    uint4 *d4 = (uint4 *)(a.st.pool + dst * a.NN);
    for (int v = lane; v < row_vecs; v += 32) d4[v] = s4[v];
    if (lane < REC_WORDS) a.st.rec[dst * REC_WORDS + lane] = a.st.rec[(size_t)slot * REC_WORDS + lane];
    if (lane == 0) a.ptr[r] = (uint32_t)dst;
  }
}

// ---------------------------------------------------------------------------------------
// Gather: dense rows of `count` candidates (first_candidate .., or the single candidate
// *index when index is not NULL) from their indices.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rowstore_gather_kernel(StoreView st, const uint32_t *__restrict__ ptr, int first_candidate, long long rows,
                       const int32_t *__restrict__ index, int J, int NN, int16_t *__restrict__ out) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long first = (long long)(index ? *index : first_candidate) * J;
  const int row_vecs = NN >> 3;
  const bool aligned = ((uintptr_t)out & 15) == 0;
  for (long long r = (long long)blockIdx.x * 8 + warp; r < rows; r += (long long)gridDim.x * 8) {
    const uint32_t slot = ptr[first + r];
    if (aligned) {
      const uint4 *s4 = (const uint4 *)(st.pool + (size_t)slot * NN);
      uint4 *d4 = (uint4 *)(out + (size_t)r * NN);
      for (int v = lane; v < row_vecs; v += 32) d4[v] = s4[v];
    } else {
      for (int n = lane; n < NN; n += 32) out[(size_t)r * NN + n] = st.pool[(size_t)slot * NN + n];
    }
  }
}

// ---------------------------------------------------------------------------------------
// One generation of one candidate per block.
// ---------------------------------------------------------------------------------------
struct GenArgs {
  StoreView st;
  const uint32_t *ptr_in;   // [P][J] parents
  uint32_t *ptr_out;        // [P][J] children
  unsigned int *state;      // {next free slot, half}
  const int16_t *cap;       // [NN]
  const int32_t *k_cap;     // [J] or NULL
  const uint8_t *active;    // [J] or NULL
  const uint32_t *fitness_bits;  // [P] parents' fitness
  const int16_t *cur;       // [J][NN] or NULL
  int P, J, NN, k_max, n_max, num_elite;
  uint32_t thr, gen;
  RngKey key;
  TermParams tp;
  int rows_per_chunk, chunks;   // the dense fitness kernel's chunking, reproduced for identical sums
  float *fitness_out;       // [P]
  int *status;
};

// what the per-node repair decides for the occupant held by this lane of a group (entry = job |
// GPUs << 13 | distributed << 31 in the first have_n <= 16 lanes): the GPUs the job keeps on the node
__device__ __forceinline__ int decide_entries(const GenArgs &a, const Grp &g, uint32_t c, int nn, int tot, int ne,
                                              int cap_n, uint32_t entry, int have_n) {
  const int J = a.J;
  const bool have = g.sub < have_n;
  const int j = (int)(entry & 0x1FFFu);
  int v = have ? (int)((entry >> 13) & 0x7FFu) : 0;
  const bool dist = have && (entry >> 31);
  if (ne >= 2) {
    const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
    int t = J;
    if (dist && v > 0) { t = j - o; if (t < 0) t += J; }
    int best = t;
#pragma unroll
    for (int off = GROUP / 2; off >= 1; off >>= 1) best = min(best, __shfl_xor_sync(g.mask, best, off, GROUP));
    int removed = 0;
    if (dist && v > 0 && t != best) { removed = v; v = 0; }
    tot -= group_sum(g, removed);
  }
  const int excess = tot - cap_n;
  if (excess > 0) {
    const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J);
    int rot = 0x7fffffff;
    if (have) { rot = j - o; if (rot < 0) rot += J; }
    int ahead = 0;                       // GPUs of the occupants that come first in rotated order
    for (int k = 0; k < have_n; ++k) {
      const int rk = __shfl_sync(g.mask, rot, k, GROUP);
      const int vk = __shfl_sync(g.mask, v, k, GROUP);
      if (rk < rot) ahead += vk;
    }
    if (have) v -= min(v, max(excess - ahead, 0));
  }
  return v;
}

// Shared-memory carve-up of the generation kernel (sizes in bytes, 16-byte aligned pieces).
struct GenSmem {
  size_t slot, summ, term, mark, acc, viol, viollist, occ, rowbuf, mut, ovf, mod, cap, rec, total;
};

__host__ __device__ inline GenSmem gen_smem_layout(int J, int NN) {
  GenSmem L;
  size_t off = 0;
#define TAKE(field, bytes) do { L.field = off; off += ((size_t)(bytes) + 15) & ~(size_t)15; } while (0)
  TAKE(slot, (size_t)J * 4);
  TAKE(summ, (size_t)J * 4);
  TAKE(term, (size_t)J * 4);
  TAKE(mark, (size_t)J * 4);
  TAKE(acc, (size_t)NN * 8);
  TAKE(viol, (size_t)NN);
  TAKE(viollist, (size_t)NN * 2);
  TAKE(occ, (size_t)NN * OCC * 4);
  // a row per group of 16 lanes
  TAKE(rowbuf, (size_t)GEN_GROUPS * NN * 2);
  TAKE(mut, (size_t)J * 2);
  TAKE(ovf, (size_t)J * 2);
  TAKE(mod, (size_t)J * 2);
  TAKE(cap, (size_t)NN * 2);
  TAKE(rec, (size_t)GEN_GROUPS * REC_WORDS * 4);
#undef TAKE
  L.total = off;
  return L;
}

// Column value of job j on node nn as the capacity pass must see it: zero when the
// interference pass removes it.
__device__ __forceinline__ int column_value(const GenArgs &a, const uint32_t *s_slot, const uint32_t *s_summ, int j,
                                            int nn, int keep, bool intf, bool &dist) {
  const int v = (int)a.st.pool[(size_t)s_slot[j] * a.NN + nn];
  dist = ((s_summ[j] >> 11) & 0x7FFu) >= 2u;
  if (intf && dist && v > 0 && j != keep) return 0;
  return v;
}

// Repair of a node whose occupants did not fit the block's list: passes over the whole
// column through the row indices.  APPLY false: only marks the rows that will change.
template <bool APPLY, typename MarkFn>
__device__ void repair_column_scan(const GenArgs &a, uint32_t c, const uint32_t *s_slot, const uint32_t *s_summ,
                                   int nn, int tot, int ne, int cap_n, int lane, MarkFn mark) {
  const int J = a.J, NN = a.NN;
  int keep = -1;
  const bool intf = ne >= 2;
  if (intf) {
    const int o = (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
    int best = J;
    for (int j = lane; j < J; j += 32) {
      const int v = (int)a.st.pool[(size_t)s_slot[j] * NN + nn];
      if (v > 0 && ((s_summ[j] >> 11) & 0x7FFu) >= 2u) {
        int t = j - o;
        if (t < 0) t += J;
        best = min(best, t);
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, off));
    keep = o + best;
    if (keep >= J) keep -= J;
    int removed = 0;
    for (int j = lane; j < J; j += 32) {
      const int v = (int)a.st.pool[(size_t)s_slot[j] * NN + nn];
      if (v > 0 && ((s_summ[j] >> 11) & 0x7FFu) >= 2u && j != keep) removed += v;
    }
    tot -= warp_sum(removed);
  }
  int excess = tot - cap_n;
  // the capacity pass walks every job once in rotated order; jobs removed by the interference
  // pass count as empty there and are written (or marked) on the way
  const int o = (excess > 0) ? (int)bounded(draw(a.key, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J) : 0;
  for (int t0 = 0; t0 < J; t0 += 32) {
    const int t = t0 + lane;
    int j = o + t;
    if (j >= J) j -= J;
    int v_old = 0, v_eff = 0;
    if (t < J) {
      bool dist;
      v_old = (int)a.st.pool[(size_t)s_slot[j] * NN + nn];
      v_eff = column_value(a, s_slot, s_summ, j, nn, keep, intf, dist);
    }
    int s = v_eff;                                // inclusive prefix over the 32 jobs
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, s, off);
      if (lane >= off) s += u;
    }
    const int take = (excess > 0) ? min(v_eff, max(excess - (s - v_eff), 0)) : 0;
    const int v_new = v_eff - take;
    if (t < J && v_new != v_old) {
      if (APPLY) a.st.pool[(size_t)s_slot[j] * NN + nn] = (int16_t)v_new;
      else mark(j);
    }
    excess -= __shfl_sync(0xffffffffu, s, 31);
  }
}

template <int PPL>
__global__ void __launch_bounds__(GEN_THREADS, 4) generation_store_kernel(GenArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int J = a.J, NN = a.NN, P = a.P;
  const GenSmem L = gen_smem_layout(J, NN);
  uint32_t *s_slot = (uint32_t *)(smem + L.slot);
  uint32_t *s_summ = (uint32_t *)(smem + L.summ);
  int *s_mark = (int *)(smem + L.mark);            // bit 0: changed by the column pass, bit 1: row is new
  float *s_term = (float *)(smem + L.term);
  // per node: GPUs placed (bits 0..31), distributed jobs on it (32..47), occupants (48..63)
  unsigned long long *s_node = (unsigned long long *)(smem + L.acc);
  uint8_t *s_viol = (uint8_t *)(smem + L.viol);
  uint16_t *s_viollist = (uint16_t *)(smem + L.viollist);
  uint32_t *s_occ = (uint32_t *)(smem + L.occ);
  int16_t *s_rowbuf = (int16_t *)(smem + L.rowbuf);
  uint16_t *s_mut = (uint16_t *)(smem + L.mut), *s_ovf = (uint16_t *)(smem + L.ovf), *s_mod = (uint16_t *)(smem + L.mod);
  int16_t *s_cap = (int16_t *)(smem + L.cap);
  uint32_t *s_rec = (uint32_t *)(smem + L.rec);
  __shared__ int s_nmut, s_novf, s_nmod, s_ncow, s_fail, s_anyscan, s_nviol;
  __shared__ unsigned int s_base_mut, s_base_cow;
  __shared__ int s_parent[2], s_rank4[4];
  __shared__ double s_acc[GEN_WARPS];
  __shared__ int s_acn[GEN_WARPS];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t c = blockIdx.x;
  const bool elite = (int)c < a.num_elite;

  // ---- parents: the candidate of rank c for an elite child, else the better-ranked of two
  // random pairs (rank = candidates ordered before, fitness descending, index ascending) ----
  if (elite) {
    // The candidate of rank c: composite keys (fitness key, then lower index first) are unique,
    // so c + 1 rounds of "largest key below the previous one" find it; one barrier per round.
    __shared__ unsigned long long s_wmax[2][GEN_WARPS];
    unsigned long long prev = ~0ull;
    for (int t = 0; t <= (int)c; ++t) {
      unsigned long long best = 0ull;
      for (int i = tid; i < P; i += GEN_THREADS) {
        const unsigned long long key = ((unsigned long long)order_key(__ldg(a.fitness_bits + i)) << 32) |
                                       (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
        if (key < prev && key > best) best = key;
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, off);
        best = o > best ? o : best;
      }
      if (lane == 0) s_wmax[t & 1][warp] = best;
      __syncthreads();
      best = 0ull;
#pragma unroll
      for (int w = 0; w < GEN_WARPS; ++w) best = s_wmax[t & 1][w] > best ? s_wmax[t & 1][w] : best;
      prev = best;
    }
    if (tid == 0) s_parent[0] = s_parent[1] = (int)(0xFFFFFFFFu - (uint32_t)(prev & 0xFFFFFFFFull));
  } else {
    const u32x4 sel = draw(a.key, 0u, c, a.gen, SLOT_SELECT);
    const int idx[4] = {(int)bounded(sel.x, P), (int)bounded(sel.y, P), (int)bounded(sel.z, P), (int)bounded(sel.w, P)};
    // the ranks of the four drawn candidates, a warp each; the keys are first staged in the (still
    // unused) dynamic shared memory when they fit, so that every key is fetched once
    uint32_t *s_keys = (uint32_t *)smem;
    const bool staged = (size_t)P * 4 <= L.total;
    if (staged) {
      for (int i = tid; i < P; i += GEN_THREADS) s_keys[i] = order_key(__ldg(a.fitness_bits + i));
      __syncthreads();
    }
    if (warp < 4) {
      const int i = idx[warp];
      const uint32_t ki = staged ? s_keys[i] : order_key(a.fitness_bits[i]);
      int rk = 0;
      for (int o = lane; o < P; o += 32) {
        const uint32_t ko = staged ? s_keys[o] : order_key(__ldg(a.fitness_bits + o));
        rk += (ko > ki || (ko == ki && o < i)) ? 1 : 0;
      }
      rk = warp_sum(rk);
      if (lane == 0) s_rank4[warp] = rk;
    }
    __syncthreads();
    if (tid == 0) {
      s_parent[0] = s_rank4[0] <= s_rank4[1] ? idx[0] : idx[1];
      s_parent[1] = s_rank4[2] <= s_rank4[3] ? idx[2] : idx[3];
    }
  }
  __syncthreads();

  for (int i = tid; i < NN; i += GEN_THREADS) {
    s_node[i] = 0ull; s_viol[i] = 0;
    s_cap[i] = (int16_t)max((int)a.cap[i], 0);
  }
  for (int i = tid; i < J; i += GEN_THREADS) s_mark[i] = 0;
  if (tid == 0) { s_nmut = 0; s_novf = 0; s_nmod = 0; s_ncow = 0; s_fail = 0; s_anyscan = 0; s_nviol = 0; }
  __syncthreads();

  // occupant (job j holds g GPUs on node n) into the node's totals and list
  auto add_occupant = [&](int j, int n, int g, bool dist) {
    uint32_t *w = (uint32_t *)&s_node[n];   // two 32-bit adds: the low word's answer is not needed
    atomicAdd(&w[0], (uint32_t)g);
    const int k = (int)(atomicAdd(&w[1], (dist ? 1u : 0u) | (1u << 16)) >> 16);
    if (k < OCC) s_occ[n * OCC + k] = (uint32_t)j | ((uint32_t)g << 13) | (dist ? 0x80000000u : 0u);
  };

  // the occupants in this lane's pieces of a row
  auto add_row_occupants = [&](const Grp &g, int j, const RowPieces<PPL> &p, bool dist) {
#pragma unroll
    for (int q = 0; q < PPL; ++q) {
      uint32_t m = p.mask[q];
      while (m) {
        const int h = __ffs(m) - 1;
        m &= m - 1;
        add_occupant(j, 8 * (g.sub * PPL + q) + h, piece_entry(p.x[q], h), dist);
      }
    }
  };

  // ---- rows, one thread each: the child row is the chosen parent's row -----------------------
  // First every row's draws (which parent; perturbed or not).  The count of perturbed rows is
  // then known and the block takes its slots - those plus a reserve for the rows the column
  // pass will change - with one atomic whose answer is not needed before the rows are done.
  uint32_t secbits = 0, mutbits = 0;   // bit r: this thread's r-th row (j = tid + r * GEN_THREADS)
  if (!elite) {
    int r = 0;
    for (int j = tid; j < J; j += GEN_THREADS, ++r) {
      if (a.active && !a.active[j]) continue;
      if (draw(a.key, (uint32_t)j, c, a.gen, SLOT_XOVER).x >> 31) secbits |= 1u << r;
      if (draw(a.key, (uint32_t)j, c, a.gen, SLOT_MUTATE).x < a.thr) {
        mutbits |= 1u << r;
        s_mut[atomicAdd(&s_nmut, 1)] = (uint16_t)j;
      }
    }
  }
  __syncthreads();
  unsigned int base_reg = 0;
  if (tid == 0) base_reg = atomicAdd(a.state, (unsigned int)(s_nmut + COW_RESERVE));

  // Then RB rows per thread at a time, so that their dependent loads (index -> record) travel
  // together.
  const uint32_t *pin_a = a.ptr_in + (size_t)s_parent[0] * J, *pin_b = a.ptr_in + (size_t)s_parent[1] * J;
  constexpr int RB = 4;
  for (int jb = tid, rb = 0; jb < J; jb += GEN_THREADS * RB, rb += RB) {
    uint32_t slot[RB];
    bool on[RB], mut[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int j = jb + r * GEN_THREADS;
      on[r] = j < J && (!a.active || a.active[j]);
      mut[r] = ((mutbits >> (rb + r)) & 1u) != 0u;
      slot[r] = on[r] ? (((secbits >> (rb + r)) & 1u) ? pin_b[j] : pin_a[j]) : a.st.zero_slot;
    }
    uint32_t rec[RB][REC_WORDS];
#pragma unroll
    for (int r = 0; r < RB; ++r) load_record(rec[r], a.st.rec + (size_t)slot[r] * REC_WORDS);
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int j = jb + r * GEN_THREADS;
      if (j >= J) continue;
      const uint32_t w = on[r] ? rec[r][REC_SUMM] : 0u;
      s_slot[j] = slot[r];
      s_summ[j] = w;
      if (!on[r] || mut[r]) continue;
      s_term[j] = __uint_as_float(rec[r][REC_TERM]);
      if (rec[r][0] == REC_OVERFLOW) {
        s_ovf[atomicAdd(&s_novf, 1)] = (uint16_t)j;
        continue;
      }
      const bool dist = ((w >> 11) & 0x7FFu) >= 2u;
#pragma unroll
      for (int k = 0; k < REC_ENTRIES; ++k) {
        const uint32_t e = rec[r][k];
        if (e) add_occupant(j, (int)(e & 0xFFFu), (int)((e >> 12) & 0x7FFu), dist);
      }
    }
  }
  if (tid == 0) {
    const unsigned long long limit = (unsigned long long)(a.state[1] + 1u) * a.st.half_cap;
    s_base_mut = base_reg;
    s_base_cow = base_reg + (unsigned int)s_nmut;
    if ((unsigned long long)base_reg + (unsigned long long)(s_nmut + COW_RESERVE) > limit) {
      s_fail = 1;
      atomicExch(a.status, SCHED_ERR_TOO_LARGE);
    }
  }
  __syncthreads();

  // ---- perturbed rows, one group of 16 lanes each: new row in a fresh slot --------------------
  const Grp g = make_group(lane, NN);
  const int grp = tid >> 4;
  int16_t *row = s_rowbuf + (size_t)grp * NN;   // this group's row
  uint32_t *recw = s_rec + grp * REC_WORDS;
  if (!s_fail) {
    for (int i = grp; i < s_nmut; i += GEN_GROUPS) {
      const int j = (int)s_mut[i];
      const uint32_t old = s_slot[j], w = s_summ[j];
      load_row<false>(g, row, a.st.pool + (size_t)old * NN);
      const CurPieces<PPL> cur = cur_pieces<PPL>(g, a.cur ? a.cur + (size_t)j * NN : nullptr);
      const int kc_in = a.k_cap ? a.k_cap[j] : a.k_max;
      __syncwarp(g.mask);
      const int rN = (int)((w >> 11) & 0x7FFu);
      const u32x4 mw = draw(a.key, (uint32_t)j, c, a.gen, SLOT_MUTATE);
      const uint32_t op = bounded(mw.y, 3u);
      if (op == 0u) {
        const int n = (int)bounded(mw.w, (uint32_t)NN);
        if (g.sub == 0) row[n] = (int16_t)min((int)row[n] + 1, (int)s_cap[n]);
      } else if (rN > 0) {
        const int ns = nth_occupied_row<PPL>(g, row, bounded(mw.z, (uint32_t)rN));
        if (op == 1u) {
          if (g.sub == 0) row[ns] = (int16_t)(row[ns] - 1);
        } else {
          const int nd = (int)bounded(mw.w, (uint32_t)NN);
          if (nd != ns && g.sub == 0) {
            row[nd] = (int16_t)min((int)row[nd] + (int)row[ns], (int)s_cap[nd]);
            row[ns] = 0;
          }
        }
      }
      __syncwarp(g.mask);
      int K, N, nd;
      RowPieces<PPL> p = summarise_row<PPL>(g, row, cur, K, N, nd, recw);
      // per-row caps: replicas above the job's cap leave from the highest node index down, then
      // occupied nodes beyond n_max are cleared from the highest index down
      const int kc = max(0, min(kc_in, a.k_max));
      if (K > kc || N > a.n_max) {
        if (g.sub == 0) {
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
        }
        __syncwarp(g.mask);
        p = summarise_row<PPL>(g, row, cur, K, N, nd, recw);
      }
      const uint32_t slot = s_base_mut + (uint32_t)i;
      // the row's speedup (and penalty factor) are asked for now and used at the end of the step
      float x_sp = 0.f, x_pen = 1.f;
      if (g.sub == 0) {
        x_sp = __ldg(a.tp.table + fitness_table_index(a.tp, j, K, N));
        if (a.tp.pen && nd != 0) x_pen = __ldg(a.tp.pen + j);
      }
      store_row(g, a.st.pool + (size_t)slot * NN, row);
      const uint32_t word = pack_summary(K, N, nd);
      if (g.sub == 0) {
        recw[REC_SUMM] = word;
        s_slot[j] = slot;
        s_summ[j] = word;
        s_mark[j] = 2;
      }
      add_row_occupants(g, j, p, N >= 2);
      if (g.sub == 0) {
        const float term = fitness_term_with(a.tp, x_sp, x_pen, nd != 0);
        s_term[j] = term;
        recw[REC_TERM] = __float_as_uint(term);
      }
      __syncwarp(g.mask);
      if (g.sub < REC_WORDS) a.st.rec[(size_t)slot * REC_WORDS + g.sub] = recw[g.sub];
      __syncwarp(g.mask);
    }
  }
  // rows with more occupied nodes than a record holds: occupants from the row itself
  for (int i = grp; i < s_novf; i += GEN_GROUPS) {
    const int j = (int)s_ovf[i];
    load_row<false>(g, row, a.st.pool + (size_t)s_slot[j] * NN);
    __syncwarp(g.mask);
    const RowPieces<PPL> p = row_pieces<PPL>(g, row);
    add_row_occupants(g, j, p, ((s_summ[j] >> 11) & 0x7FFu) >= 2u);
    __syncwarp(g.mask);
  }
  __syncthreads();

  // ---- column pass, decisions: which occupants of the violating nodes change ------------------
  auto mark_row = [&](int j) {
    if ((atomicOr(&s_mark[j], 1) & 1) == 0) {
      s_mod[atomicAdd(&s_nmod, 1)] = (uint16_t)j;
      for (int b = 0; b * 64 < NN; ++b) {   // the row and its counterpart will be read next
        prefetch_l2(a.st.pool + (size_t)s_slot[j] * NN + b * 64);
        if (a.cur) prefetch_l2(a.cur + (size_t)j * NN + b * 64);
      }
    }
  };
  // nodes that hold two distributed jobs or more GPUs than they have
  for (int n = tid; n < NN; n += GEN_THREADS) {
    const unsigned long long acc = s_node[n];
    if ((int)((acc >> 32) & 0xFFFFu) >= 2 || (int)(uint32_t)acc > (int)s_cap[n]) s_viollist[atomicAdd(&s_nviol, 1)] = (uint16_t)n;
  }
  __syncthreads();
  const int nviol = s_nviol;
  for (int i = grp; i < nviol; i += GEN_GROUPS) {   // a group of 16 lanes per listed node
    const int nn = (int)s_viollist[i];
    const unsigned long long acc = s_node[nn];
    const int have_n = (int)(acc >> 48);
    if (have_n > OCC) {   // more occupants than the list holds: left to the column scan below
      if (g.sub == 0) { s_viol[nn] = 2; s_anyscan = 1; }
      continue;
    }
    const uint32_t entry = (g.sub < have_n) ? s_occ[nn * OCC + g.sub] : 0u;
    const int v_new = decide_entries(a, g, c, nn, (int)(uint32_t)acc, (int)((acc >> 32) & 0xFFFFu), (int)s_cap[nn], entry, have_n);
    if (g.sub < have_n) {
      // the entry now carries the decision: GPUs kept, and bit 24 when that is a change
      const bool changed = v_new != (int)((entry >> 13) & 0x7FFu);
      s_occ[nn * OCC + g.sub] = (entry & 0x80001FFFu) | ((uint32_t)v_new << 13) | (changed ? (1u << 24) : 0u);
      if (changed) mark_row((int)(entry & 0x1FFFu));
    }
    if (g.sub == 0) s_viol[nn] = 1;
    __syncwarp(g.mask);
  }
  __syncthreads();
  if (s_anyscan) {
    for (int i = warp; i < nviol; i += GEN_WARPS) {   // a warp per node whose column must be scanned
      const int nn = (int)s_viollist[i];
      if (s_viol[nn] != 2) continue;
      const unsigned long long acc = s_node[nn];
      repair_column_scan<false>(a, c, s_slot, s_summ, nn, (int)(uint32_t)acc, (int)((acc >> 32) & 0xFFFFu), (int)s_cap[nn],
                                lane, mark_row);
    }
    __syncthreads();
  }

  // ---- rows the column pass changes -----------------------------------------------------------
  // Usual case (every violating node's occupants were listed): one group per changed row takes
  // the row, applies the decisions of its nodes, and writes it with its record - to a slot of
  // its own unless the row is new in this generation already.
  const int nmod = s_nmod;
  if (!s_anyscan) {
    if (nmod > COW_RESERVE) {   // more than the reserve: a run of slots of their own
      if (tid == 0) {
        const unsigned int base = atomicAdd(a.state, (unsigned int)nmod);
        const unsigned long long limit = (unsigned long long)(a.state[1] + 1u) * a.st.half_cap;
        s_base_cow = base;
        if ((unsigned long long)base + (unsigned long long)nmod > limit) { s_fail = 1; atomicExch(a.status, SCHED_ERR_TOO_LARGE); }
      }
      __syncthreads();
    }
    if (!s_fail) {
      for (int i = grp; i < nmod; i += GEN_GROUPS) {
        const int j = (int)s_mod[i];
        const bool own = (s_mark[j] & 2) != 0;
        const uint32_t src = s_slot[j];
        load_row<true>(g, row, a.st.pool + (size_t)src * NN);   // may have been written in this kernel
        const CurPieces<PPL> cur = cur_pieces<PPL>(g, a.cur ? a.cur + (size_t)j * NN : nullptr);
        __syncwarp(g.mask);
        {
          const RowPieces<PPL> p = row_pieces<PPL>(g, row);
#pragma unroll
          for (int q = 0; q < PPL; ++q) {
            uint32_t m = p.mask[q];
            while (m) {
              const int n = 8 * (g.sub * PPL + q) + __ffs(m) - 1;
              m &= m - 1;
              if (s_viol[n] != 1) continue;
              const int cnt = (int)(s_node[n] >> 48);
              for (int k = 0; k < cnt; ++k) {
                const uint32_t e = s_occ[n * OCC + k];
                if ((int)(e & 0x1FFFu) == j) {
                  if ((e >> 24) & 1u) row[n] = (int16_t)((e >> 13) & 0x7FFu);
                  break;
                }
              }
            }
          }
        }
        __syncwarp(g.mask);
        int K, N, nd;
        summarise_row<PPL>(g, row, cur, K, N, nd, recw);
        const uint32_t dst = own ? src : s_base_cow + (uint32_t)i;
        float x_sp = 0.f, x_pen = 1.f;
        if (g.sub == 0) {
          x_sp = __ldg(a.tp.table + fitness_table_index(a.tp, j, K, N));
          if (a.tp.pen && nd != 0) x_pen = __ldg(a.tp.pen + j);
        }
        store_row(g, a.st.pool + (size_t)dst * NN, row);
        const uint32_t word = pack_summary(K, N, nd);
        if (g.sub == 0) {
          const float term = fitness_term_with(a.tp, x_sp, x_pen, nd != 0);
          recw[REC_SUMM] = word;
          recw[REC_TERM] = __float_as_uint(term);
          s_slot[j] = dst;
          s_summ[j] = word;
          s_term[j] = term;
        }
        __syncwarp(g.mask);
        if (g.sub < REC_WORDS) a.st.rec[(size_t)dst * REC_WORDS + g.sub] = recw[g.sub];
        __syncwarp(g.mask);
      }
    }
    __syncthreads();
  } else {
    // Some node had more occupants than the block lists: its column is scanned through the
    // row indices, so the rows are first copied, then written in place, then summarised.
      for (int i = tid; i < nmod; i += GEN_THREADS) {
      const int j = (int)s_mod[i];
      const bool own = (s_mark[j] & 2) != 0;
      s_ovf[i] = own ? (uint16_t)0xFFFFu : (uint16_t)atomicAdd(&s_ncow, 1);
    }
    __syncthreads();
    if (tid == 0 && s_ncow > COW_RESERVE) {   // more than the reserve: a run of slots of their own
      const unsigned int base = atomicAdd(a.state, (unsigned int)s_ncow);
      const unsigned long long limit = (unsigned long long)(a.state[1] + 1u) * a.st.half_cap;
      s_base_cow = base;
      if ((unsigned long long)base + (unsigned long long)s_ncow > limit) { s_fail = 1; atomicExch(a.status, SCHED_ERR_TOO_LARGE); }
    }
    __syncthreads();
    if (!s_fail) {
      for (int i = grp; i < nmod; i += GEN_GROUPS) {
        const uint32_t k = s_ovf[i];
        if (k == 0xFFFFu) continue;
        const int j = (int)s_mod[i];
        const uint32_t slot = s_base_cow + k;
        load_row<true>(g, row, a.st.pool + (size_t)s_slot[j] * NN);
        __syncwarp(g.mask);
        store_row(g, a.st.pool + (size_t)slot * NN, row);
        __syncwarp(g.mask);
        if (g.sub == 0) s_slot[j] = slot;
      }
    }
    __syncthreads();

    // column pass, writes
    if (!s_fail && nmod > 0) {
      for (int i = tid; i < NN * OCC; i += GEN_THREADS) {
        const int n = i / OCC, k = i - n * OCC;
        if (s_viol[n] != 1 || k >= (int)(s_node[n] >> 48)) continue;
        const uint32_t entry = s_occ[i];
        if ((entry >> 24) & 1u)
          a.st.pool[(size_t)s_slot[entry & 0x1FFFu] * NN + n] = (int16_t)((entry >> 13) & 0x7FFu);
      }
      for (int nn = warp; nn < NN; nn += GEN_WARPS) {
        if (s_viol[nn] != 2) continue;
        repair_column_scan<true>(a, c, s_slot, s_summ, nn, (int)(uint32_t)s_node[nn], (int)((s_node[nn] >> 32) & 0xFFFFu),
                                 (int)s_cap[nn], lane, [](int) {});
      }
    }
    __syncthreads();

    // changed rows: summary and record from the row as it now stands
    if (!s_fail) {
      for (int i = grp; i < nmod; i += GEN_GROUPS) {
        const int j = (int)s_mod[i];
        const uint32_t slot = s_slot[j];
        load_row<true>(g, row, a.st.pool + (size_t)slot * NN);   // written in this kernel: read through to L2
        const CurPieces<PPL> cur = cur_pieces<PPL>(g, a.cur ? a.cur + (size_t)j * NN : nullptr);
        __syncwarp(g.mask);
        int K, N, nd;
        summarise_row<PPL>(g, row, cur, K, N, nd, recw);
        const uint32_t word = pack_summary(K, N, nd);
        if (g.sub == 0) {
          const float term = fitness_term(a.tp, j, K, N, nd != 0);
          recw[REC_SUMM] = word;
          recw[REC_TERM] = __float_as_uint(term);
          s_summ[j] = word;
          s_term[j] = term;
        }
        __syncwarp(g.mask);
        if (g.sub < REC_WORDS) a.st.rec[(size_t)slot * REC_WORDS + g.sub] = recw[g.sub];
        __syncwarp(g.mask);
      }
    }
    __syncthreads();
  }

  // ---- children's indices out, fitness of the candidate (Eq. 14) from the rows' terms ----------
  uint32_t *pout = a.ptr_out + (size_t)c * J;
  for (int j = tid; j < J; j += GEN_THREADS) pout[j] = s_slot[j];
  // sums in the order of the dense fitness kernel: per chunk of rows, thread t adds rows t,
  // t + 256, ... in double, a shuffle tree per warp, the warps in index order; then the chunks
  // in index order
  double ts = 0.0, ns = 0.0;
  for (int ch = 0; ch < a.chunks; ++ch) {
    const int j0 = ch * a.rows_per_chunk, j1 = min(J, j0 + a.rows_per_chunk);
    double acc = 0.0;
    int cnt = 0;
    for (int j = j0 + tid; j < j1; j += GEN_THREADS) {
      if (!a.tp.active || a.tp.active[j]) { acc += (double)s_term[j]; cnt += 1; }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      acc += __shfl_xor_sync(0xffffffffu, acc, off);
      cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    }
    if (lane == 0) { s_acc[warp] = acc; s_acn[warp] = cnt; }
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      int n = 0;
      for (int w = 0; w < GEN_WARPS; ++w) { t += s_acc[w]; n += s_acn[w]; }
      ts += t;
      ns += (double)n;
    }
    __syncthreads();
  }
  if (tid == 0) a.fitness_out[c] = fitness_finalise(a.tp.mode, a.tp.p, ts, ns);
}

// pieces per lane of a row's group: 1, 2 or 4 (a lane's pieces beyond the row's end are empty)
int store_pieces_per_lane(int num_nodes) {
  const int need = ((num_nodes >> 3) + GROUP - 1) / GROUP;
  return need <= 1 ? 1 : need == 2 ? 2 : 4;
}

StoreView store_view(const sched_ctx *ctx) {
  StoreView v;
  v.pool = ctx->rs_pool; v.rec = ctx->rs_rec;
  v.half_cap = ctx->rs_half_cap;
  v.zero_slot = (uint32_t)(2 * ctx->rs_half_cap);
  return v;
}

}  // namespace

// The row store serves rounds whose candidates span several row batches of the dense
// kernels (J > 256; smaller problems run a generation as one dense kernel already), with
// rows of whole 16-byte vectors and sizes that fit the packed fields.
bool rowstore_eligible(const sched_ctx *ctx, const int16_t *) {
  const sched_config &c = ctx->cfg;
  if (c.num_jobs <= 256 || c.num_jobs > STORE_MAX_JOBS) return false;
  if (c.num_nodes % 8 != 0 || c.num_nodes > 512 || ctx->cap_max > 2047) return false;
  if (c.k_max > 2047 || c.n_max > 2047) return false;
  const unsigned long long rows = (unsigned long long)c.population * c.num_jobs;
  const unsigned long long worst = store_worst_case(c.population, c.num_jobs);
  if (2ull * rows + 17ull * worst >= (1ull << 32)) return false;   // slot indices are 32-bit
  if (gen_smem_layout(c.num_jobs, c.num_nodes).total > 200 * 1024) return false;
  // a half holds the population plus at least two generations' worst case; beyond 8 GiB of pool
  // the dense path runs
  const unsigned long long row_bytes = (unsigned long long)c.num_nodes * 2 + REC_WORDS * 4;
  return 2ull * (rows + 2ull * worst) * row_bytes <= (8ull << 30);
}

int rowstore_ensure(sched_ctx *ctx) {
  if (ctx->rs_ready) return SCHED_OK;
  const sched_config &c = ctx->cfg;
  const unsigned long long rows = (unsigned long long)c.population * c.num_jobs;
  const unsigned long long row_bytes = (unsigned long long)c.num_nodes * 2 + REC_WORDS * 4;
  // half = the population + (gens between checks + slack) generations' worst case; shrink until
  // the pool fits 8 GiB
  int check = 4, slack = 4;
  const unsigned long long worst = store_worst_case(c.population, c.num_jobs);
  while (2ull * (rows + (check + slack) * worst) * row_bytes > (8ull << 30) && (check > 1 || slack > 1)) {
    if (slack > 1) --slack; else --check;
  }
  ctx->rs_check_every = check;
  ctx->rs_half_cap = (size_t)(rows + (check + slack) * worst);
  const size_t slots = 2 * ctx->rs_half_cap + 1;
  cudaError_t e = cudaMalloc((void **)&ctx->rs_pool, slots * c.num_nodes * sizeof(int16_t));
  if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->rs_rec, slots * REC_WORDS * sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->rs_ptr, 2 * (size_t)rows * sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->rs_state, 4 * sizeof(unsigned int));
  if (e == cudaSuccess) {
    const size_t smem = gen_smem_layout(c.num_jobs, c.num_nodes).total;
    if (smem > 48 * 1024)
    for (int k = 0; k < 3 && e == cudaSuccess; ++k)
      e = cudaFuncSetAttribute(k == 0 ? generation_store_kernel<1> : k == 1 ? generation_store_kernel<2> : generation_store_kernel<4>,
                               cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  }
  if (e != cudaSuccess) {
    set_error(ctx, "row store allocation failed: %s", cudaGetErrorString(e));
    for (void *p : {(void *)ctx->rs_pool, (void *)ctx->rs_rec, (void *)ctx->rs_ptr, (void *)ctx->rs_state})
      if (p) cudaFree(p);
    ctx->rs_pool = nullptr; ctx->rs_rec = nullptr; ctx->rs_ptr = nullptr; ctx->rs_state = nullptr;
    cudaGetLastError();
    return SCHED_ERR_CUDA;
  }
  ctx->scratch_epoch++;
  ctx->rs_ready = true;
  return SCHED_OK;
}

int rowstore_build(sched_ctx *ctx, const uint8_t *d_active, const int16_t *d_cur, const float *d_pen) {
  const sched_config &c = ctx->cfg;
  BuildArgs a;
  a.st = store_view(ctx);
  a.ptr = ctx->rs_ptr;
  a.state = ctx->rs_state;
  a.active = d_active; a.cur = d_cur;
  a.tp.table = ctx->d_tab_speedup; a.tp.pen = d_pen; a.tp.active = d_active;
  a.tp.k_max = c.k_max; a.tp.n_max = c.n_max; a.tp.mode = fitness_mode(c.p); a.tp.p = c.p;
  a.tp.floor_ = c.speedup_floor;
  a.P = c.population; a.J = c.num_jobs; a.NN = c.num_nodes;
  {
    TimedLaunch tl_(ctx, KK_STORE_BUILD);
    const int ppl = store_pieces_per_lane(c.num_nodes);
    if (ppl == 1) rowstore_build_kernel<1><<<ctx->num_sms * 8, 256, 0, ctx->stream>>>(a);
    else if (ppl == 2) rowstore_build_kernel<2><<<ctx->num_sms * 8, 256, 0, ctx->stream>>>(a);
    else rowstore_build_kernel<4><<<ctx->num_sms * 8, 256, 0, ctx->stream>>>(a);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

int rowstore_compact(sched_ctx *ctx, int parity, int state_phase) {
  const sched_config &c = ctx->cfg;
  CompactArgs a;
  a.st = store_view(ctx);
  a.ptr = ctx->rs_ptr + (size_t)parity * c.population * c.num_jobs;
  a.state_in = ctx->rs_state + 2 * state_phase;
  a.state_out = ctx->rs_state + 2 * (state_phase ^ 1);
  a.P = c.population; a.J = c.num_jobs; a.NN = c.num_nodes;
  a.gens_ahead = ctx->rs_check_every;
  {
    TimedLaunch tl_(ctx, KK_STORE_COMPACT);
    rowstore_compact_kernel<<<ctx->num_sms * 8, 256, 0, ctx->stream>>>(a);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

int rowstore_gather(sched_ctx *ctx, const uint32_t *d_ptr, int first_candidate, int count, const int32_t *d_index,
                    int16_t *d_out) {
  const sched_config &c = ctx->cfg;
  const long long rows = (long long)count * c.num_jobs;
  if (rows == 0) return SCHED_OK;
  const long long want = (rows + 7) / 8;
  const int blocks = (int)(want < (long long)ctx->num_sms * 8 ? want : (long long)ctx->num_sms * 8);
  {
    TimedLaunch tl_(ctx, KK_STORE_GATHER);
    rowstore_gather_kernel<<<blocks, 256, 0, ctx->stream>>>(store_view(ctx), d_ptr, first_candidate, rows, d_index,
                                                           c.num_jobs, c.num_nodes, d_out);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}

int rowstore_generation(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, const int16_t *d_cur,
                        const float *d_pen, const float *d_fitness_in, float *d_fitness_out, int parity,
                        int state_phase, uint32_t generation) {
  const sched_config &c = ctx->cfg;
  const size_t rows = (size_t)c.population * c.num_jobs;
  GenArgs a;
  a.st = store_view(ctx);
  a.ptr_in = ctx->rs_ptr + (size_t)parity * rows;
  a.ptr_out = ctx->rs_ptr + (size_t)(parity ^ 1) * rows;
  a.state = ctx->rs_state + 2 * state_phase;
  a.cap = ctx->d_cap; a.k_cap = d_k_cap; a.active = d_active;
  a.fitness_bits = (const uint32_t *)d_fitness_in;
  a.cur = d_cur;
  a.P = c.population; a.J = c.num_jobs; a.NN = c.num_nodes;
  a.k_max = c.k_max; a.n_max = c.n_max; a.num_elite = c.num_elite;
  a.thr = c.thr_mutate; a.gen = generation;
  a.key = make_key(c.seed, ctx->d_round);
  a.tp.table = ctx->d_tab_speedup; a.tp.pen = d_pen; a.tp.active = d_active;
  a.tp.k_max = c.k_max; a.tp.n_max = c.n_max; a.tp.mode = fitness_mode(c.p); a.tp.p = c.p;
  a.tp.floor_ = c.speedup_floor;
  fitness_chunking(ctx, c.population, a.rows_per_chunk, a.chunks);
  a.fitness_out = d_fitness_out;
  a.status = ctx->d_status;
  const size_t smem = gen_smem_layout(c.num_jobs, c.num_nodes).total;
  {
    TimedLaunch tl_(ctx, KK_GENSTORE);
    const int ppl = store_pieces_per_lane(c.num_nodes);
    if (ppl == 1) generation_store_kernel<1><<<c.population, GEN_THREADS, smem, ctx->stream>>>(a);
    else if (ppl == 2) generation_store_kernel<2><<<c.population, GEN_THREADS, smem, ctx->stream>>>(a);
    else generation_store_kernel<4><<<c.population, GEN_THREADS, smem, ctx->stream>>>(a);
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}
