// Row store: the population of a running scheduling round kept as shared rows (Sec. 4.3).
//
// A generation copies almost every child row verbatim from one of two parents; only the
// perturbed rows and the few rows the repair touches are new.  Here every distinct row is
// stored once and a candidate is an array of row indices ("slots").  A stored row is a
// 32-byte record: up to six occupied nodes (node | GPUs << 12, ascending node order), the
// row's term of the fitness sum (a stored row always serves the same job, so the term is
// fixed for the round) and its summary (K, N, entries that differ from the current
// allocation).  A row with at most six occupied nodes lives in its record alone; only a row
// with more (first word 0xFFFFFFFF) also has its contents in the pool.  A generation reads
// 36 bytes per unchanged row and writes 4.  New rows are appended (copy on write); when a
// half of the slot space runs low the live rows are copied to the other half.
//
// One block evolves one candidate per generation: parent selection, row-wise crossover,
// perturbation, per-row caps, interference and capacity repair, and the candidate's fitness.
// Rows that change are edited as lists of occupied nodes, one thread per row.  The initial
// population of a round is made by the same kernel from the current allocation's rows.
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
  uint32_t zero_slot;       // also the largest valid slot
  int *status;              // the context's status word (checked build)
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

// One 32-byte record with a single request, read from L2: records may have been written by the
// previous kernel, which can still be running when this one starts (programmatic dependent
// launch), so a line cached in this SM's L1 before that write must not serve the load.
__device__ __forceinline__ void load_record(uint32_t (&r)[REC_WORDS], const uint32_t *p) {
  asm volatile("ld.global.cg.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "l"(p) : "memory");
}

__device__ __forceinline__ uint32_t pack_summary(int K, int N, int ndiff) {
  return (uint32_t)K | ((uint32_t)N << 11) | ((uint32_t)ndiff << 22);
}

// ---------------------------------------------------------------------------------------
// Start of a round on the store: the current allocation's rows become slots 0 .. 2J - 1.
// Slot j holds job j's row as an unperturbed child of the initial population has it (entries
// forced into [0, node size], then the row caps); slot J + j holds it before the row caps, which
// is what a perturbed child starts from.  The initial population itself is then made by the
// generation kernel with this single "parent".
// ---------------------------------------------------------------------------------------
struct BuildCurArgs {
  StoreView st;
  uint32_t *ptr;            // [J] the parent's row indices
  unsigned int *state;      // {next free slot, half}
  const uint8_t *active;
  const int16_t *seed;      // [J][NN] current allocation the population starts from, or NULL (empty cluster)
  const int16_t *cur;       // [J][NN] current allocation the summaries compare with, or NULL
  const int16_t *cap;
  const int32_t *k_cap;
  TermParams tp;
  int J, NN, k_max, n_max;
};

template <int PPL>
__global__ void __launch_bounds__(256) rowstore_build_cur_kernel(BuildCurArgs a) {
  __shared__ __align__(16) int16_t s_row[16][512];
  __shared__ uint32_t s_rec[16][REC_WORDS];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 4;
  const Grp g = make_group(lane, a.NN);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    a.state[0] = 2u * (unsigned int)a.J;
    a.state[1] = 0u;
  }
  if (blockIdx.x == 0) {    // the empty row: contents and record all zero
    for (int n = threadIdx.x; n < a.NN; n += blockDim.x) a.st.pool[(size_t)a.st.zero_slot * a.NN + n] = 0;
    if (threadIdx.x < REC_WORDS) a.st.rec[(size_t)a.st.zero_slot * REC_WORDS + threadIdx.x] = 0u;
  }
  for (int j = blockIdx.x * 16 + grp; j < a.J; j += gridDim.x * 16) {
    const bool on = !a.active || a.active[j];
    if (g.sub == 0) a.ptr[j] = on ? (uint32_t)j : a.st.zero_slot;
    if (!on) continue;                                  // (uniform within the group)
    for (int v = g.sub; v < g.row_vecs; v += GROUP) {
      uint4 x = make_uint4(0u, 0u, 0u, 0u);
      if (a.seed) {
        x = load_piece<false>(a.seed + (size_t)j * a.NN, v);
        const uint4 cp = *((const uint4 *)a.cap + v);
        x.x = __vimin_s16x2_relu(x.x, __vimax_s16x2_relu(cp.x, 0u));
        x.y = __vimin_s16x2_relu(x.y, __vimax_s16x2_relu(cp.y, 0u));
        x.z = __vimin_s16x2_relu(x.z, __vimax_s16x2_relu(cp.z, 0u));
        x.w = __vimin_s16x2_relu(x.w, __vimax_s16x2_relu(cp.w, 0u));
      }
      ((uint4 *)s_row[grp])[v] = x;
    }
    const CurPieces<PPL> cur = cur_pieces<PPL>(g, a.cur ? a.cur + (size_t)j * a.NN : nullptr);
    __syncwarp(g.mask);
    const int kc = max(0, min(a.k_cap ? a.k_cap[j] : a.k_max, a.k_max));
    for (int pass = 0; pass < 2; ++pass) {              // before the row caps (slot J + j), after them (slot j)
      int K, N, nd;
      summarise_row<PPL>(g, s_row[grp], cur, K, N, nd, s_rec[grp]);
      const size_t slot = pass == 0 ? (size_t)a.J + j : (size_t)j;
      if (g.sub == 0) {
        // (before the row caps K may exceed its field: the row is only a perturbation's source then,
        // and that path adds the entries up itself)
        s_rec[grp][REC_SUMM] = pack_summary(min(K, 2047), N, nd);
        s_rec[grp][REC_TERM] = __float_as_uint(fitness_term(a.tp, j, K, N, nd != 0));
      }
      if (N > REC_ENTRIES) store_row(g, a.st.pool + slot * a.NN, s_row[grp]);
      __syncwarp(g.mask);
      if (g.sub < REC_WORDS) a.st.rec[slot * REC_WORDS + g.sub] = s_rec[grp][g.sub];
      __syncwarp(g.mask);
      if (pass == 0 && (K > kc || N > a.n_max)) {
        // replicas above the job's cap leave from the highest node index down, then occupied nodes
        // beyond n_max are cleared from the highest index down
        if (g.sub == 0) {
          int16_t *row = s_row[grp];
          int excess = K - kc;
          for (int n = a.NN - 1; n >= 0 && excess > 0; --n) {
            const int take = min((int)row[n], excess);
            row[n] = (int16_t)(row[n] - take);
            excess -= take;
          }
          int occ = 0;
          for (int n = 0; n < a.NN; ++n) {
            if (row[n] > 0) {
              ++occ;
              if (occ > a.n_max) row[n] = 0;
            }
          }
        }
        __syncwarp(g.mask);
      }
    }
  }
}

// most slots one generation can take: every row new (a row gets at most one slot per generation:
// perturbed, or copied when the column pass first changes it), plus every block's reserve
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
  unsigned int *moves;      // times the rows have moved (since the context was made)
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
    atomicAdd(a.moves, 1u);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row_vecs = a.NN >> 3;
  for (unsigned long long r = (unsigned long long)blockIdx.x * 8 + warp; r < rows; r += (unsigned long long)gridDim.x * 8) {
    const uint32_t slot = a.ptr[r];
    if (slot == a.st.zero_slot) continue;
    const size_t dst = (size_t)(base + r);
    if (!sched_index_ok(a.st.status, slot < a.st.zero_slot && dst < a.st.zero_slot, SCHED_CHK_SLOT)) continue;
    const uint32_t w = (lane < REC_WORDS) ? a.st.rec[(size_t)slot * REC_WORDS + lane] : 0u;
    if (__shfl_sync(0xffffffffu, w, 0) == REC_OVERFLOW) {   // the record does not hold the row: its contents move too
      const uint4 *s4 = (const uint4 *)(a.st.pool + (size_t)slot * a.NN);
      uint4 *d4 = (uint4 *)(a.st.pool + dst * a.NN);
      for (int v = lane; v < row_vecs; v += 32) d4[v] = s4[v];
    }
    if (lane < REC_WORDS) a.st.rec[dst * REC_WORDS + lane] = w;
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
    uint32_t slot = ptr[first + r];
    if (!sched_index_ok(st.status, slot <= st.zero_slot, SCHED_CHK_SLOT)) slot = st.zero_slot;
    // every lane reads the row's record (one address: a broadcast)
    const uint4 lo = *((const uint4 *)(st.rec + (size_t)slot * REC_WORDS));
    const uint4 hi = *((const uint4 *)(st.rec + (size_t)slot * REC_WORDS) + 1);
    if (lo.x == REC_OVERFLOW) {          // more occupied nodes than a record holds: the contents are in the pool
      if (aligned) {
        const uint4 *s4 = (const uint4 *)(st.pool + (size_t)slot * NN);
        uint4 *d4 = (uint4 *)(out + (size_t)r * NN);
        for (int v = lane; v < row_vecs; v += 32) d4[v] = s4[v];
      } else {
        for (int n = lane; n < NN; n += 32) out[(size_t)r * NN + n] = st.pool[(size_t)slot * NN + n];
      }
      continue;
    }
    const uint32_t e[REC_ENTRIES] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y};
    for (int v = lane; v < row_vecs; v += 32) {   // the row laid out from the record, a piece per lane
      uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int k = 0; k < REC_ENTRIES; ++k) {
        const int node = (int)(e[k] & 0xFFFu);
        if (e[k] && (node >> 3) == v) {
          const uint32_t val = ((e[k] >> 12) & 0x7FFu) << ((node & 1) * 16);
#pragma unroll
          for (int q = 0; q < 4; ++q) w[q] |= (((node & 7) >> 1) == q) ? val : 0u;
        }
      }
      if (aligned) {
        ((uint4 *)(out + (size_t)r * NN))[v] = make_uint4(w[0], w[1], w[2], w[3]);
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          out[(size_t)r * NN + 8 * v + 2 * q] = (int16_t)(w[q] & 0xFFFFu);
          out[(size_t)r * NN + 8 * v + 2 * q + 1] = (int16_t)(w[q] >> 16);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// One generation of one candidate per block.
// ---------------------------------------------------------------------------------------
struct GenArgs {
  StoreView st;
  const uint32_t *ptr_in;   // [P][J] parents ([J] for the initial population: the current allocation's rows)
  uint32_t *ptr_out;        // [P][J] children
  unsigned int *state;      // {next free slot, half}
  const int16_t *cap;       // [NN]
  const int32_t *k_cap;     // [J] or NULL
  const uint8_t *active;    // [J] or NULL
  const uint32_t *fitness_bits;  // [P] parents' fitness
  const int16_t *cur;       // [J][NN] or NULL
  int P, J, NN, k_max, n_max, num_elite;
  uint32_t thr, gen;        // perturbation threshold; generation number of the draws
  uint32_t init_src;        // initial population: slot of job 0's row before the row caps (perturbation source)
  RngKey key;
  TermParams tp;
  int rows_per_chunk, chunks;   // the dense fitness kernel's chunking, reproduced for identical sums
  float *fitness_out;       // [P]
  int *status;
};

// ---- a row as the list of its occupied nodes, which is what a record holds ---------------------
// e[0 .. n) = node | GPUs << 12 in ascending node order, K = GPUs in the row, nd = entries that
// differ from the current allocation's row.  One entry more than a record holds, so that a
// perturbation may add a node before the row caps take one away again.  Few rows of a generation
// are edited, each by one thread, so the helpers are plain loops (kept rolled: the kernel's
// instruction footprint matters more than their speed) over eight words of shared memory that
// belong to the thread.
constexpr int LIST_MAX = REC_ENTRIES + 1;
constexpr int LIST_WORDS = LIST_MAX + 1;

struct RowList {
  uint32_t *e;          // LIST_WORDS words of the thread's own
  int n, K, nd;
  // up to two entries changed by the perturbation whose effect on nd is still to be worked out
  // (their current-allocation values are fetched together, with the row's speedup, once K and N
  // are known)
  int pn, pnode0, pold0, pnew0, pnode1, pold1, pnew1;
};

__device__ __forceinline__ int ent_node(uint32_t e) { return (int)(e & 0xFFFu); }
__device__ __forceinline__ int ent_gpus(uint32_t e) { return (int)((e >> 12) & 0x7FFu); }

// fitness term of a row of job j from its summary: speedup looked up at (K, N), penalty when the
// row differs from the current allocation, floor, and the form that the mode sums (one copy of
// this code for all its users)
__device__ __noinline__ float row_term_from(bool has_pen, int mode, float p, float floor_, float x_sp, float x_pen,
                                            bool changed) {
  TermParams tp;
  tp.table = nullptr; tp.pen = nullptr; tp.active = nullptr;
  tp.k_max = 0; tp.n_max = 0; tp.mode = mode; tp.p = p; tp.floor_ = floor_;
  // the re-allocation penalty is applied here, the rest (floor, the form the mode sums) is shared
  return fitness_term_with(tp, (has_pen && changed) ? x_sp * x_pen : x_sp, 1.f, false);
}

__device__ __forceinline__ float row_term_of(const float *table, const float *pen, int k_max, int n_max, int mode, float p,
                                             float floor_, int j, int K, int N, int nd) {
  TermParams tp;
  tp.k_max = k_max; tp.n_max = n_max;
  const float x_sp = __ldg(table + fitness_table_index(tp, j, K, N));
  const float x_pen = (pen && nd != 0) ? __ldg(pen + j) : 1.f;
  return row_term_from(pen != nullptr, mode, p, floor_, x_sp, x_pen, nd != 0);
}

// one call of the random stream (one copy of the ten rounds for all users in this file)
__device__ __noinline__ u32x4 draw_call(uint32_t k0, uint32_t k1, uint32_t idx, uint32_t cand, uint32_t gen, uint32_t slot) {
  const u32x4 c = {idx, cand, gen, slot};
  return philox4x32_10(c, k0, k1);
}

// Two calls of the stream that differ only in their slot (the last counter word), rounds
// interleaved: the two chains of dependent multiplies hide each other's latency (a row's crossover
// and perturbation draws, a node's two repair draws).  Of the first call only word x is wanted.
// What the two calls share is worked out once: the first round entirely (the slot only enters its third
// output word), the first product of the second round and the second product of the third; the last round of
// the first call needs half a product.  35 products instead of 40.
__device__ __noinline__ void draw_pair_call(uint32_t k0, uint32_t k1, uint32_t idx, uint32_t cand, uint32_t gen,
                                            uint32_t slot_a, uint32_t slot_b, uint32_t &a_x, u32x4 &b) {
  // (the two halves of a product as two 32-bit multiplies)
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#define HI(m, v) __umulhi((m), (v))
#define LO(m, v) ((m) * (v))
  u32x4 ca, cb;
  {
    // first round, on (idx, cand, gen, slot): x, y, w do not see the slot
    const uint32_t x = HI(M1, gen) ^ cand ^ k0, y = LO(M1, gen), w = LO(M0, idx), h0 = HI(M0, idx);
    const uint32_t za = h0 ^ slot_a ^ k1, zb = h0 ^ slot_b ^ k1;
    k0 += W0; k1 += W1;
    // second round: the product of x is shared, so are the new z and w
    ca.x = HI(M1, za) ^ y ^ k0; ca.y = LO(M1, za);
    cb.x = HI(M1, zb) ^ y ^ k0; cb.y = LO(M1, zb);
    ca.z = cb.z = HI(M0, x) ^ w ^ k1;
    ca.w = cb.w = LO(M0, x);
    k0 += W0; k1 += W1;
    // third round: the product of z is shared
    const uint32_t h1 = HI(M1, ca.z), l1 = LO(M1, ca.z);
    u32x4 na, nb;
    na.x = h1 ^ ca.y ^ k0; na.y = l1; na.z = HI(M0, ca.x) ^ ca.w ^ k1; na.w = LO(M0, ca.x);
    nb.x = h1 ^ cb.y ^ k0; nb.y = l1; nb.z = HI(M0, cb.x) ^ cb.w ^ k1; nb.w = LO(M0, cb.x);
    ca = na; cb = nb;
    k0 += W0; k1 += W1;
  }
#pragma unroll
  for (int r = 3; r < 9; ++r) {
    u32x4 na, nb;
    na.x = HI(M1, ca.z) ^ ca.y ^ k0; na.y = LO(M1, ca.z); na.z = HI(M0, ca.x) ^ ca.w ^ k1; na.w = LO(M0, ca.x);
    nb.x = HI(M1, cb.z) ^ cb.y ^ k0; nb.y = LO(M1, cb.z); nb.z = HI(M0, cb.x) ^ cb.w ^ k1; nb.w = LO(M0, cb.x);
    ca = na;
    cb = nb;
    k0 += W0; k1 += W1;
  }
  // last round: of the first call only x
  a_x = HI(M1, ca.z) ^ ca.y ^ k0;
  b.x = HI(M1, cb.z) ^ cb.y ^ k0; b.y = LO(M1, cb.z); b.z = HI(M0, cb.x) ^ cb.w ^ k1; b.w = LO(M0, cb.x);
#undef HI
#undef LO
}

// GPUs of the row on `node` (0 when the node is not occupied) and where its entry is or belongs
__device__ __forceinline__ int list_find(const RowList &r, int node, int &pos, bool &found) {
  int v = 0;
  pos = 0;
  found = false;
#pragma unroll 1
  for (int k = 0; k < r.n; ++k) {
    const int nk = ent_node(r.e[k]);
    if (nk < node) pos = k + 1;
    if (nk == node) { found = true; v = ent_gpus(r.e[k]); }
  }
  return v;
}

// change in the count of entries that differ from the current allocation when A[j][node] goes
// from v_old to v_new
__device__ __forceinline__ int diff_delta(const int16_t *cur, int NN, int j, int node, int v_old, int v_new) {
  if (!cur) return 0;
  const int cv = (int)__ldg(cur + (size_t)j * NN + node);
  return (int)(v_new != cv) - (int)(v_old != cv);
}

// A[j][node] = v_new on the list form of row j (nd is brought up to date later, see RowList)
__device__ __forceinline__ void list_put(int *status, RowList &r, int node, int v_new) {
  int pos;
  bool found;
  const int v_old = list_find(r, node, pos, found);
  if (v_new == v_old) return;
  if (!sched_index_ok(status, r.n >= 0 && r.n <= LIST_MAX && pos >= 0 && pos <= r.n && r.pn < 2, SCHED_CHK_ENTRY)) return;
  if (r.pn == 0) { r.pnode0 = node; r.pold0 = v_old; r.pnew0 = v_new; }
  else { r.pnode1 = node; r.pold1 = v_old; r.pnew1 = v_new; }
  r.pn += 1;
  r.K += v_new - v_old;
  const uint32_t ent = (uint32_t)node | ((uint32_t)v_new << 12);
  if (found && v_new > 0) {
    r.e[pos] = ent;
  } else if (found) {            // the entry goes: the ones above it move down
#pragma unroll 1
    for (int k = pos; k + 1 < r.n; ++k) r.e[k] = r.e[k + 1];
    r.n -= 1;
    r.e[r.n] = 0u;
  } else if (r.n < LIST_MAX) {   // a new entry: the ones above its place move up
#pragma unroll 1
    for (int k = r.n; k > pos; --k) r.e[k] = r.e[k - 1];
    r.e[pos] = ent;
    r.n += 1;
  }
}

// the perturbation of a row (grow / shrink / relocate, chosen by the row's draw `mw`)
__device__ __forceinline__ void list_perturb(int *status, int NN, RowList &r, const u32x4 &mw, const int16_t *s_cap) {
  if (!sched_index_ok(status, r.n >= 0 && r.n <= REC_ENTRIES, SCHED_CHK_ENTRY)) return;
  const uint32_t op = bounded(mw.y, 3u);
  int pos;
  bool found;
  int node0 = -1, val0 = 0, node1 = -1, val1 = 0;   // up to two entries change
  if (op == 0u) {
    node0 = (int)bounded(mw.w, (uint32_t)NN);
    val0 = min(list_find(r, node0, pos, found) + 1, (int)s_cap[node0]);
  } else if (r.n > 0) {
    const uint32_t ent = r.e[bounded(mw.z, (uint32_t)r.n)];
    const int ns = ent_node(ent), vs = ent_gpus(ent);
    if (op == 1u) {
      node0 = ns;
      val0 = vs - 1;
    } else {
      const int nd = (int)bounded(mw.w, (uint32_t)NN);
      if (nd != ns) {
        node0 = nd;
        val0 = min(list_find(r, nd, pos, found) + vs, (int)s_cap[nd]);
        node1 = ns;
        val1 = 0;
      }
    }
  }
#pragma unroll 1
  for (int q = 0; q < 2; ++q) {
    const int node = q ? node1 : node0, val = q ? val1 : val0;
    if (node >= 0) list_put(status, r, node, val);
  }
}

// per-row caps: replicas above kc leave from the highest node index down, then occupied nodes
// beyond n_max are cleared from the highest index down
__device__ __forceinline__ void list_caps(const int16_t *cur, int NN, int n_max, RowList &r, int j, int kc) {
  if (r.K > kc) {
    int excess = r.K - kc;
#pragma unroll 1
    for (int k = r.n - 1; k >= 0 && excess > 0; --k) {
      const int node = ent_node(r.e[k]), v = ent_gpus(r.e[k]);
      const int take = min(v, excess);
      excess -= take;
      r.nd += diff_delta(cur, NN, j, node, v, v - take);
      if (v - take > 0) r.e[k] = (uint32_t)node | ((uint32_t)(v - take) << 12);
      else { r.e[k] = 0u; r.n = k; }      // everything above it has gone already
    }
    r.K = kc;
  }
#pragma unroll 1
  for (int k = r.n - 1; k >= n_max; --k) {
    const int node = ent_node(r.e[k]), v = ent_gpus(r.e[k]);
    r.K -= v;
    r.nd += diff_delta(cur, NN, j, node, v, 0);
    r.e[k] = 0u;
    r.n = k;
  }
}

__device__ __forceinline__ void list_from_record(RowList &r, uint32_t *words, uint4 lo, uint4 hi) {
  r.e = words;
  r.pnode0 = r.pold0 = r.pnew0 = r.pnode1 = r.pold1 = r.pnew1 = 0;
  r.e[0] = lo.x; r.e[1] = lo.y; r.e[2] = lo.z; r.e[3] = lo.w; r.e[4] = hi.x; r.e[5] = hi.y; r.e[6] = 0u; r.e[7] = 0u;
  r.K = (int)(hi.w & 0x7FFu);
  r.n = (int)((hi.w >> 11) & 0x7FFu);
  r.nd = (int)(hi.w >> 22);
  r.pn = 0;
}

// a record written by one thread: two 16-byte stores
__device__ __forceinline__ void store_record(uint32_t *rec, const RowList &r, float term, uint32_t word) {
  ((uint4 *)rec)[0] = make_uint4(r.e[0], r.e[1], r.e[2], r.e[3]);
  ((uint4 *)rec)[1] = make_uint4(r.e[4], r.e[5], __float_as_uint(term), word);
}

__device__ __forceinline__ uint4 piece_with(uint4 x, int h, int val) {   // entry h of the piece set to val
  const uint32_t sh = (uint32_t)(h & 1) * 16u, m = 0xFFFFu << sh, v = ((uint32_t)val & 0xFFFFu) << sh;
  if (h < 2) x.x = (x.x & ~m) | v;
  else if (h < 4) x.y = (x.y & ~m) | v;
  else if (h < 6) x.z = (x.z & ~m) | v;
  else x.w = (x.w & ~m) | v;
  return x;
}

// GPUs that the row stored in `slot` holds on node nn: from its record, or from its contents when
// the record does not hold the row (read from L2: the row may be new in this kernel)
__device__ __noinline__ int row_value_at(const uint32_t *rec, const int16_t *pool, int NN, uint32_t slot, int nn) {
  const uint4 lo = __ldcg((const uint4 *)(rec + (size_t)slot * REC_WORDS));
  if (lo.x == REC_OVERFLOW) return (int)__ldcg(pool + (size_t)slot * NN + nn);
  const uint4 hi = __ldcg((const uint4 *)(rec + (size_t)slot * REC_WORDS) + 1);
  const uint32_t e[REC_ENTRIES] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y};
  int v = 0;
#pragma unroll
  for (int k = 0; k < REC_ENTRIES; ++k)
    if (e[k] && ent_node(e[k]) == nn) v = ent_gpus(e[k]);
  return v;
}

// what the per-node repair decides for the occupant held by this lane of a group (entry = job |
// GPUs << 13 | distributed << 31 in the first have_n <= 16 lanes): the GPUs the job keeps on the node.
// o_intf, o_cap: the node's rotation offsets (its REPAIR_INTF and REPAIR_CAP draws, bounded by J).
__device__ __forceinline__ int decide_entries(const Grp &g, int J, int o_intf, int o_cap, int tot, int ne, int cap_n,
                                              uint32_t entry, int have_n) {
  const bool have = g.sub < have_n;
  const int j = (int)(entry & 0x1FFFu);
  int v = have ? (int)((entry >> 13) & 0x7FFu) : 0;
  const bool dist = have && (entry >> 31);
  if (ne >= 2) {
    const int o = o_intf;
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
    const int o = o_cap;
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

// perturbed rows of a block whose draw (and replica cap) is kept from the prologue; further ones
// draw again when their turn comes
constexpr int MUT_STASH = 128;

// Shared-memory carve-up of the generation kernel (sizes in bytes, 16-byte aligned pieces).
struct GenSmem {
  size_t slot, term, mark, acc, viol, occ, rowbuf, mut, ovf, slow, mod, cap, rec, sums, stash, total;
};

// most chunks the fitness chunking can cut J rows into (a block of the dense kernel covers at
// least 129 rows unless the whole candidate is smaller)
__host__ __device__ inline int gen_max_chunks(int J) { return J / 129 + 2; }

__host__ __device__ inline GenSmem gen_smem_layout(int J, int NN) {
  GenSmem L;
  size_t off = 0;
#define TAKE(field, bytes) do { L.field = off; off += ((size_t)(bytes) + 15) & ~(size_t)15; } while (0)
  TAKE(slot, (size_t)J * 4);
  TAKE(term, (size_t)J * 4);
  TAKE(mark, (size_t)J * 4);
  TAKE(acc, (size_t)NN * 8);
  TAKE(viol, (size_t)NN);
  TAKE(occ, (size_t)NN * OCC * 4);
  // a row per group of 16 lanes; at other times eight words per thread for the list form of a row
  TAKE(rowbuf, (size_t)GEN_GROUPS * NN * 2 > (size_t)GEN_THREADS * LIST_WORDS * 4 ? (size_t)GEN_GROUPS * NN * 2
                                                                                     : (size_t)GEN_THREADS * LIST_WORDS * 4);
  TAKE(mut, (size_t)J * 2);
  TAKE(ovf, (size_t)J * 2);
  TAKE(slow, (size_t)J * 2);
  TAKE(mod, (size_t)J * 2);
  TAKE(cap, (size_t)NN * 2);
  TAKE(rec, (size_t)GEN_GROUPS * REC_WORDS * 4);
  TAKE(sums, (size_t)gen_max_chunks(J) * GEN_WARPS * 12);
  TAKE(stash, (size_t)MUT_STASH * 16);
#undef TAKE
  L.total = off;
  return L;
}

// flags of a row inside a block (s_mark); bits 4.. hold the row's place among the perturbed rows
constexpr int MARK_CHANGED = 1;   // the column pass changes the row
constexpr int MARK_OWN = 2;       // the row's slot was made in this generation (rewritten in place)
constexpr int MARK_DIST = 4;      // the row spanned two nodes or more after the row pass (interference snapshot)

// block-wide minimum / exclusive prefix sum of one int per thread (s_red: GEN_WARPS + 1 ints);
// both end with a barrier, so s_red can be reused at once
__device__ __forceinline__ int block_min(int v, int *s_red) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, off));
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = s_red[0];
#pragma unroll
  for (int w = 1; w < GEN_WARPS; ++w) r = min(r, s_red[w]);
  __syncthreads();
  return r;
}

__device__ __forceinline__ int block_exscan(int v, int *s_red, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += u;
  }
  if (lane == 31) s_red[warp] = incl;
  __syncthreads();
  int before = 0;
  total = 0;
#pragma unroll
  for (int w = 0; w < GEN_WARPS; ++w) {
    const int t = s_red[w];
    if (w < warp) before += t;
    total += t;
  }
  __syncthreads();
  return before + incl - v;
}

template <int PPL, bool INIT>
__global__ void __launch_bounds__(GEN_THREADS, 4) generation_store_kernel(GenArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int J = a.J, NN = a.NN, P = a.P;
  const GenSmem L = gen_smem_layout(J, NN);
  uint32_t *s_slot = (uint32_t *)(smem + L.slot);
  int *s_mark = (int *)(smem + L.mark);
  float *s_term = (float *)(smem + L.term);
  // per node: GPUs placed (bits 0..31), distributed jobs on it (32..47), occupants (48..63)
  unsigned long long *s_node = (unsigned long long *)(smem + L.acc);
  uint8_t *s_viol = (uint8_t *)(smem + L.viol);       // 1: decided from the node's list, 2: column walked
  uint32_t *s_occ = (uint32_t *)(smem + L.occ);
  int16_t *s_rowbuf = (int16_t *)(smem + L.rowbuf);
  uint16_t *s_mut = (uint16_t *)(smem + L.mut), *s_ovf = (uint16_t *)(smem + L.ovf), *s_slow = (uint16_t *)(smem + L.slow);
  uint16_t *s_mod = (uint16_t *)(smem + L.mod);
  int16_t *s_cap = (int16_t *)(smem + L.cap);
  uint32_t *s_rec = (uint32_t *)(smem + L.rec);
  double *s_csum = (double *)(smem + L.sums);
  int *s_ccnt = (int *)(smem + L.sums + (size_t)gen_max_chunks(J) * GEN_WARPS * 8);
  uint4 *s_stash = (uint4 *)(smem + L.stash);         // per perturbed row: draw words y, z, w and the replica cap
  __shared__ int s_nmut, s_novf, s_nslow, s_nmod, s_nneed, s_ncow, s_fail, s_anyscan, s_po;
  __shared__ unsigned int s_base_mut, s_base_cow, s_base_cow2;
  __shared__ int s_parent, s_red[GEN_WARPS + 1];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t *my_list = (uint32_t *)s_rowbuf + tid * LIST_WORDS;
  const uint32_t c = blockIdx.x;
  // children that are plain copies: the best-ranked parents of a generation, the current allocation
  // itself in the initial population
  const bool elite = INIT ? (c == 0u) : ((int)c < a.num_elite);
  const uint32_t mut_slot = INIT ? SLOT_INIT : SLOT_MUTATE;

  // The next kernel of the stream may start while this one runs (programmatic dependent launch):
  // a following generation does its own prologue below and then waits for this grid to finish.
  asm volatile("griddepcontrol.launch_dependents;");

  // ---- prologue: nothing in it reads what the previous kernel writes, nothing is written to
  // global memory -----------------------------------------------------------------------------
  const uint32_t rkey = __ldg(a.key.round_ptr);
#pragma unroll 1
  for (int i = tid; i < NN; i += GEN_THREADS) {
    s_node[i] = 0ull; s_viol[i] = 0;
    s_cap[i] = (int16_t)max((int)a.cap[i], 0);
  }
#pragma unroll 1
  for (int i = tid; i < J; i += GEN_THREADS) s_mark[i] = 0;
  if (tid == 0) { s_nmut = 0; s_novf = 0; s_nslow = 0; s_nmod = 0; s_nneed = 0; s_ncow = 0; s_fail = 0; s_anyscan = 0; }
  __syncthreads();
  // every row's draws: which parent, perturbed or not; the perturbed rows are numbered
  uint32_t secbits = 0, mutbits = 0;   // bit r: this thread's r-th row (j = tid + r * GEN_THREADS)
  uint32_t actbits = 0;                // the thread's rows that exist and belong to active jobs
  {
    int r = 0;
#pragma unroll 1
    for (int j = tid; j < J; j += GEN_THREADS, ++r)
      if (!a.active || a.active[j]) actbits |= 1u << r;
  }
  if (!elite) {
    int r = 0;
#pragma unroll 1
    for (int j = tid; j < J; j += GEN_THREADS, ++r) {
      if (!((actbits >> r) & 1u)) continue;
      bool sec = false;
      u32x4 mw;
      if (INIT) {
        mw = draw_call(a.key.k0, rkey, (uint32_t)j, c, a.gen, mut_slot);
      } else {
        uint32_t xw;
        draw_pair_call(a.key.k0, rkey, (uint32_t)j, c, a.gen, SLOT_XOVER, mut_slot, xw, mw);
        sec = (xw >> 31) != 0u;
      }
      if (sec) secbits |= 1u << r;
      if (mw.x < a.thr) {
        mutbits |= 1u << r;
        const int i = atomicAdd(&s_nmut, 1);
        if (!sched_index_ok(a.status, i < J, SCHED_CHK_LIST)) continue;
        s_mut[i] = (uint16_t)(j | (sec ? 0x8000 : 0));          // j < 8192
        if (i < MUT_STASH)
          s_stash[i] = make_uint4(mw.y, mw.z, mw.w, (uint32_t)max(0, min(a.k_cap ? a.k_cap[j] : a.k_max, a.k_max)));
      }
    }
  }
  int idx[4] = {0, 0, 0, 0};
  if (!INIT && !elite) {
    const u32x4 sel = draw_call(a.key.k0, rkey, 0u, c, a.gen, SLOT_SELECT);
    idx[0] = (int)bounded(sel.x, P); idx[1] = (int)bounded(sel.y, P);
    idx[2] = (int)bounded(sel.z, P); idx[3] = (int)bounded(sel.w, P);
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- slots for the new rows: the perturbed ones plus a reserve for the rows the column pass
  // changes; one atomic, asked for now and needed once the parents are known -------------------
  unsigned int base_reg = 0, half_reg = 0;
  const int nmut = s_nmut;
  if (tid == GEN_THREADS - 1) {
    half_reg = __ldcg(a.state + 1);
    base_reg = atomicAdd(a.state, (unsigned int)(nmut + COW_RESERVE));
  }

  // ---- parents: the candidate of rank c for an elite child, else the better-ranked of two
  // random pairs (rank = candidates ordered before, fitness descending, index ascending) ----
  int par_a = 0, par_b = 0;
  if (INIT) {
    // every candidate descends from the current allocation
  } else if (elite) {
    // The candidate of rank c: composite keys (fitness key, then lower index first) are unique,
    // so c + 1 rounds of "largest key below the previous one" find it; one barrier per round.
    // Each thread keeps its first candidates' keys in registers.
    __shared__ unsigned long long s_wmax[2][GEN_WARPS];
    constexpr int KEEP = 4;
    unsigned long long mine[KEEP];
#pragma unroll
    for (int q = 0; q < KEEP; ++q) {
      const int i = tid + q * GEN_THREADS;
      mine[q] = (i < P) ? (((unsigned long long)order_key(__ldcg(a.fitness_bits + i)) << 32) |
                           (unsigned long long)(0xFFFFFFFFu - (uint32_t)i)) : 0ull;
    }
    unsigned long long prev = ~0ull;
#pragma unroll 1
    for (int t = 0; t <= (int)c; ++t) {
      unsigned long long best = 0ull;
#pragma unroll
      for (int q = 0; q < KEEP; ++q)
        if (mine[q] < prev && mine[q] > best) best = mine[q];
#pragma unroll 1
      for (int i = tid + KEEP * GEN_THREADS; i < P; i += GEN_THREADS) {
        const unsigned long long key = ((unsigned long long)order_key(__ldcg(a.fitness_bits + i)) << 32) |
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
    if (tid == 0) s_parent = (int)(0xFFFFFFFFu - (uint32_t)(prev & 0xFFFFFFFFull));
  } else {
    // the four drawn candidates' keys (every thread asks for the same four words)
    uint32_t k4[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) k4[q] = __ldcg(a.fitness_bits + idx[q]);
    par_a = tournament_winner(order_key(k4[0]), idx[0], order_key(k4[1]), idx[1]);
    par_b = tournament_winner(order_key(k4[2]), idx[2], order_key(k4[3]), idx[3]);
  }
  if (tid == GEN_THREADS - 1) {
    const unsigned long long limit = (unsigned long long)(half_reg + 1u) * a.st.half_cap;
    s_base_mut = base_reg;
    s_base_cow = base_reg + (unsigned int)nmut;
    if ((unsigned long long)base_reg + (unsigned long long)(nmut + COW_RESERVE) > limit) {
      s_fail = 1;
      atomicExch(a.status, SCHED_ERR_TOO_LARGE);
    }
  }
  __syncthreads();
  const bool fail = s_fail != 0;          // no slots: perturbed rows stay as their parents', nothing is repaired
  if (!INIT && elite) par_a = par_b = s_parent;

  // occupant (job j holds g GPUs on node n) into the node's totals and list
  auto add_occupant = [&](int j, int n, int g, bool dist) {
    if (!sched_index_ok(a.status, n >= 0 && n < NN && j >= 0 && j < J, SCHED_CHK_NODE)) return;
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
  // RB rows per thread at a time, so that their dependent loads (index -> record) travel together.
  // Perturbed rows are dealt out separately, row i of the block's list to thread i: a warp runs
  // through the long path for a perturbed row once whether one of its lanes has such a row or all
  // do, so the few there usually are share as few warps as possible.  The loads of a thread's first
  // perturbed row travel with those of its unperturbed rows.
  const uint32_t *pin_a = a.ptr_in + (INIT ? (size_t)0 : (size_t)par_a * J);
  const uint32_t *pin_b = a.ptr_in + (INIT ? (size_t)0 : (size_t)par_b * J);
  const int mine_first = tid;
  bool pre_loaded = mine_first < nmut;
  uint32_t pre_slot = 0;
  uint4 pre_lo = make_uint4(0u, 0u, 0u, 0u), pre_hi = pre_lo;
  if (pre_loaded) {
    const uint32_t mj = s_mut[mine_first];
    const int j = (int)(mj & 0x1FFFu);
    pre_slot = (INIT && !fail) ? a.init_src + (uint32_t)j : ((mj >> 15) ? __ldcg(pin_b + j) : __ldcg(pin_a + j));
  }
  constexpr int RB = 4;
  const int rows_per_thread = (J + GEN_THREADS - 1) / GEN_THREADS;
  const int own_batches = (rows_per_thread + RB - 1) / RB;
#pragma unroll 1
  for (int b = 0; b < own_batches; ++b) {
    uint32_t slot[RB];
    int jr[RB];
    bool on[RB], mut[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int rr = b * RB + r;                                // this thread's rr-th row
      jr[r] = tid + rr * GEN_THREADS;
      const bool sec = ((secbits >> rr) & 1u) != 0u;
      mut[r] = ((mutbits >> rr) & 1u) != 0u;
      on[r] = rr < 32 && ((actbits >> rr) & 1u) != 0u;
      const int j = jr[r];
      slot[r] = a.st.zero_slot;
      if (on[r]) {
        if (INIT && mut[r]) slot[r] = a.init_src + (uint32_t)j;   // perturbation starts before the row caps
        else slot[r] = sec ? __ldcg(pin_b + j) : __ldcg(pin_a + j);
      }
    }
    uint32_t rec[RB][REC_WORDS];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      if (!sched_index_ok(a.status, slot[r] <= a.st.zero_slot, SCHED_CHK_SLOT)) slot[r] = a.st.zero_slot;
      load_record(rec[r], a.st.rec + (size_t)slot[r] * REC_WORDS);
    }
    if (b == 0 && pre_loaded) {
      if (!sched_index_ok(a.status, pre_slot <= a.st.zero_slot, SCHED_CHK_SLOT)) pre_slot = a.st.zero_slot;
      pre_lo = __ldcg((const uint4 *)(a.st.rec + (size_t)pre_slot * REC_WORDS));
      pre_hi = __ldcg((const uint4 *)(a.st.rec + (size_t)pre_slot * REC_WORDS) + 1);
    }
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int j = jr[r];
      if (j >= J || mut[r]) continue;
      const uint32_t w = on[r] ? rec[r][REC_SUMM] : 0u;
      s_slot[j] = slot[r];
      if (!on[r]) continue;
      s_term[j] = __uint_as_float(rec[r][REC_TERM]);
      const bool dist = ((w >> 11) & 0x7FFu) >= 2u;
      if (dist) s_mark[j] = MARK_DIST;
      if (rec[r][0] == REC_OVERFLOW) {
        const int at = atomicAdd(&s_novf, 1);
        if (sched_index_ok(a.status, at < J, SCHED_CHK_LIST)) s_ovf[at] = (uint16_t)j;
        continue;
      }
#pragma unroll
      for (int k = 0; k < REC_ENTRIES; ++k) {
        const uint32_t e = rec[r][k];
        if (e) add_occupant(j, ent_node(e), ent_gpus(e), dist);
      }
    }
  }
  // ---- perturbed rows, one thread each -----------------------------------------------------------
  // The row is worked out on the list of occupied nodes its record holds and gets a record of
  // its own; only a row with more occupied nodes than a record holds needs its contents (left to
  // a group of lanes below).
#pragma unroll 1
  for (int i = mine_first; i < nmut; i += GEN_THREADS) {
    const uint32_t mj = s_mut[i];
    const int j = (int)(mj & 0x1FFFu);
    uint32_t src = pre_slot;
    uint4 lo = pre_lo, hi = pre_hi;
    if (!pre_loaded) {
      src = (INIT && !fail) ? a.init_src + (uint32_t)j : ((mj >> 15) ? __ldcg(pin_b + j) : __ldcg(pin_a + j));
      if (!sched_index_ok(a.status, src <= a.st.zero_slot, SCHED_CHK_SLOT)) src = a.st.zero_slot;
      lo = __ldcg((const uint4 *)(a.st.rec + (size_t)src * REC_WORDS));
      hi = __ldcg((const uint4 *)(a.st.rec + (size_t)src * REC_WORDS) + 1);
    }
    pre_loaded = false;
    s_slot[j] = src;
    s_mark[j] = i << 4;
    bool slow = lo.x == REC_OVERFLOW;
    if (fail) {
      // as an unperturbed row
      s_term[j] = __uint_as_float(hi.z);
      RowList rl;
      list_from_record(rl, my_list, lo, hi);
      if (slow) { s_ovf[atomicAdd(&s_novf, 1)] = (uint16_t)j; if (rl.n >= 2) s_mark[j] = MARK_DIST; continue; }
      if (rl.n >= 2) s_mark[j] = MARK_DIST;
#pragma unroll 1
      for (int k = 0; k < rl.n; ++k) add_occupant(j, ent_node(rl.e[k]), ent_gpus(rl.e[k]), rl.n >= 2);
      continue;
    }
    if (!slow) {
      RowList rl;
      list_from_record(rl, my_list, lo, hi);
      // K from the entries: the row a perturbation starts from may hold more GPUs than the summary's
      // field can say (the current allocation before the row caps)
      rl.K = 0;
#pragma unroll 1
      for (int k = 0; k < rl.n; ++k) rl.K += ent_gpus(rl.e[k]);
      u32x4 mw;
      int kc;
      if (i < MUT_STASH) {
        const uint4 st = s_stash[i];
        mw.x = 0u; mw.y = st.x; mw.z = st.y; mw.w = st.z;
        kc = (int)st.w;
      } else {
        mw = draw_call(a.key.k0, rkey, (uint32_t)j, c, a.gen, mut_slot);
        kc = max(0, min(a.k_cap ? a.k_cap[j] : a.k_max, a.k_max));
      }
      list_perturb(a.status, NN, rl, mw, s_cap);
      list_caps(a.cur, NN, a.n_max, rl, j, kc);
      slow = rl.n > REC_ENTRIES;
      if (!slow) {
        // K and N are final: the speedup, the penalty factor and the current allocation's values on
        // the nodes the perturbation touched are fetched together
        const float x_sp = __ldg(a.tp.table + fitness_table_index(a.tp, j, rl.K, rl.n));
        const float x_pen = a.tp.pen ? __ldg(a.tp.pen + j) : 1.f;
        int cv0 = 0, cv1 = 0;
        if (a.cur && rl.pn > 0) cv0 = (int)__ldg(a.cur + (size_t)j * NN + rl.pnode0);
        if (a.cur && rl.pn > 1) cv1 = (int)__ldg(a.cur + (size_t)j * NN + rl.pnode1);
        if (a.cur && rl.pn > 0) rl.nd += (int)(rl.pnew0 != cv0) - (int)(rl.pold0 != cv0);
        if (a.cur && rl.pn > 1) rl.nd += (int)(rl.pnew1 != cv1) - (int)(rl.pold1 != cv1);
        const uint32_t nslot = s_base_mut + (uint32_t)i;
        if (!sched_index_ok(a.status, nslot < a.st.zero_slot && rl.n >= 0 && rl.n <= REC_ENTRIES, SCHED_CHK_SLOT)) continue;
        const uint32_t word = pack_summary(rl.K, rl.n, rl.nd);
        const float term = row_term_from(a.tp.pen != nullptr, a.tp.mode, a.tp.p, a.tp.floor_, x_sp, x_pen, rl.nd != 0);
        store_record(a.st.rec + (size_t)nslot * REC_WORDS, rl, term, word);
        s_slot[j] = nslot;
        s_term[j] = term;
        s_mark[j] = MARK_OWN | (rl.n >= 2 ? MARK_DIST : 0);
#pragma unroll 1
        for (int k = 0; k < rl.n; ++k) add_occupant(j, ent_node(rl.e[k]), ent_gpus(rl.e[k]), rl.n >= 2);
      }
    }
    if (slow) {   // s_slot[j] is the source row, s_mark[j] >> 4 its number
      const int at = atomicAdd(&s_nslow, 1);
      if (sched_index_ok(a.status, at < J, SCHED_CHK_LIST)) s_slow[at] = (uint16_t)j;
    }
  }
  __syncthreads();

  // ---- the few rows that need their contents: a group of 16 lanes each --------------------------
  const Grp g = make_group(lane, NN);
  const int grp = tid >> 4;
  int16_t *row = s_rowbuf + (size_t)grp * NN;   // this group's row
  uint32_t *recw = s_rec + grp * REC_WORDS;
  if (s_nslow | s_novf) {
    // perturbed rows whose record does not hold them (before or after): contents from the pool, or
    // laid out from the record; perturbed, capped and summarised as a row; the contents are
    // written out only if the new record cannot hold the row either
#pragma unroll 1
    for (int i = grp; i < s_nslow; i += GEN_GROUPS) {
      const int j = (int)s_slow[i];
      const uint32_t old = s_slot[j];
      if (g.sub < REC_WORDS) recw[g.sub] = __ldcg(a.st.rec + (size_t)old * REC_WORDS + g.sub);
      const CurPieces<PPL> cur = cur_pieces<PPL>(g, a.cur ? a.cur + (size_t)j * NN : nullptr);
      const int kc_in = a.k_cap ? a.k_cap[j] : a.k_max;
      __syncwarp(g.mask);
      const int rN = (int)((recw[REC_SUMM] >> 11) & 0x7FFu);
      if (recw[0] == REC_OVERFLOW) {
        load_row<true>(g, row, a.st.pool + (size_t)old * NN);
      } else {
        for (int v = g.sub; v < g.row_vecs; v += GROUP) ((uint4 *)row)[v] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp(g.mask);
        if (g.sub < REC_ENTRIES && recw[g.sub]) row[ent_node(recw[g.sub])] = (int16_t)ent_gpus(recw[g.sub]);
      }
      __syncwarp(g.mask);
      const u32x4 mw = draw_call(a.key.k0, rkey, (uint32_t)j, c, a.gen, mut_slot);
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
      const uint32_t slot = s_base_mut + (uint32_t)(s_mark[j] >> 4);
      float term = 0.f;
      if (g.sub == 0)
        term = row_term_of(a.tp.table, a.tp.pen, a.tp.k_max, a.tp.n_max, a.tp.mode, a.tp.p, a.tp.floor_, j, K, N, nd);
      if (N > REC_ENTRIES) store_row(g, a.st.pool + (size_t)slot * NN, row);
      const uint32_t word = pack_summary(K, N, nd);
      __syncwarp(g.mask);
      if (g.sub == 0) {
        recw[REC_SUMM] = word;
        recw[REC_TERM] = __float_as_uint(term);
        s_slot[j] = slot;
        s_term[j] = term;
        s_mark[j] = MARK_OWN | (N >= 2 ? MARK_DIST : 0);
      }
      add_row_occupants(g, j, p, N >= 2);
      __syncwarp(g.mask);
      if (g.sub < REC_WORDS) a.st.rec[(size_t)slot * REC_WORDS + g.sub] = recw[g.sub];
      __syncwarp(g.mask);
    }
    // unperturbed rows with more occupied nodes than a record holds: occupants from the contents
#pragma unroll 1
    for (int i = grp; i < s_novf; i += GEN_GROUPS) {
      const int j = (int)s_ovf[i];
      load_row<true>(g, row, a.st.pool + (size_t)s_slot[j] * NN);
      __syncwarp(g.mask);
      const RowPieces<PPL> p = row_pieces<PPL>(g, row);
      add_row_occupants(g, j, p, (s_mark[j] & MARK_DIST) != 0);
      __syncwarp(g.mask);
    }
    __syncthreads();
  }

  // ---- column pass, decisions: which occupants of the violating nodes change ------------------
  // a warp looks at 32 nodes at a time, a lane each; its two groups of 16 lanes then decide the
  // nodes that hold two distributed jobs or more GPUs than they have
  if (!fail) {
#pragma unroll 1
    for (int nbase = warp * 32; nbase < NN; nbase += GEN_THREADS) {
      const int n_l = nbase + lane;
      bool bad = false;
      if (n_l < NN) {
        const unsigned long long acc_l = s_node[n_l];
        bad = (int)((acc_l >> 32) & 0xFFFFu) >= 2 || (int)(uint32_t)acc_l > (int)s_cap[n_l];
      }
      unsigned todo = __ballot_sync(0xffffffffu, bad);
      // the violating nodes' two rotation offsets, drawn by their lanes side by side
      int o_intf_l = 0, o_cap_l = 0;
      if (bad) {
        uint32_t xw;
        u32x4 cw;
        draw_pair_call(a.key.k0, rkey, (uint32_t)n_l, c, a.gen, SLOT_REPAIR_INTF, SLOT_REPAIR_CAP, xw, cw);
        o_intf_l = (int)bounded(xw, (uint32_t)J);
        o_cap_l = (int)bounded(cw.x, (uint32_t)J);
      }
#pragma unroll 1
      while (todo) {
      // the two lowest set bits: one node per group (the second group may have none)
      const int b0 = __ffs(todo) - 1;
      todo &= todo - 1;
      int b1 = -1;
      if (todo) { b1 = __ffs(todo) - 1; todo &= todo - 1; }
      const int bsel = (lane & GROUP) ? b1 : b0;
      const int o_intf = __shfl_sync(0xffffffffu, o_intf_l, max(bsel, 0));
      const int o_cap = __shfl_sync(0xffffffffu, o_cap_l, max(bsel, 0));
      if (bsel >= 0) {
      const int nn = nbase + bsel;
      const unsigned long long acc = s_node[nn];
      const int have_n = (int)(acc >> 48);
      if (have_n > OCC) {   // more occupants than the list holds: the column is walked below
        if (g.sub == 0) { s_viol[nn] = 2; s_anyscan = 1; }
      } else {
      const uint32_t entry = (g.sub < have_n) ? s_occ[nn * OCC + g.sub] : 0u;
      const int v_new = decide_entries(g, J, o_intf, o_cap, (int)(uint32_t)acc, (int)((acc >> 32) & 0xFFFFu), (int)s_cap[nn], entry, have_n);
      if (g.sub < have_n) {
        // the entry now carries the decision: GPUs kept, and bit 24 when that is a change
        const bool changed = v_new != (int)((entry >> 13) & 0x7FFu);
        s_occ[nn * OCC + g.sub] = (entry & 0x80001FFFu) | ((uint32_t)v_new << 13) | (changed ? (1u << 24) : 0u);
        if (changed) {
          const int j = (int)(entry & 0x1FFFu);
          const int before = atomicOr(&s_mark[j], MARK_CHANGED);
          if ((before & MARK_CHANGED) == 0) {
            const int at = atomicAdd(&s_nmod, 1);
            if (sched_index_ok(a.status, at < J, SCHED_CHK_LIST)) s_mod[at] = (uint16_t)j;
            if ((before & MARK_OWN) == 0) atomicAdd(&s_nneed, 1);   // will want a slot of its own
          }
        }
      }
      if (g.sub == 0) s_viol[nn] = 1;
      }
      }
      __syncwarp();
      }
    }
    __syncthreads();

    // ---- rows the column pass changes: rewritten by one thread each ----------------------------
    // The row keeps on each occupied node what the node's decision says (only_node < 0: looked up
    // in the lists of the decided nodes; else: only_value on that node).  The list of occupied
    // nodes is edited and stored as a new record - in a slot of its own (copy on write) unless the
    // row is new in this generation already; a row that only exists as contents is copied and
    // patched piece by piece.
    const int nmod = s_nmod;
    const bool scan = s_anyscan != 0;
    const int nneed = s_nneed;
    if (nneed > COW_RESERVE) {   // more rows to copy than the reserve: a further run of slots for the block
      if (tid == 0) {
        const unsigned int base = atomicAdd(a.state, (unsigned int)(nneed - COW_RESERVE));
        const unsigned long long limit = (unsigned long long)(__ldcg(a.state + 1) + 1u) * a.st.half_cap;
        s_base_cow2 = base;
        if ((unsigned long long)base + (unsigned long long)(nneed - COW_RESERVE) > limit) {
          s_fail = 1;
          atomicExch(a.status, SCHED_ERR_TOO_LARGE);
        }
      }
      __syncthreads();
    }
    const bool fail2 = s_fail != 0;
    auto rewrite_row = [&](int j, int only_node, int only_value) {
      if (!sched_index_ok(a.status, j >= 0 && j < J, SCHED_CHK_NODE)) return;
      const uint32_t src = s_slot[j];
      if (!sched_index_ok(a.status, src <= a.st.zero_slot, SCHED_CHK_SLOT)) return;
      const bool own = (s_mark[j] & MARK_OWN) != 0;
      const uint4 lo = __ldcg((const uint4 *)(a.st.rec + (size_t)src * REC_WORDS));
      const uint4 hi = __ldcg((const uint4 *)(a.st.rec + (size_t)src * REC_WORDS) + 1);
      uint32_t dst = src;
      if (!own) {   // a slot from the block's reserve, beyond it one by one
        const int k = atomicAdd(&s_ncow, 1);
        if (k < COW_RESERVE) {
          dst = s_base_cow + (uint32_t)k;
        } else if (k < nneed) {
          dst = s_base_cow2 + (uint32_t)(k - COW_RESERVE);
        } else {
          dst = atomicAdd(a.state, 1u);
          const unsigned long long limit = (unsigned long long)(__ldcg(a.state + 1) + 1u) * a.st.half_cap;
          if ((unsigned long long)dst + 1ull > limit) { atomicExch(a.status, SCHED_ERR_TOO_LARGE); return; }
        }
      }
      if (!sched_index_ok(a.status, dst < a.st.zero_slot, SCHED_CHK_SLOT)) return;
      auto new_value = [&](int node, int v) -> int {
        if (!sched_index_ok(a.status, node >= 0 && node < NN, SCHED_CHK_NODE)) return v;
        if (only_node >= 0) return node == only_node ? only_value : v;
        if (s_viol[node] != 1) return v;
        const int cnt = (int)(s_node[node] >> 48);
#pragma unroll 1
        for (int k = 0; k < cnt; ++k) {
          const uint32_t e = s_occ[node * OCC + k];
          if ((int)(e & 0x1FFFu) == j) return ((e >> 24) & 1u) ? (int)((e >> 13) & 0x7FFu) : v;
        }
        return v;
      };
      RowList rl;
      list_from_record(rl, my_list, lo, hi);
      float term;
      if (lo.x != REC_OVERFLOW) {
        int m = 0;                      // entries kept so far
#pragma unroll 1
        for (int k = 0; k < rl.n; ++k) {
          const int node = ent_node(rl.e[k]), v = ent_gpus(rl.e[k]);
          const int v_new = new_value(node, v);
          if (v_new != v) {
            // the first two changes are only noted: what the current allocation holds there is asked
            // for below, together with the row's speedup
            if (rl.pn == 0) { rl.pnode0 = node; rl.pold0 = v; rl.pnew0 = v_new; }
            else if (rl.pn == 1) { rl.pnode1 = node; rl.pold1 = v; rl.pnew1 = v_new; }
            else rl.nd += diff_delta(a.cur, NN, j, node, v, v_new);
            ++rl.pn;
            rl.K += v_new - v;
          }
          rl.e[k] = 0u;
          if (v_new > 0) rl.e[m++] = (uint32_t)node | ((uint32_t)v_new << 12);
        }
        rl.n = m;
        // K and N are final: speedup, penalty factor and the current allocation's values travel together
        const float x_sp = __ldg(a.tp.table + fitness_table_index(a.tp, j, rl.K, rl.n));
        const float x_pen = a.tp.pen ? __ldg(a.tp.pen + j) : 1.f;
        int cv0 = 0, cv1 = 0;
        if (a.cur && rl.pn > 0) cv0 = (int)__ldg(a.cur + (size_t)j * NN + rl.pnode0);
        if (a.cur && rl.pn > 1) cv1 = (int)__ldg(a.cur + (size_t)j * NN + rl.pnode1);
        if (a.cur && rl.pn > 0) rl.nd += (int)(rl.pnew0 != cv0) - (int)(rl.pold0 != cv0);
        if (a.cur && rl.pn > 1) rl.nd += (int)(rl.pnew1 != cv1) - (int)(rl.pold1 != cv1);
        term = row_term_from(a.tp.pen != nullptr, a.tp.mode, a.tp.p, a.tp.floor_, x_sp, x_pen, rl.nd != 0);
      } else {
        // contents only: pieces pass through this thread, patched on the way; the occupied nodes
        // that remain are listed, so that a row that now fits a record becomes one again
        const int16_t *from = a.st.pool + (size_t)src * NN;
        int16_t *to = a.st.pool + (size_t)dst * NN;
        int kept = 0;                   // occupied nodes that remain
#pragma unroll
        for (int k = 0; k <= LIST_MAX; ++k) rl.e[k] = 0u;
#pragma unroll 1
        for (int v = 0; v < (NN >> 3); ++v) {
          uint4 x = load_piece<true>(from, v);
          const uint4 x0 = x;
          uint32_t m = piece_mask(x);
          while (m) {
            const int h = __ffs(m) - 1;
            m &= m - 1;
            const int node = 8 * v + h, val = piece_entry(x, h);
            const int v_new = new_value(node, val);
            if (v_new != val) {
              rl.nd += diff_delta(a.cur, NN, j, node, val, v_new);
              rl.K += v_new - val;
              rl.n -= (v_new == 0) ? 1 : 0;
              x = piece_with(x, h, v_new);
            }
            if (v_new > 0) {
              if (kept < REC_ENTRIES) rl.e[kept] = (uint32_t)node | ((uint32_t)v_new << 12);
              ++kept;
            }
          }
          if (!own || x.x != x0.x || x.y != x0.y || x.z != x0.z || x.w != x0.w) ((uint4 *)to)[v] = x;
        }
        if (kept > REC_ENTRIES) {       // still more occupied nodes than a record holds
          rl.e[0] = REC_OVERFLOW;
#pragma unroll
          for (int k = 1; k < LIST_MAX; ++k) rl.e[k] = 0u;
        }
        term = row_term_of(a.tp.table, a.tp.pen, a.tp.k_max, a.tp.n_max, a.tp.mode, a.tp.p, a.tp.floor_, j, rl.K, rl.n, rl.nd);
      }
      const uint32_t word = pack_summary(rl.K, rl.n, rl.nd);
      store_record(a.st.rec + (size_t)dst * REC_WORDS, rl, term, word);
      s_slot[j] = dst;
      s_term[j] = term;
      s_mark[j] |= MARK_OWN;
    };
    // Thread work for the two uses of rewrite_row, gathered so that the code exists once: first the
    // rows the listed nodes changed (row i of the list to thread i), then, node by
    // node, the rows of the columns that had to be walked.
    const int rpt = (J + GEN_THREADS - 1) / GEN_THREADS;
    const int j_lo = min(J, tid * rpt), j_hi = min(J, j_lo + rpt);
    // ---- nodes with more occupants than a list holds: the whole block walks the column -------
    // Thread t looks after the consecutive rows [t * rpt, (t + 1) * rpt); a row's GPUs on the node
    // come from its record (or its contents).  Interference: the first distributed occupant in
    // rotated job order stays.  Capacity: a block-wide prefix sum in job order gives every row the
    // GPUs that come before it in rotated order.
#pragma unroll 1
    for (int step = -1; step < (scan ? NN : 0) && !fail2; ++step) {
      int nn = -1, keep = -1, excess = 0, o2 = 0, p_o = 0, total = 0, running = 0;
      if (step >= 0) {
        if (step == 0) __syncthreads();          // the listed rewrites are done
        nn = step;
        if (s_viol[nn] != 2) continue;
        const unsigned long long acc = s_node[nn];
        const int ne = (int)((acc >> 32) & 0xFFFFu), cap_n = (int)s_cap[nn];
        if (ne >= 2) {
          const int o = (int)bounded(draw_call(a.key.k0, rkey, (uint32_t)nn, c, a.gen, SLOT_REPAIR_INTF).x, (uint32_t)J);
          int best = J;
#pragma unroll 1
          for (int j = j_lo; j < j_hi; ++j) {
            if ((s_mark[j] & MARK_DIST) && row_value_at(a.st.rec, a.st.pool, NN, s_slot[j], nn) > 0) {
              int t = j - o;
              if (t < 0) t += J;
              best = min(best, t);
            }
          }
          best = block_min(best, s_red);
          keep = o + best;
          if (keep >= J) keep -= J;
        }
        int mine = 0;
#pragma unroll 1
        for (int j = j_lo; j < j_hi; ++j) {
          const int v = row_value_at(a.st.rec, a.st.pool, NN, s_slot[j], nn);
          mine += (keep >= 0 && (s_mark[j] & MARK_DIST) && v > 0 && j != keep) ? 0 : v;
        }
        running = block_exscan(mine, s_red, total);
        excess = total - cap_n;
        if (excess > 0) {
          o2 = (int)bounded(draw_call(a.key.k0, rkey, (uint32_t)nn, c, a.gen, SLOT_REPAIR_CAP).x, (uint32_t)J);
          if (o2 >= j_lo && o2 < j_hi) {      // GPUs of the rows before row o2 in job order
            int p = running;
#pragma unroll 1
            for (int j = j_lo; j < o2; ++j) {
              const int v = row_value_at(a.st.rec, a.st.pool, NN, s_slot[j], nn);
              p += (keep >= 0 && (s_mark[j] & MARK_DIST) && v > 0 && j != keep) ? 0 : v;
            }
            s_po = p;
          }
          __syncthreads();
          p_o = s_po;
        }
      }
      // the rows this thread rewrites in this step
      const int first = (step < 0) ? mine_first : j_lo;
      const int last = (step < 0) ? nmod : j_hi;
      const int stride = (step < 0) ? GEN_THREADS : 1;
#pragma unroll 1
      for (int i = first; i < last; i += stride) {
        if (step < 0) {
          rewrite_row((int)s_mod[i], -1, 0);
          continue;
        }
        const int j = i;
        const int v = row_value_at(a.st.rec, a.st.pool, NN, s_slot[j], nn);
        const int v_eff = (keep >= 0 && (s_mark[j] & MARK_DIST) && v > 0 && j != keep) ? 0 : v;
        int take = 0;
        if (excess > 0) {
          const int ahead = (j >= o2) ? running - p_o : total - p_o + running;
          take = min(v_eff, max(excess - ahead, 0));
        }
        running += v_eff;
        if (v_eff - take != v) rewrite_row(j, nn, v_eff - take);
      }
      if (step >= 0) __syncthreads();   // the rewritten rows are read again for the next such node
    }
  }
  __syncthreads();

  // ---- children's indices out, fitness of the candidate (Eq. 14) from the rows' terms ----------
  uint32_t *pout = a.ptr_out + (size_t)c * J;
#pragma unroll 1
  for (int j = tid; j < J; j += GEN_THREADS) pout[j] = s_slot[j];
  // sums in the order of the dense fitness kernel: per chunk of rows, thread t adds rows t,
  // t + 256, ... in double, a shuffle tree per warp, the warps in index order; then the chunks
  // in index order
#pragma unroll 1
  for (int ch = 0; ch < a.chunks; ++ch) {
    const int j0 = ch * a.rows_per_chunk, j1 = min(J, j0 + a.rows_per_chunk);
    double acc = 0.0;
    int cnt = 0;
#pragma unroll 1
    for (int j = j0 + tid; j < j1; j += GEN_THREADS) {
      if (!a.tp.active || a.tp.active[j]) { acc += (double)s_term[j]; cnt += 1; }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      acc += __shfl_xor_sync(0xffffffffu, acc, off);
      cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    }
    if (lane == 0) { s_csum[ch * GEN_WARPS + warp] = acc; s_ccnt[ch * GEN_WARPS + warp] = cnt; }
  }
  __syncthreads();
  if (tid == 0) {
    double ts = 0.0, ns = 0.0;
#pragma unroll 1
    for (int ch = 0; ch < a.chunks; ++ch) {
      double t = 0.0;
      int n = 0;
      for (int w = 0; w < GEN_WARPS; ++w) { t += s_csum[ch * GEN_WARPS + w]; n += s_ccnt[ch * GEN_WARPS + w]; }
      ts += t;
      ns += (double)n;
    }
    a.fitness_out[c] = fitness_finalise(a.tp.mode, a.tp.p, ts, ns);
  }
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
  v.status = ctx->d_status;
  return v;
}

}  // namespace

// Pool budget (default 12 GiB, sched_set_store_budget) of rows and records; the rows' part is
// address space more than traffic: a row's contents are only written when its record cannot hold
// it.  Returns how many generations' worst case a half can take on top of the population, at
// most 24.
// rows a half holds before any generation: the population, or the current allocation's two rows
// per job that a round starts from
static unsigned long long store_base_rows(const sched_config &c) {
  const unsigned long long rows = (unsigned long long)c.population * c.num_jobs;
  return rows > 2ull * c.num_jobs ? rows : 2ull * c.num_jobs;
}

static int store_units(const sched_config &c, unsigned long long budget) {
  const unsigned long long rows = store_base_rows(c);
  const unsigned long long worst = store_worst_case(c.population, c.num_jobs);
  const unsigned long long row_bytes = (unsigned long long)c.num_nodes * 2 + REC_WORDS * 4;
  const unsigned long long half_rows = budget / 2 / row_bytes;
  const unsigned long long index_rows = ((1ull << 32) - 2) / 2;      // slot indices are 32-bit
  const unsigned long long room = half_rows < index_rows ? half_rows : index_rows;
  if (room <= rows) return 0;
  const unsigned long long units = (room - rows) / worst;
  return (int)(units < 24 ? units : 24);
}

// The row store serves rounds whose candidates span several row batches of the dense
// kernels (J > 256; smaller problems run a generation as one dense kernel already), with
// rows of whole 16-byte vectors and sizes that fit the packed fields.
bool rowstore_eligible(const sched_ctx *ctx, const int16_t *) {
  const sched_config &c = ctx->cfg;
  if (c.num_jobs <= 256 || c.num_jobs > STORE_MAX_JOBS) return false;
  if (c.num_nodes % 8 != 0 || c.num_nodes > 512 || ctx->cap_max > 2047) return false;
  if (c.k_max > 2047 || c.n_max > 2047) return false;
  if (gen_smem_layout(c.num_jobs, c.num_nodes).total > 200 * 1024) return false;
  // a half holds the population plus at least two generations' worst case; if that does not fit
  // the pool's budget (or 32-bit slot indices) the dense path runs
  return store_units(c, ctx->rs_budget) >= 2;
}

int rowstore_ensure(sched_ctx *ctx) {
  if (ctx->rs_ready) return SCHED_OK;
  const sched_config &c = ctx->cfg;
  const unsigned long long rows = (unsigned long long)c.population * c.num_jobs;
  // half = the population + `units` generations' worst case.  The check runs every `check`
  // generations and moves the rows once fewer than `check` units are left, i.e. after the other
  // units - check have been used up: real generations take a few percent of the worst case, so
  // a wide margin means a move is rare and a long interval means few check launches.
  const int units = store_units(c, ctx->rs_budget);
  const int check = units / 2 < 1 ? 1 : units / 2 > 12 ? 12 : units / 2;
  const unsigned long long worst = store_worst_case(c.population, c.num_jobs);
  ctx->rs_check_every = check;
  ctx->rs_half_cap = (size_t)(store_base_rows(c) + (unsigned long long)units * worst);
  const size_t slots = 2 * ctx->rs_half_cap + 1;
  cudaError_t e = cudaMalloc((void **)&ctx->rs_pool, slots * c.num_nodes * sizeof(int16_t));
  if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->rs_rec, slots * REC_WORDS * sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->rs_ptr, 2 * (size_t)rows * sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->rs_state, 5 * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->rs_state, 0, 5 * sizeof(unsigned int), ctx->stream);
  if (e == cudaSuccess) {
    const size_t smem = gen_smem_layout(c.num_jobs, c.num_nodes).total;
    if (smem > 48 * 1024)
    for (int k = 0; k < 6 && e == cudaSuccess; ++k) {
      void (*kernel)(GenArgs) = k == 0 ? generation_store_kernel<1, false> : k == 1 ? generation_store_kernel<2, false>
                                : k == 2 ? generation_store_kernel<4, false> : k == 3 ? generation_store_kernel<1, true>
                                : k == 4 ? generation_store_kernel<2, true> : generation_store_kernel<4, true>;
      e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    }
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

int rowstore_build_current(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, const int16_t *d_seed,
                           const int16_t *d_cur, const float *d_pen) {
  const sched_config &c = ctx->cfg;
  BuildCurArgs a;
  a.st = store_view(ctx);
  a.ptr = ctx->rs_ptr;
  a.state = ctx->rs_state;
  a.active = d_active; a.seed = d_seed; a.cur = d_cur; a.cap = ctx->d_cap; a.k_cap = d_k_cap;
  a.tp.table = ctx->d_tab_speedup; a.tp.pen = d_pen; a.tp.active = d_active;
  a.tp.k_max = c.k_max; a.tp.n_max = c.n_max; a.tp.mode = fitness_mode(c.p); a.tp.p = c.p;
  a.tp.floor_ = c.speedup_floor;
  a.J = c.num_jobs; a.NN = c.num_nodes; a.k_max = c.k_max; a.n_max = c.n_max;
  {
    TimedLaunch tl_(ctx, KK_STORE_BUILD);
    const int ppl = store_pieces_per_lane(c.num_nodes);
    const int blocks = (c.num_jobs + 15) / 16;
    if (ppl == 1) rowstore_build_cur_kernel<1><<<blocks, 256, 0, ctx->stream>>>(a);
    else if (ppl == 2) rowstore_build_cur_kernel<2><<<blocks, 256, 0, ctx->stream>>>(a);
    else rowstore_build_cur_kernel<4><<<blocks, 256, 0, ctx->stream>>>(a);
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
  a.moves = ctx->rs_state + 4;
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

// generation == GEN_INIT: the initial population, made from the rows rowstore_build_current left
// (children are the current allocation perturbed with thr_init; they go to index set `parity ^ 1`)
int rowstore_generation(sched_ctx *ctx, const int32_t *d_k_cap, const uint8_t *d_active, const int16_t *d_cur,
                        const float *d_pen, const float *d_fitness_in, float *d_fitness_out, int parity,
                        int state_phase, uint32_t generation) {
  const bool init = generation == GEN_INIT;
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
  a.thr = init ? c.thr_init : c.thr_mutate; a.gen = generation; a.init_src = (uint32_t)c.num_jobs;
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
    // launched so that it may start while the previous kernel of the stream still runs: the kernel
    // does its draws first and waits for that kernel before it reads anything it wrote
    const int ppl = store_pieces_per_lane(c.num_nodes);
    void (*kernel)(GenArgs) = init ? (ppl == 1 ? generation_store_kernel<1, true>
                                      : ppl == 2 ? generation_store_kernel<2, true> : generation_store_kernel<4, true>)
                                   : (ppl == 1 ? generation_store_kernel<1, false>
                                      : ppl == 2 ? generation_store_kernel<2, false> : generation_store_kernel<4, false>);
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)c.population);
    lc.blockDim = dim3(GEN_THREADS);
    lc.dynamicSmemBytes = smem;
    lc.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, kernel, a) != cudaSuccess) {
      cudaGetLastError();
      kernel<<<c.population, GEN_THREADS, smem, ctx->stream>>>(a);
    }
  }
  SCHED_LAUNCH_CHECK(ctx);
  return SCHED_OK;
}
