// Full routing of a set of rows in ONE kernel, two sweeps over the key chunks: score GEMM on
// the tensor cores (Eq. 1), per-row TopK (Eq. 2), near-miss sentinels (Section 3.1 item 1),
// k-th score and margin (Section 3.3), mandatory global and random sentinels (Section 3.1
// items 2, 3) -- the score matrix never leaves the SM.
//
// One CTA owns 128 query rows of one problem (consecutive rows at an anchor; a segment of the
// compacted refresh list at a relay, Section 4.2) and walks the key chunks in tiles of 128,
// stopping at the last chunk any of its rows may select.
//   warp 0     : TMA producer (Kc tiles, 128-byte swizzle, a ring of five half-tile stages, no
//                multicast)
//   warps 1, 18: one thread each issues tcgen05.mma (M=128, N=128, K=16), alternating tiles, into
//                a ring of 3 TMEM accumulators; the Qc tile is the MMA's A operand in TMEM
//   warps 2-17 : selection, FOUR THREADS PER QUERY ROW: thread j of a row owns columns
//                [32j, 32j+32) of every tile (tcgen05.ld 32x32b hands it 32 consecutive
//                scores of its row).
// Sweep 1 (threshold before filtering): each thread keeps the running maximum of each of its
// 32 column positions over all tiles -- 128 disjoint groups per row -- and sorts them with a
// sorting network in registers.  The keep-th largest of the row's 128 group maxima, keep =
// k + max(m,1), has keep distinct scores of the row at or above it, so it is a valid inclusive
// lower bound tau of the row's keep-th largest score, and the tightest the maxima give (about
// 1.2 keep scores pass); one thread per row finds it by exchange over the four published sorted
// lists (exchange_select).  (A bound from a refresh row's old candidates, as the streaming
// kernel uses, bought nothing here and is not read.)
// Sweep 2 (the tile MMAs are simply issued again; Kc comes from L2): each thread appends its
// scores >= tau to a private list of 32 {score, chunk id} entries in shared memory, sorts the
// list (network on keys that carry 27 score bits and the list position, then an exact repair
// of neighbours that agree in those bits) and writes it back in rank order.  Two threads per row
// then find, again by exchange over the row's four sorted lists, how many entries of each list
// belong to the top k and to the top keep: the first give the route, the k-th score and the
// margin, the rest the near-miss sentinels; every thread moves its own entries' ids to a staging
// area and the ledger row goes out with 16-byte stores.  Ties go to the smaller chunk id.
// The mandatory global and the random sentinels of the routed rows are built by a separate
// one-thread-per-row kernel (rr_sentinels.cu) that runs at full occupancy: inside this kernel,
// which holds one CTA per SM, their serial draws would sit on every CTA's critical path.
// Rows the fast path cannot finish exactly (a list overflowed, three or more scores agreeing in
// 27 bits inside one list, equal scores across a cut) are handed to an exact slow path: one more sweep stores their
// complete score rows in shared memory, and a warp per row runs the radix select of the
// two-pass path on them.  Every mbarrier wait is bounded.
#include "rr_common.cuh"
#include "rr_sm100.cuh"
#include "rr_warp_topk.cuh"

using namespace sm100;

namespace {

constexpr int BM = 128, BN = 128, H_STAGES = 5, ACC_STAGES = 3;   // H_STAGES: Kc stages of one K-half
constexpr int TPR = 4, SLICE = BN / TPR;           // threads per row, columns per thread and tile
constexpr int SEL_WARPS = TPR * (BM / 32), ISSUE_WARPS = 2;
constexpr int LAST_SEL = 2 + SEL_WARPS;            // warps [2, LAST_SEL) select; the second issuer follows
constexpr int NT = (LAST_SEL + ISSUE_WARPS - 1) * 32;
constexpr int TMEM_COLS = 512, A_COL = ACC_STAGES * BN;   // Qc tile behind the accumulators
constexpr int CAPJ = 32;                           // entries per list
constexpr int MAX_KEEP = 48, MAX_NK = 1024;        // what the lists / bitmaps are sized for
constexpr int BM_WORDS = MAX_NK / 32;
constexpr int HARD_SLOTS = 24;                     // score rows held at once by the slow path
constexpr int MAX_SLOTS = 16;                      // candidate slots per thread of the in-place relay
constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr uint32_t ENTRY_PITCH = TPR * BM * 8;     // bytes between entries e and e+1 of a list
constexpr uint32_t LIST_PITCH = BM * 8;            // bytes between lists j and j+1 of a row

template <int D>
struct Cfg {
  static constexpr int KHALVES = D / 64;
  static constexpr int B_HALF = BN * 128;          // one stage: 128 key chunks x 64 bf16 (128 bytes)
};

struct Ctl {
  uint64_t full[H_STAGES], empty[H_STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
  uint64_t drain[ISSUE_WARPS];       // completes when all MMAs of an issuer have finished
  uint32_t tmem_base, abort_flag, hard_n, pad_;
  int row[BM], slot[BM];
  float tau_row[BM];                // the row's bound from the group maxima
  float ab[2][TPR][BM];             // in-place relay: each thread's part of alpha / beta
  uint32_t n_flagged, n_cand, pad2_[2];
  unsigned long long v_flagged;     // in-place relay: counters of the CTA
  uint8_t live[BM];                 // in-place relay: the row failed the challenge test
  uint32_t cnt[TPR][BM];            // list lengths; bit 8 = this list needs the slow path
  uint32_t cut_k[BM], cut_keep[BM]; // per row: entries of each list (8 bits each) in the top k / keep
  uint8_t cut_bad[2][BM];           // a cut could not be settled (scores tie across it)
  uint8_t hard_rows[BM];            // rows handed to the slow path, in registration order
  int8_t hard_slot[BM];             // position of a row in hard_rows, -1 = none
};
constexpr int CTL_BYTES = 12288;
static_assert(sizeof(Ctl) <= CTL_BYTES, "control block too large");
constexpr int BUF_BYTES = CAPJ * ENTRY_PITCH;             // 128 KB
static_assert(HARD_SLOTS * MAX_NK * 4 + SEL_WARPS * (256 + BM_WORDS) * 4 <= BUF_BYTES,
              "slow-path rows and per-warp scratch must fit the list area");

__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v; asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void lds64(uint32_t a, uint32_t& x, uint32_t& y) {
  asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(a) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t a, uint32_t x, uint32_t y) {
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(a), "r"(x), "r"(y) : "memory");
}
// the four warps that share a quarter of the rows (128 threads), barrier ids 1..4
__device__ __forceinline__ void quarter_sync(int quarter) {
  asm volatile("bar.sync %0, 128;" ::"r"(quarter + 1) : "memory");
}

// Batcher's odd-even merge sort as a compile-time network (descending): every index is a
// template constant, so the array stays in registers.  N a power of two.
template <class T> struct DescF {
  static __device__ __forceinline__ void ce(T& a, T& b) { const T hi = fmaxf(a, b), lo = fminf(a, b); a = hi; b = lo; }
};
template <class T> struct DescU {
  static __device__ __forceinline__ void ce(T& a, T& b) { const T hi = max(a, b), lo = min(a, b); a = hi; b = lo; }
};
// LIMIT < N prunes the network to its first LIMIT inputs: valid when the inputs from LIMIT on hold
// the smallest key and sit last, since a compare-exchange with such an input changes nothing.
template <int LO, int N, int R, class T, class OP, int LIMIT> struct OEMerge {
  static __device__ __forceinline__ void run(T* x) {
    constexpr int M = R * 2;
    if constexpr (M < N) {
      OEMerge<LO, N, M, T, OP, LIMIT>::run(x);
      OEMerge<LO + R, N, M, T, OP, LIMIT>::run(x);
#pragma unroll
      for (int i = LO + R; i + R < LO + N; i += M)
        if (i + R < LIMIT) OP::ce(x[i], x[i + R]);
    } else {
      if constexpr (LO + R < LIMIT) OP::ce(x[LO], x[LO + R]);
    }
  }
};
template <int LO, int N, class T, class OP, int LIMIT = LO + N> struct OESort {
  static __device__ __forceinline__ void run(T* x) {
    if constexpr (N > 1 && LO < LIMIT) {
      constexpr int M = N / 2;
      OESort<LO, M, T, OP, LIMIT>::run(x);
      OESort<LO + M, M, T, OP, LIMIT>::run(x);
      OEMerge<LO, N, 1, T, OP, LIMIT>::run(x);
    }
  }
};

// ---- sorting one list of sweep 2 ------------------------------------------------------------
// The list (n <= LIMIT <= 32 entries {score, id} at base + e * ENTRY_PITCH, in ascending chunk id)
// is rewritten in rank order (score descending, id ascending).  Keys = 27 score bits | (31 -
// position), sorted by a network in registers; neighbours that agree in the 27 bits are ordered
// by position at that point and are repaired with the exact scores (equal scores keep the
// position order = ascending chunk id); three in a row are reported (slow path).
template <int LIMIT>
__device__ __forceinline__ bool sort_list(uint32_t base, int n) {
  uint32_t key[CAPJ];
#pragma unroll
  for (int e = 0; e < CAPJ; ++e) {
    key[e] = 0u;
    if (e < LIMIT) {
      uint32_t sb;
      asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sb) : "r"(base + (uint32_t)e * ENTRY_PITCH) : "memory");
      const uint32_t ok = rr_order_key(__uint_as_float(sb));
      key[e] = e < n ? ((ok & ~31u) | (uint32_t)(31 - e)) : 0u;
    }
  }
  OESort<0, CAPJ, uint32_t, DescU<uint32_t>, LIMIT>::run(key);
  bool same = false, run3 = false;
#pragma unroll
  for (int i = 0; i + 1 < LIMIT; ++i) same |= key[i + 1] >= 32u && ((key[i] ^ key[i + 1]) < 32u);
  if (__any_sync(0xFFFFFFFFu, same)) {
#pragma unroll
    for (int i = 0; i + 1 < LIMIT; ++i) {
      const bool pair = key[i + 1] >= 32u && ((key[i] ^ key[i + 1]) < 32u);
      if (pair) {
        uint32_t sa, sb;
        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sa) : "r"(base + (31u - (key[i] & 31u)) * ENTRY_PITCH) : "memory");
        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sb) : "r"(base + (31u - (key[i + 1] & 31u)) * ENTRY_PITCH) : "memory");
        if (__uint_as_float(sb) > __uint_as_float(sa)) { const uint32_t t = key[i]; key[i] = key[i + 1]; key[i + 1] = t; }
        if (i + 2 < LIMIT && key[i + 2] >= 32u && ((key[i] ^ key[i + 2]) < 32u)) run3 = true;
      }
    }
  }
  // write the list back in rank order: all loads first, then all stores
  uint32_t es[LIMIT], ei[LIMIT];
#pragma unroll
  for (int i = 0; i < LIMIT; ++i)
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(es[i]), "=r"(ei[i])
                 : "r"(base + (31u - (key[i] & 31u)) * ENTRY_PITCH) : "memory");
#pragma unroll
  for (int i = 0; i < LIMIT; ++i)
    if (i < n) asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(base + (uint32_t)i * ENTRY_PITCH), "r"(es[i]), "r"(ei[i]) : "memory");
  return run3;
}


// ---- exchange selection over four sorted lists -----------------------------------------------
// The four lists of a row (scores in descending order in the score words of its list entries,
// n_j entries each) and a split a_0 + a_1 + a_2 + a_3 = T: the first a_j entries of list j are
// "in".  One entry at a time leaves the list whose last entry in is the smallest and one enters
// from the list whose first entry out is the largest, while the latter is larger; every such
// move raises the sum of what is in, so the search ends, and it ends at the split that holds the
// T largest scores: lo = the smallest score in (the T-th largest), hi = the largest score out.
// Any split reached on the way already has T scores at or above its lo.
// Every step re-reads the eight scores at the four cuts from shared memory (eight independent
// loads) instead of carrying them in registers: the register form needs chains of selects to
// address "the list that moves", and those chains, not the loads, were the step's latency.
// Warp-uniform: lanes that are done idle.
struct Exchange { int a0, a1, a2, a3; float lo, hi; };
__device__ __forceinline__ Exchange exchange_select(uint32_t row_base, int n0, int n1, int n2, int n3,
                                                    int a0, int a1, int a2, int a3, bool on,
                                                    int max_steps) {
  const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);
  float lo, hi;
  for (int it = 0;; ++it) {
    // last entry in (l) and first entry out (x) of every list; +inf / -inf where there is none
#define RR_CUT(j)                                                                                   \
    float l##j, x##j;                                                                               \
    {                                                                                               \
      const uint32_t base_ = row_base + (uint32_t)j * LIST_PITCH;                                   \
      uint32_t lb_, xb_;                                                                            \
      asm volatile("ld.shared.b32 %0, [%1];" : "=r"(lb_) : "r"(base_ + (uint32_t)max(a##j - 1, 0) * ENTRY_PITCH) : "memory"); \
      asm volatile("ld.shared.b32 %0, [%1];" : "=r"(xb_) : "r"(base_ + (uint32_t)min(a##j, CAPJ - 1) * ENTRY_PITCH) : "memory"); \
      l##j = a##j > 0 ? __uint_as_float(lb_) : pinf;                                                \
      x##j = a##j < n##j ? __uint_as_float(xb_) : ninf;                                             \
    }
    RR_CUT(0) RR_CUT(1) RR_CUT(2) RR_CUT(3)
#undef RR_CUT
    lo = fminf(fminf(l0, l1), fminf(l2, l3));
    hi = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
    // the largest entry out cannot sit in the list of the smallest entry in (lists descend), so
    // a strict gain always moves between two different lists
    const bool move = on && hi > lo && it < max_steps;
    if (!__any_sync(0xFFFFFFFFu, move)) break;
    if (move) {
      const int jm = l0 == lo ? 0 : l1 == lo ? 1 : l2 == lo ? 2 : 3;
      const int jx = x0 == hi ? 0 : x1 == hi ? 1 : x2 == hi ? 2 : 3;
      a0 += (jx == 0) - (jm == 0); a1 += (jx == 1) - (jm == 1);
      a2 += (jx == 2) - (jm == 2); a3 += (jx == 3) - (jm == 3);
    }
  }
  return Exchange{a0, a1, a2, a3, lo, hi};
}

// ---- threshold filter of sweep 2 ------------------------------------------------------------
// One score: if it passes, {score, chunk id} goes to [w] and w moves on by one entry.  Written in
// PTX so that a score costs a compare, an id add and three predicated instructions.
//   EDGE : the tile crosses the row's last valid chunk (ids >= v never pass)
//   GUARD: the list may fill up inside this group of scores: nothing is stored at or beyond
//          w_end, but w keeps counting (the overflow is detected afterwards)
template <int I, bool EDGE, bool GUARD>
__device__ __forceinline__ void filter_one(uint32_t& w, uint32_t sbits, float tau, uint32_t col0,
                                           uint32_t v, uint32_t w_end) {
  if constexpr (!EDGE && !GUARD) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 c;\n\t"
                 "setp.ge.f32 p, %1, %2;\n\t"
                 "add.u32 c, %3, %4;\n\t"
                 "@p st.shared.v2.b32 [%0], {%1, c};\n\t"
                 "@p add.u32 %0, %0, %5;\n\t}"
                 : "+r"(w) : "f"(__uint_as_float(sbits)), "f"(tau), "r"(col0), "n"(I), "n"(ENTRY_PITCH) : "memory");
  } else if constexpr (EDGE && !GUARD) {
    asm volatile("{\n\t.reg .pred p, q;\n\t.reg .b32 c;\n\t"
                 "add.u32 c, %3, %4;\n\t"
                 "setp.lt.u32 q, c, %6;\n\t"
                 "setp.ge.and.f32 p, %1, %2, q;\n\t"
                 "@p st.shared.v2.b32 [%0], {%1, c};\n\t"
                 "@p add.u32 %0, %0, %5;\n\t}"
                 : "+r"(w) : "f"(__uint_as_float(sbits)), "f"(tau), "r"(col0), "n"(I), "n"(ENTRY_PITCH), "r"(v) : "memory");
  } else {
    asm volatile("{\n\t.reg .pred p, q, s;\n\t.reg .b32 c;\n\t"
                 "add.u32 c, %3, %4;\n\t"
                 "setp.lt.u32 q, c, %6;\n\t"
                 "setp.ge.and.f32 p, %1, %2, q;\n\t"
                 "setp.lt.and.u32 s, %0, %7, p;\n\t"
                 "@s st.shared.v2.b32 [%0], {%1, c};\n\t"
                 "@p add.u32 %0, %0, %5;\n\t}"
                 : "+r"(w) : "f"(__uint_as_float(sbits)), "f"(tau), "r"(col0), "n"(I), "n"(ENTRY_PITCH), "r"(v), "r"(w_end) : "memory");
  }
}
template <int I0, bool EDGE, bool GUARD>
__device__ __forceinline__ void filter_eight(uint32_t& w, const uint32_t (&acc)[SLICE], float tau,
                                             uint32_t col0, uint32_t v, uint32_t w_end) {
  filter_one<I0 + 0, EDGE, GUARD>(w, acc[I0 + 0], tau, col0, v, w_end);
  filter_one<I0 + 1, EDGE, GUARD>(w, acc[I0 + 1], tau, col0, v, w_end);
  filter_one<I0 + 2, EDGE, GUARD>(w, acc[I0 + 2], tau, col0, v, w_end);
  filter_one<I0 + 3, EDGE, GUARD>(w, acc[I0 + 3], tau, col0, v, w_end);
  filter_one<I0 + 4, EDGE, GUARD>(w, acc[I0 + 4], tau, col0, v, w_end);
  filter_one<I0 + 5, EDGE, GUARD>(w, acc[I0 + 5], tau, col0, v, w_end);
  filter_one<I0 + 6, EDGE, GUARD>(w, acc[I0 + 6], tau, col0, v, w_end);
  filter_one<I0 + 7, EDGE, GUARD>(w, acc[I0 + 7], tau, col0, v, w_end);
}
// A group of eight scores: the unguarded form unless some lane of the warp has fewer than eight
// free entries left.
template <int I0>
__device__ __forceinline__ void filter_group(uint32_t& w, const uint32_t (&acc)[SLICE], float tau,
                                             uint32_t col0, uint32_t v, uint32_t w_end, bool inner) {
  const bool tight = __any_sync(0xFFFFFFFFu, w + 8u * ENTRY_PITCH > w_end);
  (void)inner;   // (a separate form for tiles that no row's mask cuts measured slower: more code)
  if (tight) filter_eight<I0, true, true>(w, acc, tau, col0, v, w_end);
  else filter_eight<I0, true, false>(w, acc, tau, col0, v, w_end);
}

#ifdef RR_PHASE_TIMING
__device__ unsigned long long g_sweep_phase[32];
#define PH_T0() long long ph_t0_ = clock64()
#define PH_LAP(i) do { const long long t1_ = clock64(); if ((threadIdx.x & 31) == 0) atomicAdd(&g_sweep_phase[i], (unsigned long long)(t1_ - ph_t0_)); ph_t0_ = t1_; } while (0)
#define PH_CNT(i, val_) atomicAdd(&g_sweep_phase[i], (unsigned long long)(val_))
#else
#define PH_CNT(i, val_) do {} while (0)
#define PH_T0() do {} while (0)
#define PH_LAP(i) do {} while (0)
#endif

template <int D>
__global__ void __launch_bounds__(NT, 1)
route_sweep_kernel(RRParams p, const __nv_bfloat16* __restrict__ qc,
                   const __grid_constant__ CUtensorMap tmap_k, const int32_t* __restrict__ row_list_arg,
                   uint32_t layer, int inplace, int hooks, int cta_stride) {
  // a relay call that the forced-anchor policy turned into full routing has the identity list:
  // take the anchor's path (consecutive rows, no gathers through the list)
  const bool forced_call = row_list_arg && p.force_threshold > 0 && p.force_in[0] > 0;
  // A refresh list that holds nearly every row (high drift) is served the same way, with the
  // rows that are not on it masked out: gathering 7/8 of the rows through the list costs more
  // than sweeping the missing eighth for nothing (results per row are the same either way).
  const bool dense_refresh = row_list_arg && !forced_call && !inplace &&
                             (long long)(*p.refresh_count) * 8 >= (long long)p.rows * 7;
  const int32_t* __restrict__ row_list = (forced_call || dense_refresh) ? nullptr : row_list_arg;
  const bool force_hard = hooks & 1, force_timeout = hooks & 2;      // test hooks
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sB = smem;
  Ctl* ctl = (Ctl*)(smem + H_STAGES * C::B_HALF);
  uint8_t* s_buf = (uint8_t*)ctl + CTL_BYTES;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const CUtensorMap* const tmap_ptr = &tmap_k;   // address in parameter space (what TMA needs)
  if (tid == 0) tma_prefetch_desc(tmap_ptr);     // first thing: the descriptor fetch takes a while
#ifdef RR_PHASE_TIMING
  const long long cta_t0_ = clock64();
#endif
  // Row tiles are handed out heaviest first (under the causal mask the last tile of a problem
  // walks the most key chunks), so the tail of the grid is made of the short ones.
  const int tiles_m = p.tiles_per_problem;
  const int prob = blockIdx.x % p.P, tm = tiles_m - 1 - blockIdx.x / p.P;

  int seg_lo = 0, seg_hi = p.n_q;
  if (row_list) { seg_lo = p.problem_offsets[prob]; seg_hi = p.problem_offsets[prob + 1]; }
  if (tm * BM >= seg_hi - seg_lo) return;                 // nothing to do (uniform per CTA)

  // row of the CTA's tile -> query row of the problem and its slot (position in the refresh list,
  // or global row id); -1 = no row
  auto locate = [&](int rr, int& row_out, int& slot_out) {
    const int local = tm * BM + rr;
    row_out = -1; slot_out = 0;
    if (row_list) {
      const int s = seg_lo + local;
      if (s < seg_hi) { row_out = row_list[s] - prob * p.n_q; slot_out = s; }
    } else if (local < p.n_q) {
      row_out = local; slot_out = prob * p.n_q + local;
    }
  };
  // ---- the Qc tile goes to TMEM: the first thread of row r loads the row (two bf16 per 32-bit
  // word, as they lie in memory; refresh rows are not contiguous, so this is also the gather)
  // and stores it to TMEM lane r, where the MMA reads its A operand; rows without a query are 0.
  // The loads are issued first so that their latency overlaps the rest of the set-up.
  constexpr int QW = D / 2;                                // 32-bit words per row
  uint32_t qv[QW];
  const bool q_loader = warp >= 2 && warp < 6;
  if (q_loader) {
    int qrow, qslot;
    locate((warp & 3) * 32 + lane, qrow, qslot);
    const uint4* src = reinterpret_cast<const uint4*>(qc + ((size_t)prob * p.n_q + max(qrow, 0)) * D);
#pragma unroll
    for (int i = 0; i < QW / 4; ++i) {
      uint4 t = make_uint4(0, 0, 0, 0);
      if (qrow >= 0) t = __ldg(src + i);
      qv[4 * i] = t.x; qv[4 * i + 1] = t.y; qv[4 * i + 2] = t.z; qv[4 * i + 3] = t.w;
    }
  }
  if (tid < BM) {
    int row, slot;
    locate(tid, row, slot);
    ctl->row[tid] = row; ctl->slot[tid] = slot;
    ctl->hard_slot[tid] = -1;
  }
  if (tid == 0) {
    for (int s = 0; s < H_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    for (int s = 0; s < ACC_STAGES; ++s) {
      mbar_init(&ctl->acc_full[s], 1);
      mbar_init(&ctl->acc_empty[s], SEL_WARPS);          // one arrival per selection warp
    }
    for (int s = 0; s < ISSUE_WARPS; ++s) mbar_init(&ctl->drain[s], 1);
    ctl->abort_flag = 0;
    ctl->hard_n = 0;
    ctl->n_flagged = 0; ctl->n_cand = 0; ctl->v_flagged = 0ull;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&ctl->tmem_base, TMEM_COLS);   // (warp 0's first thread is busy with the barriers)
  // The Kc loads depend on nothing but the number of key tiles (from the tile's last row: rows
  // ascend inside a tile), and the ring's stages are all free: the producer fills the ring before
  // the CTA's first barrier, while the Qc rows are on their way.
  if (warp == 0) {
    const int last_local = min(seg_hi - seg_lo, (tm + 1) * BM) - 1;
    const int last_row = row_list ? row_list[seg_lo + last_local] - prob * p.n_q : last_local;
    const int nt0 = (rr_valid_count(last_row, p.n_k, p.causal, p.causal_offset) + BN - 1) / BN;
    if (lane == 0) {
      const int pre = min(H_STAGES, 2 * nt0 * C::KHALVES);
      for (int q = 0; q < pre; ++q) {
        mbar_expect_tx(&ctl->full[q], C::B_HALF);
        tma_load_3d(sB + q * C::B_HALF, tmap_ptr, (q % C::KHALVES) * 64, ((q / C::KHALVES) % nt0) * BN, prob, &ctl->full[q]);
      }
    }
    __syncwarp();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  int last = -1;
  for (int t = BM - 1; t >= 0; --t) if (ctl->row[t] >= 0) { last = ctl->row[t]; break; }
  const int vmax = rr_valid_count(last, p.n_k, p.causal, p.causal_offset);
  const int n_tiles = (vmax + BN - 1) / BN;
  const int pre_q = min(H_STAGES, 2 * n_tiles * C::KHALVES);
  if (q_loader) {
    const uint32_t taddr = ctl->tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + A_COL;
    if constexpr (QW == 64) tmem_st_32x64(taddr, qv); else tmem_st_32x32(taddr, qv);
    tmem_st_wait();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile uint32_t* abort_flag = &ctl->abort_flag;

  // Tiles are numbered through all sweeps (gt): stage and phase of every ring follow from gt.
  // producer / issuer: `first` .. `first + count` of that numbering
  // A stage of the Kc ring holds one K-half (64 of the d values) of a tile of 128 key chunks, so
  // that the load of a tile's first half can start as soon as the MMAs of the first half of the
  // tile two before it have finished.  Halves are numbered q = gt * KHALVES + h.
  // (halves q < skip_q have been issued already)
  auto produce = [&](int first, int count, int skip_q) {
    int issued = 0;
    for (int i = 0; i < count; ++i) {
      const int gt = first + i, t = gt % n_tiles;
#pragma unroll
      for (int h = 0; h < C::KHALVES; ++h) {
        const int q = gt * C::KHALVES + h;
        if (q < skip_q) { ++issued; continue; }
        const int s = q % H_STAGES; const uint32_t ph = (q / H_STAGES) & 1;
        if (!mbar_wait_spin(&ctl->empty[s], ph ^ 1, abort_flag)) { i = count; break; }
        mbar_expect_tx(&ctl->full[s], C::B_HALF);
        tma_load_3d(sB + s * C::B_HALF, tmap_ptr, h * 64, t * BN, prob, &ctl->full[s]);
        ++issued;
      }
    }
    // do not go on while copies into this CTA's shared memory may still be in flight
    const int q_end = first * C::KHALVES + issued;
    for (int q = max(first * C::KHALVES, q_end - H_STAGES); q < q_end; ++q) {
      const int s = q % H_STAGES; const uint32_t ph = (q / H_STAGES) & 1;
      for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->full[s], ph); ++it) __nanosleep(64);
    }
  };
  // Two threads (of two warps) issue the MMAs, tile gt by issuer gt % 2: while one is held by the
  // tensor pipe inside its tile, the other already waits for the barriers of the next tile, so the
  // pipe finds the next tile's MMAs queued when it drains.  (MMAs of different tiles write
  // different accumulators; a commit covers the MMAs of the committing thread.)
  auto issue = [&](int first, int count, int which) {
    constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
    for (int i = 0; i < count; ++i) {
      const int gt = first + i;
      if ((gt & 1) != which) continue;
      const int as = gt % ACC_STAGES; const uint32_t aph = (gt / ACC_STAGES) & 1;
#ifdef RR_PIPE_PROBE
      const long long ip0_ = clock64();
#endif
      if (!mbar_wait_spin(&ctl->acc_empty[as], aph ^ 1, abort_flag)) break;
#ifdef RR_PIPE_PROBE
      PH_CNT(9, clock64() - ip0_); PH_CNT(13, 1);
#endif
      bool ok = true;
#pragma unroll
      for (int h = 0; h < C::KHALVES; ++h) {
        const int q = gt * C::KHALVES + h;
        const int s = q % H_STAGES; const uint32_t ph = (q / H_STAGES) & 1;
#ifdef RR_PIPE_PROBE
        const long long ip1_ = clock64();
#endif
        if (!mbar_wait_spin(&ctl->full[s], ph, abort_flag)) { ok = false; break; }
#ifdef RR_PIPE_PROBE
        PH_CNT(10 + h, clock64() - ip1_);
        const long long ip2_ = clock64();
#endif
        tc_fence_after();
        const uint32_t b_addr = smem_u32(sB + s * C::B_HALF);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16_ts(tmem_base + as * BN, tmem_base + A_COL + (h * 4 + k) * 8,
                       umma_desc_k_sw128(b_addr + k * 32), idesc, (h | k) > 0 ? 1u : 0u);
        umma_commit(&ctl->empty[s]);
#ifdef RR_PIPE_PROBE
        PH_CNT(12, clock64() - ip2_);
#endif
      }
      if (!ok) break;
      umma_commit(&ctl->acc_full[as]);
    }
  };

  // ---- selection-side geometry (meaningful for warps 2..) -------------------------------------
  const int quarter = warp & 3, jslice = (warp - 2) >> 2;
  const int r = quarter * 32 + lane;                       // row inside the CTA
  const bool is_sel = warp >= 2 && warp < LAST_SEL;
  const int row = is_sel ? ctl->row[r] : -1;
  const int v = row >= 0 ? rr_valid_count(row, p.n_k, p.causal, p.causal_offset) : 0;
  const int g = row >= 0 ? (row_list ? row_list[ctl->slot[r]] : ctl->slot[r]) : 0;
  const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);
  const uint32_t buf0 = smem_u32(s_buf);
  const uint32_t row_base = buf0 + (uint32_t)r * 8u;                       // list 0, entry 0
  const uint32_t my_base = row_base + (uint32_t)jslice * LIST_PITCH;       // this thread's list
  const uint32_t acc_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(jslice * SLICE);
  int vmaxw = v, vminw = row >= 0 ? v : 0x7FFFFFFF;
#pragma unroll
  for (int off = 16; off; off >>= 1) {
    vmaxw = max(vmaxw, __shfl_xor_sync(FULL, vmaxw, off));
    vminw = min(vminw, __shfl_xor_sync(FULL, vminw, off));
  }
  bool alive = true;
  // consumer side of one tile: tile_wait returns the first column of this thread's slice, or -1
  // if no row of the warp sees the slice (or a wait gave up); tile_release hands the accumulator
  // back.  The tile bodies are written out in the loops so that their arrays stay in registers.
  auto tile_wait = [&](int gt) -> int {
    const int as = gt % ACC_STAGES; const uint32_t aph = (gt / ACC_STAGES) & 1;
    if (alive) {
      // test hook: the first wait of CTA 0 counts as expired (what a wait that ran out does:
      // raise the CTA's abort flag; every role then leaves its loop at its next poll)
      if (force_timeout && blockIdx.x == 0 && gt == 0) *abort_flag = 1u;
      const bool ready = mbar_wait_warp(&ctl->acc_full[as], aph, abort_flag, 20);
      if (!__all_sync(FULL, ready)) alive = false;
    }
    if (!alive) return -1;
    tc_fence_after();
    const int col0 = (gt % n_tiles) * BN + jslice * SLICE;
    return col0 < vmaxw ? col0 : -1;
  };
  // (one arrival per warp: hundreds of per-thread arrivals on one barrier word serialise)
  auto tile_release = [&](int gt) {
    if (!alive) return;
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&ctl->acc_empty[gt % ACC_STAGES]);
  };
  auto acc_addr = [&](int gt) -> uint32_t { return acc_lane + (uint32_t)((gt % ACC_STAGES) * BN); };

  if (warp == 0) {
    // Every Kc tile of the CTA beyond the ring is asked into L2, one prefetch per lane, BEFORE
    // the first lane starts to produce: lanes of a warp whose first lane spins on a barrier may
    // not get to run for a long time, and the hints are only worth something early.
    for (int q = pre_q + lane; q < n_tiles * C::KHALVES; q += 32)
      tma_prefetch_l2_3d(tmap_ptr, (q % C::KHALVES) * 64, (q / C::KHALVES) * BN, prob);
    __syncwarp();
    if (lane == 0) {
      produce(0, 2 * n_tiles, pre_q);
    } else {
      // The Qc rows of the CTA that will start about when this one ends (CTAs start in
      // index order as SMs fall free, one CTA per SM) are asked into L2, so that its set-up waits
      // for L2 instead of DRAM.  A hint only: nothing depends on it.
      const int nb = (int)blockIdx.x + cta_stride;
      if (nb < (int)gridDim.x) {
        const int nprob = nb % p.P, ntm = tiles_m - 1 - nb / p.P;
        int nlo = 0, nhi = p.n_q;
        if (row_list) { nlo = p.problem_offsets[nprob]; nhi = p.problem_offsets[nprob + 1]; }
        for (int i = lane - 1; i < BM; i += 31) {
          const int local = ntm * BM + i;
          if (local >= nhi - nlo) break;
          const size_t grow = row_list ? (size_t)row_list[nlo + local] : (size_t)nprob * p.n_q + local;
          const char* src = reinterpret_cast<const char*>(qc + grow * D);
#pragma unroll
          for (int b = 0; b < D * 2; b += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(src + b));
        }
      }
    }
    __syncwarp();
  } else if (!is_sel) {
    if (lane == 0) issue(0, 2 * n_tiles, warp == 1 ? 0 : 1);
    __syncwarp();
  } else {
    PH_T0();
#ifdef RR_PHASE_TIMING
    if (lane == 0) PH_CNT(7, ph_t0_ - cta_t0_);
#endif
    // ===== sweep 1: group maxima -> tau ==========================================================
    // In-place relay (Section 3.2 on the same score strip): every thread also dumps its scores of
    // the tile to shared memory ([column][row], two tiles in the still unused list area), and after
    // a barrier of the row's four threads looks up the current scores of its share of the row's
    // candidates: alpha = min over route slots, beta = max over sentinel slots (Eq. 5).
    int cid[MAX_SLOTS];
    const int slots = (p.c + TPR - 1) / TPR, slot0 = jslice * slots;
    float a_part = pinf, b_part = ninf;
    int n_cand = 0; bool bad_id = false;
    if (inplace) {
#pragma unroll
      for (int q = 0; q < MAX_SLOTS; ++q) {
        const int sl = slot0 + q;
        int id = -1;
        if (row >= 0 && q < slots && sl < p.c)
          id = sl < p.k ? p.routes[(size_t)g * p.k + sl] : p.sentinels[(size_t)g * p.sw + (sl - p.k)];
        bad_id |= id >= v;
        cid[q] = id >= 0 && id < v ? id : -1;
        n_cand += cid[q] >= 0;
        if (p.debug && row >= 0 && q < slots && sl < p.c)
          p.cand_scores[(size_t)g * p.c + sl] = __int_as_float(0x7fc00000);
      }
    }
    float mx[SLICE];
#pragma unroll
    for (int i = 0; i < SLICE; ++i) mx[i] = ninf;
    for (int t = 0; t < n_tiles; ++t) {
      const int col0 = tile_wait(t);
      if (col0 >= 0) {
        uint32_t acc[SLICE];
        tmem_ld_32x32(acc_addr(t), acc);
        if (col0 + SLICE <= vminw) {
#pragma unroll
          for (int i = 0; i < SLICE; ++i) mx[i] = fmaxf(mx[i], __uint_as_float(acc[i]));
        } else {
#pragma unroll
          for (int i = 0; i < SLICE; ++i)
            mx[i] = col0 + i < v ? fmaxf(mx[i], __uint_as_float(acc[i])) : mx[i];
        }
        if (inplace) {
          const uint32_t dump = buf0 + (uint32_t)(t & 1) * (BN * BM * 4u) + (uint32_t)(jslice * SLICE) * (BM * 4u) + (uint32_t)r * 4u;
#pragma unroll
          for (int i = 0; i < SLICE; ++i) sts32(dump + (uint32_t)i * (BM * 4u), acc[i]);
        }
      }
      tile_release(t);
      if (inplace) {
        quarter_sync(quarter);
        const uint32_t tile_dump = buf0 + (uint32_t)(t & 1) * (BN * BM * 4u) + (uint32_t)r * 4u;
#pragma unroll
        for (int q = 0; q < MAX_SLOTS; ++q) {
          const int id = cid[q];
          if (id >= 0 && (id >> 7) == t) {
            const float sc = __uint_as_float(lds32(tile_dump + (uint32_t)(id & (BN - 1)) * (BM * 4u)));
            if (slot0 + q < p.k) a_part = fminf(a_part, sc); else b_part = fmaxf(b_part, sc);
            if (p.debug) p.cand_scores[(size_t)g * p.c + slot0 + q] = sc;
          }
        }
      }
    }
    if (inplace) {
      ctl->ab[0][jslice][r] = a_part; ctl->ab[1][jslice][r] = b_part;
      if (__any_sync(FULL, bad_id) && lane == 0) atomicOr(p.status, RR_STATUS_BAD_INDEX);
      n_cand = __reduce_add_sync(FULL, n_cand);
      if (lane == 0) atomicAdd(&ctl->n_cand, (uint32_t)n_cand);
      // every selection warp of the CTA has read its last dump: the list area (which the dumps of
      // all quarters share) is free
      asm volatile("bar.sync 5, %0;" ::"n"(SEL_WARPS * 32) : "memory");
    }
    PH_LAP(0);
    OESort<0, SLICE, float, DescF<float>, SLICE>::run(mx);
    // The row's keep-th largest group maximum (over the 128 groups of its four threads) has keep
    // distinct scores of the row at or above it: a valid inclusive lower bound of the row's
    // keep-th largest score, and the tightest one the maxima give (about 1.2 keep scores pass;
    // an even split of keep over the four threads would let 1.5 keep pass, and lists overflow).
    // Each thread publishes its sorted maxima in the score words of its (still empty) list; the
    // first thread of the row finds the split by exchange (exchange_select).  Rows that fit one
    // tile keep everything (their lists cannot overflow).
#pragma unroll
    for (int i = 0; i < SLICE; ++i) sts32(my_base + (uint32_t)i * ENTRY_PITCH, __float_as_uint(mx[i]));
    PH_LAP(8);
    quarter_sync(quarter);
    PH_LAP(9);
    float tau = ninf;
    if (jslice == 0) {          // one thread per row searches; the others wait at the barrier
      const int keep_cfg_ = p.k + max(p.m, 1);
      const bool bounded = row >= 0 && v >= BN;              // v >= 128 > keep: all 128 groups exist
      const int q_ = keep_cfg_ / TPR, rm_ = keep_cfg_ % TPR;
      const Exchange ex = exchange_select(row_base, SLICE, SLICE, SLICE, SLICE, q_ + (0 < rm_),
                                          q_ + (1 < rm_), q_ + (2 < rm_), q_, bounded, MAX_KEEP);
      if (bounded) tau = ex.lo;
      ctl->tau_row[r] = tau;
      if (inplace) {
        // challenge test of the row (Eq. 5 and the optional policies): only rows that fail it are
        // routed again; the others keep their ledger row
        const float alpha = fminf(fminf(ctl->ab[0][0][r], ctl->ab[0][1][r]), fminf(ctl->ab[0][2][r], ctl->ab[0][3][r]));
        const float beta = fmaxf(fmaxf(ctl->ab[1][0][r], ctl->ab[1][1][r]), fmaxf(ctl->ab[1][2][r], ctl->ab[1][3][r]));
        const bool flag = row >= 0 && rr_challenge(p, g, alpha, beta);
        ctl->live[r] = flag;
        if (row >= 0) { p.flags[g] = flag ? 1 : 0; p.alpha[g] = alpha; p.beta[g] = beta; }
        const int n_flag = __popc(__ballot_sync(FULL, flag));
        const int v_sum = __reduce_add_sync(FULL, flag ? v : 0);
        if (lane == 0) {
          atomicAdd(&ctl->n_flagged, (uint32_t)n_flag);
          atomicAdd(&ctl->v_flagged, (unsigned long long)v_sum);
        }
      }
    }
    PH_LAP(10);
    quarter_sync(quarter);                  // the published maxima have been read: lists are free
    tau = ctl->tau_row[r];
    const bool routed = row >= 0 && (!inplace || ctl->live[r] != 0) &&      // this row is (re)routed here
                        (!dense_refresh || p.flags[g] != 0);
    if (!routed) tau = pinf;                               // padding / reused rows pass nothing
    PH_LAP(1);

    // ===== sweep 2: threshold filter into this thread's list ====================================
    uint32_t waddr = my_base;
    const uint32_t wend = my_base + (uint32_t)CAPJ * ENTRY_PITCH;
    for (int t = 0; t < n_tiles; ++t) {
      const int col0 = tile_wait(n_tiles + t);
      if (col0 >= 0) {
        uint32_t acc[SLICE];
        tmem_ld_32x32(acc_addr(n_tiles + t), acc);
        const bool inner = col0 + SLICE <= vminw;
        filter_group<0>(waddr, acc, tau, (uint32_t)col0, (uint32_t)v, wend, inner);
        filter_group<8>(waddr, acc, tau, (uint32_t)col0, (uint32_t)v, wend, inner);
        filter_group<16>(waddr, acc, tau, (uint32_t)col0, (uint32_t)v, wend, inner);
        filter_group<24>(waddr, acc, tau, (uint32_t)col0, (uint32_t)v, wend, inner);
      }
      tile_release(n_tiles + t);
    }
    PH_LAP(2);
    const int n_raw = (int)((waddr - my_base) / ENTRY_PITCH);
    bool slow = n_raw > CAPJ;                              // the list overflowed
    const int n = min(n_raw, CAPJ);

    // ===== sort the list (network sized for the longest list of the warp; a third, smaller size
    // cost more in code than it saved in compare-exchanges) ========================================
    {
      const int n_warp = __reduce_max_sync(FULL, n);
      bool run3;
      if (n_warp <= 24) run3 = sort_list<24>(my_base, n);
      else run3 = sort_list<32>(my_base, n);
      slow |= run3;
    }
#ifdef RR_PHASE_COUNTS
    if (row >= 0 && n_raw > CAPJ) PH_CNT(17, 1);
    if (row >= 0 && slow && n_raw <= CAPJ) PH_CNT(18, 1);
    if (row >= 0) { PH_CNT(22, n_raw); PH_CNT(23, 1); }
#endif
    if (force_hard && routed && g % 5 == 0) slow = true;     // test hook: exercise the slow path
    ctl->cnt[jslice][r] = (uint32_t)n | (slow ? 256u : 0u);
    PH_LAP(3);
    quarter_sync(quarter);

    // ===== cuts: how many entries of each sorted list belong to the row's top k / top keep ======
    // Thread 0 of a row finds the cut for k, thread 1 the cut for keep, each by exchange: from a
    // split proportional to the list lengths, one entry at a time leaves the list whose last
    // selected entry is the smallest and enters from the list whose next entry is the largest,
    // while the latter is larger.  At the end every selected score is >= lo = the T-th largest and
    // every other one <= hi; lo > hi settles the set exactly, lo == hi (equal scores across the
    // cut) is left to the slow path.  The k cut also yields the k-th score (lo) and the margin.
    const uint32_t c0 = ctl->cnt[0][r], c1 = ctl->cnt[1][r], c2 = ctl->cnt[2][r], c3 = ctl->cnt[3][r];
    const bool have = alive && routed;
    const bool hard_list = have && ((c0 | c1 | c2 | c3) & 256u) != 0u;
    const bool go0 = have && !hard_list;
    const int n_total = (int)((c0 & 255u) + (c1 & 255u) + (c2 & 255u) + (c3 & 255u));
    const int keep_cfg = p.k + max(p.m, 1);
    const int keep_row0 = go0 ? min(keep_cfg, v) : 0, kk0 = go0 ? min(p.k, v) : 0;
    float kth = pinf, next = ninf;
    if (jslice < 2 && (jslice == 0 || p.m > 0)) {
      const int T = jslice == 0 ? kk0 : keep_row0;
      const int n0 = (int)(c0 & 255u), n1 = (int)(c1 & 255u), n2 = (int)(c2 & 255u), n3 = (int)(c3 & 255u);
      const int nt = max(n_total, 1);
      int a0 = T * n0 / nt, a1 = T * n1 / nt, a2 = T * n2 / nt, a3 = T * n3 / nt;
      int rem = T - (a0 + a1 + a2 + a3);
#pragma unroll
      for (int pass = 0; pass < 3; ++pass) {
        if (rem > 0 && a0 < n0) { ++a0; --rem; }
        if (rem > 0 && a1 < n1) { ++a1; --rem; }
        if (rem > 0 && a2 < n2) { ++a2; --rem; }
        if (rem > 0 && a3 < n3) { ++a3; --rem; }
      }
      const Exchange ex = exchange_select(row_base, n0, n1, n2, n3, a0, a1, a2, a3, T > 0, 2 * MAX_KEEP + 1);
      a0 = ex.a0; a1 = ex.a1; a2 = ex.a2; a3 = ex.a3;
      const float lo = ex.lo, hi = ex.hi;
      // not settled: scores tie across the cut, or the exchange ran out of steps
      const bool unsettled = T > 0 && !(lo > hi);
      const uint32_t cut4 = (uint32_t)a0 | ((uint32_t)a1 << 8) | ((uint32_t)a2 << 16) | ((uint32_t)a3 << 24);
      if (jslice == 0) { ctl->cut_k[r] = cut4; ctl->cut_bad[0][r] = unsettled; kth = lo; next = hi; }
      else { ctl->cut_keep[r] = cut4; ctl->cut_bad[1][r] = unsettled; }
#ifdef RR_PHASE_COUNTS
      if (unsettled) PH_CNT(19 + jslice, 1);
#endif
    }
    PH_LAP(4);
    quarter_sync(quarter);
    const bool hard = have && (hard_list || ctl->cut_bad[0][r] || (p.m > 0 && ctl->cut_bad[1][r]));
    const bool go = have && !hard;
    const int keep_row = go ? keep_row0 : 0, kk = go ? kk0 : 0;
    const int n_near = p.m > 0 ? keep_row - kk : 0;
    if (jslice == 0 && hard) {
      const uint32_t idx = atomicAdd(&ctl->hard_n, 1u);
      ctl->hard_rows[idx] = (uint8_t)r;
      ctl->hard_slot[r] = (int8_t)idx;
    }

    // ===== every thread: its own share of the route and the near-miss sentinels ===================
    const uint32_t ck4 = ctl->cut_k[r];
    const uint32_t cd4 = p.m > 0 ? ctl->cut_keep[r] : ck4;
    const int my_k = go ? (int)((ck4 >> (8 * jslice)) & 255u) : 0;
    const int my_d = go ? (int)((cd4 >> (8 * jslice)) & 255u) : 0;
    int off_k = 0, off_n = 0;
#pragma unroll
    for (int j = 0; j < TPR; ++j) {
      const int ckj = (int)((ck4 >> (8 * j)) & 255u), cdj = (int)((cd4 >> (8 * j)) & 255u);
      off_k += j < jslice ? ckj : 0;
      off_n += j < jslice ? cdj - ckj : 0;
    }
    // staging area of the CTA's outputs = the Kc ring (idle once the last tile of sweep 2 has
    // been consumed; the slow path only starts behind the CTA-wide barrier): word o of row r at
    // [o][r]; route ids in words [0, k), near-miss ids in [k, k+m).  Each thread moves the ids of
    // its own entries.
    const uint32_t stage_row = smem_u32(sB) + (uint32_t)r * 4u;
    auto stage_addr = [&](int o) -> uint32_t { return stage_row + (uint32_t)o * (BM * 4u); };
    {
      const int my_d_max = __reduce_max_sync(FULL, my_d);
#pragma unroll 1
      for (int e0 = 0; e0 < my_d_max; e0 += 4) {
        uint32_t id[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) id[u] = lds32(my_base + (uint32_t)min(e0 + u, CAPJ - 1) * ENTRY_PITCH + 4u);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int e = e0 + u;
          const int o = e < my_k ? off_k + e : p.k + off_n + (e - my_k);
          if (e < my_d) sts32(stage_addr(o), id[u]);
        }
      }
    }
    quarter_sync(quarter);
    // copy-out: thread j owns words [16j, 16j+16) of the staging area; 16-byte stores where the
    // ledger rows allow, -1 in the slots the row cannot fill
    if (go) {
      int32_t* route = p.routes + (size_t)g * p.k;
      int32_t* sent = p.sentinels + (size_t)g * p.sw;
      const bool vec = ((p.k | p.m | p.sw) & 3) == 0;
      auto word = [&](int o) -> int {
        const bool ok = o < kk || (o >= p.k && o < p.k + n_near);
        const int val = (int)lds32(stage_addr(o));
        return ok ? val : -1;
      };
      for (int o = 16 * jslice; o < 16 * jslice + 16 && o < p.k + p.m; o += 4) {
        if (vec) {
          const int4 q4 = make_int4(word(o), word(o + 1), word(o + 2), word(o + 3));
          if (o < p.k) *reinterpret_cast<int4*>(route + o) = q4;
          else *reinterpret_cast<int4*>(sent + (o - p.k)) = q4;
        } else {
          for (int t = o; t < o + 4 && t < p.k + p.m; ++t) {
            if (t < p.k) route[t] = word(t); else sent[t - p.k] = word(t);
          }
        }
      }
    }
    if (jslice == 0 && go) {
      p.kth[g] = kth;
      p.margin[g] = v > kk ? kth - next : pinf;
    }
    PH_LAP(5);
    PH_LAP(6);
  }

  // ===== slow path: rows the lists could not settle =============================================
  // One more sweep per batch of HARD_SLOTS rows stores their complete score rows (as order
  // keys) over the list area; a warp per row then runs the exact radix select on them.
  __syncthreads();
  const int n_hard = ctl->abort_flag ? 0 : (int)ctl->hard_n;
  if (tid == 0) { PH_CNT(16, n_hard); PH_CNT(21, n_hard > 0 ? 1 : 0); }
  int next_gt = 2 * n_tiles;
  for (int done = 0; done < n_hard; done += HARD_SLOTS) {
    // barrier: the previous batch's rows and scratch are free again; the vote makes the
    // decision to stop after a timed-out wait the same for every thread
    if (__syncthreads_or((int)ctl->abort_flag)) break;
    if (warp == 0) {
      if (lane == 0) produce(next_gt, n_tiles, 0);
      __syncwarp();
    } else if (!is_sel) {
      if (lane == 0) issue(next_gt, n_tiles, warp == 1 ? 0 : 1);
      __syncwarp();
    } else {
      const int hs = row >= 0 ? (int)ctl->hard_slot[r] - done : -1;
      const bool mine = hs >= 0 && hs < HARD_SLOTS;
      const uint32_t srow = buf0 + (uint32_t)max(hs, 0) * (MAX_NK * 4u);
      for (int t = 0; t < n_tiles; ++t) {
        const int col0 = tile_wait(next_gt + t);
        if (col0 >= 0 && __any_sync(FULL, mine)) {
          uint32_t acc[SLICE];
          tmem_ld_32x32(acc_addr(next_gt + t), acc);
#pragma unroll
          for (int i = 0; i < SLICE; ++i)
            if (mine && col0 + i < v)
              sts32(srow + (uint32_t)(col0 + i) * 4u, rr_order_key(__uint_as_float(acc[i])));
        }
        tile_release(next_gt + t);
      }
    }
    next_gt += n_tiles;
    __syncthreads();
    if (is_sel && !ctl->abort_flag) {
      const int sw = warp - 2;
      uint32_t* scratch = (uint32_t*)(s_buf + HARD_SLOTS * MAX_NK * 4) + sw * (256 + BM_WORDS);
      for (int hs = sw; hs < HARD_SLOTS && done + hs < n_hard; hs += SEL_WARPS) {
        const int rr = ctl->hard_rows[done + hs];
        const int hrow = ctl->row[rr];
        const int hv = rr_valid_count(hrow, p.n_k, p.causal, p.causal_offset);
        const int hg = row_list ? row_list[ctl->slot[rr]] : ctl->slot[rr];
        const uint32_t* keys = (const uint32_t*)(s_buf + (size_t)hs * MAX_NK * 4);
        warptopk::route_row(p, keys, scratch, scratch + 256, hg, hv, layer, lane);
        __syncwarp();
      }
    }
  }

  // TMEM must not be freed while an MMA can still write to it: after a wait that gave up the
  // consumers no longer vouch for that, so each issuer waits (bounded) for its own MMAs
  // (when no wait gave up, every issued tile has been waited for by the consumers: nothing is pending)
  if (!is_sel && warp != 0 && lane == 0 && ctl->abort_flag) {
    const int which = warp == 1 ? 0 : 1;
    umma_commit(&ctl->drain[which]);
    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->drain[which], 0); ++it) __nanosleep(64);
  }
  tc_fence_before();
  __syncthreads();
#ifdef RR_PHASE_TIMING
  if (tid == 0) { PH_CNT(14, clock64() - cta_t0_); PH_CNT(15, 1); }
#endif
  if (warp == 1) {                                         // the warp that allocated
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (warp == 0) {
    if (lane == 0 && ctl->abort_flag) atomicOr(p.status, RR_STATUS_TIMEOUT);
    if (lane == 0 && inplace) {      // what the compaction kernel and the work counters need
      p.tile_counts[prob * tiles_m + tm] = (int)ctl->n_flagged;
      atomicAdd(&p.counters[RR_CNT_FLAGGED_ROWS], (unsigned long long)ctl->n_flagged);
      atomicAdd(&p.counters[RR_CNT_CAND_PAIRS], (unsigned long long)ctl->n_cand);
      atomicAdd(&p.counters[RR_CNT_FULL_PAIRS], ctl->v_flagged);
    }
  }
}

size_t smem_bytes(int d) {
  (void)d;
  return 1024 + (size_t)H_STAGES * BN * 128 + CTL_BYTES + BUF_BYTES;
}

}  // namespace

#ifdef RR_PHASE_TIMING
extern "C" int rr_debug_sweep_phase_counters(unsigned long long* out32, int reset) {
  cudaDeviceSynchronize();
  if (cudaMemcpyFromSymbol(out32, g_sweep_phase, sizeof(unsigned long long) * 32) != cudaSuccess) return -1;
  if (reset) {
    unsigned long long z[32] = {};
    cudaMemcpyToSymbol(g_sweep_phase, z, sizeof z);
  }
  return 0;
}
#endif

// What the two-sweep kernel is built for: bf16 inputs, keep = k + max(m,1) <= 48 (four lists of
// 32 entries per row hold about 1.4 keep survivors), at most 1024 key chunks (exclusion bitmap
// of 32 words per row, slow-path score rows of 4 KB).
bool rr_route_sweep_supported(const RRParams& p) {
  const int keep = p.k + (p.m > 0 ? p.m : 1);
  return p.dtype == RR_BF16 && (p.d == 64 || p.d == 128) && keep <= MAX_KEEP && p.n_k <= MAX_NK &&
         smem_bytes(p.d) <= 227 * 1024;
}

// The in-place relay holds a row's candidates in 16 registers of each of its four threads.
bool rr_route_sweep_inplace_supported(const RRParams& p) {
  return rr_route_sweep_supported(p) && p.c <= TPR * MAX_SLOTS;
}

cudaError_t rr_launch_route_sweep(const RRParams& p, const void* qc, const void* kc,
                                  const int32_t* row_list, int layer, int inplace, int hooks,
                                  cudaStream_t st) {
  if (inplace && (row_list || p.c > TPR * MAX_SLOTS)) return cudaErrorInvalidConfiguration;
  if (!rr_route_sweep_supported(p)) return cudaErrorInvalidConfiguration;
  CUtensorMap tmap;
  cudaError_t e = rr_encode_tmap_bf16_3d(&tmap, kc, p.d, p.n_k, p.P, BN);
  if (e != cudaSuccess) return e;
  const int grid = p.P * p.tiles_per_problem;
  static unsigned long long attr_done = 0;      // devices on which the attributes are set
  e = rr_once_per_device(attr_done, [] {
    cudaError_t a = cudaFuncSetAttribute(route_sweep_kernel<128>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (a != cudaSuccess) return a;
    return cudaFuncSetAttribute(route_sweep_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                227 * 1024);
  });
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 148;                     // CTAs resident at a time: one per SM
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const __nv_bfloat16* q = (const __nv_bfloat16*)qc;
  const size_t smem = smem_bytes(p.d);
  if (p.d == 128)
    route_sweep_kernel<128><<<grid, NT, smem, st>>>(p, q, tmap, row_list, (uint32_t)layer, inplace, hooks, sms);
  else
    route_sweep_kernel<64><<<grid, NT, smem, st>>>(p, q, tmap, row_list, (uint32_t)layer, inplace, hooks, sms);
  rr_count_launch();
  return cudaPeekAtLastError();
}
