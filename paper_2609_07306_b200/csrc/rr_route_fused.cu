// Full routing of a set of rows in ONE kernel: score GEMM on the tensor cores (Eq. 1), per-row
// TopK (Eq. 2), near-miss sentinels (Section 3.1 item 1), k-th score and margin (Section 3.3),
// random sentinels (Section 3.1 item 2) -- the score matrix never leaves the SM.
//
// One CTA owns 128 query rows of one problem (consecutive rows at an anchor; a segment of the
// compacted refresh list at a relay, Section 4.2) and walks the key chunks in tiles of 64,
// stopping at the last chunk any of its rows may select.
//   warp 0   : TMA producer (Kc tiles, 128-byte swizzle, one stage -- the selection is the slow
//              side, so the shared memory goes to the candidate buffers --, no multicast)
//   warp 1   : one thread issues tcgen05.mma (M=128, N=64, K=16) into a ring of 4 TMEM
//              accumulators
//   warps 2-5: selection, ONE THREAD PER QUERY ROW (tcgen05.ld 32x32b hands each thread 32
//              consecutive scores of its own row).  Each thread streams its row through a
//              threshold filter into a private candidate buffer in shared memory ({score,
//              chunk id} entries laid out [slot][thread]: bank-conflict free).  When a buffer
//              nears its capacity the warp re-tightens with a persistent 32-bin histogram of
//              the buffered scores: the bin holding rank KEEP = k + max(m,1) is found, entries
//              below it are dropped in place (stable, so entries stay in ascending chunk id)
//              and the threshold moves to the smallest survivor.  After the last tile the bins
//              of rank KEEP and rank k are located together on a second map laid over the
//              stretch between them, the scores of those two bins are copied to short side
//              lists and the exact ranks found there by counting; the cut is applied by the
//              output pass.  Crowded bins, unusable ranges and wide bitmaps take the older
//              way: top-2 / bottom-2 tracking, zoom levels, a key-space radix level for ranges
//              too narrow to scale.  Ties go to the smaller chunk id.
// Random sentinels are drawn by the same thread with the counter-based generator, using a
// per-row bitmap of excluded chunks in shared memory.  Every mbarrier wait is bounded.
#include "rr_common.cuh"
#include "rr_sm100.cuh"

using namespace sm100;

namespace {

constexpr int BM = 128, BN = 64, B_STAGES = 1, ACC_STAGES = 4, NT = 192;
constexpr int A_COL = ACC_STAGES * BN;          // the Qc tile sits in TMEM behind the accumulators
constexpr int TMEM_COLS = 512;                 // 4 x 64 accumulator columns + up to 64 of Qc, power of 2
constexpr int NB = 32, NB_LOG = 5;             // histogram bins per level
constexpr int CHUNK = 32;                      // scores handed to a thread per TMEM load
constexpr unsigned FULL = 0xFFFFFFFFu;

template <int D>
struct Cfg {
  static constexpr int KHALVES = D / 64, KSTEPS = D / 16;
  static constexpr int A_BYTES = BM * D * 2, B_BYTES = BN * D * 2;
  static constexpr int A_HALF = BM * 128, B_HALF = BN * 128;   // rows x 128 bytes (64 bf16)
  static constexpr int CTL_BYTES = 2048;
  static constexpr int FIXED_BYTES = 1024 + B_STAGES * B_BYTES + CTL_BYTES;
};

struct Ctl {
  uint64_t full[B_STAGES], empty[B_STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
  uint32_t tmem_base, abort_flag;
  int row[BM], slot[BM];
};

// ---- thread-private selection state ---------------------------------------------------------
// A row's candidate buffer holds 8-byte entries {score bits, chunk id}; entry e of the thread
// that owns row r lives at buf + e*ENTRY_PITCH (ENTRY_PITCH = 128 rows * 8 bytes), so a warp's
// accesses to "entry e_lane" are bank-conflict free whatever e_lane is.  Histogram bins and
// the exclusion bitmap are 32-bit words at aux + b*AUX_PITCH.  All accesses use explicit
// shared-window addresses (32-bit) and ld/st/red.shared.
constexpr uint32_t ENTRY_PITCH = BM * 8, AUX_PITCH = BM * 4;
struct Sel { uint32_t buf, aux; };

// Optional self-check (compile with -DRR_BOUNDS_CHECK): a shared-window address beyond the
// CTA's allocation is recorded (first offender wins) and the access is skipped.
#ifdef RR_BOUNDS_CHECK
__device__ unsigned int g_oob[4];
__device__ __forceinline__ bool oob(uint32_t addr, unsigned code) {
  if (addr < 233472u) return false;
  if (atomicCAS(&g_oob[0], 0u, code) == 0u) { g_oob[1] = addr; g_oob[2] = blockIdx.x; g_oob[3] = threadIdx.x; }
  return true;
}
#define RR_OOB(addr, code) if (oob(addr, code)) return
#define RR_OOB_V(addr, code, val) if (oob(addr, code)) return val
#else
#define RR_OOB(addr, code) do {} while (0)
#define RR_OOB_V(addr, code, val) do {} while (0)
#endif

__device__ __forceinline__ void st_entry(uint32_t addr, float s, uint32_t id) {
  RR_OOB(addr, 1);
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "f"(s), "r"(id) : "memory");
}
__device__ __forceinline__ void ld_entry(uint32_t addr, float& s, uint32_t& id) {
  s = 0.f; id = 0;
  RR_OOB(addr, 2);
  asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=f"(s), "=r"(id) : "r"(addr) : "memory");
}
__device__ __forceinline__ float ld_score(uint32_t addr) {
  RR_OOB_V(addr, 3, 0.f);
  float s;
  asm volatile("ld.shared.b32 %0, [%1];" : "=f"(s) : "r"(addr) : "memory");
  return s;
}
__device__ __forceinline__ uint32_t aux_ld(uint32_t addr) {
  RR_OOB_V(addr, 4, 0u);
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void aux_st(uint32_t addr, uint32_t v) {
  RR_OOB(addr, 5);
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void aux_inc(uint32_t addr) {
  asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}
// predicated forms: no branch is emitted, the access is simply masked off
__device__ __forceinline__ void st_entry_if(bool pred, uint32_t addr, float s, uint32_t id) {
  if (pred) { RR_OOB(addr, 6); }
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %3, 0;\n\t@p st.shared.v2.b32 [%0], {%1, %2};\n\t}"
               ::"r"(addr), "f"(s), "r"(id), "r"((uint32_t)pred) : "memory");
}
__device__ __forceinline__ void aux_inc_if(bool pred, uint32_t addr) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p red.shared.add.u32 [%0], 1;\n\t}"
               ::"r"(addr), "r"((uint32_t)pred) : "memory");
}
__device__ __forceinline__ void aux_or(uint32_t addr, uint32_t bits) {
  asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(addr), "r"(bits) : "memory");
}

// Histogram update for a batch of entries.  The bins are private to the thread, so a plain
// load / add / store would do, but a chain of those is serialised by the shared-memory round
// trip of each load; shared-memory reductions measured several times slower still.  Here the
// counts of HG entries are loaded together and entries that fall into the same bin are chained
// in registers (a later store to the same word then carries the running total).
constexpr int HG = 4;
__device__ __forceinline__ void hist_add(uint32_t aux, const int (&b)[8], const uint32_t (&inc)[8]) {
#pragma unroll
  for (int g0 = 0; g0 < 8; g0 += HG) {
    uint32_t a[HG], c[HG];
#pragma unroll
    for (int i = 0; i < HG; ++i) { a[i] = aux + (uint32_t)b[g0 + i] * AUX_PITCH; c[i] = aux_ld(a[i]); }
    uint32_t tot[HG];
#pragma unroll
    for (int i = 0; i < HG; ++i) {
      uint32_t base = c[i];
#pragma unroll
      for (int h = 0; h < i; ++h) base = a[h] == a[i] ? tot[h] : base;   // the latest match wins
      tot[i] = base + inc[g0 + i];
      aux_st(a[i], tot[i]);
    }
  }
}

// All passes over a buffer walk it in batches of 8 with the loads issued first: a thread's
// passes are chains of shared-memory accesses, and with one selection warp per scheduler
// nothing else hides that latency.  Histogram increments are fire-and-forget reductions.
//
// Control flow is kept WARP-UNIFORM: every routine below is called by all 32 lanes, loops run
// to the warp-wide maximum trip count and each lane masks its own tail, and data-dependent
// decisions (another refinement level, the key-space fallback) are taken by warp vote.  Lanes
// that have nothing to do pass n = 0.  Divergent versions of the same passes executed each
// pass once per divergent lane group and were several times slower.
constexpr int BATCH = 8;

// Optional phase timing (compile with -DRR_PHASE_TIMING): cycles and event counts per phase,
// summed over selection warps (lane 0), read back with rr_debug_phase_counters().
#ifdef RR_PHASE_TIMING
__device__ unsigned long long g_phase[16];
#define PH_T0() const long long ph_t0_ = clock64()
#define PH_ADD(i) do { if ((threadIdx.x & 31) == 0) atomicAdd(&g_phase[i], (unsigned long long)(clock64() - ph_t0_)); } while (0)
#define PH_CNT(i, val_) do { if ((threadIdx.x & 31) == 0) atomicAdd(&g_phase[i], (unsigned long long)(val_)); } while (0)
#else
#define PH_T0() do {} while (0)
#define PH_ADD(i) do {} while (0)
#define PH_CNT(i, val_) do {} while (0)
#endif

__device__ __forceinline__ int warp_max(int x) { return __reduce_max_sync(FULL, x); }

// order-preserving key of a score (-0.0 and +0.0 share a key; float compares already agree)
__device__ __forceinline__ uint32_t key_of(float s) {
  const uint32_t u = __float_as_uint(s + 0.0f);           // -0.0 -> +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Finds, in the histogram the lane just built, the bin that holds its need-th largest entry.
__device__ __forceinline__ void scan_bins(const Sel& s, int need, int& bsel, int& cnt, int& above) {
  uint32_t h[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) h[b] = aux_ld(s.aux + b * AUX_PITCH);
  int cum = 0; bsel = 0; cnt = 0; above = 0; bool found = false;
#pragma unroll
  for (int b = NB - 1; b >= 0; --b) {
    const int c = (int)h[b];
    if (!found && cum + c >= need) { bsel = b; cnt = c; above = cum; found = true; }
    cum += c;
  }
}
__device__ __forceinline__ void clear_bins(const Sel& s) {
#pragma unroll
  for (int b = 0; b < NB; ++b) aux_st(s.aux + b * AUX_PITCH, 0u);
}
// Lanes that only tag along in a warp-uniform routine must keep their persistent bins.
__device__ __forceinline__ void clear_bins_if(bool pred, const Sel& s) {
  if (pred) clear_bins(s);
}

// What a narrowing pass learns about the bin that holds the wanted rank: how many entries it
// has, how many in-range entries outrank it, and its two largest / two smallest scores --
// enough to finish exactly, without another level, whenever the bin has at most 4 entries.
struct BinInfo {
  int cnt, above;
  float mx1, mx2, mn2, mn1;          // mx1 >= mx2 >= ... >= mn2 >= mn1 (bin bounds: mn1, mx1)
  __device__ __forceinline__ void reset() {
    mx1 = mx2 = __int_as_float(0xff800000); mn1 = mn2 = __int_as_float(0x7f800000);
  }
  __device__ __forceinline__ void track(bool tgt, float v) {
    const float vm = tgt ? v : __int_as_float(0xff800000);
    mx2 = fmaxf(mx2, fminf(mx1, vm)); mx1 = fmaxf(mx1, vm);
    const float vn = tgt ? v : __int_as_float(0x7f800000);
    mn2 = fminf(mn2, fmaxf(mn1, vn)); mn1 = fminf(mn1, vn);
  }
  // rank r (1-based from the top) inside the bin, cnt <= 4 or all entries equal.
  __device__ __forceinline__ bool resolve(int r, float& s_T, int& need) const {
    if (mx1 == mn1) { s_T = mx1; need = r; return true; }
    if (cnt > 4) return false;
    const float l0 = mx1, l1 = cnt == 2 ? mn1 : mx2, l2 = cnt == 3 ? mn1 : mn2, l3 = mn1;
    s_T = r == 1 ? l0 : r == 2 ? l1 : r == 3 ? l2 : l3;
    const int g = (l0 > s_T) + (cnt > 1 && l1 > s_T) + (cnt > 2 && l2 > s_T) + (cnt > 3 && l3 > s_T);
    need = r - g;
    return true;
  }
};

// One refinement level in the SCORE domain over the lane's entries with lo <= score <= hi:
// NB equal-width bins (bin = floor((score - lo) * scale), monotone in the score; equal-width
// bins of the 32-bit keys would be useless across a sign change or several binades).  Finds
// the bin b* holding the rank-th largest in-range entry, the number of in-range entries above
// b* and the score bounds [blo, bhi] of the entries in b*.  With `drop`, entries below b* (and
// below lo) are removed, stably and in place, and n is updated.
// Returns false, changing nothing, for lanes with n = 0 or an unusable range.
__device__ __forceinline__ bool lin_level(const Sel& s, int& n, int nw, float lo, float hi, int rank,
                                          bool drop, BinInfo& bi) {
  const float scale = (float)NB / (hi - lo);
  const bool valid = n > 0 && hi > lo && scale < 1e37f;
  const int ne = valid ? n : 0;
  PH_CNT(12, 1); PH_CNT(7, nw);
  clear_bins_if(valid, s);
  for (int e0 = 0; e0 < nw; e0 += BATCH) {
    float v[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) v[j] = ld_score(s.buf + min(e0 + j, max(ne - 1, 0)) * ENTRY_PITCH);
    int b[BATCH]; uint32_t inc[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      inc[j] = ((e0 + j < ne) & (v[j] >= lo) & (v[j] <= hi)) ? 1u : 0u;
      b[j] = max(0, min(NB - 1, __float2int_rz((v[j] - lo) * scale)));
    }
    hist_add(s.aux, b, inc);
  }
  int bsel;
  scan_bins(s, rank, bsel, bi.cnt, bi.above);
  bi.reset();
  uint32_t waddr = s.buf;
  const int ne_last = max(ne - 1, 0);
  for (int e0 = 0; e0 < nw; e0 += BATCH) {
    float v[BATCH]; uint32_t id[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j)      // reading past the lane's count is harmless (< cap)
      ld_entry(s.buf + min(e0 + j, ne_last) * ENTRY_PITCH, v[j], id[j]);
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const bool live = e0 + j < ne;
      const bool in = live & (v[j] >= lo) & (v[j] <= hi);
      const int b = min(NB - 1, __float2int_rz((v[j] - lo) * scale));
      bi.track(in & (b == bsel), v[j]);
      const bool keep = drop & live & ((v[j] > hi) | (in & (b >= bsel)));
      st_entry_if(keep, waddr, v[j], id[j]);
      waddr += keep ? ENTRY_PITCH : 0u;
    }
  }
  if (valid && drop) n = (int)((waddr - s.buf) / ENTRY_PITCH);
  return valid;
}

// Key-space fallback (5 key bits per level) for ranges the score-domain levels cannot split
// (differences too small to scale).  Exact key of rank T among the entries whose keys lie in
// [lo, hi]; `need` of the entries equal to it belong to the top T.
__device__ void select_keys(const Sel& s, int n, int T, uint32_t lo, uint32_t hi, uint32_t& key_T,
                            int& need_out) {
  const int nw = warp_max(n);
  uint32_t span = n > 0 ? hi - lo : 0u;
  int need = T;
  for (int level = 0; level < 8; ++level) {
    const bool work = n > 0 && span != 0;
    if (!__any_sync(FULL, work)) break;
    const int ne = work ? n : 0;
    const int shift = max(0, (32 - __clz(span | 1u)) - NB_LOG);
    clear_bins_if(work, s);
    for (int e0 = 0; e0 < nw; e0 += BATCH) {
      float v[BATCH];
#pragma unroll
      for (int j = 0; j < BATCH; ++j) v[j] = e0 + j < ne ? ld_score(s.buf + (e0 + j) * ENTRY_PITCH) : 0.f;
#pragma unroll
      for (int j = 0; j < BATCH; ++j) {
        const uint32_t off = key_of(v[j]) - lo;
        if (e0 + j < ne && off <= span) aux_inc(s.aux + (off >> shift) * AUX_PITCH);
      }
    }
    int bsel, cnt, above;
    scan_bins(s, need, bsel, cnt, above);
    if (work) {
      need -= above;
      const uint32_t base = (uint32_t)bsel << shift;
      lo += base;
      span = min(span - base, (shift ? (1u << shift) : 1u) - 1u);
    }
  }
  key_T = lo; need_out = need;
}

// Exact score of rank T (1-based, descending) among the n entries of each participating lane
// (T <= n; other lanes pass active = false), by zooming score-domain levels until the bin
// holding rank T contains equal scores only.  `need` of the entries equal to the result belong
// to the top T.  With `drop`, entries known to rank below T are removed on the way.
// With fit_limit >= 0 a lane stops as soon as its buffer has shrunk to fit_limit or fewer
// entries; it then reports exact = false and s_T = the smallest surviving score.
__device__ void select_rank(const Sel& s, bool active, int& n, int T, bool drop, int fit_limit,
                            float lo, float hi, float& s_T, int& need, bool& exact) {
  bool done = !active, fallback = false;
  int rank = T;
  exact = false; need = 0; s_T = lo;
  for (int level = 0; level < 10; ++level) {
    const bool work = !done;
    if (!__any_sync(FULL, work)) break;
    int nl = work ? n : 0;
    const int n_before = nl;
    const int nw = warp_max(nl);
    BinInfo bi;
    const bool valid = lin_level(s, nl, nw, lo, hi, rank, drop, bi);
    if (work) {
      if (!valid) { fallback = true; done = true; }
      else {
        n = nl;
        rank -= bi.above;
        if (fit_limit >= 0 && n <= fit_limit && n < n_before) { s_T = bi.mn1; done = true; }
        else if (bi.resolve(rank, s_T, need)) { exact = true; done = true; }
        else {
          // zoom into the bin; with drop the entries above stay in the buffer, so the rank
          // inside the bin is what remains to be resolved
          lo = bi.mn1; hi = bi.mx1;
        }
      }
    }
  }
  fallback = fallback || !done;
  if (__any_sync(FULL, fallback)) {
    PH_CNT(9, 1);
    uint32_t kt = 0; int nd = 0;
    select_keys(s, fallback ? n : 0, rank, key_of(lo), key_of(hi), kt, nd);
    if (fallback) { s_T = rr_key_to_float(kt); need = nd; exact = true; }
  }
}

// Keeps scores > s_T and the first `need` entries equal to it (stable, in place).
__device__ __forceinline__ int compact_exact(const Sel& s, int n, float s_T, int need) {
  const int nw = warp_max(n);
  uint32_t waddr = s.buf;
  int ties = 0;
  for (int e0 = 0; e0 < nw; e0 += BATCH) {
    float v[BATCH]; uint32_t id[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j)
      ld_entry(s.buf + min(e0 + j, max(n - 1, 0)) * ENTRY_PITCH, v[j], id[j]);
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const bool in = e0 + j < n;
      const bool eq = in & (v[j] == s_T);
      const bool keep = in & ((v[j] > s_T) | (eq & (ties < need)));
      ties += eq;
      st_entry_if(keep, waddr, v[j], id[j]);
      waddr += keep ? ENTRY_PITCH : 0u;
    }
  }
  return (int)((waddr - s.buf) / ENTRY_PITCH);
}

// The final cut and the route / near-miss split are finished on short side lists: while the
// last pass drops what lies below the bin of rank keep, it copies the scores of that bin, and
// of the bin of rank kk, into two lists of up to LMAX words each (in the histogram words, which
// are dead once the bins have been scanned).  The wanted rank inside such a list is then found
// by counting, list order breaking ties (the lists keep the buffer's ascending chunk ids).
constexpr int LMAX = NB / 2;
__device__ __forceinline__ void rank_in_list(uint32_t list, int cnt, int cmax, int T, float& s_T,
                                             int& need) {
  const int last = max(cnt - 1, 0);
  for (int i = 0; i < cmax; ++i) {
    const float si = ld_score(list + min(i, last) * AUX_PITCH);
    int gt = 0, eq = 0;
    for (int j0 = 0; j0 < cmax; j0 += 4) {
      float sj[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) sj[j] = ld_score(list + min(j0 + j, last) * AUX_PITCH);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool in = j0 + j < cnt;
        gt += in & (sj[j] > si); eq += in & (sj[j] == si);
      }
    }
    if (i < cnt && gt < T && T <= gt + eq) { s_T = si; need = T - gt; }
  }
}

// Smallest and largest score in the lane's buffer (lanes with n = 0 get +inf / -inf).
__device__ __forceinline__ void buffer_minmax(const Sel& s, int n, float& mn, float& mx) {
  const int nw = warp_max(n);
  mn = __int_as_float(0x7f800000); mx = __int_as_float(0xff800000);
  for (int e0 = 0; e0 < nw; e0 += BATCH) {
    float v[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) v[j] = ld_score(s.buf + min(e0 + j, max(n - 1, 0)) * ENTRY_PITCH);
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      mn = fminf(mn, n > 0 ? v[j] : mn); mx = fmaxf(mx, n > 0 ? v[j] : mx);
    }
  }
}
// Upper end of a search range when only a lower bound of the buffered scores is known: the
// first level then puts everything into one bin and the next one zooms into the real range.
constexpr float kNoUpperBound = 3.0e38f;

// Per-row state of the streaming threshold filter.
struct RowState {
  float tau;          // pass threshold of the filter (inclusive)
  float blo;          // lower bound of the buffered scores
  float smin, smax;   // smallest / largest buffered score when the map was laid out
  float map_lo, map_scale;   // fixed score -> bin map of the persistent histogram
  int binned;         // buffer entries [0, binned) are counted in the histogram; -1: no map yet
};

// Re-tightening with a PERSISTENT histogram: the row's score->bin map is fixed at its first
// re-tightening, so each call only has to bin the entries appended since the previous call,
// find the bin b* of rank `keep` from the top, and drop the entries below b* (stable, in
// place).  Bins below b* keep stale counts, which is harmless: the threshold only rises.  If
// b* is too crowded for the buffer to fit `fit_limit`, the cut is finished inside b* (directly
// when b* has at most 4 entries, else by score-domain zoom levels) and the histogram is
// rebuilt at the next call.
// FINAL: the last call of a row.  The cut is made exact (n becomes `keep`), and the same
// level also locates rank `kk` (the route / near-miss split): s_k and need_k are returned.
// With `lists` (FINAL only) the exact cut is not applied to the buffer: the buffer keeps the
// entries of bin b* and above, and (s_cut, need_cut) say which of them belong to the top keep
// (scores > s_cut, and the first need_cut entries equal to it); lanes that had to take the
// slow way return s_cut = -inf (everything left in the buffer belongs).
template <bool FINAL>
__device__ void retighten(const Sel& s, bool active, int& n, int keep, int fit_limit, RowState& st,
                          int kk, float& s_k, int& need_k, bool lists, float& s_cut,
                          int& need_cut) {
  // (1) map (first call) + binning of the new entries.  With d = mean - min of the buffered
  // scores the map covers [mean - 0.5 d, mean + 1.3 d]: the cut lies around or above the mean,
  // and a few far outliers (e.g. a row's own cluster) would otherwise stretch the bins;
  // whatever falls outside lands in the first / last bin.
  const bool fresh = active && st.binned < 0;
  if (__any_sync(FULL, fresh)) {
    const int nf = fresh ? n : 0;
    const int nwf = warp_max(nf);
    float sum = 0.f, mn = __int_as_float(0x7f800000), mx = __int_as_float(0xff800000);
    for (int e0 = 0; e0 < nwf; e0 += BATCH) {
      float v[BATCH];
#pragma unroll
      for (int j = 0; j < BATCH; ++j) v[j] = ld_score(s.buf + min(e0 + j, max(nf - 1, 0)) * ENTRY_PITCH);
#pragma unroll
      for (int j = 0; j < BATCH; ++j) {      // indices past nf re-read the last entry: harmless
        sum += e0 + j < nf ? v[j] : 0.f;
        mn = fminf(mn, v[j]); mx = fmaxf(mx, v[j]);
      }
    }
    if (fresh) {
      st.smin = mn; st.smax = mx;
      const float mean = sum / (float)max(nf, 1);
      const float d = mean - st.smin;
      // full distribution buffered (no threshold yet): skip its lower tail; a buffer that was
      // filtered from the start (warm threshold) is a truncated upper tail: start at its floor
      const bool truncated = st.tau > __int_as_float(0xff800000);
      const float below = truncated ? d : 0.5f * d;
      const float width = below + fminf((truncated ? 1.5f : 1.3f) * d, st.smax - mean);
      st.map_lo = mean - below;
      st.map_scale = (float)NB / width;
      st.binned = 0;
      clear_bins(s);
    }
  }
  const bool usable = active && st.smax > st.smin && st.map_scale > 0.f && st.map_scale < 1e37f;
  // lanes without a usable map (all buffered scores equal, or a range too narrow to scale)
  // search their whole buffer below: its exact bounds
  float fb_lo = 0.f, fb_hi = 0.f;
  if (__any_sync(FULL, active && !usable)) buffer_minmax(s, active && !usable ? n : 0, fb_lo, fb_hi);
  const int from = usable ? st.binned : 0, to = usable ? n : 0;
  const int nw_new = warp_max(to - from);
  float mlo = st.map_lo, msc = st.map_scale;
  float moff = -mlo * msc;           // bin coordinate of a score: fmaf(v, msc, moff), everywhere
  for (int e0 = 0; e0 < nw_new; e0 += BATCH) {
    float v[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j)
      v[j] = ld_score(s.buf + min(from + e0 + j, max(to - 1, 0)) * ENTRY_PITCH);
    int b[BATCH]; uint32_t inc[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      inc[j] = from + e0 + j < to ? 1u : 0u;
      b[j] = max(0, min(NB - 1, __float2int_rz(fmaf(v[j], msc, moff))));
    }
    hist_add(s.aux, b, inc);
  }
  // (2) bin of rank keep (and of rank kk), drop what lies below the former
  BinInfo bc, bk;
  int bsel, bsel_k = 0;
  scan_bins(s, keep, bsel, bc.cnt, bc.above);
  if (FINAL) scan_bins(s, kk, bsel_k, bk.cnt, bk.above);
  bc.reset(); bk.reset();
  const int nd = usable ? n : 0;
  const int nw = warp_max(nd);
  if (FINAL && lists) {
    // The persistent map was laid out for the row's whole score distribution; by now the
    // buffer holds its upper tail only, so the bins around the cut are crowded.  Lay a second
    // map over the stretch from the bin of rank keep to the bin of rank kk (one bin of slack at
    // either end catches what lies below / above) and count again: the bins of the two ranks
    // then hold a handful of entries each.
    const bool crowded = usable && (bc.cnt > LMAX || bk.cnt > LMAX);
    if (__any_sync(FULL, crowded)) {
      const float e_lo = mlo + (float)bsel / msc, e_hi = mlo + (float)(bsel_k + 1) / msc;
      const float w = (e_hi - e_lo) * (1.0f / (float)(NB - 2));
      const bool remap = usable && w > 0.f && (1.0f / w) < 1e37f;
      if (remap) { mlo = e_lo - w; msc = 1.0f / w; moff = -mlo * msc; }
      clear_bins_if(remap, s);
      const int nr_ = remap ? n : 0;
      for (int e0 = 0; e0 < nw; e0 += BATCH) {
        float v[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j) v[j] = ld_score(s.buf + min(e0 + j, max(nr_ - 1, 0)) * ENTRY_PITCH);
        int b[BATCH]; uint32_t inc[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j) {
          inc[j] = e0 + j < nr_ ? 1u : 0u;
          b[j] = max(0, min(NB - 1, __float2int_rz(fmaf(v[j], msc, moff))));
        }
        hist_add(s.aux, b, inc);
      }
      int b1, b2; BinInfo t1, t2;
      scan_bins(s, keep, b1, t1.cnt, t1.above);
      scan_bins(s, kk, b2, t2.cnt, t2.above);
      if (remap) { bsel = b1; bsel_k = b2; bc.cnt = t1.cnt; bc.above = t1.above; bk.cnt = t2.cnt; bk.above = t2.above; }
    }
  }
  uint32_t waddr = s.buf;
  // bin >= bsel  <=>  (v - lo) * scale >= bsel for bsel >= 1; bin 0 also holds what lies below lo
  const float tb = bsel == 0 ? __int_as_float(0xff800000) : (float)bsel;
  // FINAL, every lane with work has a usable map and short bins: side lists instead of tracking
  const bool fast_lane = FINAL && lists && usable && bc.cnt <= LMAX && bk.cnt <= LMAX;
  const bool fast = FINAL && lists && __all_sync(FULL, fast_lane || !active);
#ifdef RR_PHASE_TIMING
  if (FINAL) {
    const int n_slow_lanes = __popc(__ballot_sync(FULL, active && !fast_lane));
    const int worst = warp_max(active ? max(bc.cnt, bk.cnt) : 0);
    PH_CNT(13, fast ? 1 : 0); PH_CNT(14, n_slow_lanes); PH_CNT(15, worst);
  }
#endif
  if (fast) {
    const uint32_t list_c = s.aux, list_k = s.aux + LMAX * AUX_PITCH;
    uint32_t wc = list_c, wk = list_k;
    for (int e0 = 0; e0 < nw; e0 += BATCH) {
      float v[BATCH]; uint32_t id[BATCH];
#pragma unroll
      for (int j = 0; j < BATCH; ++j)
        ld_entry(s.buf + min(e0 + j, max(nd - 1, 0)) * ENTRY_PITCH, v[j], id[j]);
#pragma unroll
      for (int j = 0; j < BATCH; ++j) {
        const float t = fmaf(v[j], msc, moff);
        const bool live = e0 + j < nd;
        const bool keep_it = live & (t >= tb);
        const int b = max(0, min(NB - 1, __float2int_rz(t)));
        const bool in_c = live & (b == bsel), in_k = live & (b == bsel_k);
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.b32 [%0], %1;\n\t}"
                     ::"r"(wc), "f"(v[j]), "r"((uint32_t)in_c) : "memory");
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.b32 [%0], %1;\n\t}"
                     ::"r"(wk), "f"(v[j]), "r"((uint32_t)in_k) : "memory");
        wc += in_c ? AUX_PITCH : 0u; wk += in_k ? AUX_PITCH : 0u;
        st_entry_if(keep_it, waddr, v[j], id[j]);
        waddr += keep_it ? ENTRY_PITCH : 0u;
      }
    }
    if (active) n = (int)((waddr - s.buf) / ENTRY_PITCH);
    const int cnt_c = active ? bc.cnt : 0, cnt_k = active ? bk.cnt : 0;
    s_cut = __int_as_float(0xff800000); need_cut = 0;
    rank_in_list(list_c, cnt_c, warp_max(cnt_c), keep - bc.above, s_cut, need_cut);
    float ks = 0.f; int kn = 0;
    rank_in_list(list_k, cnt_k, warp_max(cnt_k), kk - bk.above, ks, kn);
    if (active) { s_k = ks; need_k = kn; }
    return;
  }
  if (FINAL) { s_cut = __int_as_float(0xff800000); need_cut = 0; }
  for (int e0 = 0; e0 < nw; e0 += BATCH) {
    float v[BATCH]; uint32_t id[BATCH];
#pragma unroll
    for (int j = 0; j < BATCH; ++j)
      ld_entry(s.buf + min(e0 + j, max(nd - 1, 0)) * ENTRY_PITCH, v[j], id[j]);
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const float t = fmaf(v[j], msc, moff);
      const bool live = e0 + j < nd;
      const bool keep_it = live & (t >= tb);
      if (FINAL) {
        const int b = max(0, min(NB - 1, __float2int_rz(t)));
        bc.track(live & (b == bsel), v[j]);
        bk.track(live & (b == bsel_k), v[j]);
      } else {
        bc.mn1 = fminf(bc.mn1, keep_it ? v[j] : bc.mn1);      // smallest survivor
      }
      st_entry_if(keep_it, waddr, v[j], id[j]);
      waddr += keep_it ? ENTRY_PITCH : 0u;
    }
  }
  if (usable) {
    n = (int)((waddr - s.buf) / ENTRY_PITCH);
    st.binned = n;
    st.blo = bc.mn1; st.tau = bc.mn1;  // >= keep seen scores reach mn1: a valid threshold
  }
  // (3) crowded bin, unusable range, or the final exact cut: finish inside b*
  const bool more = active && (!usable || n > fit_limit);
  float s_T = 0.f; int need = 0;
  const bool direct = FINAL && more && usable && bc.resolve(keep - bc.above, s_T, need);
  const bool zoom = more && !direct;
#ifdef RR_PHASE_TIMING
  if (!FINAL) {       // ballots by the whole warp first; only then the lane-0 counters
    const int nz = __popc(__ballot_sync(FULL, zoom)), nu = __popc(__ballot_sync(FULL, active && !usable));
    const int ndr = __popc(__ballot_sync(FULL, zoom && bsel == 0));
    const int ntop = __popc(__ballot_sync(FULL, zoom && bsel == NB - 1));
    (void)nz; (void)ntop; (void)ndr;
  }
#endif
  if (__any_sync(FULL, zoom)) {
    PH_CNT(9, 1);
    float zs; int zn; bool zexact;
    // FINAL and usable: everything left of interest is inside bin b* = [mn1, mx1] and `above`
    // entries outrank it; otherwise the whole (already reduced) buffer is searched
    const bool inbin = FINAL && usable;
    select_rank(s, zoom, n, inbin ? keep - bc.above : keep, true, fit_limit,
                inbin ? bc.mn1 : (usable ? bc.mn1 : fb_lo),
                inbin ? bc.mx1 : (usable ? kNoUpperBound : fb_hi), zs, zn, zexact);
    if (zoom) {
      if (zexact) { s_T = zs; need = zn; }
      else { st.tau = zs; st.blo = zs; }        // fits now; zs = smallest surviving score
    }
    // the scratch levels overwrote the bins of the lanes that zoomed
    if (zoom) { st.binned = usable ? 0 : -1; clear_bins(s); }
    const bool cut_exact = direct || (zoom && zexact);
    const int w = compact_exact(s, cut_exact ? n : 0, s_T, need);
    if (cut_exact) {
      n = w;
      st.tau = rr_key_to_float(key_of(s_T) + 1u);   // later ties have larger ids: they lose
      st.blo = s_T;
      if (st.binned > 0) { st.binned = 0; clear_bins(s); }   // counts no longer match
    }
  } else if (__any_sync(FULL, direct)) {
    const int w = compact_exact(s, direct ? n : 0, s_T, need);
    if (direct) {
      n = w;
      st.tau = rr_key_to_float(key_of(s_T) + 1u);
      st.blo = s_T;
      if (st.binned > 0) { st.binned = 0; clear_bins(s); }
    }
  }
  // (4) FINAL: the route / near-miss split at rank kk among the `keep` survivors
  if (FINAL) {
    const bool split = active && n > kk;
    float ks = 0.f; int kn = 0;
    const bool kdirect = split && usable && bk.resolve(kk - bk.above, ks, kn);
    const bool kzoom = split && !kdirect;
    if (__any_sync(FULL, kzoom)) {
      float zs; int zn; bool zexact; int n_ = n;
      select_rank(s, kzoom, n_, usable ? kk - bk.above : kk, false, -1,
                  usable ? bk.mn1 : fb_lo, usable ? bk.mx1 : fb_hi, zs, zn,
                  zexact);
      if (kzoom) { ks = zs; kn = zn; }
    }
    if (split) { s_k = ks; need_k = kn; }
  }
}

// STEP: scores filtered between two checks of the buffer fill.  32 (one TMEM load) unless the
// buffer has little room above `keep` (wide routes): there a finer step lets the buffer fill
// closer to its capacity before each re-tightening, which is worth the extra checks.
template <int D, int STEP>
__global__ void __launch_bounds__(NT, 1)
route_fused_kernel(RRParams p, const __nv_bfloat16* __restrict__ qc,
                   const __grid_constant__ CUtensorMap tmap_k, const int32_t* __restrict__ row_list,
                   uint32_t layer, int cap, int aux_words) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sB = smem;
  Ctl* ctl = (Ctl*)(smem + B_STAGES * C::B_BYTES);
  uint8_t* s_buf = (uint8_t*)ctl + C::CTL_BYTES;                      // [cap][BM] 8-byte entries
  uint8_t* s_aux = s_buf + (size_t)cap * ENTRY_PITCH;                 // [NB][BM] histogram words

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Row tiles are handed out heaviest first (under the causal mask the last tile of a problem
  // walks the most key chunks), so the tail of the grid is made of the short ones.
  const int tiles_m = p.tiles_per_problem;
  const int prob = blockIdx.x % p.P, tm = tiles_m - 1 - blockIdx.x / p.P;

  int seg_lo = 0, seg_hi = p.n_q;
  if (row_list) { seg_lo = p.problem_offsets[prob]; seg_hi = p.problem_offsets[prob + 1]; }
  if (tm * BM >= seg_hi - seg_lo) return;                 // nothing to do (uniform per CTA)

  if (tid < BM) {
    const int local = tm * BM + tid;
    int row = -1, slot = 0;
    if (row_list) {
      const int s = seg_lo + local;
      if (s < seg_hi) { row = row_list[s] - prob * p.n_q; slot = s; }
    } else if (local < p.n_q) {
      row = local; slot = prob * p.n_q + local;
    }
    ctl->row[tid] = row; ctl->slot[tid] = slot;
  }
  if (tid == 0) {
    for (int s = 0; s < B_STAGES; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    for (int s = 0; s < ACC_STAGES; ++s) { mbar_init(&ctl->acc_full[s], 1); mbar_init(&ctl->acc_empty[s], BM); }
    ctl->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmap_k);
  }
  if (warp == 0) tmem_alloc(&ctl->tmem_base, TMEM_COLS);
  __syncthreads();

  // ---- the Qc tile goes to TMEM: the thread that owns row r loads the row (two bf16 per
  // 32-bit word, as they lie in memory) and stores it to TMEM lane r, where the MMA reads its
  // A operand from; rows without a query are zero
  tc_fence_after();
  if (warp >= 2) {
    const int r = (warp & 3) * 32 + lane;
    const int row = ctl->row[r];
    constexpr int W = D / 2;                               // 32-bit words per row
    uint32_t qv[W];
    const uint4* src = reinterpret_cast<const uint4*>(qc + ((size_t)prob * p.n_q + max(row, 0)) * D);
#pragma unroll
    for (int i = 0; i < W / 4; ++i) {
      uint4 t = make_uint4(0, 0, 0, 0);
      if (row >= 0) t = __ldg(src + i);
      qv[4 * i] = t.x; qv[4 * i + 1] = t.y; qv[4 * i + 2] = t.z; qv[4 * i + 3] = t.w;
    }
    const uint32_t taddr = ctl->tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + A_COL;
    if constexpr (W == 64) tmem_st_32x64(taddr, qv); else tmem_st_32x32(taddr, qv);
    tmem_st_wait();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile uint32_t* abort_flag = &ctl->abort_flag;

  int last = -1;
  for (int t = BM - 1; t >= 0; --t) if (ctl->row[t] >= 0) { last = ctl->row[t]; break; }
  const int vmax = rr_valid_count(last, p.n_k, p.causal, p.causal_offset);
  const int n_tiles = (vmax + BN - 1) / BN;

  if (warp == 0) {
    // ===== TMA producer =====
    if (lane == 0) {
      int issued = 0;
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
        if (!mbar_wait_relaxed(&ctl->empty[s], ph ^ 1, abort_flag, 400)) break;
        mbar_expect_tx(&ctl->full[s], C::B_BYTES);
#pragma unroll
        for (int h = 0; h < C::KHALVES; ++h)
          tma_load_3d(sB + s * C::B_BYTES + h * C::B_HALF, &tmap_k, h * 64, t * BN, prob,
                      &ctl->full[s]);
        ++issued;
      }
      for (int t = max(0, issued - B_STAGES); t < issued; ++t) {
        const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->full[s], ph); ++it) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    // ===== MMA issuer =====
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
        const int as = t % ACC_STAGES; const uint32_t aph = (t / ACC_STAGES) & 1;
        if (!mbar_wait_relaxed(&ctl->acc_empty[as], aph ^ 1, abort_flag, 400)) break;
        if (!mbar_wait_relaxed(&ctl->full[s], ph, abort_flag, 100)) break;
        tc_fence_after();
        const uint32_t b_addr = smem_u32(sB + s * C::B_BYTES);
#pragma unroll
        for (int k = 0; k < C::KSTEPS; ++k) {
          const uint32_t b_off = (k >> 2) * C::B_HALF + (k & 3) * 32;
          umma_bf16_ts(tmem_base + as * BN, tmem_base + A_COL + k * 8,
                       umma_desc_k_sw128(b_addr + b_off), idesc, k > 0 ? 1u : 0u);
        }
        umma_commit(&ctl->empty[s]);
        umma_commit(&ctl->acc_full[as]);
      }
    }
  } else {
    // ===== selection: one thread per query row =====
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const int row = ctl->row[r];
    const int v = row >= 0 ? rr_valid_count(row, p.n_k, p.causal, p.causal_offset) : 0;
    const int keep_cfg = p.k + max(p.m, 1);
    const int keep = min(keep_cfg, v), kk = min(p.k, v);
    const Sel sel{smem_u32(s_buf) + r * 8u, smem_u32(s_aux) + r * 4u};
    const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);
    RowState st;
    // rows of a refresh list start from the threshold the rescoring kernel derived from the
    // old candidates' current scores (a valid lower bound); anchors start from -inf
    st.tau = row >= 0 ? (row_list ? p.tau[row_list[ctl->slot[r]]] : ninf) : pinf;   // padding rows pass nothing
    st.blo = pinf; st.smin = pinf; st.smax = ninf;
    st.map_lo = 0.f; st.map_scale = 0.f; st.binned = -1;
    uint32_t waddr = sel.buf;                 // next free entry
    const uint32_t trigger = sel.buf + (uint32_t)(cap - STEP) * ENTRY_PITCH;
    int vmaxw = v, vminw = row >= 0 ? v : 0x7FFFFFFF;
#pragma unroll
    for (int off = 16; off; off >>= 1) {
      vmaxw = max(vmaxw, __shfl_xor_sync(FULL, vmaxw, off));
      vminw = min(vminw, __shfl_xor_sync(FULL, vminw, off));
    }
    bool alive = true;
    for (int t = 0; t < n_tiles; ++t) {
      const int as = t % ACC_STAGES; const uint32_t aph = (t / ACC_STAGES) & 1;
      bool ready;
      { PH_T0(); ready = mbar_wait(&ctl->acc_full[as], aph, abort_flag); PH_ADD(0); }
      if (!__all_sync(FULL, ready)) { alive = false; break; }
      tc_fence_after();
      static_assert(BATCH == 8, "hist_add takes batches of 8");
      static_assert(BN == 2 * CHUNK, "a tile is two TMEM loads of 32 columns");
      if (t * BN < vmaxw) {                                // else: no row of this warp sees it
        uint32_t acc[2][32];
        tmem_ld_32x64(tmem_base + ((uint32_t)(quarter * 32) << 16) + as * BN, acc[0], acc[1]);
#pragma unroll
        for (int c = 0; c < BN / STEP; ++c) {
          const int col0 = t * BN + c * STEP;
          if (col0 >= vmaxw) break;
          if (__any_sync(FULL, waddr > trigger)) {
            // re-tighten: raise the threshold until the buffer fits again
            PH_T0();
            int n = (int)((waddr - sel.buf) / ENTRY_PITCH);
            const bool act = n > keep;
            float dummy_s; int dummy_n;
            retighten<false>(sel, act, n, keep, (keep + cap - STEP) / 2, st, 0, dummy_s, dummy_n,
                             false, dummy_s, dummy_n);
            if (act) waddr = sel.buf + (uint32_t)n * ENTRY_PITCH;
            PH_ADD(1); PH_CNT(8, 1);
          }
          PH_T0();
          const float tau_f = st.tau;
          const uint32_t* a = &acc[c / (CHUNK / STEP)][(c % (CHUNK / STEP)) * STEP];
          // threshold filter: branch-free appends (predicated stores); waddr is the only chain
          if (col0 + STEP <= vminw) {
#pragma unroll
            for (int q = 0; q < STEP; ++q) {
              const float sc = __uint_as_float(a[q]);
              const bool pass = sc >= tau_f;
              st_entry_if(pass, waddr, sc, (uint32_t)(col0 + q));
              waddr += pass ? ENTRY_PITCH : 0u;
            }
          } else {
#pragma unroll
            for (int q = 0; q < STEP; ++q) {
              const float sc = __uint_as_float(a[q]);
              const bool valid = col0 + q < v;
              const bool pass = valid && sc >= tau_f;
              st_entry_if(pass, waddr, sc, (uint32_t)(col0 + q));
              waddr += pass ? ENTRY_PITCH : 0u;
            }
          }
          PH_ADD(2); PH_CNT(10, 1);
        }
      }
      tc_fence_before();
      mbar_arrive(&ctl->acc_empty[as]);
    }

    if (alive) {                                    // warp-uniform
      const bool have = row >= 0;
      const int g = have ? (row_list ? row_list[ctl->slot[r]] : ctl->slot[r]) : 0;
      int n = have ? (int)((waddr - sel.buf) / ENTRY_PITCH) : 0;
      PH_CNT(11, 1);
      // ---- exact cut at rank keep and split at rank kk (entries <= keep: nothing to cut) ----------
      float s_k = ninf; int need_k = 0;        // defaults: everything buffered is selected
      float s_cut = ninf; int need_cut = 0;    // ... and everything buffered belongs to the top keep
      {
        PH_T0();
        if (__any_sync(FULL, n > kk)) {
          if (n <= keep) {
            // rows that see fewer than keep chunks keep everything; only the split remains,
            // over the whole buffer (no map was ever needed for them)
          }
          const bool cut = n > keep;
          // the side lists live in the histogram words, which also hold the exclusion bitmap
          // unless that sits in the buffer tail (where entries beyond keep would be in its way)
          retighten<true>(sel, cut, n, keep, -1, st, kk, s_k, need_k, aux_words <= NB, s_cut,
                          need_cut);
          // rows with kk < n <= keep never enter the cut: split them over the whole buffer
          const bool small = !cut && n > kk;
          if (__any_sync(FULL, small)) {
            float zs; int zn; bool zexact; int n_ = n;
            float lo_s, hi_s;
            buffer_minmax(sel, small ? n : 0, lo_s, hi_s);
            select_rank(sel, small, n_, kk, false, -1, lo_s, hi_s, zs, zn, zexact);
            if (small) { s_k = zs; need_k = zn; }
          }
        }
        PH_ADD(3);
      }
      PH_T0();
      // exclusion bitmap: in the thread's histogram words when they suffice, else in the tail of
      // the thread's OWN buffer column (entries beyond keep are dead after the final cut; two
      // words per entry slot).  Other warps may still be filtering, so nothing outside this
      // thread's column may be touched.
      const bool tail = aux_words > NB;
      const uint32_t bm_base = tail ? sel.buf + (uint32_t)keep_cfg * ENTRY_PITCH : sel.aux;
      auto bm = [&](int w) -> uint32_t {
        return tail ? bm_base + (uint32_t)(w >> 1) * ENTRY_PITCH + (uint32_t)(w & 1) * 4u
                    : bm_base + (uint32_t)w * AUX_PITCH;
      };
      for (int w = 0; w < aux_words; ++w) aux_st(bm(w), 0u);
      int32_t* route = p.routes + (size_t)g * p.k;
      int32_t* sent = p.sentinels + (size_t)g * p.sw;
      // Pass A (branch-free): classify the survivors.  Route ids are parked in the score word
      // of slots 0.., near-miss ids in the id word of slots 0.. (a slot is only overwritten
      // after its entry has been read); the exclusion bitmap is written word by word, which
      // works because the entries are in ascending chunk id.
      int nr = 0, nn = 0, ties = 0, ties_cut = 0, cur_word = 0;
      uint32_t cur_bits = 0u;
      float kth = pinf, next = ninf;
      const int nw = warp_max(n);
      for (int e0 = 0; e0 < nw; e0 += BATCH) {
        float sv[BATCH]; uint32_t id[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j)
          ld_entry(sel.buf + min(e0 + j, max(n - 1, 0)) * ENTRY_PITCH, sv[j], id[j]);
#pragma unroll
        for (int j = 0; j < BATCH; ++j) {
          const bool eq_cut = (e0 + j < n) & (sv[j] == s_cut);
          const bool live = (e0 + j < n) & ((sv[j] > s_cut) | (eq_cut & (ties_cut < need_cut)));
          ties_cut += eq_cut;
          const bool eq = live & (sv[j] == s_k);
          const bool in_route = live & ((sv[j] > s_k) | (eq & (ties < need_k)));
          const bool in_near = live & !in_route & (nn < p.m);
          ties += eq;
          kth = fminf(kth, in_route ? sv[j] : kth);
          next = fmaxf(next, (live & !in_route) ? sv[j] : next);
          asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.b32 [%0], %1;\n\t}"
                       ::"r"(sel.buf + nr * ENTRY_PITCH), "r"(id[j]), "r"((uint32_t)in_route) : "memory");
          asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.b32 [%0], %1;\n\t}"
                       ::"r"(sel.buf + nn * ENTRY_PITCH + 4u), "r"(id[j]), "r"((uint32_t)in_near) : "memory");
          nr += in_route; nn += in_near;
          const int wi = live ? (int)(id[j] >> 5) : cur_word;
          const bool flush = wi != cur_word;
          asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.b32 [%0], %1;\n\t}"
                       ::"r"(bm(cur_word)), "r"(cur_bits), "r"((uint32_t)flush) : "memory");
          cur_bits = flush ? 0u : cur_bits;
          cur_word = wi;
          cur_bits |= (in_route | in_near) ? 1u << (id[j] & 31) : 0u;
        }
      }
      aux_st(bm(cur_word), cur_bits);
      PH_ADD(5);
      if (have) {
        PH_T0();
        // Pass B: copy out, 16 bytes at a time where the row is 16-byte aligned
        if ((p.k & 3) == 0) {
          for (int q = 0; q < p.k; q += 4) {
            int4 o;
            o.x = q + 0 < nr ? (int)aux_ld(sel.buf + (q + 0) * ENTRY_PITCH) : -1;
            o.y = q + 1 < nr ? (int)aux_ld(sel.buf + (q + 1) * ENTRY_PITCH) : -1;
            o.z = q + 2 < nr ? (int)aux_ld(sel.buf + (q + 2) * ENTRY_PITCH) : -1;
            o.w = q + 3 < nr ? (int)aux_ld(sel.buf + (q + 3) * ENTRY_PITCH) : -1;
            *reinterpret_cast<int4*>(route + q) = o;
          }
        } else {
          for (int e = 0; e < p.k; ++e) route[e] = e < nr ? (int)aux_ld(sel.buf + e * ENTRY_PITCH) : -1;
        }
        if (((p.m | p.sw) & 3) == 0) {
          for (int q = 0; q < p.m; q += 4) {
            int4 o;
            o.x = q + 0 < nn ? (int)aux_ld(sel.buf + (q + 0) * ENTRY_PITCH + 4u) : -1;
            o.y = q + 1 < nn ? (int)aux_ld(sel.buf + (q + 1) * ENTRY_PITCH + 4u) : -1;
            o.z = q + 2 < nn ? (int)aux_ld(sel.buf + (q + 2) * ENTRY_PITCH + 4u) : -1;
            o.w = q + 3 < nn ? (int)aux_ld(sel.buf + (q + 3) * ENTRY_PITCH + 4u) : -1;
            *reinterpret_cast<int4*>(sent + q) = o;
          }
        } else {
          for (int e = 0; e < p.m; ++e) sent[e] = e < nn ? (int)aux_ld(sel.buf + e * ENTRY_PITCH + 4u) : -1;
        }
        p.kth[g] = kth;
        p.margin[g] = v > kk ? kth - next : pinf;

        // ---- mandatory global sentinels (sink chunk, most recent chunk): a slot each after
        // the random ones, empty if the chunk is already in the route or a near-miss sentinel
        int pool = v - (nr + nn);
        if (p.n_global) {
          int32_t* glob = sent + p.m + p.r;
          int gi = 0;
          for (int b = 0; b < 2; ++b) {
            if (!((p.global_mask >> b) & 1)) continue;
            const int j = b == 0 ? 0 : v - 1;
            int id = -1;
            if (v > 0) {
              const uint32_t wa = bm(j >> 5);
              const uint32_t w = aux_ld(wa), bit = 1u << (j & 31);
              if (!(w & bit)) { aux_st(wa, w | bit); id = j; --pool; }
            }
            glob[gi++] = id;
          }
        }
        // ---- random sentinels --------------------------------------------------------------
        int32_t* rnd = sent + p.m;
        int taken = 0;
        if (p.r > 0 && pool > 0) {
          if (pool > p.r) {
            const unsigned long long rk = rr_row_key(p.seed, (uint32_t)g);
            const int limit = 64 * p.r;
            // four draws are generated at a time (independent 64-bit mixes overlap); they are
            // still accepted strictly in draw order
            for (int t0 = 0; t0 < limit && taken < p.r; t0 += 4) {
              int j4[4];
#pragma unroll
              for (int i = 0; i < 4; ++i)
                j4[i] = (int)__umulhi(rr_draw_u32(rk, layer, (uint32_t)(t0 + i)), (uint32_t)v);
#pragma unroll
              for (int i = 0; i < 4; ++i) {              // branch-free: predicated stores
                const bool live = (t0 + i < limit) & (taken < p.r);
                const uint32_t wa = bm(j4[i] >> 5);
                const uint32_t w = aux_ld(wa), bit = 1u << (j4[i] & 31);
                const bool take = live & ((w & bit) == 0u);
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.b32 [%0], %1;\n\t}"
                             ::"r"(wa), "r"(w | bit), "r"((uint32_t)take) : "memory");
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.global.b32 [%0], %1;\n\t}"
                             ::"l"(rnd + taken), "r"(j4[i]), "r"((uint32_t)take) : "memory");
                taken += take;
              }
            }
          }
          for (int j = 0; j < v && taken < p.r; ++j)
            if (!((aux_ld(bm(j >> 5)) >> (j & 31)) & 1u)) rnd[taken++] = j;
        }
        for (int e = taken; e < p.r; ++e) rnd[e] = -1;
        PH_ADD(6);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
    if (lane == 0 && ctl->abort_flag) atomicOr(p.status, RR_STATUS_TIMEOUT);
  }
}

// Shared-memory plan: returns false if the configuration does not fit the fused kernel.
bool plan(const RRParams& p, int& cap, int& aux_words, size_t& smem_bytes) {
  const int keep = p.k + (p.m > 0 ? p.m : 1);
  const size_t fixed = p.d == 128 ? Cfg<128>::FIXED_BYTES : Cfg<64>::FIXED_BYTES;
  aux_words = (p.n_k + 31) / 32;                 // words of the exclusion bitmap
  const size_t max_smem = 227 * 1024;
  const size_t hist = (size_t)NB * AUX_PITCH;
  if (fixed + hist >= max_smem) return false;
  const int fit = (int)((max_smem - fixed - hist) / ENTRY_PITCH);
  cap = keep + 144;
  if (cap > fit) cap = fit;
  if (cap < keep + CHUNK) return false;
  // a bitmap wider than the histogram lives in the buffer entries beyond `keep`
  if (aux_words > NB && (aux_words + 1) / 2 > cap - keep) return false;
  if (p.n_k > 65535) return false;
  smem_bytes = fixed + hist + (size_t)cap * ENTRY_PITCH;
  return true;
}

}  // namespace

#ifdef RR_BOUNDS_CHECK
extern "C" int rr_debug_oob(unsigned int* out4) {
  cudaDeviceSynchronize();
  return cudaMemcpyFromSymbol(out4, g_oob, 16) == cudaSuccess ? 0 : -1;
}
#endif

#ifdef RR_PHASE_TIMING
extern "C" int rr_debug_phase_counters(unsigned long long* out16, int reset) {
  cudaDeviceSynchronize();
  if (cudaMemcpyFromSymbol(out16, g_phase, sizeof(unsigned long long) * 16) != cudaSuccess) return -1;
  if (reset) {
    unsigned long long z[16] = {};
    cudaMemcpyToSymbol(g_phase, z, sizeof z);
  }
  return 0;
}
#endif

bool rr_route_fused_supported(const RRParams& p) {
  int cap, aux; size_t smem;
  return p.dtype == RR_BF16 && plan(p, cap, aux, smem);
}

cudaError_t rr_launch_route_fused(const RRParams& p, const void* qc, const void* kc,
                                  const int32_t* row_list, int layer, cudaStream_t st) {
  int cap, aux; size_t smem;
  if (!plan(p, cap, aux, smem)) return cudaErrorInvalidConfiguration;
  CUtensorMap tmap;
  cudaError_t e = rr_encode_tmap_bf16_3d(&tmap, kc, p.d, p.n_k, p.P, BN);
  if (e != cudaSuccess) return e;
  const int grid = p.P * p.tiles_per_problem;
  const int keep = p.k + (p.m > 0 ? p.m : 1);
  const bool fine = cap - keep < 64;             // little room above keep: check the fill more often
  static unsigned long long attr_done = 0;      // devices on which the attributes are set
  e = rr_once_per_device(attr_done, [] {
    const void* fns[4] = {(const void*)route_fused_kernel<128, 32>, (const void*)route_fused_kernel<128, 8>,
                          (const void*)route_fused_kernel<64, 32>, (const void*)route_fused_kernel<64, 8>};
    for (const void* fn : fns) {
      const cudaError_t a = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (a != cudaSuccess) return a;
    }
    return cudaSuccess;
  });
  if (e != cudaSuccess) return e;
  const __nv_bfloat16* q = (const __nv_bfloat16*)qc;
  if (p.d == 128 && !fine)
    route_fused_kernel<128, 32><<<grid, NT, smem, st>>>(p, q, tmap, row_list, (uint32_t)layer, cap, aux);
  else if (p.d == 128)
    route_fused_kernel<128, 8><<<grid, NT, smem, st>>>(p, q, tmap, row_list, (uint32_t)layer, cap, aux);
  else if (!fine)
    route_fused_kernel<64, 32><<<grid, NT, smem, st>>>(p, q, tmap, row_list, (uint32_t)layer, cap, aux);
  else
    route_fused_kernel<64, 8><<<grid, NT, smem, st>>>(p, q, tmap, row_list, (uint32_t)layer, cap, aux);
  rr_count_launch();
  return cudaPeekAtLastError();
}
