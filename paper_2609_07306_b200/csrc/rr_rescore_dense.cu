// Candidate rescoring + challenge test (Section 3.2, Eq. 5) on the TENSOR CORES.
//
// The gathered kernel (rr_rescore.cu) fetches c Kc rows per query row and multiplies them on
// the FP32 ALUs: no operand is reused, so it moves c*d*2 bytes per row through L2 and is an
// order of magnitude slower on this machine than computing the whole score strip with
// tcgen05.mma.  This variant does the latter: the same kind of tile pipeline as the fused
// routing kernel produces S[128 rows, 64 chunks] tiles in TMEM, and the threads of a row pick
// out the scores of the row's candidates:
//   * at start the two threads of a row turn its ledger row into a bitmap in shared memory (two
//     planes encoding route / near-miss / random sentinel, one plane per thread), reading the
//     ids with 16-byte loads and setting bits with grouped read-modify-writes;
//   * per tile a thread reads its share of the row's scores from TMEM and takes masked minima /
//     maxima under the tile's bitmap words: alpha = min over route bits, beta = max over
//     sentinel bits, floor = min over route and near-miss bits (the refresh's warm-start
//     threshold).
// Scores are bit-identical to the ones the fused routing kernel computes (same instruction
// sequence on the same operands), so the floor needs no safety margin.
// Outputs are those of the gathered kernel: flags, alpha, beta, tau, per-tile flagged counts,
// work counters (the candidate pairs are still charged as c per row: that is what the method
// evaluates; that the hardware computes the strip is an implementation matter).
#include "rr_tc_pipeline.cuh"

using namespace sm100;

namespace {

// 64-chunk tiles in two stages keep a CTA under half an SM's shared memory: two CTAs per SM
// overlap one's set-up and bitmap build with the other's tile loop.  Two threads share a query
// row (each takes 32 of a tile's 64 columns, one bitmap word): the per-tile work is a chain of dependent ALU-pipe
// instructions, so twice the warps hide twice the latency.
constexpr int BN = 64, B_STAGES = 2, ACC_STAGES = 4;
constexpr int TPR = 2, COLS = BN / TPR;             // threads per row, columns per thread
constexpr int NCONS = tcpipe::BM * TPR, NT = 64 + NCONS;
constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr uint32_t PITCH = tcpipe::BM * 4;          // debug score column: one word per row

__device__ __forceinline__ uint32_t lds(uint32_t a) {
  uint32_t v; asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v;
}
__device__ __forceinline__ void sts(uint32_t a, uint32_t v) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void consumers_sync() {            // the NCONS consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(NCONS) : "memory");
}
// acc = min(acc, s) / max(acc, s) if (word & bit): a predicate and a predicated instruction
__device__ __forceinline__ void min_if(float& acc, float s, uint32_t word, uint32_t bit) {
  asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %2, %3;\n\tsetp.ne.u32 p, t, 0;\n\t"
      "@p min.f32 %0, %0, %1;\n\t}" : "+f"(acc) : "f"(s), "r"(word), "r"(bit));
}
__device__ __forceinline__ void max_if(float& acc, float s, uint32_t word, uint32_t bit) {
  asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %2, %3;\n\tsetp.ne.u32 p, t, 0;\n\t"
      "@p max.f32 %0, %0, %1;\n\t}" : "+f"(acc) : "f"(s), "r"(word), "r"(bit));
}

#ifdef RR_PHASE_TIMING
// cycles per phase, kept in registers and added to the global totals once per warp
__device__ unsigned long long g_rd_phase[8];
#define RD_T0() long long rd_t0_ = clock64(); long long rd_acc_[5] = {0, 0, 0, 0, 0}
#define RD_LAP(i) do { const long long t1_ = clock64(); rd_acc_[i] += t1_ - rd_t0_; rd_t0_ = t1_; } while (0)
#define RD_FLUSH() do { if ((threadIdx.x & 31) == 0) { for (int i_ = 0; i_ < 5; ++i_) atomicAdd(&g_rd_phase[i_], (unsigned long long)rd_acc_[i_]); } } while (0)
#else
#define RD_T0() do {} while (0)
#define RD_LAP(i) do {} while (0)
#define RD_FLUSH() do {} while (0)
#endif

// Per-row bitmaps: row r owns `pitch` = 2*words + 1 consecutive words (odd, so that the 32 rows
// of a warp fall into 32 different banks whenever each thread touches a word of its own row).
// Two planes encode the three candidate classes of a chunk:
//   plane A | plane B :  route = 1|0,  near-miss = 0|1,  random sentinel = 1|1.
// PRIOR: also track the weakest near-miss candidate, so that tau = the floor of the k+m old
// candidates' current scores can warm-start a refresh kernel that wants it (the streaming kernel;
// the two-sweep kernel derives a tighter bound itself and the third masked pass is a tenth of
// this kernel's time).
template <int D, bool PRIOR>
__global__ void __launch_bounds__(NT, 2)
rescore_dense_kernel(RRParams p, const __grid_constant__ CUtensorMap tmap_q,
                     const __grid_constant__ CUtensorMap tmap_k, int words, int force_timeout) {
  using P = tcpipe::Pipe<D, BN, B_STAGES, ACC_STAGES, NCONS>;
  if (p.force_threshold > 0 && p.force_in[0] > 0) return;   // forced anchor: nothing is tested
  extern __shared__ uint8_t smem_raw[];
  P pipe;
  pipe.carve(smem_raw);
  // extra: 3 counters, [128][pitch] bitmap words, [3][128] partial results of the second
  // thread of each row, (debug only) [BN][128] score column
  unsigned long long* s_cnt = (unsigned long long*)pipe.extra;
  const uint32_t pitch = 2u * words + 1u;
  const uint32_t bm_base = smem_u32(pipe.extra) + 64u;
  const uint32_t xch_base = (bm_base + tcpipe::BM * pitch * 4u + 15u) & ~15u;
  const uint32_t sc_base = xch_base + 3u * PITCH;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles_m = p.tiles_per_problem;
  const int prob = blockIdx.x % p.P, tm = tiles_m - 1 - blockIdx.x / p.P;   // heaviest first
  const int tile_id = prob * tiles_m + tm;
  if (tid == 0) { s_cnt[0] = 0; s_cnt[1] = 0; s_cnt[2] = 0; }
  RD_T0();

  // ---- who builds what ---------------------------------------------------------------------
  // Each row has two consumer threads (warps 2-5: part 0, warps 6-9: part 1).  Part 0 owns
  // plane A of its row's bitmap (route and random / global sentinels), part 1 owns plane B
  // (all sentinels), so the two never write the same word and plain read-modify-writes do.
  // A thread reads its ids 16 at a time (16-byte loads where the ledger row allows) and sets
  // their bits with shared-memory reductions (no read-modify-write round trips to wait for).
  // The first two batches are fetched before the pipeline set-up so that their memory round
  // trip overlaps it.  Without the prior-bound pass (PRIOR = false) the classes are just route
  // (plane A) and sentinel (plane B): part 0 then skips the random / global slots.
  const int cquarter = warp & 3, cpart = (warp - 2) >> 2;
  const int crow_l = cquarter * 32 + lane;                       // row inside the tile
  const int crow = tm * tcpipe::BM + crow_l;
  const bool chas = warp >= 2 && crow < p.n_q;
  const size_t cg = (size_t)prob * p.n_q + crow;
  // part 0: range 0 = route [0, k), range 1 = sentinel slots [m, sw); part 1: range 0 = [0, sw)
  const int32_t* const ptr0 = cpart == 0 ? p.routes + cg * p.k : p.sentinels + cg * p.sw;
  const int32_t* const ptr1 = p.sentinels + cg * p.sw + p.m;
  const int n0 = chas ? (cpart == 0 ? p.k : p.sw) : 0, n1 = chas && cpart == 0 && PRIOR ? p.sw - p.m : 0;
  auto load16 = [&](const int32_t* ptr, int s0, int n, int (&ids)[16]) {
    if (s0 + 16 <= n && (((uintptr_t)(ptr + s0)) & 15u) == 0) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int4 t = __ldg(reinterpret_cast<const int4*>(ptr + s0) + q);
        ids[4 * q] = t.x; ids[4 * q + 1] = t.y; ids[4 * q + 2] = t.z; ids[4 * q + 3] = t.w;
      }
    } else {
#pragma unroll
      for (int q = 0; q < 16; ++q) ids[q] = s0 + q < n ? __ldg(ptr + s0 + q) : -1;
    }
  };
  // second prefetched batch: range 1 if the thread has one, else the next 16 of range 0
  const bool pre1_is1 = n1 > 0;
  const int pre1_s0 = pre1_is1 ? 0 : 16;
  int pre0[16], pre1[16];
  load16(ptr0, 0, n0, pre0);
  load16(pre1_is1 ? ptr1 : ptr0, pre1_s0, pre1_is1 ? n1 : n0, pre1);

  pipe.setup(p, nullptr, &tmap_k, nullptr, prob, tm, 0, p.n_q, NT, &tmap_q);
  const int n_tiles = pipe.num_tiles(p);

  if (warp == 0) {
    if (lane == 0) pipe.producer(&tmap_k, prob, n_tiles, &tmap_q, tm);
  } else if (warp == 1) {
    if (lane == 0) pipe.mma_issuer(n_tiles, true);
  } else {
    // a warp may only read the TMEM lanes 32*(warp % 4) ...: warps 2-5 take the first COLS
    // columns of their quarter's rows, warps 6-9 the rest
    const int quarter = cquarter, part = cpart;
    const int r = crow_l;
    const int row = crow < p.n_q ? crow : -1;                       // rows are consecutive
    const int g = (int)cg;
    const int v = row >= 0 ? rr_valid_count(row, p.n_k, p.causal, p.causal_offset) : 0;
    const uint32_t bA = bm_base + r * pitch * 4u, bB = bA + words * 4u;
    const uint32_t col = sc_base + r * 4u;
    const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);

    RD_LAP(0);
    // ---- ledger row -> this thread's plane of the row's bitmap -----------------------------
    {
      const uint32_t plane = part == 0 ? bA : bB;
      for (int w = 0; w < words; ++w) sts(plane + w * 4u, 0u);
      RD_LAP(4);
      int n_ok = 0; bool bad = false;
      // candidates are charged once: part 0 counts what it sets, part 1 only the near-miss slots
      auto or_ids = [&](const int (&ids)[16], int s0, int count_below) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int id = ids[i];
          bad |= id >= v;
          const bool ok = id >= 0 && id < v;
          n_ok += ok && s0 + i < count_below;
          // a shared-memory reduction: the marks of a row do not wait for one another
          if (ok) asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(plane + (uint32_t)(id >> 5) * 4u), "r"(1u << (id & 31)) : "memory");
        }
      };
      const int cb0 = (part == 0 || !PRIOR) ? 0x7fffffff : p.m;   // range 0: all / the near-miss slots
      or_ids(pre0, 0, cb0);
      or_ids(pre1, pre1_s0, pre1_is1 ? 0x7fffffff : cb0);
      const int n0_max = __reduce_max_sync(FULL, n0), n1_max = __reduce_max_sync(FULL, n1);
      for (int s0 = pre1_is1 ? 16 : 32; s0 < n0_max; s0 += 16) {
        load16(ptr0, s0, n0, pre0);
        or_ids(pre0, s0, cb0);
      }
      for (int s0 = 16; s0 < n1_max; s0 += 16) {
        load16(ptr1, s0, n1, pre0);
        or_ids(pre0, s0, 0x7fffffff);
      }
      if (p.debug && part == 0 && row >= 0)
        for (int s = 0; s < p.c; ++s) p.cand_scores[(size_t)g * p.c + s] = __int_as_float(0x7fc00000);
      if (__any_sync(FULL, bad) && lane == 0) atomicOr(p.status, RR_STATUS_BAD_INDEX);
      n_ok = __reduce_add_sync(FULL, n_ok);
      if (lane == 0) atomicAdd(&s_cnt[1], (unsigned long long)n_ok);
    }
    consumers_sync();                    // a row's bitmap is read by warps that did not build it

    float amin = pinf, bmax = ninf, nmin = pinf;      // nmin: weakest near-miss candidate
    bool alive = true;
    const uint32_t sh = (uint32_t)part * COLS;
    RD_LAP(1);
    for (int t = 0; t < n_tiles; ++t) {
      // after a wait that gave up the remaining iterations only keep the barriers in step
      // (test hook: the first wait of CTA 0 counts as expired)
      if (force_timeout && blockIdx.x == 0 && t == 0) { pipe.ctl->abort_flag = 1u; alive = false; }
      if (alive) alive = pipe.consumer_wait(t);
      RD_LAP(2);
      static_assert(COLS == 32, "a thread's share of a tile is one bitmap word");
      const int wi = t * TPR + part;                       // this thread's word of either plane
      const bool in = alive && wi < words;
      const uint32_t wa = in ? lds(bA + wi * 4u) : 0u, wb = in ? lds(bB + wi * 4u) : 0u;
      const uint32_t wr = PRIOR ? wa & ~wb : wa, wn = wb & ~wa, ws = wb;
      const bool work = __any_sync(FULL, (wa | wb) != 0u);
      uint32_t a0[COLS];
      if (work) {
        tmem_ld_32x32(pipe.acc_addr(t, quarter) + sh, a0);
        // masked min / max straight from the registers: no loop over set bits (its trip
        // count and its dependent shared-memory reads made it several times slower)
#pragma unroll
        for (int q = 0; q < COLS; ++q) {
          const float s0 = __uint_as_float(a0[q]);
          min_if(amin, s0, wr, 1u << q);
          max_if(bmax, s0, ws, 1u << q);
          if constexpr (PRIOR) min_if(nmin, s0, wn, 1u << q);
        }
      }
      if (p.debug) {                                         // tests: every candidate's score
        if (work) {
#pragma unroll
          for (int q = 0; q < COLS; ++q) sts(col + (sh + q) * PITCH, a0[q]);
        }
        consumers_sync();
        if (alive && part == 0 && row >= 0) {
          const int32_t* route = p.routes + (size_t)g * p.k;
          const int32_t* sent = p.sentinels + (size_t)g * p.sw;
          for (int s = 0; s < p.c; ++s) {
            const int id = s < p.k ? route[s] : sent[s - p.k];
            const int rel = id - t * BN;
            if (id >= 0 && id < v && rel >= 0 && rel < BN)
              p.cand_scores[(size_t)g * p.c + s] = __uint_as_float(lds(col + (uint32_t)rel * PITCH));
          }
        }
        consumers_sync();
      }
      if (alive) pipe.consumer_release(t);
      RD_LAP(3);
    }

    RD_FLUSH();
    // ---- the second thread of each row hands its partial results to the first ---------------
    if (part != 0) {
      sts(xch_base + r * 4u, __float_as_uint(amin));
      sts(xch_base + PITCH + r * 4u, __float_as_uint(bmax));
      sts(xch_base + 2u * PITCH + r * 4u, __float_as_uint(nmin));
    }
    consumers_sync();
    if (part == 0) {
      amin = fminf(amin, __uint_as_float(lds(xch_base + r * 4u)));
      bmax = fmaxf(bmax, __uint_as_float(lds(xch_base + PITCH + r * 4u)));
      nmin = fminf(nmin, __uint_as_float(lds(xch_base + 2u * PITCH + r * 4u)));
      const bool ok = alive && row >= 0;
      const bool flag = ok && rr_challenge(p, g, amin, bmax);
      if (ok) {
        p.flags[g] = flag ? 1 : 0;
        p.alpha[g] = amin;
        p.beta[g] = bmax;
        p.tau[g] = (PRIOR && p.m > 0) ? fminf(amin, nmin) : ninf;    // floor of the k+m old candidates
      }
      const int n_flag = __popc(__ballot_sync(FULL, flag));
      const int v_sum = __reduce_add_sync(FULL, flag ? v : 0);
      if (lane == 0) {
        atomicAdd(&s_cnt[0], (unsigned long long)n_flag);
        atomicAdd(&s_cnt[2], (unsigned long long)v_sum);
      }
    }
  }

  pipe.teardown(p);                                           // includes a __syncthreads()
  if (tid == 0) {
    p.tile_counts[tile_id] = (int)s_cnt[0];
    atomicAdd(&p.counters[RR_CNT_FLAGGED_ROWS], s_cnt[0]);
    atomicAdd(&p.counters[RR_CNT_CAND_PAIRS], s_cnt[1]);
    atomicAdd(&p.counters[RR_CNT_FULL_PAIRS], s_cnt[2]);
  }
}

size_t smem_need(const RRParams& p, int& words) {
  words = (p.n_k + 31) / 32;
  const size_t fixed = p.d == 128 ? tcpipe::Pipe<128, BN, B_STAGES, ACC_STAGES, NCONS>::FIXED_BYTES
                                  : tcpipe::Pipe<64, BN, B_STAGES, ACC_STAGES, NCONS>::FIXED_BYTES;
  return fixed + (size_t)tcpipe::BM * (2 * words + 1) * 4 + 16 + (size_t)(3 + (p.debug ? BN : 0)) * PITCH + 64;
}

}  // namespace

#ifdef RR_PHASE_TIMING
extern "C" int rr_debug_rd_phase_counters(unsigned long long* out8, int reset) {
  cudaDeviceSynchronize();
  if (cudaMemcpyFromSymbol(out8, g_rd_phase, sizeof(unsigned long long) * 8) != cudaSuccess) return -1;
  if (reset) { unsigned long long z[8] = {}; cudaMemcpyToSymbol(g_rd_phase, z, sizeof z); }
  return 0;
}
#endif

bool rr_rescore_dense_supported(const RRParams& p) {
  int words;
  return p.dtype == RR_BF16 && smem_need(p, words) <= 227 * 1024;
}

cudaError_t rr_launch_rescore_dense(const RRParams& p, const void* qc, const void* kc,
                                    int force_timeout, bool prior, cudaStream_t st) {
  int words;
  const size_t smem = smem_need(p, words);
  CUtensorMap tmap, tmap_q;
  cudaError_t e = rr_encode_tmap_bf16_3d(&tmap, kc, p.d, p.n_k, p.P, BN);
  if (e != cudaSuccess) return e;
  e = rr_encode_tmap_bf16_3d(&tmap_q, qc, p.d, p.n_q, p.P, tcpipe::BM);
  if (e != cudaSuccess) return e;
  static unsigned long long attr_done = 0;      // devices on which the attributes are set
  e = rr_once_per_device(attr_done, [] {
    const void* kernels[4] = {(const void*)rescore_dense_kernel<128, true>, (const void*)rescore_dense_kernel<128, false>,
                              (const void*)rescore_dense_kernel<64, true>, (const void*)rescore_dense_kernel<64, false>};
    for (const void* k : kernels) {
      const cudaError_t a = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (a != cudaSuccess) return a;
      cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    }
    return cudaSuccess;
  });
  if (e != cudaSuccess) return e;
  const int grid = p.n_tiles;
  if (p.d == 128) {
    if (prior) rescore_dense_kernel<128, true><<<grid, NT, smem, st>>>(p, tmap_q, tmap, words, force_timeout);
    else rescore_dense_kernel<128, false><<<grid, NT, smem, st>>>(p, tmap_q, tmap, words, force_timeout);
  } else {
    if (prior) rescore_dense_kernel<64, true><<<grid, NT, smem, st>>>(p, tmap_q, tmap, words, force_timeout);
    else rescore_dense_kernel<64, false><<<grid, NT, smem, st>>>(p, tmap_q, tmap, words, force_timeout);
  }
  rr_count_launch();
  return cudaPeekAtLastError();
}
