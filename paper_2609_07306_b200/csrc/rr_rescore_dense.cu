// Candidate rescoring + challenge test (Section 3.2, Eq. 5) on the TENSOR CORES.
//
// The gathered kernel (rr_rescore.cu) fetches c Kc rows per query row and multiplies them on
// the FP32 ALUs: no operand is reused, so it moves c*d*2 bytes per row through L2 and is an
// order of magnitude slower on this machine than computing the whole score strip with
// tcgen05.mma.  This variant does the latter: the same tile pipeline as the fused routing
// kernel produces S[128 rows, 64 chunks] tiles in TMEM, and each row's thread picks out the
// scores of its own candidates:
//   * at start the thread turns its ledger row into three per-row bitmaps in shared memory
//     (route, near-miss, all sentinels);
//   * per tile it reads its 64 scores from TMEM and takes masked minima / maxima under the
//     tile's bitmap words: alpha = min over route bits, beta = max over sentinel bits,
//     floor = min over route and near-miss bits (the refresh's warm-start threshold).
// Scores are bit-identical to the ones the fused routing kernel computes (same instruction
// sequence on the same operands), so the floor needs no safety margin.
// Outputs are those of the gathered kernel: flags, alpha, beta, tau, per-tile flagged counts,
// work counters (the candidate pairs are still charged as c per row: that is what the method
// evaluates; that the hardware computes the strip is an implementation matter).
#include "rr_tc_pipeline.cuh"

using namespace sm100;

namespace {

// 32-chunk tiles keep a CTA under half an SM's shared memory: two CTAs per SM overlap one's
// set-up and bitmap build with the other's tile loop.
constexpr int BN = 32, B_STAGES = 3, ACC_STAGES = 4, NT = 192;
constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr uint32_t PITCH = tcpipe::BM * 4;          // one 32-bit word per row thread

__device__ __forceinline__ uint32_t lds(uint32_t a) {
  uint32_t v; asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a) : "memory"); return v;
}
__device__ __forceinline__ void sts(uint32_t a, uint32_t v) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

#ifdef RR_PHASE_TIMING
__device__ unsigned long long g_rd_phase[8];
#define RD_T0() long long rd_t0_ = clock64()
#define RD_LAP(i) do { const long long t1_ = clock64(); if ((threadIdx.x & 31) == 0) atomicAdd(&g_rd_phase[i], (unsigned long long)(t1_ - rd_t0_)); rd_t0_ = t1_; } while (0)
#else
#define RD_T0() do {} while (0)
#define RD_LAP(i) do {} while (0)
#endif

template <int D>
__global__ void __launch_bounds__(NT, 2)
rescore_dense_kernel(RRParams p, const __nv_bfloat16* __restrict__ qc,
                     const __grid_constant__ CUtensorMap tmap_k, int words) {
  using P = tcpipe::Pipe<D, BN, B_STAGES, ACC_STAGES>;
  extern __shared__ uint8_t smem_raw[];
  P pipe;
  pipe.carve(smem_raw);
  // extra: 3 counters, [3*words][128] bitmap words, (debug only) [BN][128] score column
  unsigned long long* s_cnt = (unsigned long long*)pipe.extra;
  const uint32_t bm_base = smem_u32(pipe.extra) + 64u;
  const uint32_t sc_base = bm_base + 3u * words * PITCH;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles_m = p.tiles_per_problem;
  const int prob = blockIdx.x % p.P, tm = tiles_m - 1 - blockIdx.x / p.P;   // heaviest first
  const int tile_id = prob * tiles_m + tm;
  if (tid == 0) { s_cnt[0] = 0; s_cnt[1] = 0; s_cnt[2] = 0; }
  RD_T0();
  pipe.setup(p, qc, &tmap_k, nullptr, prob, tm, 0, p.n_q, NT);
  const int n_tiles = pipe.num_tiles(p);

  if (warp == 0) {
    if (lane == 0) pipe.producer(&tmap_k, prob, n_tiles);
  } else if (warp == 1) {
    if (lane == 0) pipe.mma_issuer(n_tiles);
  } else {
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const int row = pipe.ctl->row[r];
    const int g = pipe.ctl->slot[r];
    const int v = row >= 0 ? rr_valid_count(row, p.n_k, p.causal, p.causal_offset) : 0;
    const uint32_t bR = bm_base + r * 4u, bN = bR + words * PITCH, bS = bN + words * PITCH;
    const uint32_t col = sc_base + r * 4u;
    const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);

    RD_LAP(0);
    // ---- ledger row -> bitmaps ---------------------------------------------------------------
    for (int w = 0; w < 3 * words; ++w) sts(bR + w * PITCH, 0u);
    int n_valid = 0; bool bad = false;
    if (row >= 0) {
      const int32_t* route = p.routes + (size_t)g * p.k;
      const int32_t* sent = p.sentinels + (size_t)g * p.sw;
      // ids are fetched 16 at a time, all loads first: one L2 round trip per group, not per id
      for (int s0 = 0; s0 < p.c; s0 += 16) {
        int ids[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int s = s0 + j;
          ids[j] = s < p.k ? __ldg(route + s) : (s < p.c ? __ldg(sent + (s - p.k)) : -1);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int s = s0 + j, id = ids[j];
          bad |= id >= v;
          const bool ok = (id >= 0) & (id < v);
          const uint32_t wi = ok ? (uint32_t)(id >> 5) : 0u, bit = ok ? 1u << (id & 31) : 0u;
          const uint32_t a = (s < p.k ? bR : bS) + wi * PITCH;
          sts(a, lds(a) | bit);
          if (s >= p.k && s < p.k + p.m) { const uint32_t an = bN + wi * PITCH; sts(an, lds(an) | bit); }
          n_valid += ok;
          if (p.debug && s < p.c) p.cand_scores[(size_t)g * p.c + s] = __int_as_float(0x7fc00000);
        }
      }
    }
    if (__any_sync(FULL, bad) && lane == 0) atomicOr(p.status, RR_STATUS_BAD_INDEX);

    float amin = pinf, bmax = ninf, nmin = pinf;      // nmin: weakest near-miss candidate
    bool alive = true;
    RD_LAP(1);
    for (int t = 0; t < n_tiles; ++t) {
      if (!pipe.consumer_wait(t)) { alive = false; break; }
      RD_LAP(2);
      static_assert(BN == 32, "a tile is one bitmap word");
      const bool in = t < words;
      const uint32_t wr = in ? lds(bR + t * PITCH) : 0u, wn = in ? lds(bN + t * PITCH) : 0u;
      const uint32_t ws = in ? lds(bS + t * PITCH) : 0u;
      if (__any_sync(FULL, (wr | ws) != 0u)) {
        uint32_t a0[32];
        tmem_ld_32x32(pipe.acc_addr(t, quarter), a0);
        // masked min / max straight from the registers: no loop over set bits (its trip
        // count and its dependent shared-memory reads made it several times slower)
#pragma unroll
        for (int q = 0; q < 32; ++q) {
          const float s0 = __uint_as_float(a0[q]);
          const uint32_t bit = 1u << q;
          amin = fminf(amin, (wr & bit) ? s0 : pinf);
          bmax = fmaxf(bmax, (ws & bit) ? s0 : ninf);
          nmin = fminf(nmin, (wn & bit) ? s0 : pinf);
        }
        if (p.debug) {
#pragma unroll
          for (int q = 0; q < 32; ++q) sts(col + q * PITCH, a0[q]);
        }
        if (p.debug && row >= 0) {                            // tests: every candidate's score
          const int32_t* route = p.routes + (size_t)g * p.k;
          const int32_t* sent = p.sentinels + (size_t)g * p.sw;
          for (int s = 0; s < p.c; ++s) {
            const int id = s < p.k ? route[s] : sent[s - p.k];
            const int rel = id - t * BN;
            if (id >= 0 && id < v && rel >= 0 && rel < BN)
              p.cand_scores[(size_t)g * p.c + s] = __uint_as_float(lds(col + (uint32_t)rel * PITCH));
          }
        }
      }
      pipe.consumer_release(t);
      RD_LAP(3);
    }

    if (alive && row >= 0) {
      const bool has_sent = bmax > ninf;
      const bool flag = has_sent && !(amin > bmax + p.gamma);
      p.flags[g] = flag ? 1 : 0;
      p.alpha[g] = amin;
      p.beta[g] = bmax;
      p.tau[g] = p.m > 0 ? fminf(amin, nmin) : ninf;    // floor of the k+m old candidates
      atomicAdd(&s_cnt[0], (unsigned long long)flag);
      atomicAdd(&s_cnt[1], (unsigned long long)n_valid);
      if (flag) atomicAdd(&s_cnt[2], (unsigned long long)v);
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
  const size_t fixed = p.d == 128 ? tcpipe::Pipe<128, BN, B_STAGES, ACC_STAGES>::FIXED_BYTES
                                  : tcpipe::Pipe<64, BN, B_STAGES, ACC_STAGES>::FIXED_BYTES;
  return fixed + (size_t)(3 * words + (p.debug ? BN : 0)) * PITCH + 64;
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
                                    cudaStream_t st) {
  int words;
  const size_t smem = smem_need(p, words);
  CUtensorMap tmap;
  cudaError_t e = rr_encode_tmap_bf16_3d(&tmap, kc, p.d, p.n_k, p.P, BN);
  if (e != cudaSuccess) return e;
  static bool attr_set = false;
  if (!attr_set) {
    e = cudaFuncSetAttribute(rescore_dense_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             227 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(rescore_dense_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             227 * 1024);
    if (e != cudaSuccess) return e;
    cudaFuncSetAttribute(rescore_dense_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    cudaFuncSetAttribute(rescore_dense_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    attr_set = true;
  }
  const int grid = p.n_tiles;
  if (p.d == 128)
    rescore_dense_kernel<128><<<grid, NT, smem, st>>>(p, (const __nv_bfloat16*)qc, tmap, words);
  else
    rescore_dense_kernel<64><<<grid, NT, smem, st>>>(p, (const __nv_bfloat16*)qc, tmap, words);
  rr_count_launch();
  return cudaPeekAtLastError();
}
