// The producer side of the tensor-core score kernels: one CTA owns BM = 128 query rows of one
// problem and streams score tiles S[128 rows, BN key chunks] into a ring of TMEM accumulators.
//   warp 0, lane 0 : TMA producer -- Kc tiles (bf16, 128-byte swizzle, no multicast) into a ring
//                    of B_STAGES shared-memory stages
//   warp 1, lane 0 : issues tcgen05.mma (M=128, N=BN, K=16; d/16 steps per tile) into a ring of
//                    ACC_STAGES TMEM accumulators of BN columns and commits to mbarriers
//   consumers      : CONSUMERS threads (one or more per row); wait on acc_full[stage], read
//                    TMEM with tcgen05.ld, then arrive on acc_empty[stage]
// The Qc tile is gathered by all threads with 16-byte loads straight into the swizzled layout
// the MMA descriptors expect (rows of a refresh list are not contiguous in memory); when the
// rows are consecutive the caller may hand a tensor map of Qc instead, and the producer fetches
// the tile with TMA while the consumers are already busy with their own set-up.
// Every mbarrier wait is bounded: on expiry the abort flag is raised, every role leaves its
// loop, the CTA frees its TMEM and reports RR_STATUS_TIMEOUT.
#pragma once
#include "rr_common.cuh"
#include "rr_sm100.cuh"

namespace tcpipe {

using namespace sm100;

constexpr int BM = 128;

template <int D, int BN, int B_STAGES, int ACC_STAGES, int CONSUMERS = BM>
struct Pipe {
  static constexpr int KHALVES = D / 64, KSTEPS = D / 16;
  static constexpr int A_BYTES = BM * D * 2, B_BYTES = BN * D * 2;
  static constexpr int A_HALF = BM * 128, B_HALF = BN * 128;     // rows x 128 bytes (64 bf16)
  static constexpr int TMEM_COLS = ACC_STAGES * BN;              // must be a power of two >= 32
  static constexpr int CTL_BYTES = 2048;
  static constexpr int FIXED_BYTES = 1024 + A_BYTES + B_STAGES * B_BYTES + CTL_BYTES;

  struct Ctl {
    uint64_t full[B_STAGES], empty[B_STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
    uint64_t a_full;                                      // Qc tile landed (TMA variant only)
    uint64_t drain;                                       // all MMAs of the issuer have finished
    uint32_t tmem_base, abort_flag;
    int row[BM], slot[BM];
  };
  static_assert(sizeof(Ctl) <= CTL_BYTES, "control block too large");

  uint8_t* sA; uint8_t* sB; Ctl* ctl; uint8_t* extra;   // extra: what follows the fixed part

  __device__ __forceinline__ void carve(uint8_t* smem_raw) {
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    sA = smem; sB = smem + A_BYTES;
    ctl = (Ctl*)(smem + A_BYTES + B_STAGES * B_BYTES);
    extra = (uint8_t*)ctl + CTL_BYTES;
  }

  // Row table, barriers, TMEM allocation, Qc tile.  Call with all threads; ends in a
  // __syncthreads().  rows come from row_list[seg_lo + tm*BM ...) (relay) or are consecutive.
  // tmap_q != nullptr (consecutive rows only): the Qc tile is left to producer().
  __device__ __forceinline__ void setup(const RRParams& p, const __nv_bfloat16* qc,
                                        const CUtensorMap* tmap_k, const int32_t* row_list,
                                        int prob, int tm, int seg_lo, int seg_hi, int nthreads,
                                        const CUtensorMap* tmap_q = nullptr) {
    const int tid = threadIdx.x, warp = tid >> 5;
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
      for (int s = 0; s < ACC_STAGES; ++s) { mbar_init(&ctl->acc_full[s], 1); mbar_init(&ctl->acc_empty[s], CONSUMERS); }
      mbar_init(&ctl->a_full, 1);
      mbar_init(&ctl->drain, 1);
      ctl->abort_flag = 0;
      mbar_fence_init();
      tma_prefetch_desc(tmap_k);
      if (tmap_q) tma_prefetch_desc(tmap_q);
    }
    if (warp == 0) tmem_alloc(&ctl->tmem_base, TMEM_COLS);
    if (tmap_q) {
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
      return;
    }
    __syncthreads();
    constexpr int CPR = D / 8;                            // 16-byte chunks per row
    const __nv_bfloat16* qbase = qc + (size_t)prob * p.n_q * D;
    for (int ch = tid; ch < BM * CPR; ch += nthreads) {
      const int r = ch / CPR, c16 = ch % CPR, h = c16 >> 3, cc = c16 & 7;
      const int row = ctl->row[r];
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row >= 0) v = __ldg(reinterpret_cast<const uint4*>(qbase + (size_t)row * D + c16 * 8));
      *reinterpret_cast<uint4*>(sA + h * A_HALF + r * 128 + ((cc ^ (r & 7)) << 4)) = v;
    }
    fence_proxy_async_smem();                             // generic writes -> async proxy (MMA)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }

  // rows ascend inside a tile: the last present row has the largest valid count
  __device__ __forceinline__ int num_tiles(const RRParams& p) const {
    int last = -1;
    for (int t = BM - 1; t >= 0; --t) if (ctl->row[t] >= 0) { last = ctl->row[t]; break; }
    const int vmax = rr_valid_count(last, p.n_k, p.causal, p.causal_offset);
    return (vmax + BN - 1) / BN;
  }

  __device__ __forceinline__ void producer(const CUtensorMap* tmap_k, int prob, int n_tiles,
                                           const CUtensorMap* tmap_q = nullptr, int tm = 0) {
    volatile uint32_t* abort_flag = &ctl->abort_flag;
    if (tmap_q) {                                         // rows past n_q are zero-filled
      mbar_expect_tx(&ctl->a_full, A_BYTES);
#pragma unroll
      for (int h = 0; h < KHALVES; ++h)
        tma_load_3d(sA + h * A_HALF, tmap_q, h * 64, tm * BM, prob, &ctl->a_full);
    }
    int issued = 0;
    for (int t = 0; t < n_tiles; ++t) {
      const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
      if (!mbar_wait_relaxed(&ctl->empty[s], ph ^ 1, abort_flag, 400)) break;
      mbar_expect_tx(&ctl->full[s], B_BYTES);
#pragma unroll
      for (int h = 0; h < KHALVES; ++h)
        tma_load_3d(sB + s * B_BYTES + h * B_HALF, tmap_k, h * 64, t * BN, prob, &ctl->full[s]);
      ++issued;
    }
    // do not leave while copies into this CTA's shared memory may still be in flight
    for (int t = max(0, issued - B_STAGES); t < issued; ++t) {
      const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
      for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->full[s], ph); ++it) __nanosleep(64);
    }
    if (tmap_q)
      for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->a_full, 0); ++it) __nanosleep(64);
  }

  __device__ __forceinline__ void mma_issuer(int n_tiles, bool q_by_tma = false) {
    volatile uint32_t* abort_flag = &ctl->abort_flag;
    if (q_by_tma && !mbar_wait(&ctl->a_full, 0, abort_flag)) return;
    constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
    const uint32_t a_addr = smem_u32(sA);
    const uint32_t tmem_base = ctl->tmem_base;
    for (int t = 0; t < n_tiles; ++t) {
      const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
      const int as = t % ACC_STAGES; const uint32_t aph = (t / ACC_STAGES) & 1;
      if (!mbar_wait_relaxed(&ctl->acc_empty[as], aph ^ 1, abort_flag, 400)) break;
      if (!mbar_wait_relaxed(&ctl->full[s], ph, abort_flag, 100)) break;
      tc_fence_after();
      const uint32_t b_addr = smem_u32(sB + s * B_BYTES);
#pragma unroll
      for (int k = 0; k < KSTEPS; ++k) {
        const uint32_t a_off = (k >> 2) * A_HALF + (k & 3) * 32;
        const uint32_t b_off = (k >> 2) * B_HALF + (k & 3) * 32;
        umma_bf16(tmem_base + as * BN, umma_desc_k_sw128(a_addr + a_off),
                  umma_desc_k_sw128(b_addr + b_off), idesc, k > 0 ? 1u : 0u);
      }
      umma_commit(&ctl->empty[s]);        // smem stage reusable once these MMAs have read it
      umma_commit(&ctl->acc_full[as]);    // accumulator ready for the consumers
    }
    // TMEM must not be freed while an MMA can still write to it: after a wait that gave up the
    // consumers no longer vouch for that, so the issuer waits (bounded) for its own MMAs
    umma_commit(&ctl->drain);
    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->drain, 0); ++it) __nanosleep(64);
  }

  // Consumer side of one tile: returns false (for the whole warp) if the wait gave up.
  __device__ __forceinline__ bool consumer_wait(int t) {
    const int as = t % ACC_STAGES; const uint32_t aph = (t / ACC_STAGES) & 1;
    const bool ready = mbar_wait(&ctl->acc_full[as], aph, &ctl->abort_flag);
    if (!__all_sync(0xFFFFFFFFu, ready)) return false;
    tc_fence_after();
    return true;
  }
  __device__ __forceinline__ void consumer_release(int t) {
    tc_fence_before();
    mbar_arrive(&ctl->acc_empty[t % ACC_STAGES]);
  }
  __device__ __forceinline__ uint32_t acc_addr(int t, int quarter) const {
    return ctl->tmem_base + ((uint32_t)(quarter * 32) << 16) + (t % ACC_STAGES) * BN;
  }

  // All threads; frees TMEM and reports a timed-out wait.
  __device__ __forceinline__ void teardown(const RRParams& p) {
    tc_fence_before();
    __syncthreads();
    if ((threadIdx.x >> 5) == 0) {
      tc_fence_after();
      tmem_dealloc(ctl->tmem_base, TMEM_COLS);
      if ((threadIdx.x & 31) == 0 && ctl->abort_flag) atomicOr(p.status, RR_STATUS_TIMEOUT);
    }
  }
};

}  // namespace tcpipe
