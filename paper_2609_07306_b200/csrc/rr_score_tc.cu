// Score rows on the 5th-generation tensor cores (Eq. 1): S[slot, j] = <Qc[row], Kc[j]>,
// bf16 x bf16 -> fp32, written to the score-row scratch for the TopK kernel.
//
// One CTA owns 128 query rows of one problem -- consecutive rows at an anchor, a segment of
// the compacted refresh list at a relay (Section 4.2) -- and walks the key chunks in tiles
// of 128, stopping at the last chunk any of its rows may select (causal tile skipping).
//   warp 0   : TMA producer (Kc tiles, 128-byte swizzle, 3-stage ring, no multicast)
//   warp 1   : one thread issues tcgen05.mma (M=128, N=128, K=16, d/16 steps per tile) into a
//              double-buffered TMEM accumulator and commits to mbarriers
//   warps 2-5: epilogue, one thread per query row: tcgen05.ld 32 columns at a time -> global
// The Qc tile is gathered by all threads with 16-byte loads straight into the swizzled
// layout the MMA descriptors expect (rows of a refresh list are not contiguous).
// Every mbarrier wait is bounded; on expiry the CTA sets RR_STATUS_TIMEOUT, frees its TMEM
// and returns.
#include "rr_common.cuh"
#include "rr_sm100.cuh"

using namespace sm100;

namespace {

constexpr int BM = 128, BN = 128, B_STAGES = 3, ACC_STAGES = 2, NT = 192;
constexpr int TMEM_COLS = ACC_STAGES * BN;     // 256, a power of two

template <int D>
struct Cfg {
  static constexpr int KHALVES = D / 64, KSTEPS = D / 16;
  static constexpr int A_BYTES = BM * D * 2, B_BYTES = BN * D * 2;
  static constexpr int HALF_BYTES = 128 * 128;            // 128 rows x 128 bytes
  static constexpr int SMEM_BYTES = 1024 + A_BYTES + B_STAGES * B_BYTES + 2048;
};

struct Ctl {
  uint64_t full[B_STAGES], empty[B_STAGES], acc_full[ACC_STAGES], acc_empty[ACC_STAGES];
  uint32_t tmem_base, abort_flag;
  int row[BM], slot[BM];
};

template <int D>
__global__ void __launch_bounds__(NT, 1)
score_tc_kernel(RRParams p, const __nv_bfloat16* __restrict__ qc,
                const __grid_constant__ CUtensorMap tmap_k, const int32_t* __restrict__ row_list) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + C::A_BYTES;
  Ctl* ctl = (Ctl*)(smem + C::A_BYTES + B_STAGES * C::B_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles_m = p.tiles_per_problem;
  const int prob = blockIdx.x / tiles_m, tm = blockIdx.x % tiles_m;

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

  // ---- gather the Qc tile into the K-major, 128B-swizzled layout -------------------------
  {
    constexpr int CPR = D / 8;                            // 16-byte chunks per row
    const __nv_bfloat16* qbase = qc + (size_t)prob * p.n_q * D;
    for (int ch = tid; ch < BM * CPR; ch += NT) {
      const int r = ch / CPR, c16 = ch % CPR, h = c16 >> 3, cc = c16 & 7;
      const int row = ctl->row[r];
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row >= 0) v = __ldg(reinterpret_cast<const uint4*>(qbase + (size_t)row * D + c16 * 8));
      *reinterpret_cast<uint4*>(sA + h * C::HALF_BYTES + r * 128 + ((cc ^ (r & 7)) << 4)) = v;
    }
    fence_proxy_async_smem();                             // generic writes -> async proxy (MMA)
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile uint32_t* abort_flag = &ctl->abort_flag;

  // rows ascend inside a tile: the last present row has the largest valid count
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
        if (!mbar_wait(&ctl->empty[s], ph ^ 1, abort_flag)) break;
        mbar_expect_tx(&ctl->full[s], C::B_BYTES);
#pragma unroll
        for (int h = 0; h < C::KHALVES; ++h)
          tma_load_3d(sB + s * C::B_BYTES + h * C::HALF_BYTES, &tmap_k, h * 64, t * BN, prob,
                      &ctl->full[s]);
        ++issued;
      }
      // do not leave while copies into this CTA's shared memory may still be in flight
      for (int t = max(0, issued - B_STAGES); t < issued; ++t) {
        const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&ctl->full[s], ph); ++it) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    // ===== MMA issuer =====
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
      const uint32_t a_addr = smem_u32(sA);
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t % B_STAGES; const uint32_t ph = (t / B_STAGES) & 1;
        const int as = t % ACC_STAGES; const uint32_t aph = (t / ACC_STAGES) & 1;
        if (!mbar_wait(&ctl->acc_empty[as], aph ^ 1, abort_flag)) break;
        if (!mbar_wait(&ctl->full[s], ph, abort_flag)) break;
        tc_fence_after();
        const uint32_t b_addr = smem_u32(sB + s * C::B_BYTES);
#pragma unroll
        for (int k = 0; k < C::KSTEPS; ++k) {
          const uint32_t off = (k >> 2) * C::HALF_BYTES + (k & 3) * 32;
          umma_bf16(tmem_base + as * BN, umma_desc_k_sw128(a_addr + off),
                    umma_desc_k_sw128(b_addr + off), idesc, k > 0 ? 1u : 0u);
        }
        umma_commit(&ctl->empty[s]);        // smem stage reusable once these MMAs have read it
        umma_commit(&ctl->acc_full[as]);    // accumulator ready for the epilogue
      }
    }
  } else {
    // ===== epilogue: one thread per query row =====
    const int quarter = warp & 3;                         // TMEM lane quarter of this warp
    const int r = quarter * 32 + lane;
    const int row = ctl->row[r];
    const int v = row >= 0 ? rr_valid_count(row, p.n_k, p.causal, p.causal_offset) : 0;
    float* out = p.S + (size_t)ctl->slot[r] * p.n_k;
    const bool vec_ok = (p.n_k & 3) == 0;
    for (int t = 0; t < n_tiles; ++t) {
      const int as = t % ACC_STAGES; const uint32_t aph = (t / ACC_STAGES) & 1;
      const bool ready = mbar_wait(&ctl->acc_full[as], aph, abort_flag);
      if (!__all_sync(0xFFFFFFFFu, ready)) break;         // leave as a whole warp
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t acc[32];
        __syncwarp();
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + as * BN + c * 32, acc);
        const int col0 = t * BN + c * 32;
        if (col0 + 32 <= v && vec_ok) {
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<uint4*>(out + col0 + 4 * q) =
                make_uint4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
        } else {
#pragma unroll
          for (int q = 0; q < 32; ++q)
            if (col0 + q < v) out[col0 + q] = __uint_as_float(acc[q]);
        }
      }
      tc_fence_before();
      mbar_arrive(&ctl->acc_empty[as]);
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) ==
            cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  }
  return fn;
}

}  // namespace

cudaError_t rr_encode_tmap_bf16_3d(CUtensorMap* out, const void* base, int d, int rows, int planes,
                                   int box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return cudaErrorNotSupported;
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)planes};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * (cuuint64_t)rows};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides,
                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t rr_launch_score_tc(const RRParams& p, const void* qc, const void* kc,
                               const int32_t* row_list, cudaStream_t st) {
  CUtensorMap tmap;
  cudaError_t e = rr_encode_tmap_bf16_3d(&tmap, kc, p.d, p.n_k, p.P, BN);
  if (e != cudaSuccess) return e;
  const int grid = p.P * p.tiles_per_problem;
  static unsigned long long attr_done = 0;      // devices on which the attributes are set
  e = rr_once_per_device(attr_done, [] {
    const cudaError_t a = cudaFuncSetAttribute(score_tc_kernel<128>,
                                               cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               Cfg<128>::SMEM_BYTES);
    if (a != cudaSuccess) return a;
    return cudaFuncSetAttribute(score_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Cfg<64>::SMEM_BYTES);
  });
  if (e != cudaSuccess) return e;
  if (p.d == 128)
    score_tc_kernel<128><<<grid, NT, Cfg<128>::SMEM_BYTES, st>>>(p, (const __nv_bfloat16*)qc, tmap,
                                                                  row_list);
  else
    score_tc_kernel<64><<<grid, NT, Cfg<64>::SMEM_BYTES, st>>>(p, (const __nv_bfloat16*)qc, tmap,
                                                                row_list);
  rr_count_launch();
  return cudaPeekAtLastError();
}
