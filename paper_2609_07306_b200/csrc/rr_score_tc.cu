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
#include "rr_tc_pipeline.cuh"

using namespace sm100;

namespace {

constexpr int BN = 128, B_STAGES = 3, ACC_STAGES = 2, NT = 192;
template <int D> using ScorePipe = tcpipe::Pipe<D, BN, B_STAGES, ACC_STAGES, tcpipe::BM>;

template <int D>
__global__ void __launch_bounds__(NT, 1)
score_tc_kernel(RRParams p, const __nv_bfloat16* __restrict__ qc,
                const __grid_constant__ CUtensorMap tmap_k, const int32_t* __restrict__ row_list) {
  extern __shared__ uint8_t smem_raw[];
  ScorePipe<D> pipe;
  pipe.carve(smem_raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = p.tiles_per_problem;
  const int prob = blockIdx.x / tiles_m, tm = blockIdx.x % tiles_m;

  int seg_lo = 0, seg_hi = p.n_q;
  if (row_list) { seg_lo = p.problem_offsets[prob]; seg_hi = p.problem_offsets[prob + 1]; }
  if (tm * tcpipe::BM >= seg_hi - seg_lo) return;         // nothing to do (uniform per CTA)

  // row table, barriers, TMEM, gathered Qc tile (the shared producer / issuer of the score kernels)
  pipe.setup(p, qc, &tmap_k, row_list, prob, tm, seg_lo, seg_hi, NT);
  const int n_tiles = pipe.num_tiles(p);

  if (warp == 0) {
    if (lane == 0) pipe.producer(&tmap_k, prob, n_tiles);
  } else if (warp == 1) {
    if (lane == 0) pipe.mma_issuer(n_tiles);
  } else {
    // ===== epilogue: one thread per query row =====
    const int quarter = warp & 3;                         // TMEM lane quarter of this warp
    const int r = quarter * 32 + lane;
    const int row = pipe.ctl->row[r];
    const int v = row >= 0 ? rr_valid_count(row, p.n_k, p.causal, p.causal_offset) : 0;
    float* out = p.S + (size_t)pipe.ctl->slot[r] * p.n_k;
    const bool vec_ok = (p.n_k & 3) == 0;
    for (int t = 0; t < n_tiles; ++t) {
      if (!pipe.consumer_wait(t)) break;                  // leaves as a whole warp
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t acc[32];
        __syncwarp();
        tmem_ld_32x32(pipe.acc_addr(t, quarter) + c * 32, acc);
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
      pipe.consumer_release(t);
    }
  }
  pipe.teardown(p);
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
                                               ScorePipe<128>::FIXED_BYTES);
    if (a != cudaSuccess) return a;
    return cudaFuncSetAttribute(score_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                ScorePipe<64>::FIXED_BYTES);
  });
  if (e != cudaSuccess) return e;
  if (p.d == 128)
    score_tc_kernel<128><<<grid, NT, ScorePipe<128>::FIXED_BYTES, st>>>(p, (const __nv_bfloat16*)qc, tmap,
                                                                  row_list);
  else
    score_tc_kernel<64><<<grid, NT, ScorePipe<64>::FIXED_BYTES, st>>>(p, (const __nv_bfloat16*)qc, tmap,
                                                                row_list);
  rr_count_launch();
  return cudaPeekAtLastError();
}
