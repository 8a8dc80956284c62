// Score rows on the FP32 ALUs: S[slot, j] = <Qc[row], Kc[j]>  (Eq. 1), fp32 accumulate.
//
// This is the path for fp32 inputs (the tensor-core path takes bf16 only).  A CTA computes
// a 64x64 tile of one problem's score matrix; the rows of the tile are either consecutive
// query rows (anchor) or a segment of the compacted refresh list (relay, Section 4.2:
// "complete score rows only for the compacted IDs").  Column tiles that lie entirely
// beyond the last valid chunk of the tile's rows (causal mask) are skipped.
#include "rr_common.cuh"

namespace {

constexpr int TM = 64, TN = 64, TK = 32, NT = 256;

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}

template <typename T>
__global__ void __launch_bounds__(NT)
score_simt_kernel(RRParams p, const T* __restrict__ qc, const T* __restrict__ kc,
                  const int32_t* __restrict__ row_list) {
  __shared__ float As[TK][TM + 1];
  __shared__ float Bs[TK][TN + 1];
  __shared__ int s_row[TM];      // query index inside the problem, -1 = no row
  __shared__ int s_slot[TM];     // row of S to write

  const int tiles_m = (p.n_q + TM - 1) / TM;
  const int prob = blockIdx.x / tiles_m;
  const int tm = blockIdx.x % tiles_m;
  const int col0 = blockIdx.y * TN;
  const int tid = threadIdx.x;

  int seg_lo = 0, seg_hi = p.n_q;
  if (row_list) { seg_lo = p.problem_offsets[prob]; seg_hi = p.problem_offsets[prob + 1]; }
  if (tid < TM) {
    int local = tm * TM + tid;
    int row = -1, slot = 0;
    if (row_list) {
      int s = seg_lo + local;
      if (s < seg_hi) { row = row_list[s] - prob * p.n_q; slot = s; }
    } else if (local < p.n_q) {
      row = local; slot = prob * p.n_q + local;
    }
    s_row[tid] = row; s_slot[tid] = slot;
  }
  __syncthreads();
  // rows ascend inside a tile, so the last present row has the largest valid count
  int last = -1;
  for (int t = TM - 1; t >= 0; --t) if (s_row[t] >= 0) { last = s_row[t]; break; }
  if (last < 0) return;
  const int vmax = rr_valid_count(last, p.n_k, p.causal, p.causal_offset);
  if (col0 >= vmax) return;

  const T* kbase = kc + (size_t)prob * p.n_k * p.d;
  const T* qbase = qc + (size_t)prob * p.n_q * p.d;
  const int tx = tid % 16, ty = tid / 16;      // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4] = {};
  for (int d0 = 0; d0 < p.d; d0 += TK) {
    for (int e = tid; e < TM * TK; e += NT) {
      int rr = e / TK, dd = e % TK;
      int row = s_row[rr];
      As[dd][rr] = row >= 0 ? to_f32(qbase[(size_t)row * p.d + d0 + dd]) : 0.f;
      int col = col0 + rr;
      Bs[dd][rr] = col < p.n_k ? to_f32(kbase[(size_t)col * p.d + d0 + dd]) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int dd = 0; dd < TK; ++dd) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[dd][ty * 4 + i]; b[i] = Bs[dd][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int rr = ty * 4 + i;
    int row = s_row[rr];
    if (row < 0) continue;
    int v = rr_valid_count(row, p.n_k, p.causal, p.causal_offset);
    float* out = p.S + (size_t)s_slot[rr] * p.n_k;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int col = col0 + tx * 4 + j;
      if (col < v) out[col] = acc[i][j];
    }
  }
}

}  // namespace

cudaError_t rr_launch_score_simt(const RRParams& p, const void* qc, const void* kc,
                                 const int32_t* row_list, cudaStream_t st) {
  dim3 grid(p.P * ((p.n_q + TM - 1) / TM), (p.n_k + TN - 1) / TN);
  if (p.dtype == RR_F32)
    score_simt_kernel<float><<<grid, NT, 0, st>>>(p, (const float*)qc, (const float*)kc, row_list);
  else
    score_simt_kernel<__nv_bfloat16><<<grid, NT, 0, st>>>(p, (const __nv_bfloat16*)qc,
                                                         (const __nv_bfloat16*)kc, row_list);
  rr_count_launch();
  return cudaPeekAtLastError();
}
