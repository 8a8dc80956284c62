// A minimal consumer of the routes (Eq. 3): o_i = softmax(q_i K_R^T * scale) V_R over the tokens
// R that row i's token ranges cover -- the ranges rr_route_* writes when chunk_tokens > 0, one per
// route slot or, with coalesce_ranges, one per run of consecutive chunks.  It shows that the
// range layout is directly consumable and gives the tests an end-to-end check; it is a plain
// SIMT kernel (one warp per query row, FP32 arithmetic), not a tuned attention backend: the
// paper leaves the sparse-attention backend unchanged (Section 4.3).
//
// Two passes over the row's tokens, both in ascending token order: (1) the maximum logit,
// (2) the sums of exp(logit - max) and exp(logit - max) * V.  Lane t of a step computes the
// logit of one token (a dh-long dot product); the weighted values are then accumulated token by
// token, every lane owning dh / 32 output dimensions.  Because every sum runs in token order and
// a token's logit does not depend on how tokens are grouped into ranges, coalesced and
// per-slot ranges give bit-identical outputs.
#include "rr_common.cuh"

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int WARPS = 4, MAX_DH = 256;

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__global__ void __launch_bounds__(WARPS * 32)
attend_ranges_kernel(const int32_t* __restrict__ ranges, int rows, int slots, int n_q,
                     const T* __restrict__ q, const T* __restrict__ keys, const T* __restrict__ values,
                     int tokens, int dh, float scale, float* __restrict__ out) {
  __shared__ float s_q[WARPS][MAX_DH];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * WARPS + warp;
  if (row >= rows) return;
  const int prob = row / n_q;
  for (int e = lane; e < dh; e += 32) s_q[warp][e] = to_f32(q[(size_t)row * dh + e]);
  __syncwarp();
  const T* kp = keys + (size_t)prob * tokens * dh;
  const T* vp = values + (size_t)prob * tokens * dh;
  const int32_t* rg = ranges + (size_t)row * slots * 2;
  const float ninf = __int_as_float(0xff800000);

  auto logit = [&](int t) -> float {
    const T* kr = kp + (size_t)t * dh;
    float acc = 0.f;
    for (int e = 0; e < dh; ++e) acc = fmaf(s_q[warp][e], to_f32(kr[e]), acc);
    return acc * scale;
  };
  // pass 1: the maximum logit
  float mx = ninf;
  for (int s = 0; s < slots; ++s) {
    const int lo = rg[2 * s], hi = min(rg[2 * s + 1], tokens);
    if (lo < 0) continue;
    for (int t0 = lo; t0 < hi; t0 += 32) {
      const int t = t0 + lane;
      if (t < hi) mx = fmaxf(mx, logit(t));
    }
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, off));
  // pass 2: sums in token order; lane owns output dimensions lane, lane + 32, ...
  float acc[MAX_DH / 32];
#pragma unroll
  for (int i = 0; i < MAX_DH / 32; ++i) acc[i] = 0.f;
  float denom = 0.f;
  for (int s = 0; s < slots; ++s) {
    const int lo = rg[2 * s], hi = min(rg[2 * s + 1], tokens);
    if (lo < 0) continue;
    for (int t0 = lo; t0 < hi; t0 += 32) {
      const int t = t0 + lane;
      const float w = t < hi ? expf(logit(t) - mx) : 0.f;
      const int n = min(32, hi - t0);
      for (int u = 0; u < n; ++u) {
        const float wu = __shfl_sync(FULL, w, u);
        denom += wu;
        const T* vr = vp + (size_t)(t0 + u) * dh;
#pragma unroll
        for (int i = 0; i < MAX_DH / 32; ++i)
          if (lane + 32 * i < dh) acc[i] = fmaf(wu, to_f32(vr[lane + 32 * i]), acc[i]);
      }
    }
  }
  const float inv = denom > 0.f ? 1.f / denom : 0.f;
#pragma unroll
  for (int i = 0; i < MAX_DH / 32; ++i)
    if (lane + 32 * i < dh) out[(size_t)row * dh + lane + 32 * i] = acc[i] * inv;
}

}  // namespace

extern "C" int rr_attend_token_ranges(const int32_t* ranges, int32_t rows, int32_t slots, int32_t n_q,
                                      const void* q, const void* keys, const void* values,
                                      int32_t tokens, int32_t dh, int32_t dtype, float scale,
                                      float* out, void* stream) {
  if (!ranges || !q || !keys || !values || !out) return RR_ERR_INVALID_ARG;
  if (rows <= 0 || slots <= 0 || n_q <= 0 || rows % n_q != 0 || tokens <= 0) return RR_ERR_INVALID_ARG;
  if (dh <= 0 || dh > MAX_DH) return RR_ERR_UNSUPPORTED;
  if (dtype != RR_BF16 && dtype != RR_F32) return RR_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  const int grid = (rows + WARPS - 1) / WARPS;
  if (dtype == RR_BF16)
    attend_ranges_kernel<__nv_bfloat16><<<grid, WARPS * 32, 0, st>>>(
        ranges, rows, slots, n_q, (const __nv_bfloat16*)q, (const __nv_bfloat16*)keys,
        (const __nv_bfloat16*)values, tokens, dh, scale, out);
  else
    attend_ranges_kernel<float><<<grid, WARPS * 32, 0, st>>>(
        ranges, rows, slots, n_q, (const float*)q, (const float*)keys, (const float*)values, tokens,
        dh, scale, out);
  rr_count_launch();
  return cudaPeekAtLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}
