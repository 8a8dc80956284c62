// Candidate rescoring + challenge test (Section 3.2, Eq. 5; Section 4.2 first kernel).
//
// One warp per query row.  The row's candidate ids are the ledger's route row followed by
// its sentinel row (the join is a view, never materialised).  Each candidate's Kc row is
// fetched with 16-byte loads -- `LPC` lanes cover one row, so a warp scores 32/LPC candidates
// per step -- multiplied against the query row held in registers, and reduced with
// shuffles.  alpha = min over route slots, beta = max over sentinel slots,
// flag = has_sentinel && !(alpha > beta + gamma)   (a NaN therefore flags the row).
// A CTA covers one tile of RR_ROW_TILE rows of one problem and also emits that tile's
// flagged-row count for the compaction scan, plus the work counters.
#include "rr_common.cuh"

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int WARPS = 8;

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* ptr, float (&out)[8]) {
    float4 v = __ldg(reinterpret_cast<const float4*>(ptr));
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* ptr, float (&out)[8]) {
    uint4 v = __ldg(reinterpret_cast<const uint4*>(ptr));
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      out[2 * q] = __uint_as_float(w[q] << 16);
      out[2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
    }
  }
};

template <typename T, int LPC>
__global__ void __launch_bounds__(WARPS * 32)
rescore_kernel(RRParams p, const T* __restrict__ qc, const T* __restrict__ kc) {
  constexpr int N = Vec16<T>::N;          // elements per 16-byte load; d == N * LPC
  constexpr int CPI = 32 / LPC;           // candidates per warp step
  __shared__ int s_flagged;
  __shared__ unsigned long long s_cand, s_full;
  if (p.force_threshold > 0 && p.force_in[0] > 0) return;   // forced anchor: nothing is tested
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int prob = blockIdx.x / p.tiles_per_problem;
  const int tile = blockIdx.x % p.tiles_per_problem;
  if (threadIdx.x == 0) { s_flagged = 0; s_cand = 0; s_full = 0; }
  __syncthreads();

  const T* kbase = kc + (size_t)prob * p.n_k * p.d;
  const int sub = lane % LPC, grp = lane / LPC;
  const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);
  int my_flagged = 0;
  unsigned long long my_cand = 0, my_full = 0;
  const float err_scale = 4.0f * (float)p.d * 5.9604645e-8f;     // 2 sides x safety 2

  const int row_end = min(p.n_q, (tile + 1) * RR_ROW_TILE);
  for (int i = tile * RR_ROW_TILE + warp; i < row_end; i += WARPS) {
    const int g = prob * p.n_q + i;
    const int v = rr_valid_count(i, p.n_k, p.causal, p.causal_offset);
    float q[8];
    Vec16<T>::load(qc + (size_t)g * p.d + sub * N, q);
    const int32_t* route = p.routes + (size_t)g * p.k;
    const int32_t* sent = p.sentinels + (size_t)g * p.sw;
    float amin = pinf, bmax = ninf, nmin = pinf;   // nmin: safe floor of route+near-miss scores
    int n_valid = 0;
    bool bad = false;
    for (int s0 = 0; s0 < p.c; s0 += CPI) {
      const int slot = s0 + grp;
      int idx = -1;
      if (slot < p.k) idx = route[slot];
      else if (slot < p.c) idx = sent[slot - p.k];
      if (idx >= v) { bad = true; idx = -1; }
      float acc = 0.f, mag = 0.f;            // mag = sum |q_t k_t|: scale of the rounding error
      if (idx >= 0) {
        float kv[8];
        Vec16<T>::load(kbase + (size_t)idx * p.d + sub * N, kv);
#pragma unroll
        for (int e = 0; e < N; ++e) {
          acc = fmaf(q[e], kv[e], acc);
          mag = fmaf(fabsf(q[e]), fabsf(kv[e]), mag);
        }
      }
#pragma unroll
      for (int off = LPC / 2; off; off >>= 1) {
        acc += __shfl_xor_sync(FULL, acc, off);
        mag += __shfl_xor_sync(FULL, mag, off);
      }
      if (idx >= 0) {
        if (slot < p.k) amin = fminf(amin, acc); else bmax = fmaxf(bmax, acc);
        // lower bound of this candidate's score under ANY fp32 summation order (the refresh
        // recomputes it on the tensor cores): |error| <= d * 2^-24 * sum|q_t k_t| per side
        if (slot < p.k + p.m) nmin = fminf(nmin, acc - err_scale * mag);
        if (sub == 0) ++n_valid;
      }
      if (p.debug && sub == 0 && slot < p.c)
        p.cand_scores[(size_t)g * p.c + slot] = idx >= 0 ? acc : __int_as_float(0x7fc00000);
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
      amin = fminf(amin, __shfl_xor_sync(FULL, amin, off));
      bmax = fmaxf(bmax, __shfl_xor_sync(FULL, bmax, off));
      nmin = fminf(nmin, __shfl_xor_sync(FULL, nmin, off));
      n_valid += __shfl_xor_sync(FULL, n_valid, off);
    }
    if (__any_sync(FULL, bad) && lane == 0) atomicOr(p.status, RR_STATUS_BAD_INDEX);
    const bool flag = rr_challenge(p, g, amin, bmax);
    if (lane == 0) {
      p.flags[g] = flag ? 1 : 0;
      p.alpha[g] = amin;
      p.beta[g] = bmax;
      // Warm start for the refresh: the route and near-miss candidates are k+m distinct
      // chunks, so at least k+m scores of this row reach the floor of their current scores
      // -- a valid (inclusive) lower bound for everything the new route and near-miss set
      // can contain.
      p.tau[g] = p.m > 0 ? nmin : ninf;
      my_flagged += flag;
      my_cand += (unsigned long long)n_valid;
      if (flag) my_full += (unsigned long long)v;
    }
  }
  if (lane == 0) {
    atomicAdd(&s_flagged, my_flagged);
    atomicAdd(&s_cand, my_cand);
    atomicAdd(&s_full, my_full);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    p.tile_counts[blockIdx.x] = s_flagged;
    atomicAdd(&p.counters[RR_CNT_FLAGGED_ROWS], (unsigned long long)s_flagged);
    atomicAdd(&p.counters[RR_CNT_CAND_PAIRS], s_cand);
    atomicAdd(&p.counters[RR_CNT_FULL_PAIRS], s_full);
  }
}

}  // namespace

cudaError_t rr_launch_rescore(const RRParams& p, const void* qc, const void* kc,
                              cudaStream_t st) {
  const int grid = p.n_tiles, nt = WARPS * 32;
  const int row_bytes = p.d * (p.dtype == RR_F32 ? 4 : 2);
  if (p.dtype == RR_F32) {
    const float* q = (const float*)qc; const float* k = (const float*)kc;
    if (row_bytes == 256) rescore_kernel<float, 16><<<grid, nt, 0, st>>>(p, q, k);
    else rescore_kernel<float, 32><<<grid, nt, 0, st>>>(p, q, k);
  } else {
    const __nv_bfloat16* q = (const __nv_bfloat16*)qc; const __nv_bfloat16* k = (const __nv_bfloat16*)kc;
    if (row_bytes == 256) rescore_kernel<__nv_bfloat16, 16><<<grid, nt, 0, st>>>(p, q, k);
    else rescore_kernel<__nv_bfloat16, 8><<<grid, nt, 0, st>>>(p, q, k);
  }
  rr_count_launch();
  return cudaPeekAtLastError();
}
