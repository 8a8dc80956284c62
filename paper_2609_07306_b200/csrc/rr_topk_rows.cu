// Per-row TopK over a score row held in shared memory: route (Eq. 2), near-miss sentinels
// (Section 3.1 item 1), k-th score and margin (Section 3.3), and the random sentinels
// (Section 3.1 item 2) -- one warp per row, writing straight into the ledger row.
//
// Selection is a warp-level radix select on order-preserving 32-bit keys (8 bits per pass,
// shared-memory histogram, shuffle scan), run for rank k and rank k+m.  Ties on a key are
// resolved towards the smaller chunk id by walking the row in index order with ballots.
// Input: score rows S[slot, 0..v) in global memory (fp32), slot = position in the refresh
// list (relay) or the global row id (anchor).
#include "rr_warp_topk.cuh"

namespace {

constexpr int WARPS = 4;

__global__ void __launch_bounds__(WARPS * 32)
topk_rows_kernel(RRParams p, const int32_t* __restrict__ row_list, uint32_t layer) {
  extern __shared__ uint32_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nk_pad = (p.n_k + 31) & ~31;
  const int per_warp = nk_pad + 256 + nk_pad / 32;
  uint32_t* keys = smem + (size_t)warp * per_warp;
  uint32_t* hist = keys + nk_pad;
  uint32_t* bitmap = hist + 256;

  const int slot = blockIdx.x * WARPS + warp;
  const int count = row_list ? *p.refresh_count : p.rows;
  if (slot >= count) return;
  const int g = row_list ? row_list[slot] : slot;
  const int i = g % p.n_q;
  const int v = rr_valid_count(i, p.n_k, p.causal, p.causal_offset);
  const float* srow = p.S + (size_t)slot * p.n_k;
  for (int j = lane; j < v; j += 32) keys[j] = rr_order_key(srow[j]);
  __syncwarp();
  warptopk::route_row(p, keys, hist, bitmap, g, v, layer, lane);
}

}  // namespace

cudaError_t rr_launch_topk_rows(const RRParams& p, const int32_t* row_list, int layer,
                                cudaStream_t st) {
  const int nk_pad = (p.n_k + 31) & ~31;
  const size_t smem = (size_t)WARPS * (nk_pad + 256 + nk_pad / 32) * sizeof(uint32_t);
  static unsigned long long attr_done = 0;      // devices on which the attributes are set
  const cudaError_t e = rr_once_per_device(attr_done, [] {
    return cudaFuncSetAttribute(topk_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                96 * 1024);
  });
  if (e != cudaSuccess) return e;
  const int grid = (p.rows + WARPS - 1) / WARPS;
  topk_rows_kernel<<<grid, WARPS * 32, smem, st>>>(p, row_list, (uint32_t)layer);
  rr_count_launch();
  return cudaPeekAtLastError();
}
