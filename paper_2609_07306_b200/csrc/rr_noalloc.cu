// rr_compact_flags_noalloc: row compaction for callers that cannot allocate device memory.
//
// Some embedders of this library run where cudaMalloc is off limits: inside a memory pool
// that has been frozen for the lifetime of a serving process, inside a plugin whose host
// hands it input and output buffers and nothing else, or on a latency path where an
// allocation (an implicit device synchronisation) is not acceptable.  For them this file
// offers the compaction step (flags -> ascending list of flagged row ids, count, per-problem
// offsets) with its only scratch -- the per-tile flagged counts that the scan consumes -- held
// in a fixed array that is part of the library image.
//
// Every GPU that loads the library carries that array (RR_NOALLOC_MAX_TILES * 4 bytes =
// 256 KB) until the process exits.  All calls share it: it keeps whatever the previous call
// wrote, and two calls whose kernels overlap on the GPU (different streams, or different
// host threads) race on it.  Nothing in it needs to start at zero -- the counting kernel
// overwrites every entry the scan then reads -- so no clearing pass is run.
#include <mutex>
#include "rr_common.cuh"

namespace {

constexpr int kMaxTiles = RR_NOALLOC_MAX_TILES;
constexpr int kMaxDevices = 64;
constexpr unsigned FULL = 0xFFFFFFFFu;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// table, not a device address; the address for kernel arguments comes from
// cudaGetSymbolAddress (see scratch_for_current_device).
static __device__ __align__(256) int32_t g_noalloc_tile_counts[kMaxTiles];

std::mutex g_mu;
int32_t* g_scratch_ptr[kMaxDevices] = {};

// One-time set-up per device, run with that device current: resolve the array's device
// address.  No allocation happens here either.
cudaError_t scratch_for_current_device(int32_t** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    int32_t* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_tile_counts);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

// Pass 1: flagged rows per tile of RR_ROW_TILE rows (tiles never straddle a problem).
__global__ void __launch_bounds__(RR_ROW_TILE)
noalloc_count_kernel(const uint8_t* __restrict__ flags, int n_q, int tiles_per_problem,
                     int32_t* __restrict__ tile_counts) {
  const int prob = blockIdx.x / tiles_per_problem, tile = blockIdx.x % tiles_per_problem;
  const int i = tile * RR_ROW_TILE + threadIdx.x;
  const bool f = i < n_q && flags[(size_t)prob * n_q + i] != 0;
  const int n = __syncthreads_count(f);
  if (threadIdx.x == 0) tile_counts[blockIdx.x] = n;
}

// Pass 2: same scan as the library's compaction kernel, reading the counts from the
// built-in array: base offset = sum of earlier tiles' counts, slot inside the tile from a
// ballot/popcount scan.  Output order = ascending global row id.
__global__ void __launch_bounds__(RR_ROW_TILE)
noalloc_compact_kernel(const uint8_t* __restrict__ flags, int n_problems, int n_q,
                       int tiles_per_problem, const int32_t* __restrict__ tile_counts,
                       int32_t* __restrict__ rows_out, int32_t* __restrict__ count_out,
                       int32_t* __restrict__ problem_offsets_out) {
  __shared__ int s_part[RR_ROW_TILE / 32];
  __shared__ int s_base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile_id = blockIdx.x, n_tiles = gridDim.x;
  const int prob = tile_id / tiles_per_problem, tile = tile_id % tiles_per_problem;
  int part = 0;
  for (int t = tid; t < tile_id; t += RR_ROW_TILE) part += tile_counts[t];
#pragma unroll
  for (int off = 16; off; off >>= 1) part += __shfl_xor_sync(FULL, part, off);
  if (lane == 0) s_part[warp] = part;
  __syncthreads();
  if (tid == 0) {
    int b = 0;
    for (int w = 0; w < RR_ROW_TILE / 32; ++w) b += s_part[w];
    s_base = b;
  }
  __syncthreads();
  const int base = s_base;
  __syncthreads();
  const int i = tile * RR_ROW_TILE + tid;
  const int g = prob * n_q + i;
  const bool f = i < n_q && flags[g] != 0;
  const unsigned bal = __ballot_sync(FULL, f);
  if (lane == 0) s_part[warp] = __popc(bal);
  __syncthreads();
  int before = 0;
  for (int w = 0; w < warp; ++w) before += s_part[w];
  if (f) rows_out[base + before + __popc(bal & ((1u << lane) - 1u))] = g;
  if (tid == 0) {
    if (tile == 0) problem_offsets_out[prob] = base;
    if (tile_id == n_tiles - 1) {
      int total = base;
      for (int w = 0; w < RR_ROW_TILE / 32; ++w) total += s_part[w];
      problem_offsets_out[n_problems] = total;
      *count_out = total;
    }
  }
}

}  // namespace

extern "C" int rr_compact_flags_noalloc(const uint8_t* dev_flags, int32_t n_problems, int32_t n_q,
                                        int32_t* dev_rows_out, int32_t* dev_count_out,
                                        int32_t* dev_problem_offsets_out, void* stream) {
  if (!dev_flags || !dev_rows_out || !dev_count_out || !dev_problem_offsets_out)
    return RR_ERR_INVALID_ARG;
  if (n_problems < 1 || n_q < 1) return RR_ERR_INVALID_ARG;
  const long long tiles_per_problem = ((long long)n_q + RR_ROW_TILE - 1) / RR_ROW_TILE;
  const long long n_tiles = tiles_per_problem * n_problems;
  if (n_tiles > kMaxTiles || (long long)n_problems * n_q > 0x7FFFFFFFLL)
    return RR_ERR_TOO_LARGE;             // beyond the built-in scratch: use the ledger path
  int32_t* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return RR_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  noalloc_count_kernel<<<(int)n_tiles, RR_ROW_TILE, 0, st>>>(dev_flags, n_q,
                                                             (int)tiles_per_problem, scratch);
  noalloc_compact_kernel<<<(int)n_tiles, RR_ROW_TILE, 0, st>>>(
      dev_flags, n_problems, n_q, (int)tiles_per_problem, scratch, dev_rows_out, dev_count_out,
      dev_problem_offsets_out);
  rr_count_launch(2);
  return cudaPeekAtLastError() == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}
