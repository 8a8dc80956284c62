// Row compaction (Section 4.2: "A prefix sum compacts unstable row IDs") together with the
// ledger's book-keeping (Section 4.1: stable rows keep their routes and their ages advance;
// refreshed rows restart at age 0; cumulative work counters), the anchor's fill of the same
// state, token-range expansion, and ledger reset.
#include "rr_common.cuh"

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;

// ---- compaction -----------------------------------------------------------------------
// One CTA per row tile (RR_ROW_TILE rows of one problem).  The tile's base offset is the sum
// of the flagged counts of all earlier tiles (written by the rescoring kernel); inside the
// tile a ballot/popcount scan gives each flagged row its slot.  The list is therefore in
// ascending global row id -- exactly numpy.nonzero(flags) -- with no atomics and no waits
// (the price: n_tiles^2 / 2 count reads in total, nothing at the few thousand tiles of a layer).
// The same pass advances the ages (flagged -> 0, stable -> +1) and, once per launch, the
// per-layer counters: nothing later in the layer reads either.
__global__ void __launch_bounds__(RR_ROW_TILE)
compact_kernel(RRParams p, unsigned long long dense_pairs) {
  __shared__ int s_part[RR_ROW_TILE / 32];
  __shared__ int s_base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile_id = blockIdx.x;
  const int prob = tile_id / p.tiles_per_problem, tile = tile_id % p.tiles_per_problem;

  // Forced anchor (Section 3.2, policy of rr_config.force_permille): the previous tested relay
  // flagged so many rows that this call routes every row.  The tile does what the anchor's fill
  // does for its rows; the rescoring kernel has exited without writing anything.
  if (p.force_threshold > 0 && p.force_in[0] > 0) {
    const int i = tile * RR_ROW_TILE + tid;
    const int g = prob * p.n_q + i;
    if (i < p.n_q) {
      const float qnan = __int_as_float(0x7fc00000);
      p.flags[g] = 1; p.refresh_rows[g] = g; p.ages[g] = 0;
      p.alpha[g] = qnan; p.beta[g] = qnan; p.tau[g] = __int_as_float(0xff800000);
    }
    if (tid == 0) {
      if (tile == 0) p.problem_offsets[prob] = prob * p.n_q;
      if (tile_id == 0) {
        p.counters[RR_CNT_LAYER_CALLS] += 1;
        p.counters[RR_CNT_DENSE_PAIRS] += dense_pairs;
        p.counters[RR_CNT_ANCHOR_ROWS] += (unsigned long long)p.rows;
        p.counters[RR_CNT_FULL_PAIRS] += dense_pairs;
      }
      if (tile_id == p.n_tiles - 1) {
        p.problem_offsets[p.P] = p.rows;
        *p.refresh_count = p.rows;
        p.force_out[0] = p.force_in[0] - 1; p.force_out[1] = p.force_in[1];
        p.force_stats[4] += 1; p.force_stats[5] = 1;
      }
    }
    return;
  }

  int part = 0;
  for (int t = tid; t < tile_id; t += RR_ROW_TILE) part += p.tile_counts[t];
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
  const int g = prob * p.n_q + i;
  const bool f = (i < p.n_q) && p.flags[g] != 0;
  const unsigned bal = __ballot_sync(FULL, f);
  if (lane == 0) s_part[warp] = __popc(bal);
  __syncthreads();
  int before = 0;
  for (int w = 0; w < warp; ++w) before += s_part[w];
  if (f) p.refresh_rows[base + before + __popc(bal & ((1u << lane) - 1u))] = g;
  if (i < p.n_q) p.ages[g] = f ? 0 : p.ages[g] + 1;
  if (tid == 0) {
    if (tile_id == 0) {
      p.counters[RR_CNT_LAYER_CALLS] += 1;
      p.counters[RR_CNT_DENSE_PAIRS] += dense_pairs;
      p.counters[RR_CNT_RELAY_ROWS] += (unsigned long long)p.rows;
    }
    if (tile == 0) p.problem_offsets[prob] = base;
    if (tile_id == p.n_tiles - 1) {
      int total = base;
      for (int w = 0; w < RR_ROW_TILE / 32; ++w) total += s_part[w];
      p.problem_offsets[p.P] = total;
      *p.refresh_count = total;
      if (p.force_threshold > 0) {    // this call was tested: decide about the next ones
        const int run = total >= p.force_threshold ? min(max(1, 2 * p.force_in[1]), p.force_max_run) : 0;
        p.force_out[0] = run; p.force_out[1] = run; p.force_stats[5] = 0;
      }
    }
  }
}

// ---- anchor: every row is (re)routed ----------------------------------------------------
// Flags, identity refresh list, offsets, ages and the anchor's counters.
__global__ void anchor_fill_kernel(RRParams p, unsigned long long dense_pairs) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  const float qnan = __int_as_float(0x7fc00000);
  if (g < p.rows) {
    p.flags[g] = 1;
    p.refresh_rows[g] = g;
    p.alpha[g] = qnan;
    p.beta[g] = qnan;
    p.ages[g] = 0;
  }
  if (g <= p.P) p.problem_offsets[g] = g * p.n_q;
  if (g == 0) {
    *p.refresh_count = p.rows;
    p.counters[RR_CNT_LAYER_CALLS] += 1;
    p.counters[RR_CNT_DENSE_PAIRS] += dense_pairs;
    p.counters[RR_CNT_ANCHOR_ROWS] += (unsigned long long)p.rows;
    p.counters[RR_CNT_FULL_PAIRS] += dense_pairs;
    if (p.force_threshold > 0) {      // a scheduled anchor clears a pending forced run
      p.force_out[0] = 0; p.force_out[1] = p.force_in[1]; p.force_stats[5] = 0;
    }
  }
}

// ---- token ranges of the rows that were re-routed -------------------------------------------
// One warp per row: ids are ranked by counting (they are distinct), chunk j -> [j*T, (j+1)*T),
// ascending chunk id, (-1,-1) for empty slots.
__global__ void __launch_bounds__(256)
expand_kernel(RRParams p, int is_anchor) {
  const int lane = threadIdx.x & 31;
  const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (g >= p.rows) return;
  if (!(is_anchor || p.flags[g] != 0)) return;       // stable row: ranges unchanged
  const int32_t* route = p.routes + (size_t)g * p.k;
  int32_t* out = p.token_ranges + (size_t)g * p.k * 2;
  // rows written by the fused routing kernel are already in ascending chunk id with the empty
  // slots last: their ranges are a plain map of the row (8-byte stores)
  bool ordered = true;
  for (int s = lane; s < p.k; s += 32) {
    const int id = route[s];
    if (s > 0 && id >= 0) { const int prev = route[s - 1]; ordered &= prev >= 0 && prev < id; }
  }
  const bool all_ordered = __all_sync(FULL, ordered);
  if (p.coalesce) {
    // the row's ids in ascending order (empty slots last) into shared memory, then one range
    // per run of consecutive ids: a run's first id writes its start, its last id its end
    extern __shared__ int32_t s_sorted[];
    int32_t* srt = s_sorted + (threadIdx.x >> 5) * p.k;
    for (int s = lane; s < p.k; s += 32) srt[s] = all_ordered ? route[s] : -1;
    __syncwarp();
    if (!all_ordered) {
      for (int s = lane; s < p.k; s += 32) {
        const int id = route[s];
        if (id >= 0) {
          int rank = 0;
          for (int t = 0; t < p.k; ++t) { const int o = route[t]; rank += (o >= 0 && o < id); }
          srt[rank] = id;
        }
      }
      __syncwarp();
    }
    int base = 0;
    for (int s0 = 0; s0 < p.k; s0 += 32) {
      const int s = s0 + lane;
      const int id = s < p.k ? srt[s] : -1;
      const bool valid = id >= 0;
      const bool joins_prev = valid && s > 0 && srt[s - 1] == id - 1 && srt[s - 1] >= 0;
      const bool joins_next = valid && s + 1 < p.k && srt[s + 1] == id + 1;
      const unsigned starts = __ballot_sync(FULL, valid && !joins_prev);
      const int ri = base + __popc(starts & (0xFFFFFFFFu >> (31 - lane))) - 1;
      if (valid && !joins_prev) out[2 * ri] = id * p.chunk_tokens;
      if (valid && !joins_next) out[2 * ri + 1] = (id + 1) * p.chunk_tokens;
      base += __popc(starts);
    }
    for (int s = base + lane; s < p.k; s += 32) { out[2 * s] = -1; out[2 * s + 1] = -1; }
    return;
  }
  if (all_ordered) {
    for (int s = lane; s < p.k; s += 32) {
      const int id = route[s];
      reinterpret_cast<int2*>(out)[s] =
          id >= 0 ? make_int2(id * p.chunk_tokens, (id + 1) * p.chunk_tokens) : make_int2(-1, -1);
    }
    return;
  }
  int n_valid = 0;
  for (int s = lane; s < p.k; s += 32) n_valid += route[s] >= 0;
#pragma unroll
  for (int off = 16; off; off >>= 1) n_valid += __shfl_xor_sync(FULL, n_valid, off);
  for (int s = lane; s < p.k; s += 32) {
    const int id = route[s];
    if (id >= 0) {
      int rank = 0;
      for (int t = 0; t < p.k; ++t) { const int o = route[t]; rank += (o >= 0 && o < id); }
      out[2 * rank] = id * p.chunk_tokens;
      out[2 * rank + 1] = (id + 1) * p.chunk_tokens;
    }
  }
  for (int s = n_valid + lane; s < p.k; s += 32) { out[2 * s] = -1; out[2 * s + 1] = -1; }
}

__global__ void reset_kernel(RRParams p) {
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = tid; e < (size_t)p.rows * p.k; e += stride) p.routes[e] = -1;
  for (size_t e = tid; e < (size_t)p.rows * p.sw; e += stride) p.sentinels[e] = -1;
  for (size_t e = tid; e < (size_t)p.rows; e += stride) {
    p.ages[e] = -1; p.kth[e] = 0.f; p.margin[e] = 0.f;
    p.flags[e] = 0; p.alpha[e] = 0.f; p.beta[e] = 0.f; p.refresh_rows[e] = -1;
  }
  for (size_t e = tid; e <= (size_t)p.P; e += stride) p.problem_offsets[e] = 0;
  for (size_t e = tid; e < (size_t)p.n_tiles; e += stride) p.tile_counts[e] = 0;
  if (p.token_ranges)
    for (size_t e = tid; e < (size_t)p.rows * p.k * 2; e += stride) p.token_ranges[e] = -1;
  if (tid < RR_NUM_COUNTERS) p.counters[tid] = 0;
  if (tid < 8) p.force_stats[tid] = 0;
  if (tid == 0) { *p.status = 0; *p.refresh_count = 0; }
}

}  // namespace

cudaError_t rr_launch_compact(const RRParams& p, unsigned long long dense_pairs, cudaStream_t st) {
  compact_kernel<<<p.n_tiles, RR_ROW_TILE, 0, st>>>(p, dense_pairs);
  rr_count_launch();
  return cudaPeekAtLastError();
}

cudaError_t rr_launch_anchor_fill(const RRParams& p, unsigned long long dense_pairs,
                                  cudaStream_t st) {
  const int n = p.rows > p.P + 1 ? p.rows : p.P + 1;
  anchor_fill_kernel<<<(n + 255) / 256, 256, 0, st>>>(p, dense_pairs);
  rr_count_launch();
  return cudaPeekAtLastError();
}

cudaError_t rr_launch_expand(const RRParams& p, int is_anchor, cudaStream_t st) {
  const int wpb = 8;
  const size_t smem = p.coalesce ? (size_t)wpb * p.k * sizeof(int32_t) : 0;
  expand_kernel<<<(p.rows + wpb - 1) / wpb, wpb * 32, smem, st>>>(p, is_anchor);
  rr_count_launch();
  return cudaPeekAtLastError();
}

cudaError_t rr_launch_reset(const RRParams& p, cudaStream_t st) {
  reset_kernel<<<148 * 4, 256, 0, st>>>(p);
  rr_count_launch();
  return cudaPeekAtLastError();
}
