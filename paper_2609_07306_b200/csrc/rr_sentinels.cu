// Mandatory global sentinels and the seeded random sentinel sample (Section 3.1 items 2 and 3,
// Section 3.4) of rows whose route and near-miss sentinels have just been written by the
// two-sweep routing kernel.  One thread per row, in small blocks so that a layer's rows fill every
// SM with as many warps as its registers allow: a row's draws are accepted strictly in draw
// order, a serial chain per row that only many rows in flight can hide (inside the routing
// kernel, which holds one CTA per SM, it would sit on every CTA's critical path).
//
// The thread rebuilds the set of excluded chunks (route + near-miss) as a bitmap in shared
// memory ([word][thread], private to the thread, so plain read-modify-writes do), fills the
// global slots (a slot stays -1 if its chunk is excluded already) and draws:
// pool <= r: the whole pool in ascending order; else for t = 0, 1, ...: j = floor(u_t v / 2^32),
// accept iff j is not excluded and not drawn yet; after 64 r draws the smallest free chunks.
#include "rr_common.cuh"

namespace {

constexpr int NT = 64, WORDS = 32;             // rows per block; bitmap words per row (n_k <= 1024)
constexpr int MAX_R = 32;                      // random sentinels staged per row (more: direct stores)

__global__ void __launch_bounds__(NT)
sentinel_kernel(RRParams p, const int32_t* __restrict__ row_list, uint32_t layer) {
  __shared__ uint32_t s_bits[WORDS][NT];
  // The row's random sentinels are collected here ([slot][thread]) and leave with 16-byte stores:
  // the kernel is bound by the L1's sector accesses for its per-row (uncoalesced) traffic, and a
  // 4-byte store per accepted draw costs one each.
  __shared__ int32_t s_out[MAX_R][NT];
  const int tid = threadIdx.x;
  const int slot = blockIdx.x * NT + tid;
  const int count = row_list ? *p.refresh_count : p.rows;
  if (slot >= count) return;
  const int g = row_list ? row_list[slot] : slot;
  const int v = rr_valid_count(g % p.n_q, p.n_k, p.causal, p.causal_offset);
  const int words = (v + 31) >> 5;
  for (int w = 0; w < words; ++w) s_bits[w][tid] = 0u;
  const int32_t* route = p.routes + (size_t)g * p.k;
  int32_t* sent = p.sentinels + (size_t)g * p.sw;
  int excluded = 0;
  auto mark = [&](int id) {
    if (id >= 0 && id < v) { s_bits[id >> 5][tid] |= 1u << (id & 31); ++excluded; }
  };
  if (((p.k | p.m | p.sw) & 3) == 0) {
    for (int q = 0; q < p.k; q += 4) {
      const int4 t = *reinterpret_cast<const int4*>(route + q);
      mark(t.x); mark(t.y); mark(t.z); mark(t.w);
    }
    for (int q = 0; q < p.m; q += 4) {
      const int4 t = *reinterpret_cast<const int4*>(sent + q);
      mark(t.x); mark(t.y); mark(t.z); mark(t.w);
    }
  } else {
    for (int q = 0; q < p.k; ++q) mark(route[q]);
    for (int q = 0; q < p.m; ++q) mark(sent[q]);
  }
  int pool = v - excluded;
  // ---- mandatory global sentinels: a slot each after the random ones -----------------------------
  if (p.n_global) {
    int32_t* glob = sent + p.m + p.r;
    int gi = 0;
    for (int b = 0; b < 2; ++b) {
      if (!((p.global_mask >> b) & 1)) continue;
      const int j = b == 0 ? 0 : v - 1;
      int id = -1;
      if (v > 0) {
        const uint32_t w = s_bits[j >> 5][tid], bit = 1u << (j & 31);
        if (!(w & bit)) { s_bits[j >> 5][tid] = w | bit; id = j; --pool; }
      }
      glob[gi++] = id;
    }
  }
  // ---- random sentinels ---------------------------------------------------------------------------
  int32_t* rnd = sent + p.m;
  int taken = 0;
  const bool staged = p.r <= MAX_R && ((p.m | p.r | p.sw) & 3) == 0;
  auto put = [&](int slot_, int id) { if (staged) s_out[slot_][tid] = id; else rnd[slot_] = id; };
  if (p.r > 0 && pool > 0) {
    if (pool > p.r) {
      const unsigned long long rk = rr_row_key(p.seed, (uint32_t)g);
      const int limit = 64 * p.r;
      // four draws are generated at a time (independent 64-bit mixes overlap); they are still
      // accepted strictly in draw order
      for (int t0 = 0; t0 < limit && taken < p.r; t0 += 4) {
        int j4[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          j4[i] = (int)__umulhi(rr_draw_u32(rk, layer, (uint32_t)(t0 + i)), (uint32_t)v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const bool live = (t0 + i < limit) & (taken < p.r);
          const uint32_t w = s_bits[j4[i] >> 5][tid], bit = 1u << (j4[i] & 31);
          if (live && !(w & bit)) { s_bits[j4[i] >> 5][tid] = w | bit; put(taken++, j4[i]); }
        }
      }
    }
    // whole pool (pool <= r) or the bounded-work fill: smallest free chunks first
    for (int j = 0; j < v && taken < p.r; ++j)
      if (!((s_bits[j >> 5][tid] >> (j & 31)) & 1u)) put(taken++, j);
  }
  for (int e = taken; e < p.r; ++e) put(e, -1);
  if (staged)
    for (int e = 0; e < p.r; e += 4)
      *reinterpret_cast<int4*>(rnd + e) =
          make_int4(s_out[e][tid], s_out[e + 1][tid], s_out[e + 2][tid], s_out[e + 3][tid]);
}

}  // namespace

cudaError_t rr_launch_sentinels(const RRParams& p, const int32_t* row_list, int layer,
                                cudaStream_t st) {
  if (p.n_k > WORDS * 32) return cudaErrorInvalidConfiguration;
  sentinel_kernel<<<(p.rows + NT - 1) / NT, NT, 0, st>>>(p, row_list, (uint32_t)layer);
  rr_count_launch();
  return cudaPeekAtLastError();
}
