// Warp-level exact TopK of one score row held in shared memory as order-preserving keys: route
// (Eq. 2), near-miss sentinels (Section 3.1 item 1), k-th score and margin (Section 3.3), the
// mandatory global and the random sentinels (Section 3.1 items 2, 3), written straight into the
// ledger row.  One warp per row.  Used by the two-pass path (score rows read back from memory)
// and by the fused routing kernel for the rows its fast path hands over.
//
// Selection is a radix select on the 32-bit keys (8 bits per pass, shared-memory histogram,
// shuffle scan), run for rank k and rank k+m.  Ties on a key are resolved towards the smaller
// chunk id by walking the row in index order with ballots.
#pragma once
#include "rr_common.cuh"

namespace warptopk {

constexpr unsigned FULL = 0xFFFFFFFFu;

struct Sel { uint32_t key; int need; int ties; };

// Key of rank T (1-based, descending) among keys[0..v): `need` of the `ties` keys equal to
// it belong to the top T.  Requires 1 <= T <= v.
__device__ inline Sel warp_select(const uint32_t* keys, int v, int T, uint32_t* hist, int lane) {
  uint32_t prefix = 0, mask = 0;
  int need = T, ties = 0;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int b = lane; b < 256; b += 32) hist[b] = 0;
    __syncwarp();
    for (int j = lane; j < v; j += 32) {
      uint32_t key = keys[j];
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncwarp();
    // lane owns digits 255-8*lane .. 248-8*lane, walked in descending order
    int loc[8], sum = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) { loc[q] = (int)hist[255 - 8 * lane - q]; sum += loc[q]; }
    int incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int t = __shfl_up_sync(FULL, incl, off);
      if (lane >= off) incl += t;
    }
    int excl = incl - sum;
    bool mine = (excl < need) && (need <= incl);
    int dsel = 0, before = 0, cnt = 0, run = excl;
    bool found = false;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      bool here = mine && !found && (need <= run + loc[q]);
      if (here) { dsel = 255 - 8 * lane - q; before = run; cnt = loc[q]; found = true; }
      run += loc[q];
    }
    int src = __ffs(__ballot_sync(FULL, mine)) - 1;
    dsel = __shfl_sync(FULL, dsel, src);
    before = __shfl_sync(FULL, before, src);
    cnt = __shfl_sync(FULL, cnt, src);
    need -= before;
    prefix |= (uint32_t)dsel << shift;
    mask |= 0xFFu << shift;
    ties = cnt;
    __syncwarp();
  }
  return Sel{prefix, need, ties};
}

// Mandatory global sentinels and the random sentinel sample of one row (Section 3.1 items 2 and
// 3, Section 3.4), by a whole warp.  bitmap: the row's excluded chunks (route + near-miss) as
// ceil(v / 32) words in shared memory, private to the warp and updated here; pool = valid chunks
// not excluded.  Sequential definition of the sample: pool <= r -> the whole pool in ascending
// order; else for t = 0, 1, ...: j = floor(u_t v / 2^32), accepted iff j is not excluded and was
// not drawn before, until r are accepted; after 64 r draws the smallest free chunks fill the
// rest.  32 draws are examined per step: a draw is accepted iff its chunk is free in the bitmap
// and no earlier lane of the step drew the same chunk; the accepted ones take the next slots in
// lane (= draw) order, which is exactly the sequential outcome.
__device__ __forceinline__ void sentinels_row(const RRParams& p, uint32_t* bitmap, int pool, int g,
                                              int v, uint32_t layer, int lane) {
  const unsigned lt = (1u << lane) - 1u;
  int32_t* sent = p.sentinels + (size_t)g * p.sw;
  if (p.n_global) {
    int gi = 0;
    for (int b = 0; b < 2; ++b) {
      if (!((p.global_mask >> b) & 1)) continue;
      const int j = b == 0 ? 0 : v - 1;
      int id = -1;
      if (v > 0) {
        const uint32_t word = bitmap[j >> 5], bit = 1u << (j & 31);
        if (!(word & bit)) { id = j; --pool; }
        __syncwarp();
        if (id >= 0 && lane == 0) bitmap[j >> 5] = word | bit;
        __syncwarp();
      }
      if (lane == 0) sent[p.m + p.r + gi] = id;
      ++gi;
    }
  }
  int32_t* rnd = sent + p.m;
  int taken = 0;
  if (p.r > 0 && pool > 0) {
    if (pool > p.r) {
      const unsigned long long rk = rr_row_key(p.seed, (uint32_t)g);
      const int limit = 64 * p.r;
      for (int t0 = 0; t0 < limit && taken < p.r; t0 += 32) {
        const int j = (int)__umulhi(rr_draw_u32(rk, layer, (uint32_t)(t0 + lane)), (uint32_t)v);
        const bool free_j = ((bitmap[j >> 5] >> (j & 31)) & 1u) == 0u;
        const unsigned same = __match_any_sync(FULL, j);
        const bool ok = t0 + lane < limit && free_j && (same & lt) == 0u;
        const unsigned okmask = __ballot_sync(FULL, ok);
        const int pos = taken + __popc(okmask & lt);
        if (ok && pos < p.r) { rnd[pos] = j; atomicOr(&bitmap[j >> 5], 1u << (j & 31)); }
        taken = min(p.r, taken + __popc(okmask));
        __syncwarp();
      }
    }
    // whole pool (pool <= r) or the bounded-work fill: smallest free chunks first
    for (int j0 = 0; j0 < v && taken < p.r; j0 += 32) {
      const int j = j0 + lane;
      const bool fr = j < v && !((bitmap[j0 >> 5] >> lane) & 1u);
      const unsigned bf = __ballot_sync(FULL, fr);
      const int pos = taken + __popc(bf & lt);
      if (fr && pos < p.r) rnd[pos] = j;
      taken = min(p.r, taken + __popc(bf));
    }
  }
  for (int s = taken + lane; s < p.r; s += 32) rnd[s] = -1;
}

// keys[0..v): the row's order keys (rr_order_key of the scores); hist: 256 words; bitmap:
// ceil(n_k / 32) words.  All three in shared memory, private to the calling warp; bitmap and
// hist need no initialisation.  g: global row id, v: chunks the row may select.
__device__ __forceinline__ void route_row(const RRParams& p, const uint32_t* keys, uint32_t* hist,
                                          uint32_t* bitmap, int g, int v, uint32_t layer, int lane) {
  const unsigned lt = (1u << lane) - 1u;
  for (int w = lane; w < (p.n_k + 31) / 32; w += 32) bitmap[w] = 0;
  __syncwarp();
  const int Tk = min(p.k, v), Tkeep = min(p.k + p.m, v);
  const Sel sk = warp_select(keys, v, Tk, hist, lane);
  const Sel sn = (Tkeep > Tk) ? warp_select(keys, v, Tkeep, hist, lane) : sk;

  int32_t* route = p.routes + (size_t)g * p.k;
  int32_t* sent = p.sentinels + (size_t)g * p.sw;
  int run_eqk = 0, run_eqn = 0, run_route = 0, run_near = 0;
  for (int j0 = 0; j0 < v; j0 += 32) {
    const int j = j0 + lane;
    const bool valid = j < v;
    const uint32_t key = valid ? keys[j] : 0u;
    const bool eqk = valid && key == sk.key;
    const bool eqn = valid && key == sn.key;
    const unsigned bk = __ballot_sync(FULL, eqk), bn = __ballot_sync(FULL, eqn);
    const int rank_k = run_eqk + __popc(bk & lt), rank_n = run_eqn + __popc(bn & lt);
    const bool in_route = valid && (key > sk.key || (eqk && rank_k < sk.need));
    const bool in_near = valid && !in_route && Tkeep > Tk &&
                         (key > sn.key || (eqn && rank_n < sn.need));
    const unsigned br = __ballot_sync(FULL, in_route), bnr = __ballot_sync(FULL, in_near);
    if (in_route) route[run_route + __popc(br & lt)] = j;
    if (in_near) sent[run_near + __popc(bnr & lt)] = j;
    if (lane == 0) bitmap[j0 >> 5] = br | bnr;
    run_eqk += __popc(bk); run_eqn += __popc(bn);
    run_route += __popc(br); run_near += __popc(bnr);
  }
  for (int s = run_route + lane; s < p.k; s += 32) route[s] = -1;
  for (int s = run_near + lane; s < p.m; s += 32) sent[s] = -1;

  // k-th score and margin (min selected - max unselected)
  float kth = rr_key_to_float(sk.key), margin = __int_as_float(0x7f800000);
  if (v > Tk) {
    uint32_t next = sk.key;
    if (sk.ties <= sk.need) {
      uint32_t best = 0;
      for (int j = lane; j < v; j += 32) {
        uint32_t key = keys[j];
        if (key < sk.key && key > best) best = key;
      }
#pragma unroll
      for (int off = 16; off; off >>= 1) best = max(best, __shfl_xor_sync(FULL, best, off));
      next = best;
    }
    margin = kth - rr_key_to_float(next);
  }
  if (lane == 0) { p.kth[g] = kth; p.margin[g] = margin; }
  __syncwarp();

  __syncwarp();
  sentinels_row(p, bitmap, v - Tkeep, g, v, layer, lane);
}

}  // namespace warptopk
