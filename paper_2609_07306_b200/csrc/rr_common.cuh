// Shared declarations of the route-maintenance library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <mutex>
#include <vector>
#include "../../include/routerelay.h"

#define RR_ROW_TILE 128            // rows per compaction / rescoring tile (per problem)
#define RR_MAX_NK 4096
#define RR_MAX_C 256

// Everything a kernel needs to know about one ledger; passed by value.
struct RRParams {
  int P, n_q, n_k, d, k, m, r, c, sw;      // sw = m + r + n_global (sentinel row width), c = k + sw
  int global_mask, n_global, min_reuse, h_max;   // optional policies (0 = off)
  float gamma_boost, margin_recover;
  int dtype, causal, causal_offset, chunk_tokens, debug;   // debug: bit 0 = store candidate scores
  int coalesce;                            // token ranges of adjacent chunks merged
  int rows, tiles_per_problem, n_tiles;    // row tiles of RR_ROW_TILE per problem / in total
  float gamma;
  unsigned long long seed;
  // ledger (persistent state, Section 4.1)
  int32_t* routes; int32_t* sentinels; int32_t* ages; float* kth; float* margin;
  // per-layer outputs and scratch
  uint8_t* flags; float* alpha; float* beta; float* tau;
  int32_t* refresh_rows; int32_t* refresh_count; int32_t* problem_offsets; int32_t* tile_counts;
  int32_t* token_ranges; float* cand_scores;
  unsigned long long* counters; uint32_t* status;
  float* S;                                // [rows, n_k] score rows of the two-pass path
  // forced anchors before layers of low route persistence (Section 3.2; 0 = off): a relay call
  // reads {pending forced calls, run length} at force_in and writes the next call's pair at
  // force_out (two slots, alternating per call, so that no CTA reads what another one writes)
  int force_threshold, force_max_run;
  int32_t* force_in; int32_t* force_out; int32_t* force_stats;
};

struct rr_ledger {
  rr_config cfg;
  RRParams p;
  void* dev_ledger; size_t ledger_bytes;
  void* dev_scratch; size_t scratch_bytes;
  size_t export_bytes;
  int device;
  int anchored;                            // host-side: has an anchor been enqueued since reset
  unsigned call_index;                     // layer calls since reset (parity of the force_state slots)
  int timeout_shots;                       // test hook: forced time-outs still to be fired (bit 0
                                           // routing kernel, bit 1 strip rescoring kernel)
  bool sweep;                              // full routing runs in the two-sweep fused kernel
  bool inplace;                            // relay: challenge test inside the routing kernel
  bool fused;                              // ... else in the streaming fused kernel
  bool dense_rescore;                      // relay rescoring reads the tensor-core score strip
  unsigned long long dense_pairs_per_layer;
  // benchmark-only per-kernel timing
  bool profiling = false;
  struct ProfRec { int kind; cudaEvent_t a, b; };
  std::vector<ProfRec> prof;
  // events of the pipelined host-buffer path (created on first use)
  cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_consumed[2] = {nullptr, nullptr},
              ev_snap[2] = {nullptr, nullptr}, ev_d2h[2] = {nullptr, nullptr};
};

// ---- device helpers -------------------------------------------------------------------
__host__ __device__ __forceinline__ int rr_valid_count(int i, int n_k, int causal, int off) {
  if (!causal) return n_k;
  long long v = (long long)i + 1 + off;
  return v > n_k ? n_k : (v < 0 ? 0 : (int)v);
}

// Monotone map float -> uint32 (larger float <=> larger key); -0.0 is folded onto +0.0.
__device__ __forceinline__ uint32_t rr_order_key(float s) {
  uint32_t u = __float_as_uint(s + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float rr_key_to_float(uint32_t key) {
  uint32_t u = (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key;
  return __uint_as_float(u);
}

// Counter-based generator of the random-sentinel sampler: two rounds of a 64-bit
// avalanche finaliser, keyed by (seed, global row) and then by (layer, draw index).
__host__ __device__ __forceinline__ unsigned long long rr_fmix64(unsigned long long x) {
  x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ULL;
  x ^= x >> 27; x *= 0x94D049BB133111EBULL;
  x ^= x >> 31;
  return x;
}
__host__ __device__ __forceinline__ unsigned long long rr_row_key(unsigned long long seed,
                                                                  uint32_t g) {
  return rr_fmix64(seed ^ ((unsigned long long)g * 0x9E3779B97F4A7C15ULL));
}
__host__ __device__ __forceinline__ uint32_t rr_draw_u32(unsigned long long row_key,
                                                         uint32_t layer, uint32_t t) {
  return (uint32_t)(rr_fmix64(row_key ^ (((unsigned long long)layer << 32) | t)) >> 32);
}

// Challenge test of Eq. 5 for global row g, with the optional policies of Section 3.2: a
// larger guard margin while the margin recorded at the row's last routing is below the
// recovery level, no test before the minimum reuse horizon, forced re-routing of a route
// that is h_max layers old.  Reads the ledger's ages / margins only when a policy is on.
__device__ __forceinline__ bool rr_challenge(const RRParams& p, int g, float alpha, float beta) {
  float gamma = p.gamma;
  if (p.gamma_boost > 0.f && p.margin[g] < p.margin_recover) gamma += p.gamma_boost;
  bool flag = beta > __int_as_float(0xff800000) && !(alpha > beta + gamma);
  if (p.min_reuse > 0 || p.h_max > 0) {
    const int age = p.ages[g];
    if (age < p.min_reuse) flag = false;
    if (p.h_max > 0 && age >= p.h_max) flag = true;
  }
  return flag;
}

// ---- launchers (one per .cu file) -------------------------------------------------------
// All return cudaError_t from the launch; all are asynchronous on `st`.
cudaError_t rr_launch_score_simt(const RRParams& p, const void* qc, const void* kc,
                                 const int32_t* row_list, cudaStream_t st);
cudaError_t rr_launch_score_tc(const RRParams& p, const void* qc, const void* kc,
                               const int32_t* row_list, cudaStream_t st);
bool rr_route_fused_supported(const RRParams& p);
cudaError_t rr_launch_route_fused(const RRParams& p, const void* qc, const void* kc,
                                  const int32_t* row_list, int layer, cudaStream_t st);
bool rr_route_sweep_supported(const RRParams& p);
cudaError_t rr_launch_route_sweep(const RRParams& p, const void* qc, const void* kc,
                                  const int32_t* row_list, int layer, int inplace, int hooks,
                                  cudaStream_t st);   // hooks: bit 0 slow rows, bit 1 forced time-out
bool rr_route_sweep_inplace_supported(const RRParams& p);
cudaError_t rr_launch_topk_rows(const RRParams& p, const int32_t* row_list, int layer,
                                cudaStream_t st);
// global + random sentinels of the listed rows (after rr_launch_route_sweep; n_k <= 1024)
cudaError_t rr_launch_sentinels(const RRParams& p, const int32_t* row_list, int layer,
                                cudaStream_t st);
cudaError_t rr_launch_rescore(const RRParams& p, const void* qc, const void* kc,
                              cudaStream_t st);
bool rr_rescore_dense_supported(const RRParams& p);
cudaError_t rr_launch_rescore_dense(const RRParams& p, const void* qc, const void* kc,
                                    int force_timeout, bool prior, cudaStream_t st);
// compact / anchor_fill also advance the ages and the cumulative counters of the layer
cudaError_t rr_launch_compact(const RRParams& p, unsigned long long dense_pairs, cudaStream_t st);
cudaError_t rr_launch_anchor_fill(const RRParams& p, unsigned long long dense_pairs,
                                  cudaStream_t st);
cudaError_t rr_launch_expand(const RRParams& p, int is_anchor, cudaStream_t st);
cudaError_t rr_launch_reset(const RRParams& p, cudaStream_t st);

void rr_count_launch(int n = 1);

// Function attributes (dynamic shared-memory limit) are per device: `setup` runs the first time
// the calling site is reached with a given device current, under a lock, and the device is
// marked done only if it returned cudaSuccess (so a failure is retried, and no other host
// thread launches before the attributes are in place).  `done` is the site's own bit mask.
std::mutex& rr_attr_mutex();
template <class F>
inline cudaError_t rr_once_per_device(unsigned long long& done, F&& setup) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev > 63) return setup();
  std::lock_guard<std::mutex> lock(rr_attr_mutex());
  if ((done >> dev) & 1ull) return cudaSuccess;
  const cudaError_t e = setup();
  if (e == cudaSuccess) done |= 1ull << dev;
  return e;
}
