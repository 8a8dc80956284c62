// C ABI of the route-maintenance library: handle management, buffer layout, and the two
// layer calls (anchor / relay) that enqueue the kernels.  No device allocation, no host
// synchronisation inside the layer calls.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include "rr_common.cuh"

namespace {

std::atomic<unsigned long long> g_launches{0};
thread_local char g_cuda_err[256] = "";

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", what, cudaGetErrorString(e));
  return RR_ERR_CUDA;
}
#define RR_CUDA(call)                                             \
  do {                                                            \
    cudaError_t e_ = (call);                                      \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);           \
  } while (0)

struct Layout {
  // ledger blob
  size_t routes, sentinels, ages, kth, margin, ledger_total;
  // scratch
  size_t flags, alpha, beta, tau, refresh_rows, refresh_count, problem_offsets, tile_counts,
      token_ranges, cand_scores, counters, status, force_state, S, scratch_total;
  size_t export_total;
};

int validate(const rr_config* c) {
  if (!c) return RR_ERR_INVALID_ARG;
  if (c->batch < 1 || c->heads < 1 || c->n_q < 1 || c->n_k < 1) return RR_ERR_INVALID_ARG;
  if (c->k < 1 || c->m < 0 || c->r < 0) return RR_ERR_INVALID_ARG;
  if (c->causal != 0 && c->causal != 1) return RR_ERR_INVALID_ARG;
  if (c->causal_offset < 0) return RR_ERR_INVALID_ARG;
  if (!(c->gamma >= 0.f)) return RR_ERR_INVALID_ARG;          // also rejects NaN
  if (c->chunk_tokens < 0) return RR_ERR_INVALID_ARG;
  if (c->dtype != RR_BF16 && c->dtype != RR_F32) return RR_ERR_UNSUPPORTED;
  if (c->d != 64 && c->d != 128) return RR_ERR_UNSUPPORTED;
  if (c->n_k > RR_MAX_NK) return RR_ERR_UNSUPPORTED;
  if (c->k > c->n_k) return RR_ERR_INVALID_ARG;
  if (c->global_sentinels < 0 || c->global_sentinels > 3) return RR_ERR_INVALID_ARG;
  if (c->min_reuse < 0 || c->h_max < 0 || !(c->gamma_boost >= 0.f)) return RR_ERR_INVALID_ARG;
  if (c->margin_recover != c->margin_recover) return RR_ERR_INVALID_ARG;   // NaN
  if (c->coalesce_ranges != 0 && c->coalesce_ranges != 1) return RR_ERR_INVALID_ARG;
  if (c->force_permille < 0 || c->force_permille > 1000) return RR_ERR_INVALID_ARG;
  if (c->force_permille > 0 && (c->debug_outputs & 32)) return RR_ERR_UNSUPPORTED;
  if (c->k + c->m + c->r + (c->global_sentinels & 1) + ((c->global_sentinels >> 1) & 1) > RR_MAX_C)
    return RR_ERR_UNSUPPORTED;
  const long long rows = (long long)c->batch * c->heads * c->n_q;
  if (rows > (1LL << 30)) return RR_ERR_UNSUPPORTED;
  if (c->chunk_tokens > 0 && (long long)c->n_k * c->chunk_tokens > 0x7FFFFFFFLL)
    return RR_ERR_UNSUPPORTED;
  return RR_OK;
}

// RRParams fields that decide which kernels apply (host-only; no pointers).
RRParams shape_params(const rr_config* cfg) {
  RRParams p{};
  p.P = cfg->batch * cfg->heads; p.n_q = cfg->n_q; p.n_k = cfg->n_k; p.d = cfg->d;
  p.k = cfg->k; p.m = cfg->m; p.r = cfg->r;
  p.global_mask = cfg->global_sentinels;
  p.n_global = (cfg->global_sentinels & 1) + ((cfg->global_sentinels >> 1) & 1);
  p.min_reuse = cfg->min_reuse; p.h_max = cfg->h_max;
  p.gamma_boost = cfg->gamma_boost; p.margin_recover = cfg->margin_recover;
  p.sw = cfg->m + cfg->r + p.n_global; p.c = cfg->k + p.sw;
  p.dtype = cfg->dtype; p.causal = cfg->causal; p.causal_offset = cfg->causal_offset;
  p.chunk_tokens = cfg->chunk_tokens; p.debug = cfg->debug_outputs & 1;
  p.coalesce = cfg->coalesce_ranges;
  p.rows = p.P * p.n_q;
  p.tiles_per_problem = (p.n_q + RR_ROW_TILE - 1) / RR_ROW_TILE;
  p.n_tiles = p.P * p.tiles_per_problem;
  p.gamma = cfg->gamma; p.seed = cfg->seed;
  return p;
}

// The two-sweep kernel wins where the grid fills the GPU several times over (its per-score work
// is smaller); on grids of less than two waves of CTAs a layer is a chain of kernel latencies,
// and the streaming kernel -- one sweep, sentinels inside, one launch less -- is the shorter
// chain (measured on the 32-problem chunk sweep: 5-10 % per step).  148 SMs, one CTA per SM.
bool uses_sweep(const rr_config* cfg) {
  if (cfg->debug_outputs & (2 | 16)) return false;
  const RRParams p = shape_params(cfg);
  if (!rr_route_sweep_supported(p)) return false;
  const bool forced = (cfg->debug_outputs & (32 | 256)) != 0;   // relay in place needs it; bit 8 asks for it
  return forced || p.n_tiles >= 2 * 148 || !rr_route_fused_supported(p);
}

bool uses_fused(const rr_config* cfg) {
  return !(cfg->debug_outputs & 2) && !uses_sweep(cfg) && rr_route_fused_supported(shape_params(cfg));
}

Layout make_layout(const rr_config* c) {
  Layout L{};
  const size_t P = (size_t)c->batch * c->heads, rows = P * c->n_q;
  const size_t sw = (size_t)c->m + c->r + (c->global_sentinels & 1) + ((c->global_sentinels >> 1) & 1),
               cw = (size_t)c->k + sw;
  const size_t tiles = P * ((c->n_q + RR_ROW_TILE - 1) / RR_ROW_TILE);
  size_t o = 0;
  L.routes = o;    o = align_up(o + rows * c->k * 4);
  L.sentinels = o; o = align_up(o + rows * sw * 4);
  L.ages = o;      o = align_up(o + rows * 4);
  L.kth = o;       o = align_up(o + rows * 4);
  L.margin = o;    o = align_up(o + rows * 4);
  L.ledger_total = o;
  L.export_total = rows * c->k * 4 + rows * sw * 4 + rows * 4 * 3;
  o = 0;
  L.flags = o;           o = align_up(o + rows);
  L.alpha = o;           o = align_up(o + rows * 4);
  L.beta = o;            o = align_up(o + rows * 4);
  L.tau = o;             o = align_up(o + rows * 4);
  L.refresh_rows = o;    o = align_up(o + rows * 4);
  L.refresh_count = o;   o = align_up(o + 4);
  L.problem_offsets = o; o = align_up(o + (P + 1) * 4);
  L.tile_counts = o;     o = align_up(o + tiles * 4);
  L.counters = o;        o = align_up(o + RR_NUM_COUNTERS * 8);
  L.status = o;          o = align_up(o + 4);
  L.force_state = o;     o = align_up(o + 8 * 4);
  L.token_ranges = o;    o = align_up(o + (c->chunk_tokens > 0 ? rows * c->k * 8 : 0));
  L.cand_scores = o;     o = align_up(o + ((c->debug_outputs & 1) ? rows * cw * 4 : 0));
  // score rows are only materialised by the two-pass path
  L.S = o;               o = align_up(o + (uses_fused(c) || uses_sweep(c) ? 0 : rows * (size_t)c->n_k * 4));
  L.scratch_total = o;
  return L;
}

unsigned long long dense_pairs(const rr_config* c) {
  unsigned long long per_problem = 0;
  for (int i = 0; i < c->n_q; ++i)
    per_problem += (unsigned long long)rr_valid_count(i, c->n_k, c->causal, c->causal_offset);
  return per_problem * (unsigned long long)c->batch * c->heads;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// test hooks of the next routing launch: slow rows (debug bit 3), one forced time-out (bit 6)
int sweep_hooks(rr_ledger* L) {
  int h = (L->cfg.debug_outputs >> 3) & 1;
  if (L->timeout_shots & 1) { h |= 2; L->timeout_shots &= ~1; }
  return h;
}

int route_layer(rr_ledger* L, const void* qc, const void* kc, int layer, bool anchor,
                cudaStream_t st) {
  if (!L || !qc || !kc || layer < 0) return RR_ERR_INVALID_ARG;
  if (!aligned16(qc) || !aligned16(kc)) return RR_ERR_INVALID_ARG;
  RRParams p = L->p;
  p.force_in = p.force_stats + 2 * (L->call_index & 1u);
  p.force_out = p.force_stats + 2 * ((L->call_index + 1u) & 1u);
  ++L->call_index;
  // LAUNCH(kind, call): enqueue one kernel, bracketed by events while profiling
#define LAUNCH(kind, call)                                                         \
  do {                                                                             \
    rr_ledger::ProfRec rec_{kind, nullptr, nullptr};                               \
    if (L->profiling) {                                                            \
      RR_CUDA(cudaEventCreate(&rec_.a)); RR_CUDA(cudaEventCreate(&rec_.b));        \
      RR_CUDA(cudaEventRecord(rec_.a, st));                                        \
    }                                                                              \
    RR_CUDA(call);                                                                 \
    if (L->profiling) { RR_CUDA(cudaEventRecord(rec_.b, st)); L->prof.push_back(rec_); } \
  } while (0)
  if (anchor) {
    // Section 4.1: the anchor builds the state from a complete chunk-score matrix.
    LAUNCH(RR_KIND_ANCHOR_FILL, rr_launch_anchor_fill(p, L->dense_pairs_per_layer, st));
    if (L->sweep) {
      LAUNCH(RR_KIND_ROUTE_FUSED, rr_launch_route_sweep(p, qc, kc, nullptr, layer, 0,
                                                        sweep_hooks(L), st));
      LAUNCH(RR_KIND_SENTINELS, rr_launch_sentinels(p, nullptr, layer, st));
    } else if (L->fused) {
      LAUNCH(RR_KIND_ROUTE_FUSED, rr_launch_route_fused(p, qc, kc, nullptr, layer, st));
    } else {
      if (p.dtype == RR_BF16) LAUNCH(RR_KIND_SCORE_TC, rr_launch_score_tc(p, qc, kc, nullptr, st));
      else LAUNCH(RR_KIND_SCORE_SIMT, rr_launch_score_simt(p, qc, kc, nullptr, st));
      LAUNCH(RR_KIND_TOPK_ROWS, rr_launch_topk_rows(p, nullptr, layer, st));
    }
    L->anchored = 1;
  } else {
    if (!L->anchored) return RR_ERR_STATE;
    if (L->inplace) {
      // Relay in one pass over the score strip: the routing kernel tests every row (Eq. 5) on
      // the scores of its first sweep and re-routes the failing rows in place; the compaction
      // kernel then only builds the list the caller sees (and the sentinel kernel works from).
      LAUNCH(RR_KIND_ROUTE_FUSED, rr_launch_route_sweep(p, qc, kc, nullptr, layer, 1,
                                                        sweep_hooks(L), st));
      LAUNCH(RR_KIND_COMPACT, rr_launch_compact(p, L->dense_pairs_per_layer, st));
      LAUNCH(RR_KIND_SENTINELS, rr_launch_sentinels(p, p.refresh_rows, layer, st));
      if (p.chunk_tokens > 0) LAUNCH(RR_KIND_EXPAND, rr_launch_expand(p, 0, st));
      return RR_OK;
    }
    // Section 4.2: rescoring + flags, prefix-sum compaction, refresh of the listed rows.
    if (L->dense_rescore) {
      const int shot = (L->timeout_shots >> 1) & 1;     // test hook: one forced time-out
      L->timeout_shots &= ~2;
      LAUNCH(RR_KIND_RESCORE_DENSE, rr_launch_rescore_dense(p, qc, kc, shot, /*prior=*/!L->sweep, st));
    }
    else LAUNCH(RR_KIND_RESCORE, rr_launch_rescore(p, qc, kc, st));
    LAUNCH(RR_KIND_COMPACT, rr_launch_compact(p, L->dense_pairs_per_layer, st));
    if (L->sweep) {
      LAUNCH(RR_KIND_ROUTE_FUSED, rr_launch_route_sweep(p, qc, kc, p.refresh_rows, layer, 0,
                                                        sweep_hooks(L), st));
      LAUNCH(RR_KIND_SENTINELS, rr_launch_sentinels(p, p.refresh_rows, layer, st));
    } else if (L->fused) {
      LAUNCH(RR_KIND_ROUTE_FUSED, rr_launch_route_fused(p, qc, kc, p.refresh_rows, layer, st));
    } else {
      if (p.dtype == RR_BF16)
        LAUNCH(RR_KIND_SCORE_TC, rr_launch_score_tc(p, qc, kc, p.refresh_rows, st));
      else
        LAUNCH(RR_KIND_SCORE_SIMT, rr_launch_score_simt(p, qc, kc, p.refresh_rows, st));
      LAUNCH(RR_KIND_TOPK_ROWS, rr_launch_topk_rows(p, p.refresh_rows, layer, st));
    }
  }
  if (p.chunk_tokens > 0) LAUNCH(RR_KIND_EXPAND, rr_launch_expand(p, anchor ? 1 : 0, st));
#undef LAUNCH
  return RR_OK;
}

}  // namespace

void rr_count_launch(int n) { g_launches.fetch_add((unsigned long long)n); }

std::mutex& rr_attr_mutex() {
  static std::mutex mu;
  return mu;
}

extern "C" {

int rr_workspace_bytes(const rr_config* cfg, size_t* ledger_bytes, size_t* scratch_bytes) {
  int rc = validate(cfg);
  if (rc != RR_OK) return rc;
  if (!ledger_bytes || !scratch_bytes) return RR_ERR_INVALID_ARG;
  Layout L = make_layout(cfg);
  *ledger_bytes = L.ledger_total;
  *scratch_bytes = L.scratch_total;
  return RR_OK;
}

int rr_export_bytes(const rr_config* cfg, size_t* bytes) {
  int rc = validate(cfg);
  if (rc != RR_OK) return rc;
  if (!bytes) return RR_ERR_INVALID_ARG;
  *bytes = make_layout(cfg).export_total;
  return RR_OK;
}

int rr_ledger_init(const rr_config* cfg, void* dev_ledger, size_t ledger_bytes,
                   void* dev_scratch, size_t scratch_bytes, rr_ledger** out) {
  int rc = validate(cfg);
  if (rc != RR_OK) return rc;
  if (!dev_ledger || !dev_scratch || !out) return RR_ERR_INVALID_ARG;
  if (((uintptr_t)dev_ledger & 255u) || ((uintptr_t)dev_scratch & 255u)) return RR_ERR_INVALID_ARG;
  Layout lay = make_layout(cfg);
  if (ledger_bytes < lay.ledger_total || scratch_bytes < lay.scratch_total) return RR_ERR_TOO_SMALL;
  rr_ledger* L = new (std::nothrow) rr_ledger();
  if (!L) return RR_ERR_INVALID_ARG;
  L->cfg = *cfg;
  L->dev_ledger = dev_ledger; L->ledger_bytes = ledger_bytes;
  L->dev_scratch = dev_scratch; L->scratch_bytes = scratch_bytes;
  L->export_bytes = lay.export_total;
  L->anchored = 0;
  L->timeout_shots = (cfg->debug_outputs >> 6) & 3;
  L->device = -1;
  cudaGetDevice(&L->device);           // informational; failure (no GPU) leaves -1
  cudaGetLastError();
  L->dense_pairs_per_layer = dense_pairs(cfg);
  RRParams& p = L->p;
  p = shape_params(cfg);
  char* lb = (char*)dev_ledger; char* sb = (char*)dev_scratch;
  p.routes = (int32_t*)(lb + lay.routes); p.sentinels = (int32_t*)(lb + lay.sentinels);
  p.ages = (int32_t*)(lb + lay.ages); p.kth = (float*)(lb + lay.kth);
  p.margin = (float*)(lb + lay.margin);
  p.flags = (uint8_t*)(sb + lay.flags); p.alpha = (float*)(sb + lay.alpha);
  p.beta = (float*)(sb + lay.beta); p.tau = (float*)(sb + lay.tau);
  p.refresh_rows = (int32_t*)(sb + lay.refresh_rows);
  p.refresh_count = (int32_t*)(sb + lay.refresh_count);
  p.problem_offsets = (int32_t*)(sb + lay.problem_offsets);
  p.tile_counts = (int32_t*)(sb + lay.tile_counts);
  p.counters = (unsigned long long*)(sb + lay.counters);
  p.status = (uint32_t*)(sb + lay.status);
  p.force_stats = (int32_t*)(sb + lay.force_state);
  p.force_in = p.force_out = p.force_stats;           // set per call (route_layer)
  p.force_threshold = (int)(((long long)p.rows * cfg->force_permille + 999) / 1000);
  p.force_max_run = cfg->force_max_run < 1 ? 1 : cfg->force_max_run;
  p.token_ranges = cfg->chunk_tokens > 0 ? (int32_t*)(sb + lay.token_ranges) : nullptr;
  p.cand_scores = (cfg->debug_outputs & 1) ? (float*)(sb + lay.cand_scores) : nullptr;
  p.S = (float*)(sb + lay.S);
  L->sweep = uses_sweep(cfg);
  L->inplace = L->sweep && (cfg->debug_outputs & 32) && rr_route_sweep_inplace_supported(p);
  L->fused = uses_fused(cfg);
  L->dense_rescore = !(cfg->debug_outputs & 4) && rr_rescore_dense_supported(p);
  *out = L;
  return RR_OK;
}

int rr_ledger_reset(rr_ledger* L, void* stream) {
  if (!L) return RR_ERR_INVALID_ARG;
  RR_CUDA(rr_launch_reset(L->p, (cudaStream_t)stream));
  L->anchored = 0;
  L->call_index = 0;
  return RR_OK;
}

int rr_ledger_destroy(rr_ledger* L) {
  if (!L) return RR_ERR_INVALID_ARG;
  for (int b = 0; b < 2; ++b)
    for (cudaEvent_t e : {L->ev_copied[b], L->ev_consumed[b], L->ev_snap[b], L->ev_d2h[b]})
      if (e) cudaEventDestroy(e);
  delete L;
  return RR_OK;
}

int rr_route_anchor(rr_ledger* L, const void* qc, const void* kc, int32_t layer, void* stream) {
  return route_layer(L, qc, kc, layer, true, (cudaStream_t)stream);
}

int rr_route_relay(rr_ledger* L, const void* qc, const void* kc, int32_t layer, void* stream) {
  return route_layer(L, qc, kc, layer, false, (cudaStream_t)stream);
}

int rr_route_layer_host(rr_ledger* L, const void* host_qc, const void* host_kc,
                        void* dev_qc_staging, void* dev_kc_staging, int32_t layer,
                        int32_t is_anchor, int32_t* host_routes, void* stream) {
  if (!L || !host_qc || !host_kc || !dev_qc_staging || !dev_kc_staging) return RR_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const RRParams& p = L->p;
  const size_t esz = p.dtype == RR_F32 ? 4 : 2;
  const size_t qb = (size_t)p.P * p.n_q * p.d * esz, kb = (size_t)p.P * p.n_k * p.d * esz;
  if (!is_anchor && !L->anchored) return RR_ERR_STATE;
  RR_CUDA(cudaMemcpyAsync(dev_qc_staging, host_qc, qb, cudaMemcpyHostToDevice, st));
  RR_CUDA(cudaMemcpyAsync(dev_kc_staging, host_kc, kb, cudaMemcpyHostToDevice, st));
  int rc = route_layer(L, dev_qc_staging, dev_kc_staging, layer, is_anchor != 0, st);
  if (rc != RR_OK) return rc;
  if (host_routes)
    RR_CUDA(cudaMemcpyAsync(host_routes, p.routes, (size_t)p.rows * p.k * 4,
                            cudaMemcpyDeviceToHost, st));
  return RR_OK;
}

int rr_route_layers_host(rr_ledger* L, int32_t n_layers, const void* const* host_qc,
                         const void* const* host_kc, const int32_t* is_anchor,
                         int32_t first_layer, void* const* dev_qc_staging,
                         void* const* dev_kc_staging, void* const* dev_routes_staging,
                         int32_t* const* host_routes, void* stream, void* copy_stream,
                         void* d2h_stream) {
  if (!L || n_layers < 0 || !host_qc || !host_kc || !is_anchor || !dev_qc_staging ||
      !dev_kc_staging || first_layer < 0)
    return RR_ERR_INVALID_ARG;
  if (host_routes && !dev_routes_staging) return RR_ERR_INVALID_ARG;
  for (int b = 0; b < 2; ++b)
    if (!dev_qc_staging[b] || !dev_kc_staging[b] || (host_routes && !dev_routes_staging[b]))
      return RR_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!host_qc[l] || !host_kc[l]) return RR_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream, cs = (cudaStream_t)copy_stream;
  cudaStream_t ds = d2h_stream ? (cudaStream_t)d2h_stream : cs;
  const RRParams& p = L->p;
  const size_t esz = p.dtype == RR_F32 ? 4 : 2;
  const size_t qb = (size_t)p.P * p.n_q * p.d * esz, kb = (size_t)p.P * p.n_k * p.d * esz;
  const size_t rb = (size_t)p.rows * p.k * 4;
  for (int b = 0; b < 2; ++b) {
    cudaEvent_t* evs[4] = {&L->ev_copied[b], &L->ev_consumed[b], &L->ev_snap[b], &L->ev_d2h[b]};
    for (auto e : evs)
      if (!*e) RR_CUDA(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
  }
  // inputs of layer l -> staging set l%2 once its previous user has consumed it (layer l-2, or
  // a layer of the previous call: the events live in the ledger, and waiting on an event that
  // was never recorded returns at once); issued one layer ahead so that the copy stream never
  // queues an upload behind a download that waits for compute
  auto upload = [&](int l) -> int {
    const int b = l & 1;
    RR_CUDA(cudaStreamWaitEvent(cs, L->ev_consumed[b], 0));
    RR_CUDA(cudaMemcpyAsync(dev_qc_staging[b], host_qc[l], qb, cudaMemcpyHostToDevice, cs));
    RR_CUDA(cudaMemcpyAsync(dev_kc_staging[b], host_kc[l], kb, cudaMemcpyHostToDevice, cs));
    RR_CUDA(cudaEventRecord(L->ev_copied[b], cs));
    return RR_OK;
  };
  if (n_layers > 0) { int rc = upload(0); if (rc != RR_OK) return rc; }
  for (int l = 0; l < n_layers; ++l) {
    const int b = l & 1;
    RR_CUDA(cudaStreamWaitEvent(st, L->ev_copied[b], 0));
    int rc = route_layer(L, dev_qc_staging[b], dev_kc_staging[b], first_layer + l,
                         is_anchor[l] != 0, st);
    if (rc != RR_OK) return rc;
    RR_CUDA(cudaEventRecord(L->ev_consumed[b], st));
    if (l + 1 < n_layers) { rc = upload(l + 1); if (rc != RR_OK) return rc; }
    if (host_routes && host_routes[l]) {
      // snapshot on the compute stream (device to device), copy out on the download stream
      RR_CUDA(cudaStreamWaitEvent(st, L->ev_d2h[b], 0));   // the staging set's last download
      RR_CUDA(cudaMemcpyAsync(dev_routes_staging[b], p.routes, rb, cudaMemcpyDeviceToDevice, st));
      RR_CUDA(cudaEventRecord(L->ev_snap[b], st));
      RR_CUDA(cudaStreamWaitEvent(ds, L->ev_snap[b], 0));
      RR_CUDA(cudaMemcpyAsync(host_routes[l], dev_routes_staging[b], rb, cudaMemcpyDeviceToHost, ds));
      RR_CUDA(cudaEventRecord(L->ev_d2h[b], ds));
    }
  }
  return RR_OK;
}

int rr_ledger_views(rr_ledger* L, rr_views* out) {
  if (!L || !out) return RR_ERR_INVALID_ARG;
  const RRParams& p = L->p;
  out->routes = p.routes; out->sentinels = p.sentinels; out->ages = p.ages;
  out->kth_score = p.kth; out->margin = p.margin; out->flags = p.flags;
  out->alpha = p.alpha; out->beta = p.beta; out->refresh_rows = p.refresh_rows;
  out->refresh_count = p.refresh_count; out->problem_offsets = p.problem_offsets;
  out->token_ranges = p.token_ranges; out->cand_scores = p.cand_scores;
  out->counters = (uint64_t*)p.counters; out->status = p.status;
  out->force_state = p.force_stats;
  return RR_OK;
}

static int xfer(rr_ledger* L, void* blob, size_t bytes, cudaStream_t st, bool to_host) {
  if (!L || !blob) return RR_ERR_INVALID_ARG;
  if (bytes < L->export_bytes) return RR_ERR_TOO_SMALL;
  const RRParams& p = L->p;
  const size_t rows = (size_t)p.rows;
  struct Part { void* dev; size_t n; } parts[5] = {
      {p.routes, rows * p.k * 4}, {p.sentinels, rows * p.sw * 4}, {p.ages, rows * 4},
      {p.kth, rows * 4}, {p.margin, rows * 4}};
  char* h = (char*)blob;
  for (auto& pt : parts) {
    if (pt.n) {
      if (to_host) RR_CUDA(cudaMemcpyAsync(h, pt.dev, pt.n, cudaMemcpyDeviceToHost, st));
      else RR_CUDA(cudaMemcpyAsync(pt.dev, h, pt.n, cudaMemcpyHostToDevice, st));
    }
    h += pt.n;
  }
  RR_CUDA(cudaStreamSynchronize(st));
  return RR_OK;
}

int rr_ledger_export(rr_ledger* L, void* host_blob, size_t bytes, void* stream) {
  return xfer(L, host_blob, bytes, (cudaStream_t)stream, true);
}

int rr_ledger_import(rr_ledger* L, const void* host_blob, size_t bytes, void* stream) {
  int rc = xfer(L, const_cast<void*>(host_blob), bytes, (cudaStream_t)stream, false);
  if (rc == RR_OK) {
    // a restored ledger counts as anchored iff no row carries the "never routed" age
    // (checked by the caller's data; the library trusts an imported checkpoint)
    L->anchored = 1;
  }
  return rc;
}

int rr_ledger_status(rr_ledger* L, void* stream, uint32_t* status_out) {
  if (!L || !status_out) return RR_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t s = 0;
  RR_CUDA(cudaMemcpyAsync(&s, L->p.status, 4, cudaMemcpyDeviceToHost, st));
  RR_CUDA(cudaStreamSynchronize(st));
  *status_out = s;
  return (s & RR_STATUS_TIMEOUT) ? RR_ERR_TIMEOUT : RR_OK;
}

uint32_t rr_sampler_draw_u32(uint64_t seed, uint32_t g, uint32_t layer, uint32_t t) {
  return rr_draw_u32(rr_row_key(seed, g), layer, t);
}

int rr_profile_begin(rr_ledger* L) {
  if (!L) return RR_ERR_INVALID_ARG;
  for (auto& r : L->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  L->prof.clear();
  L->profiling = true;
  return RR_OK;
}

int rr_profile_end(rr_ledger* L, void* stream, float* total_ms, int64_t* launches) {
  if (!L || !total_ms || !launches) return RR_ERR_INVALID_ARG;
  L->profiling = false;
  for (int i = 0; i < RR_NUM_KINDS; ++i) { total_ms[i] = 0.f; launches[i] = 0; }
  RR_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  for (auto& r : L->prof) {
    float ms = 0.f;
    RR_CUDA(cudaEventElapsedTime(&ms, r.a, r.b));
    total_ms[r.kind] += ms;
    launches[r.kind] += 1;
    cudaEventDestroy(r.a); cudaEventDestroy(r.b);
  }
  L->prof.clear();
  return RR_OK;
}

const char* rr_kind_name(int kind) {
  switch (kind) {
    case RR_KIND_SCORE_SIMT: return "score_simt";
    case RR_KIND_TOPK_ROWS: return "topk_rows";
    case RR_KIND_RESCORE: return "rescore";
    case RR_KIND_COMPACT: return "compact";
    case RR_KIND_ANCHOR_FILL: return "anchor_fill";
    case RR_KIND_UPDATE: return "update";
    case RR_KIND_EXPAND: return "expand";
    case RR_KIND_SCORE_TC: return "score_tc";
    case RR_KIND_ROUTE_FUSED: return "route_fused";
    case RR_KIND_RESCORE_DENSE: return "rescore_dense";
    case RR_KIND_SENTINELS: return "sentinels";
    default: return "";
  }
}

uint64_t rr_kernel_launch_count(void) { return g_launches.load(); }

const char* rr_strerror(int code) {
  switch (code) {
    case RR_OK: return "ok";
    case RR_ERR_INVALID_ARG: return "invalid argument";
    case RR_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case RR_ERR_STATE: return "ledger state does not allow this call (relay before anchor)";
    case RR_ERR_CUDA: return "CUDA runtime error";
    case RR_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case RR_ERR_TOO_SMALL: return "buffer too small";
    case RR_ERR_TOO_LARGE: return "problem exceeds a fixed built-in capacity";
    default: return "unknown error";
  }
}

const char* rr_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
