/*
 * routerelay.h -- C ABI of the B200 (sm_100a) route-maintenance library.
 *
 * The library maintains, on the device, the RouteRelay "route ledger" of a batch of
 * independent routing problems (one per batch x head pair) across Transformer layers:
 *
 *   anchor layer : full chunk routing  S = Qc Kc^T (Eq. 1), per-row TopK (Eq. 2), and a
 *                  ledger of each row's k selected chunks, its m near-miss chunks and r
 *                  seeded random sentinels (Section 3.1);
 *   relay layer  : rescoring of route + sentinels against the current layer's Qc/Kc
 *                  (Section 3.2), the challenge test alpha > beta + gamma (Eq. 5),
 *                  prefix-sum compaction of the failing rows, full re-routing of exactly
 *                  those rows, and the ledger update (Sections 4.1, 4.2).
 *
 * Conventions
 *   - Every function returns an int status: RR_OK (0) or a negative RR_ERR_* code.  Nothing
 *     throws, aborts or traps.  rr_strerror() names a code.
 *   - "device pointer" means memory of the CUDA device that was current when
 *     rr_ledger_init() ran; "host pointer" means ordinary (preferably pinned) host memory.
 *   - The library allocates no device memory.  The caller owns the ledger buffer and the
 *     scratch buffer (sizes from rr_workspace_bytes) and must keep them alive, and must not
 *     touch them while work is in flight, until rr_ledger_destroy().
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     rr_route_anchor / rr_route_relay only enqueue work: they never synchronise with the
 *     host.  Results are read through rr_ledger_views() after the caller has synchronised
 *     the stream.
 *   - Qc is [batch, heads, n_q, d], Kc is [batch, heads, n_k, d], contiguous row-major,
 *     16-byte aligned, dtype per rr_config.dtype; both are borrowed until the enqueued work
 *     has finished.
 *   - Row ids are global: g = problem * n_q + i with problem = batch_index * heads + head.
 *   - Chunk ids are int32; a slot a row cannot fill (fewer valid chunks than k, m or r)
 *     holds -1.  The order of ids inside a route / near-miss / random group carries no
 *     meaning (the paper defines them as sets).
 *   - Ties in TopK break towards the smaller chunk id; -0.0 equals +0.0.
 */
#ifndef ROUTERELAY_H_
#define ROUTERELAY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RR_OK                 0
#define RR_ERR_INVALID_ARG   -1   /* null pointer, negative size, misaligned buffer, ...        */
#define RR_ERR_UNSUPPORTED   -2   /* shape / dtype outside what the kernels are built for      */
#define RR_ERR_STATE         -3   /* e.g. relay on a ledger that was never anchored            */
#define RR_ERR_CUDA          -4   /* a CUDA runtime call failed (see rr_last_cuda_error)       */
#define RR_ERR_TIMEOUT       -5   /* a bounded device-side wait expired (device status word)   */
#define RR_ERR_TOO_SMALL     -6   /* caller-provided buffer smaller than required              */
#define RR_ERR_TOO_LARGE     -7   /* problem exceeds a fixed built-in capacity                 */

#define RR_BF16 0
#define RR_F32  1

/* bits of the device status word (rr_ledger_status) */
#define RR_STATUS_TIMEOUT      1u  /* an mbarrier wait in a kernel gave up                     */
#define RR_STATUS_BAD_INDEX    2u  /* a ledger entry outside [0, v_i) was met and skipped      */

typedef struct rr_ledger rr_ledger;   /* opaque; owns only a small host struct */

/* One routing configuration.  P = batch*heads independent problems, rows = P*n_q. */
typedef struct rr_config {
  int32_t batch, heads;
  int32_t n_q, n_k;        /* query chunks / key chunks per problem                        */
  int32_t d;               /* representation width: 64 or 128                              */
  int32_t k, m, r;         /* route width (Eq. 2), near-miss and random sentinels (Sec 3.1)*/
  int32_t dtype;           /* RR_BF16 or RR_F32 (inputs; accumulation is always fp32)      */
  int32_t causal;          /* 0: every row sees all n_k chunks; 1: row i sees chunks
                              j < min(n_k, i + 1 + causal_offset)                          */
  int32_t causal_offset;
  float   gamma;           /* guard margin of Eq. 5, >= 0 (+inf allowed)                   */
  uint64_t seed;           /* seed of the random-sentinel sampler                          */
  int32_t chunk_tokens;    /* >0: also expand routes to token ranges of this chunk size    */
  int32_t debug_outputs;   /* bit 0: relay also stores every candidate score (tests);
                              bit 1: route through the two-pass path (score rows in scratch
                              + warp-level TopK) even where the fused kernel applies;
                              bit 2: rescore candidates with the gathered FP32 kernel even
                              where the tensor-core strip kernel applies;
                              bit 3 (tests): the two-sweep routing kernel hands every fifth
                              row to its exact slow path;
                              bit 4: route with the streaming fused kernel even where the
                              two-sweep kernel applies;
                              bit 5: relay in place -- the challenge test of Eq. 5 runs inside
                              the routing kernel on the scores of its first sweep (no separate
                              rescoring kernel, no second score GEMM over a compacted list);
                              the results are the same;
                              bit 8: route with the two-sweep kernel whatever the grid size
                              (by default grids of less than two waves of CTAs use the
                              streaming kernel: fewer launches, shorter latency chain);
                              bits 6, 7 (tests): the first wait of the first CTA of the first
                              routing launch (bit 6) / strip rescoring launch (bit 7) of this
                              ledger counts as expired, once: that CTA gives up as after a real
                              time-out and the status word gets RR_STATUS_TIMEOUT          */
  /* Optional policies either side of the trigger; all zero = the plain method.             */
  int32_t global_sentinels;/* mandatory global candidates (Section 3.1, item 3): bit 0 = the
                              sink chunk 0, bit 1 = the most recent chunk the row may select.
                              Each adds one slot after the random sentinels; a slot stays -1
                              if its chunk is in the route or among the near-miss sentinels;
                              the random sentinels are drawn from what is left              */
  int32_t min_reuse;       /* hysteresis (Section 3.2): a row fully routed fewer than this
                              many layers ago is reused without the test (the paper: 1)     */
  int32_t h_max;           /* forced anchors (Section 3.2), per row: >0 = a row whose route
                              is h_max or more layers old is re-routed whatever Eq. 5 says  */
  float   gamma_boost;     /* hysteresis: added to gamma for rows whose margin (Section 3.3)
                              recorded at their last routing is below margin_recover        */
  float   margin_recover;
  int32_t coalesce_ranges; /* with chunk_tokens > 0: runs of consecutive selected chunks become
                              one token range (the form a sparse-attention kernel consumes);
                              a row then holds its merged ranges first, (-1,-1) after them  */
  int32_t force_permille;  /* forced anchors "before layers known to have low route
                              persistence" (Section 3.2), decided on the device, no host round
                              trip: >0 = a relay call whose challenge test flags at least
                              ceil(rows * force_permille / 1000) rows makes the next relay
                              calls route every row like an anchor (flags all 1, ages 0,
                              sentinels redrawn, charged as anchor rows; the rescoring kernel
                              exits at once).  While the flagged count stays that high the forced
                              runs double -- 1, 2, 4, ... up to force_max_run calls -- with one
                              tested call between two runs; a tested call below the threshold
                              resets the run length; rr_route_anchor clears a pending run.
                              0 = off.  Not available together with debug_outputs bit 5.      */
  int32_t force_max_run;   /* longest forced run (values < 1 count as 1)                       */
} rr_config;

/* Device pointers into the caller's ledger/scratch buffers (valid until destroy). */
typedef struct rr_views {
  int32_t* routes;          /* [rows, k]     selected chunk ids                             */
  int32_t* sentinels;       /* [rows, m+r+g] near-miss (m), random (r), then g mandatory global slots */
  int32_t* ages;            /* [rows]        layers since the row was last fully routed; -1 after reset */
  float*   kth_score;       /* [rows]        weakest selected score when last routed        */
  float*   margin;          /* [rows]        Section 3.3 margin when last routed (+inf if nothing is unselected) */
  uint8_t* flags;           /* [rows]        1 = row failed Eq. 5 at the last relay (anchor: all 1) */
  float*   alpha;           /* [rows]        min route score at the last relay              */
  float*   beta;            /* [rows]        max sentinel score at the last relay (-inf if none) */
  int32_t* refresh_rows;    /* [rows]        ascending global ids of the flagged rows       */
  int32_t* refresh_count;   /* [1]           how many (= rho_l * rows)                      */
  int32_t* problem_offsets; /* [P+1]         exclusive scan of per-problem flagged counts   */
  int32_t* token_ranges;    /* [rows, k, 2]  [start,end) per route slot, ascending chunk id; NULL if chunk_tokens==0 */
  float*   cand_scores;     /* [rows, k+m+r+g] candidate scores of the last relay; NULL unless debug_outputs */
  uint64_t* counters;       /* [RR_NUM_COUNTERS] cumulative since reset, see below          */
  uint32_t* status;         /* [1]           RR_STATUS_* bits                               */
  int32_t* force_state;     /* [8]           forced-anchor policy: words 0-3 = {pending forced calls,
                                             run length} of the two call parities, 4 = forced calls
                                             since reset, 5 = the last relay call was forced        */
} rr_views;

/* counters[] indices: work accounting in the sense of the paper's "rerouted rows" and
 * "score pairs" columns (Section 5): anchors charge every row its full row; relays charge
 * every row its candidates and every flagged row its full row in addition. */
#define RR_CNT_LAYER_CALLS   0
#define RR_CNT_ANCHOR_ROWS   1
#define RR_CNT_RELAY_ROWS    2
#define RR_CNT_FLAGGED_ROWS  3
#define RR_CNT_CAND_PAIRS    4
#define RR_CNT_FULL_PAIRS    5
#define RR_CNT_DENSE_PAIRS   6   /* what full routing on every layer would have scored        */
#define RR_NUM_COUNTERS      8

/* Sizes of the two caller-owned device buffers for a configuration (Section 4.4: the ledger is
 * rows * (k + m + r) 32-bit indices plus a few words per row; the scratch holds the per-layer
 * flags, alpha / beta, the refresh list and counters).  Host-only. */
int rr_workspace_bytes(const rr_config* cfg, size_t* ledger_bytes, size_t* scratch_bytes);

/* Creates the host handle over caller-owned device buffers (both 256-byte aligned, at least
 * the sizes rr_workspace_bytes reports).  Does not touch the buffers: call rr_ledger_reset. */
int rr_ledger_init(const rr_config* cfg, void* dev_ledger, size_t ledger_bytes,
                   void* dev_scratch, size_t scratch_bytes, rr_ledger** out);

/* Enqueues: routes/sentinels = -1, ages = -1, counters = 0, status = 0. */
int rr_ledger_reset(rr_ledger* L, void* stream);

/* Frees the host handle only. */
int rr_ledger_destroy(rr_ledger* L);

/* Anchor layer (Section 4.1: "constructs this state from a complete chunk-score matrix").
 * Routes every row, rebuilds all sentinels with the sampler keyed by (seed, row, layer),
 * sets ages to 0, flags to 1, refresh_rows to all rows.  qc, kc: device pointers. */
int rr_route_anchor(rr_ledger* L, const void* qc, const void* kc, int32_t layer, void* stream);

/* Relay layer (Sections 3.2, 4.1, 4.2).  Requires a previous anchor (else RR_ERR_STATE).
 * The flagged-row list, its count and the refresh all stay on the device. */
int rr_route_relay(rr_ledger* L, const void* qc, const void* kc, int32_t layer, void* stream);

/* One layer driven from HOST buffers: copies qc/kc (host pointers, same layout) into the
 * caller's device staging buffers, runs the anchor (is_anchor != 0) or relay step, and
 * copies the routes [rows,k] back to host_routes (may be NULL).  All on `stream`, no host
 * synchronisation inside; the caller synchronises before reading host_routes. */
int rr_route_layer_host(rr_ledger* L, const void* host_qc, const void* host_kc,
                        void* dev_qc_staging, void* dev_kc_staging, int32_t layer,
                        int32_t is_anchor, int32_t* host_routes, void* stream);

/* A run of consecutive layers driven from HOST buffers, with the copies overlapped with the
 * routing: layer l's inputs are copied on `copy_stream` into staging set l%2 while layer l-1
 * runs on `stream`; after each layer its routes are snapshotted device-to-device and copied
 * to the host on `copy_stream`.
 *   host_qc / host_kc   [n_layers] host pointers (pinned memory for real overlap), layout as above
 *   is_anchor           [n_layers] non-zero = anchor layer
 *   dev_qc_staging / dev_kc_staging   [2] device buffers of one layer's Qc / Kc each
 *   dev_routes_staging  [2] device buffers of rows*k int32 each (may be NULL if host_routes is)
 *   host_routes         [n_layers] host pointers (rows*k int32 each) or NULL entries / NULL
 *   d2h_stream          stream of the route downloads (NULL = copy_stream); a separate one lets
 *                       uploads and downloads use both directions of the link at once
 * Enqueue-only: the caller synchronises ALL streams before reading host_routes or touching a
 * buffer itself.  Calls on the same ledger with the same staging buffers may follow one
 * another without a synchronisation in between: the library orders each reuse of a staging
 * set behind its previous reader (events kept in the ledger; a few are created on first use,
 * no device memory).  host_routes entries must not repeat while a download may still be in
 * flight. */
int rr_route_layers_host(rr_ledger* L, int32_t n_layers, const void* const* host_qc,
                         const void* const* host_kc, const int32_t* is_anchor,
                         int32_t first_layer, void* const* dev_qc_staging,
                         void* const* dev_kc_staging, void* const* dev_routes_staging,
                         int32_t* const* host_routes, void* stream, void* copy_stream,
                         void* d2h_stream);

/* Device pointers to state and per-layer outputs. */
int rr_ledger_views(rr_ledger* L, rr_views* out);

/* Checkpoint / restore of the ledger -- the three row-major tensors of Section 4.1 (routes,
 * sentinels, ages) plus the k-th score and margin recorded at each row's last routing -- to a
 * host blob of rr_export_bytes() bytes, laid out in that order, each array as in rr_views.
 * Both synchronise `stream`. */
int rr_export_bytes(const rr_config* cfg, size_t* bytes);
int rr_ledger_export(rr_ledger* L, void* host_blob, size_t bytes, void* stream);
int rr_ledger_import(rr_ledger* L, const void* host_blob, size_t bytes, void* stream);

/* Synchronous read of the device status word (RR_STATUS_* bits); RR_ERR_TIMEOUT is
 * returned if the timeout bit is set.  A CTA whose bounded wait expired leaves its rows as
 * they were (a relay may then hold flags and a refresh list that disagree for those rows; all
 * writes stay in bounds): after RR_ERR_TIMEOUT the ledger's contents are not to be used --
 * rr_ledger_reset (which clears the status word) and a new anchor bring it back. */
int rr_ledger_status(rr_ledger* L, void* stream, uint32_t* status_out);

/* Host-callable copy of the sampler's counter-based generator (the t-th 32-bit draw of
 * global row g when its sentinels are rebuilt at `layer`); same code the kernels run. */
uint32_t rr_sampler_draw_u32(uint64_t seed, uint32_t g, uint32_t layer, uint32_t t);

/* Row compaction for callers that cannot allocate device memory.  (The paper has no
 * counterpart of this entry point; it computes the same list as the compaction step of
 * rr_route_relay, Section 4.2.)
 *
 * Who needs it: code that runs where cudaMalloc may not be called -- a serving process
 * whose device memory pool is frozen after start-up, a plugin that is handed its input
 * and output buffers and nothing more, a latency path that cannot afford the implicit
 * synchronisation of an allocation.  The ledger API above asks such a caller for a scratch
 * buffer; this call asks for nothing beyond inputs and outputs.  Its scratch (per-tile
 * flagged counts) lives in a fixed array inside the library image: every GPU that loads
 * the library holds RR_NOALLOC_MAX_TILES * 4 bytes (256 KB) for it until the process exits.
 *
 *   dev_flags               [n_problems * n_q] device, in : non-zero = row is flagged
 *   dev_rows_out            [n_problems * n_q] device, out: ascending global ids of the flagged
 *                           rows in the first *dev_count_out entries (rest untouched)
 *   dev_count_out           [1] device, out
 *   dev_problem_offsets_out [n_problems + 1] device, out: exclusive scan of per-problem counts
 *
 * Limit: ceil(n_q / 128) * n_problems <= RR_NOALLOC_MAX_TILES (8.4 M rows when n_q is a
 * multiple of 128); larger inputs return RR_ERR_TOO_LARGE and nothing is enqueued.
 * Cost: each 128-row tile's CTA re-sums the flagged counts of all earlier tiles (no waits between
 * CTAs), n_tiles^2 / 2 four-byte reads from L2 in total: negligible at a few thousand tiles,
 * milliseconds near the limit of 65536.
 * The call allocates nothing, on the host or the device, and only enqueues work on `stream`.
 * The first call on a device also looks up the array's device address (once per device,
 * with that device current); make that first call before starting any stream capture.
 * All calls share the one array, which keeps the previous call's contents (every entry
 * that is read is rewritten first, so nothing needs clearing): calls whose kernels can
 * overlap on the GPU -- different streams or threads -- race and must be serialised by
 * the caller. */
#define RR_NOALLOC_MAX_TILES 65536
int rr_compact_flags_noalloc(const uint8_t* dev_flags, int32_t n_problems, int32_t n_q,
                             int32_t* dev_rows_out, int32_t* dev_count_out,
                             int32_t* dev_problem_offsets_out, void* stream);

/* ---- Route-width buckets (Section 4.4: "Ledgers are bucketed by route width so rows with
 * compatible shapes share kernels"; Section 4.3: the ledger stores whichever route width the
 * underlying policy requests) ------------------------------------------------------------------
 * Problems (batch x head pairs) that ask for the same route width k form one bucket; a bucket is
 * an ordinary ledger over its problems (same n_q, n_k, d, m, r, policies as cfg; cfg->k is
 * ignored), and rr_bucket_route_layer runs every bucket's kernel set with one call per layer.
 *
 * Layout contract: Qc and Kc are laid out BUCKET-MAJOR -- the problems of bucket 0 first, then
 * bucket 1, ... -- in the order rr_bucket_plan reports: buckets in ascending width, the problems
 * of a bucket in ascending input index; order[s] = input index of the problem at slot s.  A
 * bucket's inputs are then one contiguous [problems, n, d] block and nothing is gathered or
 * copied.  Rows are numbered inside their bucket (position in the bucket * n_q + i); that id
 * keys the sentinel sampler, so a bucket's results equal those of a stand-alone ledger (and of
 * the method's definition) run on that bucket's problems alone.
 * widths: host array [n_problems], 1 <= widths[p] <= n_k; n_problems = cfg->batch * cfg->heads.
 * The set owns its ledgers' host handles, not the two device buffers (caller-owned, 256-byte
 * aligned, at least the sizes rr_bucket_plan reports; bucket b uses the sub-ranges at
 * rr_bucket_info.ledger_offset / scratch_offset). */
typedef struct rr_bucket_set rr_bucket_set;
typedef struct rr_bucket_info {
  int32_t k;               /* route width of the bucket                                       */
  int32_t problems;        /* how many problems it holds                                      */
  int32_t first_slot;      /* bucket-major slot of its first problem                          */
  size_t ledger_offset, scratch_offset, ledger_bytes, scratch_bytes;
} rr_bucket_info;
/* Host-only.  order_out [n_problems] (may be NULL), the number of buckets and the sizes of the
 * two device buffers that hold all buckets. */
int rr_bucket_plan(const rr_config* cfg, const int32_t* widths, int32_t n_problems,
                   int32_t* order_out, int32_t* n_buckets_out, size_t* ledger_bytes,
                   size_t* scratch_bytes);
int rr_bucket_set_init(const rr_config* cfg, const int32_t* widths, int32_t n_problems,
                       void* dev_ledger, size_t ledger_bytes, void* dev_scratch,
                       size_t scratch_bytes, rr_bucket_set** out);
int rr_bucket_set_destroy(rr_bucket_set* S);
int rr_bucket_set_count(const rr_bucket_set* S);                 /* number of buckets (>= 1)    */
int rr_bucket_set_info(const rr_bucket_set* S, int32_t b, rr_bucket_info* out);
rr_ledger* rr_bucket_set_ledger(rr_bucket_set* S, int32_t b);    /* borrowed; for rr_ledger_views */
int rr_bucket_set_reset(rr_bucket_set* S, void* stream);
/* One layer for all buckets, enqueued on `stream` bucket after bucket.  qc / kc: device,
 * bucket-major [P, n_q, d] / [P, n_k, d].  is_anchor != 0: anchor layer, else relay layer
 * (RR_ERR_STATE before the first anchor). */
int rr_bucket_route_layer(rr_bucket_set* S, const void* qc, const void* kc, int32_t layer,
                          int32_t is_anchor, void* stream);
/* OR of the buckets' status words; the first non-zero return of rr_ledger_status. Synchronous. */
int rr_bucket_set_status(rr_bucket_set* S, void* stream, uint32_t* status_out);

/* ---- A minimal consumer of token ranges (Eq. 3) ------------------------------------------------
 * out[i] = softmax(q_i K_R^T * scale) V_R over the tokens R covered by row i's token ranges
 * (views.token_ranges: [rows, slots, 2] = [start, end) per slot, (-1,-1) = empty; per route slot
 * or coalesced).  One warp per row, FP32 arithmetic in ascending token order, so coalesced and
 * per-slot ranges of the same route give bit-identical outputs.  A plain reference consumer, not
 * a tuned attention backend (Section 4.3 leaves the backend unchanged); no token-level mask.
 *   ranges  device int32 [rows, slots, 2]       q       device [rows, dh]
 *   keys    device [rows / n_q, tokens, dh]      values  device, same shape as keys
 *   dtype   RR_BF16 or RR_F32 (q, keys, values)  out     device float [rows, dh]
 * A row without tokens gets zeros.  dh <= 256. */
int rr_attend_token_ranges(const int32_t* ranges, int32_t rows, int32_t slots, int32_t n_q,
                           const void* q, const void* keys, const void* values, int32_t tokens,
                           int32_t dh, int32_t dtype, float scale, float* out, void* stream);

/* Per-kernel device timing for benchmarks.  Between rr_profile_begin and rr_profile_end
 * every kernel the layer calls launch is bracketed by CUDA events on the caller's stream
 * (this adds event records to the stream; do not leave it on in production).
 * rr_profile_end synchronises the stream and returns, per kernel kind (RR_KIND_*), the total
 * device time in milliseconds and the number of launches; arrays hold RR_NUM_KINDS entries. */
#define RR_KIND_SCORE_SIMT   0   /* score rows on FP32 ALUs (fp32 inputs)                    */
#define RR_KIND_TOPK_ROWS    1   /* warp-level TopK + sentinels over score rows in memory    */
#define RR_KIND_RESCORE      2   /* gathered candidate rescoring + challenge test            */
#define RR_KIND_COMPACT      3   /* ballot / prefix-scan row compaction + ages and counters  */
#define RR_KIND_ANCHOR_FILL  4   /* anchor: flags, identity refresh list, ages, counters     */
#define RR_KIND_UPDATE       5   /* reserved: ages and counters are written by kinds 3 and 4  */
#define RR_KIND_EXPAND       6   /* token-range expansion                                    */
#define RR_KIND_SCORE_TC     7   /* tcgen05 score GEMM                                       */
#define RR_KIND_ROUTE_FUSED  8   /* tcgen05 score GEMM fused with TopK + sentinels           */
#define RR_KIND_RESCORE_DENSE 9  /* candidate rescoring from the tensor-core score strip     */
#define RR_KIND_SENTINELS    10  /* global + random sentinels of the rows just routed         */
#define RR_NUM_KINDS        12
int rr_profile_begin(rr_ledger* L);
int rr_profile_end(rr_ledger* L, void* stream, float* total_ms, int64_t* launches);
const char* rr_kind_name(int kind);

/* How many kernels the library has launched since it was loaded (all ledgers). */
uint64_t rr_kernel_launch_count(void);

const char* rr_strerror(int code);
const char* rr_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ROUTERELAY_H_ */
