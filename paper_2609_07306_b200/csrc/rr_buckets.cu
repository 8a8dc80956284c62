// Route-width buckets (Section 4.4: "Ledgers are bucketed by route width so rows with compatible
// shapes share kernels"; Section 4.3: the ledger stores whichever route width the underlying
// policy requests).  Problems (batch x head pairs) that ask for the same route width k form one
// bucket; a bucket is an ordinary ledger over its problems, and one call per layer runs every
// bucket's kernel set on the caller's stream.  Host logic only: the kernels are the ledger's.
//
// Layout contract: the caller lays Qc / Kc out bucket-major -- the problems of bucket 0 first,
// then bucket 1, ... -- in the order rr_bucket_plan reports (buckets in ascending width,
// problems of a bucket in ascending input index).  A bucket's inputs are then one contiguous
// [problems, n, d] block and no gather or copy is needed.  Rows are numbered inside their
// bucket (row id = position in the bucket * n_q + i): that id keys the sentinel sampler.
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "rr_common.cuh"

struct rr_bucket_set {
  struct Bucket {
    rr_config cfg;
    rr_ledger* ledger;
    int first_slot, problems;
    size_t ledger_offset, scratch_offset, ledger_bytes, scratch_bytes;
  };
  std::vector<Bucket> buckets;
  std::vector<int32_t> order;       // order[s] = input index of the problem at bucket-major slot s
  rr_config base;
};

namespace {

constexpr size_t kAlign = 256;
size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Buckets (ascending width) and bucket-major order of the problems.  widths[p] >= 1.
int plan(const rr_config* cfg, const int32_t* widths, int32_t n, std::vector<int32_t>& order,
         std::vector<rr_bucket_set::Bucket>& buckets) {
  if (!cfg || !widths || n <= 0 || n != cfg->batch * cfg->heads) return RR_ERR_INVALID_ARG;
  for (int p = 0; p < n; ++p)
    if (widths[p] < 1 || widths[p] > cfg->n_k) return RR_ERR_INVALID_ARG;
  order.resize(n);
  for (int p = 0; p < n; ++p) order[p] = p;
  std::stable_sort(order.begin(), order.end(),
                   [&](int a, int b) { return widths[a] < widths[b]; });
  buckets.clear();
  size_t lo = 0, so = 0;
  for (int s = 0; s < n;) {
    int e = s;
    while (e < n && widths[order[e]] == widths[order[s]]) ++e;
    rr_bucket_set::Bucket b{};
    b.cfg = *cfg;
    b.cfg.batch = 1; b.cfg.heads = e - s; b.cfg.k = widths[order[s]];
    b.ledger = nullptr; b.first_slot = s; b.problems = e - s;
    const int rc = rr_workspace_bytes(&b.cfg, &b.ledger_bytes, &b.scratch_bytes);
    if (rc != RR_OK) return rc;
    b.ledger_offset = lo; b.scratch_offset = so;
    lo += up(b.ledger_bytes); so += up(b.scratch_bytes);
    buckets.push_back(b);
    s = e;
  }
  return RR_OK;
}

}  // namespace

extern "C" {

int rr_bucket_plan(const rr_config* cfg, const int32_t* widths, int32_t n_problems,
                   int32_t* order_out, int32_t* n_buckets_out, size_t* ledger_bytes,
                   size_t* scratch_bytes) {
  std::vector<int32_t> order;
  std::vector<rr_bucket_set::Bucket> buckets;
  const int rc = plan(cfg, widths, n_problems, order, buckets);
  if (rc != RR_OK) return rc;
  if (order_out) std::memcpy(order_out, order.data(), sizeof(int32_t) * order.size());
  if (n_buckets_out) *n_buckets_out = (int32_t)buckets.size();
  const auto& last = buckets.back();
  if (ledger_bytes) *ledger_bytes = last.ledger_offset + up(last.ledger_bytes);
  if (scratch_bytes) *scratch_bytes = last.scratch_offset + up(last.scratch_bytes);
  return RR_OK;
}

int rr_bucket_set_init(const rr_config* cfg, const int32_t* widths, int32_t n_problems,
                       void* dev_ledger, size_t ledger_bytes, void* dev_scratch,
                       size_t scratch_bytes, rr_bucket_set** out) {
  if (!out || !dev_ledger || !dev_scratch) return RR_ERR_INVALID_ARG;
  if (((uintptr_t)dev_ledger & 255u) || ((uintptr_t)dev_scratch & 255u)) return RR_ERR_INVALID_ARG;
  rr_bucket_set* S = new (std::nothrow) rr_bucket_set();
  if (!S) return RR_ERR_INVALID_ARG;
  S->base = *cfg;
  int rc = plan(cfg, widths, n_problems, S->order, S->buckets);
  if (rc == RR_OK) {
    const auto& last = S->buckets.back();
    if (ledger_bytes < last.ledger_offset + up(last.ledger_bytes) ||
        scratch_bytes < last.scratch_offset + up(last.scratch_bytes))
      rc = RR_ERR_TOO_SMALL;
  }
  for (size_t b = 0; rc == RR_OK && b < S->buckets.size(); ++b) {
    auto& B = S->buckets[b];
    rc = rr_ledger_init(&B.cfg, (char*)dev_ledger + B.ledger_offset, B.ledger_bytes,
                        (char*)dev_scratch + B.scratch_offset, B.scratch_bytes, &B.ledger);
  }
  if (rc != RR_OK) { rr_bucket_set_destroy(S); return rc; }
  *out = S;
  return RR_OK;
}

int rr_bucket_set_destroy(rr_bucket_set* S) {
  if (!S) return RR_ERR_INVALID_ARG;
  for (auto& B : S->buckets)
    if (B.ledger) rr_ledger_destroy(B.ledger);
  delete S;
  return RR_OK;
}

int rr_bucket_set_count(const rr_bucket_set* S) {
  return S ? (int)S->buckets.size() : RR_ERR_INVALID_ARG;
}

int rr_bucket_set_info(const rr_bucket_set* S, int32_t b, rr_bucket_info* out) {
  if (!S || !out || b < 0 || b >= (int)S->buckets.size()) return RR_ERR_INVALID_ARG;
  const auto& B = S->buckets[b];
  out->k = B.cfg.k; out->problems = B.problems; out->first_slot = B.first_slot;
  out->ledger_offset = B.ledger_offset; out->scratch_offset = B.scratch_offset;
  out->ledger_bytes = B.ledger_bytes; out->scratch_bytes = B.scratch_bytes;
  return RR_OK;
}

rr_ledger* rr_bucket_set_ledger(rr_bucket_set* S, int32_t b) {
  return (S && b >= 0 && b < (int)S->buckets.size()) ? S->buckets[b].ledger : nullptr;
}

int rr_bucket_set_reset(rr_bucket_set* S, void* stream) {
  if (!S) return RR_ERR_INVALID_ARG;
  for (auto& B : S->buckets) {
    const int rc = rr_ledger_reset(B.ledger, stream);
    if (rc != RR_OK) return rc;
  }
  return RR_OK;
}

// One layer for every bucket.  qc / kc: device, bucket-major [P, n_q, d] / [P, n_k, d].
int rr_bucket_route_layer(rr_bucket_set* S, const void* qc, const void* kc, int32_t layer,
                          int32_t is_anchor, void* stream) {
  if (!S || !qc || !kc) return RR_ERR_INVALID_ARG;
  const size_t esz = S->base.dtype == RR_BF16 ? 2 : 4;
  const size_t q_prob = (size_t)S->base.n_q * S->base.d * esz, k_prob = (size_t)S->base.n_k * S->base.d * esz;
  for (auto& B : S->buckets) {
    const void* q = (const char*)qc + (size_t)B.first_slot * q_prob;
    const void* k = (const char*)kc + (size_t)B.first_slot * k_prob;
    const int rc = is_anchor ? rr_route_anchor(B.ledger, q, k, layer, stream)
                             : rr_route_relay(B.ledger, q, k, layer, stream);
    if (rc != RR_OK) return rc;
  }
  return RR_OK;
}

// The worst status over the buckets (synchronous, like rr_ledger_status).
int rr_bucket_set_status(rr_bucket_set* S, void* stream, uint32_t* status_out) {
  if (!S) return RR_ERR_INVALID_ARG;
  uint32_t all = 0; int worst = RR_OK;
  for (auto& B : S->buckets) {
    uint32_t st = 0;
    const int rc = rr_ledger_status(B.ledger, stream, &st);
    all |= st;
    if (rc != RR_OK && worst == RR_OK) worst = rc;
  }
  if (status_out) *status_out = all;
  return worst;
}

}  // extern "C"
