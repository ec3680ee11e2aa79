// C ABI of libxkv: host-side argument validation, workspace sizing, status plumbing, and the
// host-only budget solver (Algorithm 1).  Device work is in xkv_score.cu, xkv_select.cu and
// xkv_decode.cu.
#include <atomic>
#include <cmath>
#include <queue>
#include <utility>
#include <thread>
#include <cstring>
#include <algorithm>
#include <vector>

#include "common.cuh"
#include "ops.h"

namespace xkv {

static std::atomic<int64_t> g_launches{0};

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

xkv_status check_launch() { return cudaGetLastError() == cudaSuccess ? XKV_OK : XKV_ERR_CUDA; }

int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

static std::atomic<uint64_t> g_wait_limit_ns{2000000000ull};
static std::atomic<int32_t> g_withhold_item{-1};

uint64_t wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }
int32_t debug_withhold_item() { return g_withhold_item.load(std::memory_order_relaxed); }

namespace {

xkv_status check_dims(const xkv_dims* d) {
  if (d == nullptr) return XKV_ERR_INVALID_ARG;
  if (d->batch <= 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->n_q_heads % d->n_kv_heads != 0)
    return XKV_ERR_INVALID_ARG;
  if (d->head_dim != 64 && d->head_dim != 128) return XKV_ERR_UNSUPPORTED;
  if (!(d->scale >= 0.f) || std::isinf(d->scale)) return XKV_ERR_INVALID_ARG;
  return XKV_OK;
}

xkv_status check_prefill_dims(const xkv_dims* d) {
  xkv_status s = check_dims(d);
  if (s != XKV_OK) return s;
  if (d->window <= 0) return XKV_ERR_INVALID_ARG;
  if (d->pool_kernel < 1 || d->pool_kernel > 63 || d->pool_kernel % 2 == 0) return XKV_ERR_INVALID_ARG;
  if (d->pool_mode != XKV_POOL_MAX && d->pool_mode != XKV_POOL_AVG) return XKV_ERR_INVALID_ARG;
  const int64_t rows = (int64_t)(d->n_q_heads / d->n_kv_heads) * d->window;
  if (rows < 1 || rows > 256) return XKV_ERR_UNSUPPORTED;
  if (d->kv_stride_head < d->head_dim || d->kv_stride_head % 8 != 0) return XKV_ERR_INVALID_ARG;
  if (d->kv_stride_token < (int64_t)d->n_kv_heads * d->head_dim || d->kv_stride_token % 8 != 0)
    return XKV_ERR_INVALID_ARG;
  return XKV_OK;
}

xkv_status check_cache(const xkv_cache* c, const xkv_dims* d) {
  if (c == nullptr) return XKV_ERR_INVALID_ARG;
  if (c->k_pages == nullptr || c->v_pages == nullptr || c->block_table == nullptr || c->seq_lens == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (!aligned16(c->k_pages) || !aligned16(c->v_pages) || !aligned16(c->block_table) || !aligned16(c->seq_lens))
    return XKV_ERR_INVALID_ARG;
  if (c->n_layers <= 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0) return XKV_ERR_INVALID_ARG;
  if (c->page_size <= 0 || c->page_size % 16 != 0 || c->page_size > 256) return XKV_ERR_INVALID_ARG;
  if ((int64_t)c->max_pages_per_seq * c->page_size > (1 << 30)) return XKV_ERR_INVALID_ARG;
  if (c->kv_format != XKV_KV_BF16 && c->kv_format != XKV_KV_INT8) return XKV_ERR_INVALID_ARG;
  if (c->kv_format == XKV_KV_INT8 &&
      (c->k_scales == nullptr || c->v_scales == nullptr || !aligned16(c->k_scales) || !aligned16(c->v_scales)))
    return XKV_ERR_INVALID_ARG;
  (void)d;
  return XKV_OK;
}

}  // namespace
}  // namespace xkv

using namespace xkv;

extern "C" {

xkv_status xkv_score(const xkv_dims* dims, const void* q_win, const void* k, const int32_t* cu_seqlens,
                     int64_t total_tokens, int32_t max_seqlen, float* scores, float* sorted, float* gains,
                     float* mass, int32_t curve_len, void* workspace, size_t workspace_bytes, void* stream) {
  xkv_status s = check_prefill_dims(dims);
  if (s != XKV_OK) return s;
  if (q_win == nullptr || k == nullptr || cu_seqlens == nullptr || scores == nullptr || workspace == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (sorted != nullptr && (gains == nullptr || curve_len < 1)) return XKV_ERR_INVALID_ARG;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(cu_seqlens) || !aligned16(scores) || !aligned16(sorted) ||
      !aligned16(gains) || !aligned16(mass) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return XKV_ERR_INVALID_ARG;
  if (total_tokens <= 0 || total_tokens >= (1ll << 31) || max_seqlen <= 0 || max_seqlen > total_tokens)
    return XKV_ERR_INVALID_ARG;
  const size_t need = score_workspace_bytes(dims, max_seqlen, total_tokens);
  if (need == 0) return XKV_ERR_INVALID_ARG;
  if (workspace_bytes < need) return XKV_ERR_WORKSPACE;
  return score(dims, q_win, k, cu_seqlens, total_tokens, max_seqlen, scores, sorted, gains, mass, curve_len,
               workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

xkv_status xkv_score_lse(const xkv_dims* dims, const void* q_win, const void* k, const int32_t* cu_seqlens,
                         int64_t total_tokens, int32_t max_seqlen, const float* lse, float* scores, float* sorted,
                         float* gains, float* mass, int32_t curve_len, void* workspace, size_t workspace_bytes,
                         void* stream) {
  xkv_status s = check_prefill_dims(dims);
  if (s != XKV_OK) return s;
  if (q_win == nullptr || k == nullptr || cu_seqlens == nullptr || scores == nullptr || workspace == nullptr ||
      lse == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (sorted != nullptr && (gains == nullptr || curve_len < 1)) return XKV_ERR_INVALID_ARG;
  if (!aligned16(q_win) || !aligned16(k) || !aligned16(cu_seqlens) || !aligned16(scores) || !aligned16(sorted) ||
      !aligned16(gains) || !aligned16(mass) || !aligned16(lse) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return XKV_ERR_INVALID_ARG;
  if (total_tokens <= 0 || total_tokens >= (1ll << 31) || max_seqlen <= 0 || max_seqlen > total_tokens)
    return XKV_ERR_INVALID_ARG;
  if (!score_lse_supported(dims, max_seqlen)) return XKV_ERR_UNSUPPORTED;
  const size_t need = score_workspace_bytes(dims, max_seqlen, total_tokens);
  if (need == 0) return XKV_ERR_INVALID_ARG;
  if (workspace_bytes < need) return XKV_ERR_WORKSPACE;
  return score(dims, q_win, k, cu_seqlens, total_tokens, max_seqlen, scores, sorted, gains, mass, curve_len,
               workspace, workspace_bytes, static_cast<cudaStream_t>(stream), lse);
}

xkv_status xkv_prefill_attn(const xkv_dims* dims, const void* q, const void* k, const void* v,
                            const int32_t* cu_seqlens, int64_t total_tokens, int32_t max_seqlen, void* out,
                            float* lse, void* workspace, size_t workspace_bytes, void* stream) {
  xkv_status s = check_dims(dims);
  if (s != XKV_OK) return s;
  if (q == nullptr || k == nullptr || v == nullptr || cu_seqlens == nullptr || out == nullptr || workspace == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(cu_seqlens) || !aligned16(out) ||
      !aligned16(lse) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return XKV_ERR_INVALID_ARG;
  if (dims->kv_stride_head < dims->head_dim || dims->kv_stride_head % 8 != 0 ||
      dims->kv_stride_token < (int64_t)dims->n_kv_heads * dims->head_dim || dims->kv_stride_token % 8 != 0)
    return XKV_ERR_INVALID_ARG;
  if (total_tokens <= 0 || total_tokens >= (1ll << 31) || max_seqlen <= 0 || max_seqlen > total_tokens)
    return XKV_ERR_INVALID_ARG;
  if (workspace_bytes < prefill_workspace_bytes()) return XKV_ERR_WORKSPACE;
  return prefill_attn(dims, q, k, v, cu_seqlens, total_tokens, max_seqlen, out, lse, workspace,
                      static_cast<cudaStream_t>(stream));
}

xkv_status xkv_select_compact(const xkv_dims* dims, int32_t layer, const int32_t* budget, int32_t per_sequence,
                              const float* scores, const float* sorted, const void* k, const void* v,
                              const int32_t* cu_seqlens, int64_t total_tokens, int32_t max_seqlen,
                              const xkv_cache* cache, int32_t* sel, int32_t sel_stride, void* workspace,
                              size_t workspace_bytes, void* stream) {
  xkv_status s = check_prefill_dims(dims);
  if (s != XKV_OK) return s;
  s = check_cache(cache, dims);
  if (s != XKV_OK) return s;
  if (budget == nullptr || scores == nullptr || sorted == nullptr || k == nullptr || v == nullptr ||
      cu_seqlens == nullptr || workspace == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (!aligned16(scores) || !aligned16(sorted) || !aligned16(k) || !aligned16(v) || !aligned16(cu_seqlens) ||
      !aligned16(sel) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return XKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= cache->n_layers) return XKV_ERR_INVALID_ARG;
  if (total_tokens <= 0 || total_tokens >= (1ll << 31) || max_seqlen <= 0 || max_seqlen > total_tokens)
    return XKV_ERR_INVALID_ARG;
  if (per_sequence != XKV_BUDGET_PER_LAYER && per_sequence != XKV_BUDGET_PER_SEQUENCE &&
      per_sequence != XKV_BUDGET_PER_HEAD)
    return XKV_ERR_INVALID_ARG;
  const int n_budgets = per_sequence == XKV_BUDGET_PER_HEAD ? dims->batch * dims->n_kv_heads
                                                            : (per_sequence ? dims->batch : 1);
  int32_t max_budget = 0;
  for (int i = 0; i < n_budgets; ++i) {
    if (budget[i] < 0) return XKV_ERR_BUDGET;
    if (budget[i] > max_budget) max_budget = budget[i];
  }
  if (sel != nullptr && sel_stride <= 0) return XKV_ERR_INVALID_ARG;
  const size_t need = select_workspace_bytes(dims, max_seqlen, total_tokens);
  if (need == 0) return XKV_ERR_INVALID_ARG;
  if (workspace_bytes < need) return XKV_ERR_WORKSPACE;
  return select_compact(dims, layer, budget, per_sequence, scores, sorted, k, v, cu_seqlens, total_tokens,
                        max_seqlen, cache, sel, sel_stride, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream));
}

xkv_status xkv_batch_curves(const float* gains, int32_t n_layers, int32_t batch, int32_t curve_len, int32_t divisor,
                            float* out, void* stream) {
  if (gains == nullptr || out == nullptr || !aligned16(gains) || !aligned16(out)) return XKV_ERR_INVALID_ARG;
  if (n_layers <= 0 || batch <= 0 || curve_len <= 0 || divisor <= 0) return XKV_ERR_INVALID_ARG;
  return batch_curves(gains, n_layers, batch, curve_len, 1.0 / (double)divisor, out, static_cast<cudaStream_t>(stream));
}

xkv_status xkv_head_curves(const xkv_dims* dims, const float* scores, const float* sorted, const int32_t* cu_seqlens,
                           int64_t total_tokens, int32_t max_seqlen, float* head_gains, int32_t curve_len,
                           void* stream) {
  xkv_status s = check_prefill_dims(dims);
  if (s != XKV_OK) return s;
  if (scores == nullptr || sorted == nullptr || cu_seqlens == nullptr || head_gains == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (!aligned16(scores) || !aligned16(sorted) || !aligned16(cu_seqlens) || !aligned16(head_gains))
    return XKV_ERR_INVALID_ARG;
  if (total_tokens <= 0 || total_tokens >= (1ll << 31) || max_seqlen <= 0 || max_seqlen > total_tokens ||
      curve_len < 1)
    return XKV_ERR_INVALID_ARG;
  return head_curves(dims, scores, sorted, cu_seqlens, total_tokens, max_seqlen, head_gains, curve_len,
                     static_cast<cudaStream_t>(stream));
}

xkv_status xkv_build_block_table(const int32_t* first_page, const int32_t* n_pages_lb, const xkv_cache* cache,
                                 int32_t batch, void* stream) {
  if (first_page == nullptr || n_pages_lb == nullptr || cache == nullptr || cache->block_table == nullptr)
    return XKV_ERR_INVALID_ARG;
  if (!aligned16(first_page) || !aligned16(n_pages_lb) || !aligned16(cache->block_table)) return XKV_ERR_INVALID_ARG;
  if (batch <= 0 || cache->n_layers <= 0 || cache->max_pages_per_seq <= 0) return XKV_ERR_INVALID_ARG;
  return build_block_table(first_page, n_pages_lb, cache->n_layers * batch, cache->block_table,
                           cache->max_pages_per_seq, static_cast<cudaStream_t>(stream));
}

xkv_status xkv_decode_attn(const xkv_dims* dims, const xkv_cache* cache, int32_t layer_begin, int32_t layer_end,
                           const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                           int32_t chunk_rows, void* workspace, size_t workspace_bytes, void* stream) {
  xkv_status s = check_dims(dims);
  if (s != XKV_OK) return s;
  s = check_cache(cache, dims);
  if (s != XKV_OK) return s;
  if (q == nullptr || out == nullptr || workspace == nullptr) return XKV_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return XKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out) || !aligned16(lse) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return XKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > cache->n_layers) return XKV_ERR_INVALID_ARG;
  if (chunk_rows < 0 || chunk_rows % 64 != 0) return XKV_ERR_INVALID_ARG;
  if (dims->n_q_heads / dims->n_kv_heads > 8) return XKV_ERR_UNSUPPORTED;
  return decode_attn(dims, cache, layer_begin, layer_end, q, k_new, v_new, out, lse, chunk_rows, workspace,
                     workspace_bytes, static_cast<cudaStream_t>(stream));
}

xkv_status xkv_decode_attn_static(const xkv_dims* dims, const xkv_cache* cache, int32_t layer_begin,
                                  int32_t layer_end, const void* q, const void* k_new, const void* v_new,
                                  void* out, float* lse, int32_t chunk_rows, int32_t* status_out, void* stream) {
  xkv_status s = check_dims(dims);
  if (s != XKV_OK) return s;
  s = check_cache(cache, dims);
  if (s != XKV_OK) return s;
  if (q == nullptr || out == nullptr) return XKV_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return XKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out) || !aligned16(lse) ||
      (reinterpret_cast<uintptr_t>(status_out) & 3u) != 0)
    return XKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > cache->n_layers) return XKV_ERR_INVALID_ARG;
  if (chunk_rows < 0 || chunk_rows % 64 != 0) return XKV_ERR_INVALID_ARG;
  if (dims->n_q_heads / dims->n_kv_heads > 8) return XKV_ERR_UNSUPPORTED;
  if (cache->kv_format != XKV_KV_BF16) return XKV_ERR_UNSUPPORTED;
  return decode_attn_static(dims, cache, layer_begin, layer_end, q, k_new, v_new, out, lse, chunk_rows,
                            status_out, static_cast<cudaStream_t>(stream));
}

size_t xkv_workspace_bytes(int32_t op, const xkv_dims* dims, int32_t max_seqlen, int64_t total_tokens,
                           int32_t n_layers, int32_t max_cache_len, int32_t chunk_rows) {
  if (dims == nullptr) return 0;
  switch (op) {
    case XKV_OP_SCORE:
      if (check_prefill_dims(dims) != XKV_OK || max_seqlen <= 0 || total_tokens <= 0) return 0;
      return score_workspace_bytes(dims, max_seqlen, total_tokens);
    case XKV_OP_SELECT_COMPACT:
      if (check_prefill_dims(dims) != XKV_OK || max_seqlen <= 0 || total_tokens <= 0) return 0;
      return select_workspace_bytes(dims, max_seqlen, total_tokens);
    case XKV_OP_PREFILL_ATTN:
      if (check_dims(dims) != XKV_OK) return 0;
      return prefill_workspace_bytes();
    case XKV_OP_DECODE_ATTN:
      if (check_dims(dims) != XKV_OK || n_layers <= 0 || max_cache_len < 0 || chunk_rows < 0 ||
          chunk_rows % 64 != 0)
        return 0;
      return decode_workspace_bytes(dims, n_layers, max_cache_len, chunk_rows);
    default:
      return 0;
  }
}

xkv_status xkv_read_device_status(void* workspace, void* stream) {
  if (workspace == nullptr) return XKV_ERR_INVALID_ARG;
  int32_t status = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&status, workspace, sizeof(status), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return XKV_ERR_CUDA;
  if (cudaMemsetAsync(workspace, 0, sizeof(status), st) != cudaSuccess) return XKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return XKV_ERR_CUDA;
  return status;
}

void xkv_profile_events(void* start, void* stop) {
  set_profile_events(static_cast<cudaEvent_t>(start), static_cast<cudaEvent_t>(stop));
}

int64_t xkv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void xkv_test_hooks(int64_t wait_limit_ns, int32_t withhold_decode_item) {
  g_wait_limit_ns.store(wait_limit_ns > 0 ? (uint64_t)wait_limit_ns : 2000000000ull, std::memory_order_relaxed);
  g_withhold_item.store(withhold_decode_item, std::memory_order_relaxed);
}

const char* xkv_status_string(xkv_status status) {
  switch (status) {
    case XKV_OK: return "ok";
    case XKV_ERR_INVALID_ARG: return "invalid argument";
    case XKV_ERR_UNSUPPORTED: return "unsupported shape";
    case XKV_ERR_WORKSPACE: return "workspace too small";
    case XKV_ERR_BUDGET: return "budget out of range";
    case XKV_ERR_CUDA: return "CUDA call failed";
    case XKV_ERR_TIMEOUT: return "bounded device wait expired";
    case XKV_ERR_CAPACITY: return "sequence outgrew its page table";
    default: return "unknown status";
  }
}

int32_t xkv_version(void) { return 100; }

// ---------------------------------------------------------------------------------------------
// Algorithm 1 (adaptive allocation).  Instead of scanning the wait list for its maximum on every
// iteration, the wait values sit in a max-heap ordered by (value, lower layer index first); the
// sequence of grants is the same as the listing's.
// ---------------------------------------------------------------------------------------------
namespace {

struct WaitEntry {
  double value;
  int layer;
  bool operator<(const WaitEntry& o) const {   // priority_queue pops the largest
    if (value != o.value) return value < o.value;
    return layer > o.layer;
  }
};

// A curve as the solver reads it: the caller's floats as they are (every float is a double, so nothing is copied or
// converted up front), or doubles computed here (a batch mean).
struct Curve {
  const float* f = nullptr;
  const double* d = nullptr;
  int64_t n = 0;
  double operator[](int64_t j) const { return f != nullptr ? (double)f[j] : d[j]; }
  int64_t size() const { return n; }
  // true if no value over [a, b) is larger than its predecessor (a plain reduction, so that it vectorises)
  bool non_increasing(int64_t a, int64_t b) const {
    int bad = 0;
    if (f != nullptr) {
      for (int64_t j = a; j < b; ++j) bad |= f[j] > f[j - 1];
    } else {
      for (int64_t j = a; j < b; ++j) bad |= d[j] > d[j - 1];
    }
    return bad == 0;
  }
};

// Order-preserving map of a double onto an unsigned integer (larger value -> larger key).
inline uint64_t ordered_key(double v) {
  uint64_t u;
  std::memcpy(&u, &v, sizeof(u));
  return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

// Total-budget mode when every curve is non-increasing over the positions still open (what sorted scores
// give): the listing then grants the open positions in the order (value descending, layer ascending,
// position ascending), so its result is "every position above the R-th largest value, and positions equal
// to it from the lowest layers first".  The R-th largest value is found by bisecting the value's bit pattern,
// counting per layer with a binary search: the same budgets as the heap below, without its R pops.
bool solve_sorted_total(const std::vector<Curve>& curve, const std::vector<int64_t>& cap, int64_t total,
                        int n_min, int32_t* budgets, double* r_avg, xkv_status* status) {
  const int L = (int)curve.size();
  std::vector<int64_t> lo(L), hi(L);           // open positions of layer l: [lo, hi); beyond the curve the gain is 0
  int64_t used = 0, open = 0;
  for (int l = 0; l < L; ++l) {
    lo[l] = n_min < cap[l] ? n_min : cap[l];
    hi[l] = cap[l];
    used += lo[l];
    open += hi[l] - lo[l];
    const int64_t n = (int64_t)curve[l].size();
    if (!curve[l].non_increasing(lo[l] + 1, hi[l] < n ? hi[l] : n)) return false;
    if (hi[l] > n && n > lo[l] && curve[l][n - 1] < 0.0) return false;       // the implicit zeros would rise again
  }
  if (total < used || total - used > open) {
    *status = XKV_ERR_BUDGET;
    return true;
  }
  const int64_t R = total - used;
  auto value_at = [&](int l, int64_t j) -> double { return j < (int64_t)curve[l].size() ? curve[l][j] : 0.0; };
  // Open positions of layer l whose key is >= key (the curve is non-increasing, so they form a prefix), given that
  // the answer lies in [a, b].
  auto count_ge = [&](int l, uint64_t key, int64_t a, int64_t b) -> int64_t {
    a += lo[l];
    b += lo[l];
    while (a < b) {
      const int64_t mid = (a + b) >> 1;
      if (ordered_key(value_at(l, mid)) >= key) a = mid + 1;
      else b = mid;
    }
    return a - lo[l];
  };
  std::vector<int64_t> alloc(lo);
  if (R > 0) {
    // Largest key with count(key) >= R, by bisection of the key.  The counts are monotone in the key, so every layer
    // keeps a bracket [below[l], above[l]] = [count at khi + 1, count at klo] that each step narrows: the 64 steps
    // together cost one binary search per layer plus a few probes a step.
    uint64_t klo = 0, khi = ~0ull;
    std::vector<int64_t> below(L, 0), above(L), at_mid(L);
    for (int l = 0; l < L; ++l) above[l] = hi[l] - lo[l];
    while (klo < khi) {
      const uint64_t mid = klo + ((khi - klo) >> 1) + 1;
      int64_t c = 0;
      for (int l = 0; l < L; ++l) {
        at_mid[l] = count_ge(l, mid, below[l], above[l]);
        c += at_mid[l];
      }
      if (c >= R) {
        klo = mid;
        above.swap(at_mid);
      } else {
        khi = mid - 1;
        below.swap(at_mid);
      }
    }
    int64_t left = R;
    for (int l = 0; l < L; ++l) {                // everything strictly above the threshold value
      const int64_t n_above = klo == ~0ull ? 0 : count_ge(l, klo + 1, 0, hi[l] - lo[l]);
      alloc[l] += n_above;
      left -= n_above;
    }
    for (int l = 0; l < L && left > 0; ++l) {    // ties at the threshold: lowest layers first
      const int64_t ties = count_ge(l, klo, 0, hi[l] - lo[l]) - (alloc[l] - lo[l]);
      const int64_t take = ties < left ? ties : left;
      alloc[l] += take;
      left -= take;
    }
  }
  double r_total = 0.0;
  for (int l = 0; l < L; ++l) {
    for (int64_t j = 0; j < alloc[l]; ++j) r_total += value_at(l, j);
    budgets[l] = (int32_t)alloc[l];
  }
  if (r_avg != nullptr) *r_avg = r_total / L;
  *status = XKV_OK;
  return true;
}

xkv_status solve_one(const std::vector<Curve>& curve, const std::vector<int64_t>& cap,
                     int64_t total, double r_target, int n_min, int32_t* budgets, double* r_avg) {
  const int L = (int)curve.size();
  if (total >= 0) {
    xkv_status st = XKV_OK;
    if (solve_sorted_total(curve, cap, total, n_min, budgets, r_avg, &st)) return st;
  }
  std::vector<int64_t> alloc(L);
  double r_total = 0.0;
  int64_t used = 0;
  auto gain_at = [&](int l, int64_t pos) -> double {
    return pos < (int64_t)curve[l].size() ? curve[l][pos] : 0.0;
  };
  std::priority_queue<WaitEntry> wait;
  for (int l = 0; l < L; ++l) {
    alloc[l] = n_min < cap[l] ? n_min : cap[l];
    for (int64_t j = 0; j < alloc[l]; ++j) r_total += gain_at(l, j);
    used += alloc[l];
    if (alloc[l] < cap[l]) wait.push({gain_at(l, alloc[l]), l});
  }
  auto grant = [&]() -> bool {
    if (wait.empty()) return false;
    const WaitEntry top = wait.top();
    wait.pop();
    alloc[top.layer] += 1;
    r_total += top.value;
    used += 1;
    if (alloc[top.layer] < cap[top.layer]) wait.push({gain_at(top.layer, alloc[top.layer]), top.layer});
    return true;
  };
  if (total >= 0) {
    if (total < used) return XKV_ERR_BUDGET;
    while (used < total)
      if (!grant()) return XKV_ERR_BUDGET;
  } else {
    if (!(r_target > 0.0) || r_target > 1.0 + 1e-12) return XKV_ERR_BUDGET;
    while (r_total / L < r_target)
      if (!grant()) return XKV_ERR_BUDGET;
  }
  for (int l = 0; l < L; ++l) budgets[l] = (int32_t)alloc[l];
  if (r_avg != nullptr) *r_avg = r_total / L;
  return XKV_OK;
}

}  // namespace

xkv_status xkv_alloc_budgets(const float* gains, int32_t n_layers, int32_t batch, int32_t curve_len,
                             const int32_t* prefix_len, int32_t per_sequence, int64_t total, double r_target,
                             int32_t n_min, int32_t n_max, int32_t* budgets, double* r_avg) {
  if (gains == nullptr || prefix_len == nullptr || budgets == nullptr) return XKV_ERR_INVALID_ARG;
  if (n_layers <= 0 || batch <= 0 || curve_len <= 0 || n_min < 0) return XKV_ERR_INVALID_ARG;
  if (per_sequence != 0 && per_sequence != 1) return XKV_ERR_INVALID_ARG;
  if (n_max > 0 && n_min > n_max) return XKV_ERR_BUDGET;
  int64_t max_prefix = 0;
  for (int b = 0; b < batch; ++b) {
    if (prefix_len[b] < 0) return XKV_ERR_INVALID_ARG;
    if (prefix_len[b] > max_prefix) max_prefix = prefix_len[b];
  }
  const size_t lstride = (size_t)batch * curve_len;
  std::vector<Curve> curve(n_layers);
  if (!per_sequence) {
    std::vector<std::vector<double>> mean;
    if (batch == 1) {
      // one curve per layer already (the session averages over the batch on the device): read it in place
      for (int l = 0; l < n_layers; ++l) {
        curve[l].f = gains + l * lstride;
        curve[l].n = curve_len;
      }
    } else {
      mean.assign(n_layers, std::vector<double>(curve_len, 0.0));
      auto mean_layers = [&](int l0, int l1) {
        for (int l = l0; l < l1; ++l) {
          double* c = mean[l].data();
          for (int b = 0; b < batch; ++b) {
            const float* g = gains + l * lstride + (size_t)b * curve_len;
            for (int j = 0; j < curve_len; ++j) c[j] += (double)g[j];
          }
          for (int j = 0; j < curve_len; ++j) c[j] /= batch;
        }
      };
      // the batch mean reads every curve once: spread the layers over a few threads when that is megabytes
      int n_threads = (int)std::min<size_t>(8, (size_t)n_layers * lstride / (4u << 20));
      const int hw = (int)std::thread::hardware_concurrency();
      if (hw > 0 && n_threads > hw) n_threads = hw;
      if (n_threads > n_layers) n_threads = n_layers;
      if (n_threads <= 1) {
        mean_layers(0, n_layers);
      } else {
        std::vector<std::thread> pool;
        for (int i = 0; i < n_threads; ++i)
          pool.emplace_back(mean_layers, (int)((int64_t)n_layers * i / n_threads),
                            (int)((int64_t)n_layers * (i + 1) / n_threads));
        for (auto& th : pool) th.join();
      }
      for (int l = 0; l < n_layers; ++l) {
        curve[l].d = mean[l].data();
        curve[l].n = curve_len;
      }
    }
    int64_t c = max_prefix;
    if (n_max > 0 && n_max < c) c = n_max;
    std::vector<int64_t> cap(n_layers, c);
    return solve_one(curve, cap, total, r_target, n_min, budgets, r_avg);
  }
  for (int b = 0; b < batch; ++b) {
    for (int l = 0; l < n_layers; ++l) {
      curve[l].f = gains + l * lstride + (size_t)b * curve_len;
      curve[l].n = curve_len;
    }
    int64_t c = prefix_len[b];
    if (n_max > 0 && n_max < c) c = n_max;
    std::vector<int64_t> cap(n_layers, c);
    xkv_status s = solve_one(curve, cap, total, r_target, n_min, budgets + (size_t)b * n_layers,
                             r_avg != nullptr ? r_avg + b : nullptr);
    if (s != XKV_OK) return s;
  }
  return XKV_OK;
}

xkv_status xkv_average_budgets(const int32_t* lists, int32_t n_tasks, int32_t n_layers, int32_t* out) {
  if (lists == nullptr || out == nullptr || n_tasks <= 0 || n_layers <= 0) return XKV_ERR_INVALID_ARG;
  std::vector<int64_t> sums(n_layers, 0);
  int64_t total = 0;
  for (int t = 0; t < n_tasks; ++t)
    for (int l = 0; l < n_layers; ++l) {
      const int32_t v = lists[(size_t)t * n_layers + l];
      if (v < 0) return XKV_ERR_INVALID_ARG;
      sums[l] += v;
      total += v;
    }
  const int64_t n = n_tasks;
  const int64_t target = (2 * total + n) / (2 * n);          // mean of the recorded totals, rounded half up
  int64_t given = 0;
  std::vector<std::pair<int64_t, int>> frac(n_layers);        // (remainder of the division by n, layer)
  for (int l = 0; l < n_layers; ++l) {
    out[l] = (int32_t)(sums[l] / n);
    given += out[l];
    frac[l] = {sums[l] % n, l};
  }
  std::stable_sort(frac.begin(), frac.end(),
                   [](const std::pair<int64_t, int>& a, const std::pair<int64_t, int>& b) { return a.first > b.first; });
  for (int64_t i = 0; i < target - given && i < n_layers; ++i) out[frac[(size_t)i].second] += 1;
  return XKV_OK;
}

}  // extern "C"
