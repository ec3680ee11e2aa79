// C ABI of libxkv: host-side argument validation, workspace sizing, status plumbing, and the
// host-only budget solver (Algorithm 1).  Device work is in xkv_score.cu, xkv_select.cu and
// xkv_decode.cu.
#include <atomic>
#include <cmath>
#include <queue>
#include <utility>
#include <vector>

#include "common.cuh"
#include "ops.h"

namespace xkv {

static std::atomic<int64_t> g_launches{0};

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

xkv_status check_launch() { return cudaGetLastError() == cudaSuccess ? XKV_OK : XKV_ERR_CUDA; }

int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

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
  if (rows % 16 != 0 || rows > 256) return XKV_ERR_UNSUPPORTED;
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
  if (per_sequence != 0 && per_sequence != 1) return XKV_ERR_INVALID_ARG;
  int32_t max_budget = 0;
  for (int i = 0; i < (per_sequence ? dims->batch : 1); ++i) {
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
    case XKV_OP_DECODE_ATTN:
      if (check_dims(dims) != XKV_OK || n_layers <= 0 || max_cache_len < 0 || chunk_rows < 0 ||
          chunk_rows % 64 != 0)
        return 0;
      return decode_workspace_bytes(dims, n_layers, max_cache_len, chunk_rows);
    default:
      return 0;
  }
}

xkv_status xkv_read_device_status(const void* workspace, void* stream) {
  if (workspace == nullptr) return XKV_ERR_INVALID_ARG;
  int32_t status = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&status, workspace, sizeof(status), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return XKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return XKV_ERR_CUDA;
  return status;
}

void xkv_profile_events(void* start, void* stop) {
  set_profile_events(static_cast<cudaEvent_t>(start), static_cast<cudaEvent_t>(stop));
}

int64_t xkv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

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

xkv_status solve_one(const std::vector<std::vector<double>>& curve, const std::vector<int64_t>& cap,
                     int64_t total, double r_target, int n_min, int32_t* budgets, double* r_avg) {
  const int L = (int)curve.size();
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
  if (!per_sequence) {
    std::vector<std::vector<double>> curve(n_layers, std::vector<double>(curve_len, 0.0));
    for (int l = 0; l < n_layers; ++l) {
      for (int b = 0; b < batch; ++b) {
        const float* g = gains + l * lstride + (size_t)b * curve_len;
        for (int j = 0; j < curve_len; ++j) curve[l][j] += (double)g[j];
      }
      for (int j = 0; j < curve_len; ++j) curve[l][j] /= batch;
    }
    int64_t c = max_prefix;
    if (n_max > 0 && n_max < c) c = n_max;
    std::vector<int64_t> cap(n_layers, c);
    return solve_one(curve, cap, total, r_target, n_min, budgets, r_avg);
  }
  for (int b = 0; b < batch; ++b) {
    std::vector<std::vector<double>> curve(n_layers, std::vector<double>(curve_len));
    for (int l = 0; l < n_layers; ++l) {
      const float* g = gains + l * lstride + (size_t)b * curve_len;
      for (int j = 0; j < curve_len; ++j) curve[l][j] = (double)g[j];
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

}  // extern "C"
