// xkv_select_compact: TopK and EvictByIndex of one layer (Alg. 2 steps 5-7).
//
//   select_kernel  one CTA per (sequence, KV head).  The k-th largest score is read from the
//                  descending sort the scoring pass produced; one ordered sweep over the prefix then
//                  keeps every position above it and the lowest positions equal to it until k are
//                  kept (ties go to the lower position), which yields the kept positions already in
//                  ascending order.  The window positions follow.
//   select_count_kernel, select_chunk_kernel
//                  the same selection for prefixes longer than one sweep step (4096 positions): one CTA per
//                  (unit, 4096-position chunk) first counts the scores above and equal to the threshold, then
//                  every chunk finds its place from the counts of the chunks before it and writes its kept
//                  positions, so a long sequence is swept by many CTAs at once instead of one.
//   gather_kernel  16-byte vectorised copy of the kept K and V rows (256-byte rows for d = 128) into
//                  the layer's cache pages; pure data movement, HBM-bound.
#include "common.cuh"
#include "ops.h"

namespace xkv {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelItems = 4;                 // consecutive positions per thread and sweep step
constexpr int kGatherThreads = 256;
constexpr int kGatherRows = 64;              // cache rows per gather CTA

struct SelectParams {
  const float* scores;
  const float* sorted;
  const int32_t* cu_seqlens;
  const int32_t* budget_dev;   // [B] per sequence, [B][Hkv] per head, else null
  int32_t budget;              // shared budget otherwise
  int32_t head_level;          // 1: budgets, cache lengths and page lists are per (sequence, KV head)
  int32_t* sel;                // [B][Hkv][sel_stride]
  int32_t sel_stride;
  int32_t* seq_lens_layer;     // seq_lens + layer*B (layer*B*Hkv when head_level)
  const int32_t* block_table_layer;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  __nv_bfloat16* k_pages;
  __nv_bfloat16* v_pages;
  float* k_scales;             // 8-bit caches only: one scale per cached row
  float* v_scales;
  int32_t kv_format;
  int64_t total_tokens, stride_token, stride_head;
  int32_t batch, n_kv_heads, head_dim, window, page_size, max_pages_per_seq, n_pages;
  int2* counts;                // [units][n_chunks] scores above / equal to the threshold per chunk (chunked path)
  int32_t n_chunks, max_seqlen;
  WorkspaceHeader* hdr;
};

__device__ __forceinline__ void unit_shape(const SelectParams& p, int b, int g, int* cu, int* t, int* P, int* kb) {
  *cu = p.cu_seqlens[b];
  *t = min(p.cu_seqlens[b + 1] - *cu, p.max_seqlen);     // a longer prompt is cut to the bound the buffers were sized for
  *P = max(*t - p.window, 0);
  const int budget = p.budget_dev == nullptr ? p.budget
                                             : (p.head_level ? p.budget_dev[b * p.n_kv_heads + g] : p.budget_dev[b]);
  *kb = min(budget, *P);
}

// Index of the cache (its seq_lens entry and page list) that holds KV head g of sequence b, and whether this
// (b, g) is the one that writes the entry: with head-level budgets every head has a cache of its own.
__device__ __forceinline__ int cache_index(const SelectParams& p, int b, int g) {
  return p.head_level ? b * p.n_kv_heads + g : b;
}
__device__ __forceinline__ bool writes_len(const SelectParams& p, int g) { return p.head_level || g == 0; }

// Exclusive block scan of one int per thread (kSelThreads threads); returns the exclusive prefix
// and writes the block total to *total.
__device__ __forceinline__ int block_scan_excl(int v, int* s_warp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += u;
  }
  __syncthreads();            // s_warp may still be read from the previous scan
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = s_warp[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += u;
    }
    s_warp[lane] = winc - w;
    if (lane == 31) s_warp[32] = winc;
  }
  __syncthreads();
  *total = s_warp[32];
  return s_warp[warp] + incl - v;
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectParams p) {
  __shared__ int s_warp[33];
  const int b = blockIdx.x / p.n_kv_heads, g = blockIdx.x % p.n_kv_heads;
  int cu, t, P, kb;
  unit_shape(p, b, g, &cu, &t, &P, &kb);
  const int n_keep = kb + (t - P);
  const bool fits = n_keep <= p.max_pages_per_seq * p.page_size;
  if (threadIdx.x == 0 && writes_len(p, g)) {
    p.seq_lens_layer[cache_index(p, b, g)] = fits ? n_keep : 0;
    if (!fits) record_status(p.hdr, XKV_ERR_CAPACITY);
  }
  if (!fits) return;
  int32_t* sel = p.sel + ((size_t)b * p.n_kv_heads + g) * p.sel_stride;
  for (int i = threadIdx.x; i < t - P; i += kSelThreads) sel[kb + i] = P + i;   // window positions
  if (kb == 0) return;
  if (kb == P) {
    for (int i = threadIdx.x; i < P; i += kSelThreads) sel[i] = i;
    return;
  }
  const float* w = p.scores + (size_t)g * p.total_tokens + cu;
  const float* srt = p.sorted + (size_t)g * p.total_tokens + cu;
  const float thr = srt[kb - 1];
  // number of scores strictly above thr (counted over the prefix; the sorted copy only supplies thr)
  int n_gt = 0;
  for (int c = threadIdx.x; c < P; c += kSelThreads) n_gt += w[c] > thr ? 1 : 0;
  int count_gt;
  block_scan_excl(n_gt, s_warp, &count_gt);
  const int eq_needed = kb - count_gt;

  int carry_eq = 0, carry_sel = 0;
  for (int base = 0; base < P; base += kSelThreads * kSelItems) {
    const int c0 = base + threadIdx.x * kSelItems;
    float x[kSelItems];
    int n_eq = 0;
#pragma unroll
    for (int i = 0; i < kSelItems; ++i) {
      x[i] = (c0 + i < P) ? w[c0 + i] : -1.f;
      n_eq += (x[i] == thr) ? 1 : 0;
    }
    int tot_eq;
    int eq_before = carry_eq + block_scan_excl(n_eq, s_warp, &tot_eq);
    bool keep[kSelItems];
    int n_sel = 0;
#pragma unroll
    for (int i = 0; i < kSelItems; ++i) {
      const bool is_eq = x[i] == thr;
      keep[i] = (c0 + i < P) && (x[i] > thr || (is_eq && eq_before < eq_needed));
      eq_before += is_eq ? 1 : 0;
      n_sel += keep[i] ? 1 : 0;
    }
    int tot_sel;
    int dst = carry_sel + block_scan_excl(n_sel, s_warp, &tot_sel);
#pragma unroll
    for (int i = 0; i < kSelItems; ++i)
      if (keep[i] && dst < kb) sel[dst++] = c0 + i;
    carry_eq += tot_eq;
    carry_sel += tot_sel;
  }
}

constexpr int kSelChunk = kSelThreads * kSelItems;     // positions one CTA sweeps in the chunked path

// grid = (units, n_chunks): scores of the chunk above and equal to the unit's threshold.
__global__ void __launch_bounds__(kSelThreads) select_count_kernel(SelectParams p) {
  __shared__ int s_warp[33];
  const int unit = blockIdx.x, chunk = blockIdx.y;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  int cu, t, P, kb;
  unit_shape(p, b, g, &cu, &t, &P, &kb);
  if (kb == 0 || kb == P || chunk * kSelChunk >= P) return;      // nothing to count: no selection by score
  const float* w = p.scores + (size_t)g * p.total_tokens + cu;
  const float thr = p.sorted[(size_t)g * p.total_tokens + cu + kb - 1];
  const int c0 = chunk * kSelChunk + threadIdx.x * kSelItems;
  int n_gt = 0, n_eq = 0;
#pragma unroll
  for (int i = 0; i < kSelItems; ++i) {
    const float x = (c0 + i < P) ? w[c0 + i] : -1.f;
    n_gt += x > thr ? 1 : 0;
    n_eq += x == thr ? 1 : 0;
  }
  int tot;
  block_scan_excl(n_gt | (n_eq << 16), s_warp, &tot);           // at most 4096 of either: 16 bits each
  if (threadIdx.x == 0) p.counts[(size_t)unit * p.n_chunks + chunk] = make_int2(tot & 0xffff, tot >> 16);
}

// grid = (units, n_chunks): the kept positions of the chunk, placed after those of the chunks before it.
__global__ void __launch_bounds__(kSelThreads) select_chunk_kernel(SelectParams p) {
  __shared__ int s_warp[33];
  __shared__ int s_base[3];
  const int unit = blockIdx.x, chunk = blockIdx.y;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  int cu, t, P, kb;
  unit_shape(p, b, g, &cu, &t, &P, &kb);
  const int n_keep = kb + (t - P);
  const bool fits = n_keep <= p.max_pages_per_seq * p.page_size;
  if (chunk == 0 && threadIdx.x == 0 && writes_len(p, g)) {
    p.seq_lens_layer[cache_index(p, b, g)] = fits ? n_keep : 0;
    if (!fits) record_status(p.hdr, XKV_ERR_CAPACITY);
  }
  if (!fits) return;
  int32_t* sel = p.sel + (size_t)unit * p.sel_stride;
  if (chunk == 0)
    for (int i = threadIdx.x; i < t - P; i += kSelThreads) sel[kb + i] = P + i;   // window positions
  const int begin = chunk * kSelChunk;
  if (kb == 0 || begin >= P) return;
  const int c0 = begin + threadIdx.x * kSelItems;
  if (kb == P) {
#pragma unroll
    for (int i = 0; i < kSelItems; ++i)
      if (c0 + i < P) sel[c0 + i] = c0 + i;
    return;
  }
  // totals over the unit and over the chunks before this one
  if (threadIdx.x < 32) {
    int gt_all = 0, gt_before = 0, eq_before = 0;
    const int n_ch = (P + kSelChunk - 1) / kSelChunk;
    for (int c = threadIdx.x; c < n_ch; c += 32) {
      const int2 v = __ldcg(&p.counts[(size_t)unit * p.n_chunks + c]);
      gt_all += v.x;
      if (c < chunk) {
        gt_before += v.x;
        eq_before += v.y;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      gt_all += __shfl_xor_sync(0xffffffffu, gt_all, o);
      gt_before += __shfl_xor_sync(0xffffffffu, gt_before, o);
      eq_before += __shfl_xor_sync(0xffffffffu, eq_before, o);
    }
    if (threadIdx.x == 0) {
      s_base[0] = kb - gt_all;        // positions equal to the threshold that are kept (the lowest ones)
      s_base[1] = gt_before;
      s_base[2] = eq_before;
    }
  }
  __syncthreads();
  const int eq_needed = s_base[0];
  const int eq_start = s_base[2];
  const int dst_start = s_base[1] + min(eq_start, eq_needed);
  const float* w = p.scores + (size_t)g * p.total_tokens + cu;
  const float thr = p.sorted[(size_t)g * p.total_tokens + cu + kb - 1];
  float x[kSelItems];
  int n_eq = 0;
#pragma unroll
  for (int i = 0; i < kSelItems; ++i) {
    x[i] = (c0 + i < P) ? w[c0 + i] : -1.f;
    n_eq += (x[i] == thr) ? 1 : 0;
  }
  int tot_eq;
  int eq_before = eq_start + block_scan_excl(n_eq, s_warp, &tot_eq);
  bool keep[kSelItems];
  int n_sel = 0;
#pragma unroll
  for (int i = 0; i < kSelItems; ++i) {
    const bool is_eq = x[i] == thr;
    keep[i] = (c0 + i < P) && (x[i] > thr || (is_eq && eq_before < eq_needed));
    eq_before += is_eq ? 1 : 0;
    n_sel += keep[i] ? 1 : 0;
  }
  int tot_sel;
  int dst = dst_start + block_scan_excl(n_sel, s_warp, &tot_sel);
#pragma unroll
  for (int i = 0; i < kSelItems; ++i)
    if (keep[i] && dst < kb) sel[dst++] = c0 + i;
}

__global__ void __launch_bounds__(kGatherThreads) gather_kernel(SelectParams p) {
  const int unit = blockIdx.x;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  int cu, t, P, kb;
  unit_shape(p, b, g, &cu, &t, &P, &kb);
  const int n_keep = kb + (t - P);
  if (n_keep > p.max_pages_per_seq * p.page_size) return;
  const int row0 = blockIdx.y * kGatherRows;
  if (row0 >= n_keep) return;
  const int32_t* sel = p.sel + (size_t)unit * p.sel_stride;
  const int32_t* bt = p.block_table_layer + (size_t)cache_index(p, b, g) * p.max_pages_per_seq;
  const int page_heads = p.head_level ? 1 : p.n_kv_heads, page_head = p.head_level ? 0 : g;
  const int lanes_per_row = p.head_dim / 8;                   // 16-byte lanes per row
  const int rows_per_pass = kGatherThreads / lanes_per_row;
  const int lr = threadIdx.x / lanes_per_row, lc = threadIdx.x % lanes_per_row;
  for (int r = row0 + lr; r < min(row0 + kGatherRows, n_keep); r += rows_per_pass) {
    const int pos = sel[r];
    int page = bt[r / p.page_size];
    if (page < 0 || page >= p.n_pages) {
      if (lc == 0) record_status(p.hdr, XKV_ERR_CAPACITY);
      continue;
    }
    const size_t src = (size_t)(cu + pos) * p.stride_token + (size_t)g * p.stride_head + lc * 8;
    const size_t slot = ((size_t)page * page_heads + page_head) * p.page_size + r % p.page_size;
    const size_t dst = slot * p.head_dim + lc * 8;
    const uint4 kv = __ldg(reinterpret_cast<const uint4*>(p.k + src));
    const uint4 vv = __ldg(reinterpret_cast<const uint4*>(p.v + src));
    if (p.kv_format == XKV_KV_INT8) {
      // the row's lanes (consecutive lanes of the warp) agree on its scale; a lane stores its eight codes
      float x[8], ks, vs;
      bf16x8_to_f32(kv, x);
      const uint2 kc = quantize_row_piece(x, lanes_per_row, &ks);
      bf16x8_to_f32(vv, x);
      const uint2 vc = quantize_row_piece(x, lanes_per_row, &vs);
      *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(p.k_pages) + dst) = kc;
      *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(p.v_pages) + dst) = vc;
      if (lc == 0) {
        p.k_scales[slot] = ks;
        p.v_scales[slot] = vs;
      }
    } else {
      *reinterpret_cast<uint4*>(p.k_pages + dst) = kv;
      *reinterpret_cast<uint4*>(p.v_pages + dst) = vv;
    }
  }
}

// block_table[l][b][i] = first_page[l][b] + i for i < n_pages_lb[l][b], else 0.  grid = (L*B), any block size.
__global__ void block_table_kernel(const int32_t* first_page, const int32_t* n_pages_lb, int32_t* block_table,
                                   int max_pages_per_seq) {
  const int lb = blockIdx.x;
  const int first = first_page[lb], n = n_pages_lb[lb];
  int32_t* row = block_table + (size_t)lb * max_pages_per_seq;
  for (int i = threadIdx.x; i < max_pages_per_seq; i += blockDim.x) row[i] = i < n ? first + i : 0;
}

// out[l][j] = scale * sum over b of gains[l][b][j], summed in the order of b in double precision (the same
// result on every run).  grid = (tiles of 256 ranks, L).
__global__ void batch_curves_kernel(const float* gains, int batch, int curve_len, double scale, float* out) {
  const int l = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= curve_len) return;
  const float* g = gains + (size_t)l * batch * curve_len + j;
  double acc = 0.0;
  for (int b = 0; b < batch; ++b) acc += (double)g[(size_t)b * curve_len];
  out[(size_t)l * curve_len + j] = (float)(acc * scale);
}

// out[g][b][j] = sorted[g][cu_b + j] / sum over the prefix of scores[g][cu_b + c] (0 for j >= P_b).  grid = B*Hkv.
// The sum runs in double precision in a fixed order (per-thread strided partial sums, then a tree), so the result
// is the same on every run.
__global__ void __launch_bounds__(1024) head_curves_kernel(const float* scores, const float* sorted,
                                                           const int32_t* cu_seqlens, int64_t total_tokens,
                                                           int max_seqlen, int window, int batch, int n_kv_heads,
                                                           int curve_len, float* out) {
  __shared__ double s_sum[1024];
  const int b = blockIdx.x / n_kv_heads, g = blockIdx.x % n_kv_heads;
  const int cu = cu_seqlens[b];
  const int t = min(cu_seqlens[b + 1] - cu, max_seqlen);
  const int P = max(t - window, 0);
  const float* w = scores + (size_t)g * total_tokens + cu;
  double acc = 0.0;
  for (int c = threadIdx.x; c < P; c += 1024) acc += (double)w[c];
  s_sum[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) s_sum[threadIdx.x] += s_sum[threadIdx.x + o];
    __syncthreads();
  }
  const double total = s_sum[0];
  const double inv = total > 0.0 ? 1.0 / total : 0.0;
  const float* srt = sorted + (size_t)g * total_tokens + cu;
  float* o = out + ((size_t)g * batch + b) * curve_len;
  for (int j = threadIdx.x; j < curve_len; j += 1024) o[j] = j < P ? (float)((double)srt[j] * inv) : 0.f;
}

struct SelectLayout {
  size_t budget, sel, counts, total;
  int sel_stride, n_chunks;
};

void select_layout(const xkv_dims* d, int max_seqlen, SelectLayout* L) {
  size_t off = kHeaderBytes;
  L->budget = off; off = align_up(off + (size_t)d->batch * d->n_kv_heads * 4, 256);
  L->sel_stride = (max_seqlen + 3) / 4 * 4;
  L->sel = off;    off = align_up(off + (size_t)d->batch * d->n_kv_heads * L->sel_stride * 4, 256);
  L->n_chunks = (max_seqlen + kSelChunk - 1) / kSelChunk;
  L->counts = off; off = align_up(off + (size_t)d->batch * d->n_kv_heads * L->n_chunks * 8, 256);
  L->total = off;
}

}  // namespace

xkv_status build_block_table(const int32_t* first_page, const int32_t* n_pages_lb, int n_lb, int32_t* block_table,
                             int max_pages_per_seq, cudaStream_t st) {
  block_table_kernel<<<n_lb, 128, 0, st>>>(first_page, n_pages_lb, block_table, max_pages_per_seq);
  count_launch();
  return check_launch();
}

xkv_status batch_curves(const float* gains, int n_layers, int batch, int curve_len, double scale, float* out,
                        cudaStream_t st) {
  batch_curves_kernel<<<dim3((curve_len + 255) / 256, n_layers), 256, 0, st>>>(gains, batch, curve_len, scale, out);
  count_launch();
  return check_launch();
}

xkv_status head_curves(const xkv_dims* d, const float* scores, const float* sorted, const int32_t* cu_seqlens,
                       int64_t total_tokens, int max_seqlen, float* out, int curve_len, cudaStream_t st) {
  head_curves_kernel<<<d->batch * d->n_kv_heads, 1024, 0, st>>>(scores, sorted, cu_seqlens, total_tokens, max_seqlen,
                                                                d->window, d->batch, d->n_kv_heads, curve_len, out);
  count_launch();
  return check_launch();
}

size_t select_workspace_bytes(const xkv_dims* d, int max_seqlen, int64_t total_tokens) {
  (void)total_tokens;
  SelectLayout L;
  select_layout(d, max_seqlen, &L);
  return L.total;
}

xkv_status select_compact(const xkv_dims* d, int layer, const int32_t* budget, int per_sequence,
                          const float* scores, const float* sorted, const void* k, const void* v,
                          const int32_t* cu_seqlens, int64_t total_tokens, int max_seqlen, const xkv_cache* c,
                          int32_t* sel, int sel_stride, void* workspace, size_t workspace_bytes, cudaStream_t st) {
  SelectLayout L;
  select_layout(d, max_seqlen, &L);
  if (workspace_bytes < L.total) return XKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);

  const int head_level = per_sequence == XKV_BUDGET_PER_HEAD ? 1 : 0;
  const int n_budgets = head_level ? d->batch * d->n_kv_heads : (per_sequence ? d->batch : 1);
  const int n_caches = head_level ? d->batch * d->n_kv_heads : d->batch;       // caches of one layer
  int max_budget = 0;
  for (int i = 0; i < n_budgets; ++i) max_budget = budget[i] > max_budget ? budget[i] : max_budget;
  const int64_t max_keep64 = (int64_t)max_budget + d->window;
  const int max_keep = (int)(max_keep64 < max_seqlen ? max_keep64 : max_seqlen);
  if (sel != nullptr && sel_stride < max_keep) return XKV_ERR_INVALID_ARG;

  SelectParams p;
  p.scores = scores;
  p.sorted = sorted;
  p.cu_seqlens = cu_seqlens;
  p.budget_dev = nullptr;
  p.budget = budget[0];
  p.sel = sel != nullptr ? sel : reinterpret_cast<int32_t*>(ws + L.sel);
  p.sel_stride = sel != nullptr ? sel_stride : L.sel_stride;
  p.head_level = head_level;
  p.seq_lens_layer = c->seq_lens + (size_t)layer * n_caches;
  p.block_table_layer = c->block_table + (size_t)layer * n_caches * c->max_pages_per_seq;
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.v = static_cast<const __nv_bfloat16*>(v);
  p.k_pages = static_cast<__nv_bfloat16*>(c->k_pages);
  p.v_pages = static_cast<__nv_bfloat16*>(c->v_pages);
  p.k_scales = c->k_scales;
  p.v_scales = c->v_scales;
  p.kv_format = c->kv_format;
  p.total_tokens = total_tokens;
  p.stride_token = d->kv_stride_token;
  p.stride_head = d->kv_stride_head;
  p.batch = d->batch;
  p.n_kv_heads = d->n_kv_heads;
  p.head_dim = d->head_dim;
  p.window = d->window;
  p.page_size = c->page_size;
  p.max_pages_per_seq = c->max_pages_per_seq;
  p.n_pages = c->n_pages;
  p.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  p.counts = reinterpret_cast<int2*>(ws + L.counts);
  p.n_chunks = L.n_chunks;
  p.max_seqlen = max_seqlen;

  if (cudaMemsetAsync(ws + 4, 0, kHeaderBytes - 4, st) != cudaSuccess) return XKV_ERR_CUDA;   // the status word stays
  if (per_sequence) {
    if (cudaMemcpyAsync(ws + L.budget, budget, (size_t)n_budgets * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return XKV_ERR_CUDA;
    p.budget_dev = reinterpret_cast<const int32_t*>(ws + L.budget);
  }
  const int n_units = d->batch * d->n_kv_heads;
  xkv_status s;
  if (L.n_chunks <= 1) {
    select_kernel<<<n_units, kSelThreads, 0, st>>>(p);
    count_launch();
    s = check_launch();
  } else {
    select_count_kernel<<<dim3(n_units, L.n_chunks), kSelThreads, 0, st>>>(p);
    count_launch();
    s = check_launch();
    if (s != XKV_OK) return s;
    select_chunk_kernel<<<dim3(n_units, L.n_chunks), kSelThreads, 0, st>>>(p);
    count_launch();
    s = check_launch();
  }
  if (s != XKV_OK) return s;
  if (max_keep > 0) {
    dim3 grid(n_units, (max_keep + kGatherRows - 1) / kGatherRows);
    gather_kernel<<<grid, kGatherThreads, 0, st>>>(p);
    count_launch();
    s = check_launch();
  }
  return s;
}

}  // namespace xkv
