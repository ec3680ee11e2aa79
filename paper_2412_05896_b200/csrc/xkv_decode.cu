// xkv_decode_attn: generation-phase attention (Eq. 1, one query row per head) over the ragged,
// compacted per-layer caches.
//
// Kernels, in stream order:
//   decode_prepare_kernel  only for more than 2048 (layer, sequence) units: one CTA per unit stores the
//                          new K/V row of every KV head in slot seq_lens[l][b] and advances seq_lens;
//                          the last CTA to finish then cuts every (layer, sequence, KV head) cache into
//                          chunks of rows and writes the work-item table.
//   decode_attn_kernel     persistent CTAs of eight independent warps.  Up to 2048 units every CTA plans
//                          for itself from the lengths as they were before the call (chunk size from the
//                          total cached length, chunks before each unit as a prefix table in shared
//                          memory) and nothing waits for anything: the warp that owns the last chunk of a
//                          (unit, KV head) takes the new K/V row from the call's arguments, patches it
//                          into its shared-memory tile and stores it to the page; seq_lens is advanced
//                          by the last CTA to leave, so a CTA that starts late still plans from the old
//                          lengths.  A warp takes work items
//                          from a global counter and streams its item's K and V rows through its own
//                          ring of shared-memory stages: 16-row TMA tensor boxes (128-byte swizzle)
//                          that complete on an mbarrier, issued by the warp itself a few tiles ahead
//                          of where it computes, across item boundaries.  Per tile it runs online
//                          softmax with mma.sync m16n8k16, transposed: S^T = K.Q^T and O^T = V^T.P^T,
//                          the 16 keys on the M axis and the G <= 8 query heads of the group on the N
//                          axis, so no accumulator row is padding.  The softmax reference maximum is
//                          raised lazily (only when a score exceeds it by 2^8), which keeps the
//                          cross-lane reduction and the rescale out of the steady state; the scores of
//                          the next tile are computed before the softmax of the current one.  A unit
//                          with one chunk is normalised and stored by its warp; otherwise the chunk's
//                          partial (m, l, acc) go to the workspace and a ticket counts the unit's
//                          published chunks.  When the work items have run out, the warps share out
//                          the split units one query head at a time (second counter) and merge the
//                          chunks by log-sum-exp, all loads of a merge in flight together; by then
//                          most of the streaming is over, so the merges neither queue behind it nor
//                          run one after another in a single warp.
// The path is HBM-bound: 4*d bytes per cached row per KV head per step; warps never wait for each
// other, so item boundaries of one warp overlap with streaming in the others.
#include <cuda.h>

#include <cmath>
#include <mutex>

#include <atomic>

#include "common.cuh"
#include "ops.h"

namespace xkv {

namespace {

constexpr int kTileRows = 16;        // cache rows per pipeline stage = one TMA box; page_size is a multiple
constexpr int kChunkAlign = 64;      // chunk_rows granularity
constexpr int kAttnWarps = 8;
constexpr int kTargetItems = 12 * 148 * kAttnWarps;  // auto chunking aims at about this many extra work items (a dozen per warp keeps the tail short)
constexpr int kMinChunkRows = 256;
constexpr int kMaxGroup = 8;
constexpr int kFifo = 4;             // work items a warp may have fetched but not yet finished
constexpr int kPrepThreads = 256;
constexpr int kMaxPlanUnits = 2048;  // (layer, sequence) units up to which the attention kernel plans for itself

struct DecodeParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  __nv_bfloat16* out;
  float* lse;
  __nv_bfloat16* k_pages;   // uint8 codes when the cache is stored in 8 bits
  __nv_bfloat16* v_pages;
  float* k_scales;          // 8-bit caches: one fp32 scale per cached row, [n_pages][Hkv][page_size]
  float* v_scales;
  const int32_t* block_table;
  int32_t* seq_lens;
  int32_t layer_begin, n_layers, batch, n_q_heads, n_kv_heads, group;
  int32_t page_size, max_pages_per_seq, n_pages;
  int32_t chunk_rows_forced, max_items;
  int32_t fused_plan, do_append;   // fused_plan: the attention kernel plans in its own prologue and appends itself
  int32_t withhold_item;           // test hook: the merge ticket of this work item is never published (-1: none)
  float scale_log2;
  uint64_t wait_ns;                // limit of every bounded wait
  WorkspaceHeader* hdr;
  int32_t* tickets;   // [n_layers*batch*n_kv_heads]
  int2* unit_info;    // [n_layers*batch]: {first item of head 0, chunks per head}
  int32_t* multi_list;  // [n_layers*batch]: the (layer, sequence) units that were cut into several chunks
  int4* items;        // [max_items]: {unit e, kv head, row_begin, row_end}
  float* part_o;      // [max_items][G][D]
  float* part_ml;     // [max_items][G][2]
};

// Q8: the cache holds 8-bit integers and per-row scales.  The ring then holds the raw tiles as they lie in the pages:
// all K tiles first (each 1024-byte aligned, 128-byte swizzled when a row is 128 bytes), then the V tiles, then the
// scales of the K rows and of the V rows; the tensor-core fragments are formed from the bytes in registers.
template <int D, bool Q8>
struct Cfg {
  static constexpr int kHalves = D / 64;                       // 128-byte swizzled column halves
  static constexpr int kBoxBytes = kTileRows * 128;            // one half of a 16-bit K or V tile (one TMA box)
  static constexpr int kTileBytes = kHalves * kBoxBytes;
  static constexpr int kRawTileBytes = kTileRows * D;          // Q8: one tile of stored bytes
  static constexpr int kScaleBytes = kTileRows * 4;            // Q8: the scales of a tile's rows
  static constexpr int kStageBytes = Q8 ? 2 * kRawTileBytes + 2 * kScaleBytes : 2 * kTileBytes;   // K tile + V tile
  // The 8-bit path has twice the work per byte (the fragments are formed in registers) and half the bytes per
  // tile: sixteen warps with rings of as many tiles keep as many bytes in flight and hide twice the instruction latency.
  static constexpr int kWarps = Q8 ? 2 * kAttnWarps : kAttnWarps;
  static constexpr int kThreads = kWarps * 32;
  static constexpr int kStages = (D == 128) ? 3 : 6;
  static constexpr int kRingBytes = (kStages * kStageBytes + 1023) / 1024 * 1024;     // per warp
  static constexpr int kSmemBytes = 1024 + kWarps * kRingBytes + kWarps * kStages * 8 +
                                    kWarps * kFifo * 20 + (kMaxPlanUnits + 1) * 4 + kMaxPlanUnits * 2 + 64;
  // Q8 ring layout
  static constexpr int kRawVOff = kStages * kRawTileBytes;
  static constexpr int kScaleOff = 2 * kStages * kRawTileBytes;
};

// fp16 tensor-core tile for the 8-bit caches (the codes are exact in fp16).
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// Plain (untiled) bulk copy global -> shared; both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// ---------------------------------------------------------------------------------------------
// Append (optional) and plan.  grid = n_layers*batch CTAs when appending, else 1.
// ---------------------------------------------------------------------------------------------
// Rows per chunk for a launch whose caches hold `total` rows over all (layer, sequence, KV head) units.
__device__ __forceinline__ int choose_chunk(long long total, int forced) {
  if (forced > 0) return forced;
  long long c = (total + kTargetItems - 1) / kTargetItems;
  c = (c + kChunkAlign - 1) / kChunkAlign * kChunkAlign;
  if (c < kMinChunkRows) c = kMinChunkRows;
  if (c > (1 << 30)) c = 1 << 30;
  return (int)c;
}

// Stores the new K/V row of every KV head of unit e = (layer, sequence) in slot seq_lens and advances seq_lens.
__device__ __forceinline__ void append_unit(const DecodeParams& p, int D, int e, int* s_page, bool q8) {
  const int tid = threadIdx.x;
  const int l_rel = e / p.batch, b = e % p.batch;
  const int le = (p.layer_begin + l_rel) * p.batch + b;
  const int n = p.seq_lens[le];
  __syncthreads();                 // s_page may still be read for the previous unit
  if (tid == 0) {
    int page = -1;
    if (n >= 0 && n < p.max_pages_per_seq * p.page_size)
      page = p.block_table[(size_t)le * p.max_pages_per_seq + n / p.page_size];
    if (page < 0 || page >= p.n_pages) {
      page = -1;
      record_status(p.hdr, XKV_ERR_CAPACITY);
    }
    *s_page = page;
  }
  __syncthreads();
  const int page = *s_page;
  if (page >= 0) {
    const int chunks = D / 8;
    for (int idx = tid; idx < p.n_kv_heads * chunks; idx += blockDim.x) {
      const int h = idx / chunks, c = idx % chunks;
      const size_t slot = ((size_t)page * p.n_kv_heads + h) * p.page_size + n % p.page_size;
      const size_t dst = slot * D + c * 8;
      const size_t src = ((size_t)e * p.n_kv_heads + h) * D + c * 8;
      const uint4 kv = *reinterpret_cast<const uint4*>(p.k_new + src);
      const uint4 vv = *reinterpret_cast<const uint4*>(p.v_new + src);
      if (q8) {
        // a row's pieces sit on consecutive threads (D/8 of them, whole rows per warp)
        float x[8], ks, vs;
        bf16x8_to_f32(kv, x);
        const uint2 kc = quantize_row_piece(x, chunks, &ks);
        bf16x8_to_f32(vv, x);
        const uint2 vc = quantize_row_piece(x, chunks, &vs);
        *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(p.k_pages) + dst) = kc;
        *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(p.v_pages) + dst) = vc;
        if (c == 0) {
          p.k_scales[slot] = ks;
          p.v_scales[slot] = vs;
        }
      } else {
        *reinterpret_cast<uint4*>(p.k_pages + dst) = kv;
        *reinterpret_cast<uint4*>(p.v_pages + dst) = vv;
      }
    }
    if (tid == 0) p.seq_lens[le] = n + 1;
  }
}

__device__ void plan_items(const DecodeParams& p) {
  __shared__ long long s_red[32];
  __shared__ int s_scan[32];
  __shared__ int s_carry;
  __shared__ int s_chunk;
  __shared__ int s_multi;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_warps = blockDim.x >> 5;
  const int n_units = p.n_layers * p.batch;

  long long rows = 0;
  for (int e = tid; e < n_units; e += blockDim.x) {
    const int n = __ldcg(&p.seq_lens[(p.layer_begin + e / p.batch) * p.batch + e % p.batch]);
    rows += n > 0 ? n : 0;
  }
  for (int o = 16; o > 0; o >>= 1) rows += __shfl_xor_sync(0xffffffffu, rows, o);
  if (lane == 0) s_red[warp] = rows;
  __syncthreads();
  if (tid == 0) {
    long long total = 0;
    for (int w = 0; w < n_warps; ++w) total += s_red[w];
    total *= p.n_kv_heads;
    const int chunk = choose_chunk(total, p.chunk_rows_forced);
    s_chunk = chunk;
    s_carry = 0;
    s_multi = 0;
    p.hdr->chunk_rows = chunk;
  }
  __syncthreads();
  const int chunk = s_chunk;

  for (int base = 0; base < n_units; base += blockDim.x) {
    const int e = base + tid;
    int n = 0, nc = 0;
    if (e < n_units) {
      n = __ldcg(&p.seq_lens[(p.layer_begin + e / p.batch) * p.batch + e % p.batch]);
      if (n < 0) n = 0;
      nc = n == 0 ? 1 : (n + chunk - 1) / chunk;
    }
    int incl = nc;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int v = lane < n_warps ? s_scan[lane] : 0, inc = v;
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
      }
      s_scan[lane] = inc - v;   // exclusive prefix of the warp totals
    }
    __syncthreads();
    const int carry = s_carry;
    const int excl = carry + s_scan[warp] + incl - nc;
    if (e < n_units && nc > 1) p.multi_list[atomicAdd(&s_multi, 1)] = e;
    if (e < n_units) {
      const int first = excl * p.n_kv_heads;
      p.unit_info[e] = make_int2(first, nc);
      if (first + nc * p.n_kv_heads <= p.max_items) {
        for (int h = 0; h < p.n_kv_heads; ++h)
          for (int c = 0; c < nc; ++c) {
            const int rb = c * chunk;
            const int re = min(n, rb + chunk);
            p.items[first + h * nc + c] = make_int4(e, h, rb, re);
          }
      }
    }
    __syncthreads();
    if (tid == blockDim.x - 1) s_carry = excl + nc;
    __syncthreads();
  }
  if (tid == 0) {
    const int n_items = s_carry * p.n_kv_heads;
    if (n_items > p.max_items) {
      record_status(p.hdr, XKV_ERR_WORKSPACE);
      p.hdr->n_items = 0;
      p.hdr->n_multi = 0;
    } else {
      p.hdr->n_items = n_items;
      p.hdr->n_multi = s_multi;
    }
  }
}

__global__ void __launch_bounds__(kPrepThreads) decode_prepare_kernel(DecodeParams p, int D, int do_append, int q8) {
  __shared__ int s_page;
  __shared__ int s_last;
  const int tid = threadIdx.x;
  if (do_append) append_unit(p, D, blockIdx.x, &s_page, q8 != 0);
  // the last CTA to get here sees every sequence length already advanced and writes the plan
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(&p.hdr->prep_ticket, 1);
    s_last = (ticket == (int)gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  plan_items(p);
}

// ---------------------------------------------------------------------------------------------
template <int D, bool Q8>
__global__ void __launch_bounds__((Cfg<D, Q8>::kThreads), 1)
decode_attn_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const DecodeParams p) {
  using C = Cfg<D, Q8>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint8_t* ring = smem + (size_t)warp * C::kRingBytes;
  // Q8: where stage s keeps its K bytes, V bytes and the two scale vectors
  auto raw_k = [&](uint32_t s) -> uint8_t* { return ring + (size_t)s * C::kRawTileBytes; };
  auto raw_v = [&](uint32_t s) -> uint8_t* { return ring + C::kRawVOff + (size_t)s * C::kRawTileBytes; };
  auto raw_scales = [&](uint32_t s) -> float* {       // [0..15] K rows, [16..31] V rows
    return reinterpret_cast<float*>(ring + C::kScaleOff + (size_t)s * 2 * C::kScaleBytes);
  };
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + (size_t)C::kWarps * C::kRingBytes) + warp * C::kStages;
  uint8_t* fifo_base = smem + (size_t)C::kWarps * C::kRingBytes + C::kWarps * C::kStages * 8;
  int4* fifo = reinterpret_cast<int4*>(fifo_base) + warp * kFifo;                        // item descriptors
  int* fifo_idx = reinterpret_cast<int*>(fifo_base + C::kWarps * kFifo * 16) + warp * kFifo;   // and their indices
  int* s_excl = reinterpret_cast<int*>(fifo_base + C::kWarps * kFifo * 20);   // [units + 1] chunks before each unit
  uint16_t* s_multi = reinterpret_cast<uint16_t*>(s_excl + kMaxPlanUnits + 1);  // units cut into several chunks
  __shared__ int s_plan[4];                                                     // chunk rows, split units, page scratch
  __shared__ int s_scan[2 * C::kWarps];
  __shared__ long long s_rows[C::kWarps];

  if (tid == 0) {
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)C::kWarps * C::kRingBytes);
    for (int s = 0; s < C::kWarps * C::kStages; ++s) mbar_init(&bars[s], 1);
    fence_mbar_init();
    prefetch_tmap(&tmap_k);
    prefetch_tmap(&tmap_v);
  }
  __syncthreads();

  const bool fused = p.fused_plan != 0;
  const int n_units = p.n_layers * p.batch;
  // Length of unit e as this launch sees it: the stored length, plus the row this call appends when it fits the
  // page table.  seq_lens itself is only advanced by the last CTA to leave, so this reads the same at any time.
  const int cap_rows = p.max_pages_per_seq * p.page_size;
  const bool self_append = fused && p.do_append != 0;
  auto unit_len = [&](int e) -> int {
    int n = __ldcg(&p.seq_lens[(p.layer_begin + e / p.batch) * p.batch + e % p.batch]);
    n = n > 0 ? n : 0;
    return n + ((self_append && n < cap_rows) ? 1 : 0);
  };
  if (fused) {
    // ---- prologue of the self-planning launch
    // the plan, computed by every CTA for itself: chunk size from the total length, then the number of chunks
    // before each unit (and the list of units with more than one)
    constexpr int kPer = kMaxPlanUnits / C::kThreads;
    int nloc[kPer];
    long long rows = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int e = tid * kPer + i;
      nloc[i] = e < n_units ? unit_len(e) : 0;
      rows += nloc[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rows += __shfl_xor_sync(0xffffffffu, rows, o);
    if (lane == 0) s_rows[warp] = rows;
    __syncthreads();
    long long total = 0;
#pragma unroll
    for (int w8 = 0; w8 < C::kWarps; ++w8) total += s_rows[w8];
    const int chunk = choose_chunk(total * p.n_kv_heads, p.chunk_rows_forced);
    int cnt = 0, mcnt = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int e = tid * kPer + i;
      const int nc = e < n_units ? (nloc[i] == 0 ? 1 : (nloc[i] + chunk - 1) / chunk) : 0;
      nloc[i] = nc;
      cnt += nc;
      mcnt += nc > 1 ? 1 : 0;
    }
    int icnt = cnt, imcnt = mcnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, icnt, o), b = __shfl_up_sync(0xffffffffu, imcnt, o);
      if (lane >= o) {
        icnt += a;
        imcnt += b;
      }
    }
    if (lane == 31) {
      s_scan[warp] = icnt;
      s_scan[C::kWarps + warp] = imcnt;
    }
    __syncthreads();
    int base = icnt - cnt, mbase = imcnt - mcnt, all = 0, mall = 0;
#pragma unroll
    for (int w8 = 0; w8 < C::kWarps; ++w8) {
      if (w8 < warp) {
        base += s_scan[w8];
        mbase += s_scan[C::kWarps + w8];
      }
      all += s_scan[w8];
      mall += s_scan[C::kWarps + w8];
    }
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int e = tid * kPer + i;
      if (e < n_units) {
        s_excl[e] = base;
        if (nloc[i] > 1) s_multi[mbase++] = (uint16_t)e;
        base += nloc[i];
      }
    }
    if (tid == 0) {
      s_excl[n_units] = all;
      s_plan[0] = chunk;
      s_plan[1] = mall;
      s_plan[2] = ((long long)all * p.n_kv_heads <= (long long)p.max_items) ? all * p.n_kv_heads : -1;
      if (blockIdx.x == 0) {
        p.hdr->chunk_rows = chunk;
        p.hdr->n_items = s_plan[2] < 0 ? 0 : s_plan[2];
        p.hdr->n_multi = mall;
        if (s_plan[2] < 0) record_status(p.hdr, XKV_ERR_WORKSPACE);
      }
    }
    __syncthreads();
  }
  const int n_items = fused ? max(s_plan[2], 0) : p.hdr->n_items;
  const int n_multi = fused ? (s_plan[2] < 0 ? 0 : s_plan[1]) : p.hdr->n_multi;
  const int plan_chunk = fused ? s_plan[0] : 0;
  // work item idx -> {unit e, KV head, first row, end row}
  auto item_desc = [&](int idx) -> int4 {
    if (!fused) return p.items[idx];
    const int q = idx / p.n_kv_heads;
    int lo = 0, hi = n_units;                      // s_excl[lo] <= q < s_excl[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_excl[mid] <= q) lo = mid;
      else hi = mid;
    }
    const int first_chunk = s_excl[lo], nc = s_excl[lo + 1] - first_chunk;
    const int local = idx - first_chunk * p.n_kv_heads;
    const int h = local / nc, c = local % nc;
    const int n = unit_len(lo);
    const int rb = c * plan_chunk;
    return make_int4(lo, h, rb, min(n, rb + plan_chunk));
  };
  // {first work item of the unit's KV head 0, chunks per KV head}
  auto unit_info = [&](int e) -> int2 {
    if (!fused) return p.unit_info[e];
    return make_int2(s_excl[e] * p.n_kv_heads, s_excl[e + 1] - s_excl[e]);
  };
  const int gid = lane >> 2, tig = lane & 3;
  const int mat = lane >> 3, mrow = lane & 7;
  const int G = p.group;
  constexpr uint32_t kTxBytes = C::kStageBytes;

  // ---- producer side of this warp: runs up to kStages tiles ahead of the consumer side
  bool p_valid = false, no_more = false, aborted = false;
  int4 p_desc = make_int4(0, 0, 0, 0);
  int p_row = 0, p_page_tile0 = 0, p_pages = 0, p_item = 0;
  const int32_t* p_bt = p.block_table;
  int fifo_head = 0, fifo_count = 0;
  uint32_t issued = 0, consumed = 0;
  int next_idx = 0;
  if (lane == 0) next_idx = atomicAdd(&p.hdr->work_counter, 1);

  auto produce_one = [&]() -> bool {
    while (true) {
      if (!p_valid) {
        if (no_more || fifo_count == kFifo) return false;
        const int idx = __shfl_sync(0xffffffffu, next_idx, 0);
        if (idx >= n_items) {
          no_more = true;
          return false;
        }
        if (lane == 0) next_idx = atomicAdd(&p.hdr->work_counter, 1);   // fetched early, used at the next item
        p_desc = item_desc(idx);
        p_item = idx;
        const int slot = (fifo_head + fifo_count) % kFifo;
        if (lane == 0) {
          fifo[slot] = p_desc;
          fifo_idx[slot] = idx;
        }
        ++fifo_count;
        p_row = p_desc.z;
        if (p_row >= p_desc.w) continue;          // empty cache: the consumer side writes zeros
        const int e = p_desc.x;
        const int le = (p.layer_begin + e / p.batch) * p.batch + e % p.batch;
        p_bt = p.block_table + (size_t)le * p.max_pages_per_seq;
        p_page_tile0 = -1000000;
        p_valid = true;
      }
      const int tile = p_row / kTileRows;
      if (tile - p_page_tile0 >= 32 || tile < p_page_tile0) {       // refill the page ids of the next 32 tiles
        p_page_tile0 = tile;
        const int slot_row = (tile + lane) * kTileRows;
        p_pages = slot_row < p_desc.w ? p_bt[slot_row / p.page_size] : 0;
      }
      int page = __shfl_sync(0xffffffffu, p_pages, tile - p_page_tile0);
      page = min(max(page, 0), p.n_pages - 1);
      if (lane == 0) {
        const int grow = (page * p.n_kv_heads + p_desc.y) * p.page_size + p_row % p.page_size;
        const int s = issued % C::kStages;
        uint8_t* ks = ring + (size_t)s * C::kStageBytes;
        mbar_arrive_expect_tx(&full_bar[s], kTxBytes);
        if constexpr (Q8) {
          // stored bytes of the 16 rows (one box of D bytes per row) and their scales (16 consecutive floats)
          tma_load_2d(raw_k(s), &tmap_k, 0, grow, &full_bar[s]);
          tma_load_2d(raw_v(s), &tmap_v, 0, grow, &full_bar[s]);
          bulk_copy_g2s(raw_scales(s), p.k_scales + grow, C::kScaleBytes, &full_bar[s]);
          bulk_copy_g2s(raw_scales(s) + kTileRows, p.v_scales + grow, C::kScaleBytes, &full_bar[s]);
        } else {
          uint8_t* vs = ks + C::kTileBytes;
#pragma unroll
          for (int hf = 0; hf < C::kHalves; ++hf) {
            tma_load_2d(ks + hf * C::kBoxBytes, &tmap_k, hf * 64, grow, &full_bar[s]);
            tma_load_2d(vs + hf * C::kBoxBytes, &tmap_v, hf * 64, grow, &full_bar[s]);
          }
        }
      }
      ++issued;
      p_row += kTileRows;
      if (p_row >= p_desc.w) p_valid = false;
      return true;
    }
  };
  auto fill = [&]() {
    while (!aborted && issued - consumed < (uint32_t)C::kStages && produce_one()) {
    }
  };

  // ---- consumer side.  Everything is computed transposed, keys on the M axis of the tensor-core tile and the
  // (at most eight) query heads of the group on its N axis: S^T = K.Q^T is one m16n8 accumulator per 16-row
  // tile, and O^T = V^T.P^T needs D/16 of them, so no accumulator row is padding.  In every fragment a lane
  // then owns the two heads 2*tig, 2*tig+1.
  const uint32_t k_lane_off = (uint32_t)(((mat & 1) * 8 + mrow) * 128 + ((((mat >> 1) & 1) ^ mrow) << 4));
  const uint32_t v_lane_off = (uint32_t)(((mat >> 1) * 8 + mrow) * 128 + (((mat & 1) ^ mrow) << 4));
  constexpr float kLazy = 8.f;        // the reference maximum is raised only when a score exceeds it by 2^8

  // waits for the tile with sequence number idx (bounded); flags the warp as aborted on failure
  auto wait_tile = [&](uint32_t idx) {
    if (aborted) return;
    const int s = idx % C::kStages;
    const uint32_t ph = (idx / C::kStages) & 1u;
    const bool ok = ((int32_t)(issued - idx) > 0) && mbar_wait_bounded(&full_bar[s], ph, p.wait_ns);
    if (!__all_sync(0xffffffffu, ok)) {
      aborted = true;
      no_more = true;
      if (lane == 0) record_status(p.hdr, XKV_ERR_TIMEOUT);
    }
  };

  while (true) {
    fill();
    if (fifo_count == 0) break;
    __syncwarp();
    const int item = fifo_idx[fifo_head];
    const int4 I = fifo[fifo_head];
    fifo_head = (fifo_head + 1) % kFifo;
    --fifo_count;
    const int e = I.x, h = I.y;
    const int nc = unit_info(e).y;
    const size_t q_row0 = ((size_t)e * p.n_q_heads + (size_t)h * G);

    // Q^T as the B operand: lane (gid, tig) holds head gid, columns 16*ks + 2*tig (+1) and + 8
    uint32_t qb[D / 16][2];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      qb[ks][0] = 0u;
      qb[ks][1] = 0u;
      if (gid < G) {
        const __nv_bfloat16* qp = p.q + (q_row0 + gid) * D + 16 * ks + 2 * tig;
        qb[ks][0] = *reinterpret_cast<const uint32_t*>(qp);
        qb[ks][1] = *reinterpret_cast<const uint32_t*>(qp + 8);
        if constexpr (Q8) {
          // The 8-bit path multiplies in fp16, and a lane's K fragment of this k-step holds the four consecutive
          // columns 16*ks + 4*tig .. + 3 (two registers of two): the query columns follow that order.
          const uint2 four = *reinterpret_cast<const uint2*>(p.q + (q_row0 + gid) * D + 16 * ks + 4 * tig);
          qb[ks][0] = pack_f16(bf16_lo(four.x), bf16_hi(four.x));
          qb[ks][1] = pack_f16(bf16_lo(four.y), bf16_hi(four.y));
        }
      }
    }
    float o[D / 16][4];               // O^T: [mt] = columns 16*mt + gid (regs 0,1) and + 8 (regs 2,3); heads 2*tig, +1
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    float m_ref[2] = {-3.0e38f, -3.0e38f};   // finite, so that (-inf) - m_ref stays -inf
    float l_part[2] = {0.f, 0.f};
    // Q8: the stored bytes enter the MMAs as kInt8Bias + q.  q_bias[i] = kInt8Bias x (sum over d of the query of head
    // 2*tig + i) comes off every logit; p_sum[i] gathers the weights P as the O^T MMAs see them, and kInt8Bias x p_sum
    // comes off every element of O^T at the end.  Both sums are formed by the tensor core itself (an A operand of
    // ones), so they are rounded exactly like the products they correct.
    const uint32_t ones[4] = {0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u};
    float q_bias[2] = {0.f, 0.f}, p_sum[4] = {0.f, 0.f, 0.f, 0.f};
    if constexpr (Q8) {
      float qs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) mma_f16_16816(qs, ones, qb[ks][0], qb[ks][1]);
      q_bias[0] = kInt8Bias * qs[0];
      q_bias[1] = kInt8Bias * qs[1];
    }

    // S^T of one 16-row tile: rows gid (regs 0,1) and gid + 8 (regs 2,3), heads 2*tig, 2*tig + 1
    // Q8: address this lane hands to ldmatrix for row `row` (0..15) and 16-byte piece `piece` of a raw tile (rows of D
    // bytes; pieces at their swizzled places when a row is the 128 bytes of the swizzle span)
    auto raw_piece = [&](uint32_t tile_base, int row, int piece) -> uint32_t {
      return D == 128 ? tile_base + row * 128 + ((piece ^ (row & 7)) << 4) : tile_base + row * D + (piece << 4);
    };
    auto qk_tile = [&](uint32_t idx, float (&acc)[4]) {
      const uint32_t s = idx % C::kStages;
      float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f};
      if constexpr (Q8) {
        // One ldmatrix.x4 covers two k-steps: matrices (rows 0-7 | 8-15) x (piece 2j | 2j+1); a lane then holds, per
        // matrix, the four consecutive bytes 4*tig .. of row gid: columns 0, 1 feed the fragment's first k pair and
        // columns 2, 3 its second one (the query fragment is loaded in the same column order).
        const uint32_t kt = smem_u32(raw_k(s));
#pragma unroll
        for (int j = 0; j < D / 32; ++j) {
          uint32_t r[4];
          ldmatrix_x4(r, raw_piece(kt, (mat & 1) * 8 + mrow, 2 * j + (mat >> 1)));
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int ks = 2 * j + half;
            const uint32_t af[4] = {int8x2_to_biased_f16x2<0x5140>(r[2 * half]),
                                    int8x2_to_biased_f16x2<0x5140>(r[2 * half + 1]),
                                    int8x2_to_biased_f16x2<0x5342>(r[2 * half]),
                                    int8x2_to_biased_f16x2<0x5342>(r[2 * half + 1])};
            if (half) mma_f16_16816(a1, af, qb[ks][0], qb[ks][1]);
            else      mma_f16_16816(a0, af, qb[ks][0], qb[ks][1]);
          }
        }
      } else {
        const uint32_t ks_base = smem_u32(ring + (size_t)s * C::kStageBytes);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          uint32_t af[4];
          ldmatrix_x4(af, ks_base + (ks >> 2) * C::kBoxBytes + (k_lane_off ^ (uint32_t)(((2 * ks) & 7) << 4)));
          if (ks & 1) mma_bf16_16816(a1, af, qb[ks][0], qb[ks][1]);
          else        mma_bf16_16816(a0, af, qb[ks][0], qb[ks][1]);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i] = a0[i] + a1[i];
      if constexpr (Q8) {
        // the rows' scales: keys gid (registers 0, 1) and gid + 8 (registers 2, 3)
        const float* kscale = raw_scales(s);
        const float s0 = kscale[gid], s1 = kscale[gid + 8];
        acc[0] = (acc[0] - q_bias[0]) * s0;
        acc[1] = (acc[1] - q_bias[1]) * s0;
        acc[2] = (acc[2] - q_bias[0]) * s1;
        acc[3] = (acc[3] - q_bias[1]) * s1;
      }
    };

    const int n_tiles = (I.w - I.z + kTileRows - 1) / kTileRows;
    // The row this call appends to (e, h) is the last row of the unit's last chunk.  Its page slot still holds
    // old bytes when the tile is copied in, so the owner of that chunk takes the row from k_new / v_new:
    // into the landed tile (16-byte pieces at their swizzled places; lanes 0-15 carry K, lanes 16-31 V) and into
    // the page, where the next call's copies will find it.
    int new_slot = -1;                                   // cache slot of the appended row if this item owns it
    if (self_append && I.w > I.z) {
      const int n_old = max(__ldcg(&p.seq_lens[(p.layer_begin + e / p.batch) * p.batch + e % p.batch]), 0);
      if (n_old < cap_rows && I.w == n_old + 1) new_slot = n_old;
    }
    auto patch_new_row = [&](uint32_t idx) {
      constexpr int kPieces = D / 8;                     // 16-byte pieces of one row
      const int r = (new_slot - I.z) % kTileRows;
      const size_t src = ((size_t)e * p.n_kv_heads + h) * D;
      const int le = (p.layer_begin + e / p.batch) * p.batch + e % p.batch;
      const int page = p.block_table[(size_t)le * p.max_pages_per_seq + new_slot / p.page_size];
      const bool page_ok = page >= 0 && page < p.n_pages;
      if (!page_ok && lane == 0) record_status(p.hdr, XKV_ERR_CAPACITY);
      if constexpr (Q8) {
        // The new row is quantised here (its D/8 pieces on consecutive lanes: K on the first D/8 lanes, V on the next
        // ones); its bytes and scales go into the landed raw tile and into the page.
        static_assert(2 * kPieces <= 32, "one warp holds the K and V pieces of a row");
        const uint32_t st = idx % C::kStages;
        if (lane < 2 * kPieces) {
          const int is_v = lane / kPieces, c = lane % kPieces;
          float x[8], sc;
          bf16x8_to_f32(*reinterpret_cast<const uint4*>((is_v ? p.v_new : p.k_new) + src + c * 8), x);
          const uint2 bytes = quantize_row_piece(x, kPieces, &sc);
          uint8_t* raw = is_v ? raw_v(st) : raw_k(st);
          const int off = D == 128 ? r * 128 + (((c >> 1) ^ (r & 7)) << 4) + (c & 1) * 8 : r * D + c * 8;
          *reinterpret_cast<uint2*>(raw + off) = bytes;
          if (c == 0) raw_scales(st)[is_v * kTileRows + r] = sc;
          if (page_ok) {
            const size_t slot = ((size_t)page * p.n_kv_heads + h) * p.page_size + new_slot % p.page_size;
            *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(is_v ? p.v_pages : p.k_pages) + slot * D + c * 8) = bytes;
            if (c == 0) (is_v ? p.v_scales : p.k_scales)[slot] = sc;
          }
        }
      } else {
        uint8_t* ks = ring + (size_t)(idx % C::kStages) * C::kStageBytes;
        for (int i = lane; i < 2 * kPieces; i += 32) {
          const int is_v = i / kPieces, c = i % kPieces;
          const uint4 val = *reinterpret_cast<const uint4*>((is_v ? p.v_new : p.k_new) + src + c * 8);
          *reinterpret_cast<uint4*>(ks + is_v * C::kTileBytes + (c >> 3) * C::kBoxBytes + r * 128 +
                                    (((c & 7) ^ (r & 7)) << 4)) = val;
          if (page_ok) {
            const size_t dst = (((size_t)page * p.n_kv_heads + h) * p.page_size + new_slot % p.page_size) * D + c * 8;
            *reinterpret_cast<uint4*>((is_v ? p.v_pages : p.k_pages) + dst) = val;
          }
        }
      }
      fence_proxy_async_smem();       // the stage is written again by a later copy
      __syncwarp();
    };
    float s_next[4] = {0.f, 0.f, 0.f, 0.f};
    if (n_tiles > 0) {
      wait_tile(consumed);
      if (!aborted && new_slot >= 0 && n_tiles == 1) patch_new_row(consumed);
      if (!aborted) qk_tile(consumed, s_next);
    }
    for (int t = 0; t < n_tiles; ++t) {
      float sv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) sv[i] = s_next[i] * p.scale_log2;
      const int s = consumed % C::kStages;
      const int wrows = min(kTileRows, I.w - (I.z + t * kTileRows));
      if (t + 1 < n_tiles) {          // the next tile's scores do not depend on this tile's softmax
        wait_tile(consumed + 1);
        if (!aborted && new_slot >= 0 && t + 2 == n_tiles) patch_new_row(consumed + 1);
        if (!aborted) qk_tile(consumed + 1, s_next);
      }
      if (!aborted) {
        float vs0 = 1.f, vs1 = 1.f;                    // Q8: scales of the V rows gid and gid + 8
        if constexpr (Q8) {
          const float* vscale = raw_scales(s) + kTileRows;
          vs0 = gid < wrows ? vscale[gid] : 0.f;       // rows past the end of the cache carry no weight at all
          vs1 = gid + 8 < wrows ? vscale[gid + 8] : 0.f;
        }
        const uint32_t vs_base = smem_u32(ring + (size_t)s * C::kStageBytes) + C::kTileBytes;
        if (wrows < kTileRows) {
          // rows past the end of the cache hold whatever the page held: mask their scores and (16-bit tiles, where the
          // leftovers may be NaN) clear V so that 0 * x stays 0; stored bytes are always finite integers
          if (gid >= wrows) sv[0] = sv[1] = -INFINITY;
          if (gid + 8 >= wrows) sv[2] = sv[3] = -INFINITY;
          if constexpr (!Q8) {
            uint8_t* vs = ring + (size_t)s * C::kStageBytes + C::kTileBytes;
            const int n_bad = kTileRows - wrows;
            for (int idx = lane; idx < n_bad * (D / 8); idx += 32) {
              const int row = wrows + idx / (D / 8);
              const int c = idx % (D / 8);
              *reinterpret_cast<uint4*>(vs + (c >> 3) * C::kBoxBytes + row * 128 + (c & 7) * 16) =
                  make_uint4(0u, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();
            __syncwarp();
          }
        }
        float mx0 = fmaxf(sv[0], sv[2]), mx1 = fmaxf(sv[1], sv[3]);
        const bool grow = (mx0 > m_ref[0] + kLazy) || (mx1 > m_ref[1] + kLazy);
        if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
          for (int x = 4; x < 32; x <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, x));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, x));
          }
          const float n0 = fmaxf(m_ref[0], mx0), n1 = fmaxf(m_ref[1], mx1);
          const float al0 = fast_exp2(m_ref[0] - n0), al1 = fast_exp2(m_ref[1] - n1);
          m_ref[0] = n0;
          m_ref[1] = n1;
          l_part[0] *= al0;
          l_part[1] *= al1;
#pragma unroll
          for (int mt = 0; mt < D / 16; ++mt) {
            o[mt][0] *= al0;
            o[mt][1] *= al1;
            o[mt][2] *= al0;
            o[mt][3] *= al1;
          }
          if constexpr (Q8) {
            p_sum[0] *= al0;
            p_sum[1] *= al1;
            p_sum[2] *= al0;
            p_sum[3] *= al1;
          }
        }
        const float p0 = fast_exp2(sv[0] - m_ref[0]), p1 = fast_exp2(sv[1] - m_ref[1]);
        const float p2 = fast_exp2(sv[2] - m_ref[0]), p3 = fast_exp2(sv[3] - m_ref[1]);
        l_part[0] += p0 + p2;
        l_part[1] += p1 + p3;
        // P^T as the B operand of O^T += V^T.P^T: transpose the two 8x8 blocks of the accumulator layout
        const uint32_t b0 = movmatrix_trans(Q8 ? pack_f16(p0 * vs0, p1 * vs0) : pack_bf16(p0, p1));
        const uint32_t b1 = movmatrix_trans(Q8 ? pack_f16(p2 * vs1, p3 * vs1) : pack_bf16(p2, p3));
        if constexpr (Q8) {
          // V^T fragments out of the raw [keys][D] tile: a transposing ldmatrix over 16-bit units hands a lane, per
          // matrix (keys 0-7 | 8-15) x (16 columns), the bytes (key 2*tig, cols 2*gid, 2*gid+1) and (key 2*tig+1, same
          // cols).  Bytes 0 and 2 are the two keys of column 2*gid, bytes 1 and 3 those of column 2*gid+1: the
          // accumulator rows gid and gid+8 of a 16-column block therefore stand for columns 2*gid and 2*gid+1.
          const uint32_t vt = smem_u32(raw_v(s));
#pragma unroll
          for (int j = 0; j < D / 32; ++j) {
            uint32_t r[4];
            ldmatrix_x4_trans(r, raw_piece(vt, (mat & 1) * 8 + mrow, 2 * j + (mat >> 1)));
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const uint32_t af[4] = {int8x2_to_biased_f16x2<0x5240>(r[2 * half]),
                                      int8x2_to_biased_f16x2<0x5341>(r[2 * half]),
                                      int8x2_to_biased_f16x2<0x5240>(r[2 * half + 1]),
                                      int8x2_to_biased_f16x2<0x5341>(r[2 * half + 1])};
              mma_f16_16816(o[2 * j + half], af, b0, b1);
            }
          }
          mma_f16_16816(p_sum, ones, b0, b1);
        } else {
#pragma unroll
          for (int mt = 0; mt < D / 16; ++mt) {
            uint32_t af[4];
            ldmatrix_x4_trans(af, vs_base + (mt >> 2) * C::kBoxBytes + (v_lane_off ^ (uint32_t)(((2 * mt) & 7) << 4)));
            mma_bf16_16816(o[mt], af, b0, b1);
          }
        }
      }
      __syncwarp();
      ++consumed;
      fill();                                   // the stage just released takes the next tile
    }

    if constexpr (Q8) {               // take the bias of the stored bytes off O^T (see p_sum above)
#pragma unroll
      for (int mt = 0; mt < D / 16; ++mt) {
        o[mt][0] -= kInt8Bias * p_sum[0];
        o[mt][1] -= kInt8Bias * p_sum[1];
        o[mt][2] -= kInt8Bias * p_sum[0];
        o[mt][3] -= kInt8Bias * p_sum[1];
      }
    }
    // ---- finish the work item: denominators of the lane's two heads over all rows
#pragma unroll
    for (int x = 4; x < 32; x <<= 1) {
      l_part[0] += __shfl_xor_sync(0xffffffffu, l_part[0], x);
      l_part[1] += __shfl_xor_sync(0xffffffffu, l_part[1], x);
    }
    // normalises an accumulator in fragment layout and stores it as bf16 rows of the output
    auto store_out = [&](float (&acc)[D / 16][4], const float (&den)[2], const float (&mx)[2]) {
      const float inv0 = den[0] > 0.f ? 1.f / den[0] : 0.f;
      const float inv1 = den[1] > 0.f ? 1.f / den[1] : 0.f;
      __nv_bfloat16* orow = p.out + (q_row0 + gid) * D;
#pragma unroll
      for (int mt = 0; mt < D / 16; ++mt) {
        // after the transpose the lane holds head gid, columns 16*mt + 2*tig (+1), then the same + 8
        const uint32_t u0 = movmatrix_trans(pack_bf16(acc[mt][0] * inv0, acc[mt][1] * inv1));
        const uint32_t u1 = movmatrix_trans(pack_bf16(acc[mt][2] * inv0, acc[mt][3] * inv1));
        if (gid < G) {
          if constexpr (Q8) {
            // accumulator rows r < 8 stand for columns 2r, rows 8 + r for columns 2r + 1: u0 holds columns 4*tig and
            // 4*tig + 2, u1 columns 4*tig + 1 and 4*tig + 3
            uint2 w;
            asm("prmt.b32 %0, %1, %2, 0x5410;" : "=r"(w.x) : "r"(u0), "r"(u1));
            asm("prmt.b32 %0, %1, %2, 0x7632;" : "=r"(w.y) : "r"(u0), "r"(u1));
            *reinterpret_cast<uint2*>(orow + 16 * mt + 4 * tig) = w;
          } else {
            *reinterpret_cast<uint32_t*>(orow + 16 * mt + 2 * tig) = u0;
            *reinterpret_cast<uint32_t*>(orow + 16 * mt + 8 + 2 * tig) = u1;
          }
        }
      }
      if (gid == 0 && p.lse != nullptr) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
          if (2 * tig + hh < G)
            p.lse[q_row0 + 2 * tig + hh] =
                den[hh] > 0.f ? (mx[hh] + log2f(den[hh])) * 0.6931471805599453f : -INFINITY;
      }
    };

    if (nc == 1) {
      store_out(o, l_part, m_ref);
    } else {
      // partial results of this chunk: [item][head][D] accumulators and [item][head] (max, sum)
#pragma unroll
      for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int head = 2 * tig + (i & 1);
          const int col = Q8 ? 2 * gid + (i >> 1) : gid + 8 * (i >> 1);     // see store_out for the 8-bit order
          if (head < G) p.part_o[((size_t)item * G + head) * D + 16 * mt + col] = o[mt][i];
        }
      if (gid == 0) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
          if (2 * tig + hh < G)
            *reinterpret_cast<float2*>(p.part_ml + ((size_t)item * G + 2 * tig + hh) * 2) =
                make_float2(m_ref[hh], l_part[hh]);
      }
      __syncwarp();                 // the lanes' partial results are ordered before lane 0's fence (cumulative)
      if (lane == 0 && item != p.withhold_item) {
        __threadfence();
        atomicAdd(&p.tickets[e * p.n_kv_heads + h], 1);     // one more chunk of this unit is published
      }
    }
  }

  // ---- merge phase.  Once the work items have run out, the warps share out the units that were cut into several
  // chunks, one query head at a time, and combine the chunks' partial results by log-sum-exp.  A job may find
  // chunks of its unit still being computed: every such chunk is held by a warp that is still streaming (a warp
  // comes here only after it has finished every item it took) and streaming warps wait for nothing but their own
  // copies, so the bounded wait below ends.
  constexpr int kCols = D / 32;
  const int n_jobs = n_multi * p.n_kv_heads * G;
  while (!aborted) {
    int job = 0;
    if (lane == 0) job = atomicAdd(&p.hdr->merge_counter, 1);
    job = __shfl_sync(0xffffffffu, job, 0);
    if (job >= n_jobs) break;
    const int g = job % G, uh = job / G;
    const int h = uh % p.n_kv_heads;
    const int e = fused ? (int)s_multi[uh / p.n_kv_heads] : p.multi_list[uh / p.n_kv_heads];
    const int2 ui = unit_info(e);
    const int nc = ui.y, first = ui.x + h * nc;
    int ready = 1;
    if (lane == 0) ready = spin_until_ge(&p.tickets[e * p.n_kv_heads + h], nc, p.wait_ns, 200) ? 1 : 0;
    ready = __shfl_sync(0xffffffffu, ready, 0);
    if (!ready) {
      if (lane == 0) record_status(p.hdr, XKV_ERR_TIMEOUT);
      break;
    }
    __threadfence();
    float m_run = -3.0e38f, den = 0.f, acc[kCols];
#pragma unroll
    for (int j = 0; j < kCols; ++j) acc[j] = 0.f;
    for (int c0 = 0; c0 < nc; c0 += 32) {
      // lane c holds the weight of chunk c0 + c; the chunks' rows are then read sixteen at a time
      const int c = c0 + lane;
      float2 ml = make_float2(-3.0e38f, 0.f);
      if (c < nc) ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + ((size_t)(first + c) * G + g) * 2));
      float bm = ml.x;
#pragma unroll
      for (int x = 16; x > 0; x >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, x));
      const float m_new = fmaxf(m_run, bm);
      const float rescale = fast_exp2(m_run - m_new);
      const float wgt = c < nc ? fast_exp2(ml.x - m_new) : 0.f;
      float ds = wgt * ml.y;
#pragma unroll
      for (int x = 16; x > 0; x >>= 1) ds += __shfl_xor_sync(0xffffffffu, ds, x);
      den = den * rescale + ds;
      m_run = m_new;
#pragma unroll
      for (int j = 0; j < kCols; ++j) acc[j] *= rescale;
      const int nb = min(32, nc - c0);
      for (int cc = 0; cc < nb; cc += 16) {
        float v[16][kCols];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const float* src = p.part_o + ((size_t)(first + c0 + cc + k) * G + g) * D + lane * kCols;
          if (cc + k < nb) {
            if constexpr (kCols == 4) {
              const float4 t = __ldcg(reinterpret_cast<const float4*>(src));
              v[k][0] = t.x; v[k][1] = t.y; v[k][2] = t.z; v[k][3] = t.w;
            } else {
              const float2 t = __ldcg(reinterpret_cast<const float2*>(src));
              v[k][0] = t.x; v[k][1] = t.y;
            }
          } else {
#pragma unroll
            for (int j = 0; j < kCols; ++j) v[k][j] = 0.f;
          }
        }
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const float wk = __shfl_sync(0xffffffffu, wgt, (cc + k) & 31);
#pragma unroll
          for (int j = 0; j < kCols; ++j) acc[j] += wk * v[k][j];
        }
      }
    }
    const size_t row = (size_t)e * p.n_q_heads + (size_t)h * G + g;
    const float inv = den > 0.f ? 1.f / den : 0.f;
#pragma unroll
    for (int j = 0; j < kCols; j += 2)
      *reinterpret_cast<uint32_t*>(p.out + row * D + lane * kCols + j) = pack_bf16(acc[j] * inv, acc[j + 1] * inv);
    if (lane == 0 && p.lse != nullptr)
      p.lse[row] = den > 0.f ? (m_run + log2f(den)) * 0.6931471805599453f : -INFINITY;
  }
  if (aborted) {
    // let copies already issued land before this CTA's shared memory can be handed on
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
  if (self_append) {
    // the last CTA to get here advances the lengths of the units whose new row was stored
    __threadfence();
    __syncthreads();
    if (tid == 0) s_plan[3] = (atomicAdd(&p.hdr->grid_arrivals, 1) == (int)gridDim.x - 1) ? 1 : 0;
    __syncthreads();
    if (s_plan[3]) {
      for (int e = tid; e < n_units; e += C::kThreads) {
        const int le = (p.layer_begin + e / p.batch) * p.batch + e % p.batch;
        const int n_old = max(p.seq_lens[le], 0);
        if (n_old < cap_rows) {
          const int page = p.block_table[(size_t)le * p.max_pages_per_seq + n_old / p.page_size];
          if (page >= 0 && page < p.n_pages) p.seq_lens[le] = n_old + 1;
        } else {
          record_status(p.hdr, XKV_ERR_CAPACITY);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

bool make_page_tmap(CUtensorMap* tmap, void* base, int D, uint64_t rows, bool q8) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (enc == nullptr) return false;
  const cuuint64_t gdim[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  const cuuint32_t estr[2] = {1u, 1u};
  if (q8) {
    // one byte per element: a box is 16 whole rows of D bytes; rows of 128 bytes are swizzled like the 16-bit tiles
    // (conflict-free ldmatrix), rows of 64 bytes are stored as they are
    const cuuint64_t gstride[1] = {(cuuint64_t)D};
    const cuuint32_t box[2] = {(cuuint32_t)D, (cuuint32_t)kTileRows};
    return enc(tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               D == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  const cuuint64_t gstride[1] = {(cuuint64_t)D * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)kTileRows};
  return enc(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct DecodeLayout {
  size_t tickets, unit_info, multi, items, part_o, part_ml, total;
  int64_t max_items;
};

bool decode_layout(const xkv_dims* d, int n_layers, int max_cache_len, int chunk_rows, DecodeLayout* L) {
  if (n_layers <= 0 || d->batch <= 0 || d->n_kv_heads <= 0) return false;
  const int64_t lb = (int64_t)n_layers * d->batch;
  const int64_t units = lb * d->n_kv_heads;
  int64_t max_items;
  if (chunk_rows > 0) {
    const int64_t per = max_cache_len > 0 ? ((int64_t)max_cache_len + chunk_rows - 1) / chunk_rows : 1;
    max_items = units * (per > 0 ? per : 1);
  } else {
    // ceil() adds at most one item per unit, the rows themselves at most kTargetItems
    max_items = units + (int64_t)kTargetItems + 1;
  }
  if (max_items > (int64_t)1 << 28) return false;
  const int G = d->n_q_heads / d->n_kv_heads;
  size_t off = kHeaderBytes;
  L->tickets = off;   off = align_up(off + (size_t)units * 4, 256);
  L->unit_info = off; off = align_up(off + (size_t)lb * 8, 256);
  L->multi = off;     off = align_up(off + (size_t)lb * 4, 256);
  L->items = off;     off = align_up(off + (size_t)max_items * 16, 256);
  L->part_o = off;    off = align_up(off + (size_t)max_items * G * d->head_dim * 4, 256);
  L->part_ml = off;   off = align_up(off + (size_t)max_items * G * 2 * 4, 256);
  L->total = off;
  L->max_items = max_items;
  return true;
}

cudaEvent_t g_ev_start = nullptr, g_ev_stop = nullptr;

template <int D, bool Q8>
xkv_status launch_attn(const CUtensorMap& tk, const CUtensorMap& tv, const DecodeParams& p, cudaStream_t st) {
  cudaError_t attr_err = cudaSuccess;
  // opt in to the large dynamic shared-memory carve-out once per process and device in use
  int dev = 0;
  cudaGetDevice(&dev);
  static std::atomic<bool> done[64];   // idempotent set-up: two threads doing it twice is harmless
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  if (!done[dev].load(std::memory_order_acquire)) {
    attr_err = cudaFuncSetAttribute(decode_attn_kernel<D, Q8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    Cfg<D, Q8>::kSmemBytes);
    if (attr_err != cudaSuccess) return XKV_ERR_CUDA;
    done[dev].store(true, std::memory_order_release);
  }
  if (g_ev_start != nullptr && g_ev_stop != nullptr) cudaEventRecord(g_ev_start, st);
  decode_attn_kernel<D, Q8><<<sm_count(), Cfg<D, Q8>::kThreads, Cfg<D, Q8>::kSmemBytes, st>>>(tk, tv, p);
  if (g_ev_start != nullptr && g_ev_stop != nullptr) cudaEventRecord(g_ev_stop, st);
  count_launch();
  return check_launch();
}

}  // namespace

void set_profile_events(cudaEvent_t start, cudaEvent_t stop) {
  g_ev_start = start;
  g_ev_stop = stop;
}

size_t decode_workspace_bytes(const xkv_dims* d, int n_layers, int max_cache_len, int chunk_rows) {
  DecodeLayout L;
  if (!decode_layout(d, n_layers, max_cache_len, chunk_rows, &L)) return 0;
  return L.total;
}

xkv_status decode_attn(const xkv_dims* d, const xkv_cache* c, int layer_begin, int layer_end, const void* q,
                       const void* k_new, const void* v_new, void* out, float* lse, int chunk_rows,
                       void* workspace, size_t workspace_bytes, cudaStream_t st, bool clear_status) {
  const int Lr = layer_end - layer_begin;
  const int G = d->n_q_heads / d->n_kv_heads;
  if (G > kMaxGroup) return XKV_ERR_UNSUPPORTED;
  if (chunk_rows < 0 || chunk_rows % kChunkAlign != 0) return XKV_ERR_INVALID_ARG;
  const int max_cache_len = c->max_pages_per_seq * c->page_size;
  DecodeLayout L;
  if (!decode_layout(d, Lr, max_cache_len, chunk_rows, &L)) return XKV_ERR_INVALID_ARG;
  if (workspace_bytes < L.total) return XKV_ERR_WORKSPACE;
  const uint64_t page_rows = (uint64_t)c->n_pages * d->n_kv_heads * c->page_size;
  if (page_rows >= (1ull << 31)) return XKV_ERR_UNSUPPORTED;

  const bool q8 = c->kv_format == XKV_KV_INT8;
  CUtensorMap tk, tv;
  if (!make_page_tmap(&tk, c->k_pages, d->head_dim, page_rows, q8) ||
      !make_page_tmap(&tv, c->v_pages, d->head_dim, page_rows, q8))
    return XKV_ERR_CUDA;

  uint8_t* ws = static_cast<uint8_t*>(workspace);
  DecodeParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  p.k_pages = static_cast<__nv_bfloat16*>(c->k_pages);
  p.v_pages = static_cast<__nv_bfloat16*>(c->v_pages);
  p.k_scales = c->k_scales;
  p.v_scales = c->v_scales;
  p.block_table = c->block_table;
  p.seq_lens = c->seq_lens;
  p.layer_begin = layer_begin;
  p.n_layers = Lr;
  p.batch = d->batch;
  p.n_q_heads = d->n_q_heads;
  p.n_kv_heads = d->n_kv_heads;
  p.group = G;
  p.page_size = c->page_size;
  p.max_pages_per_seq = c->max_pages_per_seq;
  p.n_pages = c->n_pages;
  p.chunk_rows_forced = chunk_rows;
  p.max_items = (int32_t)L.max_items;
  const float scale = d->scale != 0.f ? d->scale : 1.0f / sqrtf((float)d->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  p.wait_ns = wait_limit_ns();
  p.withhold_item = debug_withhold_item();
  p.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  p.tickets = reinterpret_cast<int32_t*>(ws + L.tickets);
  p.unit_info = reinterpret_cast<int2*>(ws + L.unit_info);
  p.multi_list = reinterpret_cast<int32_t*>(ws + L.multi);
  p.items = reinterpret_cast<int4*>(ws + L.items);
  p.part_o = reinterpret_cast<float*>(ws + L.part_o);
  p.part_ml = reinterpret_cast<float*>(ws + L.part_ml);

  const int n_units = Lr * d->batch;
  const int do_append = k_new != nullptr ? 1 : 0;
  // Up to kMaxPlanUnits units the attention kernel plans in its own prologue and appends as it goes (one
  // launch); beyond that a separate kernel appends and writes the work-item table.
  p.fused_plan = n_units <= kMaxPlanUnits ? 1 : 0;
  p.do_append = do_append;
  // counters and tickets start at zero; the status word (the first four bytes) is left alone unless asked, so an
  // error of an earlier call on this workspace stays until it is read
  const size_t keep = clear_status ? 0 : sizeof(int32_t);
  if (cudaMemsetAsync(ws + keep, 0, L.unit_info - keep, st) != cudaSuccess) return XKV_ERR_CUDA;
  if (!p.fused_plan) {
    decode_prepare_kernel<<<do_append ? n_units : 1, kPrepThreads, 0, st>>>(p, d->head_dim, do_append, q8 ? 1 : 0);
    count_launch();
    xkv_status s = check_launch();
    if (s != XKV_OK) return s;
  }
  if (q8) return d->head_dim == 128 ? launch_attn<128, true>(tk, tv, p, st) : launch_attn<64, true>(tk, tv, p, st);
  return d->head_dim == 128 ? launch_attn<128, false>(tk, tv, p, st) : launch_attn<64, false>(tk, tv, p, st);
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant: the scratch that decode_attn normally receives from the caller lives in
// a fixed device array that is part of the library image.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = XKV_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

xkv_status decode_attn_static(const xkv_dims* d, const xkv_cache* c, int layer_begin, int layer_end,
                              const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                              int chunk_rows, int32_t* status_out, cudaStream_t st) {
  // In host code g_static_scratch is only a handle for the symbol; the device address has to be
  // asked for, once per device, while that device is current.
  static std::atomic<void*> scratch_ptr[64];   // resolving the address twice from two threads gives the same value
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  void* scratch = scratch_ptr[dev].load(std::memory_order_acquire);
  if (scratch == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return XKV_ERR_CUDA;
    scratch_ptr[dev].store(ptr, std::memory_order_release);
    scratch = ptr;
  }
  const int max_cache_len = c->max_pages_per_seq * c->page_size;
  const size_t need = decode_workspace_bytes(d, layer_end - layer_begin, max_cache_len, chunk_rows);
  if (need == 0) return XKV_ERR_INVALID_ARG;
  if (need > kStaticScratchBytes) return XKV_ERR_WORKSPACE;   // problem too large for the fixed scratch
  // decode_attn clears the part of the scratch that must start at zero (status word, tickets)
  xkv_status s = decode_attn(d, c, layer_begin, layer_end, q, k_new, v_new, out, lse, chunk_rows,
                             scratch, kStaticScratchBytes, st, /*clear_status=*/true);
  if (s != XKV_OK) return s;
  if (status_out != nullptr &&
      cudaMemcpyAsync(status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return XKV_ERR_CUDA;
  return XKV_OK;
}

}  // namespace xkv
