// Window-logit passes of xkv_score on the 5th-generation tensor cores (tcgen05) with TMEM accumulators.
//
// A work item is (unit = (sequence, KV head), split of the key axis).  One persistent CTA per SM streams
// its items' keys through a four-stage shared-memory ring filled by TMA (128-byte swizzled, K-major tiles
// of 128 keys); a one-lane MMA warp issues tcgen05.mma per landed tile into one of four 128-column TMEM
// accumulator buffers (a tile with 256 query rows takes two, one per half of the rows) while two groups of
// four epilogue warps reduce earlier tiles out of the others: a group's next accumulator is filled while it
// works on the current one; stages and accumulators are handed around with mbarriers (tcgen05.commit on
// the MMA side).  Two launches with a small merge of
// the row statistics in between:
//   pass 1  D[query rows x keys] = Q K^T with the G*W query rows on the MMA's M axis: a thread owns one
//           TMEM lane = one query row, so the running (max, sum of exponentials) of the softmax is two
//           registers and needs no cross-lane traffic.  With fewer than 128 query rows the rows are
//           replicated over the four lane quarters and every warp takes a quarter of the key columns.
//   pass 2  D[keys x query rows] = K Q^T with the keys on M: a thread owns one key and sums
//           exp2(s*c - normaliser[row]) over the query rows straight out of TMEM -> column score u[key].
//           Every CTA walks its run of items backwards so that the keys pass 1 streamed last are re-read from L2.
// No CTA ever waits for another one; every mbarrier wait is bounded.
#include <atomic>

#include "tc_common.cuh"

namespace xkv {
namespace {

using namespace tc;

// ---------------------------------------------------------------------------------------------
// Kernel: warp-specialised pipeline
//   warp 8 (one lane)  producer: TMA loads of the query rows of an item and of its key tiles into a ring
//   warp 9 (one lane)  MMA issuer: tcgen05.mma per landed tile into the next of four TMEM accumulator
//                      buffers; tcgen05.commit hands the ring stage back to the producer and the accumulator
//                      to the epilogue
//   warps 0-7          epilogue, two groups of four warps: group e takes every other tile, reduces its
//                      accumulator(s) out of TMEM and hands them back
// Work items are assigned statically (a contiguous run of items per CTA), so each role walks the same sequence
// on its own and the producer runs ahead across item boundaries.
// ---------------------------------------------------------------------------------------------
struct ItemShape {
  int unit, split, b, g, cu, t, P, key_begin, key_end, n_tiles;
  bool new_unit;       // the query rows (and row normalisers) of this item's unit are not the previous item's
  bool last_of_unit;   // the next item of this CTA, if any, belongs to another unit
};

// The CTA's share of the work: a contiguous run of the non-empty items in (sequence, KV head, split) order, found
// once per CTA by one warp.  Consecutive items then mostly share their unit, so its query rows are loaded once,
// and the shares differ by at most one item whatever the lengths are.
struct WalkStart {
  int b, g, split, count;
};

// Splits of sequence b in this pass: pass 1 covers all t keys (the window rows see window keys), pass 2 the prefix.
template <int PASS>
__device__ __forceinline__ int seq_splits(const ScoreParams& p, int b, int* cu_out, int* t_out) {
  const int cu = p.cu_seqlens[b];
  const int t = min(p.cu_seqlens[b + 1] - cu, p.max_seqlen);
  if (cu_out != nullptr) *cu_out = cu;
  if (t_out != nullptr) *t_out = t;
  const int len = PASS == 1 ? t : max(t - p.window, 0);
  return (len + p.split_keys - 1) / p.split_keys;
}

// Called by one whole warp.  Items are numbered sequence-major, then KV head, then split; this CTA takes items
// [first, last) with first = cta * N / grid.  Pass 1 walks its run forwards, pass 2 backwards from last - 1 (the keys
// pass 1 streamed last are then re-read from L2), so the start is the position of item first or last - 1.
template <int PASS>
__device__ __forceinline__ void walk_start(const ScoreParams& p, WalkStart* out) {
  const int lane = threadIdx.x & 31;
  long long total = 0;
  for (int base = 0; base < p.batch; base += 32) {
    int n = base + lane < p.batch ? seq_splits<PASS>(p, base + lane, nullptr, nullptr) : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    total += n;
  }
  total *= p.n_kv_heads;
  const long long first = total * blockIdx.x / gridDim.x, last = total * (blockIdx.x + 1) / gridDim.x;
  WalkStart w = {0, 0, 0, (int)(last - first)};
  if (w.count > 0) {
    const long long want = PASS == 1 ? first : last - 1;
    long long before = 0;
    for (int base = 0; base < p.batch; base += 32) {
      const int n = base + lane < p.batch ? seq_splits<PASS>(p, base + lane, nullptr, nullptr) * p.n_kv_heads : 0;
      int incl = n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, want < before + incl);
      if (hit != 0u) {
        const int src = __ffs(hit) - 1;
        const int n_src = __shfl_sync(0xffffffffu, n, src) / p.n_kv_heads;       // splits of that sequence
        const int rem = (int)(want - before - __shfl_sync(0xffffffffu, incl - n, src));
        w.b = base + src;
        w.g = rem / n_src;
        w.split = rem % n_src;
        break;
      }
      before += __shfl_sync(0xffffffffu, incl, 31);
    }
  }
  if (lane == 0) *out = w;
}

// Steps through the CTA's items; every role keeps a walker of its own and they all see the same sequence.
template <int PASS>
struct ItemWalker {
  int b, g, split, n_b, cu, t, left;
  bool fresh;       // no item handed out yet: the first one always starts a unit

  __device__ __forceinline__ void init(const ScoreParams& p, const WalkStart& w) {
    b = w.b;
    g = w.g;
    split = w.split;
    left = w.count;
    fresh = true;
    n_b = left > 0 ? seq_splits<PASS>(p, b, &cu, &t) : 0;
  }

  __device__ __forceinline__ bool next(const ScoreParams& p, ItemShape* it) {
    if (left <= 0) return false;
    it->b = b;
    it->g = g;
    it->unit = b * p.n_kv_heads + g;
    it->split = split;
    it->cu = cu;
    it->t = t;
    it->P = max(t - p.window, 0);
    it->key_begin = split * p.split_keys;
    it->key_end = min(it->key_begin + p.split_keys, PASS == 1 ? t : it->P);
    it->n_tiles = (it->key_end - it->key_begin + kTcKeyTile - 1) / kTcKeyTile;      // at least one: empty items are not numbered
    it->new_unit = fresh || (PASS == 1 ? split == 0 : split == n_b - 1);
    fresh = false;
    --left;
    // advance to the following item
    bool same_unit;
    if (PASS == 1) {
      same_unit = split + 1 < n_b;
      if (same_unit) {
        ++split;
      } else if (g + 1 < p.n_kv_heads) {
        ++g;
        split = 0;
      } else if (left > 0) {
        do {
          ++b;
          n_b = seq_splits<PASS>(p, b, &cu, &t);
        } while (n_b == 0);
        g = 0;
        split = 0;
      }
    } else {
      same_unit = split > 0;
      if (same_unit) {
        --split;
      } else if (g > 0) {
        --g;
        split = n_b - 1;
      } else if (left > 0) {
        do {
          --b;
          n_b = seq_splits<PASS>(p, b, &cu, &t);
        } while (n_b == 0);
        g = p.n_kv_heads - 1;
        split = n_b - 1;
      }
    }
    it->last_of_unit = left == 0 || !same_unit;
    return true;
  }
};

template <int D, int M, int PASS>
__global__ void __launch_bounds__(kWsThreads) score_tc_kernel(const __grid_constant__ CUtensorMap tmap_q,
                                                             const __grid_constant__ CUtensorMap tmap_k,
                                                             const ScoreParams p) {
  using C = TcCfg<D, M>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* k_s = q_s + (size_t)C::kQBufs * C::kQBytes;
  float* s_mrow = reinterpret_cast<float*>(k_s + (size_t)kWsStages * C::kKTileBytes);   // [kMrowSlots][256]
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(s_mrow + kMrowSlots * 256);   // [kWsStages] tile landed
  uint64_t* empty_bar = full_bar + kWsStages;                        // [kWsStages] tile consumed by the MMAs
  uint64_t* qfull_bar = empty_bar + kWsStages;                       // [2] query rows landed
  uint64_t* qempty_bar = qfull_bar + 2;                              // [2] query rows no longer read
  uint64_t* accfull_bar = qempty_bar + 2;                            // [kAccBufs] accumulator complete
  uint64_t* accempty_bar = accfull_bar + kAccBufs;                   // [kAccBufs] accumulator reduced
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(accempty_bar + kAccBufs);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  WalkStart* s_walk = reinterpret_cast<WalkStart*>(s_tmem + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < kWsStages; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&qfull_bar[i], 1);
      mbar_init(&qempty_bar[i], 1);
    }
    for (int i = 0; i < kAccBufs; ++i) {
      mbar_init(&accfull_bar[i], 1);
      mbar_init(&accempty_bar[i], 4);          // one arrival per warp of the owning epilogue group
    }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_k);
  }
  if (warp == 0) {
    tmem_alloc(s_tmem, C::kTmemCols);
    tmem_relinquish();
  }
  if (warp == 1) walk_start<PASS>(p, s_walk);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  ItemWalker<PASS> walk;
  walk.init(p, *s_walk);

  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t gt = 0, uc = 0;              // tiles issued; units started (one query-row buffer each)
      ItemShape sh;
      bool ok = true;
      while (ok && walk.next(p, &sh)) {
        if (sh.new_unit) {
          const uint32_t qb = uc % C::kQBufs;
          ok = ws_wait(&qempty_bar[qb], ((uc / C::kQBufs) & 1u) ^ 1u, s_abort, p.wait_ns);
          if (!ok) break;
          mbar_arrive_expect_tx(&qfull_bar[qb], C::kQTxBytes + (PASS == 2 ? (uint32_t)(M * 4) : 0u));
          if (PASS == 2)     // the unit's row normalisers ride on the same barrier; slot reuse distance is four units
            bulk_load_1d(s_mrow + (uc % kMrowSlots) * 256, p.mrow + (size_t)sh.unit * M, M * 4, &qfull_bar[qb]);
          const int qrow0 = (sh.b * p.n_q_heads + sh.g * p.group) * p.window;
#pragma unroll
          for (int rep = 0; rep < C::kRep; ++rep)
#pragma unroll
            for (int hf = 0; hf < C::kHalves; ++hf)
              tma_load_2d(q_s + (size_t)qb * C::kQBytes + hf * C::kQHalfBytes + rep * M * 128, &tmap_q, hf * 64, qrow0,
                          &qfull_bar[qb]);
          ++uc;
        }
        for (int ti = 0; ti < sh.n_tiles; ++ti, ++gt) {
          const uint32_t s = gt % kWsStages;
          ok = ws_wait(&empty_bar[s], ((gt / kWsStages) & 1u) ^ 1u, s_abort, p.wait_ns);
          if (!ok) break;
          mbar_arrive_expect_tx(&full_bar[s], (uint32_t)C::kKTileBytes);
#pragma unroll
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_3d(k_s + (size_t)s * C::kKTileBytes + hf * C::kKHalfBytes, &tmap_k, hf * 64, sh.g,
                        sh.cu + sh.key_begin + ti * kTcKeyTile, &full_bar[s]);
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t gt = 0, uc = 0;
      ItemShape sh;
      bool ok = true;
      const uint32_t q_base = smem_u32(q_s), k_base = smem_u32(k_s);
      uint32_t qb = 0;
      uint64_t q_desc = 0;
      while (ok && walk.next(p, &sh)) {
        if (sh.new_unit) {
          qb = uc % C::kQBufs;
          ok = ws_wait(&qfull_bar[qb], (uc / C::kQBufs) & 1u, s_abort, p.wait_ns);
          if (!ok) break;
          // One descriptor per operand buffer; a k-step (16 bf16 = 32 bytes inside the swizzled 128-byte row, the
          // next 64 columns one half-tile further) only moves the start-address field, which is in 16-byte units
          // and cannot carry out of its 14 bits for addresses inside shared memory.
          q_desc = umma_desc_k128(q_base + qb * C::kQBytes);
          ++uc;
        }
        for (int ti = 0; ti < sh.n_tiles; ++ti, ++gt) {
          const uint32_t s = gt % kWsStages;
          ok = ws_wait(&full_bar[s], (gt / kWsStages) & 1u, s_abort, p.wait_ns);
          if (!ok) break;
          const uint64_t k_desc = umma_desc_k128(k_base + s * C::kKTileBytes);
          // a tile is one accumulator job of 128 columns, or two with 256 query rows (one per half of the rows)
#pragma unroll
          for (int half = 0; half < C::kJobs; ++half) {
            const uint32_t job = gt * C::kJobs + half, ab = job % kAccBufs;
            ok = ws_wait(&accempty_bar[ab], ((job / kAccBufs) & 1u) ^ 1u, s_abort, p.wait_ns);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + ab * C::kBufCols;
            const uint64_t q_half = q_desc + (uint64_t)((half * 128 * 128) >> 4);     // rows 128*half .. of the query block
#pragma unroll
            for (int k = 0; k < C::kSteps; ++k) {
              const uint64_t kd = k_desc + (uint64_t)(((k / 4) * C::kKHalfBytes + (k % 4) * 32) >> 4);
              const uint64_t qd = q_half + (uint64_t)(((k / 4) * C::kQHalfBytes + (k % 4) * 32) >> 4);
              if (PASS == 1)
                umma_bf16(d_tmem, qd, kd, umma_idesc(128, kTcKeyTile), k > 0 ? 1u : 0u);
              else
                umma_bf16(d_tmem, kd, qd, umma_idesc(kTcKeyTile, C::kJobRows), k > 0 ? 1u : 0u);
            }
            umma_commit(&accfull_bar[ab]);    // this job's accumulator is complete
          }
          if (!ok) break;
          umma_commit(&empty_bar[s]);         // the ring stage is free once the tile's MMAs have read it
        }
        if (!ok) break;
        if (sh.last_of_unit) umma_commit(&qempty_bar[qb]);   // all MMAs of the unit have read the query rows
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 0..7
    const uint32_t group = warp >> 2;                                       // takes every other tile
    const int etid = tid & (kEpiThreads - 1);                               // thread within the group = TMEM lane
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);   // this warp's quarter of the lanes
    constexpr int kEntries = M < 128 ? 128 : M;                             // statistics entries per item
    uint32_t gt = 0, uc = 0;
    ItemShape sh;
    bool ok = true;
    while (ok && walk.next(p, &sh)) {
      if (sh.new_unit) ++uc;
      float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;   // second pair: row tid+128 when M == 256
      const int limit0 = sh.t - p.window + ((etid % M) % p.window);
      const int limit1 = sh.t - p.window + ((etid + 128) % p.window);
      const int col_begin = M < 128 ? (etid / M) * C::kColsPerThread : 0;
      float* u = p.u + (size_t)sh.g * p.total_tokens + sh.cu;
      // landed before the MMA warp issued the item's first tile, whose completion this group waits for below
      const float4* mrow4 = reinterpret_cast<const float4*>(s_mrow + ((uc - 1) % kMrowSlots) * 256);
      for (int ti = 0; ti < sh.n_tiles; ++ti, ++gt) {
        if ((gt & 1u) != group) continue;        // the other group's tile
        const int tile_c0 = sh.key_begin + ti * kTcKeyTile;
        const bool masked = tile_c0 + kTcKeyTile > sh.t - p.window;      // pass 1: the tile reaches the window
        float acc = 0.f;                                                 // pass 2: this thread's key
#pragma unroll
        for (int half = 0; half < C::kJobs; ++half) {
          const uint32_t job = gt * C::kJobs + half, ab = job % kAccBufs;
          ok = __all_sync(0xffffffffu, ws_wait(&accfull_bar[ab], (job / kAccBufs) & 1u, s_abort, p.wait_ns));
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t acc_addr = tmem_lane + ab * C::kBufCols;
          if (PASS == 1) {
            // rows etid (first half) and etid + 128 (second half, only with 256 query rows)
            float& m = half == 0 ? m0 : m1;
            float& l = half == 0 ? l0 : l1;
            const int limit = half == 0 ? limit0 : limit1;
            // all of the thread's columns of this job in flight together, one wait
            constexpr int kChunks = C::kColsPerThread / 32;
            float v[kChunks][32];
#pragma unroll
            for (int j = 0; j < kChunks; ++j) tmem_ld32(acc_addr + (uint32_t)(col_begin + 32 * j), v[j]);
            tmem_wait_ld();
            p1_update<kChunks>(v, masked, tile_c0 + col_begin, limit, p.scale_log2, m, l);
          } else {
            auto add_chunk = [&](const float (&v)[32], int row0) {
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                const float4 mr = mrow4[(row0 + i) >> 2];            // same address in every thread: a broadcast
                acc += fast_exp2(fmaf(v[i + 0], p.scale_log2, -mr.x)) + fast_exp2(fmaf(v[i + 1], p.scale_log2, -mr.y)) +
                       fast_exp2(fmaf(v[i + 2], p.scale_log2, -mr.z)) + fast_exp2(fmaf(v[i + 3], p.scale_log2, -mr.w));
              }
            };
            // all query rows of this job in flight together, one wait
            constexpr int kChunks = C::kJobRows / 32;
            float v[kChunks][32];
#pragma unroll
            for (int j = 0; j < kChunks; ++j) tmem_ld32(acc_addr + (uint32_t)(32 * j), v[j]);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < kChunks; ++j) add_chunk(v[j], half * 128 + 32 * j);
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&accempty_bar[ab]);
        }
        if (!ok) break;
        if (PASS == 2) {
          const int key = tile_c0 + etid;
          if (key < sh.key_end) u[key] = acc;
        }
      }
      if (!ok) break;
      if (PASS == 1) {
        // every thread stores the statistics of its own (row, key-column quarter); tc_merge_kernel combines them
        float2* out = p.stats_part + (((size_t)sh.unit * p.n_splits + sh.split) * kEpiGroups + group) * kEntries;
        out[etid] = make_float2(m0, l0);
        if (M == 256) out[128 + etid] = make_float2(m1, l1);
      }
    }
  }

  // ---- teardown
  __syncthreads();
  if (*s_abort) {
    if (tid == 0) record_status(p.hdr, XKV_ERR_TIMEOUT);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies and MMAs already issued finish
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, C::kTmemCols);
}

// grid = (units, M / 32), blockDim = (32 query rows, up to 32 slices): mrow[r] = m_r + log2(l_r) (log2 domain; +inf for
// rows without visible keys) from the per-split, per-group, per-replica statistics pass 1 stored.  Consecutive
// rows are consecutive in every partial vector, so a warp's load is one 256-byte segment; a slice takes every
// blockDim.y-th partial, and the slices are combined through shared memory.
__global__ void __launch_bounds__(1024) tc_merge_kernel(const ScoreParams p) {
  __shared__ float2 s_part[32][33];
  const int unit = blockIdx.x;
  const int M = p.M;
  const int rl = threadIdx.x, sl = threadIdx.y, n_sl = blockDim.y;
  const int r = blockIdx.y * 32 + rl;
  const int group_entries = M < 128 ? 128 : M;
  const int group_reps = M < 128 ? 128 / M : 1;
  const int per_split = kEpiGroups * group_reps;             // partial statistics of this row per split
  const int entries = kEpiGroups * group_entries;
  const int b = unit / p.n_kv_heads;
  const int t = min(p.cu_seqlens[b + 1] - p.cu_seqlens[b], p.max_seqlen);
  const int n_splits_u = (t + p.split_keys - 1) / p.split_keys;
  const float2* part = p.stats_part + (size_t)unit * p.n_splits * entries + r;
  const int n = n_splits_u * per_split;
  float m = -INFINITY, l = 0.f;
  auto fold = [&](float2 v) {
    const float m_new = fmaxf(m, v.x);
    const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
    l = l * exp2f(m - m_ref) + v.y * exp2f(v.x - m_ref);
    m = m_new;
  };
  auto at = [&](int i) -> const float2* {
    const int s = i / per_split, q = i % per_split;
    return part + (size_t)s * entries + (q / group_reps) * group_entries + (q % group_reps) * M;
  };
  int i = sl;
  for (; i + 3 * n_sl < n; i += 4 * n_sl) {
    const float2 v0 = __ldcg(at(i)), v1 = __ldcg(at(i + n_sl)), v2 = __ldcg(at(i + 2 * n_sl)),
                 v3 = __ldcg(at(i + 3 * n_sl));
    fold(v0);
    fold(v1);
    fold(v2);
    fold(v3);
  }
  for (; i < n; i += n_sl) fold(__ldcg(at(i)));
  s_part[sl][rl] = make_float2(m, l);
  __syncthreads();
  if (sl == 0) {
    for (int k = 1; k < n_sl; ++k) fold(s_part[k][rl]);
    p.mrow[(size_t)unit * M + r] = (l > 0.f) ? m + log2f(l) : INFINITY;
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// Key tiles per work item: items are cheap (the producer prefetches across them), so keep them small
// enough to balance the static assignment.
int tc_tiles(int M, int head_dim, int units, int max_seqlen) {
  if (M != 32 && M != 64 && M != 128 && M != 256) return 0;
  if (head_dim != 64 && head_dim != 128) return 0;
  const int sms = sm_count();
  int tiles = 4;                      // a CTA's items are contiguous, so the query rows are rarely reloaded
  while (tiles > 1 && (int64_t)units * ((max_seqlen + tiles * kTcKeyTile - 1) / (tiles * kTcKeyTile)) < 8 * sms)
    tiles >>= 1;
  return tiles;
}

template <int D, int M, int PASS>
xkv_status tc_launch(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, cudaStream_t st) {
  using C = TcCfg<D, M>;
  size_t smem = C::kSmemBytes;
  if (smem < 120 * 1024) smem = 120 * 1024;      // one CTA per SM: it may hold all 512 TMEM columns
  static std::atomic<bool> done[64];   // idempotent set-up: two threads doing it twice is harmless
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  if (!done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(score_tc_kernel<D, M, PASS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)      // the kernel also has a few KB of static shared memory
      return XKV_ERR_CUDA;
    done[dev].store(true, std::memory_order_release);
  }
  int grid = sm_count();
  if (grid > p.n_work) grid = p.n_work;
  score_tc_kernel<D, M, PASS><<<grid, kWsThreads, smem, st>>>(tq, tk, p);
  count_launch();
  return check_launch();
}

template <int D, int M>
xkv_status tc_launch_both(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, cudaStream_t st) {
  xkv_status s = tc_launch<D, M, 1>(tq, tk, p, st);
  if (s != XKV_OK) return s;
  // about four partials per slice: short sequences get small CTAs, long ones many loads in flight
  const int n_part = p.n_splits * kEpiGroups * (M < 128 ? 128 / M : 1);
  int slices = 1;
  while (slices < 32 && slices * 4 < n_part) slices <<= 1;
  tc_merge_kernel<<<dim3(p.batch * p.n_kv_heads, M / 32), dim3(32, slices), 0, st>>>(p);
  count_launch();
  s = check_launch();
  if (s != XKV_OK) return s;
  return tc_launch<D, M, 2>(tq, tk, p, st);
}

}  // namespace

int score_tc_split_keys(int M, int head_dim, int units, int max_seqlen) {
#ifdef XKV_NO_TC
  return 0;
#else
  return tc_tiles(M, head_dim, units, max_seqlen) * kTcKeyTile;
#endif
}

xkv_status score_tc_pass2(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st) {
  const int units = p.batch * p.n_kv_heads;
  const int tiles = tc_tiles(p.M, head_dim, units, max_seqlen);
  if (tiles == 0 || tiles * kTcKeyTile != p.split_keys) return XKV_ERR_UNSUPPORTED;
  CUtensorMap tq, tk;
  if (!tc_make_score_tmaps(p, head_dim, &tq, &tk)) return XKV_ERR_CUDA;
#define XKV_TC_CASE(DD, MM) \
  if (head_dim == DD && p.M == MM) return tc_launch<DD, MM, 2>(tq, tk, p, st);
  XKV_TC_CASE(128, 32) XKV_TC_CASE(128, 64) XKV_TC_CASE(128, 128) XKV_TC_CASE(128, 256)
  XKV_TC_CASE(64, 32) XKV_TC_CASE(64, 64) XKV_TC_CASE(64, 128) XKV_TC_CASE(64, 256)
#undef XKV_TC_CASE
  return XKV_ERR_UNSUPPORTED;
}

xkv_status score_tc_passes(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st) {
  const int units = p.batch * p.n_kv_heads;
  const int tiles = tc_tiles(p.M, head_dim, units, max_seqlen);
  if (tiles == 0 || tiles * kTcKeyTile != p.split_keys) return XKV_ERR_UNSUPPORTED;
  CUtensorMap tq, tk;
  if (!tc_make_score_tmaps(p, head_dim, &tq, &tk)) return XKV_ERR_CUDA;
#define XKV_TC_CASE(DD, MM) \
  if (head_dim == DD && p.M == MM) return tc_launch_both<DD, MM>(tq, tk, p, st);
  XKV_TC_CASE(128, 32) XKV_TC_CASE(128, 64) XKV_TC_CASE(128, 128) XKV_TC_CASE(128, 256)
  XKV_TC_CASE(64, 32) XKV_TC_CASE(64, 64) XKV_TC_CASE(64, 128) XKV_TC_CASE(64, 256)
#undef XKV_TC_CASE
  return XKV_ERR_UNSUPPORTED;
}

}  // namespace xkv
