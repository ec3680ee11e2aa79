// Window-logit passes of xkv_score on the 5th-generation tensor cores (tcgen05) with TMEM accumulators.
//
// A work item is (unit = (sequence, KV head), split of the key axis).  One persistent CTA per SM streams
// its items' keys through a four-stage shared-memory ring filled by TMA (128-byte swizzled, K-major tiles
// of 128 keys); a one-lane MMA warp issues tcgen05.mma per landed tile into one of two TMEM accumulator
// buffers while four epilogue warps reduce the previous tile out of the other; stages and accumulators
// are handed around with mbarriers (tcgen05.commit on the MMA side).  Two launches with a small merge of
// the row statistics in between:
//   pass 1  D[query rows x keys] = Q K^T with the G*W query rows on the MMA's M axis: a thread owns one
//           TMEM lane = one query row, so the running (max, sum of exponentials) of the softmax is two
//           registers and needs no cross-lane traffic.  With fewer than 128 query rows the rows are
//           replicated over the four lane quarters and every warp takes a quarter of the key columns.
//   pass 2  D[keys x query rows] = K Q^T with the keys on M: a thread owns one key and sums
//           exp2(s*c - normaliser[row]) over the query rows straight out of TMEM -> column score u[key].
//           Items are walked in reverse so that the keys pass 1 streamed last are re-read from L2.
// No CTA ever waits for another one; every mbarrier wait is bounded.
#include <atomic>

#include "tc_common.cuh"

namespace xkv {
namespace {

using namespace tc;

// ---------------------------------------------------------------------------------------------
// Kernel: warp-specialised pipeline
//   warp 8 (one lane)  producer: TMA loads of the query rows of an item and of its key tiles into a ring
//   warp 9 (one lane)  MMA issuer: tcgen05.mma per landed tile into one of two TMEM accumulator buffers;
//                      tcgen05.commit hands the ring stage back to the producer and the accumulator to the
//                      epilogue
//   warps 0-7          epilogue, two groups of four warps: group e owns accumulator buffer e (every other
//                      tile), reduces it out of TMEM and hands it back
// Work items are assigned statically (item = CTA + n * grid), so each role walks the same sequence on its
// own and the producer runs ahead across item boundaries.
// ---------------------------------------------------------------------------------------------
struct ItemShape {
  int unit, split, b, g, cu, t, P, key_begin, key_end, n_tiles;
};

// Item n of this CTA; returns false when the sequence is exhausted.  Empty items have n_tiles == 0.  Items are
// numbered split-major (all units' split 0, then all units' split 1, ...): with ragged lengths the empty items
// are the high splits of short sequences, and this order gives every CTA the same share of every split level.
template <int PASS>
__device__ __forceinline__ bool item_shape(const ScoreParams& p, int n, ItemShape* it) {
  int idx = blockIdx.x + n * gridDim.x;
  if (idx >= p.n_work) return false;
  if (PASS == 2) idx = p.n_work - 1 - idx;       // reverse: the keys pass 1 read last are still in L2
  const int units = p.batch * p.n_kv_heads;
  it->unit = idx % units;
  it->split = idx / units;
  it->b = it->unit / p.n_kv_heads;
  it->g = it->unit % p.n_kv_heads;
  it->cu = p.cu_seqlens[it->b];
  it->t = min(p.cu_seqlens[it->b + 1] - it->cu, p.max_seqlen);
  it->P = max(it->t - p.window, 0);
  it->key_begin = it->split * p.split_keys;
  it->key_end = min(it->key_begin + p.split_keys, PASS == 1 ? it->t : it->P);
  it->n_tiles = it->key_end > it->key_begin ? (it->key_end - it->key_begin + kTcKeyTile - 1) / kTcKeyTile : 0;
  return true;
}

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
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t gt = 0, it = 0;
      ItemShape sh;
      bool ok = true;
      for (int n = 0; ok && item_shape<PASS>(p, n, &sh); ++n) {
        if (sh.n_tiles == 0) continue;
        const uint32_t qb = it % C::kQBufs;
        ok = ws_wait(&qempty_bar[qb], ((it / C::kQBufs) & 1u) ^ 1u, s_abort, p.wait_ns);
        if (!ok) break;
        mbar_arrive_expect_tx(&qfull_bar[qb], C::kQTxBytes + (PASS == 2 ? (uint32_t)(M * 4) : 0u));
        if (PASS == 2)     // the item's row normalisers ride on the same barrier; slot reuse distance is four items
          bulk_load_1d(s_mrow + (it % kMrowSlots) * 256, p.mrow + (size_t)sh.unit * M, M * 4, &qfull_bar[qb]);
        const int qrow0 = (sh.b * p.n_q_heads + sh.g * p.group) * p.window;
#pragma unroll
        for (int rep = 0; rep < C::kRep; ++rep)
#pragma unroll
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_2d(q_s + (size_t)qb * C::kQBytes + hf * C::kQHalfBytes + rep * M * 128, &tmap_q, hf * 64, qrow0,
                        &qfull_bar[qb]);
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
        ++it;
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t gt = 0, it = 0;
      ItemShape sh;
      bool ok = true;
      const uint32_t q_base = smem_u32(q_s), k_base = smem_u32(k_s);
      for (int n = 0; ok && item_shape<PASS>(p, n, &sh); ++n) {
        if (sh.n_tiles == 0) continue;
        const uint32_t qb = it % C::kQBufs;
        ok = ws_wait(&qfull_bar[qb], (it / C::kQBufs) & 1u, s_abort, p.wait_ns);
        if (!ok) break;
        // One descriptor per operand buffer; a k-step (16 bf16 = 32 bytes inside the swizzled 128-byte row, the
        // next 64 columns one half-tile further) only moves the start-address field, which is in 16-byte units
        // and cannot carry out of its 14 bits for addresses inside shared memory.
        const uint64_t q_desc = umma_desc_k128(q_base + qb * C::kQBytes);
        for (int ti = 0; ti < sh.n_tiles; ++ti, ++gt) {
          const uint32_t s = gt % kWsStages, ab = gt % kAccBufs;
          ok = ws_wait(&full_bar[s], (gt / kWsStages) & 1u, s_abort, p.wait_ns) &&
               ws_wait(&accempty_bar[ab], ((gt / kAccBufs) & 1u) ^ 1u, s_abort, p.wait_ns);
          if (!ok) break;
          tc_fence_after_sync();
          const uint64_t k_desc = umma_desc_k128(k_base + s * C::kKTileBytes);
          const uint32_t d_tmem = tmem_base + ab * C::kBufCols;
#pragma unroll
          for (int k = 0; k < C::kSteps; ++k) {
            const uint64_t kd = k_desc + (uint64_t)(((k / 4) * C::kKHalfBytes + (k % 4) * 32) >> 4);
            const uint64_t qd = q_desc + (uint64_t)(((k / 4) * C::kQHalfBytes + (k % 4) * 32) >> 4);
            if (PASS == 1) {
#pragma unroll
              for (int rb = 0; rb < (M == 256 ? 2 : 1); ++rb)
                umma_bf16(d_tmem + rb * 128u, qd + (uint64_t)((rb * 128 * 128) >> 4), kd, umma_idesc(128, kTcKeyTile),
                          k > 0 ? 1u : 0u);
            } else {
              umma_bf16(d_tmem, kd, qd, umma_idesc(kTcKeyTile, M), k > 0 ? 1u : 0u);
            }
          }
          umma_commit(&empty_bar[s]);         // the ring stage is free once these MMAs have read it
          umma_commit(&accfull_bar[ab]);      // and the accumulator is complete
        }
        if (!ok) break;
        umma_commit(&qempty_bar[qb]);         // all MMAs of the item have read the query rows
        ++it;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 0..7
    const uint32_t group = warp >> 2;                                       // owns accumulator buffer `group`
    const int etid = tid & (kEpiThreads - 1);                               // thread within the group = TMEM lane
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);   // this warp's quarter of the lanes
    constexpr int kEntries = M < 128 ? 128 : M;                             // statistics entries per item
    uint32_t gt = 0, it = 0;
    ItemShape sh;
    bool ok = true;
    for (int n = 0; ok && item_shape<PASS>(p, n, &sh); ++n, ++it) {
      if (sh.n_tiles == 0) {
        --it;                                      // empty items are not counted (same rule in every role)
        continue;
      }
      float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;   // second pair: row tid+128 when M == 256
      const int limit0 = sh.t - p.window + ((etid % M) % p.window);
      const int limit1 = sh.t - p.window + ((etid + 128) % p.window);
      const int col_begin = M < 128 ? (etid / M) * C::kColsPerThread : 0;
      float* u = p.u + (size_t)sh.g * p.total_tokens + sh.cu;
      // landed before the MMA warp issued the item's first tile, whose completion this group waits for below
      const float4* mrow4 = reinterpret_cast<const float4*>(s_mrow + (it % kMrowSlots) * 256);
      for (int ti = 0; ti < sh.n_tiles; ++ti, ++gt) {
        const uint32_t ab = gt % kAccBufs;
        if (ab != group) continue;               // the other group's tile
        ok = __all_sync(0xffffffffu, ws_wait(&accfull_bar[ab], (gt / kAccBufs) & 1u, s_abort, p.wait_ns));
        if (!ok) break;
        tc_fence_after_sync();
        const int tile_c0 = sh.key_begin + ti * kTcKeyTile;
        const uint32_t acc_addr = tmem_lane + ab * C::kBufCols;
        if (PASS == 1) {
          const bool masked = tile_c0 + kTcKeyTile > sh.t - p.window;
          if (C::kColsPerThread == 32) {
            float v[32];
            tmem_ld32(acc_addr + (uint32_t)col_begin, v);
            tmem_wait_ld();
            p1_update(v, masked, tile_c0 + col_begin, limit0, p.scale_log2, m0, l0);
          } else {
#pragma unroll
            for (int cc = 0; cc < C::kColsPerThread; cc += 64) {      // two TMEM loads in flight
              float va[32], vb[32];
              tmem_ld32(acc_addr + (uint32_t)(col_begin + cc), va);
              tmem_ld32(acc_addr + (uint32_t)(col_begin + cc + 32), vb);
              tmem_wait_ld();
              p1_update(va, masked, tile_c0 + col_begin + cc, limit0, p.scale_log2, m0, l0);
              p1_update(vb, masked, tile_c0 + col_begin + cc + 32, limit0, p.scale_log2, m0, l0);
            }
          }
          if (M == 256) {
#pragma unroll
            for (int cc = 0; cc < 128; cc += 64) {
              float va[32], vb[32];
              tmem_ld32(acc_addr + 128u + (uint32_t)cc, va);
              tmem_ld32(acc_addr + 128u + (uint32_t)(cc + 32), vb);
              tmem_wait_ld();
              p1_update(va, masked, tile_c0 + cc, limit1, p.scale_log2, m1, l1);
              p1_update(vb, masked, tile_c0 + cc + 32, limit1, p.scale_log2, m1, l1);
            }
          }
        } else {
          float acc = 0.f;
          auto add_chunk = [&](const float (&v)[32], int cc) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float4 mr = mrow4[(cc + i) >> 2];              // same address in every thread: a broadcast
              acc += fast_exp2(fmaf(v[i + 0], p.scale_log2, -mr.x)) + fast_exp2(fmaf(v[i + 1], p.scale_log2, -mr.y)) +
                     fast_exp2(fmaf(v[i + 2], p.scale_log2, -mr.z)) + fast_exp2(fmaf(v[i + 3], p.scale_log2, -mr.w));
            }
          };
          if (M == 32) {
            float v[32];
            tmem_ld32(acc_addr, v);
            tmem_wait_ld();
            add_chunk(v, 0);
          } else {
#pragma unroll
            for (int cc = 0; cc < M; cc += 64) {                    // two TMEM loads in flight
              float va[32], vb[32];
              tmem_ld32(acc_addr + (uint32_t)cc, va);
              tmem_ld32(acc_addr + (uint32_t)(cc + 32), vb);
              tmem_wait_ld();
              add_chunk(va, cc);
              add_chunk(vb, cc + 32);
            }
          }
          const int key = tile_c0 + etid;
          if (key < sh.key_end) u[key] = acc;
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&accempty_bar[ab]);
      }
      if (!ok) break;
      if (PASS == 1) {
        // every thread stores the statistics of its own (row, key-column quarter); tc_merge_kernel combines them
        float2* out = p.stats_part + (((size_t)sh.unit * p.n_splits + sh.split) * kAccBufs + group) * kEntries;
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
  const int per_split = kAccBufs * group_reps;               // partial statistics of this row per split
  const int entries = kAccBufs * group_entries;
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
  int tiles = M == 256 ? 16 : 4;      // G*W = 256 reloads a 64 KB query block per item: make items larger
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
  const int n_part = p.n_splits * kAccBufs * (M < 128 ? 128 / M : 1);
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
