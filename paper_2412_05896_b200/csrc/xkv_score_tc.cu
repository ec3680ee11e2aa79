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
#include <cuda.h>

#include <cmath>
#include <mutex>

#include "common.cuh"
#include "score_params.h"

namespace xkv {
namespace {

constexpr int kTcThreads = 128;
constexpr int kTcKeyTile = 128;                 // keys per MMA tile

// ---------------------------------------------------------------------------------------------
// tcgen05 / TMEM wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 inputs, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t"
      "}\n" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// mbarrier arrives once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane; the values may be used after tmem_wait_ld().
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major operand stored as rows of 128 bytes (64 bf16) with the
// 128-byte swizzle, eight-row groups 1024 bytes apart (what a TMA box {64, rows} with SWIZZLE_128B writes).
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: next eight-row group
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void tma_load_3d(void* dst, const void* tmap, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// Plain (untiled) bulk copy global -> shared; both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ uint64_t tc_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded mbarrier wait: two seconds at most.
__device__ __forceinline__ bool tc_mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = tc_timer_ns();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (tc_timer_ns() - t0 > 2000000000ull) return false;
  }
}
__device__ __forceinline__ int tc_ld_acquire(const int* ptr) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

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
constexpr int kWsThreads = 320;
constexpr int kEpiThreads = 128;     // threads of one epilogue group
constexpr int kWsStages = 4;       // shared-memory ring of key tiles
constexpr int kAccBufs = 2;        // TMEM accumulator buffers
constexpr int kMrowSlots = 4;      // pass 2: ring of row-normaliser vectors (one per item in flight)

template <int D, int M>
struct TcCfg {
  static constexpr int kHalves = D / 64;                         // 128-byte swizzled K segments per row
  static constexpr int kSteps = D / 16;                          // MMA k-steps per tile
  static constexpr int kQRows = M < 128 ? 128 : M;               // rows of the query operand buffer
  static constexpr int kRep = M < 128 ? 128 / M : 1;             // replicas of the query rows across lanes
  static constexpr int kQHalfBytes = kQRows * 128;
  static constexpr int kQBytes = kHalves * kQHalfBytes;
  static constexpr int kQBufs = M == 256 ? 1 : 2;
  static constexpr int kKHalfBytes = kTcKeyTile * 128;
  static constexpr int kKTileBytes = kHalves * kKHalfBytes;
  static constexpr uint32_t kBufCols = M == 256 ? 256 : 128;     // TMEM columns of one accumulator buffer
  static constexpr uint32_t kTmemCols = kAccBufs * kBufCols;
  static constexpr int kColsPerThread = M < 128 ? M : 128;       // pass-1 key columns a thread reduces per tile
  static constexpr uint32_t kQTxBytes = (uint32_t)(kRep * kHalves * (M < 128 ? M : kQRows) * 128);
  static constexpr size_t kSmemBytes = 1024 + (size_t)kQBufs * kQBytes + (size_t)kWsStages * kKTileBytes +
                                       kMrowSlots * 256 * 4 /*row normalisers*/ + 256 /*barriers*/;
};

__device__ __forceinline__ void p1_update(const float (&v)[32], bool masked, int c0, int limit, float scale,
                                          float& m, float& l) {
  float x[32];
  float vmax = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    x[i] = (masked && c0 + i > limit) ? -INFINITY : v[i];
    vmax = fmaxf(vmax, x[i]);
  }
  const float m_new = fmaxf(m, vmax * scale);
  const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) sum += fast_exp2(fmaf(x[i], scale, -m_ref));
  l = l * fast_exp2(m - m_ref) + sum;
  m = m_new;
}

struct ItemShape {
  int unit, split, b, g, cu, t, P, key_begin, key_end, n_tiles;
};

// Item n of this CTA; returns false when the sequence is exhausted.  Empty items have n_tiles == 0.
template <int PASS>
__device__ __forceinline__ bool item_shape(const ScoreParams& p, int n, ItemShape* it) {
  int idx = blockIdx.x + n * gridDim.x;
  if (idx >= p.n_work) return false;
  if (PASS == 2) idx = p.n_work - 1 - idx;       // reverse: the keys pass 1 read last are still in L2
  it->unit = idx / p.n_splits;
  it->split = idx % p.n_splits;
  it->b = it->unit / p.n_kv_heads;
  it->g = it->unit % p.n_kv_heads;
  it->cu = p.cu_seqlens[it->b];
  it->t = p.cu_seqlens[it->b + 1] - it->cu;
  it->P = max(it->t - p.window, 0);
  it->key_begin = it->split * p.split_keys;
  it->key_end = min(it->key_begin + p.split_keys, PASS == 1 ? it->t : it->P);
  it->n_tiles = it->key_end > it->key_begin ? (it->key_end - it->key_begin + kTcKeyTile - 1) / kTcKeyTile : 0;
  return true;
}

// Bounded mbarrier wait (two seconds) that also gives up when another role has raised the abort flag.
__device__ __forceinline__ bool ws_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = tc_timer_ns();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (tc_timer_ns() - t0 > 2000000000ull) {
      *abort_flag = 1;
      return false;
    }
  }
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
        ok = ws_wait(&qempty_bar[qb], ((it / C::kQBufs) & 1u) ^ 1u, s_abort);
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
          ok = ws_wait(&empty_bar[s], ((gt / kWsStages) & 1u) ^ 1u, s_abort);
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
        ok = ws_wait(&qfull_bar[qb], (it / C::kQBufs) & 1u, s_abort);
        if (!ok) break;
        const uint32_t qa = q_base + qb * C::kQBytes;
        for (int ti = 0; ti < sh.n_tiles; ++ti, ++gt) {
          const uint32_t s = gt % kWsStages, ab = gt % kAccBufs;
          ok = ws_wait(&full_bar[s], (gt / kWsStages) & 1u, s_abort) &&
               ws_wait(&accempty_bar[ab], ((gt / kAccBufs) & 1u) ^ 1u, s_abort);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t kt = k_base + s * C::kKTileBytes;
          const uint32_t d_tmem = tmem_base + ab * C::kBufCols;
#pragma unroll
          for (int k = 0; k < C::kSteps; ++k) {
            const uint32_t ko = (uint32_t)(k % 4) * 32u;      // 16 bf16 along K inside the swizzled 128-byte row
            const uint64_t kd = umma_desc_k128(kt + (k / 4) * C::kKHalfBytes + ko);
            if (PASS == 1) {
#pragma unroll
              for (int rb = 0; rb < (M == 256 ? 2 : 1); ++rb) {
                const uint64_t qd = umma_desc_k128(qa + (k / 4) * C::kQHalfBytes + rb * 128 * 128 + ko);
                umma_bf16(d_tmem + rb * 128u, qd, kd, umma_idesc(128, kTcKeyTile), k > 0 ? 1u : 0u);
              }
            } else {
              const uint64_t qd = umma_desc_k128(qa + (k / 4) * C::kQHalfBytes + ko);
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
        ok = __all_sync(0xffffffffu, ws_wait(&accfull_bar[ab], (gt / kAccBufs) & 1u, s_abort));
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

// One warp per query row of a unit: mrow[r] = m_r + log2(l_r) (log2 domain; +inf for rows without visible
// keys) from the per-split, per-group, per-replica statistics pass 1 stored.  grid = (units, M / 4).
__global__ void __launch_bounds__(128) tc_merge_kernel(const ScoreParams p) {
  const int unit = blockIdx.x;
  const int M = p.M;
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.y * 4 + (threadIdx.x >> 5);
  if (r >= M) return;
  const int group_entries = M < 128 ? 128 : M;
  const int group_reps = M < 128 ? 128 / M : 1;
  const int per_split = kAccBufs * group_reps;               // partial statistics of this row per split
  const int entries = kAccBufs * group_entries;
  const int b = unit / p.n_kv_heads;
  const int t = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
  const int n_splits_u = (t + p.split_keys - 1) / p.split_keys;
  const float2* part = p.stats_part + (size_t)unit * p.n_splits * entries + r;
  float m = -INFINITY, l = 0.f;
  for (int i = lane; i < n_splits_u * per_split; i += 32) {
    const int s = i / per_split, q = i % per_split;
    const float2 v = part[(size_t)s * entries + (q / group_reps) * group_entries + (q % group_reps) * M];
    const float m_new = fmaxf(m, v.x);
    const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
    l = l * exp2f(m - m_ref) + v.y * exp2f(v.x - m_ref);
    m = m_new;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float mo = __shfl_xor_sync(0xffffffffu, m, o), lo = __shfl_xor_sync(0xffffffffu, l, o);
    const float m_new = fmaxf(m, mo);
    const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
    l = l * exp2f(m - m_ref) + lo * exp2f(mo - m_ref);
    m = m_new;
  }
  if (lane == 0) p.mrow[(size_t)unit * M + r] = (l > 0.f) ? m + log2f(l) : INFINITY;
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tc_encode_fn() {
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

bool tc_make_tmap(CUtensorMap* tmap, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                  const cuuint32_t* box) {
  EncodeTiledFn enc = tc_encode_fn();
  if (enc == nullptr) return false;
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return enc(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box,
             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

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
  static bool done[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  if (!done[dev]) {
    if (cudaFuncSetAttribute(score_tc_kernel<D, M, PASS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             227 * 1024) != cudaSuccess)
      return XKV_ERR_CUDA;
    done[dev] = true;
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
  tc_merge_kernel<<<dim3(p.batch * p.n_kv_heads, M / 4), 128, 0, st>>>(p);
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

xkv_status score_tc_passes(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st) {
  const int units = p.batch * p.n_kv_heads;
  const int tiles = tc_tiles(p.M, head_dim, units, max_seqlen);
  if (tiles == 0 || tiles * kTcKeyTile != p.split_keys) return XKV_ERR_UNSUPPORTED;
  CUtensorMap tq, tk;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)head_dim, (cuuint64_t)p.batch * p.n_q_heads * p.window};
    const cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
    const cuuint32_t box[2] = {64u, (cuuint32_t)p.M};
    if (!tc_make_tmap(&tq, p.q_win, 2, dims, strides, box)) return XKV_ERR_CUDA;
  }
  {
    const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)p.n_kv_heads, (cuuint64_t)p.total_tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)p.stride_head * 2, (cuuint64_t)p.stride_token * 2};
    const cuuint32_t box[3] = {64u, 1u, (cuuint32_t)kTcKeyTile};
    if (!tc_make_tmap(&tk, p.k, 3, dims, strides, box)) return XKV_ERR_CUDA;
  }
#define XKV_TC_CASE(DD, MM) \
  if (head_dim == DD && p.M == MM) return tc_launch_both<DD, MM>(tq, tk, p, st);
  XKV_TC_CASE(128, 32) XKV_TC_CASE(128, 64) XKV_TC_CASE(128, 128) XKV_TC_CASE(128, 256)
  XKV_TC_CASE(64, 32) XKV_TC_CASE(64, 64) XKV_TC_CASE(64, 128) XKV_TC_CASE(64, 256)
#undef XKV_TC_CASE
  return XKV_ERR_UNSUPPORTED;
}

}  // namespace xkv
