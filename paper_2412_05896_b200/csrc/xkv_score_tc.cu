// Window-logit passes of xkv_score on the 5th-generation tensor cores (tcgen05) with TMEM accumulators.
//
// A work item is (unit = (sequence, KV head), split of the key axis).  Persistent CTAs take items from a
// global counter and stream the item's keys through a two-stage shared-memory ring filled by TMA
// (128-byte swizzled, K-major tiles of 128 keys); one thread issues the MMAs of a tile into one of two TMEM
// accumulator buffers while all threads reduce the previous tile out of the other; completion comes back
// through tcgen05.commit on an mbarrier.  Two launches:
//   pass 1  D[query rows x keys] = Q K^T with the G*W query rows on the MMA's M axis: a thread owns one
//           TMEM lane = one query row, so the running (max, sum of exponentials) of the softmax is two
//           registers and needs no cross-lane traffic.  With fewer than 128 query rows the rows are
//           replicated over the four lane quarters and every warp takes a quarter of the key columns.
//           The last split of a unit to finish (atomic ticket) merges the unit's statistics.
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
// 32 consecutive fp32 columns of this thread's TMEM lane.
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
  tmem_wait_ld();
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
// Kernel
// ---------------------------------------------------------------------------------------------
constexpr int kTcStages = 2;       // shared-memory ring of key tiles, and TMEM accumulator buffers

template <int D, int M>
struct TcCfg {
  static constexpr int kHalves = D / 64;                         // 128-byte swizzled K segments per row
  static constexpr int kSteps = D / 16;                          // MMA k-steps per tile
  static constexpr int kQRows = M < 128 ? 128 : M;               // rows of the query operand buffer
  static constexpr int kRep = M < 128 ? 128 / M : 1;             // replicas of the query rows across lanes
  static constexpr int kQHalfBytes = kQRows * 128;
  static constexpr int kQBytes = kHalves * kQHalfBytes;
  static constexpr int kKHalfBytes = kTcKeyTile * 128;
  static constexpr int kKTileBytes = kHalves * kKHalfBytes;
  static constexpr uint32_t kBufCols = M == 256 ? 256 : 128;     // TMEM columns of one accumulator buffer
  static constexpr uint32_t kTmemCols = kTcStages * kBufCols;    // 256 (two CTAs per SM) or 512
  static constexpr int kColsPerThread = M < 128 ? M : 128;       // pass-1 key columns a thread reduces per tile
  static constexpr uint32_t kQTxBytes = (uint32_t)(kRep * kHalves * (M < 128 ? M : kQRows) * 128);
  static constexpr size_t kSmemBytes =
      1024 + (size_t)kQBytes + (size_t)kTcStages * kKTileBytes + 256 * 4 /*mrow*/ + 256 * 8 /*stats*/ + 128;
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

// PASS 1: row statistics of every (unit, split) item, merged per unit by the last split to finish.
// PASS 2: column sums u, launched after pass 1 has completed; items are taken in reverse order so that the
//         keys pass 1 streamed last are still in L2.
template <int D, int M, int PASS>
__global__ void __launch_bounds__(kTcThreads) score_tc_kernel(const __grid_constant__ CUtensorMap tmap_q,
                                                             const __grid_constant__ CUtensorMap tmap_k,
                                                             const ScoreParams p) {
  using C = TcCfg<D, M>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* k_s = q_s + C::kQBytes;
  float* s_mrow = reinterpret_cast<float*>(k_s + (size_t)kTcStages * C::kKTileBytes);   // [256]
  float2* s_stat = reinterpret_cast<float2*>(s_mrow + 256);                              // [256]
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(s_stat + 256);                        // [kTcStages]
  uint64_t* mma_bar = full_bar + kTcStages;                                              // [kTcStages]
  uint64_t* q_bar = mma_bar + kTcStages;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(q_bar + 1);
  int* s_ctl = reinterpret_cast<int*>(s_tmem + 1);                                       // [0] item [1] flag

  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < kTcStages; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&mma_bar[i], 1);
    }
    mbar_init(q_bar, 1);
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
  const uint32_t tmem_lane = tmem_base + ((uint32_t)(32 * warp) << 16);   // this warp's quarter of the lanes

  uint32_t gt = 0;            // key tiles this CTA has processed: stage, accumulator buffer and phases follow it
  uint32_t q_parity = 0;      // phase of the query barrier (one use per item)
  bool aborted = false;
  const uint32_t q_base = smem_u32(q_s), k_base = smem_u32(k_s);
  int* counter = PASS == 1 ? &p.hdr->work_counter : &p.hdr->prep_ticket;

  int next = 0;
  if (tid == 0) next = atomicAdd(counter, 1);
  while (!aborted) {
    __syncthreads();
    if (tid == 0) {
      s_ctl[0] = next;
      next = atomicAdd(counter, 1);      // fetched now, used after this item (no item ever waits for another)
    }
    __syncthreads();
    int idx = s_ctl[0];
    if (idx >= p.n_work) break;
    if (PASS == 2) idx = p.n_work - 1 - idx;
    const int unit = idx / p.n_splits, split = idx % p.n_splits;
    const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
    const int cu = p.cu_seqlens[b];
    const int t = p.cu_seqlens[b + 1] - cu;
    const int P = max(t - p.window, 0);
    const int key_begin = split * p.split_keys;
    const int key_end = min(key_begin + p.split_keys, PASS == 1 ? t : P);
    if (key_begin >= key_end) continue;
    const int n_tiles = (key_end - key_begin + kTcKeyTile - 1) / kTcKeyTile;

    auto load_tile = [&](int ti) {           // thread 0: arm the stage's barrier and start the copy
      const uint32_t s = (gt + ti) % kTcStages;
      mbar_arrive_expect_tx(&full_bar[s], (uint32_t)C::kKTileBytes);
#pragma unroll
      for (int hf = 0; hf < C::kHalves; ++hf)
        tma_load_3d(k_s + (size_t)s * C::kKTileBytes + hf * C::kKHalfBytes, &tmap_k, hf * 64, g,
                    cu + key_begin + ti * kTcKeyTile, &full_bar[s]);
    };
    // thread 0: once tile ti has landed, issue its MMAs into accumulator buffer (gt+ti) % 2
    auto issue = [&](int ti) -> bool {
      const uint32_t gi = gt + ti, s = gi % kTcStages;
      if (!tc_mbar_wait(&full_bar[s], (gi / kTcStages) & 1u)) return false;
      tc_fence_after_sync();
      const uint32_t kt = k_base + s * C::kKTileBytes;
      const uint32_t d_tmem = tmem_base + s * C::kBufCols;
#pragma unroll
      for (int k = 0; k < C::kSteps; ++k) {
        const uint32_t ko = (uint32_t)(k % 4) * 32u;          // 16 bf16 along K inside the swizzled 128-byte row
        const uint64_t kd = umma_desc_k128(kt + (k / 4) * C::kKHalfBytes + ko);
        if (PASS == 1) {
#pragma unroll
          for (int rb = 0; rb < (M == 256 ? 2 : 1); ++rb) {
            const uint64_t qd = umma_desc_k128(q_base + (k / 4) * C::kQHalfBytes + rb * 128 * 128 + ko);
            umma_bf16(d_tmem + rb * 128u, qd, kd, umma_idesc(128, kTcKeyTile), k > 0 ? 1u : 0u);
          }
        } else {
          const uint64_t qd = umma_desc_k128(q_base + (k / 4) * C::kQHalfBytes + ko);
          umma_bf16(d_tmem, kd, qd, umma_idesc(kTcKeyTile, M), k > 0 ? 1u : 0u);
        }
      }
      umma_commit(&mma_bar[s]);
      return true;
    };

    // ---- prologue of the item: query rows (replicated across lane quarters) and the first key tiles
    bool issue_ok = true;
    if (tid == 0) {
      mbar_arrive_expect_tx(q_bar, C::kQTxBytes);
      const int qrow0 = (b * p.n_q_heads + g * p.group) * p.window;
#pragma unroll
      for (int rep = 0; rep < C::kRep; ++rep)
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf)
          tma_load_2d(q_s + hf * C::kQHalfBytes + rep * M * 128, &tmap_q, hf * 64, qrow0, q_bar);
      for (int ti = 0; ti < min(n_tiles, kTcStages); ++ti) load_tile(ti);
      issue_ok = tc_mbar_wait(q_bar, q_parity);
      if (issue_ok) issue_ok = issue(0);
    }
    q_parity ^= 1u;
    if (PASS == 2) {
      for (int r = tid; r < M; r += kTcThreads) s_mrow[r] = __ldcg(&p.mrow[(size_t)unit * M + r]);
      __syncthreads();
    }

    // ---- the item's tiles: MMA of tile ti+1 runs while tile ti is reduced out of TMEM
    float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;   // second pair: row tid+128 when M == 256
    const int limit0 = t - p.window + ((tid % M) % p.window);
    const int limit1 = t - p.window + ((tid + 128) % p.window);
    const int col_begin = M < 128 ? (tid / M) * C::kColsPerThread : 0;
    float* u = p.u + (size_t)g * p.total_tokens + cu;
    for (int ti = 0; ti < n_tiles; ++ti) {
      const uint32_t gi = gt + ti, s = gi % kTcStages;
      if (tid == 0 && ti + 1 < n_tiles && issue_ok) issue_ok = issue(ti + 1);
      const bool ok = issue_ok && tc_mbar_wait(&mma_bar[s], (gi / kTcStages) & 1u);
      tc_fence_after_sync();
      if (tid == 0 && ok && ti + kTcStages < n_tiles) load_tile(ti + kTcStages);   // the MMA is done with stage s
      if (ok) {
        const int tile_c0 = key_begin + ti * kTcKeyTile;
        const uint32_t acc_addr = tmem_lane + s * C::kBufCols;
        if (PASS == 1) {
          const bool masked = tile_c0 + kTcKeyTile > t - p.window;
#pragma unroll
          for (int cc = 0; cc < C::kColsPerThread; cc += 32) {
            float v[32];
            tmem_ld32(acc_addr + (uint32_t)(col_begin + cc), v);
            p1_update(v, masked, tile_c0 + col_begin + cc, limit0, p.scale_log2, m0, l0);
          }
          if (M == 256) {
#pragma unroll
            for (int cc = 0; cc < 128; cc += 32) {
              float v[32];
              tmem_ld32(acc_addr + 128u + (uint32_t)cc, v);
              p1_update(v, masked, tile_c0 + cc, limit1, p.scale_log2, m1, l1);
            }
          }
        } else {
          float acc = 0.f;
#pragma unroll
          for (int cc = 0; cc < M; cc += 32) {
            float v[32];
            tmem_ld32(acc_addr + (uint32_t)cc, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) acc += fast_exp2(fmaf(v[i], p.scale_log2, -s_mrow[cc + i]));
          }
          const int key = tile_c0 + tid;
          if (key < key_end) u[key] = acc;
        }
      }
      tc_fence_before_sync();
      aborted = __syncthreads_or(ok ? 0 : 1) != 0;
      if (aborted) break;
    }
    if (aborted) break;
    gt += (uint32_t)n_tiles;

    if (PASS == 1) {
      // ---- publish this split's row statistics; the last split of the unit merges them into
      //      mrow[r] = m_r + log2(l_r) (log2 domain; +inf for rows without visible keys)
      s_stat[tid] = make_float2(m0, l0);
      if (M == 256) s_stat[128 + tid] = make_float2(m1, l1);
      __syncthreads();
      float2* out = p.stats_part + ((size_t)unit * p.n_splits + split) * M;
      for (int r = tid; r < M; r += kTcThreads) {
        float m = -INFINITY;
#pragma unroll
        for (int rep = 0; rep < C::kRep; ++rep) m = fmaxf(m, s_stat[r + rep * M].x);
        float l = 0.f;
        if (m > -INFINITY) {
#pragma unroll
          for (int rep = 0; rep < C::kRep; ++rep) l += s_stat[r + rep * M].y * fast_exp2(s_stat[r + rep * M].x - m);
        }
        out[r] = make_float2(m, l);
      }
      __threadfence();
      __syncthreads();
      const int n_splits_u = (t + p.split_keys - 1) / p.split_keys;
      if (tid == 0) s_ctl[1] = (atomicAdd(&p.unit_ticket[unit], 1) == n_splits_u - 1) ? 1 : 0;
      __syncthreads();
      if (s_ctl[1]) {
        __threadfence();
        for (int r = tid; r < M; r += kTcThreads) {
          const float2* part = p.stats_part + (size_t)unit * p.n_splits * M + r;
          float m = -INFINITY;
          for (int sp = 0; sp < n_splits_u; ++sp) m = fmaxf(m, __ldcg(&part[(size_t)sp * M]).x);
          float l = 0.f;
          if (m > -INFINITY)
            for (int sp = 0; sp < n_splits_u; ++sp) {
              const float2 v = __ldcg(&part[(size_t)sp * M]);
              l += v.y * exp2f(v.x - m);
            }
          p.mrow[(size_t)unit * M + r] = (l > 0.f) ? m + log2f(l) : INFINITY;
        }
      }
    }
  }

  // ---- teardown: every MMA has completed (its barrier was waited on) before TMEM goes back
  if (aborted) {
    if (tid == 0) record_status(p.hdr, XKV_ERR_TIMEOUT);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies already issued land
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, C::kTmemCols);
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

// Key tiles per work item: large enough to amortise the per-item prologue, small enough to fill the GPU.
int tc_tiles(int M, int head_dim, int units, int max_seqlen, int* ctas_per_sm) {
  if (M != 32 && M != 64 && M != 128 && M != 256) return 0;
  if (head_dim != 64 && head_dim != 128) return 0;
  const int sms = sm_count();
  int tiles = 8;
  while (tiles > 1 && (int64_t)units * ((max_seqlen + tiles * kTcKeyTile - 1) / (tiles * kTcKeyTile)) < 4 * sms)
    tiles >>= 1;
  *ctas_per_sm = M == 256 ? 1 : 2;
  return tiles;
}

template <int D, int M, int PASS>
xkv_status tc_launch(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, int ctas_per_sm,
                     cudaStream_t st) {
  using C = TcCfg<D, M>;
  size_t smem = C::kSmemBytes;
  // keep further CTAs off the SM: the resident ones hold all 512 TMEM columns between them
  const size_t floor_bytes = ctas_per_sm == 2 ? 80 * 1024 : 120 * 1024;
  if (smem < floor_bytes) smem = floor_bytes;
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
  int grid = sm_count() * ctas_per_sm;
  if (grid > p.n_work) grid = p.n_work;
  score_tc_kernel<D, M, PASS><<<grid, kTcThreads, smem, st>>>(tq, tk, p);
  count_launch();
  return check_launch();
}

template <int D, int M>
xkv_status tc_launch_both(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, int ctas_per_sm,
                          cudaStream_t st) {
  xkv_status s = tc_launch<D, M, 1>(tq, tk, p, ctas_per_sm, st);
  if (s != XKV_OK) return s;
  return tc_launch<D, M, 2>(tq, tk, p, ctas_per_sm, st);
}

}  // namespace

int score_tc_split_keys(int M, int head_dim, int units, int max_seqlen) {
#ifdef XKV_NO_TC
  return 0;
#else
  int ctas = 1;
  return tc_tiles(M, head_dim, units, max_seqlen, &ctas) * kTcKeyTile;
#endif
}

xkv_status score_tc_passes(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st) {
  const int units = p.batch * p.n_kv_heads;
  int ctas = 1;
  const int tiles = tc_tiles(p.M, head_dim, units, max_seqlen, &ctas);
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
  if (head_dim == DD && p.M == MM) return tc_launch_both<DD, MM>(tq, tk, p, ctas, st);
  XKV_TC_CASE(128, 32) XKV_TC_CASE(128, 64) XKV_TC_CASE(128, 128) XKV_TC_CASE(128, 256)
  XKV_TC_CASE(64, 32) XKV_TC_CASE(64, 64) XKV_TC_CASE(64, 128) XKV_TC_CASE(64, 256)
#undef XKV_TC_CASE
  return XKV_ERR_UNSUPPORTED;
}

}  // namespace xkv
