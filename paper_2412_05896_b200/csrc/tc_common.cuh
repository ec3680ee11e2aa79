// tcgen05 / TMEM / TMA wrappers and the tile configuration shared by the tensor-core scoring kernels
// (xkv_score_tc.cu: two streaming passes; xkv_score_fused.cu: both passes in one cluster kernel).
#pragma once

#include <cuda.h>

#include <cmath>
#include <mutex>

#include "common.cuh"
#include "score_params.h"

namespace xkv {
namespace tc {

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

constexpr int kWsThreads = 320;
constexpr int kEpiThreads = 128;     // threads of one epilogue group
constexpr int kWsStages = 4;       // shared-memory ring of key tiles
constexpr int kAccBufs = 4;        // TMEM accumulator buffers of 128 columns
constexpr int kEpiGroups = 2;      // epilogue groups (each takes every other tile)
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
  static constexpr uint32_t kBufCols = 128;                      // TMEM columns of one accumulator buffer
  static constexpr uint32_t kTmemCols = kAccBufs * kBufCols;
  static constexpr int kJobs = M == 256 ? 2 : 1;                 // accumulator jobs per key tile
  static constexpr int kJobRows = M == 256 ? 128 : M;            // pass 2: query rows (MMA N) of one job
  static constexpr int kColsPerThread = M < 128 ? M : 128;       // pass-1 key columns a thread reduces per tile
  static constexpr uint32_t kQTxBytes = (uint32_t)(kRep * kHalves * (M < 128 ? M : kQRows) * 128);
  static constexpr size_t kSmemBytes = 1024 + (size_t)kQBufs * kQBytes + (size_t)kWsStages * kKTileBytes +
                                       kMrowSlots * 256 * 4 /*row normalisers*/ + 256 /*barriers*/;
};

// Online-softmax update of one query row with 32*N more logits v (raw dot products; scale > 0 folds 1/sqrt(d) and
// log2 e).  Tiles that reach into the observation window mask the keys the row must not see; all other tiles
// skip that work (masked is the same for every thread of a tile).  Maximum and sum run as four independent
// chains so that neither is one long dependent sequence, and the running sum is rescaled once per call.
template <int N>
__device__ __forceinline__ void p1_update(float (&x)[N][32], bool masked, int c0, int limit, float scale, float& m,
                                          float& l) {
  if (masked) {
#pragma unroll
    for (int j = 0; j < N; ++j)
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (c0 + 32 * j + i > limit) x[j][i] = -INFINITY;
  }
  float mx[4] = {x[0][0], x[0][1], x[0][2], x[0][3]};
#pragma unroll
  for (int j = 0; j < N; ++j)
#pragma unroll
    for (int i = (j == 0 ? 4 : 0); i < 32; i += 4) {
      mx[0] = fmaxf(mx[0], x[j][i]);
      mx[1] = fmaxf(mx[1], x[j][i + 1]);
      mx[2] = fmaxf(mx[2], x[j][i + 2]);
      mx[3] = fmaxf(mx[3], x[j][i + 3]);
    }
  const float vmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
  const float m_new = fmaxf(m, vmax * scale);
  const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
  float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int j = 0; j < N; ++j)
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
      sm[0] += fast_exp2(fmaf(x[j][i], scale, -m_ref));
      sm[1] += fast_exp2(fmaf(x[j][i + 1], scale, -m_ref));
      sm[2] += fast_exp2(fmaf(x[j][i + 2], scale, -m_ref));
      sm[3] += fast_exp2(fmaf(x[j][i + 3], scale, -m_ref));
    }
  l = l * fast_exp2(m - m_ref) + ((sm[0] + sm[1]) + (sm[2] + sm[3]));
  m = m_new;
}

// Bounded mbarrier wait that also gives up when another role has raised the abort flag.
__device__ __forceinline__ bool ws_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint64_t limit_ns) {
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_timer_ns() - t0 > limit_ns) {
      *abort_flag = 1;
      return false;
    }
  }
}


typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tc_encode_fn() {
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

inline bool tc_make_tmap(CUtensorMap* tmap, const void* base, int rank, const cuuint64_t* dims,
                         const cuuint64_t* strides, const cuuint32_t* box) {
  EncodeTiledFn enc = tc_encode_fn();
  if (enc == nullptr) return false;
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return enc(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box,
             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor maps of the query rows (2-D, box {64, M}) and of the packed keys (3-D, box {64, 1, 128 keys}).
inline bool tc_make_score_tmaps(const ScoreParams& p, int head_dim, CUtensorMap* tq, CUtensorMap* tk) {
  {
    const cuuint64_t dims[2] = {(cuuint64_t)head_dim, (cuuint64_t)p.batch * p.n_q_heads * p.window};
    const cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
    const cuuint32_t box[2] = {64u, (cuuint32_t)p.M};
    if (!tc_make_tmap(tq, p.q_win, 2, dims, strides, box)) return false;
  }
  const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)p.n_kv_heads, (cuuint64_t)p.total_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)p.stride_head * 2, (cuuint64_t)p.stride_token * 2};
  const cuuint32_t box[3] = {64u, 1u, (cuuint32_t)kTcKeyTile};
  return tc_make_tmap(tk, p.k, 3, dims, strides, box);
}

}  // namespace tc
}  // namespace xkv
