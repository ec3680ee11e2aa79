// Shared host/device helpers of libxkv (sm_100a): status plumbing, bf16 packing, mbarrier / TMA /
// ldmatrix / mma.sync wrappers in inline PTX.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/xkv.h"

namespace xkv {

// ---------------------------------------------------------------------------------------------
// Workspace header: the first 256 bytes of every op's workspace.
// ---------------------------------------------------------------------------------------------
struct WorkspaceHeader {
  int32_t status;      // XKV_OK or the first XKV_ERR_* recorded by a kernel
  int32_t n_items;     // decode: number of work items planned on the device
  int32_t chunk_rows;  // decode: rows per chunk chosen by the plan
  int32_t work_counter;  // decode: next work item to hand to a warp
  int32_t prep_ticket;   // decode: CTAs of the prepare kernel that have finished
  int32_t n_multi;       // decode: (layer, sequence) units cut into more than one chunk
  int32_t merge_counter; // decode: next split-K merge job to hand to a warp
  int32_t grid_arrivals; // decode: CTAs of the self-planning launch that have finished all their work
  int32_t reserved[56];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header is 256 bytes");

constexpr int kHeaderBytes = 256;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Launch bookkeeping shared by all translation units.
void count_launch(int n = 1);
xkv_status check_launch();
int sm_count();
// Limit, in nanoseconds, of every bounded wait inside a kernel (two seconds unless a test shortened it).
uint64_t wait_limit_ns();
// Test hook: index of the decode work item whose merge ticket is withheld (-1: none).
int32_t debug_withhold_item();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__device__ __forceinline__ void record_status(WorkspaceHeader* hdr, int32_t code) {
  atomicCAS(&hdr->status, XKV_OK, code);
}

// ---------------------------------------------------------------------------------------------
// Small device utilities
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------------------------------------
// Cache rows stored as 8-bit integers with one fp32 scale per row: scale = max|x| / 127 (1 for an all-zero row),
// q = x / scale rounded to nearest, ties to even, within [-127, 127]; the stored byte is q + 128.  Both divisions are
// IEEE fp32 divisions, so that the bytes are the same wherever they are computed.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t int8_stored_byte(float x, float scale) {
  int q = __float2int_rn(__fdiv_rn(x, scale));
  q = max(-127, min(127, q));
  return (uint32_t)(q + 128);
}
// Quantises one row spread over consecutive lanes of a warp, eight consecutive elements per lane (x = this lane's
// elements as fp32, group = D / 8 lanes per row, a power of two, rows aligned to multiples of `group` lanes; every lane
// of the row must be here).  Returns the lane's eight stored bytes; *scale is the row's scale in every lane of the row.
__device__ __forceinline__ uint2 quantize_row_piece(const float (&x)[8], int group, float* scale) {
  const unsigned lane = threadIdx.x & 31u;
  const unsigned mask = (group >= 32 ? 0xffffffffu : ((1u << group) - 1u)) << (lane & ~(unsigned)(group - 1));
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(x[i]));
  for (int o = 1; o < group; o <<= 1) amax = fmaxf(amax, __shfl_xor_sync(mask, amax, o));
  const float s = amax > 0.f ? __fdiv_rn(amax, 127.f) : 1.f;
  *scale = s;
  uint2 out;
  out.x = int8_stored_byte(x[0], s) | (int8_stored_byte(x[1], s) << 8) | (int8_stored_byte(x[2], s) << 16) |
          (int8_stored_byte(x[3], s) << 24);
  out.y = int8_stored_byte(x[4], s) | (int8_stored_byte(x[5], s) << 8) | (int8_stored_byte(x[6], s) << 16) |
          (int8_stored_byte(x[7], s) << 24);
  return out;
}
// Two stored bytes of a 32-bit word -> two fp16 integers (exact).  kSelector picks the bytes (a prmt selector whose
// odd result bytes take the constant 0x64): 0x64nn read as fp16 is 1024 + nn, and 1024 + 128 is subtracted.
template <uint32_t kSelector>
__device__ __forceinline__ uint32_t int8x2_to_f16x2(uint32_t word) {
  uint32_t r;
  asm("{\n\t.reg .b32 t, c;\n\t"
      "prmt.b32 t, %1, 0x64646464, %2;\n\t"
      "mov.b32 c, 0x64806480;\n\t"
      "sub.f16x2 %0, t, c;\n\t}"
      : "=r"(r)
      : "r"(word), "n"(kSelector));
  return r;
}
// The same without the subtraction: the two fp16 values are 1024 + stored byte = kInt8Bias + q.  A product summed
// over such operands carries kInt8Bias times the sum of the other operand, which the caller removes once per output
// instead of once per element (every value involved is an integer below 2048 times an fp16: exact until the fp32 sum).
constexpr float kInt8Bias = 1152.f;
template <uint32_t kSelector>
__device__ __forceinline__ uint32_t int8x2_to_biased_f16x2(uint32_t word) {
  uint32_t r;
  asm("prmt.b32 %0, %1, 0x64646464, %2;" : "=r"(r) : "r"(word), "n"(kSelector));
  return r;
}
// The eight bf16 of a 16-byte piece as fp32.
__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float (&x)[8]) {
  x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
  x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
}

// ---------------------------------------------------------------------------------------------
// mbarrier (shared::cta) and TMA tensor loads.  Every wait is bounded.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t* ptr) {
  int32_t v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

// Waits for the phase with the given parity for at most limit_ns of wall time; false on expiry.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint64_t limit_ns) {
  for (int i = 0; i < 128; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (global_timer_ns() - t0 > limit_ns) return false;
  }
}

// Polls a counter in global memory until it reaches `target`, for at most limit_ns; false on expiry.
__device__ __forceinline__ bool spin_until_ge(const int32_t* ptr, int32_t target, uint64_t limit_ns, unsigned sleep_ns) {
  if (ld_acquire_gpu(ptr) >= target) return true;
  const uint64_t t0 = global_timer_ns();
  while (ld_acquire_gpu(ptr) < target) {
    if (global_timer_ns() - t0 > limit_ns) return false;
    __nanosleep(sleep_ns);
  }
  return true;
}

// 2-D tiled TMA load global -> shared, completion counted on an mbarrier.  x is the innermost
// coordinate; x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* dst, const void* tmap, int32_t x, int32_t y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void prefetch_tmap(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}

// Named barrier among a subset of the CTA's warps.
__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Tensor-core fragments: ldmatrix and mma.sync m16n8k16 (bf16 x bf16 -> fp32)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Transposes an 8x8 matrix of 16-bit elements held one row pair per lane (lane = 4*row + column/2).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// cp.async 16-byte copy global -> shared (zero-fills when src_bytes < 16).
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

}  // namespace xkv
