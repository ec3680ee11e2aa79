// xkv_prefill_attn: causal attention of the whole prompt (Eq. 1 with the weights of Eq. 2) on the 5th-generation
// tensor cores, writing next to its output the softmax normaliser of every row.  The normalisers of the last W
// rows are what the scoring step needs of W_attn (Alg. 2 step 1): with them xkv_score_lse forms the column
// scores in one pass over the keys.
//
// One CTA per (sequence, tile of 128 query rows, query head), 256 threads, key tiles of 64; two CTAs share an SM
// (half of its shared memory and of its tensor memory each), so that one CTA's softmax runs under the other's MMAs:
//   warps 0-3  softmax: thread = query row = TMEM lane.  Per key tile: the row's 64 logits out of TMEM into registers
//              (once), row maximum, a reference maximum that is exact on the first tile and raised lazily
//              afterwards (only when a logit exceeds it by 2^8, which is when the warp waits for the previous
//              O += P V and rescales the O accumulator in TMEM: load, multiply, store), P = exp2(s*c - ref) rounded
//              to bf16 and stored as pairs over the first 32 columns of the tile's S buffer, where the MMA reads it
//              as its A operand; row sum in fp32.  At the end O / l -> bf16 rows, lse.
//   warps 4, 6 producers (one lane each): TMA loads of the Q tile and the K tiles, and of the V tiles (two stages
//              each), so that a K tile never queues behind the V stage of an earlier tile
//   warps 5, 7 MMA issuers (one lane each), one per product: S = Q K^T into one of two 64-column TMEM buffers, one
//              tile ahead of the softmax (and not before the product that last read P out of that buffer is
//              complete); O += P V with P out of tensor memory and V as an MN-major B operand straight from its
//              [keys][d] tile
// Hand-overs between the roles go through one mbarrier per S buffer for each of "logits ready", "P ready" and
// "product complete": a softmax warp may be a tile ahead of the others, and a warp that did not rescale for a while
// has not waited for any product, so a single barrier counted over all tiles could take a later phase for an earlier.
// Every wait is bounded; an expired wait sets the status word and lets the CTA drain.
#include <atomic>

#include "tc_common.cuh"
#include "ops.h"

namespace xkv {
namespace {

using namespace tc;

constexpr int kPfThreads = 256;
constexpr int kPfRows = 128;          // query rows per CTA
constexpr int kPfKeys = 64;           // keys per tile
constexpr float kPfLazy = 8.f;        // log2 slack before the reference maximum is raised

struct PrefillParams {
  const int32_t* cu_seqlens;
  __nv_bfloat16* out;     // [T][Hq][D]
  float* lse;             // [Hq][T]
  WorkspaceHeader* hdr;
  int64_t total_tokens;
  int32_t batch, n_q_heads, n_kv_heads, group, max_seqlen;
  float scale_log2;
  uint64_t wait_ns;
};

template <int D>
struct PfCfg {
  static constexpr int kHalves = D / 64;
  static constexpr int kSteps = D / 16;                      // k-steps of S = Q K^T
  static constexpr int kQHalfBytes = kPfRows * 128;          // 64 columns of the query tile: rows of 128 bytes
  static constexpr int kQTileBytes = kHalves * kQHalfBytes;
  static constexpr int kKvHalfBytes = kPfKeys * 128;         // 64 columns of a K or V tile
  static constexpr int kKvTileBytes = kHalves * kKvHalfBytes;
  static constexpr int kKStages = 2;                         // S runs one tile ahead of the softmax
  static constexpr int kVStages = 2;
  static constexpr uint32_t kSCols = kPfKeys;                // one S buffer
  static constexpr uint32_t kOCol = 2 * kPfKeys;             // O accumulator starts here
  static constexpr uint32_t kTmemCols = 256;                 // two CTAs share an SM's 512 columns
  static constexpr size_t kSmemBytes = 1024 + (size_t)kQTileBytes + (size_t)kKvTileBytes * (kKStages + kVStages) + 256;
  static_assert(2 * (kSmemBytes + 1024) <= 233472, "two CTAs per SM");
};

__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 consecutive 32-bit columns of this thread's TMEM lane from registers (here: 64 bf16 values of a row of P).
__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem desc], bf16 inputs, fp32 accumulate; A is 128 rows (one per TMEM lane) of K-major
// bf16 pairs, one pair per 32-bit column (16 K elements = 8 columns a step); issued by one thread.
__device__ __forceinline__ void umma_bf16_a_tmem(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t"
      "}\n" ::"r"(tmem_d),
      "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}

// 16 consecutive fp32 columns of this thread's TMEM lane (the rescale of O works in these smaller pieces so that the
// tile's logits can stay in registers beside it).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
      : "memory");
}

// Shared-memory descriptor of an MN-major operand tile stored as rows of 128 bytes (64 bf16 along MN) per K index
// with the 128-byte swizzle: eight K rows form a 1024-byte group (stride byte offset), the next 64 MN elements
// start `mn_block_bytes` further (leading byte offset).  This is what a TMA box {64, rows} of a [keys][d] tile is
// when d is the MMA's N and the keys its K.
__device__ __forceinline__ uint64_t umma_desc_mn128(uint32_t smem_addr, uint32_t mn_block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
  d |= (uint64_t)(mn_block_bytes >> 4) << 16;     // leading byte offset: next block of 64 MN elements
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: next group of eight K rows
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}

// bf16 x bf16 -> fp32, A K-major, B MN-major.
__host__ __device__ constexpr uint32_t umma_idesc_b_mn(int M, int N) { return umma_idesc(M, N) | (1u << 16); }

// The (sequence, query tile) of CTA-tile index `idx`, counted from the end so that the long tiles of the last
// sequence start first; false when idx is beyond the tiles that exist.  Computed by every warp for itself: a lane
// takes one sequence, a warp scan gives the tiles before it.
__device__ __forceinline__ bool pf_tile(const PrefillParams& p, int idx, int* b_out, int* q0_out, int* cu_out,
                                        int* t_out) {
  const int lane = threadIdx.x & 31;
  int before = 0;                                   // tiles of the sequences already passed
  for (int base = 0; base < p.batch; base += 32) {
    const int b = p.batch - 1 - (base + lane);
    int cu = 0, t = 0, n = 0;
    if (b >= 0) {
      cu = p.cu_seqlens[b];
      t = min(p.cu_seqlens[b + 1] - cu, p.max_seqlen);
      n = (t + kPfRows - 1) / kPfRows;
    }
    int incl = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, idx < before + incl);
    if (hit != 0u) {
      const int src = __ffs(hit) - 1;
      const int first = before + __shfl_sync(0xffffffffu, incl - n, src);     // tiles before that sequence
      const int n_src = __shfl_sync(0xffffffffu, n, src);
      *b_out = p.batch - 1 - (base + src);
      *q0_out = (n_src - 1 - (idx - first)) * kPfRows;
      *cu_out = __shfl_sync(0xffffffffu, cu, src);
      *t_out = __shfl_sync(0xffffffffu, t, src);
      return true;
    }
    before += __shfl_sync(0xffffffffu, incl, 31);
  }
  return false;
}

template <int D>
__global__ void __launch_bounds__(kPfThreads, 2)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const PrefillParams p) {
  using C = PfCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* k_s = q_s + C::kQTileBytes;
  uint8_t* v_s = k_s + (size_t)C::kKStages * C::kKvTileBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(v_s + (size_t)C::kVStages * C::kKvTileBytes);
  uint64_t* q_full = bars;             // [1]
  uint64_t* k_full = bars + 1;         // [2]
  uint64_t* k_empty = bars + 3;        // [2]
  uint64_t* v_full = bars + 5;         // [2]
  uint64_t* v_empty = bars + 7;        // [2]
  uint64_t* s_full = bars + 9;         // [2] S buffer complete (MMA -> softmax)
  // [2] P written over the tile's S buffer, O rescaled (softmax -> MMA), one barrier per S buffer: a softmax warp that
  // does not have to rescale O may be a tile ahead of the others, and its arrival for tile j+1 must not count for tile j
  uint64_t* p_full = bars + 13;
  // [2] O += P V of a tile complete (MMA -> softmax, and MMA -> its own next use of the S buffer), one barrier per S
  // buffer as well: softmax warps wait here only when they rescale O and at the very end, so between two waits of a
  // warp several products may complete, and with one barrier for all tiles the parity of "tile j-1 done" would also
  // match "tile j-3 done"
  uint64_t* p_empty = bars + 15;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 17);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int b, q0, cu, t;
  const int h = blockIdx.x % p.n_q_heads;
  if (!pf_tile(p, blockIdx.x / p.n_q_heads, &b, &q0, &cu, &t)) return;      // uniform over the CTA
  const int g = h / p.group;
  const int n_kt = (q0 + kPfRows) / kPfKeys;         // key tiles up to and including the last one a row of the tile sees

  if (tid == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&v_full[i], 1);
      mbar_init(&v_empty[i], 1);
    }
    mbar_init(&p_full[0], 4);
    mbar_init(&p_full[1], 4);
    mbar_init(&p_empty[0], 1);
    mbar_init(&p_empty[1], 1);
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_k);
    prefetch_tmap(&tmap_v);
  }
  if (warp == 0) {
    tmem_alloc(s_tmem, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 4) {
    // ------------------------------------------------------------------ producer of Q and the K tiles
    if (lane == 0) {
      mbar_arrive_expect_tx(q_full, (uint32_t)C::kQTileBytes);
#pragma unroll
      for (int hf = 0; hf < C::kHalves; ++hf) tma_load_3d(q_s + hf * C::kQHalfBytes, &tmap_q, hf * 64, h, cu + q0, q_full);
      bool ok = true;
      for (int j = 0; ok && j < n_kt; ++j) {
        const uint32_t s = j & 1u, ph = ((j >> 1) & 1u) ^ 1u;
        ok = ws_wait(&k_empty[s], ph, s_abort, p.wait_ns);
        if (!ok) break;
        mbar_arrive_expect_tx(&k_full[s], (uint32_t)C::kKvTileBytes);
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf)
          tma_load_3d(k_s + (size_t)s * C::kKvTileBytes + hf * C::kKvHalfBytes, &tmap_k, hf * 64, g, cu + j * kPfKeys,
                      &k_full[s]);
      }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ producer of the V tiles (two stages)
    if (lane == 0) {
      bool ok = true;
      for (int j = 0; ok && j < n_kt; ++j) {
        const uint32_t s = j & 1u;
        ok = ws_wait(&v_empty[s], ((j >> 1) & 1u) ^ 1u, s_abort, p.wait_ns);
        if (!ok) break;
        mbar_arrive_expect_tx(&v_full[s], (uint32_t)C::kKvTileBytes);
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf)
          tma_load_3d(v_s + (size_t)s * C::kKvTileBytes + hf * C::kKvHalfBytes, &tmap_v, hf * 64, g, cu + j * kPfKeys,
                      &v_full[s]);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ issuer of the logit MMAs
    // Two issuing threads, one per product: a `tcgen05.mma` holds its thread until the pipe (shared with the SM's
    // other CTA) takes it, and with one thread for both products that time, not the softmax, set the pace of a tile.
    if (lane == 0) {
      bool ok = ws_wait(q_full, 0u, s_abort, p.wait_ns);
      const uint64_t q_desc = umma_desc_k128(smem_u32(q_s));
      for (int j = 0; ok && j < n_kt; ++j) {
        const uint32_t s = j & 1u;
        // S buffer s holds P of tile j-2 until that tile's O += P V, issued by the other thread, has read it
        if (j >= 2) {
          ok = ws_wait(&p_empty[s], (uint32_t)((j - 2) >> 1) & 1u, s_abort, p.wait_ns);
          if (!ok) break;
        }
        ok = ws_wait(&k_full[s], (j >> 1) & 1u, s_abort, p.wait_ns);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t k_desc = umma_desc_k128(smem_u32(k_s) + s * C::kKvTileBytes);
#pragma unroll
        for (int k = 0; k < C::kSteps; ++k) {
          const uint64_t q_off = (uint64_t)(((k / 4) * C::kQHalfBytes + (k % 4) * 32) >> 4);
          const uint64_t k_off = (uint64_t)(((k / 4) * C::kKvHalfBytes + (k % 4) * 32) >> 4);
          umma_bf16(tmem_base + s * C::kSCols, q_desc + q_off, k_desc + k_off, umma_idesc(kPfRows, kPfKeys),
                    k > 0 ? 1u : 0u);
        }
        umma_commit(&k_empty[s]);
        umma_commit(&s_full[s]);
      }
    }
  } else if (warp == 7) {
    // ------------------------------------------------------------------ issuer of O += P V
    if (lane == 0) {
      bool ok = true;
      for (int j = 0; ok && j < n_kt; ++j) {
        const uint32_t vs = j & 1u;
        ok = ws_wait(&p_full[j & 1u], (j >> 1) & 1u, s_abort, p.wait_ns) &&
             ws_wait(&v_full[vs], (j >> 1) & 1u, s_abort, p.wait_ns);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t v_base = smem_u32(v_s) + vs * C::kKvTileBytes;
        const uint32_t p_tmem = tmem_base + (j & 1u) * C::kSCols;      // P over the first columns of the tile's S buffer
#pragma unroll
        for (int k = 0; k < kPfKeys / 16; ++k) {
          // A: P[rows][keys 16k .. 16k+15] out of TMEM (eight columns of bf16 pairs); B: V[keys 16k ..][d], MN-major
          // (16 keys = two 8-row groups)
          const uint64_t vd = umma_desc_mn128(v_base + k * 16 * 128, C::kKvHalfBytes);
          umma_bf16_a_tmem(tmem_base + C::kOCol, p_tmem + (uint32_t)(k * 8), vd, umma_idesc_b_mn(kPfRows, D),
                           (j > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(&v_empty[vs]);
        umma_commit(&p_empty[j & 1u]);
      }
    }
  } else if (warp < 4) {
    // ------------------------------------------------------------------ softmax warps 0..3
    const int r = tid;                                       // query row of the tile = TMEM lane
    const uint32_t lane_base = tmem_base + ((uint32_t)(32 * warp) << 16);
    const int row_pos = q0 + r;                              // position in the sequence
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; ok && j < n_kt; ++j) {
      const uint32_t s = j & 1u;
      ok = __all_sync(0xffffffffu, ws_wait(&s_full[s], (j >> 1) & 1u, s_abort, p.wait_ns));
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t s_addr = lane_base + s * C::kSCols;
      const bool diag = (j + 1) * kPfKeys - 1 > q0;          // the tile holds keys beyond some row's position
      const int c_base = j * kPfKeys;
      // ---- the tile's 64 logits of this row leave TMEM once; keys beyond the row's position (only tiles on the diagonal
      //      hold any) become -inf here, so neither the maximum nor the exponentials below mask again
      static_assert(kPfKeys == 64, "the softmax keeps one tile of 64 logits per row in registers");
      float v[2][32];
      tmem_ld32(s_addr, v[0]);
      tmem_ld32(s_addr + 32u, v[1]);
      tmem_wait_ld();
      if (diag) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (c_base + i > row_pos) v[0][i] = -INFINITY;
          if (c_base + 32 + i > row_pos) v[1][i] = -INFINITY;
        }
      }
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one dependent sequence
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        m4[0] = fmaxf(m4[0], fmaxf(v[0][i], v[1][i]));
        m4[1] = fmaxf(m4[1], fmaxf(v[0][i + 1], v[1][i + 1]));
        m4[2] = fmaxf(m4[2], fmaxf(v[0][i + 2], v[1][i + 2]));
        m4[3] = fmaxf(m4[3], fmaxf(v[0][i + 3], v[1][i + 3]));
      }
      float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
      mx *= p.scale_log2;                                    // key 0 is always visible, so mx is finite
      const bool grow = mx > m_ref + kPfLazy;                // also true on the first tile (m_ref = -inf)
      float alpha = 1.f;
      if (grow) {
        alpha = j == 0 ? 0.f : fast_exp2(m_ref - mx);
        m_ref = mx;
        l *= alpha;
      }
      // ---- O is rescaled only once the previous tile's O += P V is complete; a warp none of whose rows grew does
      //      not wait for it (P of this tile goes to this tile's own S buffer)
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
        ok = __all_sync(0xffffffffu,
                        ws_wait(&p_empty[(j - 1) & 1u], (uint32_t)((j - 1) >> 1) & 1u, s_abort, p.wait_ns));
        if (!ok) break;
        tc_fence_after_sync();
        {
#pragma unroll
          for (int cc = 0; cc < D; cc += 16) {
            float o[16];
            tmem_ld16(lane_base + C::kOCol + (uint32_t)cc, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] *= alpha;
            tmem_st16(lane_base + C::kOCol + (uint32_t)cc, o);
          }
          tmem_wait_st();
        }
      }
      // ---- P = exp2(s*c - ref) as bf16 pairs over the first 32 columns of the tile's S buffer (the logits are in
      //      registers by now), row sum in fp32
      float sm[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t packed[32];
#pragma unroll
      for (int cc = 0; cc < kPfKeys; cc += 32) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float e0 = fast_exp2(fmaf(v[cc >> 5][i], p.scale_log2, -m_ref));
          const float e1 = fast_exp2(fmaf(v[cc >> 5][i + 1], p.scale_log2, -m_ref));
          const float e2 = fast_exp2(fmaf(v[cc >> 5][i + 2], p.scale_log2, -m_ref));
          const float e3 = fast_exp2(fmaf(v[cc >> 5][i + 3], p.scale_log2, -m_ref));
          sm[0] += e0;
          sm[1] += e1;
          sm[2] += e2;
          sm[3] += e3;
          packed[(cc + i) >> 1] = pack_bf16(e0, e1);
          packed[((cc + i) >> 1) + 1] = pack_bf16(e2, e3);
        }
      }
      tmem_st32u(s_addr, packed);
      const float sum = (sm[0] + sm[1]) + (sm[2] + sm[3]);
      l += sum;
      // P and O are ready for the MMA
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[s]);
    }
    // ---- epilogue: O / l -> bf16, lse
    if (ok)
      ok = __all_sync(0xffffffffu,
                      ws_wait(&p_empty[(n_kt - 1) & 1u], (uint32_t)((n_kt - 1) >> 1) & 1u, s_abort, p.wait_ns));
    if (ok) {
      tc_fence_after_sync();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const bool live = row_pos < t;
      __nv_bfloat16* orow = p.out + ((size_t)(cu + row_pos) * p.n_q_heads + h) * D;
#pragma unroll
      for (int cc = 0; cc < D; cc += 32) {
        float o[32];
        tmem_ld32(lane_base + C::kOCol + (uint32_t)cc, o);
        tmem_wait_ld();
        if (live) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 w;
            w.x = pack_bf16(o[8 * q + 0] * inv, o[8 * q + 1] * inv);
            w.y = pack_bf16(o[8 * q + 2] * inv, o[8 * q + 3] * inv);
            w.z = pack_bf16(o[8 * q + 4] * inv, o[8 * q + 5] * inv);
            w.w = pack_bf16(o[8 * q + 6] * inv, o[8 * q + 7] * inv);
            *reinterpret_cast<uint4*>(orow + cc + 8 * q) = w;
          }
        }
      }
      if (live && p.lse != nullptr)
        p.lse[(size_t)h * p.total_tokens + cu + row_pos] = (m_ref + log2f(l)) * 0.6931471805599453f;
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

template <int D>
xkv_status pf_launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const PrefillParams& p,
                     int grid, cudaStream_t st) {
  static std::atomic<bool> done[64];   // idempotent set-up: two threads doing it twice is harmless
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  if (!done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(prefill_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)PfCfg<D>::kSmemBytes) != cudaSuccess)
      return XKV_ERR_CUDA;
    done[dev].store(true, std::memory_order_release);
  }
  prefill_attn_kernel<D><<<grid, kPfThreads, PfCfg<D>::kSmemBytes, st>>>(tq, tk, tv, p);
  count_launch();
  return check_launch();
}

// 3-D map {d, heads, tokens} with box {64, 1, box_rows} over a packed [T][heads][d] bf16 tensor.
bool pf_make_tmap(CUtensorMap* tmap, const void* base, int head_dim, int heads, int64_t tokens, int64_t stride_token,
                  int64_t stride_head, int box_rows) {
  const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)heads, (cuuint64_t)tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)stride_head * 2, (cuuint64_t)stride_token * 2};
  const cuuint32_t box[3] = {64u, 1u, (cuuint32_t)box_rows};
  return tc_make_tmap(tmap, base, 3, dims, strides, box);
}

}  // namespace

size_t prefill_workspace_bytes() { return kHeaderBytes; }

xkv_status prefill_attn(const xkv_dims* d, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                        int64_t total_tokens, int max_seqlen, void* out, float* lse, void* workspace,
                        cudaStream_t st) {
  PrefillParams p;
  p.cu_seqlens = cu_seqlens;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  p.hdr = reinterpret_cast<WorkspaceHeader*>(workspace);
  p.total_tokens = total_tokens;
  p.batch = d->batch;
  p.n_q_heads = d->n_q_heads;
  p.n_kv_heads = d->n_kv_heads;
  p.group = d->n_q_heads / d->n_kv_heads;
  p.max_seqlen = max_seqlen;
  const float scale = d->scale != 0.f ? d->scale : 1.0f / sqrtf((float)d->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  p.wait_ns = wait_limit_ns();
  CUtensorMap tq, tk, tv;
  if (!pf_make_tmap(&tq, q, d->head_dim, d->n_q_heads, total_tokens, (int64_t)d->n_q_heads * d->head_dim, d->head_dim,
                    kPfRows) ||
      !pf_make_tmap(&tk, k, d->head_dim, d->n_kv_heads, total_tokens, d->kv_stride_token, d->kv_stride_head, kPfKeys) ||
      !pf_make_tmap(&tv, v, d->head_dim, d->n_kv_heads, total_tokens, d->kv_stride_token, d->kv_stride_head, kPfKeys))
    return XKV_ERR_CUDA;
  // an upper bound of the query tiles that exist: every sequence adds at most one partial tile
  const int64_t tiles = total_tokens / kPfRows + d->batch;
  const int64_t grid = tiles * d->n_q_heads;
  if (grid > 0x7fffffffll) return XKV_ERR_UNSUPPORTED;
  if (d->head_dim == 128) return pf_launch<128>(tq, tk, tv, p, (int)grid, st);
  return pf_launch<64>(tq, tk, tv, p, (int)grid, st);
}

}  // namespace xkv
