// xkv_score: importance scoring of one layer (Eq. 2, Eq. 3, Eq. 4; Alg. 2 steps 1-4).
//
// Kernels, in stream order:
//   score_resident_kernel<D> / score_stream_kernel<D>  persistent CTAs working through key splits:
//                           pass 1  softmax row statistics (max, sum of exponentials) of the G*W
//                                   window query rows over their visible keys; the last split of a
//                                   unit merges them into one log2-domain normaliser per row
//                           pass 2  recompute the logits and accumulate the column sums u[c] over
//                                   the G*W rows (Select + Merge; the GQA group is summed before
//                                   pooling)
//                           The resident variant keeps a split's keys in shared memory between the
//                           passes (K is read from HBM once); the streaming variant, for sequences
//                           too long for that, runs all pass-1 items and then all pass-2 items.
//   pool_sort_kernel        1-D pooling (max or zero-padded average) of u into the scores w, and a
//                           descending bitonic sort of each 4096-score chunk (registers, warp
//                           shuffles, shared memory only for the longest exchanges)
//   merge_kernel            merge-path passes that combine the sorted chunks of a segment
//   gains_kernel / mass_kernel  the per-sequence retained-importance curve of the layer
//
// Both logit passes are the one dense contraction of the path and run on tensor cores
// (mma.sync m16n8k16, bf16 in, fp32 accumulate): a warp owns 32 keys of a 128-key tile, keeps
// their B fragments in registers and sweeps all G*W query rows, so per-row statistics stay with a
// thread quad and column sums complete inside the warp.  The exact method needs two passes: the
// row normalisers must be final before a column sum can be formed.
#include <cmath>

#include <atomic>

#include "common.cuh"
#include "ops.h"
#include "score_params.h"

namespace xkv {
namespace {

constexpr int kPassThreads = 128;     // 4 warps
constexpr int kKeyTile = 128;         // keys per tile, 32 per warp
constexpr int kSortChunk = 4096;      // scores sorted per CTA
constexpr int kSortThreads = 512;
constexpr int kSortItems = kSortChunk / kSortThreads;   // 8 scores per thread, kept in registers
constexpr int kMergeTile = 2048;
constexpr int kMergeThreads = 256;
constexpr int kMergeItems = kMergeTile / kMergeThreads;


constexpr int kPassStages = 3;        // cp.async ring of key tiles (streaming variant)

template <int D>
struct PassCfg {
  static constexpr int kRowBytes = D * 2;                 // unpadded rows, 16-byte chunks XOR-swizzled
  static constexpr int kTileBytes = kKeyTile * kRowBytes;
  static size_t smem_bytes(int M, int tiles) {
    return (size_t)M * kRowBytes + (size_t)tiles * kTileBytes + (size_t)4 * M * 8 + 64;
  }
};

// Byte offset of 16-byte chunk c of row r: chunks are XOR-swizzled inside each 128-byte segment so that
// ldmatrix reads of eight consecutive rows hit distinct banks.
__device__ __forceinline__ uint32_t swz(int r, int c, int row_bytes) {
  return (uint32_t)(r * row_bytes + ((c >> 3) << 7) + (((c & 7) ^ (r & 7)) << 4));
}

struct UnitShape {
  int b, g, cu, t, P;
};

__device__ __forceinline__ UnitShape unit_shape(const ScoreParams& p, int unit) {
  UnitShape s;
  s.b = unit / p.n_kv_heads;
  s.g = unit % p.n_kv_heads;
  s.cu = p.cu_seqlens[s.b];
  s.t = min(p.cu_seqlens[s.b + 1] - s.cu, p.max_seqlen);
  s.P = max(s.t - p.window, 0);
  return s;
}

template <int D>
__device__ __forceinline__ void load_q(const ScoreParams& p, const UnitShape& us, uint8_t* q_s) {
  constexpr int kChunks = D / 8;
  const __nv_bfloat16* qg = p.q_win + ((size_t)us.b * p.n_q_heads + (size_t)us.g * p.group) * p.window * D;
  for (int idx = threadIdx.x; idx < p.M * kChunks; idx += kPassThreads) {
    const int r = idx / kChunks, c = idx % kChunks;
    const bool real = r < p.M_real;               // rows that only pad G*W to a multiple of 16 are zero-filled
    cp_async_16(smem_u32(q_s) + swz(r, c, D * 2), qg + (size_t)(real ? r : 0) * D + c * 8, real ? 16 : 0);
  }
}

template <int D>
__device__ __forceinline__ void load_k_tile(const ScoreParams& p, const UnitShape& us, uint8_t* dst, int tile_c0) {
  constexpr int kChunks = D / 8;
  const __nv_bfloat16* kg = p.k + (size_t)us.cu * p.stride_token + (size_t)us.g * p.stride_head;
  for (int idx = threadIdx.x; idx < kKeyTile * kChunks; idx += kPassThreads) {
    const int r = idx / kChunks, c = idx % kChunks;
    const int key = tile_c0 + r;
    const bool in = key < us.t;
    const __nv_bfloat16* src = kg + (size_t)(in ? key : 0) * p.stride_token + c * 8;
    cp_async_16(smem_u32(dst) + swz(r, c, D * 2), src, in ? 16 : 0);
  }
}

// One 128-key tile against all G*W query rows.  A warp owns 32 keys, keeps their B fragments in
// registers and sweeps the query rows 16 at a time.
// PASS 1: online (max, sum of exponentials) per query row in `st` = this warp's [M][2] state.
// PASS 2: `st` = [M] row normalisers (log2 domain); column sums of the tile go to u for keys < key_end.
template <int D, int PASS>
__device__ __forceinline__ void compute_tile(const ScoreParams& p, const UnitShape& us, uint32_t q_base,
                                             uint32_t k_base, float* st, int tile_c0, int key_end) {
  constexpr int kRB = D * 2;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gid = lane >> 2, tig = lane & 3, mat = lane >> 3, mrow_l = lane & 7;
  const int MT = p.M / 16;

  uint32_t bf[2][D / 16][4];
#pragma unroll
  for (int ntp = 0; ntp < 2; ++ntp)
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const int key = 32 * warp + 16 * ntp + (mat >> 1) * 8 + mrow_l;
      ldmatrix_x4(bf[ntp][ks], k_base + swz(key, 2 * ks + (mat & 1), kRB));
    }

  float colsum[4][2];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) colsum[nt][0] = colsum[nt][1] = 0.f;
  const int c_base = tile_c0 + 32 * warp + 2 * tig;

  for (int mt = 0; mt < MT; ++mt) {
    float acc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      uint32_t a[4];
      const int row = 16 * mt + (mat & 1) * 8 + mrow_l;
      ldmatrix_x4(a, q_base + swz(row, 2 * ks + (mat >> 1), kRB));
      // The tensor core adds into its fp32 accumulator with truncation; summing the per-k-step
      // partial products with ordinary round-to-nearest adds keeps the logits accurate enough for
      // the top-k decision.
      float part[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) part[nt][0] = part[nt][1] = part[nt][2] = part[nt][3] = 0.f;
      mma_bf16_16816(part[0], a, bf[0][ks][0], bf[0][ks][1]);
      mma_bf16_16816(part[1], a, bf[0][ks][2], bf[0][ks][3]);
      mma_bf16_16816(part[2], a, bf[1][ks][0], bf[1][ks][1]);
      mma_bf16_16816(part[3], a, bf[1][ks][2], bf[1][ks][3]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[nt][j] += part[nt][j];
    }
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int row = 16 * mt + gid + 8 * half;
      if (PASS == 1) {
        const int limit = us.t - p.window + (row % p.window);   // last visible key of this query row
        float sv[4][2];
        float vmax = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = c_base + 8 * nt + j;
            sv[nt][j] = (c <= limit) ? acc[nt][2 * half + j] * p.scale_log2 : -INFINITY;
            vmax = fmaxf(vmax, sv[nt][j]);
          }
        vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 1));
        vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 2));
        const float m_old = st[2 * row], l_old = st[2 * row + 1];
        const float m_new = fmaxf(m_old, vmax);
        const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
        float sum = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) sum += fast_exp2(sv[nt][0] - m_ref) + fast_exp2(sv[nt][1] - m_ref);
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        const float l_new = l_old * fast_exp2(m_old - m_ref) + sum;
        __syncwarp();
        if (tig == 0) {
          st[2 * row] = m_new;
          st[2 * row + 1] = l_new;
        }
      } else {
        const float mr = st[row];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          colsum[nt][0] += fast_exp2(fmaf(acc[nt][2 * half + 0], p.scale_log2, -mr));
          colsum[nt][1] += fast_exp2(fmaf(acc[nt][2 * half + 1], p.scale_log2, -mr));
        }
      }
    }
  }

  if (PASS == 2) {
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float v = colsum[nt][j];
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        colsum[nt][j] = v;
      }
    if (gid == 0) {
      float* u = p.u + (size_t)us.g * p.total_tokens + us.cu;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int c = c_base + 8 * nt + j;
          if (c < key_end) u[c] = colsum[nt][j];
        }
    }
  }
}

// Combine the four warps' pass-1 states of a split, publish them, and let the last split of the unit
// (atomic ticket) merge all splits into mrow[r] = m_r + log2(l_r) (log2 domain; +inf for rows without
// visible keys) and raise the unit's ready flag.  All threads of the CTA call it.
__device__ __forceinline__ void publish_stats(const ScoreParams& p, const UnitShape& us, int unit, int split,
                                              const float* state, int* s_flag) {
  const int M = p.M, tid = threadIdx.x;
  float2* out = p.stats_part + ((size_t)unit * p.n_splits + split) * M;
  for (int r = tid; r < M; r += kPassThreads) {
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) m = fmaxf(m, state[((size_t)w * M + r) * 2]);
    float l = 0.f;
    if (m > -INFINITY) {
#pragma unroll
      for (int w = 0; w < 4; ++w)
        l += state[((size_t)w * M + r) * 2 + 1] * fast_exp2(state[((size_t)w * M + r) * 2] - m);
    }
    out[r] = make_float2(m, l);
  }
  __threadfence();
  __syncthreads();
  const int n_splits_u = (us.t + p.split_keys - 1) / p.split_keys;
  if (tid == 0) *s_flag = (atomicAdd(&p.unit_ticket[unit], 1) == n_splits_u - 1) ? 1 : 0;
  __syncthreads();
  if (*s_flag) {
    __threadfence();
    for (int r = tid; r < M; r += kPassThreads) {
      const float2* part = p.stats_part + (size_t)unit * p.n_splits * M + r;
      float m = -INFINITY;
      for (int s = 0; s < n_splits_u; ++s) m = fmaxf(m, __ldcg(&part[(size_t)s * M]).x);
      float l = 0.f;
      if (m > -INFINITY)
        for (int s = 0; s < n_splits_u; ++s) {
          const float2 v = __ldcg(&part[(size_t)s * M]);
          l += v.y * exp2f(v.x - m);
        }
      // a normaliser of +inf makes a row contribute exp2(-inf) = 0: rows without visible keys, padding rows
      p.mrow[(size_t)unit * M + r] = (l > 0.f && r < p.M_real) ? m + log2f(l) : INFINITY;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) atomicExch(&p.unit_ready[unit], 1);
  }
}

// Bounded wait for a unit's row normalisers.  Thread 0 polls; returns false on expiry.
__device__ __forceinline__ bool wait_unit_ready(const ScoreParams& p, int unit, int* s_flag) {
  if (threadIdx.x == 0) {
    const int ok = spin_until_ge(&p.unit_ready[unit], 1, p.wait_ns, 100) ? 1 : 0;
    if (!ok) record_status(p.hdr, XKV_ERR_TIMEOUT);
    *s_flag = ok;
  }
  __syncthreads();
  return *s_flag != 0;
}

// Resident variant: a work item is (unit, split); the split's keys stay in shared memory between the two
// passes, so K is read from HBM once.  A CTA runs pass 1 on its split, publishes its row statistics, waits
// (bounded) until all splits of the unit have done so, and runs pass 2 from shared memory.  Items are
// handed out in order from a global counter, and a CTA asks for its next item only when it is free: an
// item that has been handed out is being worked on.  So a waiting CTA depends only on items that are
// running or will be picked up by the next CTA that finishes, and the host uses this variant only when a
// unit has far fewer splits than there are resident CTAs.
template <int D>
__global__ void __launch_bounds__(kPassThreads) score_resident_kernel(const ScoreParams p) {
  using C = PassCfg<D>;
  extern __shared__ __align__(128) uint8_t smem[];
  const int M = p.M;
  uint8_t* q_s = smem;
  uint8_t* k_s = smem + (size_t)M * C::kRowBytes;
  float* state = reinterpret_cast<float*>(k_s + (size_t)p.slice_tiles * C::kTileBytes);
  int* s_ctl = reinterpret_cast<int*>(state + (size_t)4 * M * 2);
  const int tid = threadIdx.x, warp = tid >> 5;

  while (true) {
    __syncthreads();
    if (tid == 0) s_ctl[0] = atomicAdd(&p.hdr->work_counter, 1);
    __syncthreads();
    const int idx = s_ctl[0];
    if (idx >= p.n_work) break;
    const int unit = idx / p.n_splits, split = idx % p.n_splits;
    const UnitShape us = unit_shape(p, unit);
    const int key_begin = split * p.split_keys;
    const int key_end1 = min(key_begin + p.split_keys, us.t);
    if (key_begin >= key_end1) continue;
    const int n_tiles = (key_end1 - key_begin + kKeyTile - 1) / kKeyTile;

    load_q<D>(p, us, q_s);
    for (int ti = 0; ti < n_tiles; ++ti)
      load_k_tile<D>(p, us, k_s + (size_t)ti * C::kTileBytes, key_begin + ti * kKeyTile);
    cp_async_commit();
    for (int i = tid; i < 4 * M; i += kPassThreads) {
      state[2 * i] = -INFINITY;
      state[2 * i + 1] = 0.f;
    }
    cp_async_wait<0>();
    __syncthreads();

    const uint32_t q_base = smem_u32(q_s);
    for (int ti = 0; ti < n_tiles; ++ti)
      compute_tile<D, 1>(p, us, q_base, smem_u32(k_s + (size_t)ti * C::kTileBytes), state + (size_t)warp * M * 2,
                         key_begin + ti * kKeyTile, 0);
    __syncthreads();
    publish_stats(p, us, unit, split, state, &s_ctl[1]);

    const int key_end2 = min(key_end1, us.P);
    if (key_begin >= key_end2) continue;           // a split that holds window keys only
    if (!wait_unit_ready(p, unit, &s_ctl[2])) continue;
    for (int r = tid; r < M; r += kPassThreads) state[r] = __ldcg(&p.mrow[(size_t)unit * M + r]);
    __syncthreads();
    const int n_tiles2 = (key_end2 - key_begin + kKeyTile - 1) / kKeyTile;
    for (int ti = 0; ti < n_tiles2; ++ti)
      compute_tile<D, 2>(p, us, q_base, smem_u32(k_s + (size_t)ti * C::kTileBytes), state, key_begin + ti * kKeyTile,
                         key_end2);
  }
}

// Streaming variant for sequences too long for the resident one: all pass-1 items, then all pass-2 items,
// from one global counter; key tiles go through a cp.async ring.  A pass-2 item waits (bounded) for its
// unit's ready flag, which is long set except right at the boundary between the two phases.  Pass-1 items
// never wait, and every pass-1 item has a lower index than every pass-2 item, so fetching the next index
// early cannot hold back an item somebody waits for.
template <int D>
__global__ void __launch_bounds__(kPassThreads) score_stream_kernel(const ScoreParams p) {
  using C = PassCfg<D>;
  extern __shared__ __align__(128) uint8_t smem[];
  const int M = p.M;
  uint8_t* q_s = smem;
  uint8_t* k_s = smem + (size_t)M * C::kRowBytes;
  float* state = reinterpret_cast<float*>(k_s + (size_t)kPassStages * C::kTileBytes);
  int* s_ctl = reinterpret_cast<int*>(state + (size_t)4 * M * 2);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int half_work = p.n_work / 2;

  int next = 0;
  if (tid == 0) next = atomicAdd(&p.hdr->work_counter, 1);
  while (true) {
    __syncthreads();
    if (tid == 0) {
      s_ctl[0] = next;
      next = atomicAdd(&p.hdr->work_counter, 1);      // fetched now, used after this item
    }
    __syncthreads();
    const int idx = s_ctl[0];
    if (idx >= p.n_work) break;
    const int pass = idx < half_work ? 1 : 2;
    const int rem = idx < half_work ? idx : idx - half_work;
    const int unit = rem / p.n_splits, split = rem % p.n_splits;
    const UnitShape us = unit_shape(p, unit);
    const int key_begin = split * p.split_keys;
    const int key_end = min(key_begin + p.split_keys, pass == 1 ? us.t : us.P);
    if (key_begin >= key_end) continue;
    if (pass == 2) {
      if (!wait_unit_ready(p, unit, &s_ctl[2])) continue;
      for (int r = tid; r < M; r += kPassThreads) state[r] = __ldcg(&p.mrow[(size_t)unit * M + r]);
    } else {
      for (int i = tid; i < 4 * M; i += kPassThreads) {
        state[2 * i] = -INFINITY;
        state[2 * i + 1] = 0.f;
      }
    }

    const int n_tiles = (key_end - key_begin + kKeyTile - 1) / kKeyTile;
    load_q<D>(p, us, q_s);
#pragma unroll
    for (int s = 0; s < kPassStages - 1; ++s) {
      if (s < n_tiles) load_k_tile<D>(p, us, k_s + (size_t)s * C::kTileBytes, key_begin + s * kKeyTile);
      cp_async_commit();
    }
    const uint32_t q_base = smem_u32(q_s);
    for (int ti = 0; ti < n_tiles; ++ti) {
      cp_async_wait<kPassStages - 2>();
      __syncthreads();          // tile ti has landed for everyone; the buffer of tile ti-1 is free
      if (ti + kPassStages - 1 < n_tiles)
        load_k_tile<D>(p, us, k_s + (size_t)((ti + kPassStages - 1) % kPassStages) * C::kTileBytes,
                       key_begin + (ti + kPassStages - 1) * kKeyTile);
      cp_async_commit();
      const uint32_t k_base = smem_u32(k_s + (size_t)(ti % kPassStages) * C::kTileBytes);
      if (pass == 1)
        compute_tile<D, 1>(p, us, q_base, k_base, state + (size_t)warp * M * 2, key_begin + ti * kKeyTile, 0);
      else
        compute_tile<D, 2>(p, us, q_base, k_base, state, key_begin + ti * kKeyTile, key_end);
    }
    cp_async_wait<0>();
    __syncthreads();
    if (pass == 1) publish_stats(p, us, unit, split, state, &s_ctl[1]);
  }
}

// ---------------------------------------------------------------------------------------------
// Pooling + chunk sort.  grid = (units, n_chunks).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSortThreads) pool_sort_kernel(const ScoreParams p, float* sort_out) {
  __shared__ float s_u[kSortChunk + 64];
  __shared__ __align__(16) float s_key[kSortChunk];
  __shared__ float s_red[32];
  const int unit = blockIdx.x, chunk = blockIdx.y;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  const int cu = p.cu_seqlens[b];
  const int t_given = p.cu_seqlens[b + 1] - cu;
  const int t = min(t_given, p.max_seqlen);
  if (t_given > p.max_seqlen && chunk == 0 && g == 0 && threadIdx.x == 0)
    record_status(p.hdr, XKV_ERR_INVALID_ARG);       // a prompt longer than the bound the grids were sized for
  const int P = max(t - p.window, 0);
  const int c0 = chunk * kSortChunk;
  const int tid = threadIdx.x;
  const size_t seg = (size_t)g * p.total_tokens + cu;
  const int half = p.pool_kernel / 2;
  if (c0 >= t) return;

  // u with halo; positions outside the prefix read as "absent"
  for (int i = tid; i < kSortChunk + 2 * half; i += kSortThreads) {
    const int c = c0 - half + i;
    s_u[i] = (c >= 0 && c < P) ? p.u[seg + c] : -1.f;
  }
  __syncthreads();

  float local = 0.f;
  for (int i = tid; i < kSortChunk; i += kSortThreads) {
    const int c = c0 + i;
    float w = -1.f;
    if (c < P) {
      if (p.pool_mode == XKV_POOL_MAX) {
        w = 0.f;
        for (int j = 0; j <= 2 * half; ++j) w = fmaxf(w, s_u[i + j]);   // absent entries are -1
      } else {
        float acc = 0.f;
        for (int j = 0; j <= 2 * half; ++j) acc += fmaxf(s_u[i + j], 0.f);
        w = acc / (float)p.pool_kernel;
      }
      p.scores[seg + c] = w;
      local += w;
    } else if (c < t) {
      p.scores[seg + c] = 0.f;
      if (sort_out != nullptr) {
        p.sorted[seg + c] = 0.f;
        p.tmp_sorted[seg + c] = 0.f;
      }
    }
    s_key[i] = w;
  }
  // deterministic block sum of this chunk's scores
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((tid & 31) == 0) s_red[tid >> 5] = local;
  __syncthreads();
  if (tid < 32) {
    float v = tid < kSortThreads / 32 ? s_red[tid] : 0.f;
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (tid == 0) p.part_sum[(size_t)unit * p.n_chunks + chunk] = v;
  }
  if (sort_out == nullptr) return;
  if (c0 >= P) return;

  // Bitonic sort, descending; absent entries (-1) end up last.  Thread t holds elements 8t..8t+7 in
  // registers: exchanges at distance < 8 stay in the thread, distances 8..128 are warp shuffles, and
  // only the ten steps at distance >= 256 go through shared memory.
  static_assert(kSortItems == 8, "the exchange pattern below assumes 8 scores per thread");
  __syncthreads();
  float e[kSortItems];
  {
    const float4 lo = *reinterpret_cast<const float4*>(&s_key[8 * tid]);
    const float4 hi = *reinterpret_cast<const float4*>(&s_key[8 * tid + 4]);
    e[0] = lo.x; e[1] = lo.y; e[2] = lo.z; e[3] = lo.w;
    e[4] = hi.x; e[5] = hi.y; e[6] = hi.z; e[7] = hi.w;
  }
#pragma unroll
  for (int k = 2; k <= kSortChunk; k <<= 1) {
#pragma unroll
    for (int j = k >> 1; j > 0; j >>= 1) {
      if (j >= 8) {
        const int m = j >> 3;                                   // partner thread = tid ^ m
        const bool lower = (tid & m) == 0;
        const bool desc = (tid & (k >> 3)) == 0;
        const bool want_max = lower == desc;
        float o[kSortItems];
        if (m >= 32) {
          __syncthreads();
          *reinterpret_cast<float4*>(&s_key[8 * tid]) = make_float4(e[0], e[1], e[2], e[3]);
          *reinterpret_cast<float4*>(&s_key[8 * tid + 4]) = make_float4(e[4], e[5], e[6], e[7]);
          __syncthreads();
          const float4 lo = *reinterpret_cast<const float4*>(&s_key[8 * (tid ^ m)]);
          const float4 hi = *reinterpret_cast<const float4*>(&s_key[8 * (tid ^ m) + 4]);
          o[0] = lo.x; o[1] = lo.y; o[2] = lo.z; o[3] = lo.w;
          o[4] = hi.x; o[5] = hi.y; o[6] = hi.z; o[7] = hi.w;
        } else {
#pragma unroll
          for (int r = 0; r < kSortItems; ++r) o[r] = __shfl_xor_sync(0xffffffffu, e[r], m);
        }
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) e[r] = want_max ? fmaxf(e[r], o[r]) : fminf(e[r], o[r]);
      } else {
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) {
          if ((r & j) == 0) {
            const bool desc = k < 8 ? ((r & k) == 0) : ((tid & (k >> 3)) == 0);
            const float hi = fmaxf(e[r], e[r | j]), lo = fminf(e[r], e[r | j]);
            e[r] = desc ? hi : lo;
            e[r | j] = desc ? lo : hi;
          }
        }
      }
    }
  }
  __syncthreads();
  *reinterpret_cast<float4*>(&s_key[8 * tid]) = make_float4(e[0], e[1], e[2], e[3]);
  *reinterpret_cast<float4*>(&s_key[8 * tid + 4]) = make_float4(e[4], e[5], e[6], e[7]);
  __syncthreads();
  const int n_valid = min(kSortChunk, P - c0);
  for (int i = tid; i < n_valid; i += kSortThreads) sort_out[seg + c0 + i] = s_key[i];
}

// ---------------------------------------------------------------------------------------------
// One merge pass: runs of length `run` (descending) are merged pairwise.  grid = (units, tiles).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int merge_path(const float* A, int la, const float* B, int lb, int diag) {
  int lo = max(0, diag - lb), hi = min(diag, la);
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (A[mid] >= B[diag - 1 - mid]) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// The same split point found by a whole warp: 32 probes per round instead of one, so a run of 64K scores takes four
// rounds of global loads instead of sixteen.  All lanes return the result.
__device__ __forceinline__ int merge_path_warp(const float* A, int la, const float* B, int lb, int diag) {
  const int lane = threadIdx.x & 31;
  int lo = max(0, diag - lb), hi = min(diag, la);
  while (lo < hi) {
    const int step = (hi - lo + 31) / 32;
    const int q = lo + (lane + 1) * step - 1;                 // probe positions, ascending with the lane
    const bool in = q < hi;
    const bool ge = in && A[q] >= B[diag - 1 - q];            // true on a prefix of the lanes
    const unsigned m = __ballot_sync(0xffffffffu, ge);
    const int c = __popc(m);                                   // the split lies beyond the first c probes
    const int q_c = lo + (c + 1) * step - 1;                   // first probe that failed (if it exists)
    lo = lo + c * step;
    if (c < 32 && q_c < hi) hi = q_c;
    if (lo > hi) lo = hi;
  }
  return lo;
}

__global__ void __launch_bounds__(kMergeThreads) merge_kernel(const ScoreParams p, const float* src, float* dst,
                                                             int run) {
  __shared__ float s_in[kMergeTile];
  __shared__ int s_split[2];
  const int unit = blockIdx.x;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  const int cu = p.cu_seqlens[b];
  const int t = min(p.cu_seqlens[b + 1] - cu, p.max_seqlen);
  const int P = max(t - p.window, 0);
  const int o0 = blockIdx.y * kMergeTile;
  if (o0 >= P) return;
  const size_t seg = (size_t)g * p.total_tokens + cu;
  const int pair0 = (o0 / (2 * run)) * (2 * run);
  const int la = min(run, P - pair0);
  const int lb = max(0, min(run, P - pair0 - run));
  const float* A = src + seg + pair0;
  const float* B = A + run;
  const int d0 = o0 - pair0;
  const int d1 = min(d0 + kMergeTile, la + lb);
  if (threadIdx.x < 64) {                      // warp 0 finds the tile's start, warp 1 its end
    const int w = threadIdx.x >> 5;
    const int split = merge_path_warp(A, la, B, lb, w == 0 ? d0 : d1);
    if ((threadIdx.x & 31) == 0) s_split[w] = split;
  }
  __syncthreads();
  const int a0 = s_split[0], a1 = s_split[1];
  const int b0 = d0 - a0, b1 = d1 - a1;
  const int na = a1 - a0, nb = b1 - b0;
  for (int i = threadIdx.x; i < na; i += kMergeThreads) s_in[i] = A[a0 + i];
  for (int i = threadIdx.x; i < nb; i += kMergeThreads) s_in[na + i] = B[b0 + i];
  __syncthreads();
  const float* SA = s_in;
  const float* SB = s_in + na;
  const int n_out = d1 - d0;
  const int my0 = min(threadIdx.x * kMergeItems, n_out);
  const int my1 = min(my0 + kMergeItems, n_out);
  int ia = merge_path(SA, na, SB, nb, my0);
  int ib = my0 - ia;
  for (int o = my0; o < my1; ++o) {
    const bool take_a = (ib >= nb) || (ia < na && SA[ia] >= SB[ib]);
    dst[seg + pair0 + d0 + o] = take_a ? SA[ia++] : SB[ib++];
  }
}

// ---------------------------------------------------------------------------------------------
// gains[b][j] = mean over KV heads of sorted[g][j] / sum_c w_g[c].  grid = (tiles, B).
// ---------------------------------------------------------------------------------------------
__global__ void gains_kernel(const ScoreParams p) {
  extern __shared__ float s_inv[];   // [Hkv]
  const int b = blockIdx.y;
  const int cu = p.cu_seqlens[b];
  const int t = min(p.cu_seqlens[b + 1] - cu, p.max_seqlen);
  const int P = max(t - p.window, 0);
  for (int g = threadIdx.x; g < p.n_kv_heads; g += blockDim.x) {
    const float* ps = p.part_sum + ((size_t)b * p.n_kv_heads + g) * p.n_chunks;
    float s = 0.f;
    const int used = (P + kSortChunk - 1) / kSortChunk;
    for (int c = 0; c < used; ++c) s += ps[c];
    s_inv[g] = s > 0.f ? 1.f / s : 0.f;
  }
  __syncthreads();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= p.curve_len) return;
  float acc = 0.f;
  if (j < P)
    for (int g = 0; g < p.n_kv_heads; ++g) acc += p.sorted[(size_t)g * p.total_tokens + cu + j] * s_inv[g];
  p.gains[(size_t)b * p.curve_len + j] = acc / (float)p.n_kv_heads;
}

// mass[b][n] = inclusive prefix sum of gains[b].  grid = B, 1024 threads.
__global__ void __launch_bounds__(1024) mass_kernel(const ScoreParams p) {
  __shared__ float s_warp[32];
  __shared__ float s_carry;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_carry = 0.f;
  __syncthreads();
  for (int base = 0; base < p.curve_len; base += 1024) {
    const int j = base + tid;
    const float v = j < p.curve_len ? p.gains[(size_t)b * p.curve_len + j] : 0.f;
    float incl = v;
    for (int o = 1; o < 32; o <<= 1) {
      const float u = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += u;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      float w = s_warp[lane];
      float winc = w;
      for (int o = 1; o < 32; o <<= 1) {
        const float u = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += u;
      }
      s_warp[lane] = winc - w;
    }
    __syncthreads();
    const float carry = s_carry;
    const float r = carry + s_warp[warp] + incl;
    if (j < p.curve_len) p.mass[(size_t)b * p.curve_len + j] = r;
    __syncthreads();
    if (tid == 1023) s_carry = r;
    __syncthreads();
  }
}

// mrow[unit][row] = the given softmax normaliser (natural log of the row's sum of exponentials) of window row
// `row` = (query head within the group) * W + r, in log2 units; +inf for rows before the start of a sequence shorter
// than the window, so that they contribute nothing.  grid = units, block = M.
__global__ void mrow_from_lse_kernel(const ScoreParams p, const float* lse) {
  const int unit = blockIdx.x, row = threadIdx.x;
  if (row >= p.M) return;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  const int cu = p.cu_seqlens[b];
  const int t = min(p.cu_seqlens[b + 1] - cu, p.max_seqlen);
  const int h = g * p.group + row / p.window;
  const int pos = t - p.window + row % p.window;
  p.mrow[(size_t)unit * p.M + row] =
      pos >= 0 ? lse[(size_t)h * p.total_tokens + cu + pos] * 1.4426950408889634f : INFINITY;
}

struct ScoreLayout {
  size_t flags, u, tmp_sorted, stats_part, mrow, part_sum, total;
  int split_keys, n_splits, n_chunks, slice_tiles, ctas_per_sm;
  bool resident, use_tc;
};

void score_layout(const xkv_dims* d, int max_seqlen, int64_t T, ScoreLayout* L) {
  const int units = d->batch * d->n_kv_heads;
  const int M_real = (d->n_q_heads / d->n_kv_heads) * d->window;
  const int M = (M_real + 15) / 16 * 16;
  const int sms = sm_count();
  // Resident variant: key tiles per split chosen so that two CTAs fit on an SM (one for G*W = 256).
  int tiles = M <= 64 ? 3 : (M <= 128 ? 2 : 4);
  while (tiles > 1 && (int64_t)units * ((max_seqlen + tiles * kKeyTile - 1) / (tiles * kKeyTile)) < 2 * sms) --tiles;
  const size_t tile_bytes = (size_t)kKeyTile * d->head_dim * 2;
  const size_t fixed = (size_t)M * d->head_dim * 2 + (size_t)4 * M * 8 + 64;
  auto ctas_for = [&](size_t smem) {
    int c = (int)((227u * 1024u) / (smem + 1024));
    return c < 1 ? 1 : (c > 3 ? 3 : c);
  };
  const int res_ctas = ctas_for(fixed + tiles * tile_bytes);
  const int res_splits = (max_seqlen + tiles * kKeyTile - 1) / (tiles * kKeyTile);
  // every split of a unit must be in flight at once with room to spare (CTAs of a unit wait for each other)
  L->resident = res_splits * 4 <= sms * (res_ctas < 2 ? res_ctas : 2);
  if (L->resident) {
    L->slice_tiles = tiles;
    L->split_keys = tiles * kKeyTile;
    L->ctas_per_sm = res_ctas;
  } else {
    int split = 1024;
    while (split > kKeyTile && (int64_t)units * ((max_seqlen + split - 1) / split) < 2 * sms) split >>= 1;
    L->slice_tiles = kPassStages;
    L->split_keys = split;
    L->ctas_per_sm = ctas_for(fixed + kPassStages * tile_bytes);
  }
  // the tcgen05 kernel takes the passes over when it covers the shape (it is a resident variant too)
  const int tc_split = M_real == M ? score_tc_split_keys(M, d->head_dim, units, max_seqlen) : 0;
  L->use_tc = tc_split > 0;
  if (L->use_tc) {
    L->resident = true;            // one work item per (unit, split); the kernel runs as two launches
    L->split_keys = tc_split;
    L->slice_tiles = tc_split / kKeyTile;
  }
  L->n_splits = (max_seqlen + L->split_keys - 1) / L->split_keys;
  L->n_chunks = (max_seqlen + kSortChunk - 1) / kSortChunk;
  size_t off = kHeaderBytes;
  L->flags = off;      off = align_up(off + (size_t)units * 8, 256);
  L->u = off;          off = align_up(off + (size_t)d->n_kv_heads * T * 4, 256);
  L->tmp_sorted = off; off = align_up(off + (size_t)d->n_kv_heads * T * 4, 256);
  // sized for the smallest split either variant may choose, so the size does not depend on the device
  L->stats_part = off; off = align_up(off + (size_t)units * ((max_seqlen + kKeyTile - 1) / kKeyTile) * (M < 128 ? 128 : M) * 2 * 8, 256);
  L->mrow = off;       off = align_up(off + (size_t)units * M * 4, 256);
  L->part_sum = off;   off = align_up(off + (size_t)units * L->n_chunks * 4, 256);
  L->total = off;
}

template <int D>
xkv_status launch_passes(const ScoreParams& p, const ScoreLayout& L, cudaStream_t st) {
  const size_t smem = PassCfg<D>::smem_bytes(p.M, L.slice_tiles);
  static std::atomic<bool> done[64];   // idempotent set-up: two threads doing it twice is harmless
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  if (!done[dev].load(std::memory_order_acquire)) {
    const int max_smem = 227 * 1024;
    if (cudaFuncSetAttribute(score_stream_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) !=
            cudaSuccess ||
        cudaFuncSetAttribute(score_resident_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) !=
            cudaSuccess)
      return XKV_ERR_CUDA;
    done[dev].store(true, std::memory_order_release);
  }
  int grid = sm_count() * L.ctas_per_sm;
  if (grid > p.n_work) grid = p.n_work;
  if (L.resident)
    score_resident_kernel<D><<<grid, kPassThreads, smem, st>>>(p);
  else
    score_stream_kernel<D><<<grid, kPassThreads, smem, st>>>(p);
  count_launch();
  return check_launch();
}

}  // namespace

int score_lse_supported(const xkv_dims* d, int max_seqlen) {
  ScoreLayout L;
  score_layout(d, max_seqlen, max_seqlen, &L);
  return L.use_tc ? 1 : 0;
}

size_t score_workspace_bytes(const xkv_dims* d, int max_seqlen, int64_t total_tokens) {
  ScoreLayout L;
  score_layout(d, max_seqlen, total_tokens, &L);
  return L.total;
}

xkv_status score(const xkv_dims* d, const void* q_win, const void* k, const int32_t* cu_seqlens,
                 int64_t total_tokens, int max_seqlen, float* scores, float* sorted, float* gains, float* mass,
                 int curve_len, void* workspace, size_t workspace_bytes, cudaStream_t st, const float* lse) {
  ScoreLayout L;
  score_layout(d, max_seqlen, total_tokens, &L);
  if (workspace_bytes < L.total) return XKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const int units = d->batch * d->n_kv_heads;

  ScoreParams p;
  p.q_win = static_cast<const __nv_bfloat16*>(q_win);
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.cu_seqlens = cu_seqlens;
  p.scores = scores;
  p.sorted = sorted;
  p.gains = gains;
  p.mass = mass;
  p.u = reinterpret_cast<float*>(ws + L.u);
  p.tmp_sorted = reinterpret_cast<float*>(ws + L.tmp_sorted);
  p.stats_part = reinterpret_cast<float2*>(ws + L.stats_part);
  p.mrow = reinterpret_cast<float*>(ws + L.mrow);
  p.part_sum = reinterpret_cast<float*>(ws + L.part_sum);
  p.total_tokens = total_tokens;
  p.stride_token = d->kv_stride_token;
  p.stride_head = d->kv_stride_head;
  p.batch = d->batch;
  p.n_q_heads = d->n_q_heads;
  p.n_kv_heads = d->n_kv_heads;
  p.group = d->n_q_heads / d->n_kv_heads;
  p.window = d->window;
  p.M_real = p.group * d->window;
  p.M = (p.M_real + 15) / 16 * 16;
  p.pool_kernel = d->pool_kernel;
  p.pool_mode = d->pool_mode;
  p.split_keys = L.split_keys;
  p.n_splits = L.n_splits;
  p.n_chunks = L.n_chunks;
  p.curve_len = curve_len;
  p.hdr = reinterpret_cast<WorkspaceHeader*>(ws);
  p.unit_ticket = reinterpret_cast<int32_t*>(ws + L.flags);
  p.unit_ready = p.unit_ticket + units;
  p.slice_tiles = L.slice_tiles;
  p.n_work = (L.resident ? 1 : 2) * units * L.n_splits;
  const float scale = d->scale != 0.f ? d->scale : 1.0f / sqrtf((float)d->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  p.max_seqlen = max_seqlen;
  p.wait_ns = wait_limit_ns();

  // counters, tickets and ready flags start at zero; the status word (first four bytes) keeps an unread error
  if (cudaMemsetAsync(ws + 4, 0, L.u - 4, st) != cudaSuccess) return XKV_ERR_CUDA;
  xkv_status s;
  if (lse != nullptr) {
    // the row normalisers come from the prefill attention: only the column-sum pass runs
    if (!L.use_tc) return XKV_ERR_UNSUPPORTED;
    mrow_from_lse_kernel<<<units, p.M, 0, st>>>(p, lse);
    count_launch();
    s = check_launch();
    if (s != XKV_OK) return s;
    s = score_tc_pass2(p, d->head_dim, max_seqlen, st);
  } else if (L.use_tc && score_fused_covers(p.M, d->head_dim, units, max_seqlen)) {
    s = score_fused_pass(p, d->head_dim, max_seqlen, st);      // both passes in one cluster kernel, keys read once
  } else if (L.use_tc) {
    s = score_tc_passes(p, d->head_dim, max_seqlen, st);
  } else {
    s = d->head_dim == 128 ? launch_passes<128>(p, L, st) : launch_passes<64>(p, L, st);
  }
  if (s != XKV_OK) return s;

  // chunk sort, then log2(n_chunks) merge passes ping-ponging so that the last one lands in `sorted`
  int n_pass = 0;
  for (int run = kSortChunk; run < max_seqlen; run <<= 1) ++n_pass;
  float* first_out = sorted == nullptr ? nullptr : ((n_pass % 2 == 0) ? sorted : p.tmp_sorted);
  pool_sort_kernel<<<dim3(units, L.n_chunks), kSortThreads, 0, st>>>(p, first_out);
  count_launch();
  s = check_launch();
  if (s != XKV_OK || sorted == nullptr) return s;
  {
    float* src = first_out;
    float* dst = (src == sorted) ? p.tmp_sorted : sorted;
    const int tiles = (max_seqlen + kMergeTile - 1) / kMergeTile;
    for (int run = kSortChunk; run < max_seqlen; run <<= 1) {
      merge_kernel<<<dim3(units, tiles), kMergeThreads, 0, st>>>(p, src, dst, run);
      count_launch();
      s = check_launch();
      if (s != XKV_OK) return s;
      float* tmp = src; src = dst; dst = tmp;
    }
  }
  gains_kernel<<<dim3((curve_len + 255) / 256, d->batch), 256, d->n_kv_heads * sizeof(float), st>>>(p);
  count_launch();
  s = check_launch();
  if (s != XKV_OK) return s;
  if (mass != nullptr) {
    mass_kernel<<<d->batch, 1024, 0, st>>>(p);
    count_launch();
    s = check_launch();
  }
  return s;
}

}  // namespace xkv
