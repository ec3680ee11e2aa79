// xkv_score: importance scoring of one layer (Eq. 2, Eq. 3, Eq. 4; Alg. 2 steps 1-4).
//
// Kernels, in stream order:
//   score_pass_kernel<D,1>  softmax row statistics (max, sum of exponentials) of the G*W window
//                           query rows over their visible keys, per split of the key axis
//   stats_merge_kernel      merge the per-split statistics into one log2-domain normaliser per row
//   score_pass_kernel<D,2>  recompute the logits and accumulate the column sums u[c] over the
//                           G*W rows (Select + Merge; the GQA group is summed before pooling)
//   pool_sort_kernel        1-D pooling (max or zero-padded average) of u into the scores w, and a
//                           descending bitonic sort of each 4096-score chunk in shared memory
//   merge_kernel            merge-path passes that combine the sorted chunks of a segment
//   gains_kernel / mass_kernel  the per-sequence retained-importance curve of the layer
//
// Both logit passes are the one dense contraction of the path and run on tensor cores
// (mma.sync m16n8k16, bf16 in, fp32 accumulate): a warp owns 32 keys of a 128-key tile, keeps
// their B fragments in registers and sweeps all G*W query rows, so per-row statistics stay with a
// thread quad and column sums complete inside the warp.  The exact method needs two passes: the
// row normalisers must be final before a column sum can be formed.
#include <cmath>

#include "common.cuh"
#include "ops.h"

namespace xkv {
namespace {

#ifndef XKV_SPLIT_ACC
#define XKV_SPLIT_ACC 1
#endif

constexpr int kPassThreads = 128;     // 4 warps
constexpr int kKeyTile = 128;         // keys per tile, 32 per warp
constexpr int kSortChunk = 4096;      // scores sorted per CTA
constexpr int kSortThreads = 1024;
constexpr int kMergeTile = 2048;
constexpr int kMergeThreads = 256;
constexpr int kMergeItems = kMergeTile / kMergeThreads;

struct ScoreParams {
  const __nv_bfloat16* q_win;
  const __nv_bfloat16* k;
  const int32_t* cu_seqlens;
  float* scores;
  float* sorted;
  float* gains;
  float* mass;
  float* u;            // [Hkv][T] un-pooled column sums
  float* tmp_sorted;   // [Hkv][T] ping-pong buffer of the merge passes
  float2* stats_part;  // [units][n_splits][M]
  float* mrow;         // [units][M]
  float* part_sum;     // [units][n_chunks]
  int64_t total_tokens, stride_token, stride_head;
  int32_t batch, n_q_heads, n_kv_heads, group, window, M, pool_kernel, pool_mode;
  int32_t split_keys, n_splits, n_chunks, curve_len;
  float scale_log2;
};

template <int D>
struct PassCfg {
  static constexpr int kRowElems = D + 8;   // padded shared-memory row: conflict-free ldmatrix
  static constexpr int kRowBytes = kRowElems * 2;
  static constexpr int kTileBytes = kKeyTile * kRowBytes;
  static size_t smem_bytes(int M) { return (size_t)M * kRowBytes + 2 * kTileBytes + (size_t)4 * M * 8; }
};

// One CTA: unit (b, g) = blockIdx.x, key range split = blockIdx.y.
template <int D, int PASS>
__global__ void __launch_bounds__(kPassThreads) score_pass_kernel(const ScoreParams p) {
  using C = PassCfg<D>;
  extern __shared__ __align__(16) uint8_t smem[];
  const int M = p.M;
  uint8_t* q_s = smem;
  uint8_t* k_s = smem + (size_t)M * C::kRowBytes;
  float* state = reinterpret_cast<float*>(k_s + 2 * C::kTileBytes);   // pass 1: [4][M][2]; pass 2: [M]

  const int unit = blockIdx.x;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  const int cu = p.cu_seqlens[b];
  const int t = p.cu_seqlens[b + 1] - cu;
  const int P = max(t - p.window, 0);
  const int key_end_all = (PASS == 1) ? t : P;
  const int key_begin = blockIdx.y * p.split_keys;
  const int key_end = min(key_begin + p.split_keys, key_end_all);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3, mat = lane >> 3, mrow_l = lane & 7;

  if (PASS == 1) {
    float2* out = p.stats_part + ((size_t)unit * p.n_splits + blockIdx.y) * M;
    if (key_begin >= key_end) {       // empty split: neutral statistics
      for (int r = tid; r < M; r += kPassThreads) out[r] = make_float2(-INFINITY, 0.f);
      return;
    }
  } else if (key_begin >= key_end) {
    return;
  }

  // ---- stage the query rows of the group (G*W x D) and the first key tile
  const __nv_bfloat16* qg = p.q_win + ((size_t)b * p.n_q_heads + (size_t)g * p.group) * p.window * D;
  constexpr int kChunksPerRow = D / 8;
  for (int idx = tid; idx < M * kChunksPerRow; idx += kPassThreads) {
    const int r = idx / kChunksPerRow, c = idx % kChunksPerRow;
    cp_async_16(smem_u32(q_s + r * C::kRowBytes + c * 16), qg + (size_t)r * D + c * 8, 16);
  }
  const __nv_bfloat16* kg = p.k + (size_t)cu * p.stride_token + (size_t)g * p.stride_head;
  auto load_tile = [&](int tile_c0, int buf) {
    uint8_t* dst = k_s + buf * C::kTileBytes;
    for (int idx = tid; idx < kKeyTile * kChunksPerRow; idx += kPassThreads) {
      const int r = idx / kChunksPerRow, c = idx % kChunksPerRow;
      const int key = tile_c0 + r;
      const bool in = key < t;
      const __nv_bfloat16* src = kg + (size_t)(in ? key : 0) * p.stride_token + c * 8;
      cp_async_16(smem_u32(dst + r * C::kRowBytes + c * 16), src, in ? 16 : 0);
    }
  };
  load_tile(key_begin, 0);
  cp_async_commit();

  if (PASS == 1) {
    for (int i = tid; i < 4 * M; i += kPassThreads) {
      state[2 * i] = -INFINITY;
      state[2 * i + 1] = 0.f;
    }
  } else {
    for (int r = tid; r < M; r += kPassThreads) state[r] = p.mrow[(size_t)unit * M + r];
  }

  const int n_tiles = (key_end - key_begin + kKeyTile - 1) / kKeyTile;
  const int MT = M / 16;
  const uint32_t q_base = smem_u32(q_s);
  float* my_state = state + (size_t)warp * M * 2;

  for (int ti = 0; ti < n_tiles; ++ti) {
    const int tile_c0 = key_begin + ti * kKeyTile;
    if (ti + 1 < n_tiles) {
      load_tile(tile_c0 + kKeyTile, (ti + 1) & 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();

    const uint32_t k_base = smem_u32(k_s + (ti & 1) * C::kTileBytes);
    uint32_t bf[2][D / 16][4];
#pragma unroll
    for (int ntp = 0; ntp < 2; ++ntp)
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const int key = 32 * warp + 16 * ntp + (mat >> 1) * 8 + mrow_l;
        const int col = 16 * ks + (mat & 1) * 8;
        ldmatrix_x4(bf[ntp][ks], k_base + key * C::kRowBytes + col * 2);
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
        const int col = 16 * ks + (mat >> 1) * 8;
        ldmatrix_x4(a, q_base + row * C::kRowBytes + col * 2);
#if XKV_SPLIT_ACC
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
#else
        mma_bf16_16816(acc[0], a, bf[0][ks][0], bf[0][ks][1]);
        mma_bf16_16816(acc[1], a, bf[0][ks][2], bf[0][ks][3]);
        mma_bf16_16816(acc[2], a, bf[1][ks][0], bf[1][ks][1]);
        mma_bf16_16816(acc[3], a, bf[1][ks][2], bf[1][ks][3]);
#endif
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int row = 16 * mt + gid + 8 * half;
        if (PASS == 1) {
          const int limit = t - p.window + (row % p.window);   // last visible key of this query row
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
          const float m_old = my_state[2 * row], l_old = my_state[2 * row + 1];
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
            my_state[2 * row] = m_new;
            my_state[2 * row + 1] = l_new;
          }
        } else {
          const float mr = state[row];
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
        float* u = p.u + (size_t)g * p.total_tokens + cu;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = c_base + 8 * nt + j;
            if (c < key_end) u[c] = colsum[nt][j];
          }
      }
    }
    __syncthreads();   // the tile buffer is overwritten by the load issued in the next iteration
  }

  if (PASS == 1) {
    float2* out = p.stats_part + ((size_t)unit * p.n_splits + blockIdx.y) * M;
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
  }
}

// One CTA per unit: mrow[r] = m_r + log2(l_r) in the log2 domain, +inf for rows without keys.
__global__ void stats_merge_kernel(const ScoreParams p) {
  const int unit = blockIdx.x;
  const int M = p.M;
  for (int r = threadIdx.x; r < M; r += blockDim.x) {
    const float2* part = p.stats_part + (size_t)unit * p.n_splits * M + r;
    float m = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) m = fmaxf(m, part[(size_t)s * M].x);
    float l = 0.f;
    if (m > -INFINITY)
      for (int s = 0; s < p.n_splits; ++s) {
        const float2 v = part[(size_t)s * M];
        l += v.y * exp2f(v.x - m);
      }
    p.mrow[(size_t)unit * M + r] = (l > 0.f) ? m + log2f(l) : INFINITY;
  }
}

// ---------------------------------------------------------------------------------------------
// Pooling + chunk sort.  grid = (units, n_chunks).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSortThreads) pool_sort_kernel(const ScoreParams p, float* sort_out) {
  __shared__ float s_u[kSortChunk + 64];
  __shared__ float s_key[kSortChunk];
  __shared__ float s_red[32];
  const int unit = blockIdx.x, chunk = blockIdx.y;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  const int cu = p.cu_seqlens[b];
  const int t = p.cu_seqlens[b + 1] - cu;
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
    float v = s_red[tid];
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (tid == 0) p.part_sum[(size_t)unit * p.n_chunks + chunk] = v;
  }
  if (sort_out == nullptr) return;
  if (c0 >= P) return;

  // bitonic sort, descending; absent entries (-1) end up last
  for (int k = 2; k <= kSortChunk; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      __syncthreads();
      for (int x = tid; x < kSortChunk / 2; x += kSortThreads) {
        const int i = ((x & ~(j - 1)) << 1) | (x & (j - 1));   // index with bit j clear
        const int l = i | j;
        const float a = s_key[i], c = s_key[l];
        const bool desc = (i & k) == 0;
        if (desc ? (a < c) : (a > c)) {
          s_key[i] = c;
          s_key[l] = a;
        }
      }
    }
  }
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

__global__ void __launch_bounds__(kMergeThreads) merge_kernel(const ScoreParams p, const float* src, float* dst,
                                                             int run) {
  __shared__ float s_in[kMergeTile];
  __shared__ int s_split[2];
  const int unit = blockIdx.x;
  const int b = unit / p.n_kv_heads, g = unit % p.n_kv_heads;
  const int cu = p.cu_seqlens[b];
  const int t = p.cu_seqlens[b + 1] - cu;
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
  if (threadIdx.x < 2) s_split[threadIdx.x] = merge_path(A, la, B, lb, threadIdx.x == 0 ? d0 : d1);
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
  const int t = p.cu_seqlens[b + 1] - cu;
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

struct ScoreLayout {
  size_t u, tmp_sorted, stats_part, mrow, part_sum, total;
  int split_keys, n_splits, n_chunks;
};

void score_layout(const xkv_dims* d, int max_seqlen, int64_t T, ScoreLayout* L) {
  const int units = d->batch * d->n_kv_heads;
  const int M = (d->n_q_heads / d->n_kv_heads) * d->window;
  int split = 1024;
  while (split > kKeyTile && (int64_t)units * ((max_seqlen + split - 1) / split) < 2 * 148) split >>= 1;
  L->split_keys = split;
  L->n_splits = (max_seqlen + split - 1) / split;
  L->n_chunks = (max_seqlen + kSortChunk - 1) / kSortChunk;
  size_t off = kHeaderBytes;
  L->u = off;          off = align_up(off + (size_t)d->n_kv_heads * T * 4, 256);
  L->tmp_sorted = off; off = align_up(off + (size_t)d->n_kv_heads * T * 4, 256);
  L->stats_part = off; off = align_up(off + (size_t)units * L->n_splits * M * 8, 256);
  L->mrow = off;       off = align_up(off + (size_t)units * M * 4, 256);
  L->part_sum = off;   off = align_up(off + (size_t)units * L->n_chunks * 4, 256);
  L->total = off;
}

template <int D>
xkv_status launch_passes(const ScoreParams& p, int units, cudaStream_t st) {
  const size_t smem = PassCfg<D>::smem_bytes(p.M);
  static bool done[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  if (!done[dev]) {
    if (cudaFuncSetAttribute(score_pass_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)PassCfg<D>::smem_bytes(256)) != cudaSuccess ||
        cudaFuncSetAttribute(score_pass_kernel<D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)PassCfg<D>::smem_bytes(256)) != cudaSuccess)
      return XKV_ERR_CUDA;
    done[dev] = true;
  }
  dim3 grid(units, p.n_splits);
  score_pass_kernel<D, 1><<<grid, kPassThreads, smem, st>>>(p);
  count_launch();
  xkv_status s = check_launch();
  if (s != XKV_OK) return s;
  stats_merge_kernel<<<units, 256, 0, st>>>(p);
  count_launch();
  s = check_launch();
  if (s != XKV_OK) return s;
  score_pass_kernel<D, 2><<<grid, kPassThreads, smem, st>>>(p);
  count_launch();
  return check_launch();
}

}  // namespace

size_t score_workspace_bytes(const xkv_dims* d, int max_seqlen, int64_t total_tokens) {
  ScoreLayout L;
  score_layout(d, max_seqlen, total_tokens, &L);
  return L.total;
}

xkv_status score(const xkv_dims* d, const void* q_win, const void* k, const int32_t* cu_seqlens,
                 int64_t total_tokens, int max_seqlen, float* scores, float* sorted, float* gains, float* mass,
                 int curve_len, void* workspace, size_t workspace_bytes, cudaStream_t st) {
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
  p.M = p.group * d->window;
  p.pool_kernel = d->pool_kernel;
  p.pool_mode = d->pool_mode;
  p.split_keys = L.split_keys;
  p.n_splits = L.n_splits;
  p.n_chunks = L.n_chunks;
  p.curve_len = curve_len;
  const float scale = d->scale != 0.f ? d->scale : 1.0f / sqrtf((float)d->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;

  if (cudaMemsetAsync(ws, 0, kHeaderBytes, st) != cudaSuccess) return XKV_ERR_CUDA;
  xkv_status s = d->head_dim == 128 ? launch_passes<128>(p, units, st) : launch_passes<64>(p, units, st);
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
