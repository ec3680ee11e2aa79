// Both window-logit passes of xkv_score in one kernel that reads every key once, for G*W = 32 query rows
// and units of at most kClusterMax * 1024 keys.
//
// A thread-block cluster owns one unit = (sequence, KV head) at a time (units are dealt to the clusters
// round-robin) and every CTA of the cluster takes a contiguous share of at most eight 128-key tiles.  With
// the keys on the M axis of the tensor-core tile, S[128 keys x 32 query rows] of one tile is 32 columns of
// tensor memory, so a CTA keeps the logits of its whole share (8 x 32 columns) in TMEM, and those of the
// next unit in the other half of the 512 columns.  Per unit a CTA
//   A. streams its tiles by TMA, one tcgen05.mma chain per tile into the tile's TMEM slot; an epilogue
//      thread owns one key, so the softmax statistics of a query row run across the lanes of a warp: the
//      thread sums its key slot's exponentials per row over the warp's tiles, and once per unit the warp
//      exchanges the 32 x 32 block by a halving butterfly (31 shuffles) so that lane r holds the (reference,
//      sum of exponentials) of row r.  The reference is the row maximum at the warp's first
//      tile and is raised only when a logit exceeds it by 2^8; it reaches the other lanes through a
//      32-float strip of shared memory;
//   X. sends its per-warp statistics to every CTA of the cluster with st.async into their shared memory
//      (the stores complete a transaction count on the receiver's mbarrier), waits until the statistics of
//      the whole cluster have landed in its own, and merges them into the row normalisers m_r + log2(l_r);
//   B. reads the logits again, from TMEM, and sums exp2(s*c - normaliser[row]) over the query rows: the
//      column score u[key] (Eq. 2 summed over the window, before pooling).  The slot is then free for the
//      unit after next.
// The producer and the MMA issuer run up to a whole unit ahead of the epilogue, and the epilogue runs steps X
// (the wait) and B of a unit after step A of the next one, so neither the keys nor the epilogue wait for the
// exchange; the statistics of up to four units can sit in a CTA's shared memory.  The only waits on other
// CTAs are those of step X, within a cluster, whose CTAs the hardware schedules together; they are bounded
// like every other wait here, and a CTA leaves only after a cluster-wide barrier, so no store can reach the
// shared memory of a CTA that has gone.
#include <atomic>

#include "tc_common.cuh"

namespace xkv {
namespace {

using namespace tc;

constexpr int kRows = 32;                    // G*W this kernel covers
constexpr int kSlotsPerUnit = 8;             // 128-key tiles of one unit a CTA holds in TMEM
constexpr int kSlots = 2 * kSlotsPerUnit;    // x 32 columns = all 512 columns
constexpr int kEpiAll = 2 * kEpiThreads;     // epilogue threads of a CTA
constexpr int kClusterMax = 8;
constexpr int kStatSlots = 4;                // units whose exchanged statistics may be in a CTA's shared memory
constexpr float kLazyRaise = 8.f;

template <int D, int CS>
struct FusedCfg {
  static constexpr int kHalves = D / 64;
  static constexpr int kSteps = D / 16;
  static constexpr int kQHalfBytes = kRows * 128;
  static constexpr int kQBytes = kHalves * kQHalfBytes;
  static constexpr int kKHalfBytes = kTcKeyTile * 128;
  static constexpr int kKTileBytes = kHalves * kKHalfBytes;
  static constexpr int kStages = D == 128 ? (CS <= 4 ? 5 : 4) : 8;
  static constexpr size_t kStatsBytes = kStatSlots * (size_t)CS * kEpiAll * 8;   // [slot][source CTA][thread]
  static constexpr size_t kSmemBytes = 1024 + (size_t)2 * kQBytes + (size_t)kStages * kKTileBytes + kStatsBytes +
                                       2 * kRows * 4 /*row normalisers*/ + 16 * kRows * 4 /*reference and rescale strips*/ +
                                       512 /*barriers*/;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t n_clusters_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in the CTA with the given rank of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// Eight-byte store into a cluster CTA's shared memory that counts eight bytes on that CTA's mbarrier.
__device__ __forceinline__ void st_async_f2(uint32_t remote_addr, float a, float b, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(
                   remote_addr),
               "f"(a), "f"(b), "r"(remote_bar)
               : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// x[r] of every lane -> lane r holds op over the 32 lanes of x[r]; x is consumed.
template <class Op>
__device__ __forceinline__ float warp_transpose_reduce(float (&x)[32], int lane, Op op) {
#pragma unroll
  for (int step = 16; step >= 1; step >>= 1) {
    const bool up = (lane & step) != 0;
#pragma unroll
    for (int i = 0; i < step; ++i) {
      const float send = up ? x[i] : x[i + step];
      const float keep = up ? x[i + step] : x[i];
      x[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, step));
    }
  }
  return x[0];
}

struct UnitShape {
  int unit, b, g, cu, t, P, tile_begin, n1, n2;
};

// Unit n of this cluster and this CTA's share of its tiles: tiles [tile_begin, tile_begin + n1) cover the keys
// below t, the first n2 <= n1 of them hold keys below P = t - W (those get a score).
template <int CS>
__device__ __forceinline__ bool unit_shape(const ScoreParams& p, int n, uint32_t cluster, uint32_t n_clusters,
                                           uint32_t rank, UnitShape* u) {
  const int unit = (int)cluster + n * (int)n_clusters;
  if (unit >= p.batch * p.n_kv_heads) return false;
  u->unit = unit;
  u->b = unit / p.n_kv_heads;
  u->g = unit % p.n_kv_heads;
  u->cu = p.cu_seqlens[u->b];
  u->t = min(p.cu_seqlens[u->b + 1] - u->cu, p.max_seqlen);
  u->P = max(u->t - p.window, 0);
  const int nt1 = (u->t + kTcKeyTile - 1) / kTcKeyTile, nt2 = (u->P + kTcKeyTile - 1) / kTcKeyTile;
  const int per = (nt1 + CS - 1) / CS;              // <= kSlotsPerUnit: the host checks max_seqlen
  u->tile_begin = (int)rank * per;
  u->n1 = min(max(nt1 - u->tile_begin, 0), per);
  u->n2 = min(max(nt2 - u->tile_begin, 0), per);
  return true;
}

template <int D, int CS>
__global__ void __launch_bounds__(kWsThreads, 1) score_fused_kernel(const __grid_constant__ CUtensorMap tmap_q,
                                                                const __grid_constant__ CUtensorMap tmap_k,
                                                                const ScoreParams p) {
  using C = FusedCfg<D, CS>;
  extern __shared__ uint8_t smem_raw[];
  // the same offset in every CTA of the cluster (mapa maps equal offsets): align within the window itself
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* q_s = smem;
  uint8_t* k_s = q_s + (size_t)2 * C::kQBytes;
  float2* s_stats = reinterpret_cast<float2*>(k_s + (size_t)C::kStages * C::kKTileBytes);   // [4][CS][256]
  float* s_mrow = reinterpret_cast<float*>(s_stats + kStatSlots * CS * kEpiAll);            // [2][32]
  float* s_ref = s_mrow + 2 * kRows;                                                        // [8 warps][32]
  float* s_fac = s_ref + 8 * kRows;                                                         // [8 warps][32]
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(s_fac + 8 * kRows);
  uint64_t* empty_bar = full_bar + C::kStages;
  uint64_t* qfull_bar = empty_bar + C::kStages;
  uint64_t* qempty_bar = qfull_bar + 2;
  uint64_t* resfull_bar = qempty_bar + 2;            // [kSlots] the tile's logits are complete in TMEM
  uint64_t* resempty_bar = resfull_bar + kSlots;     // [kSlots] both readings of the slot are over
  uint64_t* stats_bar = resempty_bar + kSlots;       // [4] statistics of the whole cluster have landed here
  uint64_t* mrow_bar = stats_bar + kStatSlots;       // [2] this CTA's row normalisers are written
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(mrow_bar + 2);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank(), cluster = cluster_id_x(), n_clusters = n_clusters_x();
  if (tid == 0) {
    for (int i = 0; i < C::kStages; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&qfull_bar[i], 1);
      mbar_init(&qempty_bar[i], 1);
      mbar_init(&mrow_bar[i], 8);              // one arrival per epilogue warp
    }
    for (int i = 0; i < kStatSlots; ++i) mbar_init(&stats_bar[i], 1);   // one arrival (with the byte count) per unit
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(&resfull_bar[i], 1);
      mbar_init(&resempty_bar[i], 4);          // one arrival per warp of the group that reads the slot
    }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_k);
  }
  if (warp == 0) {
    tmem_alloc(s_tmem, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  cluster_sync_all();          // every CTA's barriers exist before any store from a neighbour can arrive
  const uint32_t tmem_base = *s_tmem;

  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t gt = 0, it = 0;
      UnitShape sh;
      bool ok = true;
      for (int n = 0; ok && unit_shape<CS>(p, n, cluster, n_clusters, rank, &sh); ++n) {
        if (sh.n1 == 0) continue;
        const uint32_t qb = it & 1u;
        ok = ws_wait(&qempty_bar[qb], ((it >> 1) & 1u) ^ 1u, s_abort, p.wait_ns);
        if (!ok) break;
        mbar_arrive_expect_tx(&qfull_bar[qb], (uint32_t)C::kQBytes);
        const int qrow0 = (sh.b * p.n_q_heads + sh.g * p.group) * p.window;
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf)
          tma_load_2d(q_s + (size_t)qb * C::kQBytes + hf * C::kQHalfBytes, &tmap_q, hf * 64, qrow0, &qfull_bar[qb]);
        for (int ti = 0; ti < sh.n1; ++ti, ++gt) {
          const uint32_t s = gt % C::kStages;
          ok = ws_wait(&empty_bar[s], ((gt / C::kStages) & 1u) ^ 1u, s_abort, p.wait_ns);
          if (!ok) break;
          mbar_arrive_expect_tx(&full_bar[s], (uint32_t)C::kKTileBytes);
#pragma unroll
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_3d(k_s + (size_t)s * C::kKTileBytes + hf * C::kKHalfBytes, &tmap_k, hf * 64, sh.g,
                        sh.cu + (sh.tile_begin + ti) * kTcKeyTile, &full_bar[s]);
        }
        ++it;
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t gt = 0, it = 0, slot_uses = 0;       // slot_uses: bit s = parity of the uses of TMEM slot s so far
      UnitShape sh;
      bool ok = true;
      const uint32_t q_base = smem_u32(q_s), k_base = smem_u32(k_s);
      for (int n = 0; ok && unit_shape<CS>(p, n, cluster, n_clusters, rank, &sh); ++n) {
        if (sh.n1 == 0) continue;
        const uint32_t qb = it & 1u;
        ok = ws_wait(&qfull_bar[qb], (it >> 1) & 1u, s_abort, p.wait_ns);
        if (!ok) break;
        const uint64_t q_desc = umma_desc_k128(q_base + qb * C::kQBytes);   // k-steps only move the start-address field
        for (int ti = 0; ti < sh.n1; ++ti, ++gt) {
          const uint32_t s = gt % C::kStages;
          const uint32_t slot = (it & 1u) * kSlotsPerUnit + (uint32_t)ti;
          ok = ws_wait(&full_bar[s], (gt / C::kStages) & 1u, s_abort, p.wait_ns) &&
               ws_wait(&resempty_bar[slot], ((slot_uses >> slot) & 1u) ^ 1u, s_abort, p.wait_ns);
          if (!ok) break;
          slot_uses ^= 1u << slot;
          tc_fence_after_sync();
          const uint64_t k_desc = umma_desc_k128(k_base + s * C::kKTileBytes);
#pragma unroll
          for (int k = 0; k < C::kSteps; ++k) {
            const uint64_t kd = k_desc + (uint64_t)(((k / 4) * C::kKHalfBytes + (k % 4) * 32) >> 4);
            const uint64_t qd = q_desc + (uint64_t)(((k / 4) * C::kQHalfBytes + (k % 4) * 32) >> 4);
            umma_bf16(tmem_base + slot * kRows, kd, qd, umma_idesc(kTcKeyTile, kRows), k > 0 ? 1u : 0u);
          }
          umma_commit(&empty_bar[s]);           // the ring stage is free once these MMAs have read it
          umma_commit(&resfull_bar[slot]);      // and the tile's logits are complete
        }
        if (!ok) break;
        umma_commit(&qempty_bar[qb]);
        ++it;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 0..7
    const uint32_t group = warp >> 2;                                       // takes the tiles with ti % 2 == group
    const int etid = tid & (kEpiThreads - 1);                               // TMEM lane = key within the tile
    const int eall = (int)group * kEpiThreads + etid;                       // 0..255; its query row is lane = eall % 32
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
    const uint32_t stats_base = smem_u32(s_stats), stats_bar_base = smem_u32(stats_bar);
    float* ref = s_ref + warp * kRows;
    const float4* ref4 = reinterpret_cast<const float4*>(ref);
    float* fac = s_fac + warp * kRows;
    const float4* fac4 = reinterpret_cast<const float4*>(fac);
    uint32_t it = 0, useq = 0, slot_uses = 0;
    UnitShape sh;
    bool ok = true;
    // The unit whose statistics have been sent but whose column sums are still to be formed: its steps X (wait)
    // and B run after step A of the next unit, so the exchange has a whole unit's worth of work to land behind.
    bool have_pend = false;
    UnitShape pend;
    uint32_t pend_useq = 0, pend_slot0 = 0;
    auto finish = [&](const UnitShape& u, uint32_t q, uint32_t slot0) {
      const uint32_t st = q % kStatSlots, st_phase = (q / kStatSlots) & 1u;
      const uint32_t par = q & 1u, phase = (q >> 1) & 1u;
      ok = __all_sync(0xffffffffu, ws_wait(&stats_bar[st], st_phase, s_abort, p.wait_ns));
      if (!ok) return;
      // row normalisers: thread r < 32 merges every entry of query row r (entries r, r + 32, ... of each CTA)
      if (eall < kRows) {
        float m = -INFINITY, l = 0.f;
        for (int src = 0; src < CS; ++src)
          for (int k = eall; k < kEpiAll; k += kRows) {
            const float2 v = s_stats[(st * CS + src) * kEpiAll + k];
            const float m_new = fmaxf(m, v.x);
            const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
            l = l * exp2f(m - m_ref) + v.y * exp2f(v.x - m_ref);
            m = m_new;
          }
        s_mrow[par * kRows + eall] = (l > 0.f) ? m + log2f(l) : INFINITY;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&mrow_bar[par]);
      if (u.n1 == 0) return;
      ok = __all_sync(0xffffffffu, ws_wait(&mrow_bar[par], phase, s_abort, p.wait_ns));
      if (!ok) return;
      // ---- B: column sums out of TMEM; a thread owns one key
      float* uo = p.u + (size_t)u.g * p.total_tokens + u.cu;
      const float4* mrow4 = reinterpret_cast<const float4*>(s_mrow + par * kRows);
      for (int ti = (int)group; ti < u.n1; ti += 2) {
        const uint32_t slot = slot0 + (uint32_t)ti;
        slot_uses ^= 1u << slot;
        if (ti < u.n2) {
          float v[32];
          tmem_ld32(tmem_lane + slot * kRows, v);
          tmem_wait_ld();
          float sum = 0.f;
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 mr = mrow4[i >> 2];
            sum += fast_exp2(fmaf(v[i + 0], p.scale_log2, -mr.x)) + fast_exp2(fmaf(v[i + 1], p.scale_log2, -mr.y)) +
                   fast_exp2(fmaf(v[i + 2], p.scale_log2, -mr.z)) + fast_exp2(fmaf(v[i + 3], p.scale_log2, -mr.w));
          }
          const int key = (u.tile_begin + ti) * kTcKeyTile + etid;
          if (key < u.P) uo[key] = sum;
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&resempty_bar[slot]);
      }
    };
    for (int n = 0; ok && unit_shape<CS>(p, n, cluster, n_clusters, rank, &sh); ++n) {
      if (sh.t == 0) continue;                       // nothing to exchange: every CTA of the cluster skips it
      const uint32_t my_useq = useq++;
      const uint32_t st = my_useq % kStatSlots;
      const uint32_t slot0 = (it & 1u) * kSlotsPerUnit;
      if (sh.n1 > 0) ++it;
      // ---- A: statistics of row `lane` over the keys of this warp.  The exponentials are summed per thread
      // (one key slot, 32 rows) over the warp's tiles of the unit and exchanged across the lanes once at the end.
      float r_run = -INFINITY;                       // reference (log2 domain) of row `lane`
      float acc[32];                                 // this key slot's sum of exp2(x - reference[row]) per row
#pragma unroll
      for (int i = 0; i < 32; ++i) acc[i] = 0.f;
      bool first = true;
      for (int ti = (int)group; ti < sh.n1; ti += 2) {
        const uint32_t slot = slot0 + (uint32_t)ti;
        ok = __all_sync(0xffffffffu, ws_wait(&resfull_bar[slot], (slot_uses >> slot) & 1u, s_abort, p.wait_ns));
        if (!ok) break;
        tc_fence_after_sync();
        float x[32];
        tmem_ld32(tmem_lane + slot * kRows, x);
        tmem_wait_ld();
        const int key = (sh.tile_begin + ti) * kTcKeyTile + etid;
        const bool masked = key + p.window >= sh.t;          // a window key (causal inside the window) or past the end
        if (masked) {
          const int lim0 = sh.t - p.window;                  // row i sees the keys up to lim0 + i % W
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (key > lim0 + (i % p.window)) x[i] = -INFINITY;
        }
        float y[32], dmax = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 r4 = ref4[i >> 2];
          y[i] = fmaf(x[i], p.scale_log2, -r4.x);            // raw logit * (log2 e / sqrt(d)) - reference
          y[i + 1] = fmaf(x[i + 1], p.scale_log2, -r4.y);
          y[i + 2] = fmaf(x[i + 2], p.scale_log2, -r4.z);
          y[i + 3] = fmaf(x[i + 3], p.scale_log2, -r4.w);
          dmax = fmaxf(fmaxf(dmax, fmaxf(y[i], y[i + 1])), fmaxf(y[i + 2], y[i + 3]));
        }
        if (__any_sync(0xffffffffu, first || dmax > kLazyRaise || r_run == -INFINITY)) {
          // exact maximum of every row over this warp's 32 keys; lane r raises (or first sets) its reference and
          // tells the other lanes by how much the sums gathered so far shrink
          float tcopy[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) tcopy[i] = x[i] * p.scale_log2;
          const float tmax = warp_transpose_reduce(tcopy, lane, [](float a, float b) { return fmaxf(a, b); });
          float shrink = 1.f;
          if (tmax > r_run) {
            shrink = (r_run == -INFINITY) ? 1.f : fast_exp2(r_run - tmax);   // nothing was gathered under -inf
            r_run = tmax;
          }
          __syncwarp();
          ref[lane] = (r_run == -INFINITY) ? 0.f : r_run;
          fac[lane] = shrink;
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 r4 = ref4[i >> 2];
            y[i] = fmaf(x[i], p.scale_log2, -r4.x);
            y[i + 1] = fmaf(x[i + 1], p.scale_log2, -r4.y);
            y[i + 2] = fmaf(x[i + 2], p.scale_log2, -r4.z);
            y[i + 3] = fmaf(x[i + 3], p.scale_log2, -r4.w);
          }
          if (!first) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float4 f4 = fac4[i >> 2];
              acc[i] *= f4.x;
              acc[i + 1] *= f4.y;
              acc[i + 2] *= f4.z;
              acc[i + 3] *= f4.w;
            }
          }
          first = false;
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[i] += fast_exp2(y[i]);
      }
      const float l_run = warp_transpose_reduce(acc, lane, [](float a, float b) { return a + b; });
      if (!ok) break;
      // ---- X: the statistics of row `lane` from this warp go to slot [st][rank][eall] of every CTA of the cluster
      if (eall == 0) mbar_arrive_expect_tx(&stats_bar[st], (uint32_t)(CS * kEpiAll * 8));
      {
        const uint32_t slot = stats_base + (uint32_t)(((st * CS + rank) * kEpiAll + eall) * 8);
        const uint32_t bar = stats_bar_base + st * 8u;
#pragma unroll
        for (uint32_t dst = 0; dst < (uint32_t)CS; ++dst)
          st_async_f2(map_to_rank(slot, dst), r_run, l_run, map_to_rank(bar, dst));
      }
      if (have_pend) {
        finish(pend, pend_useq, pend_slot0);
        if (!ok) break;
      }
      pend = sh;
      pend_useq = my_useq;
      pend_slot0 = slot0;
      have_pend = true;
    }
    if (ok && have_pend) finish(pend, pend_useq, pend_slot0);
  }

  // ---- teardown
  __syncthreads();
  if (*s_abort) {
    if (tid == 0) record_status(p.hdr, XKV_ERR_TIMEOUT);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies and MMAs already issued finish
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, 512);
  cluster_sync_all();          // no CTA leaves while a neighbour may still store into its shared memory
}

template <int D, int CS>
xkv_status fused_launch(const CUtensorMap& tq, const CUtensorMap& tk, const ScoreParams& p, cudaStream_t st) {
  using F = FusedCfg<D, CS>;
  const size_t smem = F::kSmemBytes;             // > 113 KB: one CTA per SM, which owns all 512 TMEM columns
  static std::atomic<int> max_clusters[64];   // the occupancy query gives the same answer from any thread
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return XKV_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kWsThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_clusters[dev].load(std::memory_order_acquire) == 0) {
    if (cudaFuncSetAttribute(score_fused_kernel<D, CS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return XKV_ERR_CUDA;
    // clusters that can be resident together: units are dealt to exactly that many, so none waits for an SM
    cfg.gridDim = dim3((unsigned)(sm_count() / CS * CS));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, score_fused_kernel<D, CS>, &cfg) != cudaSuccess || n < 1) {
      cudaGetLastError();
      return XKV_ERR_CUDA;
    }
    max_clusters[dev].store(n, std::memory_order_release);
  }
  int n_clusters = max_clusters[dev].load(std::memory_order_acquire);
  const int units = p.batch * p.n_kv_heads;
  if (n_clusters > units) n_clusters = units;
  cfg.gridDim = dim3((unsigned)(n_clusters * CS));
  if (cudaLaunchKernelEx(&cfg, score_fused_kernel<D, CS>, tq, tk, p) != cudaSuccess) {
    cudaGetLastError();
    return XKV_ERR_CUDA;
  }
  count_launch();
  return check_launch();
}

}  // namespace

bool score_fused_covers(int M, int head_dim, int units, int max_seqlen) {
#ifdef XKV_NO_TC
  return false;
#else
  (void)units;
  if (M != kRows) return false;
  if (head_dim != 64 && head_dim != 128) return false;
  return max_seqlen <= kClusterMax * kSlotsPerUnit * kTcKeyTile;
#endif
}

xkv_status score_fused_pass(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st) {
  const int units = p.batch * p.n_kv_heads;
  if (!score_fused_covers(p.M, head_dim, units, max_seqlen)) return XKV_ERR_UNSUPPORTED;
  CUtensorMap tq, tk;
  if (!tc_make_score_tmaps(p, head_dim, &tq, &tk)) return XKV_ERR_CUDA;
  const bool small = max_seqlen <= 4 * kSlotsPerUnit * kTcKeyTile;       // clusters of four cover 4096 keys
  if (head_dim == 128) return small ? fused_launch<128, 4>(tq, tk, p, st) : fused_launch<128, 8>(tq, tk, p, st);
  return small ? fused_launch<64, 4>(tq, tk, p, st) : fused_launch<64, 8>(tq, tk, p, st);
}

}  // namespace xkv
