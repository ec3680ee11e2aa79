/*
 * xkv.h -- C ABI of libxkv: the data-parallel hot path of XKV (personalised per-layer
 * KV-cache budgets) on one NVIDIA B200 (sm_100a).
 *
 * The path, in call order:
 *   0. xkv_prefill_attn   optional, the step before the path: causal attention of the whole prompt, which also
 *                         yields the softmax normalisers of the window rows   (Eq. 1, Eq. 2; Alg. 2 step 1)
 *   1. xkv_score          per layer: observation-window attention weights -> pooled importance
 *                         scores per KV head, their descending sort, and the layer's
 *                         retained-importance curve               (Eq. 2, Eq. 3, Eq. 4; Alg. 2 steps 1-4)
 *      xkv_score_lse      the same from normalisers that xkv_prefill_attn (or the model's own attention)
 *                         already produced: one pass over the keys instead of two      (Alg. 2 steps 1-4)
 *      xkv_batch_curves   device: one curve per layer from the batch's curves         (Alg. 1, input W)
 *      xkv_head_curves    device: one curve per (layer, KV head) for head-level budgets      (Sec. II-C)
 *   2. xkv_alloc_budgets  host: greedy split of a global budget across layers        (Alg. 1; Eq. 17, Eq. 18)
 *      xkv_average_budgets  host: the averaged list of the online scenario           (Sec. IV-C)
 *   3. xkv_select_compact per layer: top-k per (sequence, KV head) and gather of the kept K/V
 *                         rows into a ragged paged cache                             (Alg. 2 steps 5-7)
 *   4. xkv_decode_attn    per generation step: attention over the ragged compacted caches,
 *                         new K/V appended first                                     (Eq. 1; Sec. IV-A, generation phase)
 *
 * Conventions that hold for every entry point
 *   - Plain C types only. "dev" = pointer to device memory of the current CUDA device,
 *     "host" = pointer to host memory. bf16 = IEEE bfloat16 stored as uint16_t bit patterns.
 *   - The caller owns every buffer (inputs, outputs, cache pages, workspace). The library
 *     allocates nothing, frees nothing and never synchronises the stream; work is enqueued on
 *     `stream` (a cudaStream_t passed as void*, NULL = default stream).
 *   - Device pointers must be 16-byte aligned; violations are rejected with XKV_ERR_INVALID_ARG.
 *   - Arguments are validated on the host and rejected before anything is enqueued. A negative
 *     return value means nothing was launched. Conditions only the device can see (a cache slot
 *     beyond its page table, a bounded wait that expired, a prompt longer than max_seqlen) are
 *     recorded in a status word, the first four bytes of the workspace. The word is sticky: a call
 *     never clears it, it keeps the first error recorded since it was last read, so one workspace
 *     can serve many calls (the layers of a phase) and be checked once. xkv_read_device_status
 *     returns the word and resets it. A workspace must be zero-filled before its first use.
 *   - The first call of an entry point on a device does one-time set-up (kernel attributes, symbol
 *     addresses); these steps are idempotent and safe from several host threads.
 *   - Sequences are packed: token c of sequence b is row cu_seqlens[b] + c. t_b = cu_seqlens[b+1]
 *     - cu_seqlens[b] is the prompt length, W = dims.window, P_b = max(t_b - W, 0) the prefix
 *     length (the tokens that can be evicted); the last min(W, t_b) tokens are always kept.
 *   - G = n_q_heads / n_kv_heads query heads share KV head g = h / G.
 */
#ifndef XKV_H_
#define XKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t xkv_status;
#define XKV_OK               0
#define XKV_ERR_INVALID_ARG (-1) /* null/misaligned pointer, non-positive size, inconsistent dims    */
#define XKV_ERR_UNSUPPORTED (-2) /* head_dim not in {64,128}, G*W > 256, ... */
#define XKV_ERR_WORKSPACE   (-3) /* workspace_bytes smaller than xkv_workspace_bytes() reports        */
#define XKV_ERR_BUDGET      (-4) /* negative budget, total beyond capacity, unreachable R target      */
#define XKV_ERR_CUDA        (-5) /* a CUDA runtime/driver call or a launch failed                     */
#define XKV_ERR_TIMEOUT     (-6) /* device status: a bounded wait inside a kernel expired             */
#define XKV_ERR_CAPACITY    (-7) /* device status: a sequence outgrew its page table                  */

#define XKV_POOL_MAX 0
#define XKV_POOL_AVG 1

/* What the `budget` argument of xkv_select_compact holds. */
#define XKV_BUDGET_PER_LAYER    0 /* [1]: one count for every sequence and KV head of the layer (Alg. 1's n_i) */
#define XKV_BUDGET_PER_SEQUENCE 1 /* [B]: one count per sequence (the paper's offline mode, one list per task) */
#define XKV_BUDGET_PER_HEAD     2 /* [B][Hkv]: head-level budgets inside the layer (Sec. II-C)                 */

#define XKV_KV_BF16 0
#define XKV_KV_INT8 1

#define XKV_OP_SCORE          0
#define XKV_OP_SELECT_COMPACT 1
#define XKV_OP_DECODE_ATTN    2
#define XKV_OP_PREFILL_ATTN   3

/* Problem shape shared by the device entry points. */
typedef struct xkv_dims {
  int32_t batch;         /* B, number of sequences                                            */
  int32_t n_q_heads;     /* Hq                                                                 */
  int32_t n_kv_heads;    /* Hkv, divides Hq                                                    */
  int32_t head_dim;      /* d, 64 or 128                                                       */
  int32_t window;        /* W = ows, observation-window size (Eq. 3); G*W <= 256 */
  int32_t pool_kernel;   /* ps, odd, 1..63 (Alg. 2 step 4); 1 = no pooling                     */
  int32_t pool_mode;     /* XKV_POOL_MAX or XKV_POOL_AVG                                       */
  float   scale;         /* logit scale; 0 selects 1/sqrt(d) (Eq. 2)                           */
  int64_t kv_stride_token; /* elements between consecutive tokens of k and v (>= Hkv*d, mult. of 8) */
  int64_t kv_stride_head;  /* elements between KV heads of one token (>= d, mult. of 8)        */
} xkv_dims;

/*
 * The ragged paged cache of all layers (the reduced caches of Sec. IV-A whose sizes differ per layer).
 * A page holds page_size consecutive cache slots of every KV head:
 *   k_pages / v_pages : dev bf16 [n_pages][Hkv][page_size][d]
 *   block_table       : dev int32 [n_layers][B][max_pages_per_seq], page ids, filled by the caller;
 *                       slot s of (layer, b) lives in page block_table[layer][b][s / page_size]
 *   seq_lens          : dev int32 [n_layers][B], number of filled slots; written by
 *                       xkv_select_compact, advanced by xkv_decode_attn when it appends
 * page_size is a multiple of 16 (at most 256).
 *
 * A cache stored with few bits (Sec. II-B: quantisation is compatible with eviction; the paper names no format, this
 * one is the library's): with kv_format = XKV_KV_INT8 the pages hold one byte per element,
 *   k_pages / v_pages : dev uint8 [n_pages][Hkv][page_size][d], the byte is q + 128 with q an integer in [-127, 127]
 *   k_scales / v_scales : dev fp32 [n_pages][Hkv][page_size]
 * and a cached row stands for q * scale with scale = max|x| / 127 over the row (1 for an all-zero row) and
 * q = x / scale rounded to the nearest integer (ties to even), both divisions in fp32.
 * xkv_select_compact and the append of xkv_decode_attn store rows that way; xkv_decode_attn multiplies the scales back
 * in (K: on the logits, V: on the weights) and computes in fp16 x fp16 -> fp32: query magnitudes must stay below
 * 65504, and so must 256 * max|v| / 127 of a row. head_dim 64 and 128.
 *
 * Head-level budgets (XKV_BUDGET_PER_HEAD) give every KV head of a sequence a cache of its own length. The same
 * structure then describes B*Hkv caches of one KV head each per layer:
 *   k_pages / v_pages : dev bf16 [n_pages][1][page_size][d]
 *   block_table       : dev int32 [n_layers][B*Hkv][max_pages_per_seq], cache index b*Hkv + g
 *   seq_lens          : dev int32 [n_layers][B*Hkv]
 * xkv_select_compact fills it when called with XKV_BUDGET_PER_HEAD, and xkv_decode_attn reads it when called
 * with dims {batch = B*Hkv, n_q_heads = G, n_kv_heads = 1}: q, k_new, v_new, out and lse keep their memory
 * layout ([Lr][B][Hq][d] is [Lr][B*Hkv][G][d]).
 */
typedef struct xkv_cache {
  void*    k_pages;
  void*    v_pages;
  int32_t* block_table;
  int32_t* seq_lens;
  int32_t  n_layers;
  int32_t  page_size;
  int32_t  max_pages_per_seq;
  int32_t  n_pages;
  float*   k_scales;   /* XKV_KV_INT8 only: dev fp32 [n_pages][Hkv][page_size], one scale per cached row */
  float*   v_scales;
  int32_t  kv_format;  /* XKV_KV_BF16 (0) or XKV_KV_INT8 */
  int32_t  reserved;   /* 0 */
} xkv_cache;

/*
 * xkv_score -- importance scoring of one layer (Eq. 2, Eq. 3; Alg. 2 steps 1-4; Eq. 4).
 *
 * For every sequence b and KV head g:
 *   a[h,r,c] = softmax over the visible keys c <= P_b + r of scale * q_win[b,h,r,:] . k[c,g,:]
 *              (the model's causal attention weights of the last W tokens, Eq. 2)
 *   u[c]     = sum over the G query heads h of group g and the W window rows r of a[h,r,c], c < P_b
 *              (the ows x (t-ows) block, reduced along its first dimension)
 *   w[c]     = 1-D pooling of u, stride 1, same length, centred kernel ps:
 *              max over the part of the kernel inside [0, P_b)   (XKV_POOL_MAX), or
 *              sum over that part divided by ps                   (XKV_POOL_AVG, zero padding)
 *   sorted   = w in descending order
 *   gains[b][j] = mean over g of sorted[g][j] / sum_c w[c]   (0 for j >= P_b): the increase of the
 *              layer's retained-importance ratio R (Eq. 4) when every head keeps one more token;
 *   mass[b][n]  = sum_{j<=n} gains[b][j] = R at n+1 kept tokens.
 *
 * q_win      dev bf16 [B][Hq][W][d]; row r is the query of position t_b - W + r. Sequences shorter
 *            than W use rows W - t_b .. W-1 only.
 * k          dev bf16, token row cu_seqlens[b]+c, head g at element offset
 *            (cu_seqlens[b]+c)*kv_stride_token + g*kv_stride_head
 * cu_seqlens dev int32 [B+1], non-decreasing, cu_seqlens[0] = 0, cu_seqlens[B] = total_tokens
 * total_tokens, max_seqlen  host values: T and an upper bound of every t_b. The launch grids and buffers are
 *            sized from max_seqlen: a prompt found longer on the device is processed as if cut to
 *            max_seqlen tokens and the device status becomes XKV_ERR_INVALID_ARG.
 * scores     dev out fp32 [Hkv][T]: w at column cu_seqlens[b]+c for c < P_b; window columns are 0
 * sorted     dev out fp32 [Hkv][T]: per (g, b) the P_b values of w in descending order at columns
 *            cu_seqlens[b] .. cu_seqlens[b]+P_b-1; window columns are 0. NULL skips the sort and
 *            the curves (gains and mass are then not written).
 * gains      dev out fp32 [B][curve_len]
 * mass       dev out fp32 [B][curve_len], may be NULL
 * curve_len  number of ranks reported, >= 1
 * workspace  dev, at least xkv_workspace_bytes(XKV_OP_SCORE, ...) bytes, 256-byte aligned
 */
xkv_status xkv_score(const xkv_dims* dims, const void* q_win, const void* k,
                     const int32_t* cu_seqlens, int64_t total_tokens, int32_t max_seqlen,
                     float* scores, float* sorted, float* gains, float* mass, int32_t curve_len,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * xkv_prefill_attn -- causal attention of the prompt (Eq. 1 with the weights of Eq. 2), the layer's own attention
 * in which the paper computes W_attn (Alg. 2 step 1; Sec. IV-A, prefill phase).
 *
 * For every sequence b, query head h and position i < t_b:
 *   out[i,h,:] = softmax over the keys c <= i of scale * q[i,h,:] . k[c,g,:]  times  v[c,g,:]     (g = h / G)
 *   lse[h][i]  = natural log of the sum over c <= i of exp(scale * q[i,h,:] . k[c,g,:])
 * bf16 inputs, fp32 accumulation, the weights rounded to bf16 before they multiply v, bf16 output.
 * The lse entries of the last W positions of a sequence are the normalisers of the observation-window rows
 * of W_attn; xkv_score_lse takes them instead of recomputing them with a pass over the keys.
 *
 * q          dev bf16 [T][Hq][d], packed like k (row cu_seqlens[b] + i)
 * k, v       dev bf16, layout and strides of xkv_score (dims.kv_stride_*)
 * out        dev out bf16 [T][Hq][d]
 * lse        dev out fp32 [Hq][T], may be NULL
 * workspace  dev, at least xkv_workspace_bytes(XKV_OP_PREFILL_ATTN, ...) bytes (the status word), 256-byte aligned
 * dims.window, pool_kernel and pool_mode are not used. Device status XKV_ERR_TIMEOUT if a bounded wait expired.
 */
xkv_status xkv_prefill_attn(const xkv_dims* dims, const void* q, const void* k, const void* v,
                            const int32_t* cu_seqlens, int64_t total_tokens, int32_t max_seqlen, void* out,
                            float* lse, void* workspace, size_t workspace_bytes, void* stream);

/*
 * xkv_score_lse -- xkv_score when the normalisers of the window rows are already known (Alg. 2 step 1 takes
 * W_attn from the layer's attention; only Select, Merge, Pooling and the curves remain: Alg. 2 steps 2-4, Eq. 4).
 *
 *   a[h,r,c] = exp(scale * q_win[b,h,r,:] . k[c,g,:] - lse[h][cu_seqlens[b] + t_b - W + r])
 * and everything after it as in xkv_score; the keys are read once. With the "nothing cached" mini-prefill of
 * Sec. IV-A the caller has no normalisers and uses xkv_score, which forms them from the window queries alone.
 *
 * lse        dev fp32 [Hq][T] as xkv_prefill_attn writes it (only the last min(W, t_b) positions of every
 *            sequence are read)
 * other arguments, outputs and workspace: those of xkv_score.
 * Returns XKV_ERR_UNSUPPORTED unless G*W is 32, 64, 128 or 256.
 */
xkv_status xkv_score_lse(const xkv_dims* dims, const void* q_win, const void* k, const int32_t* cu_seqlens,
                         int64_t total_tokens, int32_t max_seqlen, const float* lse, float* scores, float* sorted,
                         float* gains, float* mass, int32_t curve_len, void* workspace, size_t workspace_bytes,
                         void* stream);

/*
 * xkv_alloc_budgets -- Algorithm 1 (adaptive allocation), host only, no CUDA call.
 *
 * gains      host fp32 [n_layers][batch][curve_len] as written by xkv_score, layer by layer
 * prefix_len host int32 [batch], P_b; a layer can hold at most max_b P_b (or n_max) tokens per head
 * per_sequence 0: one list for the batch from the mean over b of the gains (budgets [n_layers]);
 *              1: one list per sequence (budgets [batch][n_layers]), sequence b capped at P_b
 * total      N = sum of the per-layer budgets to hand out (Eq. 17). If total < 0 the R_avg mode
 *            of Eq. 18 runs instead: hand out slots until mean-over-layers retained ratio
 *            reaches r_target (in (0,1]).
 * n_min,n_max box per layer: every layer starts at n_min and stops at n_max
 *            (n_max <= 0 means no upper bound other than the capacity, n_min 0 = the paper's form)
 * budgets    host out int32
 * r_avg      host out double [1] or [batch]: the mean over layers of the retained ratio reached
 *
 * Each iteration grants one slot to the layer whose next-largest normalised score is largest;
 * ties go to the lowest layer index. Errors: XKV_ERR_BUDGET if total exceeds the summed
 * capacities (or is below n_layers*n_min), or r_target is not reachable.
 */
xkv_status xkv_alloc_budgets(const float* gains, int32_t n_layers, int32_t batch,
                             int32_t curve_len, const int32_t* prefix_len, int32_t per_sequence,
                             int64_t total, double r_target, int32_t n_min, int32_t n_max,
                             int32_t* budgets, double* r_avg);

/*
 * xkv_batch_curves -- the batch's curve of every layer, formed on the device (Alg. 1 takes one w per
 * layer: for a batch that is the mean over its sequences of the per-sequence curves xkv_score wrote).
 *
 *   out[l][j] = (sum over b of gains[l][b][j]) / divisor      summed in the order of b, in double precision
 *
 * gains      dev fp32 [n_layers][batch][curve_len]
 * divisor    batch for the mean of one GPU's batch; the total number of sequences of all ranks when the
 *            per-rank results are afterwards summed across ranks
 * out        dev out fp32 [n_layers][curve_len]; copied to the host it is the `gains` argument of
 *            xkv_alloc_budgets with batch = 1 and prefix_len = max_b P_b, which gives the list that
 *            per_sequence = 0 gives on the full array (up to the rounding of the mean to fp32), while only
 *            n_layers * curve_len numbers cross to the host.
 */
xkv_status xkv_batch_curves(const float* gains, int32_t n_layers, int32_t batch, int32_t curve_len, int32_t divisor,
                            float* out, void* stream);

/*
 * xkv_head_curves -- the curve of every KV head of one layer on its own: what Algorithm 1 consumes when the
 * unit that waits for slots is a (layer, KV head) pair instead of a layer (head-level cache sizes working
 * together with the layer-level allocation, Sec. II-C; per head the curve is Sort(w)/Sum(w) of Eq. 21).
 *
 *   head_gains[g][b][j] = sorted[g][cu_seqlens[b] + j] / sum over c < P_b of scores[g][cu_seqlens[b] + c]
 *                         for j < min(P_b, curve_len), 0 for the other j < curve_len
 *
 * scores, sorted  dev fp32 [Hkv][T] as xkv_score wrote them for this layer
 * head_gains      dev out fp32 [Hkv][B][curve_len]. The arrays of all layers, stacked, are [L*Hkv][B][curve_len]:
 *                 the `gains` argument of xkv_batch_curves / xkv_alloc_budgets with n_layers = L*Hkv, whose
 *                 budgets [L*Hkv] are then one count per (layer, KV head) and whose total is the number of
 *                 cached prefix tokens summed over all heads of all layers.
 */
xkv_status xkv_head_curves(const xkv_dims* dims, const float* scores, const float* sorted,
                           const int32_t* cu_seqlens, int64_t total_tokens, int32_t max_seqlen,
                           float* head_gains, int32_t curve_len, void* stream);

/*
 * xkv_average_budgets -- the averaged allocation list of the online scenario (Sec. IV-C), host only.
 *
 * The lists that xkv_alloc_budgets produced for a sample of tasks of one type are averaged layer by
 * layer; later tasks of that type skip the allocation and are evicted under the averaged list.
 *
 * lists      host int32 [n_tasks][n_layers], every entry >= 0
 * out        host out int32 [n_layers]
 *
 * The paper leaves the rounding open. Here every layer gets the floor of its mean, and the slots that
 * leaves over -- up to the mean of the recorded totals rounded half up -- go one each to the layers with
 * the largest fractional parts, the lower layer first among equals; lists that all add up to N therefore
 * give a list that adds up to N. Errors: XKV_ERR_INVALID_ARG for null pointers, non-positive counts or a
 * negative entry.
 */
xkv_status xkv_average_budgets(const int32_t* lists, int32_t n_tasks, int32_t n_layers, int32_t* out);

/*
 * xkv_select_compact -- top-k and eviction of one layer (Alg. 2 steps 5-7).
 *
 * For every (b, g): keep the kb = min(budget, P_b) prefix positions with the largest w, ordered by
 * (score descending, position ascending) so that among equal scores the lower position is kept,
 * plus all window positions P_b .. t_b-1. The kept positions, in ascending order, are copied
 * bit-exactly from k and v into cache slots 0 .. kb + (t_b - P_b) - 1 of (layer, b) and
 * seq_lens[layer][b] is set to that count.
 *
 * per_sequence  XKV_BUDGET_PER_LAYER (0), XKV_BUDGET_PER_SEQUENCE (1) or XKV_BUDGET_PER_HEAD (2)
 * budget     host int32 [1], [B] or [B][Hkv] accordingly, each >= 0. Arrays of more than one entry are
 *            copied to the device on `stream`: from pageable memory that copy waits
 *            for the stream's earlier work; from pinned memory it is asynchronous, and the array
 *            must then stay alive and unchanged until the stream has passed this call.
 *            With XKV_BUDGET_PER_HEAD, `cache` is the per-head form described at xkv_cache, kb and the
 *            slot count are those of (b, g), and seq_lens[layer][b*Hkv + g] is set.
 * scores     dev fp32 [Hkv][T] (w of xkv_score, or any non-negative finite scores)
 * sorted     dev fp32 [Hkv][T] (descending per (g,b), as xkv_score writes it)
 * k, v       dev bf16, same layout and strides (dims.kv_stride_*)
 * sel        dev out int32 [B][Hkv][sel_stride], may be NULL: the kept positions in cache order;
 *            sel_stride >= min(budget, max_seqlen) + W
 * workspace  dev, at least xkv_workspace_bytes(XKV_OP_SELECT_COMPACT, ...) bytes
 * Device status XKV_ERR_CAPACITY if a sequence needs more than max_pages_per_seq pages
 * (nothing is copied for that sequence and its seq_lens entry is set to 0).
 */
xkv_status xkv_select_compact(const xkv_dims* dims, int32_t layer, const int32_t* budget,
                              int32_t per_sequence, const float* scores, const float* sorted,
                              const void* k, const void* v, const int32_t* cu_seqlens,
                              int64_t total_tokens, int32_t max_seqlen, const xkv_cache* cache,
                              int32_t* sel, int32_t sel_stride,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * xkv_build_block_table -- fills cache->block_table for runs of consecutive pages (no counterpart in the
 * paper: bookkeeping of the reduced caches whose sizes differ per layer, Sec. IV-A).
 *   block_table[l][b][i] = first_page[l][b] + i  for i < n_pages_lb[l][b],  0 otherwise
 * first_page, n_pages_lb  dev int32 [n_layers][batch]; which pages a (layer, sequence) gets is the caller's
 *            decision (it owns the pool), the library only expands it on the device.
 */
xkv_status xkv_build_block_table(const int32_t* first_page, const int32_t* n_pages_lb, const xkv_cache* cache,
                                 int32_t batch, void* stream);

/*
 * xkv_decode_attn -- one generation step of attention over the reduced caches of layers
 * [layer_begin, layer_end) (Eq. 1 with one query row per head; Sec. IV-A generation phase).
 *
 * If k_new and v_new are given, row (l, b, g) is first appended to slot seq_lens[l][b] of the cache
 * and seq_lens[l][b] advances by one (newly generated tokens are stored too and never evicted).
 * Then for every query head h:  out[l,b,h,:] = softmax_c(scale * q[l,b,h,:] . K_c) V_c  over all
 * n filled slots c of (l, b) and KV head h / G, computed with fp32 accumulation in chunks of
 * cache rows whose partial results are merged by log-sum-exp.
 *
 * q          dev bf16 [Lr][B][Hq][d], Lr = layer_end - layer_begin
 * k_new,v_new dev bf16 [Lr][B][Hkv][d], both NULL or both given
 * out        dev out bf16 [Lr][B][Hq][d]; rows of empty caches (n = 0) are zero
 * lse        dev out fp32 [Lr][B][Hq], may be NULL: natural-log sum of exp of the scaled logits
 * chunk_rows 0 = chosen on the device from the cache lengths; otherwise a multiple of 64
 * workspace  dev, at least xkv_workspace_bytes(XKV_OP_DECODE_ATTN, ...) bytes
 * Device status XKV_ERR_CAPACITY if an append does not fit its page table (that row is neither stored
 * nor attended to and its seq_lens entry stays), XKV_ERR_WORKSPACE if the work items planned on the
 * device exceed what the workspace was sized for, XKV_ERR_TIMEOUT if a bounded wait expired.
 * Launches: up to 2048 (layer, sequence) units the call is one small memset and one kernel whose blocks
 * plan their work themselves from the lengths before the call; the block that handles the end of a
 * cache takes the new row from k_new / v_new and stores it, and seq_lens is advanced when the last
 * block leaves. No block waits for another one to start, so the launch needs no particular
 * residency. Larger problems run a separate append-and-plan kernel first.
 */
xkv_status xkv_decode_attn(const xkv_dims* dims, const xkv_cache* cache, int32_t layer_begin,
                           int32_t layer_end, const void* q, const void* k_new, const void* v_new,
                           void* out, float* lse, int32_t chunk_rows,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * xkv_decode_attn_static -- xkv_decode_attn for callers that cannot hand the library a workspace.
 * (The paper has no counterpart: this is the same operation with a different memory arrangement.)
 *
 * Some hosts of this library may not allocate device memory at the point where they decode: code
 * that runs inside a fixed memory plan (every buffer sized before the serving loop starts), plug-ins
 * that only receive their input and output tensors from the framework around them, or code on a
 * path where a cudaMalloc would stall the device. For them the scratch memory of the decode step
 * (status word, merge tickets, work-item table, split-K partial results) is a fixed array of
 * XKV_STATIC_SCRATCH_BYTES inside the library image. Every GPU that loads the library holds that
 * array until the process exits. The call itself allocates and frees nothing.
 *
 * Arguments and results are those of xkv_decode_attn without workspace/workspace_bytes, plus
 *   status_out  dev out int32 [1], may be NULL: receives the device status word of this call
 *               (XKV_OK, XKV_ERR_CAPACITY, XKV_ERR_WORKSPACE, XKV_ERR_TIMEOUT) in stream order; copy it to
 *               the host to read it. Unlike a caller's workspace the array's status word is cleared by
 *               every call.
 * Limits and rules
 *   - Returns XKV_ERR_WORKSPACE, launching nothing, when the scratch this problem needs
 *     (xkv_workspace_bytes(XKV_OP_DECODE_ATTN, ...)) exceeds XKV_STATIC_SCRATCH_BYTES. With
 *     chunk_rows = 0 the library reserves room for about 14 000 chunks beyond one per (layer,
 *     sequence, KV head), which alone passes the limit once G * head_dim >= 256 (any grouped-query
 *     model with head_dim 128): such callers pass an explicit chunk_rows, which sizes the scratch
 *     from the longest cache instead.
 *   - The first call on a device looks up the array's device address (a one-time set-up step);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each call
 *     clears what it needs zeroed. Two calls that overlap on the GPU (different streams) race on
 *     it: keep calls of this entry point on one stream, or order them yourself.
 */
#define XKV_STATIC_SCRATCH_BYTES (16u << 20)
xkv_status xkv_decode_attn_static(const xkv_dims* dims, const xkv_cache* cache, int32_t layer_begin,
                                  int32_t layer_end, const void* q, const void* k_new, const void* v_new,
                                  void* out, float* lse, int32_t chunk_rows, int32_t* status_out, void* stream);

/*
 * Workspace size in bytes for one call of `op` (XKV_OP_*). Unused arguments may be 0.
 *   XKV_OP_SCORE, XKV_OP_SELECT_COMPACT: dims, max_seqlen, total_tokens
 *   XKV_OP_PREFILL_ATTN: dims
 *   XKV_OP_DECODE_ATTN: dims, n_layers (layers per call), max_cache_len (upper bound of any
 *                       seq_lens entry, e.g. max_pages_per_seq*page_size), chunk_rows as passed
 * Returns 0 for invalid arguments.
 */
size_t xkv_workspace_bytes(int32_t op, const xkv_dims* dims, int32_t max_seqlen,
                           int64_t total_tokens, int32_t n_layers, int32_t max_cache_len,
                           int32_t chunk_rows);

/*
 * Copies the device status word of `workspace` to the host, resets the word to XKV_OK, waits for
 * `stream`, and returns what it read: XKV_OK, or the first XKV_ERR_* a kernel recorded in any call
 * on that workspace since the word was last read. This is the only entry point that synchronises.
 */
xkv_status xkv_read_device_status(void* workspace, void* stream);

/*
 * Profiling hook (no counterpart in the paper): while both events are set, every xkv_decode_attn call
 * records `start` on its stream immediately before its attention kernel and `stop` immediately after
 * it, so a caller can time that kernel alone with cudaEventElapsedTime. Events are cudaEvent_t handles
 * owned by the caller; pass NULL, NULL to switch the hook off (the default). Not thread-safe.
 */
void xkv_profile_events(void* start, void* stop);

/*
 * Test hook (no counterpart in the paper), process-wide: the limit of every bounded wait inside the kernels
 * (nanoseconds; <= 0 restores the default of two seconds), and the index of one decode work item whose
 * split-K merge ticket is never published (-1: none), so that a test can watch a wait run out: the kernel
 * returns, the device status reads XKV_ERR_TIMEOUT and the workspace stays usable.
 */
void xkv_test_hooks(int64_t wait_limit_ns, int32_t withhold_decode_item);

/* Number of kernel launches the library enqueued since it was loaded (all entry points). */
int64_t xkv_launch_count(void);

const char* xkv_status_string(xkv_status status);
int32_t xkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* XKV_H_ */
