/*
 * rkv.h - C ABI of the RefreshKV decode-attention library (CUDA, sm_100a).
 *
 * The library implements the per-layer attention work of RefreshKV
 * (arXiv 2411.05787, Sec. 2.2): the periodic FULL step (attention over the
 * whole KV cache C_f, attention scores a_L aggregated over the query heads of
 * each grouped-query group, top-K positions, rebuild of the small cache C_p)
 * and the cheap PARTIAL steps (attention over C_p), plus the cache append and
 * the query-similarity refresh trigger.
 *
 * General conventions
 *  - Every pointer is a DEVICE pointer unless its comment says "host".
 *  - Every call except create/destroy/get_device_status only enqueues work on
 *    the given stream (a cudaStream_t passed as void*; NULL = default stream)
 *    and returns; nothing synchronises, nothing is copied to the host.
 *  - The caller owns all tensors and the stream.  The context owns only its
 *    scratch workspace (split partials, per-head logits, tickets, a status
 *    word), sized once in rkv_create.  Calls on one context must not overlap
 *    on the GPU (they share that workspace): issue them on one stream.
 *  - bf16 tensors are plain arrays of 16-bit brain floats.  head_dim is 128.
 *    Every bf16 tensor (q, out, k_new, v_new, cache buffers) starts on a
 *    16-byte boundary; a misaligned base is RKV_ERR_INVALID_ARG.
 *  - Query head h reads KV head h / G, G = n_q_heads / n_kv_heads (1..8).
 *  - Errors: every call returns an rkv_status.  Bad arguments are detected on
 *    the host before anything is launched.  Conditions only the device can
 *    see (append past capacity, a length above the configured maximum,
 *    a non-finite score, a bounded wait that ran out) set bits in a sticky
 *    device status word (RKV_DEV_*) and the offending access is skipped or
 *    clamped; nothing traps.
 *
 * Cache layout (rkv_cache).  K and V are each ONE buffer of n_rows rows of 128
 * bf16 channels (256 bytes per row, base 16-byte aligned).  Sequence b,
 * KV head g, position p is row  row_offset[b] + g * cap[b] + p.
 * Ragged batches are packed by choosing row_offset/cap per sequence.
 */
#ifndef RKV_H_
#define RKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RKV_HEAD_DIM 128
#define RKV_MAX_GROUP 8

typedef struct rkv_ctx rkv_ctx; /* opaque */

typedef enum {
  RKV_OK = 0,
  RKV_ERR_INVALID_ARG = 1, /* null pointer, size out of the configured range        */
  RKV_ERR_UNSUPPORTED = 2, /* head_dim != 128, G > 8, mode not built                */
  RKV_ERR_WORKSPACE = 3,   /* workspace allocation failed                           */
  RKV_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (rkv_last_cuda_error)*/
  RKV_ERR_DEVICE_CHECK = 5 /* rkv_get_device_status found device-side flags set     */
} rkv_status;

/* bits of the device status word */
#define RKV_DEV_APPEND_OVERFLOW 1 /* rkv_append: len == cap, row not written            */
#define RKV_DEV_LEN_CLAMPED 2     /* a seq_len exceeded cap or max_len and was clamped   */
#define RKV_DEV_NONFINITE 4       /* a NaN/Inf attention logit was seen                  */
#define RKV_DEV_BAD_INDEX 8       /* rkv_gather_small: index outside [0, len), row skipped*/
#define RKV_DEV_TIMEOUT 16        /* a bounded wait inside an attention kernel (for a copy into shared memory,
                                     or for a peer CTA's partial result) ran out: the out[] rows of that call
                                     are not valid.  Never seen in a healthy run; the waits are bounded so that
                                     a lost copy cannot hang the GPU                                          */

/* score aggregation over the query heads of a group (Sec. 2.2 footnote; App. A.3, Table 6) */
typedef enum { RKV_AGG_MAX = 0, RKV_AGG_MEAN = 1, RKV_AGG_FIRST = 2 } rkv_agg;

typedef struct {
  int32_t n_seq;         /* B                                                          */
  int32_t n_q_heads;     /* Hq                                                         */
  int32_t n_kv_heads;    /* Hkv; Hq % Hkv == 0, Hq / Hkv <= 8                          */
  int32_t head_dim;      /* must be 128                                                */
  int32_t max_len;       /* largest full-cache length any call will see (<= 327680)    */
  int32_t max_small;     /* largest small-cache length any call will see               */
  int32_t agg;           /* rkv_agg; RKV_AGG_MAX is the paper's rule                   */
  int32_t pool_kernel;   /* 1 = no pooling; odd w in 3..31 = the scores are max-pooled over w neighbouring
                            positions before the top-K (App. A.1: 7)                                   */
  float softmax_scale;   /* 0 -> 1/sqrt(head_dim)                                      */
} rkv_config;

typedef struct {
  void* k;                   /* bf16 [n_rows][128]                                     */
  void* v;                   /* bf16 [n_rows][128]                                     */
  int64_t n_rows;            /* host value: rows in each buffer (< 2^31)               */
  const int64_t* row_offset; /* [B] first row of sequence b      } constant while calls  */
  const int32_t* cap;        /* [B] capacity of sequence b       } are in flight: kernels */
                             /*     in positions                 } may read them early    */
  int32_t* len;              /* [B] current length; append / gather_small update it    */
} rkv_cache;

/* Host.  Creates a context on the current device and allocates its workspace
 * (cudaMalloc).  *out is NULL on failure. */
rkv_status rkv_create(const rkv_config* cfg /*host*/, rkv_ctx** out /*host*/);
/* Host.  Frees the workspace.  The caller must have synchronised its streams. */
rkv_status rkv_destroy(rkv_ctx* ctx);
/* Host.  Bytes of device workspace rkv_create allocates for this config (0 if cfg is invalid). */
size_t rkv_workspace_bytes(const rkv_config* cfg /*host*/);

/*
 * FULL step (Sec. 2.2 "Decoding with full cache"; App. A.1 on obtaining the
 * scores; Sec. 2.2 footnote on the group aggregation).  For every sequence b
 * with active[b] != 0 (active == NULL: all) and n = full->len[b]:
 *   s[h][j]   = scale * <q[b][h], K[b][h/G][j]>               j < n
 *   p[h][j]   = softmax_j(s[h][:])
 *   out[b][h] = sum_j p[h][j] V[b][h/G][j]                     (bf16)
 *   score[b][g][j] = agg_{h in group g} p[h][j]                (fp32, optional output);
 *       with cfg.pool_kernel = w > 1:  score[j] <- max over |i - j| <= (w-1)/2, 0 <= i < n  (Sec. 2.2
 *       "Prefilling stage": max pooling over the scores of surrounding tokens)
 *   topk_idx[b][g][0..m) = the m = min(k_small[b], n) positions of largest
 *       score, ties to the lower position, listed in ASCENDING position
 *       order; entries m..k_max-1 are -1.
 * If q_last_full != NULL, q[b] is copied there for the active sequences (the
 * reference query of the refresh trigger).  Inactive sequences: nothing is
 * read or written.
 *   q            bf16 [B][Hq][128]
 *   k_small      int32 [B]  small-cache size per sequence, 0 <= k_small[b] <= k_max
 *   k_max        host value, 1..max_small
 *   out          bf16 [B][Hq][128]
 *   scores       fp32 [B][Hkv][score_stride] or NULL; positions >= n are not written
 *   score_stride host value >= max length in this call (ignored if scores == NULL)
 *   topk_idx     int32 [B][Hkv][k_max]
 *   max_len_hint host value: upper bound of full->len[b] over active b in this
 *                call (0 = cfg.max_len).  Only launch geometry depends on it;
 *                a longer sequence is clamped and flagged RKV_DEV_LEN_CLAMPED.
 */
rkv_status rkv_full_step(rkv_ctx* ctx, const void* q, const rkv_cache* full /*host struct*/,
                         const int32_t* k_small, int32_t k_max, const int32_t* active,
                         void* out, float* scores, int64_t score_stride, int32_t* topk_idx,
                         void* q_last_full, int32_t max_len_hint, void* stream);

/*
 * The two halves of rkv_full_step as calls of their own (Sec. 2.2: the full step's attention output is
 * what the decoder needs next; the refreshed partial cache is first read by the NEXT token's partial
 * step).  A caller that wants the attention output early - and the selection and the rebuild of C_p
 * off the layer's critical path, e.g. on a second stream under the next layer's work - calls
 *   rkv_full_attention   attention over C_f: out is complete when this call's two kernels end (the
 *                        streaming pass, then a short merge of its split partials); the logits
 *                        and softmax statistics stay in the context's workspace
 *                        (rkv_append_full_attention: the same behind the token's append);
 *   rkv_select_topk      scores, topk_idx, q_last_full from that workspace (same values as
 *                        rkv_full_step; out differs from rkv_full_step's by summation order only).
 * rkv_select_topk completes the LAST rkv_[append_]full_attention of the same context and must be given the same
 * cache and mask (otherwise RKV_ERR_INVALID_ARG; also when there is no attention pass to complete).  The
 * workspace holds one pass: no other rkv_full_step / rkv_score_step / rkv_full_attention on this
 * context may run between the two (stream order, or an event, must put them after rkv_select_topk);
 * callers that overlap the halves of consecutive layers use one context per layer in flight.
 * Arguments as in rkv_full_step; q may be NULL in rkv_select_topk when q_last_full is.
 */
rkv_status rkv_full_attention(rkv_ctx* ctx, const void* q, const rkv_cache* full /*host struct*/,
                              const int32_t* active, void* out, int32_t max_len_hint, void* stream);
/* The same with the token's new rows appended to C_f first, inside the streaming pass's kernel (no launch of
 * its own; the result is that of rkv_append(ctx, k_new, v_new, full, NULL) followed by rkv_full_attention): every sequence's
 * cache grows by one row - inactive ones too, as in rkv_append - and the attention of the active ones
 * covers the new row.  max_len_hint bounds the lengths AFTER the append.  A cache already at capacity
 * sets RKV_DEV_APPEND_OVERFLOW and is attended as it is.  (Sec. 2.2: new KV pairs are appended to both
 * caches; the full step that follows rebuilds C_p, so only C_f needs the row here.) */
rkv_status rkv_append_full_attention(rkv_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                     const rkv_cache* full /*host struct*/, const int32_t* active, void* out,
                                     int32_t max_len_hint, void* stream);
rkv_status rkv_select_topk(rkv_ctx* ctx, const void* q, const rkv_cache* full /*host struct*/,
                           const int32_t* k_small, int32_t k_max, const int32_t* active, float* scores,
                           int64_t score_stride, int32_t* topk_idx, void* q_last_full, void* stream);
/* The second half cut once more, for callers that want its first launch early: rkv_score_keys runs the score pass
 * alone - the logits the attention pass left in the workspace become aggregated scores (written to scores[] when it
 * is not NULL), their order-preserving keys and the per-(sequence, KV head) histogram, and q goes to q_last_full when
 * that is not NULL - and the NEXT rkv_select_topk on the context (same cache, mask and k_max; scores and q_last_full
 * NULL, they have been written) launches the selection alone.  Right behind the attention pass the logits are
 * still in L2; the top-K and the rebuild can then follow whenever the caller likes (Sec. 2.2: the refreshed C_p is
 * first needed by the next token).  Same indices and scores as rkv_full_step. */
rkv_status rkv_score_keys(rkv_ctx* ctx, const void* q, const rkv_cache* full /*host struct*/, const int32_t* k_small,
                          int32_t k_max, const int32_t* active, float* scores, int64_t score_stride,
                          void* q_last_full, void* stream);

/*
 * Score-only refresh step (Sec. 4.2 "Impact of full attention steps", the "w/o full attention" setting:
 * at the stride the attention scores over the entire cache update the partial cache, and the step then
 * attends to the UPDATED partial cache instead of the full one; the paper reports the same quality as
 * the regular method).  Computes exactly the scores / topk_idx / q_last_full of rkv_full_step but reads
 * the K half of C_f only and produces no attention output: half the bytes of a full step.  The caller
 * follows it with rkv_gather_small and rkv_small_step.  Arguments as in rkv_full_step (without out).
 */
rkv_status rkv_score_step(rkv_ctx* ctx, const void* q, const rkv_cache* full /*host struct*/,
                          const int32_t* k_small, int32_t k_max, const int32_t* active, float* scores,
                          int64_t score_stride, int32_t* topk_idx, void* q_last_full, int32_t max_len_hint,
                          void* stream);

/*
 * Rebuild C_p from the selected positions (Sec. 2.2 "refresh the partial
 * cache").  For active b, KV head g, r < m = min(k_small[b], full->len[b]):
 *   small.K[b][g][r] = full.K[b][g][topk_idx[b][g][r]]   (same for V; bit copy)
 * and small->len[b] = m.  Entries of topk_idx that are -1 are skipped; an
 * index outside [0, full->len[b]) is skipped and flagged RKV_DEV_BAD_INDEX.
 * Requires m <= small->cap[b].
 */
rkv_status rkv_gather_small(rkv_ctx* ctx, const int32_t* topk_idx, const int32_t* k_small,
                            int32_t k_max, const rkv_cache* full /*host struct*/,
                            const rkv_cache* small_cache /*host struct*/, const int32_t* active,
                            void* stream);

/*
 * PARTIAL step (Sec. 2.2 "Decoding with partial cache"): softmax attention of
 * q over the first small->len[b] rows of the small cache, for sequences with
 * active[b] != 0 (NULL: all).  out as in rkv_full_step.  max_len_hint: upper
 * bound of small->len[b] (0 = cfg.max_small).
 */
rkv_status rkv_small_step(rkv_ctx* ctx, const void* q, const rkv_cache* small_cache /*host struct*/,
                          const int32_t* active, void* out, int32_t max_len_hint, void* stream);

/*
 * Append the current token's key/value (Sec. 2.1: the cache is updated with
 * the current token's pair; Sec. 2.2: both C_p and C_f receive it).  For each
 * non-NULL cache c and every b: row len[b] of every KV head receives
 * k_new[b][g] / v_new[b][g], then c->len[b] += 1.  If len[b] == cap[b] nothing
 * is written for that sequence and RKV_DEV_APPEND_OVERFLOW is set.
 *   k_new, v_new  bf16 [B][Hkv][128]
 */
rkv_status rkv_append(rkv_ctx* ctx, const void* k_new, const void* v_new,
                      const rkv_cache* full /*host struct or NULL*/,
                      const rkv_cache* small_cache /*host struct or NULL*/, void* stream);

/*
 * Append + PARTIAL step in one call (Sec. 2.2 "Decoding with partial cache": the step attends over
 * C_p and stores the input token's K/V; C_f receives the pair as well).  Same result as
 *   rkv_append(k_new, v_new, full, small_cache)  followed by  rkv_small_step(q, small_cache, active, out):
 * every sequence (active or not) gets the new row in both caches and its lengths bumped; sequences with
 * active[b] != 0 (NULL: all) attend over the small cache including the new row.  When the length bound
 * allows the clustered partial step (see RKV_OPT_SMALL_CLUSTER) this is ONE kernel launch; otherwise the
 * two kernels are launched back to back.  full may be NULL (only the small cache receives the row).
 * max_len_hint bounds small->len[b] AFTER the append (0 = cfg.max_small).
 */
rkv_status rkv_append_small_step(rkv_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                 const rkv_cache* full /*host struct or NULL*/,
                                 const rkv_cache* small_cache /*host struct*/, const int32_t* active,
                                 void* out, int32_t max_len_hint, void* stream);

/*
 * Fixed-size partial cache (Sec. 2.2 "Decoding with partial cache": to keep |C_p| = K while decoded tokens
 * are stored, the entry with the lowest attention score of the last full step is removed for each new
 * token).  Two calls replace rkv_gather_small / rkv_append_small_step:
 *
 * rkv_gather_small_evict  = rkv_gather_small, and additionally, from the scores of the rkv_full_step /
 *   rkv_score_step issued just before on the same context and stream, the eviction order of the rebuilt
 *   cache: evict_order[b][g][i] = row of the small cache (0 .. m-1) that the i-th new token will replace,
 *   lowest score first, the later position first among equal scores; -1 beyond m.  evict_count[b] <- 0.
 * rkv_append_small_step_evict = rkv_append_small_step, except that a sequence whose small cache has
 *   reached k_small[b] rows does not grow: the new row overwrites row evict_order[b][g][evict_count[b]]
 *   of every KV head and evict_count[b] += 1 (a shorter cache still grows).  After max_evict evictions
 *   without a refresh the row is not stored in the small cache and RKV_DEV_APPEND_OVERFLOW is set.
 *   evict_order  int32 [B][Hkv][max_evict];  evict_count  int32 [B];  max_evict  host value, 1..4096
 *   k_max <= 4096.  Needs the clustered partial step (RKV_OPT_SMALL_CLUSTER on, length bound <= 8192).
 */
rkv_status rkv_gather_small_evict(rkv_ctx* ctx, const int32_t* topk_idx, const int32_t* k_small, int32_t k_max,
                                  const rkv_cache* full /*host struct*/, const rkv_cache* small_cache /*host struct*/,
                                  const int32_t* active, int32_t* evict_order, int32_t* evict_count,
                                  int32_t max_evict, void* stream);
rkv_status rkv_append_small_step_evict(rkv_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                       const rkv_cache* full /*host struct or NULL*/,
                                       const rkv_cache* small_cache /*host struct*/, const int32_t* k_small,
                                       const int32_t* active, void* out, const int32_t* evict_order,
                                       int32_t* evict_count, int32_t max_evict, int32_t max_len_hint,
                                       void* stream);

/*
 * Refresh trigger (Sec. 2.2 "Deciding when to decode with full cache").
 *   qbar  = mean over the Hq heads of q_now[b];  qbar' likewise from q_last_full[b]
 *   sim   = <qbar, qbar'> / (|qbar| |qbar'|)          (fp32)
 *   flag[b] = 0 (partial step) if sim > threshold, else 1 (full step);
 *   equality and NaN (a zero mean vector) give 1.
 *   keep[b] = 1 - flag[b]: the mask of the sequences that stay on the partial cache, ready to be
 *   passed as `active` to rkv_small_step / rkv_append_small_step while flag goes to rkv_full_step.
 *   q_now, q_last_full  bf16 [B][Hq][128];  flag int32 [B];  keep int32 [B] or NULL;  sim fp32 [B] or NULL
 */
rkv_status rkv_should_refresh(rkv_ctx* ctx, const void* q_now, const void* q_last_full,
                              float threshold, int32_t* flag, int32_t* keep, float* sim, void* stream);

/*
 * Partial step without a context and without any allocation (the paper has no counterpart: this
 * exists for deployment reasons only).
 *
 * Who needs it: hosts that cannot call cudaMalloc where they run attention - a serving runtime
 * whose own arena already owns the device heap, a plugin that must stay inside another program's
 * memory budget, a latency path on which an allocation (which synchronises the device) is not
 * allowed.  rkv_create allocates a workspace, so such callers cannot hold an rkv_ctx.  This call
 * computes exactly what rkv_small_step computes, but its scratch (split partials, arrival
 * tickets, a status word) is a fixed array inside the library image: every device that loads the
 * library holds those ~2.1 MB until the process exits.  The call never calls cudaMalloc, cudaFree
 * or any other allocating routine; the caller passes inputs and outputs as usual.
 *
 * Limits (the array is sized for them; beyond them the call returns RKV_ERR_UNSUPPORTED and, if
 * err_msg is given, says which limit was hit):
 *   cfg->n_seq * cfg->n_kv_heads <= RKV_NOALLOC_MAX_PROBLEMS
 *   length bound (max_len_hint, or cfg->max_small when the hint is 0) <= RKV_NOALLOC_MAX_LEN
 * Of cfg only n_seq, n_q_heads, n_kv_heads, head_dim, max_small and softmax_scale are read.
 *
 * First call on a device: looks up the array's device address, sets the kernel's shared-memory
 * attribute and resolves the tensor-map encoder (host work, once per device, under a lock).  If the
 * library's device code has not been loaded on that device yet, the CUDA runtime loads it during
 * this first call, which is when the device memory for the code and for the array itself is taken;
 * from the second call on, device memory use does not change.  Make that first call outside any
 * stream capture.
 * Sharing: every call on a device uses the same array, which keeps the previous call's contents;
 * the call clears the tickets (and the built-in status word) on the stream before it launches.
 * Two calls that overlap on the GPU (different streams, no ordering) race on the array: order them.
 *   device_status  optional device int32: receives the RKV_DEV_* bits the kernel raises (sticky,
 *                  the caller clears it).  NULL: the bits go to the built-in word and are dropped.
 *   err_msg        optional host buffer of err_cap bytes for a one-line reason on failure.
 * Other arguments as in rkv_small_step.
 */
#define RKV_NOALLOC_MAX_PROBLEMS 32
#define RKV_NOALLOC_MAX_SPLITS 16
#define RKV_NOALLOC_MAX_LEN 65536
rkv_status rkv_small_step_noalloc(const rkv_config* cfg /*host*/, const void* q,
                                  const rkv_cache* small_cache /*host struct*/, const int32_t* active,
                                  void* out, int32_t max_len_hint, int32_t* device_status, void* stream,
                                  char* err_msg /*host*/, size_t err_cap);

/* Host.  Synchronises the stream, copies the sticky device status word to
 * *host_bits, clears it, and returns RKV_ERR_DEVICE_CHECK if it was non-zero. */
rkv_status rkv_get_device_status(rkv_ctx* ctx, int32_t* host_bits /*host*/, void* stream);

/* Host.  Static strings; never NULL. */
const char* rkv_status_string(rkv_status s);
const char* rkv_last_cuda_error(const rkv_ctx* ctx);

/* Host.  Number of kernels this context has launched since creation (each call
 * above launches a fixed, documented number; used by benchmarks to report it). */
int64_t rkv_launch_count(const rkv_ctx* ctx);

/*
 * Launch-geometry knobs (no counterpart in the paper).  Results never depend on them beyond
 * floating-point summation order.
 *   RKV_OPT_SMALL_MIN_CHUNK   positions per CTA (at least) in rkv_small_step when its splits are merged
 *                             through the workspace; default 256, >= 64
 *   RKV_OPT_SMALL_CLUSTER     1 (default): rkv_small_step merges the splits of one (sequence, KV head)
 *                             inside a thread-block cluster (no workspace traffic) when the length
 *                             bound is at most 8192 positions; 0: always through the workspace
 *   RKV_OPT_DEPENDENT_LAUNCH  1 (default): kernels are launched with programmatic stream
 *                             serialisation so that a kernel's launch overlaps the tail of its
 *                             predecessor; 0: plain stream order.  Process-wide.
 *   RKV_OPT_EARLY_CACHE_READ  1 (default): an attention kernel may request its first tiles of the attended cache
 *                             before its stream dependency has resolved - the clustered partial step its whole
 *                             share, the full-cache pass (one sequence, no mask) the first one to three tiles per
 *                             CTA - when the library's previous launch on the same stream wrote no row of that
 *                             cache (the library keeps a host-side record per stream; the row a call appends
 *                             itself is patched in on chip; kernels of other origin complete before a kernel of
 *                             this library starts, unless they themselves release their dependents early while
 *                             still writing the cache - turn the option off in that case); 0: never.
 *   RKV_OPT_INTERLEAVE_TILES  1 (default): the full-cache pass deals the 64-position tiles of a (sequence,
 *                             KV head) out to its CTAs in turn, so that every CTA walks the whole length and
 *                             all carry the same number of tiles up to one; 0: each CTA takes one contiguous
 *                             chunk.  Either way the assignment is fixed by the launch geometry, so results
 *                             are reproducible bit for bit (the two settings differ in summation order).
 *   RKV_OPT_SELECT_KEYS_PER_CTA  keys (positions) one CTA of a top-K cluster takes, 512..40960; default 4096.
 *                             The cluster has 1, 2, 4 or 8 CTAs per (sequence, KV head): fewer keys per CTA give
 *                             the shortest chain for a single selection, more keys per CTA occupy fewer SMs
 *                             when many selections run side by side.  The selected set does not depend on it.
 *   RKV_OPT_SCORE_SLICE       fewest positions one CTA of the score pass takes: 0 (default) = chosen per launch
 *                             alone (the smallest of 1024, 2048, 4096, 8192 that keeps the grid near four CTAs per
 *                             SM); 1024, 2048, 4096 or 8192 = that choice, but no less than this.  Longer slices mean
 *                             fewer CTAs that each pay the log-sum-exp and the histogram flush once: slower for a
 *                             single selection, cheaper when many run side by side.  Keys, scores and the selected
 *                             set do not depend on it.
 */
#define RKV_OPT_SMALL_MIN_CHUNK 1
#define RKV_OPT_DEPENDENT_LAUNCH 2
#define RKV_OPT_SMALL_CLUSTER 3
#define RKV_OPT_EARLY_CACHE_READ 4
#define RKV_OPT_INTERLEAVE_TILES 5
#define RKV_OPT_SELECT_KEYS_PER_CTA 6
#define RKV_OPT_SCORE_SLICE 7
rkv_status rkv_set_option(rkv_ctx* ctx, int32_t option, int32_t value);
/* The option's current value (host memory); RKV_ERR_INVALID_ARG for an unknown option or a NULL pointer. */
rkv_status rkv_get_option(const rkv_ctx* ctx, int32_t option, int32_t* value);

/*
 * Optional per-kernel timing (no counterpart in the paper, which reports wall-clock decode time
 * only).  While profiling is on, every kernel launch is bracketed by CUDA events on the caller's
 * stream; rkv_get_profile waits for them, adds up the elapsed device time per kernel kind, returns
 * the sums and the launch counts and forgets the samples.  Do not enable it during stream capture.
 *   total_us, launches   host arrays of RKV_KERNEL_KINDS entries
 */
#define RKV_KERNEL_ATTN_FULL 0  /* full-cache attention + logit emission (rkv_full_step, 1st kernel) */
#define RKV_KERNEL_SELECT 1     /* top-K from the keys' histogram        (rkv_full_step, 3rd kernel) */
#define RKV_KERNEL_ATTN_SMALL 2 /* small-cache attention                 (rkv_small_step)            */
#define RKV_KERNEL_GATHER 3     /* rkv_gather_small                                                  */
#define RKV_KERNEL_APPEND 4     /* rkv_append                                                        */
#define RKV_KERNEL_TRIGGER 5    /* rkv_should_refresh                                                */
#define RKV_KERNEL_FOLD 6       /* output from the split partials        (rkv_[append_]full_attention, 2nd kernel) */
#define RKV_KERNEL_SCORE 7      /* logits -> scores, keys, histogram     (rkv_full_step, 2nd kernel) */
#define RKV_KERNEL_KINDS 8
rkv_status rkv_set_profiling(rkv_ctx* ctx, int32_t on);
rkv_status rkv_get_profile(rkv_ctx* ctx, double* total_us /*host*/, int64_t* launches /*host*/);

#ifdef __cplusplus
}
#endif
#endif /* RKV_H_ */
