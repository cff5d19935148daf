// Internal declarations shared by the translation units of librkv (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <map>
#include <utility>
#include <vector>

#include "rkv.h"

namespace rkv {

constexpr int kHeadDim = 128;
constexpr int kMaxGroup = 8;
constexpr int kMaxSplits = 128;        // split-K partials kept per (sequence, KV head)
constexpr int kTile = 64;              // positions per pipeline stage
constexpr int kStages = 3;
constexpr int kAttnThreads = 160;      // 4 MMA warps + 1 copy warp
constexpr int kSelectCluster = 8;      // CTAs that share one top-K problem
constexpr int kAttnCluster = 8;        // most CTAs that share one (sequence, KV head) in the clustered partial step
constexpr int kSelectThreads = 512;
constexpr int kScoreThreads = 256;
constexpr int kSelectMaxKeysPerCta = 40960;   // max_len <= kSelectCluster * this
constexpr int kSelectBins = 4096;      // bins of the per-(sequence, KV head) score histogram in the workspace
constexpr int kSelectMaxSlice = 8192;  // most positions one CTA of the score pass takes

struct PartialLayout {                 // split-K partial of one (b, g, split)
  // o: [8 heads][128] fp32 unnormalised, then m[8], l[8]
  static constexpr int kFloats = kMaxGroup * kHeadDim + 2 * kMaxGroup;
};

struct AttnParams {
  const void* q;              // bf16 [B][Hq][128]
  const int64_t* row_offset;  // [B]
  const int32_t* cap;         // [B]
  const int32_t* len;         // [B]
  const int32_t* active;      // [B] or null
  void* out;                  // bf16 [B][Hq][128]
  float* partials;            // [B*Hkv][max_splits][PartialLayout::kFloats]
  float* ml_t;                // [B*Hkv][16][max_splits]: the (m, l) of the partials again, split-contiguous, or null
  int32_t* tickets;           // [B*Hkv]
  float* logits;              // [B*Hkv][logit_stride][gp] (position-major) or null
  int32_t* status;
  int64_t logit_stride;
  int32_t n_q_heads, n_kv_heads, group;
  int32_t gp;                 // floats per position in the logit scratch: 4 (G <= 4) or 8
  int32_t chunk;              // positions per CTA
  int32_t max_splits;
  int32_t max_len;            // clamp for len[b]
  int32_t spec;               // 1: every CTA has work by construction, first tiles may be requested before len is read
  int32_t early;              // > 0 (with spec): request them before the dependency wait as well - all of them in the
                              // clustered step, this many in the streaming forms
  int32_t interleave;         // 1 (streaming forms): tile j of a (sequence, KV head) goes to CTA j mod gridDim.x
  float scale;
  // fused append (clustered partial step only): the new token's rows and where they go
  const void* k_new;          // bf16 [B][Hkv][128]
  const void* v_new;
  void* small_k; void* small_v;         // the cache being attended (same buffers the tensor maps describe)
  int32_t* small_len;                   // [B] updated by the kernel
  void* full_k; void* full_v;           // optional second cache that receives the rows
  const int64_t* full_row_offset; const int32_t* full_cap; int32_t* full_len;
  int32_t* len_tickets;       // [B] arrival counters of the (sequence, KV head) clusters
  int32_t has_full;
  // fixed-size small cache: the new row replaces the lowest-scoring survivor of the last refresh
  const int32_t* evict_order; // [B][Hkv][max_evict] slots in eviction order, or null (the cache grows)
  int32_t* evict_count;       // [B] evictions since the refresh
  const int32_t* k_small;     // [B] size of the small cache
  int32_t max_evict;
};

// Score pass of the full step: logits -> keys (+ scores) and the histogram of the keys; optionally the fold of out[].
struct ScoreParams {
  const float* logits;        // [B*Hkv][logit_stride][gp]
  const float* partials;      // split partials written by the attention kernel (read when out != null)
  const float* ml_t;          // [B*Hkv][16][max_splits]: m of head j (j < 8) / l of head j - 8, contiguous over the splits
  const void* q;              // bf16 [B][Hq][128] (read when q_last_full != null)
  void* out;                  // bf16 [B][Hq][128], or null: the attention output has been folded already
  void* q_last_full;          // bf16 [B][Hq][128] or null
  const int32_t* cap;
  const int32_t* len;
  const int32_t* k_small;     // [B]
  const int32_t* active;
  float* scores;              // [B][Hkv][score_stride] or null
  uint32_t* keys;             // [B*Hkv][logit_stride]: key of every position
  uint32_t* hist;             // [B*Hkv][kSelectBins]: all zero on entry
  int32_t* anchor;            // [B*Hkv]: where each histogram's window starts (whole nats of -log p)
  int32_t* status;
  int64_t logit_stride, score_stride;
  int32_t n_q_heads, n_kv_heads, group, agg;
  int32_t k_max, max_len;
  int32_t slice, n_slices;    // positions per CTA; CTAs per (sequence, KV head)
  int32_t chunk, max_splits;  // split geometry of the attention launch that produced the partials
  int32_t grid_splits;        // CTAs per (sequence, KV head) that launch had
  int32_t pool_half;          // (pool_kernel - 1) / 2
};

struct SelectParams {
  const uint32_t* keys;       // [B*Hkv][logit_stride]
  uint32_t* hist;             // [B*Hkv][kSelectBins]: read, then cleared
  const int32_t* anchor;      // [B*Hkv]: written by the score pass
  const int32_t* cap;
  const int32_t* len;
  const int32_t* k_small;     // [B]
  const int32_t* active;
  int32_t* topk_idx;          // [B][Hkv][k_max]
  uint32_t* win_keys;         // [B*Hkv][win_stride]: key of every winner, in output order (for the eviction order)
  int32_t win_stride;
  int64_t logit_stride;
  int32_t n_kv_heads;
  int32_t k_max, max_len;
  int32_t keys_per_thread;    // keys per thread of a selection CTA at the host's length bound
  int32_t per_fixed;          // 1: slices are rank * keys_per_thread * threads (one sequence); 0: cut by each sequence's own length
};

struct CacheDev {
  void* k; void* v;
  const int64_t* row_offset; const int32_t* cap; int32_t* len;
};

cudaError_t launch_attention(const AttnParams& p, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                             int n_seq, int grid_x, bool write_logits, cudaStream_t st, bool append = false);
cudaError_t launch_attention_cluster(const AttnParams& p, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                     int n_seq, int cluster, bool append, bool wide, cudaStream_t st);
cudaError_t launch_attention_scores(const AttnParams& p, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                    int n_seq, int grid_x, cudaStream_t st);
cudaError_t launch_evict_order(const uint32_t* win_keys, int win_stride, const int32_t* k_small, int k_max,
                               const int32_t* full_len, const int32_t* active, int32_t* evict_order,
                               int32_t* evict_count, int max_evict, int n_seq, int n_kv_heads, cudaStream_t st);
cudaError_t launch_score(const ScoreParams& p, int n_seq, cudaStream_t st);
cudaError_t launch_select(const SelectParams& p, int n_seq, int cluster, cudaStream_t st);
int score_slice_for(int n_max, int problems, int sm_count);   // positions per CTA of the score pass
int select_cluster_for(int n_max, int keys_per_cta);          // CTAs per (sequence, KV head) of the selection
int select_keys_per_thread(int n_max, int cluster);           // keys per thread of a CTA of such a cluster
cudaError_t launch_gather(const int32_t* topk_idx, const int32_t* k_small, int k_max, CacheDev full,
                          CacheDev small_cache, const int32_t* active, int n_seq, int n_kv_heads,
                          int32_t* status, cudaStream_t st);
cudaError_t launch_append(const void* k_new, const void* v_new, CacheDev full, CacheDev small_cache,
                          bool has_full, bool has_small, int n_seq, int n_kv_heads, int32_t* status,
                          cudaStream_t st);
cudaError_t launch_fold(const float* partials, const float* ml_t, const int32_t* len, const int32_t* cap,
                        const int32_t* active, void* out, int n_seq, int n_q_heads, int n_kv_heads, int chunk,
                        int max_splits, int max_len, int grid_splits, cudaStream_t st);
cudaError_t launch_trigger(const void* q_now, const void* q_last, float threshold, int32_t* flag, int32_t* keep,
                           float* sim, int n_seq, int n_q_heads, cudaStream_t st);
// Launch with optional programmatic dependent launch (the kernel may start while its predecessor on
// the stream drains; every kernel waits with pdl_wait() before touching global memory) and an
// optional thread-block cluster along x.  Every kernel calls pdl_launch() only AFTER its own pdl_wait():
// a kernel can then begin no earlier than the moment its predecessor's own dependency has resolved, so at
// most one earlier launch of this library is still running while a kernel executes the part above its wait.
// The partial step's early cache read (AttnParams::early, early_read_safe below) relies on exactly that.
// (Releasing at the top would also let an attention kernel's CTAs occupy every SM while its predecessor
// drains, shutting out work that another stream wants to run beside it.)
extern bool g_use_pdl;
template <typename... KArgs, typename... Args>
inline cudaError_t launch_ex(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (g_use_pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
// Programmatic dependent launch: let the next kernel on the stream begin its launch now / wait until
// everything the previous kernel wrote is visible.  Both are no-ops without the launch attribute.
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// The library's most recent launch on each stream (host-side record): the K/V buffers it writes (either may be
// NULL).  early_read_safe: the launch before this one on the stream writes no row of cache c, or nothing of
// this library was ever launched on the stream (kernels of other origin complete before a kernel of this
// library starts).
void note_launch(cudaStream_t st, const rkv_cache* a, const rkv_cache* b, bool fold = false);
bool early_read_safe(cudaStream_t st, const rkv_cache* c);
bool last_launch_was_fold(cudaStream_t st);   // the library's last launch on the stream was the full step's merge kernel

cudaError_t prepare_attention();  // one-time function attributes (dynamic shared memory sizes)
cudaError_t prepare_select();
size_t attention_smem_bytes();
size_t select_smem_bytes(int keys_per_thread);

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of one cache buffer ([n_rows][128] bf16) as the attention kernel reads it: a box is 64 rows of both
// 64-channel halves, {channel 0..63, row, half}, so that ONE copy instruction lands a whole K (or V) tile in
// shared memory as [half][row][64 channels] with the 128-byte swizzle - the layout the ldmatrix addressing
// expects.  (The copy engine's cost per instruction is what makes one large box better than two small ones.)
inline CUresult encode_cache_map(EncodeTiledFn encode, void* base, int64_t n_rows, CUtensorMap* out) {
  const cuuint64_t dims[3] = {64, (cuuint64_t)n_rows, 2};
  const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, 128};   // bytes: next row, next half
  const cuuint32_t box[3] = {64, (cuuint32_t)kTile, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

}  // namespace rkv

struct rkv_ctx {
  rkv_config cfg;
  int group;
  int max_splits;
  int64_t logit_stride;
  char* workspace;
  size_t workspace_bytes;
  float* partials;
  float* ml_t;
  int32_t* tickets;
  int32_t* len_tickets;
  uint32_t* win_keys;
  uint32_t* keys;      // key of every position of the last score pass
  uint32_t* hist;      // per (sequence, KV head) histogram of those keys; all zero between selections
  int32_t* anchor;     // per (sequence, KV head): start of the histogram's window
  bool hist_dirty;     // a score pass was launched whose selection (which clears the histogram) was not
  float* logits;
  int32_t* status;
  int64_t launches;
  int device;
  int sm_count;
  int small_min_chunk;
  int small_cluster;   // 1: the partial step merges its splits inside a thread-block cluster when the length allows
  int early_read;      // 1: the attention kernels may request their first cache tiles before their dependency wait
  int interleave;      // 1: the full-cache pass deals a head's tiles out to its CTAs in turn
  int select_keys_per_cta;   // keys one CTA of a selection cluster takes (about): fewer = shorter chain, more = fewer CTAs
  int score_slice;           // positions per CTA of the score pass; 0: chosen per launch
  // geometry of the last rkv_full_attention, for the rkv_select_topk that completes it
  struct { bool valid; int chunk, gx, n_max; const void* full_k; const int32_t* active; } pending_full;
  // ... and of the last rkv_score_keys, for the rkv_select_topk that launches the selection alone
  struct { bool valid; int n_max, k_max; const void* full_k; const int32_t* active; } pending_keys;
  int gp;              // floats per position in the logit scratch
  std::string last_error;
  std::map<std::pair<uint64_t, int64_t>, CUtensorMap> tmaps;   // (base address, rows) -> tensor map
  // optional per-kernel timing (rkv_set_profiling): event pairs recorded around every launch
  bool profiling;
  struct Timed { int kind; cudaEvent_t start, stop; };
  std::vector<Timed> timed;
  std::vector<cudaEvent_t> event_pool;
};
