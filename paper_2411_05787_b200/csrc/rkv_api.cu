// C ABI of librkv: argument validation, workspace, tensor maps, launches.
#include <math.h>
#include <string.h>

#include <mutex>
#include <new>
#include <utility>

#include "rkv_internal.h"

namespace {

using rkv::AttnParams;
using rkv::CacheDev;
using rkv::ScoreParams;
using rkv::SelectParams;

rkv::EncodeTiledFn g_encode = nullptr;
// kernel attributes (dynamic shared-memory sizes) are set per device, once
constexpr int kMaxDevices = 64;
bool g_prepared[kMaxDevices] = {};
std::mutex g_prepare_mu;

bool config_ok(const rkv_config* c, rkv_status* why) {
  if (c == nullptr) { *why = RKV_ERR_INVALID_ARG; return false; }
  if (c->n_seq < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->max_len < 1 || c->max_small < 1 ||
      c->n_q_heads % c->n_kv_heads != 0) { *why = RKV_ERR_INVALID_ARG; return false; }
  if (c->head_dim != rkv::kHeadDim || c->n_q_heads / c->n_kv_heads > rkv::kMaxGroup ||
      c->agg < RKV_AGG_MAX || c->agg > RKV_AGG_FIRST || c->pool_kernel < 1 || c->pool_kernel > 31 ||
      c->pool_kernel % 2 == 0 ||
      (int64_t)c->max_len > (int64_t)rkv::kSelectCluster * rkv::kSelectMaxKeysPerCta ||
      (int64_t)c->n_seq * c->n_kv_heads > 65535 * 8) { *why = RKV_ERR_UNSUPPORTED; return false; }
  if (!(c->softmax_scale >= 0.f) || isinf(c->softmax_scale)) { *why = RKV_ERR_INVALID_ARG; return false; }
  return true;
}

int splits_for(const rkv_config* c) {
  int s = (c->max_len + rkv::kTile - 1) / rkv::kTile;
  return s < rkv::kMaxSplits ? (s < 1 ? 1 : s) : rkv::kMaxSplits;
}

struct WsLayout { size_t partials, ml_t, tickets, len_tickets, win_keys, keys, hist, anchor, logits, status, total; int64_t logit_stride; };

WsLayout ws_layout(const rkv_config* c) {
  WsLayout w;
  const size_t bg = (size_t)c->n_seq * c->n_kv_heads;
  const int group = c->n_q_heads / c->n_kv_heads;
  auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
  w.logit_stride = ((int64_t)c->max_len + 63) & ~int64_t(63);
  size_t off = 0;
  w.partials = off; off = up(off + bg * splits_for(c) * rkv::PartialLayout::kFloats * sizeof(float));
  w.ml_t = off;     off = up(off + bg * 16 * (size_t)splits_for(c) * sizeof(float));
  w.tickets = off;  off = up(off + bg * sizeof(int32_t));
  w.len_tickets = off; off = up(off + (size_t)c->n_seq * sizeof(int32_t));
  w.win_keys = off; off = up(off + bg * (size_t)c->max_small * sizeof(uint32_t));
  w.keys = off;     off = up(off + bg * (size_t)w.logit_stride * sizeof(uint32_t));
  w.hist = off;     off = up(off + bg * (size_t)rkv::kSelectBins * sizeof(uint32_t));
  w.anchor = off;   off = up(off + bg * sizeof(int32_t));
  const int gp = group <= 4 ? 4 : 8;   // position-major logits, padded to a vector width
  w.logits = off;   off = up(off + bg * gp * (size_t)w.logit_stride * sizeof(float));
  w.status = off;   off = up(off + sizeof(int32_t));
  w.total = off;
  return w;
}

rkv_status cuda_fail(rkv_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) ctx->last_error = std::string(where) + ": " + cudaGetErrorString(e);
  return RKV_ERR_CUDA;
}

bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15) == 0; }   // NULL counts as aligned
bool cache_ok(const rkv_cache* c) {
  return c && c->k && c->v && c->row_offset && c->cap && c->len && c->n_rows > 0 && c->n_rows < (int64_t(1) << 31) &&
         (reinterpret_cast<uintptr_t>(c->k) & 15) == 0 && (reinterpret_cast<uintptr_t>(c->v) & 15) == 0;
}

// Brackets one kernel launch with events when profiling is on.
struct LaunchScope {
  rkv_ctx* ctx; cudaStream_t st; int kind; cudaEvent_t stop = nullptr;
  static cudaEvent_t get(rkv_ctx* c) {
    cudaEvent_t e = nullptr;
    if (!c->event_pool.empty()) { e = c->event_pool.back(); c->event_pool.pop_back(); return e; }
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
  }
  LaunchScope(rkv_ctx* c, cudaStream_t s, int k) : ctx(c), st(s), kind(k) {
    if (!ctx->profiling) return;
    cudaEvent_t start = get(ctx);
    stop = get(ctx);
    if (start == nullptr || stop == nullptr) { stop = nullptr; return; }
    cudaEventRecord(start, st);
    ctx->timed.push_back({kind, start, stop});
  }
  ~LaunchScope() { if (stop != nullptr) cudaEventRecord(stop, st); }
};

CacheDev dev_of(const rkv_cache* c) { return CacheDev{c->k, c->v, c->row_offset, c->cap, c->len}; }

// [n_rows][128] bf16 as {64 channels, row, half}: one box = 64 rows x both halves, 128-byte swizzle
rkv_status tensor_map(rkv_ctx* ctx, void* base, int64_t n_rows, CUtensorMap* out) {
  const std::pair<uint64_t, int64_t> key(reinterpret_cast<uint64_t>(base), n_rows);   // the map depends on nothing else
  auto it = ctx->tmaps.find(key);
  if (it != ctx->tmaps.end()) { *out = it->second; return RKV_OK; }
  if (g_encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess)
      return cuda_fail(ctx, e == cudaSuccess ? cudaErrorUnknown : e, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
    g_encode = reinterpret_cast<rkv::EncodeTiledFn>(fn);
  }
  CUtensorMap tm;
  CUresult r = rkv::encode_cache_map(g_encode, base, n_rows, &tm);
  if (r != CUDA_SUCCESS) {
    ctx->last_error = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
    return RKV_ERR_CUDA;
  }
  if (ctx->tmaps.size() > 8192) ctx->tmaps.clear();
  ctx->tmaps.emplace(key, tm);
  *out = tm;
  return RKV_OK;
}

// Positions per CTA.  Full step: one balanced wave over 2 CTAs per SM when that keeps chunks moderate,
// otherwise fixed 2048-position chunks over several waves (ragged batches then balance by count).
// Small step: the work is tiny and latency-bound, so chunks of at least 256 positions keep the
// number of partials that the last CTA has to fold small.
int choose_chunk(const rkv_ctx* ctx, int n_max, bool full, int* grid_x) {
  const int bg = ctx->cfg.n_seq * ctx->cfg.n_kv_heads;
  const int slots = 2 * ctx->sm_count;
  int splits = slots / bg;
  if (splits < 1) splits = 1;
  if (splits > ctx->max_splits) splits = ctx->max_splits;
  int chunk = (n_max + splits - 1) / splits;
  if (chunk > 4096) chunk = 2048;
  const int floor_chunk = full ? rkv::kTile : ctx->small_min_chunk;
  if (chunk < floor_chunk) chunk = floor_chunk;
  chunk = (chunk + 15) & ~15;
  int gx = (n_max + chunk - 1) / chunk;
  while (gx > ctx->max_splits) {  // keep the partial buffer's bound
    chunk *= 2;
    gx = (n_max + chunk - 1) / chunk;
  }
  *grid_x = gx < 1 ? 1 : gx;
  return chunk;
}

// Longest small cache that the clustered partial step takes (8 CTAs x 1024 positions).
constexpr int kClusterMaxLen = 8192;

struct AppendArgs {
  const void* k_new; const void* v_new; const rkv_cache* full;
  const int32_t* evict_order; int32_t* evict_count; const int32_t* k_small; int max_evict;   // all null / 0: the cache grows
};

bool cluster_eligible(const rkv_ctx* ctx, int n_max) { return ctx->small_cluster != 0 && n_max <= kClusterMaxLen; }

rkv_status run_attention(rkv_ctx* ctx, const void* q, const rkv_cache* cache, const int32_t* active, void* out,
                         int n_max, int limit, bool logits, cudaStream_t st, int* chunk_out, int* gx_out,
                         const AppendArgs* app = nullptr, bool score_only = false) {
  if (!aligned16(q) || !aligned16(out) || (app != nullptr && (!aligned16(app->k_new) || !aligned16(app->v_new))))
    return RKV_ERR_INVALID_ARG;   // the kernels read and write these 16 bytes at a time
  CUtensorMap tm_k, tm_v;
  rkv_status s = tensor_map(ctx, cache->k, cache->n_rows, &tm_k);
  if (s != RKV_OK) return s;
  s = tensor_map(ctx, cache->v, cache->n_rows, &tm_v);
  if (s != RKV_OK) return s;
  AttnParams p;
  memset(&p, 0, sizeof(p));
  int gx = 1;
  const bool cluster = !logits && cluster_eligible(ctx, n_max);
  if (cluster) {   // 1, 2, 4 or 8 CTAs per (sequence, KV head), whole tiles each
    const int tiles = (n_max + rkv::kTile - 1) / rkv::kTile;
    gx = tiles >= 5 ? 8 : tiles >= 3 ? 4 : tiles >= 2 ? 2 : 1;
    // with many (sequence, KV head) pairs one wave of CTAs is enough: fewer, longer CTAs per pair spend a smaller
    // share of their time on the exchange inside the cluster
    const int bg = ctx->cfg.n_seq * ctx->cfg.n_kv_heads;
    while (gx > 1 && (int64_t)gx * bg > 2 * ctx->sm_count) gx >>= 1;
    p.chunk = ((tiles + gx - 1) / gx) * rkv::kTile;
  } else {
    p.chunk = choose_chunk(ctx, n_max, logits, &gx);
  }
  // Streaming forms: the head's tiles are dealt out to the gx CTAs in turn; the partial slots in use are then
  // min(tiles, gx), which is what the consumers of (chunk, gx) compute when they are told chunk = one tile.
  p.interleave = (logits && ctx->interleave) ? 1 : 0;
  if (chunk_out) *chunk_out = p.interleave ? rkv::kTile : p.chunk;
  if (gx_out) *gx_out = gx;
  p.q = q;
  p.row_offset = cache->row_offset;
  p.cap = cache->cap;
  p.len = cache->len;
  p.active = active;
  p.out = out;
  p.partials = ctx->partials;
  p.tickets = ctx->tickets;
  p.ml_t = ctx->ml_t;
  p.logits = logits ? ctx->logits : nullptr;
  p.status = ctx->status;
  p.logit_stride = ctx->logit_stride;
  p.n_q_heads = ctx->cfg.n_q_heads;
  p.n_kv_heads = ctx->cfg.n_kv_heads;
  p.group = ctx->group;
  p.gp = ctx->gp;
  p.max_splits = ctx->max_splits;
  p.max_len = limit;
  p.scale = ctx->cfg.softmax_scale;
  // without a mask: a cluster per head always has work; a streaming grid has when it serves a single sequence
  p.spec = (active == nullptr && (cluster || (logits && ctx->cfg.n_seq == 1))) ? 1 : 0;
  // Early cache read: only when the launch before this one on the stream leaves the attended cache alone (a
  // gather or an append into it forbids it; so does an unknown history).
  p.early = (cluster && p.spec != 0 && ctx->early_read && rkv::early_read_safe(st, cache)) ? 1 : 0;
  // The streaming pass does the same with its first tiles: all stages of its ring, or - when the launch before it
  // is the short merge kernel of the previous pass, whose few loads would queue behind them - one tile.
  if (logits && p.spec != 0 && ctx->early_read && rkv::early_read_safe(st, cache))
    p.early = rkv::last_launch_was_fold(st) ? 1 : rkv::kStages;
  if (app != nullptr) {   // the clustered partial step and the full step's attention pass can take the append with them
    if (!cluster && !(logits && !score_only)) return RKV_ERR_INVALID_ARG;
    p.k_new = app->k_new;
    p.v_new = app->v_new;
    p.small_k = cache->k;
    p.small_v = cache->v;
    p.small_len = cache->len;
    p.len_tickets = ctx->len_tickets;
    p.has_full = app->full != nullptr;
    p.evict_order = app->evict_order;
    p.evict_count = app->evict_count;
    p.k_small = app->k_small;
    p.max_evict = app->max_evict;
    if (app->full != nullptr) {
      p.full_k = app->full->k;
      p.full_v = app->full->v;
      p.full_row_offset = app->full->row_offset;
      p.full_cap = app->full->cap;
      p.full_len = app->full->len;
    }
  }
  cudaError_t e;
  {
    LaunchScope scope(ctx, st, logits ? RKV_KERNEL_ATTN_FULL : RKV_KERNEL_ATTN_SMALL);
    // few clusters (half the SMs or fewer): the wide form of the clustered kernel, one CTA per SM
    const bool wide = cluster && (int64_t)gx * ctx->cfg.n_kv_heads * ctx->cfg.n_seq * 2 <= ctx->sm_count;
    e = cluster      ? rkv::launch_attention_cluster(p, tm_k, tm_v, ctx->cfg.n_seq, gx, app != nullptr, wide, st)
        : score_only ? rkv::launch_attention_scores(p, tm_k, tm_v, ctx->cfg.n_seq, gx, st)
                     : rkv::launch_attention(p, tm_k, tm_v, ctx->cfg.n_seq, gx, logits, st, app != nullptr);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "attention launch");
  ctx->launches += 1;
  rkv::note_launch(st, app != nullptr ? cache : nullptr, app != nullptr ? app->full : nullptr);
  return RKV_OK;
}

}  // namespace

namespace rkv {
bool g_use_pdl = true;

namespace {
struct ByteRange { uintptr_t lo, hi; };
std::mutex g_writes_mu;
struct LastLaunch { std::vector<ByteRange> writes; bool fold = false; };
std::map<cudaStream_t, LastLaunch> g_writes;   // per stream: the library's last launch
bool g_writes_lost = false;   // the record was dropped once: a stream without an entry is then unknown, not clean
constexpr size_t kMaxTrackedStreams = 1024;
void add_ranges(std::vector<ByteRange>* v, const rkv_cache* c) {
  if (c == nullptr || c->k == nullptr || c->v == nullptr) return;
  const uintptr_t bytes = (uintptr_t)c->n_rows * kHeadDim * 2;
  v->push_back({reinterpret_cast<uintptr_t>(c->k), reinterpret_cast<uintptr_t>(c->k) + bytes});
  v->push_back({reinterpret_cast<uintptr_t>(c->v), reinterpret_cast<uintptr_t>(c->v) + bytes});
}
}  // namespace

void note_launch(cudaStream_t st, const rkv_cache* a, const rkv_cache* b, bool fold) {
  std::lock_guard<std::mutex> lock(g_writes_mu);
  if (g_writes.size() >= kMaxTrackedStreams && g_writes.find(st) == g_writes.end()) {
    g_writes.clear();
    g_writes_lost = true;
  }
  LastLaunch& v = g_writes[st];
  v.fold = fold;
  v.writes.clear();
  add_ranges(&v.writes, a);
  add_ranges(&v.writes, b);
}

bool last_launch_was_fold(cudaStream_t st) {
  std::lock_guard<std::mutex> lock(g_writes_mu);
  auto it = g_writes.find(st);
  return it != g_writes.end() && it->second.fold;
}

bool early_read_safe(cudaStream_t st, const rkv_cache* c) {
  std::lock_guard<std::mutex> lock(g_writes_mu);
  auto it = g_writes.find(st);
  if (it == g_writes.end()) return !g_writes_lost;   // never launched here: whatever runs before is not ours and
                                                     // therefore complete before a kernel of ours starts
  std::vector<ByteRange> mine;
  add_ranges(&mine, c);
  for (const ByteRange& w : it->second.writes)
    for (const ByteRange& r : mine)
      if (w.lo < r.hi && r.lo < w.hi) return false;
  return true;
}
}  // namespace rkv

extern "C" {

size_t rkv_workspace_bytes(const rkv_config* cfg) {
  rkv_status why;
  if (!config_ok(cfg, &why)) return 0;
  return ws_layout(cfg).total;
}

rkv_status rkv_create(const rkv_config* cfg, rkv_ctx** out) {
  if (out == nullptr) return RKV_ERR_INVALID_ARG;
  *out = nullptr;
  rkv_status why;
  if (!config_ok(cfg, &why)) return why;
  rkv_ctx* ctx = new (std::nothrow) rkv_ctx();
  if (ctx == nullptr) return RKV_ERR_WORKSPACE;
  ctx->cfg = *cfg;
  if (ctx->cfg.softmax_scale == 0.f) ctx->cfg.softmax_scale = 1.0f / sqrtf((float)cfg->head_dim);
  ctx->group = cfg->n_q_heads / cfg->n_kv_heads;
  ctx->max_splits = splits_for(cfg);
  ctx->launches = 0;
  ctx->profiling = false;
  ctx->small_min_chunk = 256;
  ctx->small_cluster = 1;
  ctx->early_read = 1;
  ctx->interleave = 1;
  ctx->select_keys_per_cta = 4096;
  ctx->score_slice = 0;
  ctx->gp = ctx->group <= 4 ? 4 : 8;
  ctx->workspace = nullptr;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e != cudaSuccess) { delete ctx; return RKV_ERR_CUDA; }
  if (ctx->device < 0 || ctx->device >= kMaxDevices) { delete ctx; return RKV_ERR_UNSUPPORTED; }
  {
    std::lock_guard<std::mutex> lock(g_prepare_mu);
    if (!g_prepared[ctx->device]) {
      e = rkv::prepare_attention();
      if (e == cudaSuccess) e = rkv::prepare_select();
      if (e != cudaSuccess) { delete ctx; return RKV_ERR_CUDA; }
      g_prepared[ctx->device] = true;
    }
  }
  const WsLayout w = ws_layout(cfg);
  e = cudaMalloc(reinterpret_cast<void**>(&ctx->workspace), w.total);
  if (e != cudaSuccess) { delete ctx; return RKV_ERR_WORKSPACE; }
  e = cudaMemset(ctx->workspace, 0, w.total);
  if (e != cudaSuccess) { cudaFree(ctx->workspace); delete ctx; return RKV_ERR_CUDA; }
  ctx->workspace_bytes = w.total;
  ctx->partials = reinterpret_cast<float*>(ctx->workspace + w.partials);
  ctx->ml_t = reinterpret_cast<float*>(ctx->workspace + w.ml_t);
  ctx->tickets = reinterpret_cast<int32_t*>(ctx->workspace + w.tickets);
  ctx->len_tickets = reinterpret_cast<int32_t*>(ctx->workspace + w.len_tickets);
  ctx->win_keys = reinterpret_cast<uint32_t*>(ctx->workspace + w.win_keys);
  ctx->keys = reinterpret_cast<uint32_t*>(ctx->workspace + w.keys);
  ctx->hist = reinterpret_cast<uint32_t*>(ctx->workspace + w.hist);   // zeroed with the rest of the workspace above
  ctx->anchor = reinterpret_cast<int32_t*>(ctx->workspace + w.anchor);
  ctx->hist_dirty = false;
  ctx->pending_keys.valid = false;
  ctx->pending_full.valid = false;
  ctx->logits = reinterpret_cast<float*>(ctx->workspace + w.logits);
  ctx->status = reinterpret_cast<int32_t*>(ctx->workspace + w.status);
  ctx->logit_stride = w.logit_stride;
  *out = ctx;
  return RKV_OK;
}

rkv_status rkv_destroy(rkv_ctx* ctx) {
  if (ctx == nullptr) return RKV_ERR_INVALID_ARG;
  cudaError_t e = cudaSuccess;
  if (ctx->workspace) e = cudaFree(ctx->workspace);
  for (auto& t : ctx->timed) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
  for (auto ev : ctx->event_pool) cudaEventDestroy(ev);
  delete ctx;
  return e == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

// First half of the full step: attention over the full cache, logits and softmax statistics to the workspace.
// fold_out: a second kernel finishes out from the partials right away (otherwise the selection kernel does).
static rkv_status full_attention_part(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* active,
                                      void* out, int32_t max_len_hint, cudaStream_t st, bool score_only,
                                      bool fold_out, const AppendArgs* app = nullptr) {
  if (!ctx || !q || !cache_ok(full) || (!out && !score_only)) return RKV_ERR_INVALID_ARG;
  int n_max = max_len_hint == 0 ? ctx->cfg.max_len : max_len_hint;
  if (n_max < 1 || n_max > ctx->cfg.max_len) return RKV_ERR_INVALID_ARG;
  int chunk = 0, gx = 1;
  ctx->pending_full.valid = false;
  ctx->pending_keys.valid = false;   // the logits those keys came from are about to be overwritten
  rkv_status s = run_attention(ctx, q, full, active, out, n_max, n_max, true, st, &chunk, &gx, app, score_only);
  if (s != RKV_OK) return s;
  if (fold_out && !score_only) {
    cudaError_t e;
    {
      LaunchScope scope(ctx, st, RKV_KERNEL_FOLD);
      e = rkv::launch_fold(ctx->partials, ctx->ml_t, full->len, full->cap, active, out, ctx->cfg.n_seq,
                           ctx->cfg.n_q_heads, ctx->cfg.n_kv_heads, chunk, ctx->max_splits, n_max, gx, st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "fold launch");
    ctx->launches += 1;
    rkv::note_launch(st, nullptr, nullptr, true);
  }
  ctx->pending_full = {true, chunk, gx, n_max, full->k, active};
  return RKV_OK;
}

// Second half: scores and top-K from what the first half left in the workspace; folds out unless it is NULL.
// stage: both launches (the score pass, then the selection), or one of them - rkv_score_keys launches the score pass
// alone and leaves a record for the rkv_select_topk that launches the selection alone.
enum SelectStage { kStageBoth, kStageScore, kStageSelect };
static rkv_status select_part(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* k_small,
                              int32_t k_max, const int32_t* active, void* out, float* scores, int64_t score_stride,
                              int32_t* topk_idx, void* q_last_full, cudaStream_t st, SelectStage stage = kStageBoth) {
  if (!ctx || !cache_ok(full) || !k_small || (!topk_idx && stage != kStageScore) ||
      (q_last_full != nullptr && q == nullptr))
    return RKV_ERR_INVALID_ARG;
  if (k_max < 1 || k_max > ctx->cfg.max_small) return RKV_ERR_INVALID_ARG;
  int n_max, chunk, gx;
  if (stage == kStageSelect) {
    if (!ctx->pending_keys.valid || ctx->pending_keys.k_max != k_max) return RKV_ERR_INVALID_ARG;
    n_max = ctx->pending_keys.n_max;
    chunk = gx = 0;                 // (geometry of the attention pass: the score pass has used it)
    ctx->pending_keys.valid = false;
  } else {
    if (!ctx->pending_full.valid) return RKV_ERR_INVALID_ARG;   // no attention pass to take the logits from
    n_max = ctx->pending_full.n_max, chunk = ctx->pending_full.chunk, gx = ctx->pending_full.gx;
    if (scores != nullptr && score_stride < n_max) return RKV_ERR_INVALID_ARG;
    ctx->pending_full.valid = false;
    ctx->pending_keys.valid = false;
  }
  // two launches: the score pass over all positions (keys, scores, histogram; folds out[] when asked to), then
  // the selection proper, one small cluster per (sequence, KV head)
  const int bg = ctx->cfg.n_seq * ctx->cfg.n_kv_heads;
  if (ctx->hist_dirty && stage != kStageSelect) {   // an earlier score pass was never followed by its selection, which clears the histogram
    cudaError_t e0 = cudaMemsetAsync(ctx->hist, 0, (size_t)bg * rkv::kSelectBins * sizeof(uint32_t), st);
    if (e0 != cudaSuccess) return cuda_fail(ctx, e0, "histogram reset");
    ctx->hist_dirty = false;
  }
  ScoreParams cp;
  memset(&cp, 0, sizeof(cp));
  cp.logits = ctx->logits;
  cp.partials = ctx->partials;
  cp.ml_t = ctx->ml_t;
  cp.q = q;
  cp.out = out;
  cp.q_last_full = q_last_full;
  cp.cap = full->cap;
  cp.len = full->len;
  cp.k_small = k_small;
  cp.active = active;
  cp.scores = scores;
  cp.keys = ctx->keys;
  cp.hist = ctx->hist;
  cp.anchor = ctx->anchor;
  cp.status = ctx->status;
  cp.logit_stride = ctx->logit_stride;
  cp.score_stride = score_stride;
  cp.n_q_heads = ctx->cfg.n_q_heads;
  cp.n_kv_heads = ctx->cfg.n_kv_heads;
  cp.group = ctx->group;
  cp.agg = ctx->cfg.agg;
  cp.k_max = k_max;
  cp.max_len = n_max;
  cp.slice = rkv::score_slice_for(n_max, bg, ctx->sm_count);
  if (cp.slice < ctx->score_slice) cp.slice = ctx->score_slice;   // the option is a floor
  cp.n_slices = (n_max + cp.slice - 1) / cp.slice;
  cp.chunk = chunk;
  cp.max_splits = ctx->max_splits;
  cp.grid_splits = gx;
  cp.pool_half = (ctx->cfg.pool_kernel - 1) / 2;
  SelectParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.keys = ctx->keys;
  sp.hist = ctx->hist;
  sp.anchor = ctx->anchor;
  sp.cap = full->cap;
  sp.len = full->len;
  sp.k_small = k_small;
  sp.active = active;
  sp.topk_idx = topk_idx;
  sp.win_keys = ctx->win_keys;
  sp.win_stride = ctx->cfg.max_small;
  sp.logit_stride = ctx->logit_stride;
  sp.n_kv_heads = ctx->cfg.n_kv_heads;
  sp.k_max = k_max;
  sp.max_len = n_max;
  const int cluster = rkv::select_cluster_for(n_max, ctx->select_keys_per_cta);
  sp.keys_per_thread = rkv::select_keys_per_thread(n_max, cluster);
  sp.per_fixed = ctx->cfg.n_seq == 1 ? 1 : 0;
  cudaError_t e;
  if (stage != kStageSelect) {
    ctx->hist_dirty = true;
    {
      LaunchScope scope(ctx, st, RKV_KERNEL_SCORE);
      e = rkv::launch_score(cp, ctx->cfg.n_seq, st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "score launch");
    ctx->launches += 1;
    if (stage == kStageScore) {
      ctx->pending_keys = {true, n_max, k_max, full->k, active};
      rkv::note_launch(st, nullptr, nullptr);
      return RKV_OK;
    }
  }
  {
    LaunchScope scope(ctx, st, RKV_KERNEL_SELECT);
    e = rkv::launch_select(sp, ctx->cfg.n_seq, cluster, st);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "select launch");
  ctx->hist_dirty = false;
  ctx->launches += 1;
  rkv::note_launch(st, nullptr, nullptr);
  return RKV_OK;
}

static rkv_status full_step_impl(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* k_small,
                                 int32_t k_max, const int32_t* active, void* out, float* scores, int64_t score_stride,
                                 int32_t* topk_idx, void* q_last_full, int32_t max_len_hint, void* stream,
                                 bool score_only) {
  // everything the second half would reject is rejected before the first half launches
  if (!ctx || !q || !cache_ok(full) || !k_small || (!out && !score_only) || !topk_idx) return RKV_ERR_INVALID_ARG;
  if (k_max < 1 || k_max > ctx->cfg.max_small) return RKV_ERR_INVALID_ARG;
  const int n_max = max_len_hint == 0 ? ctx->cfg.max_len : max_len_hint;
  if (n_max < 1 || n_max > ctx->cfg.max_len) return RKV_ERR_INVALID_ARG;
  if (scores != nullptr && score_stride < n_max) return RKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rkv_status s = full_attention_part(ctx, q, full, active, out, max_len_hint, st, score_only, false);
  if (s != RKV_OK) return s;
  return select_part(ctx, q, full, k_small, k_max, active, out, scores, score_stride, topk_idx, q_last_full, st);
}

rkv_status rkv_full_step(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* k_small, int32_t k_max,
                         const int32_t* active, void* out, float* scores, int64_t score_stride, int32_t* topk_idx,
                         void* q_last_full, int32_t max_len_hint, void* stream) {
  return full_step_impl(ctx, q, full, k_small, k_max, active, out, scores, score_stride, topk_idx, q_last_full,
                        max_len_hint, stream, false);
}

rkv_status rkv_score_step(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* k_small, int32_t k_max,
                          const int32_t* active, float* scores, int64_t score_stride, int32_t* topk_idx,
                          void* q_last_full, int32_t max_len_hint, void* stream) {
  return full_step_impl(ctx, q, full, k_small, k_max, active, nullptr, scores, score_stride, topk_idx, q_last_full,
                        max_len_hint, stream, true);
}

rkv_status rkv_full_attention(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* active, void* out,
                              int32_t max_len_hint, void* stream) {
  return full_attention_part(ctx, q, full, active, out, max_len_hint, static_cast<cudaStream_t>(stream), false, true);
}

rkv_status rkv_append_full_attention(rkv_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                     const rkv_cache* full, const int32_t* active, void* out, int32_t max_len_hint,
                                     void* stream) {
  if (!k_new || !v_new) return RKV_ERR_INVALID_ARG;
  const AppendArgs app = {k_new, v_new, nullptr, nullptr, nullptr, nullptr, 0};   // one cache: the attended one
  return full_attention_part(ctx, q, full, active, out, max_len_hint, static_cast<cudaStream_t>(stream), false, true,
                             &app);
}

rkv_status rkv_select_topk(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* k_small, int32_t k_max,
                           const int32_t* active, float* scores, int64_t score_stride, int32_t* topk_idx,
                           void* q_last_full, void* stream) {
  if (ctx != nullptr && ctx->pending_keys.valid) {   // rkv_score_keys has run: the selection alone is left
    if (full == nullptr || ctx->pending_keys.full_k != full->k || ctx->pending_keys.active != active ||
        scores != nullptr || q_last_full != nullptr)
      return RKV_ERR_INVALID_ARG;   // (scores and q_last_full are outputs of the score pass)
    return select_part(ctx, q, full, k_small, k_max, active, nullptr, nullptr, 0, topk_idx, nullptr,
                       static_cast<cudaStream_t>(stream), kStageSelect);
  }
  if (ctx != nullptr && ctx->pending_full.valid && full != nullptr &&
      (ctx->pending_full.full_k != full->k || ctx->pending_full.active != active))
    return RKV_ERR_INVALID_ARG;   // not the cache / mask of the attention pass it completes
  return select_part(ctx, q, full, k_small, k_max, active, nullptr, scores, score_stride, topk_idx, q_last_full,
                     static_cast<cudaStream_t>(stream));
}

rkv_status rkv_score_keys(rkv_ctx* ctx, const void* q, const rkv_cache* full, const int32_t* k_small, int32_t k_max,
                          const int32_t* active, float* scores, int64_t score_stride, void* q_last_full,
                          void* stream) {
  if (ctx != nullptr && ctx->pending_full.valid && full != nullptr &&
      (ctx->pending_full.full_k != full->k || ctx->pending_full.active != active))
    return RKV_ERR_INVALID_ARG;   // not the cache / mask of the attention pass it completes
  return select_part(ctx, q, full, k_small, k_max, active, nullptr, scores, score_stride, nullptr, q_last_full,
                     static_cast<cudaStream_t>(stream), kStageScore);
}

rkv_status rkv_gather_small(rkv_ctx* ctx, const int32_t* topk_idx, const int32_t* k_small, int32_t k_max,
                            const rkv_cache* full, const rkv_cache* small_cache, const int32_t* active,
                            void* stream) {
  if (!ctx || !topk_idx || !k_small || !cache_ok(full) || !cache_ok(small_cache)) return RKV_ERR_INVALID_ARG;
  if (k_max < 1 || k_max > ctx->cfg.max_small) return RKV_ERR_INVALID_ARG;
  cudaError_t e;
  {
    LaunchScope scope(ctx, static_cast<cudaStream_t>(stream), RKV_KERNEL_GATHER);
    e = rkv::launch_gather(topk_idx, k_small, k_max, dev_of(full), dev_of(small_cache), active, ctx->cfg.n_seq,
                           ctx->cfg.n_kv_heads, ctx->status, static_cast<cudaStream_t>(stream));
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "gather launch");
  ctx->launches += 1;
  rkv::note_launch(static_cast<cudaStream_t>(stream), small_cache, nullptr);
  return RKV_OK;
}

rkv_status rkv_small_step(rkv_ctx* ctx, const void* q, const rkv_cache* small_cache, const int32_t* active,
                          void* out, int32_t max_len_hint, void* stream) {
  if (!ctx || !q || !cache_ok(small_cache) || !out) return RKV_ERR_INVALID_ARG;
  int n_max = max_len_hint == 0 ? ctx->cfg.max_small : max_len_hint;
  if (n_max < 1 || n_max > ctx->cfg.max_small) return RKV_ERR_INVALID_ARG;
  return run_attention(ctx, q, small_cache, active, out, n_max, n_max, false, static_cast<cudaStream_t>(stream),
                       nullptr, nullptr);
}

rkv_status rkv_append_small_step(rkv_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                 const rkv_cache* full, const rkv_cache* small_cache, const int32_t* active,
                                 void* out, int32_t max_len_hint, void* stream) {
  if (!ctx || !q || !k_new || !v_new || !cache_ok(small_cache) || !out) return RKV_ERR_INVALID_ARG;
  if (full != nullptr && !cache_ok(full)) return RKV_ERR_INVALID_ARG;
  int n_max = max_len_hint == 0 ? ctx->cfg.max_small : max_len_hint;
  if (n_max < 1 || n_max > ctx->cfg.max_small) return RKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cluster_eligible(ctx, n_max)) {   // one launch: the attention kernel appends
    const AppendArgs app = {k_new, v_new, full, nullptr, nullptr, nullptr, 0};
    return run_attention(ctx, q, small_cache, active, out, n_max, n_max, false, st, nullptr, nullptr, &app);
  }
  rkv_status s = rkv_append(ctx, k_new, v_new, full, small_cache, stream);
  if (s != RKV_OK) return s;
  return run_attention(ctx, q, small_cache, active, out, n_max, n_max, false, st, nullptr, nullptr);
}

// Largest small cache whose eviction order one block can sort in shared memory.
constexpr int kEvictMaxK = 4096;

rkv_status rkv_gather_small_evict(rkv_ctx* ctx, const int32_t* topk_idx, const int32_t* k_small, int32_t k_max,
                                  const rkv_cache* full, const rkv_cache* small_cache, const int32_t* active,
                                  int32_t* evict_order, int32_t* evict_count, int32_t max_evict, void* stream) {
  if (!evict_order || !evict_count || max_evict < 1 || max_evict > kEvictMaxK) return RKV_ERR_INVALID_ARG;
  if (k_max > kEvictMaxK) return RKV_ERR_UNSUPPORTED;
  rkv_status s = rkv_gather_small(ctx, topk_idx, k_small, k_max, full, small_cache, active, stream);
  if (s != RKV_OK) return s;
  cudaError_t e;
  {
    LaunchScope scope(ctx, static_cast<cudaStream_t>(stream), RKV_KERNEL_GATHER);
    e = rkv::launch_evict_order(ctx->win_keys, ctx->cfg.max_small, k_small, k_max, full->len, active, evict_order,
                                evict_count, max_evict, ctx->cfg.n_seq, ctx->cfg.n_kv_heads,
                                static_cast<cudaStream_t>(stream));
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "eviction-order launch");
  ctx->launches += 1;
  rkv::note_launch(static_cast<cudaStream_t>(stream), nullptr, nullptr);
  return RKV_OK;
}

rkv_status rkv_append_small_step_evict(rkv_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                       const rkv_cache* full, const rkv_cache* small_cache, const int32_t* k_small,
                                       const int32_t* active, void* out, const int32_t* evict_order,
                                       int32_t* evict_count, int32_t max_evict, int32_t max_len_hint, void* stream) {
  if (!ctx || !q || !k_new || !v_new || !cache_ok(small_cache) || !out || !k_small || !evict_order || !evict_count)
    return RKV_ERR_INVALID_ARG;
  if (full != nullptr && !cache_ok(full)) return RKV_ERR_INVALID_ARG;
  if (max_evict < 1 || max_evict > kEvictMaxK) return RKV_ERR_INVALID_ARG;
  int n_max = max_len_hint == 0 ? ctx->cfg.max_small : max_len_hint;
  if (n_max < 1 || n_max > ctx->cfg.max_small) return RKV_ERR_INVALID_ARG;
  if (!cluster_eligible(ctx, n_max)) return RKV_ERR_UNSUPPORTED;   // the evicting append lives in the clustered kernel
  const AppendArgs app = {k_new, v_new, full, evict_order, evict_count, k_small, max_evict};
  return run_attention(ctx, q, small_cache, active, out, n_max, n_max, false, static_cast<cudaStream_t>(stream), nullptr,
                       nullptr, &app);
}

rkv_status rkv_append(rkv_ctx* ctx, const void* k_new, const void* v_new, const rkv_cache* full,
                      const rkv_cache* small_cache, void* stream) {
  if (!ctx || !k_new || !v_new || (full == nullptr && small_cache == nullptr)) return RKV_ERR_INVALID_ARG;
  if ((full && !cache_ok(full)) || (small_cache && !cache_ok(small_cache))) return RKV_ERR_INVALID_ARG;
  CacheDev none = {nullptr, nullptr, nullptr, nullptr, nullptr};
  cudaError_t e;
  {
    LaunchScope scope(ctx, static_cast<cudaStream_t>(stream), RKV_KERNEL_APPEND);
    e = rkv::launch_append(k_new, v_new, full ? dev_of(full) : none, small_cache ? dev_of(small_cache) : none,
                           full != nullptr, small_cache != nullptr, ctx->cfg.n_seq, ctx->cfg.n_kv_heads, ctx->status,
                           static_cast<cudaStream_t>(stream));
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "append launch");
  ctx->launches += 1;
  rkv::note_launch(static_cast<cudaStream_t>(stream), full, small_cache);
  return RKV_OK;
}

rkv_status rkv_should_refresh(rkv_ctx* ctx, const void* q_now, const void* q_last_full, float threshold,
                              int32_t* flag, int32_t* keep, float* sim, void* stream) {
  if (!ctx || !q_now || !q_last_full || !flag) return RKV_ERR_INVALID_ARG;
  cudaError_t e;
  {
    LaunchScope scope(ctx, static_cast<cudaStream_t>(stream), RKV_KERNEL_TRIGGER);
    e = rkv::launch_trigger(q_now, q_last_full, threshold, flag, keep, sim, ctx->cfg.n_seq, ctx->cfg.n_q_heads,
                            static_cast<cudaStream_t>(stream));
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "trigger launch");
  ctx->launches += 1;
  rkv::note_launch(static_cast<cudaStream_t>(stream), nullptr, nullptr);
  return RKV_OK;
}

rkv_status rkv_get_device_status(rkv_ctx* ctx, int32_t* host_bits, void* stream) {
  if (!ctx || !host_bits) return RKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t bits = 0;
  cudaError_t e = cudaMemcpyAsync(&bits, ctx->status, sizeof(bits), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status, 0, sizeof(int32_t), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "status read");
  *host_bits = bits;
  return bits == 0 ? RKV_OK : RKV_ERR_DEVICE_CHECK;
}

const char* rkv_status_string(rkv_status s) {
  switch (s) {
    case RKV_OK: return "ok";
    case RKV_ERR_INVALID_ARG: return "invalid argument";
    case RKV_ERR_UNSUPPORTED: return "unsupported configuration";
    case RKV_ERR_WORKSPACE: return "workspace allocation failed";
    case RKV_ERR_CUDA: return "CUDA error";
    case RKV_ERR_DEVICE_CHECK: return "device-side check failed";
  }
  return "unknown status";
}

const char* rkv_last_cuda_error(const rkv_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

int64_t rkv_launch_count(const rkv_ctx* ctx) { return ctx ? ctx->launches : 0; }

rkv_status rkv_set_option(rkv_ctx* ctx, int32_t option, int32_t value) {
  if (!ctx) return RKV_ERR_INVALID_ARG;
  switch (option) {
    case RKV_OPT_SMALL_MIN_CHUNK:
      if (value < rkv::kTile || value > (1 << 20)) return RKV_ERR_INVALID_ARG;
      ctx->small_min_chunk = value;
      return RKV_OK;
    case RKV_OPT_SMALL_CLUSTER:
      ctx->small_cluster = value != 0;
      return RKV_OK;
    case RKV_OPT_DEPENDENT_LAUNCH:
      rkv::g_use_pdl = value != 0;
      return RKV_OK;
    case RKV_OPT_EARLY_CACHE_READ:
      ctx->early_read = value != 0;
      return RKV_OK;
    case RKV_OPT_INTERLEAVE_TILES:
      ctx->interleave = value != 0;
      return RKV_OK;
    case RKV_OPT_SELECT_KEYS_PER_CTA:
      if (value < 512 || value > rkv::kSelectMaxKeysPerCta) return RKV_ERR_INVALID_ARG;
      ctx->select_keys_per_cta = value;
      return RKV_OK;
    case RKV_OPT_SCORE_SLICE:
      if (value != 0 && value != 1024 && value != 2048 && value != 4096 && value != rkv::kSelectMaxSlice)
        return RKV_ERR_INVALID_ARG;
      ctx->score_slice = value;
      return RKV_OK;
    default:
      return RKV_ERR_INVALID_ARG;
  }
}

rkv_status rkv_get_option(const rkv_ctx* ctx, int32_t option, int32_t* value) {
  if (!ctx || !value) return RKV_ERR_INVALID_ARG;
  switch (option) {
    case RKV_OPT_SMALL_MIN_CHUNK: *value = ctx->small_min_chunk; return RKV_OK;
    case RKV_OPT_SMALL_CLUSTER: *value = ctx->small_cluster; return RKV_OK;
    case RKV_OPT_DEPENDENT_LAUNCH: *value = rkv::g_use_pdl ? 1 : 0; return RKV_OK;
    case RKV_OPT_EARLY_CACHE_READ: *value = ctx->early_read; return RKV_OK;
    case RKV_OPT_INTERLEAVE_TILES: *value = ctx->interleave; return RKV_OK;
    case RKV_OPT_SELECT_KEYS_PER_CTA: *value = ctx->select_keys_per_cta; return RKV_OK;
    case RKV_OPT_SCORE_SLICE: *value = ctx->score_slice; return RKV_OK;
    default: return RKV_ERR_INVALID_ARG;
  }
}

rkv_status rkv_set_profiling(rkv_ctx* ctx, int32_t on) {
  if (!ctx) return RKV_ERR_INVALID_ARG;
  ctx->profiling = on != 0;
  return RKV_OK;
}

rkv_status rkv_get_profile(rkv_ctx* ctx, double* total_us, int64_t* launches) {
  if (!ctx || !total_us || !launches) return RKV_ERR_INVALID_ARG;
  for (int i = 0; i < RKV_KERNEL_KINDS; ++i) { total_us[i] = 0.0; launches[i] = 0; }
  for (auto& t : ctx->timed) {
    cudaError_t e = cudaEventSynchronize(t.stop);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.start, t.stop);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "profile read");
    total_us[t.kind] += 1000.0 * ms;
    launches[t.kind] += 1;
    ctx->event_pool.push_back(t.start);
    ctx->event_pool.push_back(t.stop);
  }
  ctx->timed.clear();
  return RKV_OK;
}

}  // extern "C"
