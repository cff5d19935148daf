// rkv_small_step_noalloc: the partial step for callers that may not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need attention:
// a serving runtime that hands the whole device heap to its own arena at start-up, a plugin
// that runs inside someone else's memory budget, code on a latency path where an allocation
// (an implicit device synchronisation) is forbidden.  rkv_create allocates a workspace, so those
// callers cannot own a context.  This file gives them the partial step without one: the split
// partials, the arrival tickets and the status word live in a fixed array that is part of the
// library image on every device that loads it.
//
// The array's name is only a host-side handle.  Its device address is looked up once per device
// with cudaGetSymbolAddress (with that device current) and that address is what the kernel gets.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "rkv_internal.h"

namespace {

constexpr int kMaxProblems = RKV_NOALLOC_MAX_PROBLEMS;   // n_seq * n_kv_heads
constexpr int kMaxSplitsNA = RKV_NOALLOC_MAX_SPLITS;     // CTAs that share one (sequence, KV head)
constexpr int kMaxLenNA = RKV_NOALLOC_MAX_LEN;
constexpr size_t kPartialBytes = (size_t)kMaxProblems * kMaxSplitsNA * rkv::PartialLayout::kFloats * sizeof(float);
constexpr size_t kTicketOff = (kPartialBytes + 255) & ~size_t(255);
constexpr size_t kStatusOff = kTicketOff + 256;          // tickets: kMaxProblems int32 <= 256 bytes
constexpr size_t kScratchBytes = kStatusOff + 256;
static_assert(kMaxProblems * sizeof(int32_t) <= 256, "tickets fit their slot");

// Held by every device that loads the library until the process exits (about 2.1 MB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal
bool g_device_ready[kMaxDevices] = {};

rkv::EncodeTiledFn g_encode_na = nullptr;

rkv_status fail(char* err, size_t cap, rkv_status code, const char* fmt, const char* detail = "") {
  if (err != nullptr && cap > 0) snprintf(err, cap, fmt, detail);
  return code;
}

// One-time work for the current device: resolve the array's device address, set the kernels'
// shared-memory attribute, find the tensor-map encoder.  None of it allocates device memory.
rkv_status setup_device(int dev, char* err, size_t cap) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_device_ready[dev]) return RKV_OK;
  void* addr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
  if (e != cudaSuccess || addr == nullptr)
    return fail(err, cap, RKV_ERR_CUDA, "cudaGetSymbolAddress(static scratch) failed: %s", cudaGetErrorString(e));
  e = rkv::prepare_attention();
  if (e != cudaSuccess)
    return fail(err, cap, RKV_ERR_CUDA, "setting the attention kernel's shared-memory size failed: %s",
                cudaGetErrorString(e));
  if (g_encode_na == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || fn == nullptr || q != cudaDriverEntryPointSuccess)
      return fail(err, cap, RKV_ERR_CUDA, "cuTensorMapEncodeTiled is not available: %s", cudaGetErrorString(e));
    g_encode_na = reinterpret_cast<rkv::EncodeTiledFn>(fn);
  }
  g_scratch_addr[dev] = static_cast<unsigned char*>(addr);
  g_device_ready[dev] = true;
  return RKV_OK;
}

bool encode_map(void* base, int64_t n_rows, CUtensorMap* out) {
  return rkv::encode_cache_map(g_encode_na, base, n_rows, out) == CUDA_SUCCESS;
}

}  // namespace

extern "C" rkv_status rkv_small_step_noalloc(const rkv_config* cfg, const void* q, const rkv_cache* small_cache,
                                             const int32_t* active, void* out, int32_t max_len_hint,
                                             int32_t* device_status, void* stream, char* err_msg, size_t err_cap) {
  if (err_msg != nullptr && err_cap > 0) err_msg[0] = '\0';
  if (cfg == nullptr || q == nullptr || small_cache == nullptr || out == nullptr)
    return fail(err_msg, err_cap, RKV_ERR_INVALID_ARG, "cfg, q, small_cache and out must not be NULL");
  if (cfg->n_seq < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads != 0 ||
      cfg->max_small < 1)
    return fail(err_msg, err_cap, RKV_ERR_INVALID_ARG, "bad sizes in rkv_config");
  if (cfg->head_dim != rkv::kHeadDim || cfg->n_q_heads / cfg->n_kv_heads > rkv::kMaxGroup)
    return fail(err_msg, err_cap, RKV_ERR_UNSUPPORTED, "head_dim must be 128 and the group size at most 8");
  if (!(cfg->softmax_scale >= 0.f) || isinf(cfg->softmax_scale))
    return fail(err_msg, err_cap, RKV_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0");
  if ((int64_t)cfg->n_seq * cfg->n_kv_heads > kMaxProblems) {
    if (err_msg != nullptr && err_cap > 0)
      snprintf(err_msg, err_cap, "n_seq * n_kv_heads = %lld exceeds RKV_NOALLOC_MAX_PROBLEMS = %d: the static scratch "
               "holds partials for that many (sequence, KV head) pairs only",
               (long long)cfg->n_seq * cfg->n_kv_heads, kMaxProblems);
    return RKV_ERR_UNSUPPORTED;
  }
  const int n_max = max_len_hint == 0 ? cfg->max_small : max_len_hint;
  if (n_max < 1 || n_max > cfg->max_small)
    return fail(err_msg, err_cap, RKV_ERR_INVALID_ARG, "max_len_hint must lie in 1..cfg.max_small (or be 0)");
  if (n_max > kMaxLenNA) {
    if (err_msg != nullptr && err_cap > 0)
      snprintf(err_msg, err_cap, "small-cache length bound %d exceeds RKV_NOALLOC_MAX_LEN = %d", n_max, kMaxLenNA);
    return RKV_ERR_UNSUPPORTED;
  }
  if ((reinterpret_cast<uintptr_t>(q) & 15) != 0 || (reinterpret_cast<uintptr_t>(out) & 15) != 0)
    return fail(err_msg, err_cap, RKV_ERR_INVALID_ARG, "q and out must start on a 16-byte boundary");
  const rkv_cache* c = small_cache;
  if (!c->k || !c->v || !c->row_offset || !c->cap || !c->len || c->n_rows <= 0 || c->n_rows >= (int64_t(1) << 31) ||
      (reinterpret_cast<uintptr_t>(c->k) & 15) != 0 || (reinterpret_cast<uintptr_t>(c->v) & 15) != 0)
    return fail(err_msg, err_cap, RKV_ERR_INVALID_ARG, "bad rkv_cache (null field, row count, or misaligned base)");

  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(err_msg, err_cap, RKV_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices)
    return fail(err_msg, err_cap, RKV_ERR_UNSUPPORTED, "device ordinal beyond the per-device address table");
  rkv_status s = setup_device(dev, err_msg, err_cap);
  if (s != RKV_OK) return s;
  unsigned char* scratch = g_scratch_addr[dev];

  CUtensorMap tm_k, tm_v;
  if (!encode_map(c->k, c->n_rows, &tm_k) || !encode_map(c->v, c->n_rows, &tm_v))
    return fail(err_msg, err_cap, RKV_ERR_CUDA, "cuTensorMapEncodeTiled failed for the small cache");

  // positions per CTA: at least 256, and few enough CTAs per (sequence, KV head) for the partial slots
  int chunk = (n_max + kMaxSplitsNA - 1) / kMaxSplitsNA;
  if (chunk < 256) chunk = 256;
  chunk = (chunk + 15) & ~15;
  const int grid_x = (n_max + chunk - 1) / chunk;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the last call left: the tickets must start at zero, and so does the
  // built-in status word when the caller supplies none.
  e = cudaMemsetAsync(scratch + kTicketOff, 0, 512, st);
  if (e != cudaSuccess) return fail(err_msg, err_cap, RKV_ERR_CUDA, "clearing the tickets failed: %s", cudaGetErrorString(e));

  rkv::AttnParams p;
  memset(&p, 0, sizeof(p));
  p.q = q;
  p.row_offset = c->row_offset;
  p.cap = c->cap;
  p.len = c->len;
  p.active = active;
  p.out = out;
  p.partials = reinterpret_cast<float*>(scratch);
  p.tickets = reinterpret_cast<int32_t*>(scratch + kTicketOff);
  p.logits = nullptr;
  p.status = device_status != nullptr ? device_status : reinterpret_cast<int32_t*>(scratch + kStatusOff);
  p.logit_stride = 0;
  p.n_q_heads = cfg->n_q_heads;
  p.n_kv_heads = cfg->n_kv_heads;
  p.group = cfg->n_q_heads / cfg->n_kv_heads;
  p.chunk = chunk;
  p.max_splits = kMaxSplitsNA;
  p.max_len = n_max;
  p.scale = cfg->softmax_scale == 0.f ? 1.0f / sqrtf((float)cfg->head_dim) : cfg->softmax_scale;
  e = rkv::launch_attention(p, tm_k, tm_v, cfg->n_seq, grid_x, false, st);
  if (e != cudaSuccess) return fail(err_msg, err_cap, RKV_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(e));
  rkv::note_launch(st, nullptr, nullptr);   // host-side record only: this launch writes no cache rows
  return RKV_OK;
}
