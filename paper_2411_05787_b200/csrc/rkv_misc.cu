// Small kernels of the RefreshKV decode path: small-cache rebuild (gather), cache append,
// and the query-similarity refresh trigger (arXiv 2411.05787, Sec. 2.2).
#include <cuda_bf16.h>

#include "rkv_internal.h"

namespace rkv {
namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* ptr) { return (uint32_t)__cvta_generic_to_shared(ptr); }

// small.K[b][g][r] = full.K[b][g][idx[b][g][r]] (and V).  One CTA of 128 threads per tile of 64 output rows: the
// rows come into shared memory with 16-byte asynchronous copies (no register holds data, so the 32 KB of a tile are
// in flight at once and the CTA fits beside register-heavy kernels), and since the output rows of a tile are
// contiguous they leave with ONE bulk copy per cache.  Indices are requested together with the sizes (every slot
// below k_max is readable), so the kernel costs two memory round trips.
constexpr int kGatherRows = 64;
constexpr int kGatherThreads = 128;

__global__ void __launch_bounds__(kGatherThreads, 16) gather_kernel(const int32_t* __restrict__ topk_idx,
                                                                const int32_t* __restrict__ k_small, int k_max,
                                                                CacheDev full, CacheDev small_cache,
                                                                const int32_t* __restrict__ active, int n_kv_heads,
                                                                int32_t* status) {
  __shared__ __align__(128) uint4 tile_k[kGatherRows * 16];
  __shared__ __align__(128) uint4 tile_v[kGatherRows * 16];
  const int b = blockIdx.z, g = blockIdx.y, tid = threadIdx.x;
  const int sub = tid & 15, slot = tid >> 4;   // thread: 16 bytes of rows slot, slot + 8, ..
  const int r_base = blockIdx.x * kGatherRows;
  constexpr int kPer = kGatherRows / (kGatherThreads / 16);   // rows per thread
  // the caches' geometry is never written by a kernel: read above the dependency wait
  const int cap_s = small_cache.cap[b], cap_f = full.cap[b];
  const int64_t src0 = full.row_offset[b] + (int64_t)g * cap_f;
  const int64_t dst0 = small_cache.row_offset[b] + (int64_t)g * cap_s;
  const int32_t* idx = topk_idx + (int64_t)(b * n_kv_heads + g) * k_max;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)
  const int act = active != nullptr ? __ldcg(active + b) : 1;
  const int n = __ldcg(full.len + b);
  int m = __ldcg(k_small + b);
  int j[kPer];
#pragma unroll
  for (int u = 0; u < kPer; ++u) {
    const int r = r_base + slot + u * (kGatherThreads / 16);
    j[u] = r < k_max ? __ldcg(idx + r) : -1;
  }
  if (act == 0) return;
  if (m > k_max) m = k_max;
  if (m > n) m = n;
  if (m < 0) m = 0;
  if (m > cap_s) {
    m = cap_s;
    if (tid == 0 && blockIdx.x == 0) atomicOr(status, RKV_DEV_LEN_CLAMPED);
  }
  if (blockIdx.x == 0 && g == 0 && tid == 0) small_cache.len[b] = m;
  if (r_base >= m) return;
  const uint4* fk = static_cast<const uint4*>(full.k);
  const uint4* fv = static_cast<const uint4*>(full.v);
  int ok = 1;
#pragma unroll
  for (int u = 0; u < kPer; ++u) {
    const int rl = slot + u * (kGatherThreads / 16);
    if (r_base + rl >= m) {
      j[u] = -1;                                   // beyond the rows to rebuild: not part of the tile
      continue;
    }
    if (j[u] >= n || j[u] < -1) {                  // -1 is the padding of topk_idx; anything else outside [0, len) is flagged
      if (sub == 0) atomicOr(status, RKV_DEV_BAD_INDEX);
      j[u] = -1;
    }
    if (j[u] < 0) {
      ok = 0;                                      // a row of the tile stays as it is: no bulk store for this tile
      continue;
    }
    const uint32_t dk = smem_u32(&tile_k[rl * 16 + sub]), dv = smem_u32(&tile_v[rl * 16 + sub]);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dk), "l"(fk + (src0 + j[u]) * 16 + sub) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dv), "l"(fv + (src0 + j[u]) * 16 + sub) : "memory");
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy below reads what the copies above wrote
  const int all_ok = __syncthreads_and(ok);
  uint4* sk = static_cast<uint4*>(small_cache.k) + (dst0 + r_base) * 16;
  uint4* sv = static_cast<uint4*>(small_cache.v) + (dst0 + r_base) * 16;
  if (all_ok) {
    if (tid == 0) {
      const int rows = m - r_base < kGatherRows ? m - r_base : kGatherRows;
      const uint32_t bytes = (uint32_t)rows * 256u;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(sk), "r"(smem_u32(tile_k)), "r"(bytes)
                   : "memory");
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(sv), "r"(smem_u32(tile_v)), "r"(bytes)
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    return;
  }
  // a tile with skipped rows (bad or padding indices): row by row
#pragma unroll
  for (int u = 0; u < kPer; ++u) {
    const int rl = slot + u * (kGatherThreads / 16);
    if (j[u] >= 0) {
      sk[rl * 16 + sub] = tile_k[rl * 16 + sub];
      sv[rl * 16 + sub] = tile_v[rl * 16 + sub];
    }
  }
}

// One block per sequence; thread t moves 16 bytes of one head's new K row and V row.  Every load is
// issued before the first dependent use, so the kernel costs one memory round trip.
__global__ void __launch_bounds__(128) append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                                     CacheDev full, CacheDev small_cache, int has_full,
                                                     int has_small, int n_kv_heads, int32_t* status) {
  const int b = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)
  int pos_f = -1, cap_f = 0, pos_s = -1, cap_s = 0;
  int64_t off_f = 0, off_s = 0;
  if (has_full) {
    pos_f = full.len[b];
    cap_f = full.cap[b];
    off_f = full.row_offset[b];
  }
  if (has_small) {
    pos_s = small_cache.len[b];
    cap_s = small_cache.cap[b];
    off_s = small_cache.row_offset[b];
  }
  const bool ok_f = has_full && pos_f >= 0 && pos_f < cap_f;
  const bool ok_s = has_small && pos_s >= 0 && pos_s < cap_s;
  for (int i = tid; i < n_kv_heads * 16; i += blockDim.x) {
    const int g = i >> 4, sub = i & 15;
    const uint4 kv = k_new[((int64_t)b * n_kv_heads + g) * 16 + sub];
    const uint4 vv = v_new[((int64_t)b * n_kv_heads + g) * 16 + sub];
    if (ok_f) {
      const int64_t row = off_f + (int64_t)g * cap_f + pos_f;
      static_cast<uint4*>(full.k)[row * 16 + sub] = kv;
      static_cast<uint4*>(full.v)[row * 16 + sub] = vv;
    }
    if (ok_s) {
      const int64_t row = off_s + (int64_t)g * cap_s + pos_s;
      static_cast<uint4*>(small_cache.k)[row * 16 + sub] = kv;
      static_cast<uint4*>(small_cache.v)[row * 16 + sub] = vv;
    }
  }
  __syncthreads();   // every thread has read the old lengths
  if (tid == 0) {
    if (ok_f) full.len[b] = pos_f + 1;
    if (ok_s) small_cache.len[b] = pos_s + 1;
    if ((has_full && !ok_f) || (has_small && !ok_s)) atomicOr(status, RKV_DEV_APPEND_OVERFLOW);
  }
}

// one block of 128 threads per sequence: thread d owns channel d of the head-averaged queries
__global__ void __launch_bounds__(128) trigger_kernel(const __nv_bfloat16* __restrict__ q_now,
                                                      const __nv_bfloat16* __restrict__ q_last, float threshold,
                                                      int32_t* flag, int32_t* keep, float* sim, int n_q_heads) {
  const int b = blockIdx.x, d = threadIdx.x;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)
  float a = 0.f, c = 0.f;
  for (int h = 0; h < n_q_heads; ++h) {
    a += __bfloat162float(q_now[((int64_t)b * n_q_heads + h) * kHeadDim + d]);
    c += __bfloat162float(q_last[((int64_t)b * n_q_heads + h) * kHeadDim + d]);
  }
  const float inv = 1.f / (float)n_q_heads;
  a *= inv;
  c *= inv;
  float dot = a * c, na = a * a, nc = c * c;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    dot += __shfl_xor_sync(0xffffffffu, dot, o);
    na += __shfl_xor_sync(0xffffffffu, na, o);
    nc += __shfl_xor_sync(0xffffffffu, nc, o);
  }
  __shared__ float red[3][4];
  if ((d & 31) == 0) {
    red[0][d >> 5] = dot;
    red[1][d >> 5] = na;
    red[2][d >> 5] = nc;
  }
  __syncthreads();
  if (d == 0) {
    const float dt = (red[0][0] + red[0][1]) + (red[0][2] + red[0][3]);
    const float n1 = (red[1][0] + red[1][1]) + (red[1][2] + red[1][3]);
    const float n2 = (red[2][0] + red[2][1]) + (red[2][2] + red[2][3]);
    const float cs = dt / (sqrtf(n1) * sqrtf(n2));  // 0/0 -> NaN -> not "higher" -> refresh
    const int refresh = (cs > threshold) ? 0 : 1;
    flag[b] = refresh;
    if (keep != nullptr) keep[b] = 1 - refresh;
    if (sim != nullptr) sim[b] = cs;
  }
}

// Attention output of the full step from the split partials its streaming pass left in the workspace (the
// flash-decoding merge: M = max_s m_s, w_s = exp(m_s - M), out = sum_s w_s O_s / sum_s w_s l_s).  A kernel of its
// own, for rkv_full_attention: hundreds of small blocks finish in about one memory round trip, where the last
// CTA of the streaming pass would need several microseconds of dependent round trips on an otherwise idle GPU.
// One block per (sequence, KV head, head of the group, quarter of the channels); warp w takes the splits
// s = w (mod 4), lane c the channel; every load is issued before the first is used.
__global__ void __launch_bounds__(128) fold_kernel(const float* __restrict__ partials, const float* __restrict__ ml_t,
                                                   const int32_t* __restrict__ len, const int32_t* __restrict__ cap,
                                                   const int32_t* __restrict__ active, __nv_bfloat16* __restrict__ out,
                                                   int n_q_heads, int n_kv_heads, int group, int chunk, int max_splits,
                                                   int max_len, int grid_splits) {
  constexpr int kU = 10;  // splits per warp in the first batch of loads (4 * kU = 40 splits: one batch at batch 1, L = 32K)
  constexpr float kLog2e = 1.4426950408889634f;
  const int h = blockIdx.x >> 2, c = (blockIdx.x & 3) * 32 + (threadIdx.x & 31);
  const int g = blockIdx.y, b = blockIdx.z, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float sm_e[kMaxSplits];
  __shared__ float sm_red[4][32];
  __shared__ float sm_L;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)
  // One round trip: the sizes and every slot a CTA of the pass can have written (grid_splits of them; slots the
  // current length does not reach hold older partials and are left out below, once the length is known).
  const int act = active != nullptr ? __ldcg(active + b) : 1;
  int n = __ldcg(len + b);
  const int cp = __ldg(cap + b), lim = cp < max_len ? cp : max_len;
  const int64_t bg = (int64_t)b * n_kv_heads + g;
  const float* po = partials + bg * max_splits * PartialLayout::kFloats + h * kHeadDim + c;
  float v[kU];
#pragma unroll
  for (int k = 0; k < kU; ++k) {
    const int s = warp + 4 * k;
    v[k] = s < grid_splits ? __ldcg(po + (int64_t)s * PartialLayout::kFloats) : 0.f;
  }
  float m[4], l[4];
  if (warp == 0) {   // (m, l) of all splits (at most kMaxSplits = 4 per lane)
    const float* pm = ml_t + bg * 16 * max_splits + (int64_t)h * max_splits;
    const float* pl = pm + (int64_t)kMaxGroup * max_splits;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int s = lane + 32 * i;
      m[i] = s < grid_splits ? __ldcg(pm + s) : -INFINITY;
      l[i] = s < grid_splits ? __ldcg(pl + s) : 0.f;
    }
  }
  if (act == 0) return;
  n = n < lim ? n : lim;            // the clamp of the streaming pass
  if (n <= 0) return;               // nothing cached: the streaming pass has written zeros
  int n_splits = (n + chunk - 1) / chunk;
  if (n_splits > grid_splits) n_splits = grid_splits;   // (interleaved tiles: every CTA of the pass carries some)
  if (warp == 0) {   // weights of the splits in use, their sum of denominators
    float M = -INFINITY, L = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (lane + 32 * i >= n_splits) {
        m[i] = -INFINITY;
        l[i] = 0.f;
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) M = fmaxf(M, m[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float e = (m[i] == -INFINITY) ? 0.f : exp2f((m[i] - M) * kLog2e);
      L = fmaf(l[i], e, L);
      sm_e[lane + 32 * i] = e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    if (lane == 0) sm_L = L;
  }
  __syncthreads();
  float acc = 0.f;
#pragma unroll
  for (int k = 0; k < kU; ++k) {
    const int s = warp + 4 * k;
    if (s < n_splits) acc = fmaf(v[k], sm_e[s], acc);
  }
  for (int s = warp + 4 * kU; s < n_splits; s += 4) acc = fmaf(__ldcg(po + (int64_t)s * PartialLayout::kFloats), sm_e[s], acc);
  sm_red[warp][lane] = acc;
  __syncthreads();
  if (warp == 0) {
    const float sum = (sm_red[0][lane] + sm_red[1][lane]) + (sm_red[2][lane] + sm_red[3][lane]);
    out[((int64_t)b * n_q_heads + (int64_t)g * group + h) * kHeadDim + c] = __float2bfloat16(sum / sm_L);
  }
}

// Eviction order of a freshly rebuilt small cache (Sec. 2.2 "Decoding with partial cache": to keep C_p at a fixed
// size, the entry with the lowest attention score of the last full step is dropped for each new token).  One block
// per (sequence, KV head): bitonic sort of (key, slot) pairs, largest key = lowest score first, the higher slot
// (= later position) first among equal keys; the first max_evict slots are written out.
constexpr int kEvictMaxK = 4096;
__global__ void __launch_bounds__(1024) evict_order_kernel(const uint32_t* __restrict__ win_keys, int win_stride,
                                                           const int32_t* __restrict__ k_small, int k_max,
                                                           const int32_t* __restrict__ full_len,
                                                           const int32_t* __restrict__ active, int32_t* evict_order,
                                                           int32_t* evict_count, int max_evict, int n_kv_heads) {
  __shared__ unsigned long long sk[kEvictMaxK];
  const int b = blockIdx.y, g = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)
  if (active != nullptr && active[b] == 0) return;
  int m = k_small[b];
  const int n = full_len[b];
  if (m > k_max) m = k_max;
  if (m > n) m = n;
  if (m < 0) m = 0;
  int np2 = 1;
  while (np2 < m) np2 <<= 1;
  const uint32_t* wk = win_keys + (int64_t)(b * n_kv_heads + g) * win_stride;
  for (int i = tid; i < np2; i += blockDim.x)
    sk[i] = i < m ? (((unsigned long long)wk[i] << 32) | (unsigned)i) : 0ull;   // padding sorts last
  __syncthreads();
  for (int k2 = 2; k2 <= np2; k2 <<= 1) {
    for (int j = k2 >> 1; j > 0; j >>= 1) {
      for (int i = tid; i < np2; i += blockDim.x) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const unsigned long long a = sk[i], c = sk[ixj];
          const bool desc = (i & k2) == 0;          // descending overall
          if (desc ? (a < c) : (a > c)) {
            sk[i] = c;
            sk[ixj] = a;
          }
        }
      }
      __syncthreads();
    }
  }
  int32_t* eo = evict_order + (int64_t)(b * n_kv_heads + g) * max_evict;
  for (int i = tid; i < max_evict; i += blockDim.x) eo[i] = i < m ? (int32_t)(sk[i] & 0xffffffffull) : -1;
  if (g == 0 && tid == 0) evict_count[b] = 0;
}

}  // namespace

cudaError_t launch_evict_order(const uint32_t* win_keys, int win_stride, const int32_t* k_small, int k_max,
                               const int32_t* full_len, const int32_t* active, int32_t* evict_order,
                               int32_t* evict_count, int max_evict, int n_seq, int n_kv_heads, cudaStream_t st) {
  return launch_ex(evict_order_kernel, dim3(n_kv_heads, n_seq), dim3(1024), 0, st, 1, win_keys, win_stride, k_small,
                   k_max, full_len, active, evict_order, evict_count, max_evict, n_kv_heads);
}

cudaError_t launch_gather(const int32_t* topk_idx, const int32_t* k_small, int k_max, CacheDev full,
                          CacheDev small_cache, const int32_t* active, int n_seq, int n_kv_heads,
                          int32_t* status, cudaStream_t st) {
  const int gx = (k_max + kGatherRows - 1) / kGatherRows;   // one CTA per tile of output rows
  dim3 grid(gx < 1 ? 1 : gx, n_kv_heads, n_seq);
  return launch_ex(gather_kernel, grid, dim3(kGatherThreads), 0, st, 1, topk_idx, k_small, k_max, full, small_cache, active,
                   n_kv_heads, status);
}

cudaError_t launch_append(const void* k_new, const void* v_new, CacheDev full, CacheDev small_cache,
                          bool has_full, bool has_small, int n_seq, int n_kv_heads, int32_t* status,
                          cudaStream_t st) {
  return launch_ex(append_kernel, dim3(n_seq), dim3(128), 0, st, 1, static_cast<const uint4*>(k_new),
                   static_cast<const uint4*>(v_new), full, small_cache, has_full ? 1 : 0, has_small ? 1 : 0,
                   n_kv_heads, status);
}

cudaError_t launch_fold(const float* partials, const float* ml_t, const int32_t* len, const int32_t* cap,
                        const int32_t* active, void* out, int n_seq, int n_q_heads, int n_kv_heads, int chunk,
                        int max_splits, int max_len, int grid_splits, cudaStream_t st) {
  const int group = n_q_heads / n_kv_heads;
  return launch_ex(fold_kernel, dim3(4 * group, n_kv_heads, n_seq), dim3(128), 0, st, 1, partials, ml_t, len, cap,
                   active, static_cast<__nv_bfloat16*>(out), n_q_heads, n_kv_heads, group, chunk, max_splits, max_len,
                   grid_splits);
}

cudaError_t launch_trigger(const void* q_now, const void* q_last, float threshold, int32_t* flag, int32_t* keep,
                           float* sim, int n_seq, int n_q_heads, cudaStream_t st) {
  return launch_ex(trigger_kernel, dim3(n_seq), dim3(128), 0, st, 1, static_cast<const __nv_bfloat16*>(q_now),
                   static_cast<const __nv_bfloat16*>(q_last), threshold, flag, keep, sim, n_q_heads);
}

}  // namespace rkv
