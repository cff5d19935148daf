// Split-K grouped-query decode attention over a packed bf16 KV cache (sm_100a).
//
// What it computes (RefreshKV, arXiv 2411.05787, Sec. 2.2 "Decoding with full
// cache" / "Decoding with partial cache"): for one query token per sequence,
//   s[h][j] = scale <q[h], K[g][j]>,  p = softmax_j s,  out[h] = sum_j p[h][j] V[g][j],
// g = h / G.  The full step additionally needs the attention scores a_L of the
// current token (App. A.1: the paper recomputes them in a second pass because
// its library attention hides them); here the scaled logits are written out by
// the same pass that streams K, so the cache is read from HBM exactly once.
//
// Shape of the kernel: one CTA per (sequence, KV head, chunk of positions).
// A copy warp streams 64-position tiles of K and V into a shared-memory ring (3 stages,
// 5 in the wide form of the clustered partial step) with tensor-map TMA loads, one per K or
// V tile (128-byte swizzle, completion on mbarriers).  The MMA warps own bands of a tile
// (16 positions; 32 in the wide form): S^T = K Q^T and O^T += V^T P^T with m16n8k16 bf16
// tensor-core MMAs (fp32 accumulate), where the N=8 dimension holds all query heads of the
// group, so K/V are read once per group.  Online softmax lives in registers; the warps of a
// CTA merge by a sum of accumulators pre-scaled to the CTA-wide maximum.  Three ways to
// merge the splits:
//   full step      partials go to the workspace; the selection kernel folds them, or - for
//                  rkv_full_attention - a small fold kernel right behind this one (the
//                  score-only variant streams K alone: logits and softmax statistics);
//   partial step   (a) the CTAs of one (sequence, KV head) form a thread-block cluster:
//                  each pushes its slice of the partial output into the peer that owns
//                  that slice through distributed shared memory, with stores that credit
//                  an mbarrier of the receiver (no cluster barrier behind the dependency
//                  wait); each CTA finishes 128/C channels of every head;
//                  (b) long small caches: partials to the workspace, folded by the last
//                  CTA of each (sequence, KV head) to arrive (atomic ticket, no spin).
// The clustered partial step and the full step's pass can take the append with them
// (Sec. 2.2: the input token's K/V is stored in C_p, and C_f receives it too): the new rows
// are written to the cache(s), patched into the shared-memory tile that covers the new
// position, and the lengths are bumped by the last ticket holder of a sequence.
// The clustered partial step may also request its tiles before its stream dependency has
// resolved (AttnParams::early): see the comment at the dependency wait.
#include <cuda_bf16.h>

#include "rkv_fold.cuh"
#include "rkv_internal.h"

namespace rkv {
namespace {

constexpr int kStageBytes = 4 * kTile * 128;  // K lo/hi + V lo/hi halves, 64 rows x 128 B each
constexpr int kHalfBytes = kTile * 128;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kOPad = 132;  // floats per head row in the merge buffer (bank spread)
constexpr int kQPad = 68;   // 32-bit words per query row in shared memory (64 + 4: the fragment reads spread over all banks)
constexpr int kRecvFloats = kMaxGroup * kHeadDim + kAttnCluster * kMaxGroup * 2;   // pushed slices + (m, l) pairs

enum : int { kModeFull = 0, kModeTicket = 1, kModeCluster = 2, kModeClusterAppend = 3, kModeScore = 4,
              kModeFullAppend = 5 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls so that a lost copy can never hang the GPU.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// One K (or V) tile: the box {64 channels, 64 rows, 2 halves} at row y.
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* tm, int y, uint32_t bar,
                                              uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
      "l"(tm), "r"(0), "r"(y), "r"(0), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
template <int kThreadsN>
__device__ __forceinline__ void consumer_bar_n() {   // barrier among the MMA warps only (the copy warp is elsewhere)
  asm volatile("bar.sync 1, %0;" ::"n"(kThreadsN) : "memory");
}
__device__ __forceinline__ uint32_t map_rank(uint32_t local_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_shared_v2(uint32_t addr, uint2 v) {
  asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(v.x), "r"(v.y) : "memory");
}
// Store that asks L2 to keep the line (the selection kernel reads the logits right after this kernel, while
// 134 MB of K/V stream through the same cache with evict-first priority).
__device__ __forceinline__ void st_keep_f2(float* addr, float a, float b, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1, %2}, %3;" ::"l"(addr), "f"(a), "f"(b), "l"(policy) : "memory");
}
// Store into a peer CTA's shared memory that also credits the bytes to an mbarrier of that peer: data and the
// "it has arrived" signal travel together, one way.
__device__ __forceinline__ void st_async_f32x4(uint32_t addr, float4 v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(remote_bar)
               : "memory");
}
__device__ __forceinline__ void st_async_f32x2(uint32_t addr, float a, float b, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(addr),
               "f"(a), "f"(b), "r"(remote_bar)
               : "memory");
}
__device__ __forceinline__ void cluster_sync_alive() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Stage ring: normally two CTAs per SM with three 32 KiB stages each.  The clustered partial step with few
// clusters (batch 1) is a pure latency chain on half-empty SMs: its "wide" form takes the whole SM, keeps five
// tiles in flight and splits the tiles over five pairs of MMA warps.  With many clusters the narrow form wins
// (two CTAs per SM place clusters more freely and overlap each other's latencies).
template <int kMode, bool kWideT>
struct Ring {
  static constexpr bool kWide = kWideT && (kMode == kModeCluster || kMode == kModeClusterAppend);
  // (stages = groups of MMA warps in the wide form: tile t and the tile t + kStg that reuses its stage must
  // belong to the same group, because a warp may only wait for a stage's second phase after it has seen the
  // first - a parity wait on a phase the warp has skipped returns at once)
  static constexpr int kStg = kWide ? 5 : kStages;
  static constexpr int kMinBlocks = kWide ? 1 : 2;
  // The clustered partial step is bound by the length of one warp's MMA / softmax instruction chain, not by
  // bandwidth: five pairs of MMA warps take alternate tiles, so that a chunk of up to five tiles (a small
  // cache of 2048 rows plus the rows appended since, over eight CTAs) is one pass for every warp.
  static constexpr int kMmaWarps = kWide ? 10 : 4;
  static constexpr int kThreads = 32 * (kMmaWarps + 1);
};

template <int kMode, bool kWideT = false>
__global__ void __launch_bounds__(Ring<kMode, kWideT>::kThreads, Ring<kMode, kWideT>::kMinBlocks)
attn_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
            const AttnParams p) {
  constexpr bool kLogits = (kMode == kModeFull || kMode == kModeScore || kMode == kModeFullAppend);
  constexpr bool kScoreOnly = (kMode == kModeScore);   // logits and softmax statistics only: V is never read
  constexpr bool kCluster = (kMode == kModeCluster || kMode == kModeClusterAppend);
  constexpr bool kAppend = (kMode == kModeClusterAppend || kMode == kModeFullAppend);
  constexpr int kStg = Ring<kMode, kWideT>::kStg;
  constexpr int kMW = Ring<kMode, kWideT>::kMmaWarps;      // MMA warps; warp kMW is the copy warp
  // Rows of a tile per MMA warp.  The bandwidth-bound forms use 16 (four warps per tile).  The clustered
  // partial step is bound by the length of one warp's instruction chain: there a warp takes 32 rows, two
  // independent 16-row blocks that share one softmax update, and two warps cover a tile.
  constexpr int kNB = Ring<kMode, kWideT>::kWide ? 2 : 1;   // 16-row blocks per warp
  constexpr int kBand = 16 * kNB;
  constexpr int kWT = kTile / kBand;                // warps per tile
  constexpr int kGroups = kMW / kWT;                // groups of warps that take alternate tiles
  static_assert(kStg % kGroups == 0, "a stage must always be consumed by the same group of warps");
  auto consumer_bar = [] { consumer_bar_n<32 * kMW>(); };
  extern __shared__ uint8_t smem_raw[];
  __shared__ int s_last;

  const int b = blockIdx.z, g = blockIdx.y, split = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // shared memory: [stages][K lo | K hi | V lo | V hi], the barriers, then (cluster mode) the receive buffer
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_full = smem_base + kStg * kStageBytes;
  const uint32_t bar_empty = bar_full + 8 * kStg;
  const uint32_t bar_recv = bar_empty + 8 * kStg;   // cluster mode: completes when every peer's slice has arrived
  if (tid == 0) {
    for (int s = 0; s < kStg; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, kWT);   // one arrival per MMA warp that reads the tile
    }
    if (kCluster) mbar_init(bar_recv, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid == 32 * kMW) {
    prefetch_tensormap(&tm_k);
    prefetch_tensormap(&tm_v);
  }
  const int G = p.group;
  const int64_t head0 = ((int64_t)b * p.n_q_heads + (int64_t)g * G) * kHeadDim;
  __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out) + head0;
  const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + head0;
  const int qd = lane >> 2;       // row inside an 8-row group
  const int qc = (lane & 3) * 2;  // first of the two columns this lane holds
  // The geometry of the cache (capacity, first row) is never written by any kernel, so it may be read while the
  // stream predecessor is still running; everything else waits for the dependency.
  const int cap = __ldg(p.cap + b);
  const int64_t roff = __ldg(p.row_offset + b);
  __syncthreads();   // barrier initialisation (above) is visible to every warp
  if (kCluster) {
    // The receive barrier expects, from every CTA of the cluster, its slice of the partial outputs (G heads x
    // 128 / C channels) and its (m, l) of all eight head slots.  It is armed before the one cluster-wide barrier
    // of the kernel, which sits up here, above the dependency wait, where it costs nothing: behind it every
    // peer's receive barrier exists, and the merge needs no further barrier - the pushes carry their own signal.
    if (gridDim.x > 1) {
      if (tid == 0) mbar_expect_tx(bar_recv, (uint32_t)(p.group * kHeadDim * 4 + (int)gridDim.x * kMaxGroup * 8));
      cluster_sync_alive();
    }
  }

  // Which positions a CTA's t-th tile covers.  Contiguous: the CTA owns the chunk [split * chunk, (split + 1) * chunk).
  // Interleaved (streaming forms, AttnParams::interleave): the tiles of a (sequence, KV head) are dealt out to its
  // CTAs in turn - tile j goes to CTA j mod gridDim.x - so that every CTA walks the whole length, all CTAs carry the
  // same number of tiles up to one, and which CTA sums which positions stays fixed by the launch geometry alone.
  const bool il = kLogits && p.interleave != 0;
  auto tile_pos = [&](int t) { return il ? (split + t * (int)gridDim.x) * kTile : split * p.chunk + t * kTile; };
  // One tile = K (and V) rows [y, y + 64) into stage t % kStg, completion on that stage's barrier.
  auto issue_tile = [&](int t, int64_t row_first, uint64_t policy) {
    const int s = t % kStg;
    const uint32_t dst = smem_base + s * kStageBytes, bar = bar_full + 8 * s;
    const int y = (int)(row_first + (int64_t)tile_pos(t));
    mbar_expect_tx(bar, kScoreOnly ? 2 * kHalfBytes : kStageBytes);
    tma_load_tile(dst, &tm_k, y, bar, policy);
    if (!kScoreOnly) tma_load_tile(dst + 2 * kHalfBytes, &tm_v, y, bar, policy);
  };
  // Tiles requested ahead of the length (see below).  When the host has established that the launch before
  // this one on the stream does not write this cache (p.early), they are requested even before the
  // dependency wait: a clustered step usually sits at that wait while its predecessor runs, and a CTA's
  // share of the cache takes longer to arrive (about 64 bytes per cycle per SM) than the rest of the step
  // takes to get ready; the streaming pass gains the latency of its first tiles (p.early says how many: a
  // predecessor with memory traffic of its own is slowed by what is queued in front of it).  Every kernel of
  // this library releases its dependents only after its own wait, so the predecessor is the only kernel that
  // can still be running at that point.
  auto issue_spec = [&](int t_first, int t_end) {
    if (tid == 32 * kMW) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      const int64_t row_s = roff + (int64_t)g * cap;
      for (int t = t_first; t < t_end; ++t) issue_tile(t, row_s, policy);
    }
  };
  int n_spec = 0;
  if (p.spec != 0) n_spec = (!il && (p.chunk + kTile - 1) / kTile < kStg) ? (p.chunk + kTile - 1) / kTile : kStg;
  // tiles requested above the dependency wait: all of them in the clustered step, p.early of them in the streaming forms
  int n_early = 0;
  if (kCluster) {
    if (p.early != 0) issue_spec(0, n_spec);
  } else if (kLogits && p.early != 0) {
    n_early = p.early < n_spec ? p.early : n_spec;
    issue_spec(0, n_early);
  }
  // The output accumulators are cleared up here (and pinned to registers), not on the path between the query's
  // arrival and the first product, where every instruction of a warp is paid for in full.
  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    asm volatile("" : "+f"(o[i][0]), "+f"(o[i][1]), "+f"(o[i][2]), "+f"(o[i][3]));
  }
  pdl_wait();
  pdl_launch();   // after the wait: at most one predecessor is ever in flight behind a kernel of this library
  if (kCluster) {
    if (p.early == 0) issue_spec(0, n_spec);
  } else {
    issue_spec(n_early, n_spec);
  }

  // (When the host knows that every CTA of the grid has work - no mask; one sequence, or a cluster per head - the
  // chunk of this CTA follows from the launch geometry alone, so its first tiles have been requested above, before
  // the length has even been read; tiles past the length are waited for and ignored.)

  // per-sequence sizes and (MMA warps) the query fragments: independent loads, one round trip
  const int act = (p.active != nullptr) ? __ldcg(p.active + b) : 1;
  int n = __ldcg(p.len + b);
  // The G query rows go through shared memory: G * 16 coalesced 16-byte loads for the whole CTA instead of
  // sixteen 4-byte loads per lane (the memory pipe's request rate, not its latency, is what those cost).
  uint32_t* sm_q = reinterpret_cast<uint32_t*>(smem_gen + kStg * kStageBytes + 16 * kStg + 16 + kRecvFloats * 4);
  const bool q_lane = warp < kMW && tid < G * 16;
  const bool q_row = warp < kMW && tid < kMaxGroup * 16;   // rows of heads beyond the group are stored as zeros
  uint4 qv = make_uint4(0u, 0u, 0u, 0u);
  if (q_lane) qv = __ldcg(reinterpret_cast<const uint4*>(qg) + tid);
  // fused append: this lane's 8 bytes of the new K and V rows, and the second cache's sizes
  uint2 kn = make_uint2(0u, 0u), vn = make_uint2(0u, 0u);
  int pos_new = -1;            // where the new row lands in the attended cache (-1: no room, or no append)
  int new_len_s = -1, new_len_f = -1;
  bool bump_evict = false;
  if (kAppend) {
    int len_f = 0, cap_f = 0;
    int64_t roff_f = 0;
    if (p.has_full) {
      len_f = __ldcg(p.full_len + b);
      cap_f = __ldcg(p.full_cap + b);
      roff_f = __ldcg(p.full_row_offset + b);
    }
    if (warp < kMW) {
      const int64_t nrow = ((int64_t)b * p.n_kv_heads + g) * 32;   // uint2 units: 256 bytes per row
      kn = __ldcg(static_cast<const uint2*>(p.k_new) + nrow + lane);
      vn = __ldcg(static_cast<const uint2*>(p.v_new) + nrow + lane);
    }
    // (the query's store to shared memory waits for its load; it comes after every other load has been issued)
    if (q_row) *reinterpret_cast<uint4*>(sm_q + (tid >> 4) * kQPad + (tid & 15) * 4) = qv;
    // Where the new row goes in the attended cache: behind the last row (the cache grows), or - fixed-size small
    // cache that has reached its size - into the slot of the lowest-scoring survivor of the last refresh.
    int slot = n;
    bool evicting = false, ok_s = n >= 0 && n < cap;
    if (p.evict_order != nullptr) {
      const int kk = __ldcg(p.k_small + b);
      if (kk > 0 && n >= kk) {
        evicting = true;
        const int t = __ldcg(p.evict_count + b);
        slot = (t >= 0 && t < p.max_evict)
                   ? __ldcg(p.evict_order + ((int64_t)b * p.n_kv_heads + g) * p.max_evict + t) : -1;
        ok_s = slot >= 0 && slot < n && slot < cap;     // out of eviction slots: flagged like a full cache
      }
    }
    const bool ok_f = p.has_full && len_f >= 0 && len_f < cap_f;
    if (split == 0 && warp == 0) {   // one warp per (sequence, KV head) writes the rows to global memory
      if (ok_s) {
        const int64_t row = (roff + (int64_t)g * cap + slot) * 32;
        static_cast<uint2*>(p.small_k)[row + lane] = kn;
        static_cast<uint2*>(p.small_v)[row + lane] = vn;
      }
      if (ok_f) {
        const int64_t row = (roff_f + (int64_t)g * cap_f + len_f) * 32;
        static_cast<uint2*>(p.full_k)[row + lane] = kn;
        static_cast<uint2*>(p.full_v)[row + lane] = vn;
      }
      if (lane == 0 && (!ok_s || (p.has_full && !ok_f))) atomicOr(p.status, RKV_DEV_APPEND_OVERFLOW);
    }
    new_len_s = (ok_s && !evicting) ? n + 1 : -1;
    new_len_f = ok_f ? len_f + 1 : -1;
    bump_evict = evicting && ok_s;
    if (ok_s) {
      pos_new = slot;
      if (!evicting) n = n + 1;
    }
  }
  if (!kAppend && q_row) *reinterpret_cast<uint4*>(sm_q + (tid >> 4) * kQPad + (tid & 15) * 4) = qv;
  uint32_t qb[8][2];              // B fragments of Q^T: [k = channel][n = head]
  if (warp < kMW) {
    consumer_bar();               // the query rows are in shared memory
    // four 8x8 blocks [head][8 channels] per instruction: block m of load i is channels 32 i + 8 m .. + 7
    const uint32_t q_at = smem_u32(sm_q) + (uint32_t)(lane & 7) * (kQPad * 4) + (uint32_t)(lane >> 3) * 16u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t r[4];
      ldsm_x4(r, q_at + 64u * i);
      qb[2 * i][0] = r[0];
      qb[2 * i][1] = r[1];
      qb[2 * i + 1][0] = r[2];
      qb[2 * i + 1][1] = r[3];
    }
  }
  // Fused append: the lengths are bumped by the last ticket holder of the sequence.  A ticket is taken only
  // after the old lengths have been read by everyone it stands for - one per cluster, taken behind the cluster
  // barrier, or (streaming form, no barrier) one per CTA - so nobody can still see them change.
  // (In a cluster the ticket goes to the last MMA thread, not to thread 0: the atomic's round trip would otherwise
  // hold up warp 0, which finishes the CTA's share of the output right behind it.)
  bool ticket_due = kAppend && tid == (kCluster ? 32 * kMW - 1 : 0) && (!kCluster || split == 0);
  // Streaming form: the CTA takes its ticket right here - it has read the old lengths above - and looks at the
  // number it drew only when it is done, so that the atomic's round trip through L2 (about 900 cycles) is not spent
  // at the end of every CTA, where it would hold the SM and, in the last CTA, the whole kernel.
  int ticket_old = -1;
  if (!kCluster && ticket_due) {
    // (the increment is made to depend on the lengths just loaded, so that the atomic cannot be issued before
    // those loads have returned: a ticket says "this CTA HAS read the old lengths")
    int one;
    asm volatile("{\n\t.reg .b32 t;\n\tand.b32 t, %1, 0;\n\tadd.s32 %0, t, 1;\n\t}" : "=r"(one) : "r"(n ^ new_len_f ^ new_len_s));
    ticket_old = atomicAdd(p.len_tickets + b, one);
  }
  auto take_len_ticket = [&] {
    if (ticket_due) {
      ticket_due = false;
      const int holders = kCluster ? p.n_kv_heads : p.n_kv_heads * (int)gridDim.x;
      const int old = kCluster ? atomicAdd(p.len_tickets + b, 1) : ticket_old;
      if (old == holders - 1) {
        if (new_len_s >= 0) p.small_len[b] = new_len_s;
        if (new_len_f >= 0) p.full_len[b] = new_len_f;
        if (bump_evict) p.evict_count[b] += 1;   // the same decision in every cluster of the sequence
        p.len_tickets[b] = 0;   // ready for the next call on this stream
      }
    }
  };
  if (act == 0) {   // the same for every CTA of a cluster
    take_len_ticket();
    return;
  }
  {
    const int lim = cap < p.max_len ? cap : p.max_len;
    if (n > lim) {
      n = lim;
      if (tid == 0 && split == 0) atomicOr(p.status, RKV_DEV_LEN_CLAMPED);
    }
    if (n < 0) n = 0;
  }
  if (n == 0) {  // nothing cached: the output is defined as zero
    if (n_spec > 0) {   // tiles requested ahead of the length must land before the CTA may go
      if (tid == 0)
        for (int t = 0; t < n_spec; ++t) mbar_wait(bar_full + 8 * t, 0);
      __syncthreads();
    }
    if (split == 0 && tid < kHeadDim)
      for (int h = 0; h < G; ++h) out[h * kHeadDim + tid] = __float2bfloat16(0.f);
    take_len_ticket();
    return;
  }
  const int start = il ? split * kTile : split * p.chunk;   // the CTA's first position
  if (!kCluster && start >= n) {   // in a cluster an idle CTA still owns a slice of the output
    if (n_spec > 0) {
      if (tid == 0)
        for (int t = 0; t < n_spec; ++t) mbar_wait(bar_full + 8 * t, 0);
      __syncthreads();
    }
    take_len_ticket();
    return;
  }
  const int end = (il || start + p.chunk >= n) ? n : start + p.chunk;
  const int total_tiles = (n + kTile - 1) / kTile;
  const int n_tiles = il ? (total_tiles > split ? (total_tiles - split + (int)gridDim.x - 1) / (int)gridDim.x : 0)
                         : ((end > start) ? (end - start + kTile - 1) / kTile : 0);
  const int n_splits = (n + p.chunk - 1) / p.chunk;
  const int64_t row0 = roff + (int64_t)g * cap;

  if (warp == kMW) {
    // ------------------------------------------------------------ copy warp
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      for (int t = n_spec; t < n_tiles; ++t) {
        const int s = t % kStg, use = t / kStg;
        if (use > 0 && !mbar_wait(bar_empty + 8 * s, (use - 1) & 1)) {
          atomicOr(p.status, RKV_DEV_TIMEOUT);
          break;
        }
        issue_tile(t, row0, policy);
      }
    }
    return;
  }

  // ---------------------------------------------------------------- MMA warps
  const float ninf = -INFINITY;
  float m0 = ninf, m1 = ninf, l0 = 0.f, l1 = 0.f;

  // logit scratch is position-major: [position][GP] floats, GP = 4 or 8; this lane holds heads qc, qc+1
  float* lg0 = nullptr;
  if (kLogits) lg0 = p.logits + (int64_t)(b * p.n_kv_heads + g) * p.logit_stride * p.gp + qc;
  const bool lg_on = kLogits && qc < p.gp;
  uint64_t keep_policy = 0;
  if (kLogits) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep_policy));

  // A warp owns a band of kNB 16-row blocks of every tile its group takes (kWT warps per tile).
  const int wb = warp % kWT, grp = warp / kWT;
  const int band0 = kBand * wb;               // first row of the band inside a tile
  bool ok = true;

  const int n_wait = n_tiles > n_spec ? n_tiles : n_spec;   // tiles requested ahead of the length are always consumed
  for (int t = grp; t < n_wait; t += kGroups) {
    const int s = t % kStg;
    if (!mbar_wait(bar_full + 8 * s, (t / kStg) & 1)) {
      if (lane == 0) atomicOr(p.status, RKV_DEV_TIMEOUT);
      ok = false;
      break;
    }
    const int pos_base = tile_pos(t) + band0;
    if (kAppend) {
      // The tile came from global memory, where the new row may not have landed yet: the warp that owns the
      // row writes it into the tile itself (same 128-byte swizzle as the copy engine uses).
      const int rel = pos_new - tile_pos(t);
      if (rel >= 0 && rel < kTile && rel / kBand == wb) {
        const uint32_t at = smem_base + s * kStageBytes + (lane >> 4) * kHalfBytes + rel * 128 +
                            ((((lane & 15) >> 1) ^ (rel & 7)) << 4) + (lane & 1) * 8;
        st_shared_v2(at, kn);
        st_shared_v2(at + 2 * kHalfBytes, vn);
        __syncwarp();
      }
    }
    if (t < n_tiles && pos_base < end) {
      const uint32_t kbase = smem_base + s * kStageBytes;
      // S^T = K Q^T for the band: two accumulator chains per block (half the dependent MMA latency)
      float c[kNB][4], c2[kNB][4];
#pragma unroll
      for (int i = 0; i < kNB; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = c2[i][j] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int chunk = 2 * ks + (lane >> 4);
#pragma unroll
        for (int i = 0; i < kNB; ++i) {
          const int krow = band0 + 16 * i + (lane & 15);
          uint32_t a[4];
          ldsm_x4(a, kbase + (chunk >> 3) * kHalfBytes + krow * 128 + (((chunk & 7) ^ (krow & 7)) << 4));
          if (ks & 1) mma_bf16(c2[i], a, qb[ks][0], qb[ks][1]);
          else mma_bf16(c[i], a, qb[ks][0], qb[ks][1]);
        }
      }
      float sc[kNB][4];
      float t0 = ninf, t1 = ninf;
#pragma unroll
      for (int i = 0; i < kNB; ++i) {
        const int r0 = pos_base + 16 * i + qd, r1 = r0 + 8;
#pragma unroll
        for (int j = 0; j < 4; ++j) sc[i][j] = (c[i][j] + c2[i][j]) * p.scale;
        if (kLogits) {
          if (lg_on) {
            if (r0 < end) st_keep_f2(lg0 + (int64_t)r0 * p.gp, sc[i][0], sc[i][1], keep_policy);
            if (r1 < end) st_keep_f2(lg0 + (int64_t)r1 * p.gp, sc[i][2], sc[i][3], keep_policy);
          }
        }
        if (r0 >= end) sc[i][0] = sc[i][1] = ninf;
        if (r1 >= end) sc[i][2] = sc[i][3] = ninf;
        t0 = fmaxf(t0, fmaxf(sc[i][0], sc[i][2]));
        t1 = fmaxf(t1, fmaxf(sc[i][1], sc[i][3]));
      }
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, sh));
        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, sh));
      }
      const float n0 = fmaxf(m0, t0), n1 = fmaxf(m1, t1);
      if (__any_sync(0xffffffffu, (n0 > m0) || (n1 > m1))) {
        const float a0 = (n0 == m0) ? 1.f : ex2((m0 - n0) * kLog2e);
        const float a1 = (n1 == m1) ? 1.f : ex2((m1 - n1) * kLog2e);
        l0 *= a0;
        l1 *= a1;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          o[i][0] *= a0;
          o[i][1] *= a1;
          o[i][2] *= a0;
          o[i][3] *= a1;
        }
        m0 = n0;
        m1 = n1;
      }
      const float nm0 = (m0 == ninf) ? 0.f : -m0 * kLog2e;
      const float nm1 = (m1 == ninf) ? 0.f : -m1 * kLog2e;
      uint32_t pb[kNB][2];   // P^T as the B operand: the two 8x8 [position][head] blocks transposed inside the warp
#pragma unroll
      for (int i = 0; i < kNB; ++i) {
        const float p0 = ex2(fmaf(sc[i][0], kLog2e, nm0)), p1 = ex2(fmaf(sc[i][1], kLog2e, nm1));
        const float p2 = ex2(fmaf(sc[i][2], kLog2e, nm0)), p3 = ex2(fmaf(sc[i][3], kLog2e, nm1));
        l0 += p0 + p2;
        l1 += p1 + p3;
        if (!kScoreOnly) {
          pb[i][0] = movmatrix_t(pack_bf16(p0, p1));
          pb[i][1] = movmatrix_t(pack_bf16(p2, p3));
        }
      }
      if (!kScoreOnly) {
        const uint32_t vbase = kbase + 2 * kHalfBytes;
#pragma unroll
        for (int i = 0; i < kNB; ++i) {
          const int pos_i = pos_base + 16 * i;
          if (pos_i >= end) continue;   // the whole block lies past the end: its probabilities are zero
          const int vrow = band0 + 16 * i + ((lane >> 4) << 3) + (lane & 7);
          const bool tail = pos_i + 16 > end;
          uint32_t mk0 = 0xffffffffu, mk1 = 0xffffffffu;
          if (tail) {  // rows past the end may hold anything (even NaN): zero them so that 0 * x stays 0
            const int pa = pos_i + qc;
            mk0 = (pa < end ? 0x0000ffffu : 0u) | (pa + 1 < end ? 0xffff0000u : 0u);
            mk1 = (pa + 8 < end ? 0x0000ffffu : 0u) | (pa + 9 < end ? 0xffff0000u : 0u);
          }
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            const int chunk = 2 * mt + ((lane >> 3) & 1);
            uint32_t a[4];
            ldsm_x4_t(a, vbase + (chunk >> 3) * kHalfBytes + vrow * 128 + (((chunk & 7) ^ (vrow & 7)) << 4));
            if (tail) {
              a[0] &= mk0;
              a[1] &= mk0;
              a[2] &= mk1;
              a[3] &= mk1;
            }
            mma_bf16(o[mt], a, pb[i][0], pb[i][1]);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty + 8 * s);
  }

#pragma unroll
  for (int sh = 4; sh <= 16; sh <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
    l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
  }

  // ------------------------------------------------ merge the MMA warps
  // Every warp publishes its (m, l); after one barrier each warp knows the CTA-wide maximum of its two heads
  // and writes its accumulators already scaled to it, so that the merge itself is a plain sum (few
  // instructions per thread: this phase is bound by instruction issue, not by memory).
  float* sm_wm = reinterpret_cast<float*>(sm_q + kMaxGroup * kQPad);   // [kMW][8]: per-warp maximum (own memory)
  if (lane < 4) *reinterpret_cast<float2*>(sm_wm + warp * 8 + qc) = make_float2(m0, m1);
  consumer_bar();   // (m) of every warp is visible, and the stage memory is free
  float* sm_o = reinterpret_cast<float*>(smem_gen);   // [kMW][8][kOPad] scaled accumulators
  float* sm_l = sm_o + kMW * 8 * kOPad;               // [kMW][8] scaled denominators
  float* sm_M = sm_l + kMW * 8;                       // [8] CTA-wide maximum per head
  {
    float M0 = ninf, M1 = ninf;
#pragma unroll
    for (int w = 0; w < kMW; ++w) {
      const float2 mw = *reinterpret_cast<const float2*>(sm_wm + w * 8 + qc);   // qc is even
      M0 = fmaxf(M0, mw.x);
      M1 = fmaxf(M1, mw.y);
    }
    const float e0 = (m0 == ninf) ? 0.f : ex2((m0 - M0) * kLog2e);
    const float e1 = (m1 == ninf) ? 0.f : ex2((m1 - M1) * kLog2e);
    float* base = sm_o + (warp * 8 + qc) * kOPad + qd;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      base[16 * mt] = o[mt][0] * e0;
      base[kOPad + 16 * mt] = o[mt][1] * e1;
      base[16 * mt + 8] = o[mt][2] * e0;
      base[kOPad + 16 * mt + 8] = o[mt][3] * e1;
    }
    if (lane < 4) {
      sm_l[warp * 8 + qc] = l0 * e0;
      sm_l[warp * 8 + qc + 1] = l1 * e1;
      if (warp == 0) {
        sm_M[qc] = M0;
        sm_M[qc + 1] = M1;
      }
    }
  }
  consumer_bar();

  // The merged accumulators as items of (head, four channels): G * 32 items over the MMA threads.
  constexpr int kNT = 32 * kMW;
  constexpr int kIt = (kMaxGroup * 32 + kNT - 1) / kNT;
  const int n_items = G * 32;
  float4 acc4[kIt];
#pragma unroll
  for (int it = 0; it < kIt; ++it) {
    acc4[it] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int item = tid + it * kNT;
    if (item < n_items) {
      const float* src = sm_o + (item >> 5) * kOPad + (item & 31) * 4;
#pragma unroll
      for (int w = 0; w < kMW; ++w) {
        const float4 v = *reinterpret_cast<const float4*>(src + w * 8 * kOPad);
        acc4[it].x += v.x;
        acc4[it].y += v.y;
        acc4[it].z += v.z;
        acc4[it].w += v.w;
      }
    }
  }
  // (m, l) of one head for the whole CTA; heads beyond the group read as (-inf, 0)
  auto head_ml = [&](int h, float& M, float& L) {
    M = ninf;
    L = 0.f;
    if (h < G) {
      M = sm_M[h];
#pragma unroll
      for (int w = 0; w < kMW; ++w) L += sm_l[w * 8 + h];
    }
  };

  const int bg = b * p.n_kv_heads + g;

  if (kCluster) {
    // ---------------------------------------------- merge the CTAs of the cluster through shared memory
    const int C = (int)gridDim.x;                       // cluster size = CTAs per (sequence, KV head): 1, 2, 4 or 8
    const int c_sh = __ffs(C) - 1;                      // C is a power of two: shifts instead of divisions below
    const int dchunk = kHeadDim >> c_sh;                // channels of every head that one CTA finishes
    if (C == 1) {   // a "cluster" of one: nothing to exchange (and no remote stores from a launch without clusters)
      take_len_ticket();
      if (!ok) return;
#pragma unroll
      for (int it = 0; it < kIt; ++it) {
        const int item = tid + it * kNT;
        if (item < n_items) {
          const int h = item >> 5, d4 = (item & 31) * 4;
          float Mh, Lh;
          head_ml(h, Mh, Lh);
          const float inv = __fdividef(1.f, Lh);
          uint2 o2;
          o2.x = pack_bf16(acc4[it].x * inv, acc4[it].y * inv);
          o2.y = pack_bf16(acc4[it].z * inv, acc4[it].w * inv);
          *reinterpret_cast<uint2*>(out + h * kHeadDim + d4) = o2;
        }
      }
      return;
    }
    float* recv = reinterpret_cast<float*>(smem_gen + kStg * kStageBytes + 16 * kStg + 16);
    float* recv_ml = recv + kMaxGroup * kHeadDim;       // [source CTA][head][2]
    const uint32_t recv_u32 = smem_u32(recv), recv_ml_u32 = smem_u32(recv_ml);
#pragma unroll
    for (int it = 0; it < kIt; ++it) {
      const int item = tid + it * kNT;
      if (item < n_items) {   // four channels never straddle two owners: dchunk is a multiple of 16
        const int h = item >> 5, d4 = (item & 31) * 4;
        const int owner = d4 >> (7 - c_sh), dd = d4 & (dchunk - 1);
        st_async_f32x4(map_rank(recv_u32 + 4u * ((split * kMaxGroup + h) * dchunk + dd), owner), acc4[it],
                       map_rank(bar_recv, owner));
      }
    }
    if (tid < kMaxGroup * C) {   // (m, l) of head tid % 8 to peer tid / 8
      const int h = tid & 7, peer = tid >> 3;
      float Md, Ld;
      head_ml(h, Md, Ld);
      st_async_f32x2(map_rank(recv_ml_u32 + 4u * ((split * kMaxGroup + h) * 2), peer), Md, Ld, map_rank(bar_recv, peer));
    }
    if (!mbar_wait(bar_recv, 0)) {   // every peer's slice is here (bounded: a lost peer cannot hang the GPU)
      if (lane == 0) atomicOr(p.status, RKV_DEV_TIMEOUT);
      ok = false;
    }
    take_len_ticket();
    if (!ok) return;
    // This CTA finishes dchunk channels of every head: G * dchunk / 4 items of four channels, one thread each, which
    // reads the C sources' slices straight from the receive buffer (independent loads, no shuffles: with one or two
    // warps per scheduler a chain of dependent shuffles costs more than the loads it saves; two lanes per item with
    // one round of shuffles measured the same).
    const int ph_sh = 5 - c_sh;             // log2 of the items per head, dchunk / 4
    if (tid < (n_items >> c_sh)) {
      const int h = tid >> ph_sh, dd = (tid & ((1 << ph_sh) - 1)) * 4;
      float2 ml[kAttnCluster];
      float4 v[kAttnCluster];
      float M = ninf;
#pragma unroll
      for (int r = 0; r < kAttnCluster; ++r) {
        if (r < C) {
          ml[r] = *reinterpret_cast<const float2*>(recv_ml + (r * kMaxGroup + h) * 2);
          v[r] = *reinterpret_cast<const float4*>(recv + (r * kMaxGroup + h) * dchunk + dd);
          M = fmaxf(M, ml[r].x);
        }
      }
      float L = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int r = 0; r < kAttnCluster; ++r) {
        if (r < C) {
          const float e = (ml[r].x == ninf) ? 0.f : ex2((ml[r].x - M) * kLog2e);
          L = fmaf(ml[r].y, e, L);
          acc.x = fmaf(v[r].x, e, acc.x);
          acc.y = fmaf(v[r].y, e, acc.y);
          acc.z = fmaf(v[r].z, e, acc.z);
          acc.w = fmaf(v[r].w, e, acc.w);
        }
      }
      const float inv = __fdividef(1.f, L);
      uint2 o2;
      o2.x = pack_bf16(acc.x * inv, acc.y * inv);
      o2.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2*>(out + h * kHeadDim + split * dchunk + dd) = o2;
    }
    return;
  }

  const int d = tid;   // the other forms run with four MMA warps: one thread per channel below
  const bool single = (kMode == kModeTicket) && n_splits == 1;   // the full step always leaves its partials to the selector
  if (single) {
    if (!ok) return;
#pragma unroll
    for (int it = 0; it < kIt; ++it) {
      const int item = tid + it * kNT;
      if (item < n_items) {
        const int h = item >> 5, d4 = (item & 31) * 4;
        float Mh, Lh;
        head_ml(h, Mh, Lh);
        const float inv = 1.f / Lh;
        uint2 o2;
        o2.x = pack_bf16(acc4[it].x * inv, acc4[it].y * inv);
        o2.y = pack_bf16(acc4[it].z * inv, acc4[it].w * inv);
        *reinterpret_cast<uint2*>(out + h * kHeadDim + d4) = o2;
      }
    }
    return;
  }
  {
    float* part = p.partials + ((int64_t)bg * p.max_splits + split) * PartialLayout::kFloats;
    if (!kScoreOnly) {
#pragma unroll
      for (int it = 0; it < kIt; ++it) {
        const int item = tid + it * kNT;
        if (item < n_items) *reinterpret_cast<float4*>(part + (item >> 5) * kHeadDim + (item & 31) * 4) = acc4[it];
      }
    }
    if (d < kMaxGroup) {
      float Md, Ld;
      head_ml(d, Md, Ld);
      part[kMaxGroup * kHeadDim + d] = Md;
      part[kMaxGroup * kHeadDim + kMaxGroup + d] = Ld;
      if (kLogits && p.ml_t != nullptr) {   // the selection kernel reads these across the splits: keep a contiguous copy
        float* t = p.ml_t + (int64_t)bg * 16 * p.max_splits + split;
        t[(int64_t)d * p.max_splits] = Md;
        t[(int64_t)(kMaxGroup + d) * p.max_splits] = Ld;
      }
    }
    take_len_ticket();     // streaming form with the append: the ticket drawn at the start is looked at here
    if (kLogits) return;   // full step: the selection kernel (or the fold kernel) finishes out from the partials
    __threadfence();
    consumer_bar();
    if (tid == 0) {
      const int old = atomicAdd(p.tickets + bg, 1);
      s_last = (old == n_splits - 1) ? 1 : 0;
    }
    consumer_bar();
    if (!s_last) return;
    __threadfence();
    // last CTA of this (sequence, KV head): fold all split partials
    const float* pbase = p.partials + (int64_t)bg * p.max_splits * PartialLayout::kFloats;
    float* sm_red = reinterpret_cast<float*>(smem_gen);                 // [4][8][128]
    float* sm_w = sm_red + 4 * kMaxGroup * kHeadDim;                    // [n_splits][16]
    float* sm_ML = sm_w + kMaxSplits * 16;                              // [16]
    auto bar = [] { consumer_bar_n<128>(); };
    fold_weights<128>(pbase, n_splits, tid, sm_w, sm_ML, bar);
    fold_out<128, kMaxGroup>(pbase, n_splits, 0, G, tid, sm_w, sm_red, bar);
    if (tid == 0) p.tickets[bg] = 0;  // ready for the next call on this stream
    if (!ok) return;
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h)
      if (h < G) out[h * kHeadDim + d] = __float2bfloat16(sm_red[h * kHeadDim + d] / sm_ML[8 + h]);
  }
}

}  // namespace

static size_t ring_smem_bytes(int stages) {
  return (size_t)stages * kStageBytes + 16 * stages + 16 + (size_t)kRecvFloats * sizeof(float) +
         (size_t)kMaxGroup * kQPad * 4 + 16 * 8 * sizeof(float) + 1024;   // ring, barriers, receive buffer, query, warp maxima
}
size_t attention_smem_bytes() { return ring_smem_bytes(kStages); }
static size_t cluster_smem_bytes(bool wide) { return ring_smem_bytes(wide ? Ring<kModeCluster, true>::kStg : kStages); }

cudaError_t prepare_attention() {
  const int bytes = (int)attention_smem_bytes();
  cudaError_t e = cudaFuncSetAttribute(attn_kernel<kModeFull>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_kernel<kModeTicket>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_kernel<kModeScore>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_kernel<kModeFullAppend>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_kernel<kModeCluster, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_kernel<kModeClusterAppend, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_kernel<kModeCluster, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)cluster_smem_bytes(true));
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_kernel<kModeClusterAppend, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)cluster_smem_bytes(true));
  return e;
}

cudaError_t launch_attention(const AttnParams& p, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                             int n_seq, int grid_x, bool write_logits, cudaStream_t st, bool append) {
  dim3 grid(grid_x, p.n_kv_heads, n_seq);
  if (write_logits && append)
    return launch_ex(attn_kernel<kModeFullAppend>, grid, dim3(kAttnThreads), attention_smem_bytes(), st, 1, tm_k, tm_v,
                     p);
  if (write_logits)
    return launch_ex(attn_kernel<kModeFull>, grid, dim3(kAttnThreads), attention_smem_bytes(), st, 1, tm_k, tm_v, p);
  return launch_ex(attn_kernel<kModeTicket>, grid, dim3(kAttnThreads), attention_smem_bytes(), st, 1, tm_k, tm_v, p);
}

cudaError_t launch_attention_scores(const AttnParams& p, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                    int n_seq, int grid_x, cudaStream_t st) {
  dim3 grid(grid_x, p.n_kv_heads, n_seq);
  return launch_ex(attn_kernel<kModeScore>, grid, dim3(kAttnThreads), attention_smem_bytes(), st, 1, tm_k, tm_v, p);
}

cudaError_t launch_attention_cluster(const AttnParams& p, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                     int n_seq, int cluster, bool append, bool wide, cudaStream_t st) {
  dim3 grid(cluster, p.n_kv_heads, n_seq);
  const size_t smem = cluster_smem_bytes(wide);
  if (wide) {
    const dim3 block(Ring<kModeCluster, true>::kThreads);
    if (append) return launch_ex(attn_kernel<kModeClusterAppend, true>, grid, block, smem, st, cluster, tm_k, tm_v, p);
    return launch_ex(attn_kernel<kModeCluster, true>, grid, block, smem, st, cluster, tm_k, tm_v, p);
  }
  const dim3 block(kAttnThreads);
  if (append) return launch_ex(attn_kernel<kModeClusterAppend, false>, grid, block, smem, st, cluster, tm_k, tm_v, p);
  return launch_ex(attn_kernel<kModeCluster, false>, grid, block, smem, st, cluster, tm_k, tm_v, p);
}

}  // namespace rkv
