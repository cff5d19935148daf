// Full-step epilogue: fold of the split-K partials, score finalisation and exact top-K selection.
// One thread-block cluster (8 CTAs) per (sequence, KV head).
//
// RefreshKV (arXiv 2411.05787) Sec. 2.2: the partial cache is rebuilt from the
// top-K positions of the current token's attention scores a_L; for grouped-query
// attention the scores of the query heads of a group are aggregated by max
// (footnote of Sec. 2.2; mean / first head are the ablation modes of App. A.3).
//
// Input: the scaled logits s[j][h] (position-major, GP = 4 or 8 floats per position)
// and the split partials the attention kernel wrote.  Every CTA derives the
// log-sum-exp of all heads of the group from the partials and folds one eighth of
// out[] of the group.  Then
//   ell[j] = agg_h (s[j][h] - LSE[h])            (log of the aggregated probability)
// and the K largest scores are the K smallest keys  key = bits(max(-ell, 0)),  an
// order-preserving 31-bit image of -ell (equal images are ties and go to the lower
// position).  The kernel is a chain of latencies, so it is laid out to have few links:
//   1  one round trip fetches the per-sequence sizes, the split weights, this CTA's
//      slice of the partial outputs and its first logits, all at once;
//   2  keys + a 2048-bin histogram (1/64 nat per bin) in shared memory (with neighbour max-pooling
//      of the scores, App. A.1, the keys of a window are min-reduced first);
//   3  cluster barrier; the eight histograms are merged through distributed shared
//      memory and the bin T that holds the K-th key is located (while T holds more
//      than 256 keys, a finer histogram over T's key range repeats this step);
//   4  every CTA pushes its few keys of bin T into a flat array in all peers, plus
//      its count of keys below T;
//   5  cluster barrier; every CTA finds the threshold key by brute force over the
//      <= 256 pushed keys and knows how many winners precede its slice;
//   6  winners are written in ascending position order (deterministic, and the later
//      gather walks the cache monotonically).
// No global store precedes the first barrier (a release would wait for it); the
// score output is regenerated from the keys between arrive and wait of the second.
#include <cuda_bf16.h>

#include <cstddef>

#include "rkv_internal.h"

namespace rkv {
namespace {

constexpr int NT = kSelectThreads;
constexpr int NW = NT / 32;
constexpr int kBins = 2048;
constexpr int kHistWords = kBins / 2;     // two 16-bit counters per word (a CTA holds at most 40960 keys)
constexpr int kCandMax = 256;             // keys of the final bin that are resolved by brute force
constexpr int kMaxPasses = 5;             // pass 0 + refinements of 11 bits each cover the 31-bit key
constexpr int kOPre = 10;                 // partial-output values per thread fetched in the first round trip
constexpr uint32_t kWorstKey = 0x7f800000u;   // bits of +inf: probability 0, or a NaN score
constexpr uint32_t kPadKey = 0xffffffffu;     // filler behind a CTA's last key: never a winner, never in a bin
constexpr float kLog2eF = 1.4426950408889634f;
constexpr float kLn2F = 0.6931471805599453f;
static_assert(kSelectMaxKeysPerCta < 65536, "packed 16-bit histogram counters");
static_assert(kSelectCluster == 8 && NT == 512, "merge and finish assume 8 CTAs of 16 warps");
static_assert(kMaxSplits <= 128, "four weight loads per lane cover every split");

struct SelectShared {
  alignas(16) uint32_t hist[2][kHistWords];   // double-buffered: peers may still read the previous pass
  alignas(16) uint32_t flat[kCandMax];        // final-bin keys of the whole cluster, in CTA order (pushed by peers)
  alignas(16) float w[kMaxSplits * 8];        // w[s][h]: weight of split s for head h
  alignas(16) float red[4][kHeadDim];
  float lse[kMaxGroup], linv[kMaxGroup];
  uint32_t below[kSelectCluster];             // pushed by CTA r: its keys below the final bin
  uint32_t inbin[kSelectCluster];             // per CTA: its keys inside the located bin (from the merge)
  uint32_t warp_a[NW];
  uint32_t sel_bin, sel_want, sel_count;
  uint32_t own_below, own_in, cand_fill;
  uint32_t tau, ties, less_pre, eq_pre;
  uint32_t bad;
};
static_assert(offsetof(SelectShared, hist) % 16 == 0 && offsetof(SelectShared, flat) % 16 == 0, "vector access");

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint32_t map_rank(uint32_t local_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ uint4 ld_cluster_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared::cluster.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void st_cluster(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Split cluster barrier: work placed between arrive and wait hides the barrier's latency.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2f(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max_nan(float a, float b) {   // NaN if either operand is NaN
  float y;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
  return y;
}
__device__ __forceinline__ uint32_t warp_sum(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// After a cluster barrier: merge hist[buf] of the eight CTAs and locate the bin that holds the
// want-th smallest key.  Leaves sel_bin / sel_want (rank inside the bin) / sel_count (bin size) and
// inbin[r] (CTA r's share of the bin) in shared memory.
__device__ __forceinline__ void merge_locate(SelectShared* sh, int buf, uint32_t want) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t m[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
  uint4 v[kSelectCluster];
  if (tid < kHistWords / 4) {
    const uint32_t local = smem_u32(&sh->hist[buf][tid * 4]);
#pragma unroll
    for (int r = 0; r < kSelectCluster; ++r) v[r] = ld_cluster_v4(map_rank(local, r));
#pragma unroll
    for (int r = 0; r < kSelectCluster; ++r) {
      m[0] += v[r].x & 0xffffu; m[1] += v[r].x >> 16;
      m[2] += v[r].y & 0xffffu; m[3] += v[r].y >> 16;
      m[4] += v[r].z & 0xffffu; m[5] += v[r].z >> 16;
      m[6] += v[r].w & 0xffffu; m[7] += v[r].w >> 16;
    }
  }
  uint32_t sum = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) sum += m[i];
  uint32_t inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) sh->warp_a[warp] = inc;
  __syncthreads();
  if (tid < kHistWords / 4) {
    uint32_t base = 0;
#pragma unroll
    for (int w2 = 0; w2 < kHistWords / 128; ++w2)
      if (w2 < warp) base += sh->warp_a[w2];
    const uint32_t excl = base + inc - sum;
    if (excl < want && want <= excl + sum) {   // exactly one thread
      uint32_t run = excl;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (run < want && want <= run + m[i]) {
          sh->sel_bin = tid * 8 + i;
          sh->sel_want = want - run;
          sh->sel_count = m[i];
#pragma unroll
          for (int r = 0; r < kSelectCluster; ++r) {
            const uint32_t word = (i >> 1) == 0 ? v[r].x : (i >> 1) == 1 ? v[r].y : (i >> 1) == 2 ? v[r].z : v[r].w;
            sh->inbin[r] = (i & 1) ? (word >> 16) : (word & 0xffffu);
          }
        }
        run += m[i];
      }
    }
  }
  __syncthreads();
}

// GP: floats per position in the logit scratch, 4 (G <= 4) or 8.  kMinBlocks = 2 trades a few spilled
// registers for two resident CTAs per SM: with more clusters than one wave holds, their latency chains overlap.
template <int GP, int kMinBlocks>
__global__ void __launch_bounds__(NT, kMinBlocks) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int rank = (int)cluster_rank();
  const int b = blockIdx.z, g = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  SelectShared* sh = reinterpret_cast<SelectShared*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + ((sizeof(SelectShared) + 15) & ~size_t(15)));
  for (int i = tid; i < 2 * kHistWords; i += NT) (&sh->hist[0][0])[i] = 0u;
  if (tid == 0) {
    sh->cand_fill = 0u;
    sh->own_below = 0u;
    sh->own_in = 0u;
    sh->bad = 0u;
  }
  const int G = p.group;
  const int bg = b * p.n_kv_heads + g;
  // Positions per CTA: with one sequence the host fixes the slices from its length bound, so the first logits
  // can be requested before the length arrives; with a batch (ragged lengths) each sequence is cut in eight
  // by its own length once that is known, so that short sequences still use the whole cluster.
  const bool per_fixed = p.per_fixed != 0;
  int per = p.per_cta;
  int lo = rank * per;
  const float* pbase = p.partials + (int64_t)bg * p.max_splits * PartialLayout::kFloats;
  const int half = p.pool_half;               // neighbour max-pooling of the scores over 2*half+1 positions (0: none)
  // keys are made for positions lo-half .. lo+per+half-1 (the pooling window reaches into the neighbours' slices)
  const float* lg = p.logits + ((int64_t)bg * p.logit_stride + lo - half) * GP;   // re-based below if the slices move
  uint32_t* raw = half > 0 ? keys + p.keys_cap : keys;   // unpooled keys; the same array when there is no pooling
  constexpr int U = 32 / GP;                  // positions per thread per round: all their loads are in flight together
  const int gx = p.grid_splits;               // splits the attention launch had room for (>= the sequence's own count)
  // slice of out[] this CTA folds: 16*G consecutive (head, channel) pairs of the group
  const int o_local = tid & 127, sgrp = tid >> 7;
  const bool o_on = o_local < 16 * G;
  const bool fold_on = o_on && p.out != nullptr;   // the score-only step has no attention output to fold
  const int o_flat = rank * 16 * G + o_local;
  const int64_t hrow0 = ((int64_t)b * p.n_q_heads + (int64_t)g * G) * kHeadDim;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)

  // ---------------------------------------------------------------- 1: everything the kernel reads, in one round trip
  const int act = (p.active != nullptr) ? __ldcg(p.active + b) : 1;
  int n = __ldcg(p.len + b);
  const int cap = __ldcg(p.cap + b);
  int kk = __ldcg(p.k_small + b);
  float wm[4], wl[4];                          // warps 0..7: (m, l) of head `warp` for splits lane, lane+32, ...
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int s = lane + 32 * k;
    const bool on = warp < kMaxGroup && s < gx;
    const float* pt = p.ml_t + ((int64_t)bg * 16 + warp) * p.max_splits + s;   // contiguous over the splits
    wm[k] = on ? __ldcg(pt) : -INFINITY;
    wl[k] = on ? __ldcg(pt + (int64_t)kMaxGroup * p.max_splits) : 0.f;
  }
  float opre[kOPre];
#pragma unroll
  for (int k = 0; k < kOPre; ++k) {
    const int s = sgrp + 4 * k;
    opre[k] = (fold_on && s < gx) ? __ldcg(pbase + (int64_t)s * PartialLayout::kFloats + o_flat) : 0.f;
  }
  __nv_bfloat16 qv = __float2bfloat16(0.f);
  if (p.q_last_full != nullptr && sgrp == 0 && o_on) qv = static_cast<const __nv_bfloat16*>(p.q)[hrow0 + o_flat];
  float4 v[U][GP / 4], vnext[U][GP / 4];     // the round being turned into keys, and the one in flight behind it
  auto load_round = [&](float4 (&dst)[U][GP / 4], int i0) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT + tid;
      const int pos = lo - half + i;
      const bool on = i < per + 2 * half && pos >= 0 && pos < p.logit_stride;
#pragma unroll
      for (int c = 0; c < GP / 4; ++c)
        dst[u][c] = on ? __ldcg(reinterpret_cast<const float4*>(lg + (int64_t)i * GP) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  if (per_fixed) load_round(v, 0);

  if (act == 0) return;   // same decision in all CTAs of the cluster
  {
    const int lim = cap < p.max_len ? cap : p.max_len;
    if (n > lim) n = lim;
    if (n < 0) n = 0;
  }
  if (kk > p.k_max) kk = p.k_max;
  if (kk > n) kk = n;
  if (kk < 0) kk = 0;
  int32_t* idx_out = p.topk_idx + (int64_t)bg * p.k_max;
  if (n == 0) {   // the attention kernel has zeroed out[]
    for (int i = rank * NT + tid; i < p.k_max; i += kSelectCluster * NT) idx_out[i] = -1;
    return;
  }
  if (!per_fixed) {
    per = (((n + kSelectCluster - 1) / kSelectCluster) + 3) & ~3;   // never above the host's per_cta (n <= its bound)
    lo = rank * per;
    lg = p.logits + ((int64_t)bg * p.logit_stride + lo - half) * GP;
    load_round(v, 0);
  }
  const int cnt = (n - lo < 0) ? 0 : (n - lo < per ? n - lo : per);
  const int R = (((cnt + NT - 1) / NT) + 3) & ~3;   // keys per thread in the ordered phases (multiple of 4)
  const int cnt_pad = R * NT;
  const bool all_selected = (kk == n);
  const bool need_keys = (!all_selected && kk > 0) || p.scores != nullptr;
  int n_splits = (n + p.chunk - 1) / p.chunk;
  if (n_splits > gx) n_splits = gx;

  // ---------------------------------------------------------------- log-sum-exp and split weights, one warp per head
  if (warp < kMaxGroup) {
    float M = -INFINITY;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (lane + 32 * k >= n_splits) wm[k] = -INFINITY;
      M = fmaxf(M, wm[k]);
    }
    M = warp_max_f(M);
    float L = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float e = (wm[k] == -INFINITY) ? 0.f : ex2f((wm[k] - M) * kLog2eF);
      L = fmaf(wl[k], e, L);
      if (lane + 32 * k < kMaxSplits) sh->w[(lane + 32 * k) * 8 + warp] = e;
    }
    L = warp_sum_f(L);
    if (lane == 0) {
      sh->lse[warp] = M + logf(L);
      sh->linv[warp] = 1.f / L;
    }
  }
  __syncthreads();

  // this CTA's slice of out[] (and of the trigger's reference query); run where it hides a cluster barrier
  auto fold_slice = [&] {
    const int h = o_flat >> 7;
    float acc = 0.f;
    if (fold_on) {
#pragma unroll
      for (int k = 0; k < kOPre; ++k) {
        const int s = sgrp + 4 * k;
        if (s < n_splits) acc = fmaf(opre[k], sh->w[s * 8 + h], acc);
      }
      for (int s = sgrp + 4 * kOPre; s < n_splits; s += 4)
        acc = fmaf(__ldcg(pbase + (int64_t)s * PartialLayout::kFloats + o_flat), sh->w[s * 8 + h], acc);
    }
    sh->red[sgrp][o_local] = acc;
    __syncthreads();
    if (sgrp == 0 && o_on) {
      const float o = (sh->red[0][o_local] + sh->red[1][o_local]) + (sh->red[2][o_local] + sh->red[3][o_local]);
      if (fold_on) static_cast<__nv_bfloat16*>(p.out)[hrow0 + o_flat] = __float2bfloat16(o * sh->linv[h]);
      if (p.q_last_full != nullptr) static_cast<__nv_bfloat16*>(p.q_last_full)[hrow0 + o_flat] = qv;
    }
    for (int i = kk + rank * NT + tid; i < p.k_max; i += kSelectCluster * NT) idx_out[i] = -1;   // padding
  };
  // score[j] = exp(ell[j]) regenerated from the keys (a NaN score has been flagged and reads as 0)
  auto write_scores = [&] {
    if (p.scores != nullptr) {
      float* sc = p.scores + (int64_t)bg * p.score_stride + lo;
      for (int i = tid; i < cnt; i += NT) sc[i] = ex2f(-__uint_as_float(keys[i]) * kLog2eF);
    }
    if (tid == 0 && sh->bad != 0u) atomicOr(p.status, RKV_DEV_NONFINITE);
  };

  // ---------------------------------------------------------------- 2: keys and the pass-0 histogram
  if (need_keys) {
    float lse_r[GP];
#pragma unroll
    for (int h = 0; h < GP; ++h) lse_r[h] = (h < G) ? sh->lse[h] : INFINITY;
    const int agg = p.agg;
    const float inv_g = 1.f / (float)G;
    bool bad = false;
    const int n_raw = half > 0 ? (cnt > 0 ? cnt + 2 * half : 0) : cnt_pad;   // without pooling the padding is written here too
    for (int i0 = 0; i0 < n_raw; i0 += U * NT) {
      const bool more = i0 + U * NT < n_raw;
      if (more) load_round(vnext, i0 + U * NT);   // overlaps the arithmetic below
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * NT + tid;
        if (i >= n_raw) continue;
        const float* x = reinterpret_cast<const float*>(&v[u][0]);
        float ell;
        if (agg == RKV_AGG_MAX) {   // heads >= G carry LSE = +inf and drop out of the max
          ell = x[0] - lse_r[0];
#pragma unroll
          for (int h = 1; h < GP; ++h) ell = max_nan(ell, x[h] - lse_r[h]);
        } else if (agg == RKV_AGG_MEAN) {
          float acc = 0.f;
#pragma unroll
          for (int h = 0; h < GP; ++h) acc += ex2f((x[h] - lse_r[h]) * kLog2eF);   // ex2(-inf) = 0 for heads >= G
          ell = lg2f(acc * inv_g) * kLn2F;
        } else {
          ell = x[0] - lse_r[0];
        }
        uint32_t key = kPadKey;
        const int pos = lo - half + i;
        if (i < cnt + 2 * half && pos >= 0 && pos < n) {
          uint32_t bin;
          if (ell != ell) {
            bad = true;
            key = kWorstKey;
            bin = kBins - 1;
          } else {
            const float nl = fmaxf(-ell, 0.f);
            key = __float_as_uint(nl) & 0x7fffffffu;
            bin = __float2uint_rz(fminf(nl * 64.f, (float)(kBins - 1)));
          }
          if (!all_selected && half == 0) atomicAdd(&sh->hist[0][bin >> 1], 1u << ((bin & 1u) << 4));
        }
        raw[i] = key;
      }
      if (more) {
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
          for (int c = 0; c < GP / 4; ++c) v[u][c] = vnext[u][c];
      }
    }
    if (bad) sh->bad = 1u;
    if (half > 0) {
      // pooled score = max over the window = smallest key of the window (App. A.1: kernel size 7 in the paper)
      __syncthreads();
      for (int i = tid; i < cnt_pad; i += NT) {
        uint32_t key = kPadKey;
        if (i < cnt) {
          for (int d = 0; d <= 2 * half; ++d) key = min(key, raw[i + d]);
          const uint32_t bin = __float2uint_rz(fminf(__uint_as_float(key) * 64.f, (float)(kBins - 1)));
          if (!all_selected) atomicAdd(&sh->hist[0][bin >> 1], 1u << ((bin & 1u) << 4));
        }
        keys[i] = key;
      }
    }
  }

  if (all_selected || kk == 0) {   // uniform over the cluster: nothing to choose
    __syncthreads();
    fold_slice();
    write_scores();
    if (all_selected)
      for (int i = tid; i < cnt; i += NT) {
        idx_out[lo + i] = lo + i;
        if (p.win_keys != nullptr && need_keys) p.win_keys[(int64_t)bg * p.win_stride + lo + i] = keys[i];
      }
    return;
  }

  // ---------------------------------------------------------------- 3: locate the bin of the kk-th smallest key
  uint32_t lo_key = 0u, hi_key = kWorstKey, want = (uint32_t)kk, count = 0u;
  int shb = 0;
  for (int pass = 0; pass < kMaxPasses; ++pass) {
    if (pass > 0) {   // refine inside [lo_key, hi_key]: bins of 2^shb key values
      const uint32_t span = hi_key - lo_key;
      shb = 32 - __clz(span) - 11;
      if (shb < 0) shb = 0;
      uint32_t* h = sh->hist[pass & 1];
      for (int i = tid; i < kHistWords; i += NT) h[i] = 0u;
      __syncthreads();
      for (int i = tid; i < cnt; i += NT) {
        const uint32_t key = keys[i];
        if (key >= lo_key && key <= hi_key) {
          const uint32_t bin = (key - lo_key) >> shb;
          atomicAdd(&h[bin >> 1], 1u << ((bin & 1u) << 4));
        }
      }
    }
    cluster_arrive();
    if (pass == 0) fold_slice();
    cluster_wait();
    merge_locate(sh, pass & 1, want);
    const uint32_t T = sh->sel_bin;
    want = sh->sel_want;
    count = sh->sel_count;
    if (pass == 0) {   // bin T of pass 0 is  T/64 <= -ell < (T+1)/64  (the last bin is open-ended)
      lo_key = __float_as_uint((float)T * (1.f / 64.f));
      hi_key = (T == kBins - 1) ? kWorstKey : __float_as_uint((float)(T + 1) * (1.f / 64.f)) - 1u;
    } else {
      lo_key = lo_key + (T << shb);
      const uint32_t top = lo_key + ((1u << shb) - 1u);
      hi_key = top < hi_key ? top : hi_key;
    }
    if (count <= (uint32_t)kCandMax || lo_key == hi_key) break;
  }
  // count > kCandMax here means the bin is a single key value shared by all its members
  const bool ident = count > (uint32_t)kCandMax;

  // ---------------------------------------------------------------- 4: exchange the final bin
  if (tid < kCandMax && tid >= (int)count) sh->flat[tid] = kPadKey;   // nobody pushes there: lets the search read vectors
  uint32_t flat_base = 0;   // where this CTA's keys start in the flat array (CTA order)
#pragma unroll
  for (int r = 0; r < kSelectCluster; ++r)
    if (r < rank) flat_base += sh->inbin[r];
  const uint4* my_keys = reinterpret_cast<const uint4*>(keys + (size_t)tid * R);   // thread t owns keys [t*R, (t+1)*R)
  {
    uint32_t c_below = 0;
    const uint32_t flat0 = smem_u32(&sh->flat[0]);
    for (int j = 0; j < R / 4; ++j) {
      const uint4 k4 = my_keys[j];
      const uint32_t kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        c_below += (kv[e] < lo_key);
        if (!ident && kv[e] >= lo_key && kv[e] <= hi_key) {   // rare: a handful per CTA
          const uint32_t slot = flat_base + atomicAdd(&sh->cand_fill, 1u);
          if (slot < (uint32_t)kCandMax) {
#pragma unroll
            for (int r = 0; r < kSelectCluster; ++r) st_cluster(map_rank(flat0 + 4u * slot, r), kv[e]);
          }
        }
      }
    }
    c_below = warp_sum(c_below);
    if (lane == 0 && c_below != 0u) atomicAdd(&sh->own_below, c_below);
  }
  __syncthreads();
  if (tid < kSelectCluster) st_cluster(map_rank(smem_u32(&sh->below[rank]), tid), sh->own_below);
  cluster_arrive();
  write_scores();
  cluster_wait();
  // from here on nobody touches a peer's shared memory

  // ---------------------------------------------------------------- 5: threshold key; winners before this slice
  if (ident) {
    if (tid == 0) {
      sh->tau = lo_key;
      sh->ties = want;
      sh->less_pre = 0u;
      sh->eq_pre = flat_base;
    }
  } else {
    // P threads share one candidate (P a power of two, P * count <= 512): each counts over 1/P of the flat array
    int lp = 0;                                   // log2(P)
    while (lp < 5 && ((int)count << (lp + 1)) <= NT) ++lp;
    const int ci = tid >> lp, part = tid & ((1 << lp) - 1);
    if (ci < (int)count) {                        // whole groups of P lanes take this branch together
      const int len = ((((int)count + (1 << lp) - 1) >> lp) + 3) & ~3;   // a multiple of four: 16-byte reads
      const int j0 = part * len;
      const uint32_t c = sh->flat[ci];
      uint32_t less = 0, eq = 0, less_p = 0, eq_p = 0;
      for (int j = j0; j < j0 + len && j < kCandMax; j += 4) {
        const uint4 x4 = *reinterpret_cast<const uint4*>(&sh->flat[j]);
        const uint32_t xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool pre = j + e < (int)flat_base;
          less += (xs[e] < c);
          eq += (xs[e] == c);
          less_p += (pre && xs[e] < c);
          eq_p += (pre && xs[e] == c);
        }
      }
      const uint32_t gmask = __activemask();
      for (int o = 1; o < (1 << lp); o <<= 1) {
        less += __shfl_xor_sync(gmask, less, o);
        eq += __shfl_xor_sync(gmask, eq, o);
        less_p += __shfl_xor_sync(gmask, less_p, o);
        eq_p += __shfl_xor_sync(gmask, eq_p, o);
      }
      if (part == 0 && less < want && want <= less + eq) {
        // every thread that holds the threshold value writes the same four numbers
        sh->tau = c;
        sh->ties = want - less;
        sh->less_pre = less_p;
        sh->eq_pre = eq_p;
      }
    }
  }
  __syncthreads();
  const uint32_t tau = sh->tau, ties_to_take = sh->ties;
  uint32_t winners_before = sh->less_pre + (sh->eq_pre < ties_to_take ? sh->eq_pre : ties_to_take);
#pragma unroll
  for (int r = 0; r < kSelectCluster; ++r)
    if (r < rank) winners_before += sh->below[r];
  const uint32_t ties_before = sh->eq_pre;

  // ---------------------------------------------------------------- 6: ordered output
  uint32_t c_less = 0, c_eq = 0;
  for (int j = 0; j < R / 4; ++j) {
    const uint4 k4 = my_keys[j];
    c_less += (k4.x < tau) + (k4.y < tau) + (k4.z < tau) + (k4.w < tau);
    c_eq += (k4.x == tau) + (k4.y == tau) + (k4.z == tau) + (k4.w == tau);
  }
  // exclusive block scan of both counts at once (each total fits 16 bits)
  const uint32_t packed = c_less | (c_eq << 16);
  uint32_t inc = packed;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) sh->warp_a[warp] = inc;
  __syncthreads();
  uint32_t wbase = (lane < warp) ? sh->warp_a[lane] : 0u;   // NW = 16 <= 32 lanes
  wbase = warp_sum(wbase);
  const uint32_t excl = wbase + inc - packed;
  const uint32_t e_less = excl & 0xffffu;
  uint32_t eq_seen = ties_before + (excl >> 16);
  // ties are kept in position order: the first ties_to_take of them (cluster-wide) win
  uint32_t offs = winners_before + e_less +
                  ((eq_seen < ties_to_take ? eq_seen : ties_to_take) - (ties_before < ties_to_take ? ties_before : ties_to_take));
  const int i_base = tid * R;
  for (int j = 0; j < R / 4; ++j) {
    const uint4 k4 = my_keys[j];
    const uint32_t kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      bool win = kv[e] < tau;
      if (kv[e] == tau) {
        win = eq_seen < ties_to_take;
        ++eq_seen;
      }
      if (win) {
        if (offs < (uint32_t)kk) {
          idx_out[offs] = lo + i_base + 4 * j + e;
          if (p.win_keys != nullptr) p.win_keys[(int64_t)bg * p.win_stride + offs] = kv[e];
        }
        ++offs;
      }
    }
  }
}

}  // namespace

int select_keys_cap(int keys_per_cta) {   // R * NT keys, R a multiple of 4
  return (int)(((size_t)keys_per_cta + 4 * NT - 1) / (4 * NT) * (4 * NT));
}

size_t select_smem_bytes(int keys_per_cta, int pool_half) {
  const size_t padded = (size_t)select_keys_cap(keys_per_cta);
  const size_t raw = pool_half > 0 ? padded + 2 * (size_t)pool_half + 4 : 0;   // unpooled keys with their halo
  return ((sizeof(SelectShared) + 15) & ~size_t(15)) + (padded + raw) * 4;
}

cudaError_t prepare_select() {
  const int bytes = (int)select_smem_bytes(kSelectMaxKeysPerCta, 0);
  cudaError_t e = cudaFuncSetAttribute(select_kernel<4, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(select_kernel<8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(select_kernel<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(select_kernel<8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  return e;
}

cudaError_t launch_select(const SelectParams& p, int n_seq, int sm_count, cudaStream_t st) {
  const dim3 grid(kSelectCluster, p.n_kv_heads, n_seq);
  const size_t smem = select_smem_bytes(p.per_cta, p.pool_half);
  // two CTAs per SM when one wave cannot hold every cluster and two CTAs' shared memory fits
  const bool dense = (int64_t)kSelectCluster * p.n_kv_heads * n_seq > sm_count && 2 * (smem + 1024) <= 227 * 1024;
  if (p.group <= 4) {
    if (dense) return launch_ex(select_kernel<4, 2>, grid, dim3(NT), smem, st, kSelectCluster, p);
    return launch_ex(select_kernel<4, 1>, grid, dim3(NT), smem, st, kSelectCluster, p);
  }
  if (dense) return launch_ex(select_kernel<8, 2>, grid, dim3(NT), smem, st, kSelectCluster, p);
  return launch_ex(select_kernel<8, 1>, grid, dim3(NT), smem, st, kSelectCluster, p);
}

}  // namespace rkv
