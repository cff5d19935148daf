// Full-step epilogue: score finalisation and exact top-K selection, as two kernels.
//
// RefreshKV (arXiv 2411.05787) Sec. 2.2: the partial cache is rebuilt from the
// top-K positions of the current token's attention scores a_L; for grouped-query
// attention the scores of the query heads of a group are aggregated by max
// (footnote of Sec. 2.2; mean / first head are the ablation modes of App. A.3), and the
// scores may be max-pooled over neighbouring positions first (App. A.1: kernel size 7).
//
// Input: the scaled logits s[j][h] (position-major, GP = 4 or 8 floats per position)
// and the softmax statistics (m, l) of the split partials the attention kernel wrote.
//   ell[j] = agg_h (s[j][h] - LSE[h])            (log of the aggregated probability)
// and the K largest scores are the K smallest keys  key = bits(max(-ell, 0)),  an
// order-preserving 31-bit image of -ell (equal images are ties and go to the lower position).
//
// score_kernel   grid-wide and bandwidth-shaped: one CTA per slice of positions of one
//                (sequence, KV head).  Every CTA derives the log-sum-exp of the group's
//                heads from the split statistics, turns its logits into keys (written to
//                the workspace, 4 bytes per position, and - optionally - as scores) and counts
//                them in the (sequence, KV head)'s histogram of 4096 bins (1/128 nat each) in
//                global memory, one reduction per warp and distinct bin.
//                Optional extra CTAs fold out[] from the split partials (rkv_full_step).
// select_kernel  one thread-block cluster (1..8 CTAs) per (sequence, KV head), a short chain:
//   1  one round trip fetches the sizes, the histogram and this CTA's slice of the keys;
//   2  a block scan of the histogram locates the bin T that holds the K-th key (when T holds
//      more than 256 keys - long runs of near-equal scores - finer histograms over T's key
//      range, merged through distributed shared memory, narrow it down);
//   3  every thread counts its keys below T (a block scan turns the counts into output
//      offsets) and pushes its few keys inside T, with their positions, to all peers;
//   4  one cluster barrier; every CTA ranks the <= 256 pushed (key, position) pairs by brute
//      force - the ones of rank below the K-th's rank inside T are selected - and knows how
//      many winners precede its slice;
//   5  winners are written in ascending position order (deterministic, and the later
//      gather walks the cache monotonically).
//      The histogram is cleared again by the cluster that used it.
#include <cuda_bf16.h>

#include <cstddef>

#include "rkv_internal.h"

namespace rkv {
namespace {

constexpr int NT = kSelectThreads;        // threads of a selection CTA
constexpr int NW = NT / 32;
constexpr int NTS = kScoreThreads;        // threads of a score-pass CTA
constexpr int kBins = kSelectBins;        // level-1 histogram: bins of 1/128 nat over -log p, the last one open-ended
constexpr float kBinsPerNat = 128.f;
constexpr int kFineBins = 2048;           // refinement histograms of the selection
constexpr int kFineWords = kFineBins / 2; // packed 16-bit counters (a CTA holds fewer than 65536 keys)
constexpr int kCandMax = 256;             // keys of the final bin that are resolved by brute force
constexpr int kMaxPasses = 5;             // refinements of 11 bits each cover the 31-bit key
constexpr int kFoldU = 10;                // splits per warp in the fold's first batch of loads
constexpr uint32_t kWorstKey = 0x7f800000u;   // bits of +inf: probability 0, or a NaN score
constexpr uint32_t kPadKey = 0xffffffffu;     // filler behind a CTA's last key: never a winner, never in a bin
constexpr float kLog2eF = 1.4426950408889634f;
constexpr float kLn2F = 0.6931471805599453f;
static_assert(kSelectMaxKeysPerCta + NT < 65536, "packed 16-bit counters in the refinement histograms and the tie scan");
static_assert(NT == 512 && kBins == 8 * NT, "the histogram scan gives every thread 8 bins");
static_assert(kFineWords == 2 * NT, "the refinement merge gives every thread two words");
static_assert(kCandMax <= NT, "one thread per candidate when the flat list is built");
static_assert(kMaxSplits <= 128 && NTS / 32 == kMaxGroup, "score pass: one warp per head, four split statistics per lane");

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint32_t map_rank(uint32_t local_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
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
__device__ __forceinline__ uint32_t warp_scan_incl(uint32_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// The sizes both kernels work with: the length clamped as the attention pass clamped it, the number of
// positions to select, and whether there is anything to choose (only then is the histogram used at all,
// and both kernels must agree on that: the one adds to it, the other clears it).
struct Sizes {
  int n, kk;
  bool choose;
};
__device__ __forceinline__ Sizes clamp_sizes(int len, int cap, int max_len, int k_small, int k_max) {
  Sizes s;
  const int lim = cap < max_len ? cap : max_len;
  s.n = len > lim ? lim : len;
  if (s.n < 0) s.n = 0;
  s.kk = k_small > k_max ? k_max : k_small;
  if (s.kk > s.n) s.kk = s.n;
  if (s.kk < 0) s.kk = 0;
  s.choose = s.kk > 0 && s.kk < s.n;
  return s;
}

// key of a position from its GP logits (heads >= G carry LSE = +inf and drop out)
template <int GP, int AGG>
__device__ __forceinline__ uint32_t make_key(const float* x, const float* lse_r, float inv_g, bool* bad) {
  float ell;
  if (AGG == RKV_AGG_MAX) {
    ell = x[0] - lse_r[0];
#pragma unroll
    for (int h = 1; h < GP; ++h) ell = max_nan(ell, x[h] - lse_r[h]);
  } else if (AGG == RKV_AGG_MEAN) {
    float acc = 0.f;
#pragma unroll
    for (int h = 0; h < GP; ++h) acc += ex2f((x[h] - lse_r[h]) * kLog2eF);   // ex2(-inf) = 0 for heads >= G
    ell = lg2f(acc * inv_g) * kLn2F;
  } else {
    ell = x[0] - lse_r[0];
  }
  if (ell != ell) {
    *bad = true;
    return kWorstKey;
  }
  return __float_as_uint(fmaxf(-ell, 0.f)) & 0x7fffffffu;
}
// The histogram's window: bin T of a (sequence, KV head) holds  A + T/128 <= -ell < A + (T+1)/128,  bin 0 also
// everything below A and the last bin everything above.  For logits of spread sigma the bulk of the keys sits
// around the log-sum-exp of the group's heads (a position of average logit has -ell = LSE) and the K-th key a few
// sigma below it, so the window starts kWindowBelow nats below the smallest LSE of the group: sharply peaked
// attention, whose keys all lie dozens of nats up, is resolved as finely as flat attention.  A is an integer, which
// keeps  -ell - A  and the bin edges exact in fp32: both kernels agree on every key's bin.
constexpr float kWindowBelow = 26.f;
__device__ __forceinline__ int window_anchor(float lse_min) {
  const float a = floorf(lse_min - kWindowBelow);
  return a > 0.f ? (a < 1024.f ? (int)a : 1024) : 0;   // (NaN compares false: 0)
}
__device__ __forceinline__ uint32_t bin_of(uint32_t key, float anchor) {
  return __float2uint_rz(fminf(fmaxf((__uint_as_float(key) - anchor) * kBinsPerNat, 0.f), (float)(kBins - 1)));
}

// ------------------------------------------------------------------------------------------------ score_kernel
// GP: floats per position in the logit scratch, 4 (G <= 4) or 8.  kPool: neighbour max-pooling of the scores.
// The kernel is a chain of a few hundred instructions per warp, so it is written for few of them.  The slice's
// keys are counted in a shared-memory histogram, which ONE bulk reduction (cp.reduce.async.bulk: the copy engine
// adds 16 KiB of counters to the (sequence, KV head)'s histogram in global memory) sends on: with bins this fine
// a slice hardly ever puts two keys into one, and a reduction instruction per key costs an SM about two cycles.
template <int GP, int AGG, bool kPool>
__global__ void __launch_bounds__(NTS) score_kernel(const ScoreParams p) {
  extern __shared__ __align__(16) uint32_t raw[];     // pooling only: unpooled keys of the slice and its halo
  __shared__ __align__(128) uint32_t s_hist[kBins];
  __shared__ uint32_t s_bmin, s_bmax;                 // range of bins the slice's keys fall into
  __shared__ float s_lse[kMaxGroup];
  __shared__ float s_e[kMaxSplits];
  __shared__ float s_red[NTS / 32][32];
  __shared__ float s_L;
  const int b = blockIdx.z, g = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.group;
  const int64_t bg = (int64_t)b * p.n_kv_heads + g;
  const int gx = p.grid_splits;               // splits the attention launch had room for (>= the sequence's own count)

  if ((int)blockIdx.x >= p.n_slices) {
    // ---------------------------------------------------------------- extra CTAs: out[] from the split partials
    // (flash-decoding merge: M = max_s m_s, w_s = exp(m_s - M), out = sum_s w_s O_s / sum_s w_s l_s).  One CTA
    // per (head of the group, half of the channels); warp w takes the splits s = w (mod 4) of one 32-channel
    // quarter; every load is issued before the first is used.
    const int fx = (int)blockIdx.x - p.n_slices;
    const int h = fx >> 1, quarter = (fx & 1) * 2 + (warp >> 2), w4 = warp & 3;
    const int c = quarter * 32 + lane;
    pdl_wait();
    pdl_launch();
    const int act = p.active != nullptr ? __ldcg(p.active + b) : 1;
    const int len = __ldcg(p.len + b);
    const int cap = __ldg(p.cap + b);
    const float* po = p.partials + bg * p.max_splits * PartialLayout::kFloats + h * kHeadDim + c;
    float v[kFoldU];
#pragma unroll
    for (int k = 0; k < kFoldU; ++k) {
      const int s = w4 + 4 * k;
      v[k] = s < gx ? __ldcg(po + (int64_t)s * PartialLayout::kFloats) : 0.f;
    }
    float m[4], l[4];
    if (warp == 0) {
      const float* pm = p.ml_t + bg * 16 * p.max_splits + (int64_t)h * p.max_splits;
      const float* pl = pm + (int64_t)kMaxGroup * p.max_splits;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int s = lane + 32 * i;
        m[i] = s < gx ? __ldcg(pm + s) : -INFINITY;
        l[i] = s < gx ? __ldcg(pl + s) : 0.f;
      }
    }
    if (act == 0) return;
    const Sizes sz = clamp_sizes(len, cap, p.max_len, 0, 0);
    if (sz.n <= 0) return;                    // nothing cached: the attention pass has written zeros
    int n_splits = (sz.n + p.chunk - 1) / p.chunk;
    if (n_splits > gx) n_splits = gx;
    if (warp == 0) {
      float M = -INFINITY, L = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (lane + 32 * i >= n_splits) {
          m[i] = -INFINITY;
          l[i] = 0.f;
        }
        M = fmaxf(M, m[i]);
      }
      M = warp_max_f(M);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float e = (m[i] == -INFINITY) ? 0.f : ex2f((m[i] - M) * kLog2eF);
        L = fmaf(l[i], e, L);
        s_e[lane + 32 * i] = e;
      }
      L = warp_sum_f(L);
      if (lane == 0) s_L = L;
    }
    __syncthreads();
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < kFoldU; ++k) {
      const int s = w4 + 4 * k;
      if (s < n_splits) acc = fmaf(v[k], s_e[s], acc);
    }
    for (int s = w4 + 4 * kFoldU; s < n_splits; s += 4)
      acc = fmaf(__ldcg(po + (int64_t)s * PartialLayout::kFloats), s_e[s], acc);
    s_red[warp][lane] = acc;
    __syncthreads();
    if (w4 == 0) {
      const float sum = (s_red[warp][lane] + s_red[warp + 1][lane]) + (s_red[warp + 2][lane] + s_red[warp + 3][lane]);
      static_cast<__nv_bfloat16*>(p.out)[((int64_t)b * p.n_q_heads + (int64_t)g * G + h) * kHeadDim + c] =
          __float2bfloat16(sum / s_L);
    }
    return;
  }

  // -------------------------------------------------------------------- a slice of positions of one (sequence, KV head)
  const int lo = (int)blockIdx.x * p.slice;
  const int half = kPool ? p.pool_half : 0;
#pragma unroll
  for (int k = 0; k < kBins / 4 / NTS; ++k)
    reinterpret_cast<uint4*>(s_hist)[k * NTS + tid] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {
    s_bmin = kBins - 1;
    s_bmax = 0u;
  }
  constexpr int U = 4;                        // positions per thread per round: all their loads are in flight together
  // positions lo - half .. lo + slice + half - 1 become keys (the pooling window reaches into the neighbours' slices)
  const int n_pos = p.slice + 2 * half;
  const float4* lg = reinterpret_cast<const float4*>(p.logits + (bg * p.logit_stride + lo - half + tid) * GP);
  // Addresses and predicates of everything the CTA reads are worked out above the dependency wait, so that
  // behind it only the loads themselves are left to issue.
  const int32_t* a_act = p.active != nullptr ? p.active + b : nullptr;
  const int32_t* a_len = p.len + b;
  const int32_t* a_cap = p.cap + b;
  const int32_t* a_ks = p.k_small + b;
  const float* a_ml = p.ml_t + (bg * 16 + warp) * p.max_splits + lane;   // warp h: (m, l) of head h, contiguous over the splits
  const int ml_l = kMaxGroup * p.max_splits;
  bool ml_on[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) ml_on[k] = lane + 32 * k < gx;
  bool lg_on[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int i = u * NTS + tid;
    const int pos = lo - half + i;
    lg_on[u] = i < n_pos && pos >= 0 && pos < p.logit_stride;
  }
  const int64_t hrow0 = ((int64_t)b * p.n_q_heads + (int64_t)g * G) * kHeadDim;
  const bool q_copy = blockIdx.x == 0 && p.q_last_full != nullptr && tid < G * 16;
  const uint4* a_q = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.q) + hrow0) + tid;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)

  // everything the CTA reads, in one round trip
  const int act = (a_act != nullptr) ? __ldcg(a_act) : 1;
  const int len = __ldcg(a_len);
  const int cap = __ldg(a_cap);
  const int k_small = __ldcg(a_ks);
  float wm[4], wl[4];                          // (m, l) for splits lane, lane + 32, ...
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    wm[k] = ml_on[k] ? __ldcg(a_ml + 32 * k) : -INFINITY;
    wl[k] = ml_on[k] ? __ldcg(a_ml + 32 * k + ml_l) : 0.f;
  }
  float4 v[U][GP / 4];
#pragma unroll
  for (int u = 0; u < U; ++u)
#pragma unroll
    for (int c = 0; c < GP / 4; ++c)
      v[u][c] = lg_on[u] ? __ldcg(lg + (int64_t)(u * NTS) * (GP / 4) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
  float4 vnext[U][GP / 4];                     // the round in flight behind the one being turned into keys
  int n_hint = 0x7fffffff;                     // the sequence's length (+ halo), once known: nothing is loaded beyond it
  auto load_round = [&](int i0) {   // positions lo - half + i0 + u * NTS + tid (rounds after the first)
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NTS + tid;
      const int pos = lo - half + i;
      const bool on = i < n_pos && pos >= 0 && pos < p.logit_stride && pos < n_hint;
#pragma unroll
      for (int c = 0; c < GP / 4; ++c)
        vnext[u][c] = on ? __ldcg(lg + (int64_t)(i0 + u * NTS) * (GP / 4) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };

  uint4 qv = make_uint4(0u, 0u, 0u, 0u);
  if (q_copy) qv = __ldcg(a_q);

  if (act == 0) return;
  if (q_copy) reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.q_last_full) + hrow0)[tid] = qv;
  const Sizes sz = clamp_sizes(len, cap, p.max_len, k_small, p.k_max);
  const int n = sz.n;
  if (lo >= n) return;
  int n_splits = (n + p.chunk - 1) / p.chunk;
  if (n_splits > gx) n_splits = gx;

  // log-sum-exp of every head of the group, one warp per head
  {
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
    }
    L = warp_sum_f(L);
    if (lane == 0) s_lse[warp] = M + lg2f(L) * kLn2F;
  }
  __syncthreads();
  float lse_r[GP];
  float lse_min = INFINITY;
#pragma unroll
  for (int h = 0; h < GP; ++h) {
    lse_r[h] = (h < G) ? s_lse[h] : INFINITY;
    lse_min = fminf(lse_min, lse_r[h]);
  }
  const int anchor_i = window_anchor(lse_min);
  const float anchor = (float)anchor_i;
  if (blockIdx.x == 0 && tid == 0) p.anchor[bg] = anchor_i;   // the selection kernel turns bins back into key ranges
  const float inv_g = 1.f / (float)G;
  bool bad = false;
  uint32_t* keys_out = p.keys + bg * p.logit_stride;
  float* sc_out = p.scores != nullptr ? p.scores + bg * p.score_stride : nullptr;
  uint32_t bmin = kBins - 1, bmax = 0u;
  // a key leaves the kernel: the workspace copy, the optional score, the histogram
  auto emit = [&](int pos, uint32_t key) {
    keys_out[pos] = key;
    if (sc_out != nullptr) sc_out[pos] = ex2f(-__uint_as_float(key) * kLog2eF);   // a NaN score has been flagged and reads as 0
    if (sz.choose) {
      const uint32_t bin = bin_of(key, anchor);
      atomicAdd(&s_hist[bin], 1u);
      bmin = min(bmin, bin);
      bmax = max(bmax, bin);
    }
  };
  n_hint = n + half;
  for (int i0 = 0; i0 < n_pos; i0 += U * NTS) {
    const bool more = i0 + U * NTS < n_pos && lo - half + i0 + U * NTS < n + half;
    if (more) load_round(i0 + U * NTS);        // overlaps the arithmetic below
    if (lo - half + i0 >= n + half) break;     // uniform over the CTA: the rest of the slice lies beyond the sequence
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NTS + tid;
      const int pos = lo - half + i;
      if (i0 + u * NTS >= n_pos) continue;     // uniform over the CTA
      const bool on = i < n_pos && pos >= 0 && pos < n;
      uint32_t key = kPadKey;
      if (on) key = make_key<GP, AGG>(reinterpret_cast<const float*>(&v[u][0]), lse_r, inv_g, &bad);
      if (kPool) {
        if (i < n_pos) raw[i] = key;
      } else if (on) {
        emit(pos, key);
      }
    }
    if (more) {
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int c = 0; c < GP / 4; ++c) v[u][c] = vnext[u][c];
    }
  }
  if (kPool) {
    // pooled score = max over the window = smallest key of the window (positions outside the sequence do not count)
    __syncthreads();
    for (int i = tid; i < p.slice; i += NTS) {
      const int pos = lo + i;
      if (pos >= n) break;
      uint32_t key = kPadKey;
      for (int d = 0; d <= 2 * half; ++d) key = min(key, raw[i + d]);
      emit(pos, key);
    }
  }
  // The counters go from the generic proxy (the atomics above) to the copy engine: fence, then barrier, then one
  // issue - of the occupied range of bins only (16-byte granules), which is a fraction of the histogram.
  if (sz.choose) {
    bmin = __reduce_min_sync(0xffffffffu, bmin);
    bmax = __reduce_max_sync(0xffffffffu, bmax);
    if (lane == 0) {
      atomicMin(&s_bmin, bmin);
      atomicMax(&s_bmax, bmax);
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  const int any_bad = __syncthreads_or(bad);
  if (tid == 0) {
    if (sz.choose) {
      const uint32_t b0 = s_bmin & ~3u, b1 = (s_bmax | 3u) + 1u;
      if (b1 > b0) {
        asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.u32 [%0], [%1], %2;" ::"l"(p.hist + bg * kBins + b0),
                     "r"(smem_u32(s_hist + b0)), "r"((uint32_t)((b1 - b0) * sizeof(uint32_t)))
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    }
    if (any_bad) atomicOr(p.status, RKV_DEV_NONFINITE);
    // the CTA's shared memory must outlive the engine's read of it
    if (sz.choose) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
}

// ------------------------------------------------------------------------------------------------ select_kernel
struct SelectShared {
  alignas(16) unsigned long long seg[kSelectCluster][kCandMax];   // (key << 32 | position) of the final-bin keys of CTA r
  alignas(16) unsigned long long flat[kCandMax];                  // the same in one array, in CTA order
  alignas(16) uint32_t fine[2][kFineWords];   // refinement histograms, double-buffered: peers may still read the previous pass
  int32_t mywin[kCandMax];                    // positions of this CTA's final-bin keys that are selected
  uint32_t below[kSelectCluster];             // pushed by CTA r: its keys below the final bin
  uint32_t candn[kSelectCluster];             // pushed by CTA r: its keys inside the final bin
  uint32_t warp_a[NW];
  uint32_t sel_bin, sel_want, sel_count;
  uint32_t cand_fill, own_in, n_mywin, win_before;
};

// Merge fine[buf] of the C CTAs and locate the bin that holds the want-th smallest key.  Leaves sel_bin /
// sel_want (rank inside the bin) / sel_count (bin size) in shared memory.  Called behind a cluster barrier.
__device__ __noinline__ void merge_locate(SelectShared* sh, int buf, uint32_t want, int C) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t m[4] = {0u, 0u, 0u, 0u};
  const uint32_t local = smem_u32(&sh->fine[buf][tid * 2]);
  for (int r = 0; r < C; ++r) {
    uint2 v;
    if (C == 1) {
      v = *reinterpret_cast<const uint2*>(&sh->fine[buf][tid * 2]);
    } else {
      asm volatile("ld.shared::cluster.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(map_rank(local, r)));
    }
    m[0] += v.x & 0xffffu; m[1] += v.x >> 16;
    m[2] += v.y & 0xffffu; m[3] += v.y >> 16;
  }
  const uint32_t sum = (m[0] + m[1]) + (m[2] + m[3]);
  const uint32_t inc = warp_scan_incl(sum, lane);
  if (lane == 31) sh->warp_a[warp] = inc;
  __syncthreads();
  uint32_t base = 0;
#pragma unroll
  for (int w2 = 0; w2 < NW; ++w2)
    if (w2 < warp) base += sh->warp_a[w2];
  const uint32_t excl = base + inc - sum;
  if (excl < want && want <= excl + sum) {   // exactly one thread
    uint32_t run = excl;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (run < want && want <= run + m[i]) {
        sh->sel_bin = tid * 4 + i;
        sh->sel_want = want - run;
        sh->sel_count = m[i];
      }
      run += m[i];
    }
  }
  __syncthreads();
}

// Narrow [lo_key, hi_key] down with finer histograms until it holds at most kCandMax keys or a single key value.
__device__ __noinline__ void refine(SelectShared* sh, const uint32_t* keys, int per, int C, uint32_t* lo_key_io,
                                    uint32_t* hi_key_io, uint32_t* want_io, uint32_t* count_io) {
  const int tid = threadIdx.x;
  uint32_t lo_key = *lo_key_io, hi_key = *hi_key_io, want = *want_io, count = *count_io;
  for (int pass = 0; pass < kMaxPasses; ++pass) {
    const uint32_t span = hi_key - lo_key;
    int shb = 32 - __clz(span) - 11;          // bins of 2^shb key values
    if (shb < 0) shb = 0;
    uint32_t* h = sh->fine[pass & 1];
    for (int i = tid; i < kFineWords; i += NT) h[i] = 0u;
    __syncthreads();
    for (int i = tid; i < per; i += NT) {
      const uint32_t key = keys[i];
      if (key - lo_key <= span) {
        const uint32_t bin = (key - lo_key) >> shb;
        atomicAdd(&h[bin >> 1], 1u << ((bin & 1u) << 4));
      }
    }
    if (C > 1) {
      cluster_arrive();
      cluster_wait();
    } else {
      __syncthreads();
    }
    merge_locate(sh, pass & 1, want, C);
    const uint32_t T = sh->sel_bin;
    want = sh->sel_want;
    count = sh->sel_count;
    lo_key = lo_key + (T << shb);
    const uint32_t top = lo_key + ((1u << shb) - 1u);
    hi_key = top < hi_key ? top : hi_key;
    if (count <= (uint32_t)kCandMax || lo_key == hi_key) break;
  }
  *lo_key_io = lo_key;
  *hi_key_io = hi_key;
  *want_io = want;
  *count_io = count;
}

// Output when the final bin is one key value shared by more than kCandMax keys (long runs of equal scores): the
// keys below it win, and of the equal ones the first ties_to_take in position order, cluster-wide.
__device__ __noinline__ void write_ties(SelectShared* sh, const uint32_t* my, int R, int first, uint32_t tau,
                                        uint32_t ties_to_take, uint32_t ties_before, uint32_t below_before, int kk,
                                        int32_t* idx_out, uint32_t* win_out) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t c_less = 0, c_eq = 0;
  for (int j = 0; j < R; ++j) {
    const uint32_t key = my[j];
    c_less += key < tau;
    c_eq += key == tau;
  }
  // exclusive block scan of both counts at once (each total fits 16 bits)
  const uint32_t packed = c_less | (c_eq << 16);
  const uint32_t inc = warp_scan_incl(packed, lane);
  __syncthreads();   // warp_a may still be read by the scan before the exchange
  if (lane == 31) sh->warp_a[warp] = inc;
  __syncthreads();
  uint32_t wbase = (lane < warp) ? sh->warp_a[lane] : 0u;   // NW = 16 <= 32 lanes
  wbase = warp_sum(wbase);
  const uint32_t excl = wbase + inc - packed;
  uint32_t eq_seen = ties_before + (excl >> 16);
  const uint32_t tb = ties_before < ties_to_take ? ties_before : ties_to_take;
  uint32_t offs = below_before + tb + (excl & 0xffffu) + ((eq_seen < ties_to_take ? eq_seen : ties_to_take) - tb);
  for (int j = 0; j < R; ++j) {
    const uint32_t key = my[j];
    bool win = key < tau;
    if (key == tau) {
      win = eq_seen < ties_to_take;
      ++eq_seen;
    }
    if (win) {
      if (offs < (uint32_t)kk) {
        idx_out[offs] = first + j;
        if (win_out != nullptr) win_out[offs] = key;
      }
      ++offs;
    }
  }
}

// Keys per thread of a CTA when n keys are cut over C CTAs of NT threads: a multiple of four (16-byte reads).
__host__ __device__ __forceinline__ int keys_per_thread(int n, int C) {
  int q = (n + 4 * C * NT - 1) / (4 * C * NT);
  if (q < 1) q = 1;
  return 4 * q;
}

__global__ void __launch_bounds__(NT, 2) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int C = (int)gridDim.x;               // CTAs per (sequence, KV head) = cluster size
  const int rank = C > 1 ? (int)cluster_rank() : 0;
  const int b = blockIdx.z, g = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  SelectShared* sh = reinterpret_cast<SelectShared*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + ((sizeof(SelectShared) + 15) & ~size_t(15)));
  if (tid == 0) {
    sh->cand_fill = 0u;
    sh->own_in = 0u;
    sh->n_mywin = 0u;
    sh->win_before = 0u;
    sh->sel_bin = kBins - 1;
    sh->sel_want = 1u;
    sh->sel_count = 0u;
  }
  const int64_t bg = (int64_t)b * p.n_kv_heads + g;
  // One sequence: the slices are fixed by the host's length bound, so that the keys can be requested before the
  // length is known.  A batch (ragged lengths): each sequence is cut in C by its own length once that is known, so
  // that short sequences use the whole cluster too.
  const bool per_fixed = p.per_fixed != 0;
  int R = p.keys_per_thread;
  int per = R * NT;                           // a multiple of four
  int lo = rank * per;
  int n4 = per / 4;
  const uint4* kg4 = reinterpret_cast<const uint4*>(p.keys + bg * p.logit_stride + lo);
  int lim4 = lo < p.logit_stride ? (int)((p.logit_stride - lo) / 4) : 0;   // vectors of this slice inside the buffer
  // The one barrier that makes every peer's shared memory addressable sits above the dependency wait, where it is free.
  if (C > 1) {
    cluster_arrive();
    cluster_wait();
  } else {
    __syncthreads();
  }
  // addresses and predicates are worked out above the dependency wait: behind it only the loads are left to issue
  const int32_t* a_act = p.active != nullptr ? p.active + b : nullptr;
  const int32_t* a_len = p.len + b;
  const int32_t* a_cap = p.cap + b;
  const int32_t* a_ks = p.k_small + b;
  const int32_t* a_anchor = p.anchor + bg;
  const uint4* hg = reinterpret_cast<const uint4*>(p.hist + bg * kBins) + tid * 2;
  constexpr int KU = 4;
  bool kq_on[KU];
#pragma unroll
  for (int u = 0; u < KU; ++u) kq_on[u] = per_fixed && u * NT + tid < n4 && u * NT + tid < lim4;
  int32_t* idx_out = p.topk_idx + bg * p.k_max;
  uint32_t* win_out = p.win_keys != nullptr ? p.win_keys + bg * p.win_stride : nullptr;
  pdl_wait();
  pdl_launch();   // dependents are released only after this kernel's own wait (see launch_ex)

  // ---------------------------------------------------------------- 1: sizes, histogram and keys, one round trip
  const int act = (a_act != nullptr) ? __ldcg(a_act) : 1;
  const int len = __ldcg(a_len);
  const int cap = __ldg(a_cap);
  const int k_small = __ldcg(a_ks);
  const float anchor = (float)__ldcg(a_anchor);
  uint4 hv[2];                                 // thread t: bins 8 t .. 8 t + 7
  hv[0] = __ldcg(hg);
  hv[1] = __ldcg(hg + 1);
  const uint4 pad4 = make_uint4(kPadKey, kPadKey, kPadKey, kPadKey);
  uint4 kq[KU];
#pragma unroll
  for (int u = 0; u < KU; ++u) kq[u] = kq_on[u] ? __ldcg(kg4 + u * NT + tid) : pad4;
  if (act == 0) return;   // same decision in all CTAs of the cluster
  const Sizes sz = clamp_sizes(len, cap, p.max_len, k_small, p.k_max);
  const int n = sz.n, kk = sz.kk;
  for (int i = kk + rank * NT + tid; i < p.k_max; i += C * NT) idx_out[i] = -1;   // padding
  if (n == 0) return;
  if (!per_fixed) {
    R = keys_per_thread(n, C);                // never above the host's bound (n <= its length bound)
    per = R * NT;
    lo = rank * per;
    n4 = per / 4;
    kg4 = reinterpret_cast<const uint4*>(p.keys + bg * p.logit_stride + lo);
    lim4 = lo < p.logit_stride ? (int)((p.logit_stride - lo) / 4) : 0;
#pragma unroll
    for (int u = 0; u < KU; ++u) {
      const int i4 = u * NT + tid;
      kq[u] = (i4 < n4 && i4 < lim4 && lo + 4 * i4 < n) ? __ldcg(kg4 + i4) : pad4;
    }
  }
  const int first = lo + tid * R;              // thread t owns keys [t R, (t + 1) R) of the slice
  const uint32_t* my = keys + tid * R;
  {
    uint4* keys4 = reinterpret_cast<uint4*>(keys);
    const bool inside = lo + per <= n;        // the whole slice lies inside the sequence: nothing to pad
    auto put = [&](int i4, uint4 k4) {        // keys at and beyond the length become padding
      if (!inside) {
        const int pos0 = lo + 4 * i4;
        if (pos0 >= n) k4.x = kPadKey;
        if (pos0 + 1 >= n) k4.y = kPadKey;
        if (pos0 + 2 >= n) k4.z = kPadKey;
        if (pos0 + 3 >= n) k4.w = kPadKey;
      }
      keys4[i4] = k4;
    };
#pragma unroll
    for (int u = 0; u < KU; ++u) {
      const int i4 = u * NT + tid;
      if (i4 < n4) put(i4, kq[u]);
    }
    for (int base = KU * NT; base < n4; base += KU * NT) {
#pragma unroll
      for (int u = 0; u < KU; ++u) {
        const int i4 = base + u * NT + tid;
        kq[u] = (i4 < n4 && i4 < lim4 && lo + 4 * i4 < n) ? __ldcg(kg4 + i4) : pad4;
      }
#pragma unroll
      for (int u = 0; u < KU; ++u) {
        const int i4 = base + u * NT + tid;
        if (i4 < n4) put(i4, kq[u]);
      }
    }
  }
  if (!sz.choose) {   // uniform over the cluster: nothing to choose (kk == 0, or every position is selected)
    if (kk > 0) {
      __syncthreads();
      for (int j = 0; j < R; ++j)
        if (first + j < n) {
          idx_out[first + j] = first + j;
          if (win_out != nullptr) win_out[first + j] = my[j];
        }
    }
    return;
  }

  // ---------------------------------------------------------------- 2: the bin of the kk-th smallest key
  uint32_t want = (uint32_t)kk, count;
  {
    const uint32_t hw[8] = {hv[0].x, hv[0].y, hv[0].z, hv[0].w, hv[1].x, hv[1].y, hv[1].z, hv[1].w};
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += hw[i];
    const uint32_t inc = warp_scan_incl(sum, lane);
    if (lane == 31) sh->warp_a[warp] = inc;
    __syncthreads();   // also: the staged keys are visible
    uint32_t wv = lane < NW ? sh->warp_a[lane] : 0u;
    const uint32_t base = warp_sum(lane < warp ? wv : 0u);
    const uint32_t excl = base + inc - sum;
    if (excl < want && want <= excl + sum) {   // exactly one thread
      uint32_t run = excl;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (run < want && want <= run + hw[i]) {
          sh->sel_bin = tid * 8 + i;
          sh->sel_want = want - run;
          sh->sel_count = hw[i];
        }
        run += hw[i];
      }
    }
    __syncthreads();
  }
  const uint32_t T = sh->sel_bin;
  want = sh->sel_want;
  count = sh->sel_count;
  // bin T back into its range of keys (exact: the anchor is a small integer, the edges multiples of 1/128)
  uint32_t lo_key = (T == 0u) ? 0u : __float_as_uint(anchor + (float)T * (1.f / kBinsPerNat));
  uint32_t hi_key = (T == kBins - 1) ? kWorstKey : __float_as_uint(anchor + (float)(T + 1) * (1.f / kBinsPerNat)) - 1u;
  if (count > (uint32_t)kCandMax && lo_key != hi_key) refine(sh, keys, per, C, &lo_key, &hi_key, &want, &count);
  // count > kCandMax here means the bin is a single key value shared by all its members
  const bool ident = count > (uint32_t)kCandMax;

  // ---------------------------------------------------------------- 3: count below the bin; exchange the bin's keys
  const uint32_t span = hi_key - lo_key;
  uint32_t c_below = 0, c_in = 0;
  {
    const uint32_t seg0 = smem_u32(&sh->seg[rank][0]);
    const uint4* my4 = reinterpret_cast<const uint4*>(my);
    for (int j4 = 0; j4 < R / 4; ++j4) {        // (R is the same for every thread: whole warps stay together)
      const uint4 k4 = my4[j4];
      const uint32_t kv[4] = {k4.x, k4.y, k4.z, k4.w};
      c_below += (k4.x < lo_key) + (k4.y < lo_key) + (k4.z < lo_key) + (k4.w < lo_key);
      // inside the bin (keys below it wrap around to huge values): rare
      const bool any_in = k4.x - lo_key <= span || k4.y - lo_key <= span || k4.z - lo_key <= span || k4.w - lo_key <= span;
      if (__any_sync(0xffffffffu, any_in)) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool in = kv[e] - lo_key <= span;
          if (ident) {
            c_in += in;
            continue;
          }
          // the warp pushes its candidates together: each of them goes to peer `lane` from lane `lane`
          uint32_t slot = 0;
          if (in) slot = atomicAdd(&sh->cand_fill, 1u);
          const unsigned long long kp = ((unsigned long long)kv[e] << 32) | (uint32_t)(first + 4 * j4 + e);
          uint32_t todo = __ballot_sync(0xffffffffu, in && slot < (uint32_t)kCandMax);
          while (todo != 0u) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1u;
            const unsigned long long v = __shfl_sync(0xffffffffu, kp, src);
            const uint32_t at = __shfl_sync(0xffffffffu, slot, src);
            if (C == 1) {
              if (lane == 0) sh->seg[0][at] = v;
            } else if (lane < C) {
              asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(map_rank(seg0 + 8u * at, lane)), "l"(v) : "memory");
            }
          }
        }
      }
    }
  }
  // exclusive block scan of the counts below the bin: the thread's output offset inside the CTA, and the CTA's total
  const uint32_t inc_b = warp_scan_incl(c_below, lane);
  if (lane == 31) sh->warp_a[warp] = inc_b;
  if (ident) {
    c_in = warp_sum(c_in);
    if (lane == 0 && c_in != 0u) atomicAdd(&sh->own_in, c_in);
  }
  __syncthreads();
  uint32_t excl_below, own_below;
  {
    const uint32_t wv = lane < NW ? sh->warp_a[lane] : 0u;
    const uint32_t wi = warp_scan_incl(wv, lane);                   // lane w: keys below the bin in warps 0..w
    own_below = __shfl_sync(0xffffffffu, wi, NW - 1);
    const uint32_t before = __shfl_sync(0xffffffffu, wi, warp > 0 ? warp - 1 : 0);
    excl_below = (warp > 0 ? before : 0u) + inc_b - c_below;
  }
  {
    uint32_t own_c = ident ? sh->own_in : sh->cand_fill;
    if (!ident && own_c > (uint32_t)kCandMax) own_c = kCandMax;   // cannot happen: the bin holds at most kCandMax keys
    if (C == 1) {
      if (tid == 0) {
        sh->below[0] = own_below;
        sh->candn[0] = own_c;
      }
      __syncthreads();
    } else {
      if (tid < C) {
        st_cluster(map_rank(smem_u32(&sh->below[rank]), tid), own_below);
        st_cluster(map_rank(smem_u32(&sh->candn[rank]), tid), own_c);
      }
      cluster_arrive();
      cluster_wait();
    }
  }
  // From here on nobody touches a peer's shared memory, and every CTA of the cluster has read the histogram:
  // clear it for the next selection on this workspace (each CTA its share).
  {
    uint4* hz = reinterpret_cast<uint4*>(p.hist + bg * kBins);
    for (int i = rank * NT + tid; i < kBins / 4; i += C * NT) hz[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  uint32_t flat_base = 0, below_before = 0, total = 0;
  int src = 0;                                // (threads below the candidate count) the CTA whose segment holds candidate tid
  uint32_t pre = 0;                           // ... and the candidates of the CTAs before it
#pragma unroll
  for (int r = 0; r < kSelectCluster; ++r) {
    const uint32_t c_r = r < C ? sh->candn[r] : 0u;
    if (r < rank) {
      flat_base += c_r;
      below_before += sh->below[r];
    }
    total += c_r;
    if (r < kSelectCluster - 1 && (uint32_t)tid >= total) {
      src = r + 1;
      pre = total;
    }
  }
  if (ident) {
    write_ties(sh, my, R, first, lo_key, want, flat_base, below_before, kk, idx_out, win_out);
    return;
  }

  // ---------------------------------------------------------------- 4: which keys of the bin are selected
  // (key, position) pairs are distinct, so the `want` smallest of them - ties to the lower position - are simply
  // those of rank < want; P threads share one candidate (P a power of two, P * total <= NT).
  if (total > (uint32_t)kCandMax) total = kCandMax;
  if (tid < kCandMax) {
    unsigned long long val = ~0ull;
    if (tid < (int)total) val = sh->seg[src][tid - pre];
    sh->flat[tid] = val;
  }
  __syncthreads();
  {
    int lp = 0;                                   // log2(P)
    while (lp < 5 && ((int)total << (lp + 1)) <= NT) ++lp;
    const int ci = tid >> lp, part = tid & ((1 << lp) - 1);
    if (ci < (int)total) {                        // whole groups of P lanes take this branch together
      const unsigned long long c = sh->flat[ci];
      uint32_t less = 0;
      for (int j = part; j < (int)total; j += (1 << lp)) less += sh->flat[j] < c;
      const uint32_t gmask = __activemask();
      for (int o = 1; o < (1 << lp); o <<= 1) less += __shfl_xor_sync(gmask, less, o);
      if (part == 0 && less < want) {             // selected
        if ((uint32_t)ci < flat_base) atomicAdd(&sh->win_before, 1u);
        else if ((uint32_t)ci < flat_base + sh->candn[rank]) sh->mywin[atomicAdd(&sh->n_mywin, 1u)] = (int32_t)(uint32_t)c;
      }
    }
  }
  __syncthreads();

  // ---------------------------------------------------------------- 5: ordered output
  const int n_my = (int)sh->n_mywin;
  uint32_t offs = below_before + sh->win_before + excl_below;
  for (int i = 0; i < n_my; ++i) offs += sh->mywin[i] < first;   // selected keys of the bin that precede this thread's run
  const uint4* my4 = reinterpret_cast<const uint4*>(my);
  for (int j0 = 0; j0 < R; j0 += 32) {        // a mask of winners per 32 keys, then one store per winner
    const int qn = (R - j0 < 32 ? R - j0 : 32) / 4;
    uint32_t mask = 0;
    for (int q = 0; q < qn; ++q) {
      const uint4 k4 = my4[j0 / 4 + q];
      uint32_t nib = (uint32_t)(k4.x < lo_key) | ((uint32_t)(k4.y < lo_key) << 1) | ((uint32_t)(k4.z < lo_key) << 2) |
                     ((uint32_t)(k4.w < lo_key) << 3);
      if (k4.x - lo_key <= span || k4.y - lo_key <= span || k4.z - lo_key <= span || k4.w - lo_key <= span) {
        const uint32_t kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (kv[e] - lo_key <= span)
            for (int i = 0; i < n_my; ++i) nib |= (uint32_t)(sh->mywin[i] == first + j0 + 4 * q + e) << e;
      }
      mask |= nib << (4 * q);
    }
    while (mask != 0u) {
      const int j = __ffs(mask) - 1;
      mask &= mask - 1u;
      if (offs < (uint32_t)kk) {
        idx_out[offs] = first + j0 + j;
        if (win_out != nullptr) win_out[offs] = my[j0 + j];
      }
      ++offs;
    }
  }
}

template <int GP, bool kPool>
cudaError_t launch_score_agg(const ScoreParams& p, dim3 grid, size_t smem, cudaStream_t st) {
  switch (p.agg) {
    case RKV_AGG_MEAN: return launch_ex(score_kernel<GP, RKV_AGG_MEAN, kPool>, grid, dim3(NTS), smem, st, 1, p);
    case RKV_AGG_FIRST: return launch_ex(score_kernel<GP, RKV_AGG_FIRST, kPool>, grid, dim3(NTS), smem, st, 1, p);
    default: return launch_ex(score_kernel<GP, RKV_AGG_MAX, kPool>, grid, dim3(NTS), smem, st, 1, p);
  }
}

}  // namespace

int select_cluster_for(int n_max, int keys_per_cta) {   // CTAs per (sequence, KV head): a power of two up to 8
  int c = 1;
  while (c < kSelectCluster && ((int64_t)c * keys_per_cta < n_max || (int64_t)c * kSelectMaxKeysPerCta < n_max)) c <<= 1;
  return c;
}

int select_keys_per_thread(int n_max, int cluster) { return keys_per_thread(n_max, cluster); }

size_t select_smem_bytes(int keys_per_thr) {
  return ((sizeof(SelectShared) + 15) & ~size_t(15)) + (size_t)keys_per_thr * NT * 4;
}

cudaError_t prepare_select() {
  const int r_max = keys_per_thread(kSelectCluster * kSelectMaxKeysPerCta, kSelectCluster);
  return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)select_smem_bytes(r_max));
}

// Positions per CTA of the score pass: the smallest slice that keeps the grid within about four CTAs per SM.
int score_slice_for(int n_max, int problems, int sm_count) {
  int slice = 1024;
  while (slice < kSelectMaxSlice && (int64_t)problems * ((n_max + slice - 1) / slice) > 4 * (int64_t)sm_count) slice <<= 1;
  return slice;
}

cudaError_t launch_score(const ScoreParams& p, int n_seq, cudaStream_t st) {
  const dim3 grid(p.n_slices + (p.out != nullptr ? 2 * p.group : 0), p.n_kv_heads, n_seq);
  const size_t smem = p.pool_half > 0 ? (size_t)(p.slice + 2 * p.pool_half) * 4 : 0;
  if (p.group <= 4) {
    if (p.pool_half > 0) return launch_score_agg<4, true>(p, grid, smem, st);
    return launch_score_agg<4, false>(p, grid, smem, st);
  }
  if (p.pool_half > 0) return launch_score_agg<8, true>(p, grid, smem, st);
  return launch_score_agg<8, false>(p, grid, smem, st);
}

cudaError_t launch_select(const SelectParams& p, int n_seq, int cluster, cudaStream_t st) {
  const dim3 grid(cluster, p.n_kv_heads, n_seq);
  return launch_ex(select_kernel, grid, dim3(NT), select_smem_bytes(p.keys_per_thread), st, cluster, p);
}

}  // namespace rkv
