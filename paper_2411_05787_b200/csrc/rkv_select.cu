// Score finalisation + exact top-K selection, one thread-block cluster per (sequence, KV head).
//
// RefreshKV (arXiv 2411.05787) Sec. 2.2: the partial cache is rebuilt from the
// top-K positions of the current token's attention scores a_L; for grouped-query
// attention the scores of the query heads of a group are aggregated by max
// (footnote of Sec. 2.2; mean / first head are the ablation modes of App. A.3).
//
// Input: the scaled logits s[h][j] the attention kernel wrote and the
// log-sum-exp of every head.  log p[h][j] = s[h][j] - LSE[h], so the aggregated
// log-score is  ell[j] = agg_h log p[h][j]  and the K largest scores are the K
// largest ell.  Selection works on a 31-bit fixed-point image of -ell
// (2^-24 resolution, i.e. 6e-8 relative in the score; equal images are ties and
// go to the lower position), by a 3-pass radix select whose histograms are
// merged across the 8 CTAs of the cluster through distributed shared memory.
// The winners are written in ascending position order, so the result is
// deterministic and the later gather walks the cache monotonically.
#include <cooperative_groups.h>

#include "rkv_internal.h"

namespace cg = cooperative_groups;

namespace rkv {
namespace {

constexpr int kBins1 = 2048;  // bits 30..20
constexpr int kBins2 = 1024;  // bits 19..10
constexpr int kBins3 = 1024;  // bits 9..0
constexpr uint32_t kWorstKey = 0x7fffffffu;

struct SelectShared {
  uint32_t hist1[kBins1];
  uint32_t hist2[kBins2];
  uint32_t hist3[kBins3];
  uint32_t merged[kBins1];
  uint32_t warp_tot[3][8];
  uint32_t totals[2];   // this CTA's count of keys below / equal to the threshold key
  uint32_t digit;
  uint32_t want;
  double lse[kMaxGroup];
};

// exclusive block scan of one value per thread (256 threads); returns exclusive prefix, total via *total
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  uint32_t base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kSelectThreads / 32; ++w) {
    const uint32_t t = warp_tot[w];
    if (w < warp) base += t;
    tot += t;
  }
  __syncthreads();
  *total = tot;
  return base + inc - v;
}

// Merge the 8 CTAs' histograms of this pass and find the bin holding the `want`-th smallest key.
template <int kBins>
__device__ __forceinline__ void find_bin(cg::cluster_group& cluster, SelectShared* sh, uint32_t* my_hist,
                                         uint32_t want) {
  constexpr int kPer = kBins / kSelectThreads;
  const int tid = threadIdx.x;
  cluster.sync();  // every CTA's histogram of this pass is complete
  uint32_t local[kPer];
#pragma unroll
  for (int i = 0; i < kPer; ++i) local[i] = 0;
  for (int r = 0; r < kSelectCluster; ++r) {
    const uint32_t* remote = cluster.map_shared_rank(my_hist, r);
#pragma unroll
    for (int i = 0; i < kPer; ++i) local[i] += remote[tid * kPer + i];
  }
  uint32_t sum = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) sum += local[i];
  uint32_t total;
  uint32_t excl = block_excl_scan(sum, sh->warp_tot[0], &total);
  if (excl < want && want <= excl + sum) {
    uint32_t run = excl;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      if (run < want && want <= run + local[i]) {
        sh->digit = tid * kPer + i;
        sh->want = want - run;
      }
      run += local[i];
    }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kSelectThreads, 1) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int b = blockIdx.z, g = blockIdx.y, tid = threadIdx.x;
  if (p.active != nullptr && p.active[b] == 0) return;  // same decision in all CTAs of the cluster

  SelectShared* sh = reinterpret_cast<SelectShared*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + ((sizeof(SelectShared) + 15) & ~size_t(15)));

  const int G = p.group;
  int n = p.len[b];
  if (n > p.max_len) n = p.max_len;
  if (n < 0) n = 0;
  int kk = p.k_small[b];
  if (kk > p.k_max) kk = p.k_max;
  if (kk > n) kk = n;
  if (kk < 0) kk = 0;
  int32_t* idx_out = p.topk_idx + (int64_t)(b * p.n_kv_heads + g) * p.k_max;

  // padding entries
  for (int i = kk + rank * kSelectThreads + tid; i < p.k_max; i += kSelectCluster * kSelectThreads) idx_out[i] = -1;
  if (n == 0) return;

  int per = (n + kSelectCluster - 1) / kSelectCluster;
  per = (per + 3) & ~3;
  if (per > p.keys_per_cta) per = p.keys_per_cta;  // host guarantees this never bites
  const int lo = (rank * per < n) ? rank * per : n;
  const int hi = (lo + per < n) ? lo + per : n;
  const int cnt = hi - lo;

  if (tid < kMaxGroup) sh->lse[tid] = (tid < G) ? p.lse[(int64_t)b * p.n_q_heads + g * G + tid] : 0.0;
  for (int i = tid; i < kBins1; i += kSelectThreads) sh->hist1[i] = 0;
  for (int i = tid; i < kBins2; i += kSelectThreads) {
    sh->hist2[i] = 0;
    sh->hist3[i] = 0;
  }
  __syncthreads();

  // ---------------------------------------------------------------- keys (+ optional score output)
  const float* lg = p.logits + (int64_t)(b * p.n_kv_heads + g) * G * p.logit_stride;
  float* sc = p.scores ? p.scores + (int64_t)(b * p.n_kv_heads + g) * p.score_stride : nullptr;
  bool bad = false;
  const bool all_selected = (kk == n);
  for (int i = tid; i < cnt; i += kSelectThreads) {
    const int j = lo + i;
    double ell;
    if (p.agg == RKV_AGG_MAX) {
      ell = -INFINITY;
      for (int h = 0; h < G; ++h) {
        const double v = (double)lg[(int64_t)h * p.logit_stride + j] - sh->lse[h];
        if (v != v) bad = true;
        ell = fmax(ell, v);
      }
    } else if (p.agg == RKV_AGG_MEAN) {
      double acc = 0.0;
      for (int h = 0; h < G; ++h) acc += exp((double)lg[(int64_t)h * p.logit_stride + j] - sh->lse[h]);
      if (acc != acc) bad = true;
      ell = log(acc / (double)G);
    } else {
      ell = (double)lg[j] - sh->lse[0];
      if (ell != ell) bad = true;
    }
    uint32_t key;
    if (ell != ell) {
      key = kWorstKey;
    } else {
      const double u = -ell * 16777216.0;
      key = (u <= 0.0) ? 0u : (u >= 2147483647.0 ? kWorstKey : (uint32_t)u);
    }
    keys[i] = key;
    if (sc) sc[j] = (float)exp(ell);
    if (!all_selected) atomicAdd(&sh->hist1[key >> 20], 1u);
  }
  if (bad) atomicOr(p.status, RKV_DEV_NONFINITE);

  if (all_selected) {  // K >= n: every position is kept (uniform over the cluster)
    for (int i = tid; i < cnt; i += kSelectThreads) idx_out[lo + i] = lo + i;
    return;
  }

  // ---------------------------------------------------------------- 3-pass radix select of the kk-th smallest key
  find_bin<kBins1>(cluster, sh, sh->hist1, (uint32_t)kk);
  const uint32_t d1 = sh->digit;
  uint32_t want = sh->want;
  for (int i = tid; i < cnt; i += kSelectThreads) {
    const uint32_t key = keys[i];
    if ((key >> 20) == d1) atomicAdd(&sh->hist2[(key >> 10) & 1023u], 1u);
  }
  find_bin<kBins2>(cluster, sh, sh->hist2, want);
  const uint32_t d12 = (d1 << 10) | sh->digit;
  want = sh->want;
  for (int i = tid; i < cnt; i += kSelectThreads) {
    const uint32_t key = keys[i];
    if ((key >> 10) == d12) atomicAdd(&sh->hist3[key & 1023u], 1u);
  }
  find_bin<kBins3>(cluster, sh, sh->hist3, want);
  const uint32_t tau = (d12 << 10) | sh->digit;
  const uint32_t ties_to_take = sh->want;  // how many keys equal to tau are kept (lowest positions first)

  // ---------------------------------------------------------------- ordered output
  const int run = (cnt + kSelectThreads - 1) / kSelectThreads;
  const int r_lo = (tid * run < cnt) ? tid * run : cnt;
  const int r_hi = (r_lo + run < cnt) ? r_lo + run : cnt;
  uint32_t c_less = 0, c_eq = 0;
  for (int i = r_lo; i < r_hi; ++i) {
    const uint32_t key = keys[i];
    c_less += (key < tau);
    c_eq += (key == tau);
  }
  uint32_t tot_less, tot_eq;
  block_excl_scan(c_less, sh->warp_tot[1], &tot_less);
  const uint32_t e_eq = block_excl_scan(c_eq, sh->warp_tot[2], &tot_eq);
  if (tid == 0) {
    sh->totals[0] = tot_less;
    sh->totals[1] = tot_eq;
  }
  cluster.sync();
  uint32_t ties_before = 0, winners_before = 0, my_quota = 0;
  for (int r = 0; r <= rank; ++r) {
    const uint32_t* t = cluster.map_shared_rank(sh->totals, r);
    const uint32_t less_r = t[0], eq_r = t[1];
    const uint32_t left = ties_to_take > ties_before ? ties_to_take - ties_before : 0u;
    const uint32_t take = left < eq_r ? left : eq_r;
    if (r < rank) {
      winners_before += less_r + take;
      ties_before += eq_r;
    } else {
      my_quota = take;
    }
  }
  const uint32_t my_eq_take = (my_quota > e_eq) ? ((my_quota - e_eq < c_eq) ? my_quota - e_eq : c_eq) : 0u;
  uint32_t tot_w;
  uint32_t offs = block_excl_scan(c_less + my_eq_take, sh->warp_tot[0], &tot_w) + winners_before;
  uint32_t eq_seen = e_eq;
  for (int i = r_lo; i < r_hi; ++i) {
    const uint32_t key = keys[i];
    bool win = key < tau;
    if (key == tau) {
      win = eq_seen < my_quota;
      ++eq_seen;
    }
    if (win) {
      if (offs < (uint32_t)kk) idx_out[offs] = lo + i;
      ++offs;
    }
  }
  cluster.sync();  // nobody leaves while its shared memory may still be read by a peer
}

}  // namespace

size_t select_smem_bytes(int keys_per_cta) {
  return ((sizeof(SelectShared) + 15) & ~size_t(15)) + (size_t)keys_per_cta * 4;
}

cudaError_t prepare_select() {
  return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)select_smem_bytes(kSelectMaxKeysPerCta));
}

cudaError_t launch_select(const SelectParams& p, int n_seq, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kSelectCluster, p.n_kv_heads, n_seq);
  cfg.blockDim = dim3(kSelectThreads, 1, 1);
  cfg.dynamicSmemBytes = select_smem_bytes(p.keys_per_cta);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kSelectCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, select_kernel, p);
}

}  // namespace rkv
