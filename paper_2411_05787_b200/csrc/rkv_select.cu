// Full-step epilogue: fold of the split-K partials, score finalisation and exact top-K selection.
// One thread-block cluster (8 CTAs) per (sequence, KV head).
//
// RefreshKV (arXiv 2411.05787) Sec. 2.2: the partial cache is rebuilt from the
// top-K positions of the current token's attention scores a_L; for grouped-query
// attention the scores of the query heads of a group are aggregated by max
// (footnote of Sec. 2.2; mean / first head are the ablation modes of App. A.3).
//
// Input: the scaled logits s[h][j] and the split partials the attention kernel
// wrote.  The cluster first folds the partials (CTA r produces out[] of query
// head r of the group; every CTA derives the log-sum-exp of all heads), then
//   log p[h][j] = s[h][j] - LSE[h],   ell[j] = agg_h log p[h][j],
// and the K largest scores are the K largest ell.  Selection works on a 31-bit
// fixed-point image of -ell (2^-24 resolution = 6e-8 relative in the score;
// equal images are ties and go to the lower position): a histogram pass over
// the top 11 bits, merged across the cluster through distributed shared
// memory, isolates the bin that holds the K-th key; while that bin is too
// crowded further histogram passes refine it; then the few candidates are
// pooled in CTA 0's shared memory and every CTA finishes the exact selection
// locally.  Winners are written in ascending position order (deterministic,
// and the later gather walks the cache monotonically).
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include <cstddef>

#include "rkv_fold.cuh"
#include "rkv_internal.h"

namespace cg = cooperative_groups;

namespace rkv {
namespace {

constexpr int NT = kSelectThreads;
constexpr int kBins = 2048;        // pass over bits 30..20; later passes use 1024 of them
constexpr int kCand = 2048;        // candidate pool (keys) kept in CTA 0
constexpr uint32_t kWorstKey = 0x7fffffffu;

struct SelectShared {
  alignas(16) uint32_t hist[3][kBins];   // one histogram per cluster-wide pass (kept: peers may still read them)
  alignas(16) uint32_t cand[kCand];      // CTA 0: pooled candidates; every CTA: its local copy afterwards
  alignas(16) uint32_t lhist[1024];      // local passes over the candidate pool
  alignas(16) float w[kMaxSplits * 16];  // fold weights
  alignas(16) float red[(NT / 32) * kHeadDim];
  alignas(16) double lse[kMaxGroup];
  alignas(16) float ML[16];
  uint32_t warp_tot[NT / 32];
  uint32_t peer_totals[kSelectCluster];  // per CTA of the cluster: keys below (low 16 bits) / equal to (high) the threshold key
  uint32_t cand_count;                   // CTA 0 only: pool fill
  uint32_t digit, want, count;
};
static_assert(offsetof(SelectShared, red) % 16 == 0 && offsetof(SelectShared, hist) % 16 == 0, "vector access");

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
__device__ __forceinline__ uint32_t ld_cluster(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void st_cluster(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t atom_add_cluster(uint32_t addr, uint32_t v) {
  uint32_t old;
  asm volatile("atom.shared::cluster.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
  return old;
}

// exclusive block scan of one value per thread; *total receives the block sum
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
  for (int w = 0; w < NT / 32; ++w) {
    const uint32_t t = warp_tot[w];
    if (w < warp) base += t;
    tot += t;
  }
  __syncthreads();
  *total = tot;
  return base + inc - v;
}

// Given a histogram of kB bins (4 per thread held in `mine`), find the bin holding the want-th
// smallest element; results in sh->digit / sh->want (rank inside the bin) / sh->count (bin size).
__device__ __forceinline__ void locate(SelectShared* sh, const uint32_t (&mine)[4], uint32_t want) {
  const int tid = threadIdx.x;
  const uint32_t sum = mine[0] + mine[1] + mine[2] + mine[3];
  uint32_t total;
  const uint32_t excl = block_excl_scan(sum, sh->warp_tot, &total);
  if (excl < want && want <= excl + sum) {
    uint32_t run = excl;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (run < want && want <= run + mine[i]) {
        sh->digit = tid * 4 + i;
        sh->want = want - run;
        sh->count = mine[i];
      }
      run += mine[i];
    }
  }
  __syncthreads();
}

// cluster-wide pass: every CTA has filled sh->hist[pass]; merge the 8 copies and locate the bin
__device__ __forceinline__ void cluster_pass(cg::cluster_group& cluster, SelectShared* sh, int pass, int bins,
                                             uint32_t want) {
  cluster.sync();
  const int tid = threadIdx.x;
  uint32_t mine[4] = {0u, 0u, 0u, 0u};
  if (tid * 4 < bins) {
    const uint32_t local = smem_u32(&sh->hist[pass][tid * 4]);
#pragma unroll
    for (int r = 0; r < kSelectCluster; ++r) {
      const uint4 v = ld_cluster_v4(map_rank(local, r));
      mine[0] += v.x;
      mine[1] += v.y;
      mine[2] += v.z;
      mine[3] += v.w;
    }
  }
  locate(sh, mine, want);
}

// local pass over the candidate pool: digits (key >> shift) & 1023 of candidates whose bits above match `prefix`
__device__ __forceinline__ void local_pass(SelectShared* sh, int n_cand, uint32_t prefix, int prefix_shift, int shift,
                                           uint32_t want) {
  const int tid = threadIdx.x;
  for (int i = tid; i < 1024; i += NT) sh->lhist[i] = 0;
  __syncthreads();
  for (int i = tid; i < n_cand; i += NT) {
    const uint32_t key = sh->cand[i];
    if ((key >> prefix_shift) == prefix) atomicAdd(&sh->lhist[(key >> shift) & 1023u], 1u);
  }
  __syncthreads();
  uint32_t mine[4] = {0u, 0u, 0u, 0u};
  if (tid * 4 < 1024) {
#pragma unroll
    for (int i = 0; i < 4; ++i) mine[i] = sh->lhist[tid * 4 + i];
  }
  locate(sh, mine, want);
}

template <int GMAX>
__global__ void __launch_bounds__(NT, 1) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int b = blockIdx.z, g = blockIdx.y, tid = threadIdx.x;
  pdl_launch();
  pdl_wait();
  if (p.active != nullptr && p.active[b] == 0) return;  // same decision in all CTAs of the cluster

  SelectShared* sh = reinterpret_cast<SelectShared*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + ((sizeof(SelectShared) + 15) & ~size_t(15)));

  const int G = p.group;
  int n = p.len[b];
  {
    const int cap = p.cap[b];
    const int lim = cap < p.max_len ? cap : p.max_len;
    if (n > lim) n = lim;
    if (n < 0) n = 0;
  }
  int kk = p.k_small[b];
  if (kk > p.k_max) kk = p.k_max;
  if (kk > n) kk = n;
  if (kk < 0) kk = 0;
  const int bg = b * p.n_kv_heads + g;
  int32_t* idx_out = p.topk_idx + (int64_t)bg * p.k_max;

  // padding entries
  for (int i = kk + rank * NT + tid; i < p.k_max; i += kSelectCluster * NT) idx_out[i] = -1;
  if (n == 0) return;  // the attention kernel has zeroed out[]

  // ---------------------------------------------------------------- fold the split partials
  const int n_splits = (n + p.chunk - 1) / p.chunk;
  const float* pbase = p.partials + (int64_t)bg * p.max_splits * PartialLayout::kFloats;
  auto bar = [] { __syncthreads(); };
  fold_weights<NT>(pbase, n_splits, tid, sh->w, sh->ML, bar);
  if (tid < kMaxGroup) sh->lse[tid] = (double)sh->ML[tid] + log((double)sh->ML[8 + tid]);
  if (rank < G) {  // CTA r writes the attention output of query head r of this group
    fold_out<NT, 1>(pbase, n_splits, rank, 1, tid, sh->w, sh->red, bar);
    const int64_t hrow = ((int64_t)b * p.n_q_heads + (int64_t)g * G + rank) * kHeadDim;
    if (tid < kHeadDim) {
      static_cast<__nv_bfloat16*>(p.out)[hrow + tid] = __float2bfloat16(sh->red[tid] / sh->ML[8 + rank]);
      if (p.q_last_full != nullptr)
        static_cast<__nv_bfloat16*>(p.q_last_full)[hrow + tid] = static_cast<const __nv_bfloat16*>(p.q)[hrow + tid];
    }
  }
  for (int i = tid; i < kBins; i += NT) {
    sh->hist[0][i] = 0;
    sh->hist[1][i] = 0;
    sh->hist[2][i] = 0;
  }
  if (tid == 0) sh->cand_count = 0;
  __syncthreads();

  int per = (n + kSelectCluster - 1) / kSelectCluster;
  per = (per + 3) & ~3;
  if (per > p.keys_per_cta) per = p.keys_per_cta;  // host guarantees this never bites
  const int lo = (rank * per < n) ? rank * per : n;
  const int hi = (lo + per < n) ? lo + per : n;
  const int cnt = hi - lo;

  // ---------------------------------------------------------------- keys (+ optional score output)
  const float* lg = p.logits + (int64_t)bg * G * p.logit_stride;
  float* sc = p.scores ? p.scores + (int64_t)bg * p.score_stride : nullptr;
  bool bad = false;
  const bool all_selected = (kk == n);
  const int agg = p.agg;
  double lse_r[GMAX];
#pragma unroll
  for (int h = 0; h < GMAX; ++h) lse_r[h] = sh->lse[h];
  constexpr int U = 32 / GMAX;   // positions per thread per round: all their loads are in flight together
  for (int i0 = 0; i0 < cnt; i0 += U * NT) {
    float v[U][GMAX];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT + tid;
#pragma unroll
      for (int h = 0; h < GMAX; ++h)
        v[u][h] = (h < G && i < cnt && (agg != RKV_AGG_FIRST || h == 0))
                      ? __ldcg(lg + (int64_t)h * p.logit_stride + lo + i)
                      : 0.f;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * NT + tid;
      if (i >= cnt) continue;
      double ell;
      if (agg == RKV_AGG_MAX) {
        ell = -INFINITY;
#pragma unroll
        for (int h = 0; h < GMAX; ++h) {
          if (h < G) {
            const double x = (double)v[u][h] - lse_r[h];
            if (x != x) bad = true;
            ell = fmax(ell, x);
          }
        }
      } else if (agg == RKV_AGG_MEAN) {
        double acc = 0.0;
#pragma unroll
        for (int h = 0; h < GMAX; ++h)
          if (h < G) acc += exp((double)v[u][h] - lse_r[h]);
        if (acc != acc) bad = true;
        ell = log(acc / (double)G);
      } else {
        ell = (double)v[u][0] - lse_r[0];
        if (ell != ell) bad = true;
      }
      uint32_t key;
      if (ell != ell) {
        key = kWorstKey;
      } else {
        const double uu = -ell * 16777216.0;
        key = (uu <= 0.0) ? 0u : (uu >= 2147483647.0 ? kWorstKey : (uint32_t)uu);
      }
      keys[i] = key;
      if (sc) sc[lo + i] = expf((float)ell);
      if (!all_selected) atomicAdd(&sh->hist[0][key >> 20], 1u);
    }
  }
  if (bad) atomicOr(p.status, RKV_DEV_NONFINITE);

  if (all_selected) {  // K >= n: every position is kept (uniform over the cluster)
    for (int i = tid; i < cnt; i += NT) idx_out[lo + i] = lo + i;
    return;
  }
  if (kk == 0) return;  // nothing to select (uniform over the cluster); scores and out are written

  // ---------------------------------------------------------------- locate the kk-th smallest key
  // prefix = the key's bits above `shift` that are already fixed
  cluster_pass(cluster, sh, 0, kBins, (uint32_t)kk);
  uint32_t prefix = sh->digit, want = sh->want, count = sh->count;
  int shift = 20;
  int pass = 0;
  while (count > (uint32_t)kCand && shift > 0) {  // crowded bin: refine by the next 10 bits, cluster-wide
    ++pass;
    const int nshift = shift - 10;
    for (int i = tid; i < cnt; i += NT) {
      const uint32_t key = keys[i];
      if ((key >> shift) == prefix) atomicAdd(&sh->hist[pass][(key >> nshift) & 1023u], 1u);
    }
    cluster_pass(cluster, sh, pass, 1024, want);
    prefix = (prefix << 10) | sh->digit;
    want = sh->want;
    count = sh->count;
    shift = nshift;
  }
  uint32_t tau, ties_to_take;
  if (shift == 0) {  // fully resolved by histograms (only when > kCand keys are identical in all 31 bits... or share 21)
    tau = prefix;
    ties_to_take = want;
  } else {
    // pool the candidates (keys whose fixed bits match) in CTA 0, then finish locally in every CTA
    const uint32_t pool = map_rank(smem_u32(&sh->cand[0]), 0);
    const uint32_t pool_cnt = map_rank(smem_u32(&sh->cand_count), 0);
    uint32_t mine_c = 0;
    for (int i = tid; i < cnt; i += NT) mine_c += ((keys[i] >> shift) == prefix);
    uint32_t tot_c;
    uint32_t slot = block_excl_scan(mine_c, sh->warp_tot, &tot_c);
    if (tid == 0) sh->digit = tot_c ? atom_add_cluster(pool_cnt, tot_c) : 0u;   // one reservation per CTA
    __syncthreads();
    slot += sh->digit;
    for (int i = tid; i < cnt && mine_c; i += NT) {
      const uint32_t key = keys[i];
      if ((key >> shift) == prefix) {
        if (slot < (uint32_t)kCand) st_cluster(pool + 4 * slot, key);
        ++slot;
      }
    }
    cluster.sync();
    const int n_cand = (int)(count < (uint32_t)kCand ? count : (uint32_t)kCand);
    if (rank != 0) {
      for (int i = tid; i < n_cand; i += NT) sh->cand[i] = ld_cluster(pool + 4 * i);
    }
    __syncthreads();
    while (shift > 0) {
      const int nshift = shift - 10;
      local_pass(sh, n_cand, prefix, shift, nshift, want);
      prefix = (prefix << 10) | sh->digit;
      want = sh->want;
      shift = nshift;
    }
    tau = prefix;
    ties_to_take = want;
  }

  // ---------------------------------------------------------------- ordered output
  // thread t owns positions t, t + NT, ... of a block of NT*? no: contiguous runs keep the order simple
  const int run = (cnt + NT - 1) / NT;
  const int r_lo = (tid * run < cnt) ? tid * run : cnt;
  const int r_hi = (r_lo + run < cnt) ? r_lo + run : cnt;
  uint32_t c_less = 0, c_eq = 0;
  for (int i = r_lo; i < r_hi; ++i) {
    const uint32_t key = keys[i];
    c_less += (key < tau);
    c_eq += (key == tau);
  }
  // counts fit 16 bits each (at most 40960 keys per CTA): one packed scan gives both prefixes
  uint32_t tot_packed;
  const uint32_t e_packed = block_excl_scan(c_less | (c_eq << 16), sh->warp_tot, &tot_packed);
  const uint32_t e_less = e_packed & 0xffffu, e_eq = e_packed >> 16;
  if (tid < kSelectCluster) {  // push this CTA's totals to every peer: no remote read is needed later
    const uint32_t dst = map_rank(smem_u32(&sh->peer_totals[rank]), tid);
    st_cluster(dst, tot_packed);
  }
  cluster.sync();
  uint32_t ties_before = 0, winners_before = 0, my_quota = 0;
  for (int r = 0; r <= rank; ++r) {
    const uint32_t t = sh->peer_totals[r];
    const uint32_t less_r = t & 0xffffu, eq_r = t >> 16;
    const uint32_t left = ties_to_take > ties_before ? ties_to_take - ties_before : 0u;
    const uint32_t take = left < eq_r ? left : eq_r;
    if (r < rank) {
      winners_before += less_r + take;
      ties_before += eq_r;
    } else {
      my_quota = take;
    }
  }
  // ties are kept in position order, so min(e_eq, quota) of them precede this thread's run
  uint32_t offs = winners_before + e_less + (e_eq < my_quota ? e_eq : my_quota);
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
  // no cluster barrier here: after the one above nobody touches a peer's shared memory any more
}

}  // namespace

size_t select_smem_bytes(int keys_per_cta) {
  return ((sizeof(SelectShared) + 15) & ~size_t(15)) + (size_t)keys_per_cta * 4;
}

cudaError_t prepare_select() {
  cudaError_t e = cudaFuncSetAttribute(select_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)select_smem_bytes(kSelectMaxKeysPerCta));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(select_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)select_smem_bytes(kSelectMaxKeysPerCta));
}

cudaError_t launch_select(const SelectParams& p, int n_seq, cudaStream_t st) {
  const dim3 grid(kSelectCluster, p.n_kv_heads, n_seq);
  if (p.group <= 4)
    return launch_ex(select_kernel<4>, grid, dim3(NT), select_smem_bytes(p.keys_per_cta), st, kSelectCluster, p);
  return launch_ex(select_kernel<8>, grid, dim3(NT), select_smem_bytes(p.keys_per_cta), st, kSelectCluster, p);
}

}  // namespace rkv
