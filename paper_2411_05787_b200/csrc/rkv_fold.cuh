// Folding of split-K partials (flash-decoding merge): given per-split (m_s, l_s, O_s) with
// O_s = sum_j exp(s_j - m_s) v_j over the split's positions, the merged softmax output is
//   M = max_s m_s,  w_s = exp(m_s - M),  L = sum_s l_s w_s,  out = sum_s O_s w_s / L.
// Written so that every global load of a thread is independent of the others (one L2 round
// trip), because the fold runs on the critical path at the end of a decode step.
#pragma once
#include "rkv_internal.h"

namespace rkv {

__device__ __forceinline__ float fold_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Phase 1: weights.  sm_w[s*16 + h] <- w_s for head h (h < 8), sm_ML[h] <- M, sm_ML[8+h] <- L.
// All NT threads of the block call it; `bar` synchronises exactly those threads.
template <int NT, typename Bar>
__device__ __forceinline__ void fold_weights(const float* pbase, int n_splits, int tid, float* sm_w, float* sm_ML,
                                             Bar bar) {
  constexpr float kLog2e = 1.4426950408889634f;
  for (int i = tid; i < n_splits * 16; i += NT)
    sm_w[i] = __ldcg(pbase + (int64_t)(i >> 4) * PartialLayout::kFloats + kMaxGroup * kHeadDim + (i & 15));
  bar();
  const int warp = tid >> 5, lane = tid & 31;
  for (int h = warp; h < kMaxGroup; h += NT / 32) {
    float M = -INFINITY;
    for (int s = lane; s < n_splits; s += 32) M = fmaxf(M, sm_w[s * 16 + h]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float L = 0.f;
    for (int s = lane; s < n_splits; s += 32) {
      const float ms = sm_w[s * 16 + h];
      const float e = (ms == -INFINITY) ? 0.f : fold_ex2((ms - M) * kLog2e);
      L += sm_w[s * 16 + 8 + h] * e;
      sm_w[s * 16 + h] = e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    if (lane == 0) {
      sm_ML[h] = M;
      sm_ML[8 + h] = L;
    }
  }
  bar();
}

// Phase 2: sm_red[hh * 128 + d] <- sum_s w_s O_s[h0 + hh][d] for hh < NH.  sm_red needs
// (NT / 32) * NH * 128 floats; the result sits in its first NH * 128 floats after the call.
template <int NT, int NH, typename Bar>
__device__ __forceinline__ void fold_out(const float* pbase, int n_splits, int h0, int n_heads, int tid,
                                         const float* sm_w, float* sm_red, Bar bar) {
  constexpr int NSG = NT / 32;
  const int sg = tid >> 5, d4 = (tid & 31) * 4;
  float4 acc[NH];
#pragma unroll
  for (int hh = 0; hh < NH; ++hh) acc[hh] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
  for (int s = sg; s < n_splits; s += NSG) {
    const float* ps = pbase + (int64_t)s * PartialLayout::kFloats;
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
      if (hh < n_heads) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(ps + (h0 + hh) * kHeadDim + d4));
        const float e = sm_w[s * 16 + h0 + hh];
        acc[hh].x = fmaf(v.x, e, acc[hh].x);
        acc[hh].y = fmaf(v.y, e, acc[hh].y);
        acc[hh].z = fmaf(v.z, e, acc[hh].z);
        acc[hh].w = fmaf(v.w, e, acc[hh].w);
      }
    }
  }
#pragma unroll
  for (int hh = 0; hh < NH; ++hh)
    if (hh < n_heads) *reinterpret_cast<float4*>(sm_red + ((sg * NH + hh) * kHeadDim) + d4) = acc[hh];
  bar();
  for (int i = tid; i < n_heads * kHeadDim; i += NT) {
    const int hh = i >> 7, d = i & 127;
    float sum = 0.f;
#pragma unroll
    for (int g2 = 0; g2 < NSG; ++g2) sum += sm_red[(g2 * NH + hh) * kHeadDim + d];
    // safe in place: element (0, hh, d) is read only by the thread that overwrites it
    sm_red[hh * kHeadDim + d] = sum;
  }
  bar();
}

}  // namespace rkv
