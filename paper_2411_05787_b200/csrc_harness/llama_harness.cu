// Batch-1 decoder kernels around the attention calls (see include/rkv_harness.h).
// All of them are bound by streaming bf16 weights once per token; the matrix-vector kernels keep
// two batches of 128 bytes per lane in flight, request the first one before their stream dependency
// has resolved (weights are constants) and reduce inside a warp.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rkv_harness.h"

namespace {

constexpr int kGemvThreads = 512;
constexpr int kMaxIn = 16384;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
// Programmatic dependent launch: a kernel may be scheduled while its predecessor on the stream still runs and
// waits here before it touches anything the predecessor writes.  Weights are constants, so the matrix-vector
// kernels request their first batch of weights BEFORE this wait: launch latency and the staging of x then hide
// behind the first memory round trip.  Dependents are released only after the kernel's own wait, so at most one
// earlier kernel is ever still running.  Both are no-ops for a launch without the attribute.
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

constexpr int kFly = 4;   // 16-byte chunks per lane in one batch: 2 KiB per warp, two batches in flight

// One batch of a weight row: lane l takes chunks b * 256 + l, + 32, ...  (nothing is read past the row or the matrix)
__device__ __forceinline__ void load_batch(uint4 (&u)[kFly], const uint4* __restrict__ w, int64_t row, bool row_ok,
                                           int b, int n_chunks, int lane) {
#pragma unroll
  for (int k = 0; k < kFly; ++k) {
    const int c = b * 32 * kFly + lane + 32 * k;
    u[k] = (row_ok && c < n_chunks) ? __ldcs(w + row * n_chunks + c) : make_uint4(0u, 0u, 0u, 0u);
  }
}
// <batch, x>: x sits in shared memory as fp32
__device__ __forceinline__ float batch_dot(const uint4 (&u)[kFly], const float* xs, int b, int n_chunks, int lane, float acc) {
#pragma unroll
  for (int k = 0; k < kFly; ++k) {
    const int c = b * 32 * kFly + lane + 32 * k;
    if (c < n_chunks) {
      float f[8];
      unpack8(u[k], f);
      const float4 x0 = *reinterpret_cast<const float4*>(xs + 8 * c);
      const float4 x1 = *reinterpret_cast<const float4*>(xs + 8 * c + 4);
      acc = fmaf(f[0], x0.x, acc); acc = fmaf(f[1], x0.y, acc); acc = fmaf(f[2], x0.z, acc); acc = fmaf(f[3], x0.w, acc);
      acc = fmaf(f[4], x1.x, acc); acc = fmaf(f[5], x1.y, acc); acc = fmaf(f[6], x1.z, acc); acc = fmaf(f[7], x1.w, acc);
    }
  }
  return acc;
}
// Bring x into shared memory as fp32; with a norm weight, apply RMSNorm on the way (every block recomputes the
// mean square of the few thousand inputs, which is cheaper than a separate launch).  A thread requests four 16-byte
// pieces of x (and of the norm weight) before it uses the first: a hidden-size input is one round trip to L2, the
// FFN-size input of the down projection two - not one per piece.
constexpr int kStagePieces = 4;
__device__ __forceinline__ float4 bf16x4_to_float4(uint2 u) {
  const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
  const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ void stage_x(const void* x, int x_is_bf16, const __nv_bfloat16* norm_w, float eps, float* xs,
                                        int n_in) {
  __shared__ float red[32];
  const int n4 = n_in / 4;
  float4* xs4 = reinterpret_cast<float4*>(xs);
  const uint2* wn = reinterpret_cast<const uint2*>(norm_w);
  uint2 nw[kStagePieces];          // norm weights of the first round (the only round for a hidden-size input)
  float ss = 0.f;
  for (int base = 0; base < n4; base += kStagePieces * kGemvThreads) {
    float4 v[kStagePieces];
#pragma unroll
    for (int k = 0; k < kStagePieces; ++k) {
      const int i = base + threadIdx.x + k * kGemvThreads;
      v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i < n4) v[k] = x_is_bf16 ? bf16x4_to_float4(__ldcg(static_cast<const uint2*>(x) + i))
                                   : __ldcg(static_cast<const float4*>(x) + i);
      if (norm_w != nullptr && base == 0) nw[k] = i < n4 ? __ldg(wn + i) : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int k = 0; k < kStagePieces; ++k) {
      const int i = base + threadIdx.x + k * kGemvThreads;
      if (i < n4) xs4[i] = v[k];
      ss += (v[k].x * v[k].x + v[k].y * v[k].y) + (v[k].z * v[k].z + v[k].w * v[k].w);
    }
  }
  if (norm_w != nullptr) {
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < kGemvThreads / 32; ++i) tot += red[i];
    const float r = rsqrtf(tot / (float)n_in + eps);
    for (int base = 0; base < n4; base += kStagePieces * kGemvThreads) {
#pragma unroll
      for (int k = 0; k < kStagePieces; ++k) {
        const int i = base + threadIdx.x + k * kGemvThreads;
        if (i < n4) {          // the thread's own pieces: no barrier needed in between
          const float4 wv = bf16x4_to_float4(base == 0 ? nw[k] : __ldg(wn + i));
          const float4 t = xs4[i];
          xs4[i] = make_float4(t.x * r * wv.x, t.y * r * wv.y, t.z * r * wv.z, t.w * r * wv.w);
        }
      }
    }
  }
  __syncthreads();
}

// y[o] = <W[o], x> (+ residual[o]); kSwiglu: y[f] = silu(<W[f], x>) * <W[f + n_out], x>.  A warp walks its rows
// (o = first, first + stride, ...) as one stream of weight batches: the loads of the next batch - of the same row
// or of the warp's next row - are issued before the current batch is multiplied.
template <bool kSwiglu>
__global__ void __launch_bounds__(kGemvThreads) gemv_kernel(const uint4* __restrict__ w, const void* x, int x_is_bf16,
                                                            const __nv_bfloat16* norm_w, float eps, const float* residual,
                                                            float* y, int n_out, int n_in) {
  extern __shared__ float xs[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = kGemvThreads / 32;
  const int n_chunks = n_in / 8;
  const int bpr = (n_chunks + 32 * kFly - 1) / (32 * kFly);   // batches per weight row
  const int stride = gridDim.x * wpb;
  constexpr int kParts = kSwiglu ? 2 : 1;                      // weight rows per output
  int o = blockIdx.x * wpb + warp, part = 0, b = 0;            // the batch being multiplied
  // the warp's first batch is requested before the stream dependency has resolved
  uint4 cur[kFly], nxt[kFly];
  load_batch(cur, w, (int64_t)o + (int64_t)part * n_out, o < n_out, 0, n_chunks, lane);
  dep_wait();
  dep_launch();
  stage_x(x, x_is_bf16, norm_w, eps, xs, n_in);
  float acc = 0.f, gate = 0.f;
  while (o < n_out) {
    int no = o, np = part, nb = b + 1;                         // the batch after this one
    if (nb == bpr) {
      nb = 0;
      if (++np == kParts) {
        np = 0;
        no = o + stride;
      }
    }
    load_batch(nxt, w, (int64_t)no + (int64_t)np * n_out, no < n_out, nb, n_chunks, lane);
    acc = batch_dot(cur, xs, b, n_chunks, lane, acc);
    if (b == bpr - 1) {                                        // a weight row is complete
      acc = warp_sum(acc);
      if (kSwiglu && part == 0) {
        gate = acc;
      } else if (lane == 0) {
        y[o] = kSwiglu ? gate / (1.f + __expf(-gate)) * acc : acc + (residual != nullptr ? residual[o] : 0.f);
      }
      acc = 0.f;
    }
#pragma unroll
    for (int k = 0; k < kFly; ++k) cur[k] = nxt[k];
    o = no;
    part = np;
    b = nb;
  }
}

__global__ void __launch_bounds__(1024) rmsnorm_kernel(const float* x, const __nv_bfloat16* w, float eps, float* y, int n) {
  __shared__ float red[32];
  float ss = 0.f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) ss = fmaf(x[i], x[i], ss);
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += red[i];
  const float r = rsqrtf(tot / (float)n + eps);
  for (int i = threadIdx.x; i < n; i += blockDim.x) y[i] = x[i] * r * __bfloat162float(w[i]);
}

// one thread per (head, channel pair c, c + 64); v heads are copied
__global__ void __launch_bounds__(256) rope_split_kernel(const float* qkv, const int32_t* pos, float theta, __nv_bfloat16* q,
                                                         __nv_bfloat16* k, __nv_bfloat16* v, int n_q, int n_kv) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int n_rot = (n_q + n_kv) * 64;
  dep_wait();
  dep_launch();
  if (t < n_rot) {
    const int head = t >> 6, c = t & 63;
    // the angle reaches tens of thousands of radians: form it and its sine / cosine in double
    const double ang = (double)pos[0] * pow((double)theta, -(double)c / 64.0);
    double snd, csd;
    sincos(ang, &snd, &csd);
    const float sn = (float)snd, cs = (float)csd;
    const float a = qkv[head * 128 + c], b = qkv[head * 128 + c + 64];
    __nv_bfloat16* dst = head < n_q ? q + head * 128 : k + (head - n_q) * 128;
    dst[c] = __float2bfloat16(a * cs - b * sn);
    dst[c + 64] = __float2bfloat16(b * cs + a * sn);
  } else if (t < n_rot + n_kv * 128) {
    const int i = t - n_rot;
    v[i] = __float2bfloat16(qkv[(n_q + n_kv) * 128 + i]);
  }
}

__global__ void __launch_bounds__(256) embed_kernel(const __nv_bfloat16* table, const int32_t* token, float* x, int hidden,
                                                    int vocab) {
  int tok = token[0];
  tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < hidden; i += gridDim.x * blockDim.x)
    x[i] = __bfloat162float(table[(int64_t)tok * hidden + i]);
}

__global__ void __launch_bounds__(1024) argmax_kernel(const float* logits, int n, int32_t* token) {
  __shared__ float bv[32];
  __shared__ int bi[32];
  float best = -INFINITY;
  int idx = 0x7fffffff;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {   // indices ascend, so a strict compare keeps the lowest
    const float vv = logits[i];
    if (vv > best || idx == 0x7fffffff) {
      best = vv;
      idx = i;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (ov > best || (ov == best && oi < idx)) {
      best = ov;
      idx = oi;
    }
  }
  if ((threadIdx.x & 31) == 0) {
    bv[threadIdx.x >> 5] = best;
    bi[threadIdx.x >> 5] = idx;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w2 = 1; w2 < (int)(blockDim.x >> 5); ++w2)
      if (bv[w2] > best || (bv[w2] == best && bi[w2] < idx)) {
        best = bv[w2];
        idx = bi[w2];
      }
    token[0] = idx == 0x7fffffff ? 0 : idx;
  }
}

// per-device state: SM count and whether the kernels' shared-memory attribute has been set there
constexpr int kMaxDevices = 64;
int g_sm_count[kMaxDevices] = {};
bool g_attr_set[kMaxDevices] = {};
int current_device() {
  int dev = 0;
  cudaGetDevice(&dev);
  return (dev >= 0 && dev < kMaxDevices) ? dev : 0;
}
int sm_count() {
  const int dev = current_device();
  if (g_sm_count[dev] == 0) {
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    g_sm_count[dev] = n > 0 ? n : 148;
  }
  return g_sm_count[dev];
}
int ensure_attrs() {
  const int dev = current_device();
  if (g_attr_set[dev]) return 0;
  cudaError_t e = cudaFuncSetAttribute(gemv_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxIn * 4);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemv_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxIn * 4);
  if (e != cudaSuccess) return (int)e;
  g_attr_set[dev] = true;
  return 0;
}
int gemv_grid(int n_rows) {
  const int per_block = kGemvThreads / 32;
  int blocks = (n_rows + per_block - 1) / per_block;
  const int cap = sm_count() * 2;   // two blocks of 16 warps per SM: few copies of x, many rows in flight
  return blocks < cap ? (blocks < 1 ? 1 : blocks) : cap;
}

// launch with programmatic stream serialisation (see dep_wait above)
template <bool kSwiglu>
int launch_gemv(const void* w, const void* x, int x_is_bf16, const void* norm_w, float eps, const float* residual, float* y,
                int n_out, int n_in, void* stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(gemv_grid(n_out));
  cfg.blockDim = dim3(kGemvThreads);
  cfg.dynamicSmemBytes = (size_t)n_in * 4;
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return (int)cudaLaunchKernelEx(&cfg, gemv_kernel<kSwiglu>, static_cast<const uint4*>(w), x, x_is_bf16,
                                 static_cast<const __nv_bfloat16*>(norm_w), eps, residual, y, n_out, n_in);
}

}  // namespace

extern "C" {

int llh_rmsnorm(const float* x, const void* w, float eps, float* y, int32_t n, void* stream) {
  if (!x || !w || !y || n < 4 || n > kMaxIn || n % 4) return -1;
  rmsnorm_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(x, static_cast<const __nv_bfloat16*>(w), eps, y, n);
  return (int)cudaGetLastError();
}

int llh_gemv(const void* w, const void* x, int32_t x_is_bf16, const void* norm_w, float eps, const float* residual,
             float* y, int32_t n_out, int32_t n_in, void* stream) {
  if (!w || !x || !y || n_out < 1 || n_in < 256 || n_in > kMaxIn || n_in % 256) return -1;
  if (int e = ensure_attrs()) return e;
  return launch_gemv<false>(w, x, x_is_bf16, norm_w, eps, residual, y, n_out, n_in, stream);
}

int llh_gemv_swiglu(const void* w_gate_up, const float* x, const void* norm_w, float eps, float* y, int32_t n_ff,
                    int32_t n_in, void* stream) {
  if (!w_gate_up || !x || !y || n_ff < 1 || n_in < 256 || n_in > kMaxIn || n_in % 256) return -1;
  if (int e = ensure_attrs()) return e;
  return launch_gemv<true>(w_gate_up, x, 0, norm_w, eps, nullptr, y, n_ff, n_in, stream);
}

int llh_rope_split(const float* qkv, const int32_t* pos, float theta, void* q, void* k, void* v, int32_t n_q,
                   int32_t n_kv, void* stream) {
  if (!qkv || !pos || !q || !k || !v || n_q < 1 || n_kv < 1 || !(theta > 1.f)) return -1;
  const int n = (n_q + n_kv) * 64 + n_kv * 128;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((n + 255) / 256);
  cfg.blockDim = dim3(256);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return (int)cudaLaunchKernelEx(&cfg, rope_split_kernel, qkv, pos, theta, static_cast<__nv_bfloat16*>(q),
                                 static_cast<__nv_bfloat16*>(k), static_cast<__nv_bfloat16*>(v), (int)n_q, (int)n_kv);
}

int llh_embed(const void* table, const int32_t* token, float* x, int32_t hidden, int32_t vocab, void* stream) {
  if (!table || !token || !x || hidden < 1 || vocab < 1) return -1;
  embed_kernel<<<(hidden + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(table), token, x, hidden, vocab);
  return (int)cudaGetLastError();
}

int llh_argmax(const float* logits, int32_t n, int32_t* token, void* stream) {
  if (!logits || !token || n < 1) return -1;
  argmax_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(logits, n, token);
  return (int)cudaGetLastError();
}

}  // extern "C"
