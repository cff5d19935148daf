/*
 * rkv_harness.h - C ABI of the batch-1 Llama-shaped decoder kernels that surround the RefreshKV
 * attention calls in the end-to-end decode workload (hidden 4096, 32 q / 8 kv heads of 128,
 * SwiGLU FFN, RMSNorm, rotary embedding).  The paper (arXiv 2411.05787, Sec. 3 "Inference
 * settings") runs its method inside off-the-shelf Llama-3.1-8B / Qwen2-7B; these kernels stand in
 * for the rest of such a model so that tokens/s and the attention share of a decode step can be
 * measured.  They are a measuring harness, not part of librkv.
 *
 * Conventions: every pointer is a DEVICE pointer; every call only enqueues work on the given stream
 * (cudaStream_t passed as void*) and returns 0 on success or the cudaError_t of the failed launch;
 * bad sizes return -1 before anything is launched.  Weights are bf16, row-major [out][in];
 * activations are fp32 unless stated.  Nothing is allocated; the caller owns all buffers.
 */
#ifndef RKV_HARNESS_H_
#define RKV_HARNESS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* y[i] = x[i] / sqrt(mean(x^2) + eps) * w[i];  n <= 16384, n % 4 == 0.  x, y fp32 [n]; w bf16 [n]. */
int llh_rmsnorm(const float* x, const void* w, float eps, float* y, int32_t n, void* stream);

/* y[o] = sum_i W[o][i] * x'[i] (+ residual[o]).  W bf16 [n_out][n_in], n_in % 256 == 0, n_in <= 16384.
 * x is fp32 [n_in] (x_is_bf16 == 0) or bf16 [n_in] (x_is_bf16 != 0).  With norm_w != NULL (bf16 [n_in]) the input
 * is RMS-normalised on the way in: x'[i] = x[i] / sqrt(mean(x^2) + eps) * norm_w[i]; otherwise x' = x.
 * y, residual fp32 [n_out]; residual may be NULL and may alias y (but not x). */
int llh_gemv(const void* w, const void* x, int32_t x_is_bf16, const void* norm_w, float eps, const float* residual,
             float* y, int32_t n_out, int32_t n_in, void* stream);

/* SwiGLU feed-forward input half: y[f] = silu(<Wg[f], x'>) * <Wu[f], x'>, with W = [Wg ; Wu] stacked as
 * bf16 [2 * n_ff][n_in]; silu(t) = t / (1 + exp(-t)); x' as in llh_gemv.  x fp32 [n_in], y fp32 [n_ff]. */
int llh_gemv_swiglu(const void* w_gate_up, const float* x, const void* norm_w, float eps, float* y, int32_t n_ff,
                    int32_t n_in, void* stream);

/* Rotary embedding (rotate-half pairing: channel c with c + 64, angle pos * theta^(-c/64), c < 64) of the
 * query and key heads of one token, and the split of the fused projection into bf16 tensors:
 *   qkv fp32 [(n_q + 2 n_kv) * 128] = [q heads | k heads | v heads];  pos: device int32 (token position)
 *   q bf16 [n_q][128] rotated, k bf16 [n_kv][128] rotated, v bf16 [n_kv][128] copied. */
int llh_rope_split(const float* qkv, const int32_t* pos, float theta, void* q, void* k, void* v,
                   int32_t n_q, int32_t n_kv, void* stream);

/* x[i] = table[token][i]: table bf16 [vocab][hidden], token device int32 (clamped to [0, vocab)). */
int llh_embed(const void* table, const int32_t* token, float* x, int32_t hidden, int32_t vocab, void* stream);

/* token = argmax_i logits[i] (lowest index among equal maxima); logits fp32 [n], n >= 1. */
int llh_argmax(const float* logits, int32_t n, int32_t* token, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RKV_HARNESS_H_ */
