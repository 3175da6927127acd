// Step 1 of the hot path: utility logits (Eq. 1) and the threshold flag (Eq. 2).
//
// The sigmoid is monotone, so the decision u >= tau is taken as logit >= tau_logit on
// the float32 logit; the sigmoid itself is never evaluated.  bf16 inputs, float32
// accumulation in a fixed order (the result does not depend on the launch shape).
//
// Traffic: n_tok * d_in * 2 B of activations in, n_tok * n_kv_heads * 4 B out; the
// weights (a few KB to a few hundred KB) stay in L1/L2.
#include "spkv_internal.cuh"

namespace spkv {

// Linear predictor: one warp per token, all KV heads.
__global__ void __launch_bounds__(256)
score_linear_kernel(const __nv_bfloat16 *__restrict__ x, int n_tok, int d_in,
                    const __nv_bfloat16 *__restrict__ W, const float *__restrict__ b, int Hkv,
                    float tau_logit, float *__restrict__ logits, uint8_t *__restrict__ flags) {
  pdl_chain_link();
  const int lane = threadIdx.x & 31;
  const int tok = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (tok >= n_tok) return;
  const __nv_bfloat16 *xr = x + (size_t)tok * d_in;
  for (int h = 0; h < Hkv; ++h) {
    const float v = warp_dot_bf16(xr, W + (size_t)h * d_in, d_in, lane) + b[h];
    if (lane == 0) {
      logits[(size_t)tok * Hkv + h] = v;
      if (flags) flags[(size_t)tok * Hkv + h] = v >= tau_logit ? 1 : 0;
    }
  }
}

// Two-layer perceptron: one block per token; hidden activations kept in shared memory.
__global__ void __launch_bounds__(256)
score_mlp_kernel(const __nv_bfloat16 *__restrict__ x, int n_tok, int d_in,
                 const __nv_bfloat16 *__restrict__ W1, const float *__restrict__ b1, int hidden,
                 const __nv_bfloat16 *__restrict__ W2, const float *__restrict__ b2, int Hkv,
                 float tau_logit, float *__restrict__ logits, uint8_t *__restrict__ flags) {
  extern __shared__ float act[];  // [hidden]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const int tok = blockIdx.x;
  const __nv_bfloat16 *xr = x + (size_t)tok * d_in;
  for (int j = warp; j < hidden; j += n_warps) {
    const float z = warp_dot_bf16(xr, W1 + (size_t)j * d_in, d_in, lane) + b1[j];
    if (lane == 0) act[j] = z / (1.f + __expf(-z));  // SiLU
  }
  __syncthreads();
  for (int h = warp; h < Hkv; h += n_warps) {
    float acc = 0.f;
    for (int j = lane; j < hidden; j += 32)
      acc = fmaf(__bfloat162float(W2[(size_t)h * hidden + j]), act[j], acc);
    acc = warp_sum(acc) + b2[h];
    if (lane == 0) {
      logits[(size_t)tok * Hkv + h] = acc;
      if (flags) flags[(size_t)tok * Hkv + h] = acc >= tau_logit ? 1 : 0;
    }
  }
}

}  // namespace spkv

using namespace spkv;

extern "C" int spkv_score(spkv_cache_t *cache, const spkv_predictor_t *p, const void *d_x,
                          int32_t n_tok, float *d_logits_out, uint8_t *d_flags_out,
                          spkv_stream_t stream) {
  if (!cache || !p || n_tok < 0) return SPKV_E_INVALID;
  if (n_tok == 0) return SPKV_OK;
  if (!d_x || !d_logits_out || !p->d_W1 || !p->d_b1) return SPKV_E_INVALID;
  if (p->d_in < 8 || (p->d_in & 7) || ((uintptr_t)d_x & 15) || ((uintptr_t)p->d_W1 & 15))
    return SPKV_E_INVALID;
  const int Hkv = cache->view.Hkv;
  cudaStream_t s = as_stream(stream);
  cache->last_kind = kLastOther;
  const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(d_x);
  if (p->kind == 0) {
    return check_stream_error(launch_link(
        n_tok < 64, score_linear_kernel, dim3((n_tok + 7) / 8), dim3(256), 0, s, x, n_tok, (int)p->d_in,
        static_cast<const __nv_bfloat16 *>(p->d_W1), p->d_b1, Hkv, cache->tau_logit, d_logits_out, d_flags_out));
  } else if (p->kind == 1) {
    if (!p->d_W2 || !p->d_b2 || p->hidden < 1 || p->hidden > 8192) return SPKV_E_INVALID;
    // chunks of tokens at model width go to the tensor cores; a handful of tokens (decode) or an
    // unusual shape stay on the CUDA cores.  Each token is scored once, by one of the two.
    const int rc = launch_score_mlp_tc(cache, p, d_x, n_tok, d_logits_out, d_flags_out, s);
    if (rc <= 0) return rc;
    score_mlp_kernel<<<n_tok, 256, (size_t)p->hidden * 4, s>>>(
        x, n_tok, p->d_in, static_cast<const __nv_bfloat16 *>(p->d_W1), p->d_b1, p->hidden,
        static_cast<const __nv_bfloat16 *>(p->d_W2), p->d_b2, Hkv, cache->tau_logit,
        d_logits_out, d_flags_out);
  } else {
    return SPKV_E_INVALID;
  }
  return check_stream_error(cudaGetLastError());
}
