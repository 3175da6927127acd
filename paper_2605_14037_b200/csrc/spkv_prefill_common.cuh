// Declarations shared by the prefill kernels.
#pragma once
#include "spkv_internal.cuh"

namespace spkv {

constexpr int kHdrInts = 64;
enum { H_T0 = 0, H_LEN0, H_NOLD, H_N, H_NCOMMIT, H_LEN1, H_FAIL };

struct PrefillArgs {
  CacheView c;
  int layer, seq, C;
  const __nv_bfloat16 *q, *k, *v;  // [C][Hq][128], [C][Hkv][128]
  const float *logits;             // [C][Hkv]
  __nv_bfloat16 *out;              // [C][Hq][128]
  float tau_logit, scale_log2;
  int32_t *ws;                     // [Hkv][ws_stride]
  int ws_stride;
  __nv_bfloat16 *stage_pages;      // [Hkv][n_stage_pages] pages: old ring pairs + chunk pairs in
  int n_stage_pages;               //   position order, page format (tensor-core kernel only)
};

__device__ inline int32_t *unit_ws(const PrefillArgs &a, int kvh) { return a.ws + (size_t)kvh * a.ws_stride; }


// staging pages + chunk attention on tcgen05 (two heads per block when G is even)
int launch_prefill_attn_tc5(const PrefillArgs &a, cudaStream_t s);
int launch_prefill_attn_tc5x2(const PrefillArgs &a, cudaStream_t s);

}  // namespace spkv
