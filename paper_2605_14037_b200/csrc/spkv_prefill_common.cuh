// Declarations shared by the prefill kernels.
#pragma once
#include "spkv_internal.cuh"

namespace spkv {

constexpr int kHdrInts = 64;
enum { H_T0 = 0, H_LEN0, H_NOLD, H_N, H_NCOMMIT, H_LEN1, H_FAIL,
       // fp32 bit pattern of the largest finite |value| a query of this call can see: the unit's kept
       // pairs so far (plan kernel) and every staged pair, old ring and chunk (stage kernel)
       H_VMAX };

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
  int pair_tiles;                  // fp16 two-slot kernel: a single head's blocks take two query tiles each
  int n_split;                     // fp16 two-slot kernel: blocks per page walk (the most shares a walk is cut into), >= 1
  int walks_per_kvh;               //   page walks per KV head, and
  float split_unit;                //   SMs of the device (a walk's fair share of the launch = all pages / this);
                                   //   0: fewer walks than SMs, every walk is cut into runs of 16 pages
  float *partials;                 // [walk][slot][split]: 128 rows x (128 O + pad) and (m, l); n_split > 1 only
  int force_wide;                  // SPKV_FLAG_PREFILL_PV_BF16: every unit takes the two-term bf16 P.V
  // Soft-gated whole-sequence forward (spkv_softgate_forward; Eq. 6): no cache behind the call,
  // the staging sequence is the whole sequence, a query walks every causal page of it, and a key
  // beyond the query's window gets the bias gate2[key] (log2 of its gate) instead of a mask.
  int soft;
  const float *gate2;              // [Hkv][n_stage_pages * 64] (soft only)
  float *lse;                      // [C][Hq] natural-log sum-exp of the biased scaled scores, or null
  int chained;                     // host: launch the call's kernels as a chain of dependent launches (small chunks)
};

__device__ inline int32_t *unit_ws(const PrefillArgs &a, int kvh) { return a.ws + (size_t)kvh * a.ws_stride; }

// Work order of the tensor-core attention kernel (1-D grid, blocks start in index order):
// heaviest blocks first, so that the last wave is made of short ones.  A block's length is the
// number of pages it walks: KV heads are taken by descending number of kept pairs after the
// chunk (the plan kernel has counted them), and inside a head the query tiles run from the end
// of the chunk backwards.
//
// The KV head with the rank-th most keys per query in this chunk (ties by index).  Called by whole
// warps; every warp computes the same answer.  More KV heads than lanes: plain order.
__device__ inline int prefill_kvh_by_rank(const PrefillArgs &a, int rank) {
  const int lane = threadIdx.x & 31, Hkv = a.c.Hkv;
  if (Hkv > 32 || a.soft) return rank;   // (soft-gated forward: every KV head walks the same pages)
  int key = -1;
  if (lane < Hkv) {
    const int32_t *hdr = unit_ws(a, lane);
    key = hdr[H_LEN0] + hdr[kHdrInts + hdr[H_N]];
  }
  int my_rank = 0;
  for (int k = 0; k < Hkv; ++k) {
    const int other = __shfl_sync(0xffffffffu, key, k);
    my_rank += (other > key || (other == key && k < lane)) ? 1 : 0;
  }
  return __ffs(__ballot_sync(0xffffffffu, lane < Hkv && my_rank == rank)) - 1;
}
// staging pages (old ring pairs + chunk pairs as pages in the workspace), then the chunk attention
// on tcgen05 (two 128-row slots per block)
int launch_prefill_stage(const PrefillArgs &a, cudaStream_t s);
int launch_prefill_attn_tc5x2h(const PrefillArgs &a, cudaStream_t s);
size_t prefill_split_bytes(const spkv_config_t *cfg, int C);   // partial results of split page walks (small chunks)

}  // namespace spkv
