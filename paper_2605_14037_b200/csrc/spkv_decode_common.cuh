// Declarations of the decode-attention kernel: arguments, workspace layout, block scan.
#pragma once
#include "spkv_internal.cuh"

namespace spkv {

constexpr int kMaxGrid = 256;   // blocks per decode launch (one per SM; B200 has 148)
constexpr int kMaxSlots = kMaxGrid;  // one partial slot per (block + item): see the merge
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecodeArgs {
  CacheView c;
  int layer, B, n_items, G;
  const int32_t *seq_ids;
  const __nv_bfloat16 *q;  // [B][Hq][128]
  __nv_bfloat16 *out;      // [B][Hq][128]
  float *out_f32;          // [B][Hq][128] or null: the same rows before the rounding to bf16
  float *lse;              // [B][Hq] or null
  float scale_log2;        // sm_scale * log2(e)
  int snap;                // range cuts within this many positions of a unit boundary move onto it
  int min_pos;             // positions a block takes at least when the launch has half a grid of such ranges
  int wait_mode;           // 0: griddepcontrol.wait; 1: overlap mode, wait for the launches it shares data with
  int prev_half_layer;     // layer of the decode launch that last used this workspace half (-1: none)
  int32_t *counters;       // [n_items] arrival counters
  int32_t *group_counters; // [n_items][kMaxGrid / 8] arrival counters of the first-level merge groups
  float *part_ml;          // [slots][G][2]
  float *part_acc;         // [slots][G][128]
};

// Exclusive prefix sum over s_np[0..n) -> s_pre[0..n], s_pre[n] = total.  All threads call.
__device__ inline void block_exclusive_scan(const int *s_np, int *s_pre, int n, int *s_tmp) {
  const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (n + nt - 1) / nt;
  const int a = min(tid * per, n), b = min(a + per, n);
  int sum = 0;
  for (int i = a; i < b; ++i) sum += s_np[i];
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_tmp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int v = lane < (nt >> 5) ? s_tmp[lane] : 0;
    int inc2 = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int x = __shfl_up_sync(0xffffffffu, inc2, o);
      if (lane >= o) inc2 += x;
    }
    s_tmp[32 + lane] = inc2 - v;  // exclusive offset of each warp
  }
  __syncthreads();
  int run = s_tmp[32 + warp] + incl - sum;
  for (int i = a; i < b; ++i) {
    s_pre[i] = run;
    run += s_np[i];
  }
  if (tid == nt - 1) s_pre[n] = run;
  __syncthreads();
}



struct DecodeWs {
  size_t off_gcnt, off_ml, off_acc, total;
};
inline DecodeWs decode_ws_layout(int n_items, int G) {
  DecodeWs w;
  const size_t slots = (size_t)kMaxSlots + n_items;
  w.off_gcnt = ((size_t)(n_items + 2) * 4 + 255) / 256 * 256;
  w.off_ml = w.off_gcnt + ((size_t)n_items * (kMaxGrid / 8) * 4 + 255) / 256 * 256;
  w.off_acc = w.off_ml + (slots * G * 2 * 4 + 255) / 256 * 256;
  w.total = w.off_acc + slots * G * kD * 4;
  return w;
}

}  // namespace spkv
