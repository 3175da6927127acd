// Declarations shared by the decode-attention kernels (one launch per layer; the whole stack in one
// launch): arguments, workspace layout, block scan, range cuts, the merges of partial results.
#pragma once
#include "spkv_internal.cuh"
#include "spkv_mma.cuh"

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


constexpr int kConsumerWarps = 8;  // two groups of four: group g takes the pages with k % 2 == g
constexpr int kTcThreads = (kConsumerWarps + 2) * 32;  // + producer warp + epilogue warp
constexpr int kMaxStages = 8;
constexpr int kMergeCap = 256;  // (slot, head) pairs staged in shared memory by a merge
constexpr int kMergeGroup = 8;  // blocks per first-level merge group of a unit split over many blocks
constexpr int kMaxMergeGroups = kMaxGrid / kMergeGroup;
enum { F_BEGIN = 1, F_END = 2, F_STOP = 4 };

struct StageMeta {  // valid rows (bits 0-7) | flags (8-11) | item (12+); stack kernel: the page's range and layer
  int packed, chunk, layer, pad;
};

// Cut of the axis of VP positions into nb ranges: equal lengths (exact integer arithmetic,
// every block computes identical boundaries), except that a cut that falls within `snap`
// positions of a unit boundary moves onto it -- the unit is then not split, which saves two
// partial results and a merge at the price of a few pages of imbalance.  The nb + 1 cuts are
// computed once per block, in parallel, into shared memory.
__device__ inline int range_cut(int c, int nb, int VP, int snap, const int *pre, int n) {
  if (c <= 0) return 0;
  if (c >= nb) return VP;
  const int p = (int)(((unsigned long long)(unsigned)c * (unsigned)VP) / (unsigned)nb);
  int lo = 0, hi = n;  // unit containing position p
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (pre[mid] <= p) lo = mid; else hi = mid;
  }
  if (p - pre[lo] <= snap) return pre[lo];
  if (pre[lo + 1] - p <= snap) return pre[lo + 1];
  return p;
}
struct Ranges {
  int nb;
  const int *cut;  // [nb + 1], non-decreasing, cut[0] = 0, cut[nb] = VP
  __device__ int start(int c) const { return cut[min(c, nb)]; }
  // last block c with cut[c] <= p (its range is non-empty).  The cuts sit within `snap` positions
  // of c * VP / nb, so the proportional guess is off by a step or two at most.
  __device__ int of_pos(int p) const {
    const unsigned VP = (unsigned)cut[nb];
    int c = min(nb - 1, (int)(((unsigned long long)(unsigned)p * (unsigned)nb) / VP));
    while (c > 0 && cut[c] > p) --c;
    while (c + 1 < nb && cut[c + 1] <= p) ++c;
    return c;
  }
};

// false (and the sticky status set) if the wait ran out
__device__ inline bool wait_or_flag(uint64_t *bar, uint32_t parity, const CacheView &c) {
  if (mbar_wait_bounded(bar, parity)) return true;
  set_status(c, SPKV_E_TIMEOUT);
  return false;
}

// Epilogue warp: merge the consumer warps' (m, l, O) of one finished segment for all GG heads of
// the group, fully unrolled so that every shared-memory load is issued before the first use
// (a loop over the heads pays the load latency once per head and lets finished segments queue
// up behind the epilogue warp when a block's range ends in several short units).
template <int GG>
__device__ inline void merge_warps(const float *red, int GP, int lane, float (&M)[GG], float (&Ls)[GG],
                                   float4 (&Os)[GG]) {
  float m[kConsumerWarps][GG], l[kConsumerWarps][GG];
  float4 v[kConsumerWarps][GG];
#pragma unroll
  for (int w4 = 0; w4 < kConsumerWarps; ++w4)
#pragma unroll
    for (int gh = 0; gh < GG; ++gh) {
      const float *src = red + ((size_t)w4 * GP + gh) * 132;
      m[w4][gh] = src[128];
      l[w4][gh] = src[129];
      v[w4][gh] = *reinterpret_cast<const float4 *>(src + lane * 4);
    }
#pragma unroll
  for (int gh = 0; gh < GG; ++gh) {
    M[gh] = -INFINITY;
#pragma unroll
    for (int w4 = 0; w4 < kConsumerWarps; ++w4) M[gh] = fmaxf(M[gh], m[w4][gh]);
    Ls[gh] = 0.f;
    Os[gh] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w4 = 0; w4 < kConsumerWarps; ++w4) {
      const float f = m[w4][gh] == -INFINITY ? 0.f : fast_exp2(m[w4][gh] - M[gh]);
      Ls[gh] += l[w4][gh] * f;
      Os[gh].x += v[w4][gh].x * f; Os[gh].y += v[w4][gh].y * f;
      Os[gh].z += v[w4][gh].z * f; Os[gh].w += v[w4][gh].w * f;
    }
  }
}

// Merge of `cnt` partial slots (slot si at row offset si * stride slots from g_acc) for all GG heads
// of a group.  s_ml: the (m, l) pairs staged in shared memory, [cnt][GG].  The accumulator rows
// are fetched 16 at a time with unconditional loads (indices past the end are clamped and get
// weight 0), so every load of a round is in flight before the first use: a round costs one
// trip to L2 whatever the shape.  Lane l owns dims 4l..4l+3.
template <int GG>
__device__ inline void merge_rows(const float *g_acc /* first slot, + lane * 4 */, const float2 *s_ml, int stride,
                                  int cnt, float (&M)[GG], float (&L)[GG], float4 (&O)[GG]) {
  constexpr int NS = 16 / GG;
#pragma unroll
  for (int gh = 0; gh < GG; ++gh) {
    M[gh] = -INFINITY;
    L[gh] = 0.f;
    O[gh] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int si = 0; si < cnt; ++si)
#pragma unroll
    for (int gh = 0; gh < GG; ++gh) M[gh] = fmaxf(M[gh], s_ml[si * GG + gh].x);
  for (int s0 = 0; s0 < cnt; s0 += NS) {
    float4 v[NS][GG];
#pragma unroll
    for (int x = 0; x < NS; ++x) {
      const size_t row = (size_t)min(s0 + x, cnt - 1) * stride * GG;
#pragma unroll
      for (int gh = 0; gh < GG; ++gh) v[x][gh] = __ldcg(reinterpret_cast<const float4 *>(g_acc + (row + gh) * kD));
    }
#pragma unroll
    for (int x = 0; x < NS; ++x)
#pragma unroll
      for (int gh = 0; gh < GG; ++gh) {
        const float2 ml = s_ml[min(s0 + x, cnt - 1) * GG + gh];
        const float f = (s0 + x < cnt && ml.x != -INFINITY) ? fast_exp2(ml.x - M[gh]) : 0.f;
        L[gh] += ml.y * f;
        O[gh].x += v[x][gh].x * f; O[gh].y += v[x][gh].y * f; O[gh].z += v[x][gh].z * f; O[gh].w += v[x][gh].w * f;
      }
  }
}


// ---- the consumer warps' state for one segment (shared by the per-layer and the stack kernel) ----
// A consumer warp keeps, for its 16 of every page's 64 pairs, the query fragments of the group's
// heads (qb) and the running maximum, sum and output accumulators (m, l, o) in the MMA tiles'
// register layout: lane = 4 g + t4 holds heads 2 t4, 2 t4 + 1 of every 8-head tile.

// First page of a segment: the group's query rows (in the stage, behind the page) -> fragments;
// accumulators cleared.
template <int NH>
__device__ inline void segment_begin(uint32_t (&qb)[NH][8][2], float (&m)[NH][2], float (&l)[NH][2],
                                     float (&o)[NH][8][4], const __nv_bfloat16 *qs, int GP, int lane) {
  load_q_frags_t<NH>(qb, [&](int h) -> const __nv_bfloat16 * { return h < GP ? qs + h * kD : nullptr; }, lane);
#pragma unroll
  for (int hn = 0; hn < NH; ++hn) {
    m[hn][0] = m[hn][1] = -INFINITY;
    l[hn][0] = l[hn][1] = 0.f;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) o[hn][mt][0] = o[hn][mt][1] = o[hn][mt][2] = o[hn][mt][3] = 0.f;
  }
}

// Last page of a segment: this warp's (m, l, O) of the G heads into its rows of the hand-over
// buffer `red` ([warp][GP][132]: 128 output dims, then m and l), for the epilogue warp.
template <int NH>
__device__ inline void segment_hand_over(float *red, int warp, int GP, int G, const float (&m)[NH][2],
                                         const float (&l)[NH][2], const float (&o)[NH][8][4], int lane) {
  const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
  for (int hn = 0; hn < NH; ++hn)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float lv = l[hn][j];
      lv += __shfl_xor_sync(0xffffffffu, lv, 4);
      lv += __shfl_xor_sync(0xffffffffu, lv, 8);
      lv += __shfl_xor_sync(0xffffffffu, lv, 16);
      const int h = hn * 8 + t4 * 2 + j;
      if (h < G) {
        float *dst = red + ((size_t)warp * GP + h) * 132;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          dst[mt * 16 + g] = o[hn][mt][j];
          dst[mt * 16 + 8 + g] = o[hn][mt][2 + j];
        }
        if (g == 0) { dst[128] = m[hn][j]; dst[129] = lv; }
      }
    }
}

// Where the segments of one launch (or of one layer of a stack launch) put their results.
struct SegOut {
  __nv_bfloat16 *out;       // [B][Hq][128]
  float *out_f32;           // or null
  float *lse;               // or null
  int32_t *counters;        // [n_items]
  int32_t *group_counters;  // [n_items][kMaxMergeGroups]
  float *part_ml;           // [slots][G][2]
  float *part_acc;          // [slots][G][128]
};

// The epilogue warp's work for one finished segment -- the piece of unit `item` that lies in
// range `cidx`: merges the consumer warps' (m, l, O) from `red` (lane l owns dims 4l..4l+3), gives
// the buffer back (red_release), writes the output rows or, for a unit that sticks out of the
// range, the partial result, counts itself in on the unit and, if it arrived last, merges the
// unit's partials by their log-sum-exp weights (on two levels for a unit cut into many ranges).
// rg, s_pre: the launch's (layer's) range cuts and position prefix sums.
__device__ inline void finish_segment(const CacheView &c, int G, int GP, const SegOut &o, const Ranges &rg,
                                      const int *s_pre, const float *red, float2 *s_mrg, uint64_t *red_release,
                                      int item, int cidx, int lane) {
  const int b = item / c.Hkv, kvh = item % c.Hkv;
  // blocks that share the unit (searched only when it sticks out of this block's range)
  const int u_first = s_pre[item] + 1, u_last = s_pre[item + 1] - 1;
  const int c_first = u_first >= rg.start(cidx) ? cidx : rg.of_pos(u_first);
  const int c_last = u_last < rg.start(cidx + 1) ? cidx : rg.of_pos(u_last);
  const int nseg = c_last - c_first + 1;
  const int slot = cidx + item;
  // writes one head's merged result: the output if the unit lies inside this block, else a partial
  auto emit = [&](int gh, float M, float Ls, const float4 &Os) {
    const size_t row = (size_t)b * c.Hq + kvh * G + gh;
    if (nseg == 1) {
      const float inv = 1.f / Ls;
      uint2 pk;
      pk.x = pack_bf16(Os.x * inv, Os.y * inv);
      pk.y = pack_bf16(Os.z * inv, Os.w * inv);
      *reinterpret_cast<uint2 *>(o.out + row * kD + lane * 4) = pk;
      if (o.out_f32)
        *reinterpret_cast<float4 *>(o.out_f32 + row * kD + lane * 4) =
            make_float4(Os.x * inv, Os.y * inv, Os.z * inv, Os.w * inv);
      if (o.lse && lane == 0) o.lse[row] = (M + log2f(Ls)) * kLn2;
    } else {
      *reinterpret_cast<float4 *>(o.part_acc + ((size_t)slot * G + gh) * kD + lane * 4) = Os;
      if (lane == 0) {
        o.part_ml[((size_t)slot * G + gh) * 2 + 0] = M;
        o.part_ml[((size_t)slot * G + gh) * 2 + 1] = Ls;
      }
    }
  };
  if (G == 4) {
    float M[4], Ls[4];
    float4 Os[4];
    merge_warps<4>(red, GP, lane, M, Ls, Os);
#pragma unroll
    for (int gh = 0; gh < 4; ++gh) emit(gh, M[gh], Ls[gh], Os[gh]);
  } else if (G == 2) {
    float M[2], Ls[2];
    float4 Os[2];
    merge_warps<2>(red, GP, lane, M, Ls, Os);
#pragma unroll
    for (int gh = 0; gh < 2; ++gh) emit(gh, M[gh], Ls[gh], Os[gh]);
  } else {
    int gh = 0;
    for (; gh + 4 <= G; gh += 4) {  // G = 8, 12, 16: four heads at a time
      float M[4], Ls[4];
      float4 Os[4];
      merge_warps<4>(red + (size_t)gh * 132, GP, lane, M, Ls, Os);
#pragma unroll
      for (int x = 0; x < 4; ++x) emit(gh + x, M[x], Ls[x], Os[x]);
    }
    for (; gh < G; ++gh) {
      float M[1], Ls[1];
      float4 Os[1];
      merge_warps<1>(red + (size_t)gh * 132, GP, lane, M, Ls, Os);
      emit(gh, M[0], Ls[0], Os[0]);
    }
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(red_release);  // the consumers may fill the buffer again
  if (nseg > 1) {
    // Merge of `cnt` partial slots first, first + stride, ... of this unit (one warp; lane l owns
    // dims 4l..4l+3).  dst_slot < 0: normalise and write the output rows; otherwise write the
    // merged (m, l, O) back as a partial into dst_slot.
    auto merge_slots = [&](int first, int stride, int cnt, int dst_slot) {
      // (m, l) of every slot and head go through shared memory first (one round of loads for
      // the whole warp); the accumulator loads below are then independent
      const int n_ml = cnt * G;
      const bool staged = n_ml <= kMergeCap;
      const float2 *g_ml = reinterpret_cast<const float2 *>(o.part_ml) + (size_t)first * G;
      if (staged) {
        for (int idx = lane; idx < n_ml; idx += 32)
          s_mrg[idx] = __ldcg(g_ml + (size_t)(idx / G) * stride * G + idx % G);
        __syncwarp();
      }
      const float *g_acc = o.part_acc + (size_t)first * G * kD + lane * 4;
      auto ml_of = [&](int si, int gh) {
        return staged ? s_mrg[si * G + gh] : __ldcg(g_ml + ((size_t)si * stride) * G + gh);
      };
      const size_t row0 = (size_t)b * c.Hq + kvh * G;
      // writes one head's merged (m, l, O): normalised output row, or a partial into dst_slot
      auto put = [&](int gh, float Mx, float Ls, const float4 &Os) {
        if (dst_slot < 0) {
          const float inv = 1.f / Ls;
          uint2 pk;
          pk.x = pack_bf16(Os.x * inv, Os.y * inv);
          pk.y = pack_bf16(Os.z * inv, Os.w * inv);
          *reinterpret_cast<uint2 *>(o.out + (row0 + gh) * kD + lane * 4) = pk;
          if (o.out_f32)
            *reinterpret_cast<float4 *>(o.out_f32 + (row0 + gh) * kD + lane * 4) =
                make_float4(Os.x * inv, Os.y * inv, Os.z * inv, Os.w * inv);
          if (o.lse && lane == 0) o.lse[row0 + gh] = (Mx + log2f(Ls)) * kLn2;
        } else {
          *reinterpret_cast<float4 *>(o.part_acc + ((size_t)dst_slot * G + gh) * kD + lane * 4) = Os;
          if (lane == 0) {
            o.part_ml[((size_t)dst_slot * G + gh) * 2 + 0] = Mx;
            o.part_ml[((size_t)dst_slot * G + gh) * 2 + 1] = Ls;
          }
        }
      };
      if (staged && (G == 1 || G == 2 || G == 4 || G == 8)) {
        if (G == 4) {
          float M[4], L[4]; float4 O[4];
          merge_rows<4>(g_acc, s_mrg, stride, cnt, M, L, O);
#pragma unroll
          for (int gh = 0; gh < 4; ++gh) put(gh, M[gh], L[gh], O[gh]);
        } else if (G == 8) {
          float M[8], L[8]; float4 O[8];
          merge_rows<8>(g_acc, s_mrg, stride, cnt, M, L, O);
#pragma unroll
          for (int gh = 0; gh < 8; ++gh) put(gh, M[gh], L[gh], O[gh]);
        } else if (G == 2) {
          float M[2], L[2]; float4 O[2];
          merge_rows<2>(g_acc, s_mrg, stride, cnt, M, L, O);
#pragma unroll
          for (int gh = 0; gh < 2; ++gh) put(gh, M[gh], L[gh], O[gh]);
        } else {
          float M[1], L[1]; float4 O[1];
          merge_rows<1>(g_acc, s_mrg, stride, cnt, M, L, O);
          put(0, M[0], L[0], O[0]);
        }
        return;
      }
      // general case: two heads x eight slots at a time, 16 independent 16-byte loads in flight
      for (int gh0 = 0; gh0 < G; gh0 += 2) {
        float Mx[2], Ls[2];
        float4 Os[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          Mx[h] = -INFINITY; Ls[h] = 0.f; Os[h] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (gh0 + h < G)
            for (int si = 0; si < cnt; ++si) Mx[h] = fmaxf(Mx[h], ml_of(si, gh0 + h).x);
        }
        for (int s0 = 0; s0 < cnt; s0 += 8) {
          float4 v[8][2];
#pragma unroll
          for (int x = 0; x < 8; ++x)
#pragma unroll
            for (int h = 0; h < 2; ++h)
              v[x][h] = (s0 + x < cnt && gh0 + h < G)
                            ? __ldcg(reinterpret_cast<const float4 *>(
                                  g_acc + (((size_t)(s0 + x) * stride) * G + gh0 + h) * kD))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int x = 0; x < 8; ++x)
#pragma unroll
            for (int h = 0; h < 2; ++h)
              if (s0 + x < cnt && gh0 + h < G) {
                const float2 ml = ml_of(s0 + x, gh0 + h);
                const float f = ml.x == -INFINITY ? 0.f : fast_exp2(ml.x - Mx[h]);
                Ls[h] += ml.y * f;
                Os[h].x += v[x][h].x * f; Os[h].y += v[x][h].y * f;
                Os[h].z += v[x][h].z * f; Os[h].w += v[x][h].w * f;
              }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h)
          if (gh0 + h < G) put(gh0 + h, Mx[h], Ls[h], Os[h]);
      }
    };
    // this block's arrival on a counter; true for the last of `target` arrivals (which also
    // resets the counter for the next launch)
    auto arrive_last = [&](int32_t *counter, int target) {
      // The warp's partial stores are ordered before lane 0's release by the warp barrier
      // (release is cumulative), and the other lanes' later loads after its acquire the same
      // way: one acq_rel atomic instead of fence + atomic + fence.
      __syncwarp();
      int last = 0;
      if (lane == 0) {
        int old;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
        last = old == target - 1;
        if (last) *counter = 0;
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      return last != 0;
    };
    // A unit split over up to kMergeGroup blocks is merged by its last arriver.  A longer one
    // (a near-full head at 128 K spans dozens of blocks) is merged on two levels, so that no
    // single warp has to pull dozens of partials through its own few loads in flight: the
    // parts form groups of kMergeGroup consecutive blocks, the last arriver of a group merges
    // it into the group's first slot, and the last group to finish merges the group results.
    const int first_slot = c_first + item, part = cidx - c_first;
    if (nseg <= kMergeGroup) {
      if (arrive_last(&o.counters[item], nseg)) {
        merge_slots(first_slot, 1, nseg, -1);
      }
    } else {
      const int g = part / kMergeGroup, n_groups = (nseg + kMergeGroup - 1) / kMergeGroup;
      const int g_parts = min(kMergeGroup, nseg - g * kMergeGroup);
      if (arrive_last(&o.group_counters[(size_t)item * kMaxMergeGroups + g], g_parts)) {
        if (g_parts > 1) merge_slots(first_slot + g * kMergeGroup, 1, g_parts, first_slot + g * kMergeGroup);
        if (arrive_last(&o.counters[item], n_groups)) merge_slots(first_slot, kMergeGroup, n_groups, -1);
      }
    }
  }
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
