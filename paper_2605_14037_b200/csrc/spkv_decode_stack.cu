// One decode step of a whole attention-only layer stack in two launches (spkv_decode_stack):
// the appends of every layer (append_stack_kernel), then ONE persistent decode-attention
// kernel over all layers (Eq. 3-5 per layer, exactly what spkv_decode_attention computes).
//
// Why.  Launched layer by layer, a decode block spends ~7 us before its first page arrives
// (lengths, prefix sums, range cuts, page-table entry, HBM latency) and ~4 us after its last page
// waiting for its own epilogue warp (partial result, arrival count, perhaps a merge), and the next
// launch's block cannot start on the SM before it has left: 11 of every ~66 us at the 32 K
// workload, on every SM, with nothing streaming.  Here the block never leaves.  Per layer the
// page axis is cut exactly as in the per-layer kernel (units laid end to end, one marker
// position each, equal ranges snapped to unit boundaries); the ranges of all layers form one
// list, layer after layer, and a block takes the next one from an atomic counter whenever its
// producer has resolved the previous one.  So
//   - the page stream of a block runs on across range and layer boundaries: the producer warp
//     issues the first pages of the next range while the consumers still work on the last pages of
//     this one and the epilogue warp on its result;
//   - the lengths, prefix sums and cuts of layer l + 1 are worked out by a warp of their own (the
//     planner) while layer l streams;
//   - SMs that stream faster take more ranges (under full load the fastest SM of a B200 draws
//     about a fifth more than the mean, the slowest a fifth less, by position on the chip).
// Every layer's appends have finished before this kernel starts (stream order), so all blocks
// compute identical plans and nobody waits for another block: partial results and arrival
// counters live in per-layer regions of the workspace, merged by whoever arrives last.
//
// Warps: 8 consumers (two groups taking alternate pages), producer, epilogue, planner.
// Shared memory: page stages, two hand-over buffers, two to four plans (layer modulo their number).
// Hand-shakes inside the block (mbarriers, every wait bounded):
//   plan_ready[p]  planner -> producer: the plan in buffer p is complete;
//   plan_free[p]   epilogue -> planner: nobody needs that plan any more.  The producer sends a
//                  marker down the page pipeline when it moves on to the next layer; the
//                  consumers pass it on, and the epilogue warp, which sees it after the last segment
//                  of the layer, gives the plan back.  Every block visits every layer in order,
//                  with or without ranges of its own there, so the phases of both barriers
//                  advance in step.
#include "spkv_decode_common.cuh"

namespace spkv {

constexpr int kStackThreads = (kConsumerWarps + 3) * 32;  // + producer, epilogue, planner
constexpr int kMaxPlans = 4;  // plan buffers: the planner may be this many layers ahead of the epilogue warp
enum { F_LAYER = 8 };  // stage flag: no page, "the producer has left this layer"

struct StackArgs {
  CacheView c;
  int layer0, n_layers, B, n_items, G;   // layers layer0 ... layer0 + n_layers - 1 of the cache
  const int32_t *seq_ids;
  const __nv_bfloat16 *q;  // [L][B][Hq][128], first row: layer0's
  __nv_bfloat16 *out;      // [L][B][Hq][128]
  float *lse;              // [L][B][Hq] or null
  float scale_log2;
  int snap, min_pos;
  int nb;                  // ranges per layer in the list (a layer with fewer leaves the rest empty)
  int32_t *claim;          // the launch's range counter
  char *ws;                // per-layer regions (from layer0's on): arrival counters, partial results
  size_t ws_layer_bytes, off_gcnt, off_ml, off_acc;
};

struct StackPlan {  // offsets (ints) inside one plan
  int hdr, pre, unit, len, ring, row, cut, ints;
};
__host__ __device__ inline StackPlan stack_plan_layout(int n) {
  StackPlan p;
  int o = 0;
  p.hdr = o;  o += 4;  // VP, nb_eff
  p.pre = o;  o += n + 1;
  p.unit = o; o += n;
  p.len = o;  o += n;
  p.ring = o; o += n;
  p.row = o;  o += n;
  p.cut = o;  o += kMaxGrid + 1;
  p.ints = (o + 3) / 4 * 4;
  return p;
}

struct StackSmem {
  int n_stages, n_plans, stage_bytes, off_bar, off_meta, off_seq, off_np, off_plan, plan_bytes, off_red, off_mrg, off_flags,
      total;
};
__host__ __device__ inline StackSmem stack_smem_layout(int n_items, int B, int GP, int n_stages, int n_plans) {
  StackSmem L;
  L.n_stages = n_stages;
  L.n_plans = n_plans;
  L.stage_bytes = kPageBytes + GP * kRowBytes;
  int o = n_stages * L.stage_bytes;
  o = (o + 15) / 16 * 16;
  L.off_bar = o;   o += (2 * kMaxStages + 4 + 2 * kMaxPlans) * 8;  // full[], empty[], red_full[2], red_empty[2], plan_ready[], plan_free[]
  L.off_meta = o;  o += kMaxStages * (int)sizeof(StageMeta);
  L.off_seq = o;   o += B * 4;
  L.off_np = o;    o += n_items * 4;
  o = (o + 15) / 16 * 16;
  L.plan_bytes = stack_plan_layout(n_items).ints * 4;
  L.off_plan = o;  o += n_plans * L.plan_bytes;
  L.off_red = o;   o += 2 * kConsumerWarps * GP * 132 * 4;
  L.off_mrg = o;   o += kMergeCap * 8;
  L.off_flags = o; o += 32;
  L.total = o;
  return L;
}

template <int NH>  // 8-head tiles on the N side: 1 for G <= 8, 2 for G <= 16
__global__ void __launch_bounds__(kStackThreads, 1)
decode_stack_kernel(StackArgs a, int GP, int n_stages, int n_plans) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const CacheView &c = a.c;
  const int n = a.n_items;
  const StackSmem L = stack_smem_layout(n, a.B, GP, n_stages, n_plans);
  const StackPlan PL = stack_plan_layout(n);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + L.off_bar);
  uint64_t *empty = full + kMaxStages;
  uint64_t *red_full = empty + kMaxStages, *red_empty = red_full + 2;
  uint64_t *plan_ready = red_empty + 2, *plan_free = plan_ready + kMaxPlans;
  volatile StageMeta *s_meta = reinterpret_cast<volatile StageMeta *>(smem + L.off_meta);
  int *s_seq = reinterpret_cast<int *>(smem + L.off_seq);
  int *s_np = reinterpret_cast<int *>(smem + L.off_np);
  float *s_red = reinterpret_cast<float *>(smem + L.off_red);
  float2 *s_mrg = reinterpret_cast<float2 *>(smem + L.off_mrg);
  volatile int *s_redmeta = reinterpret_cast<volatile int *>(smem + L.off_flags);  // [rb]: item, [2+rb]: range, [4+rb]: layer
  auto plan_of = [&](int layer) { return reinterpret_cast<int *>(smem + L.off_plan + (layer % n_plans) * L.plan_bytes); };

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NB = a.nb;                           // ranges per layer in the global numbering
  const int n_ranges = a.n_layers * NB;

  if (tid == 0) {
    for (int i = 0; i < n_stages; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], kConsumerWarps);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&red_full[i], kConsumerWarps);
      mbar_init(&red_empty[i], 1);
    }
    for (int i = 0; i < n_plans; ++i) {
      mbar_init(&plan_ready[i], 1);
      mbar_init(&plan_free[i], 1);
    }
    mbar_fence_init();
  }
  // query rows past the group size are never written by a copy: zero them once
  for (int i = tid; i < n_stages * (GP - a.G) * (kRowBytes / 16); i += kStackThreads) {
    const int per = (GP - a.G) * (kRowBytes / 16);
    const int st = i / per, r = i % per;
    reinterpret_cast<uint4 *>(smem + (size_t)st * L.stage_bytes + kPageBytes + a.G * kRowBytes)[r] =
        make_uint4(0, 0, 0, 0);
  }
  for (int i = tid; i < a.B; i += kStackThreads) s_seq[i] = a.seq_ids[i];
  // Everything above touched only this block's shared memory and an input of the call; the launch
  // is a programmatic dependent one, so it may have run under the tail of the append launch.  From
  // here on the cache is read: wait for that launch (and everything before it) to complete.
  pdl_wait();
  __syncthreads();

  if (warp == kConsumerWarps + 2) {
    // ------------------------------------------------------------------- planner warp
    // Layer by layer: every unit's page count, the prefix sums over (pages + 1 marker), the range
    // cuts -- what the per-layer kernel's whole block does before its first page, here by one warp
    // while the previous layer streams.
    for (int l = 0; l < a.n_layers; ++l) {
      if (l >= n_plans && !wait_or_flag(&plan_free[l % n_plans], ((l / n_plans) - 1) & 1, c)) break;
      int *P = plan_of(l);
      for (int i = lane; i < n; i += 32) {
        const int b = i / c.Hkv, kvh = i % c.Hkv;
        const int seq = s_seq[b];
        int np = 0, u = 0, len = 0, n_ring = 0, trow = -1;
        if (seq >= 0 && seq < c.S) {
          u = unit_index(c, a.layer0 + l, seq, kvh);
          trow = unit_table_row(c, u);
          len = ldcg_keep(&c.len[u]);
          n_ring = min(ldcg_keep(&c.t[u]), c.w);
          np = (len + kP - 1) / kP + (n_ring + kP - 1) / kP;
        } else if (blockIdx.x == 0) {
          set_status(c, SPKV_E_BOUNDS);
        }
        s_np[i] = np > 0 ? np + 1 : 0;  // + the marker position
        P[PL.unit + i] = u; P[PL.len + i] = len; P[PL.ring + i] = n_ring; P[PL.row + i] = trow;
        if (np == 0 && blockIdx.x == 0) {  // nothing to attend to: defined output
          for (int g = 0; g < a.G; ++g) {
            const size_t row = ((size_t)l * a.B + b) * c.Hq + kvh * a.G + g;
            for (int d = 0; d < kD; ++d) a.out[row * kD + d] = __float2bfloat16(0.f);
            if (a.lse) a.lse[row] = -INFINITY;
          }
        }
      }
      __syncwarp();
      // exclusive prefix sums, a contiguous stretch per lane
      const int per = (n + 31) / 32, i0 = min(lane * per, n), i1 = min(i0 + per, n);
      int sum = 0;
      for (int i = i0; i < i1; ++i) sum += s_np[i];
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int run = incl - sum;
      for (int i = i0; i < i1; ++i) {
        P[PL.pre + i] = run;
        run += s_np[i];
      }
      const int VP = __shfl_sync(0xffffffffu, incl, 31);
      if (lane == 0) P[PL.pre + n] = VP;
      __syncwarp();
      // ranges of the layer: as many as have a.min_pos positions each (a small layer: four), at most NB
      const int nb_eff = VP >= a.min_pos * (NB / 2) ? min(NB, (VP + a.min_pos - 1) / a.min_pos)
                                                    : max(1, min(NB, (VP + 3) / 4));
      for (int cc = lane; cc <= nb_eff; cc += 32)
        P[PL.cut + cc] = range_cut(cc, nb_eff, VP, min(a.snap, VP / nb_eff / 4), P + PL.pre, n);
      if (lane == 0) {
        P[PL.hdr] = VP;
        P[PL.hdr + 1] = nb_eff;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&plan_ready[l % n_plans]);
    }
  } else if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer warp
    // kind 0: nothing follows; 1: `count` positions of a range; 2: no pages, only the news that the
    // producer has moved on from layer `mark`
    struct Group { int gpage, valid, flags, item, count, chunk, layer, kind, mark; };
    int k = 0;          // stages used so far (pages and markers)
    int gave_up = 0;
    int layer = -1;     // layer whose plan is in use (-1: none yet)
    const int *P = nullptr;
    int cidx = 0, r_ps = 0, r_pe = 0, cur_base = 0;
    bool more = true;
    // the next range of the global list, claimed one ahead so that the answer is there when needed
    int pending = 0;
    if (lane == 0) pending = atomicAdd(a.claim, 1);
    // takes one stage for a marker (no bytes): flags and layer only
    auto marker = [&](int flags, int lyr) {
      const int stage = k % n_stages, use = k / n_stages;
      int ok = 1;
      if (lane == 0 && use > 0) ok = wait_or_flag(&empty[stage], (use - 1) & 1, c);
      if (!__shfl_sync(0xffffffffu, ok, 0)) {
        gave_up = 1;
        return;
      }
      if (lane == 0) {
        s_meta[stage].packed = flags << 8;
        s_meta[stage].layer = lyr;
        mbar_arrive(&full[stage]);
      }
      ++k;
    };
    // The range held for this block (claimed, not yet walked), or the end of the list.  Every block
    // claims until the counter has run past the list, i.e. fails exactly once: the claim that brings
    // the counter to n_ranges + gridDim.x is the launch's last, and its owner leaves it at zero.
    // A block whose list is exhausted still visits the remaining layers (markers only): the planner
    // walks them all, each only after this block has left the layer that held its plan buffer before.
    bool have_g = false, finishing = false;
    int tgt_layer = 0, g_cidx = 0;
    // Resolves the next (up to) 32 positions of the range (markers come out with valid = 0), taking a
    // new range when the current one is done.  Entering the next layer is a step of its own -- one
    // layer per call, a group of kind 2 -- because the marker of the layer left must go down the
    // pipeline behind that layer's last pages and before this warp waits for a later plan.
    auto resolve = [&]() {
      Group gq = {0, 0, 0, 0, 0, 0, 0, 0, -1};
      if (!more) return gq;
      while (cur_base >= r_pe) {
        if (!have_g && !finishing) {
          const int g = __shfl_sync(0xffffffffu, pending, 0);
          if (g >= n_ranges) {
            if (g == n_ranges + (int)gridDim.x - 1 && lane == 0) *a.claim = 0;
            finishing = true;
            tgt_layer = a.n_layers - 1;
          } else {
            if (lane == 0) pending = atomicAdd(a.claim, 1);
            have_g = true;
            tgt_layer = g / NB;
            g_cidx = g % NB;
          }
        }
        if (layer < tgt_layer) {
          gq.kind = 2;
          gq.mark = layer;  // (-1 before the first layer: nothing to tell)
          ++layer;
          int ok = 1;
          if (lane == 0) ok = wait_or_flag(&plan_ready[layer % n_plans], (layer / n_plans) & 1, c);
          if (!__shfl_sync(0xffffffffu, ok, 0)) {
            gave_up = 1;
            more = false;
            gq.kind = 0;
          }
          P = plan_of(layer);
          return gq;
        }
        if (finishing) {
          more = false;
          return gq;
        }
        have_g = false;
        cidx = g_cidx;
        if (P[PL.hdr] == 0 || cidx >= P[PL.hdr + 1]) continue;  // the layer has fewer ranges than the numbering
        r_ps = P[PL.cut + cidx];
        r_pe = P[PL.cut + cidx + 1];
        cur_base = r_ps;
      }
      gq.kind = 1;
      gq.chunk = cidx;
      gq.layer = layer;
      gq.count = min(32, r_pe - cur_base);
      const int pp = cur_base + lane;
      if (pp < r_pe) {
        const int *pre = P + PL.pre;
        int lo = 0, hi = n;
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (pre[mid] <= pp) lo = mid; else hi = mid;
        }
        const int item = lo, j = pp - pre[item] - 1;  // j = -1: the unit's marker position
        if (j >= 0) {
          const int u = P[PL.unit + item], len = P[PL.len + item], nk = (len + kP - 1) / kP;
          if (j < nk) {
            gq.gpage = checked_page(c, ldcg_keep(&unit_table(c, P[PL.row + item])[j]), (int)ring_page(c, u, 0));
            gq.valid = min(kP, len - j * kP);
          } else {
            gq.gpage = (int)ring_page(c, u, j - nk);
            gq.valid = min(kP, P[PL.ring + item] - (j - nk) * kP);
          }
          gq.item = item;
          gq.flags = ((pp == r_ps || j == 0) ? F_BEGIN : 0) |
                     ((pp == r_pe - 1 || pp == pre[item + 1] - 1) ? F_END : 0);
        }
      }
      cur_base += 32;
      return gq;
    };

    const uint64_t l2pol = l2_evict_first_policy();  // keys and values are read once per step
    Group cur = resolve();
    while (cur.kind != 0 && !gave_up) {
      if (cur.mark >= 0) marker(F_LAYER, cur.mark);  // before the next resolve, which may wait for a plan that needs it
      if (gave_up) break;
      const Group nxt = resolve();  // resolved before this group is issued: its table loads overlap the copies
      for (int i = 0; i < cur.count; ++i) {
        const int gp = __shfl_sync(0xffffffffu, cur.gpage, i), va = __shfl_sync(0xffffffffu, cur.valid, i);
        const int fl = __shfl_sync(0xffffffffu, cur.flags, i), it = __shfl_sync(0xffffffffu, cur.item, i);
        if (va == 0) continue;  // marker position
        const int stage = k % n_stages, use = k / n_stages;
        int ok = 1;
        if (lane == 0 && use > 0) ok = wait_or_flag(&empty[stage], (use - 1) & 1, c);
        if (!__shfl_sync(0xffffffffu, ok, 0)) {
          gave_up = 1;
          break;
        }
        if (lane == 0) {
          s_meta[stage].packed = va | (fl << 8) | (it << 12);
          s_meta[stage].chunk = cur.chunk;
          s_meta[stage].layer = cur.layer;
          unsigned char *dst = smem + (size_t)stage * L.stage_bytes;
          const uint32_t qbytes = (fl & F_BEGIN) ? (uint32_t)(a.G * kRowBytes) : 0u;
          mbar_arrive_expect_tx(&full[stage], kPageBytes + qbytes);
          bulk_load_hint(dst, c.pages + (int64_t)gp * kPageElems, kPageBytes, &full[stage], l2pol);
          if (qbytes)
            bulk_load(dst + kPageBytes,
                      a.q + (((size_t)cur.layer * a.B + (size_t)(it / c.Hkv)) * c.Hq + (size_t)(it % c.Hkv) * a.G) * kD,
                      qbytes, &full[stage]);
        }
        ++k;
      }
      cur = nxt;
    }
    if (!gave_up) marker(F_STOP, 0);  // tell the consumers that nothing follows
    if (lane == 0 && gave_up) {
      // do not leave while copies may still be landing in shared memory
      for (int kk = max(0, k - n_stages); kk < k; ++kk)
        mbar_wait_bounded(&full[kk % n_stages], (kk / n_stages) & 1);
    }
  } else if (warp < kConsumerWarps) {
    // ----------------------------------------------------------------- consumer warps
    // (the per-layer kernel's consumers: a warp takes 16 of the 64 pairs of its group's pages;
    // S^T = K Q^T and O^T += V^T P^T as m16n8k16 tiles, online softmax in registers)
    uint32_t qb[NH][8][2];
    float m[NH][2], l[NH][2], o[NH][8][4];
    int seg_k = 0;  // pages of the current segment so far: group g takes those with seg_k % 2 == g, so that a
                    // segment's sums do not depend on what the block streamed before it
    int n_seg = 0;  // hand-overs so far (segments and layer markers)
    // waits for the hand-over buffer of this turn; false if the wait ran out
    auto hand_over_begin = [&](int &rb) {
      rb = n_seg & 1;
      const int ruse = n_seg >> 1;
      ++n_seg;
      return ruse == 0 || wait_or_flag(&red_empty[rb], (ruse - 1) & 1, c);
    };
    for (int k = 0;; ++k) {
      const int stage = k % n_stages, use = k / n_stages;
      if (!wait_or_flag(&full[stage], use & 1, c)) break;
      const int meta = s_meta[stage].packed;
      const int flags = (meta >> 8) & 15;
      if (flags & F_STOP) break;
      const int chunk = s_meta[stage].chunk, layer = s_meta[stage].layer;
      if (flags & F_LAYER) {  // the producer has left `layer`: pass the news on behind the layer's last segment
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        int rb;
        if (!hand_over_begin(rb)) break;
        if (tid == 0) {
          s_redmeta[rb] = -2;
          s_redmeta[4 + rb] = layer;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&red_full[rb]);
        continue;
      }
      const int valid = meta & 255, item = meta >> 12;
      unsigned char *sbase = smem + (size_t)stage * L.stage_bytes;
      if (flags & F_BEGIN) {
        seg_k = 0;
        segment_begin<NH>(qb, m, l, o, reinterpret_cast<const __nv_bfloat16 *>(sbase + kPageBytes), GP, lane);
      }
      const int tok0 = (warp & 3) * 16;
      if ((seg_k & 1) == (warp >> 2) && tok0 < valid) {
        const uint32_t sK = smem_u32(sbase), sV = sK + kBlockElems * 2;
        float s[NH][4];
        qk_tile_t<NH>(s, qb, sK, tok0, lane);
        softmax_pv_tile_t<NH>(s, valid, a.scale_log2, m, l, o, sV, tok0, lane);
      }
      ++seg_k;
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);
      if (!(flags & F_END)) continue;

      // last page of the segment: hand this warp's (m, l, O) to the epilogue warp
      int rb;
      if (!hand_over_begin(rb)) break;
      segment_hand_over<NH>(s_red + (size_t)rb * kConsumerWarps * GP * 132, warp, GP, a.G, m, l, o, lane);
      if (tid == 0) {
        s_redmeta[rb] = item;
        s_redmeta[2 + rb] = chunk;
        s_redmeta[4 + rb] = layer;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&red_full[rb]);
    }
    // tell the epilogue warp that nothing follows
    {
      int rb;
      if (hand_over_begin(rb)) {
        if (tid == 0) s_redmeta[rb] = -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(&red_full[rb]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warp
    for (int e = 0;; ++e) {
      const int rb = e & 1;
      if (!wait_or_flag(&red_full[rb], (e >> 1) & 1, c)) break;
      const int item = s_redmeta[rb];
      if (item == -1) break;
      const int layer = s_redmeta[4 + rb];
      if (item == -2) {  // every segment of `layer` has passed: the planner may reuse its plan
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&plan_free[layer % n_plans]);
          mbar_arrive(&red_empty[rb]);
        }
        continue;
      }
      const int cidx = s_redmeta[2 + rb];
      const int *P = plan_of(layer);
      const Ranges rg = {P[PL.hdr + 1], P + PL.cut};
      char *wsl = a.ws + (size_t)layer * a.ws_layer_bytes;
      const size_t rows = (size_t)layer * a.B * c.Hq;
      const SegOut so = {a.out + rows * kD, nullptr, a.lse ? a.lse + rows : nullptr,
                         reinterpret_cast<int32_t *>(wsl), reinterpret_cast<int32_t *>(wsl + a.off_gcnt),
                         reinterpret_cast<float *>(wsl + a.off_ml), reinterpret_cast<float *>(wsl + a.off_acc)};
      finish_segment(c, a.G, GP, so, rg, P + PL.pre, s_red + (size_t)rb * kConsumerWarps * GP * 132, s_mrg,
                     &red_empty[rb], item, cidx, lane);
    }
  }
}

}  // namespace spkv

using namespace spkv;

static size_t stack_a256(size_t x) { return (x + 255) / 256 * 256; }

extern "C" size_t spkv_decode_stack_workspace_bytes(const spkv_config_t *cfg, int32_t B) {
  if (!cfg || B < 0 || cfg->n_kv_heads < 1 || cfg->n_layers < 1) return 0;
  // the range counter, one region of arrival counters and partial results per layer, and (for the
  // layer-by-layer fallback) the workspace of spkv_decode_attention
  const size_t per_layer = stack_a256(decode_ws_layout(B * cfg->n_kv_heads, cfg->n_q_heads / cfg->n_kv_heads).total);
  return 256 + (size_t)cfg->n_layers * per_layer + spkv_decode_workspace_bytes(cfg, B);
}

// Layers l0 ... l1 - 1 of a stack step.  The input and output pointers name layer 0's rows (the
// whole stack's arrays), whatever the range.
int spkv::decode_stack_layers(spkv_cache *cache, int l0, int l1, const spkv_predictor_t *preds, const int32_t *d_seq_ids,
                              int32_t B, const void *d_x, const void *d_q, const void *d_k, const void *d_v, void *d_out,
                              float *d_logits_out, float *d_lse_opt, float sm_scale, void *d_workspace,
                              size_t workspace_bytes, spkv_stream_t stream) {
  if (!cache || !preds || B < 0 || B > cache->cfg.max_seqs || l0 < 0 || l1 > cache->cfg.n_layers || l0 > l1)
    return SPKV_E_INVALID;
  if (l0 == l1) return SPKV_OK;
  if (B == 0) return SPKV_OK;
  if (!d_seq_ids || !d_x || !d_q || !d_k || !d_v || !d_out) return SPKV_E_INVALID;
  if (((uintptr_t)d_x | (uintptr_t)d_q | (uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_out) & 15) return SPKV_E_INVALID;
  const spkv_config_t &cfg = cache->cfg;
  const CacheView &v = cache->view;
  const int L = cfg.n_layers, n_items = B * v.Hkv, d_in = preds[0].d_in, nl = l1 - l0;
  if (n_items > 1024) return SPKV_E_UNSUPPORTED;
  for (int l = 0; l < L; ++l)
    if (preds[l].d_in != d_in) return SPKV_E_INVALID;
  if (!d_workspace || ((uintptr_t)d_workspace & 255) || workspace_bytes < spkv_decode_stack_workspace_bytes(&cfg, B))
    return SPKV_E_WORKSPACE;
  const DecodeWs wl = decode_ws_layout(n_items, v.G);
  const size_t per_layer = stack_a256(wl.total);
  char *ws = static_cast<char *>(d_workspace);
  const size_t x_l = (size_t)B * d_in * 2, q_l = (size_t)B * cfg.n_q_heads * kD * 2, kv_l = (size_t)n_items * kD * 2;
  cudaStream_t s = as_stream(stream);

  // shared memory of the persistent kernel: as many page stages as fit beside two plans; then as
  // many plans (up to four: small layers are paced by how far ahead the planner may run) as fit
  // without costing a stage
  int GP = 1;
  while (GP < v.G) GP <<= 1;
  const int limit = 227 * 1024;
  int n_stages = 6, n_plans = 2;
  StackSmem SL = stack_smem_layout(n_items, B, GP, n_stages, n_plans);
  while (SL.total > limit && n_stages > 2) SL = stack_smem_layout(n_items, B, GP, --n_stages, n_plans);
  while (SL.total <= limit && n_plans < kMaxPlans &&
         stack_smem_layout(n_items, B, GP, n_stages, n_plans + 1).total <= limit)
    SL = stack_smem_layout(n_items, B, GP, n_stages, ++n_plans);

  bool fused = nl <= kMaxStackLayers && d_in >= 8 && (d_in & 7) == 0 && (x_l & 15) == 0 && SL.total <= limit;
  for (int l = l0; l < l1 && fused; ++l)
    fused = preds[l].kind == 0 && preds[l].d_W1 && preds[l].d_b1 && ((uintptr_t)preds[l].d_W1 & 15) == 0;
  if (!fused) {
    // two-layer predictors (scored by a kernel of their own), very deep stacks, and batches whose
    // plans leave no room for two page stages: layer by layer
    void *ws1 = ws + 256 + (size_t)L * per_layer;
    for (int l = l0; l < l1; ++l) {
      float *lg = d_logits_out ? d_logits_out + (size_t)l * n_items : nullptr;
      int rc = spkv_score_append_evict(cache, l, &preds[l], d_seq_ids, B, static_cast<const char *>(d_x) + l * x_l,
                                       static_cast<const char *>(d_k) + l * kv_l,
                                       static_cast<const char *>(d_v) + l * kv_l, lg, stream);
      if (rc) return rc;
      rc = spkv_decode_attention(cache, l, d_seq_ids, B, static_cast<const char *>(d_q) + l * q_l,
                                 static_cast<char *>(d_out) + l * q_l,
                                 d_lse_opt ? d_lse_opt + (size_t)l * B * cfg.n_q_heads : nullptr, sm_scale, ws1,
                                 spkv_decode_workspace_bytes(&cfg, B), stream);
      if (rc) return rc;
    }
    return SPKV_OK;
  }

  // both launches are ordinary stream-ordered ones: whatever the cache's previous launch was, they
  // wait for it, and the next per-layer call must wait for them
  cache->last_kind = kLastOther;
  StackPreds sp;
  for (int l = l0; l < l1; ++l) {
    sp.W[l - l0] = static_cast<const __nv_bfloat16 *>(preds[l].d_W1);
    sp.bias[l - l0] = preds[l].d_b1;
    sp.local_mask[l - l0] = cache->local_mask[l];
  }
  int rc = launch_append_stack(cache, sp, l0, nl, d_seq_ids, B, static_cast<const char *>(d_k) + l0 * kv_l,
                               static_cast<const char *>(d_v) + l0 * kv_l, static_cast<const char *>(d_x) + l0 * x_l, d_in,
                               d_logits_out ? d_logits_out + (size_t)l0 * n_items : nullptr, s);
  if (rc) return rc;

  StackArgs a;
  a.c = v; a.layer0 = l0; a.n_layers = nl; a.B = B; a.n_items = n_items; a.G = v.G;
  a.seq_ids = d_seq_ids;
  a.q = reinterpret_cast<const __nv_bfloat16 *>(static_cast<const char *>(d_q) + l0 * q_l);
  a.out = reinterpret_cast<__nv_bfloat16 *>(static_cast<char *>(d_out) + l0 * q_l);
  a.lse = d_lse_opt ? d_lse_opt + (size_t)l0 * B * cfg.n_q_heads : nullptr;
  a.scale_log2 = sm_scale * kLog2e;
  a.snap = 6;
  // the per-layer kernel's rule, so that both paths cut a layer's pages the same way: a cache in
  // overlap mode gives a range at least 56 positions when the layer has half a grid of such ranges
  a.min_pos = (cfg.flags & SPKV_FLAG_OVERLAP) ? 56 : 4;
  a.nb = min(kMaxGrid, cache->sm_count);
  a.claim = reinterpret_cast<int32_t *>(ws);
  a.ws = ws + 256 + (size_t)l0 * per_layer;
  a.ws_layer_bytes = per_layer;
  a.off_gcnt = wl.off_gcnt; a.off_ml = wl.off_ml; a.off_acc = wl.off_acc;
  void (*kernel)(StackArgs, int, int, int) = GP > 8 ? decode_stack_kernel<2> : decode_stack_kernel<1>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SL.total) != cudaSuccess)
    return SPKV_E_CUDA;
  const int grid = min(kMaxGrid, cache->sm_count);
  return check_stream_error(
      launch_overlapped(kernel, dim3(grid), dim3(kStackThreads), (size_t)SL.total, s, a, GP, n_stages, n_plans));
}

extern "C" int spkv_decode_stack(spkv_cache_t *cache, const spkv_predictor_t *preds, const int32_t *d_seq_ids, int32_t B,
                                 const void *d_x, const void *d_q, const void *d_k, const void *d_v, void *d_out,
                                 float *d_logits_out, float *d_lse_opt, float sm_scale, void *d_workspace,
                                 size_t workspace_bytes, spkv_stream_t stream) {
  if (!cache) return SPKV_E_INVALID;
  return decode_stack_layers(cache, 0, cache->cfg.n_layers, preds, d_seq_ids, B, d_x, d_q, d_k, d_v, d_out, d_logits_out,
                             d_lse_opt, sm_scale, d_workspace, workspace_bytes, stream);
}
