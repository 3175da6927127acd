// Step 3 of the hot path: ragged split-K decode attention (Eq. 3-5) over
// ring window U compact cache, log-sum-exp merge fused in.  The kernel that takes one layer per
// launch, and the host entry points.  (spkv_decode_stack.cu holds the kernel that takes every
// layer of a step in one launch; the two share their consumers, epilogue and range cuts through
// spkv_decode_common.cuh.)
//
// Work decomposition.  The call covers n_items = B * n_kv_heads units.  Unit i owns np_i
// pages (its kept pages followed by its ring pages).  All page lists are laid end to end
// on one axis, each preceded by one "marker" position that stands for the fixed cost of
// starting and finishing a unit (query fetch, merge of the warps, output); the axis is cut
// into gridDim.x contiguous ranges of equal length, one per block ("chunk" = range).  A
// block that gets many short units (local-only heads) therefore gets fewer pages, one that
// sits inside a long unit gets more.  Keep rates from 0 to 100 % need no special handling:
// the axis is in pages, not in heads.  Every block recomputes the prefix sums itself
// (lengths live on the device and change every step): no extra launch, no host sync.
//
// Merge.  A (chunk, unit) intersection is a "segment".  A segment that covers its whole
// unit writes the output directly.  Otherwise it stores (m, l, acc) in workspace slot
// (chunk + item) -- unique because consecutive segments differ in chunk or item -- and
// bumps the unit's arrival counter; the block that arrives last merges all slots of the
// unit by their log-sum-exp weights and resets the counter.  A unit cut into more than
// kMergeGroup ranges is merged on two levels: groups of kMergeGroup consecutive ranges, each
// by the last arriver of the group into the group's first slot, then the group results by
// the last group.  Nobody ever waits.
//
// Block = 8 consumer warps (two groups of four that take alternate pages, so that one group's
// waits overlap the other's arithmetic) + producer warp + epilogue warp, one block per SM, a
// pipeline of whole pages:
//   producer  walks the block's range, resolves each page (unit, page-table entry, valid rows) with its
//       32 lanes in parallel, then issues one 32 KB linear bulk copy HBM -> shared memory
//       per page (cp.async.bulk on an mbarrier) plus, at the start of a segment, the
//       G query rows.  The page in HBM already is the swizzled shared-memory image.
//   consumers each take 16 of the 64 pairs of their group's pages.  The 16 keys are the rows and the group's
//       G query heads the (8-wide) columns of the tiles, so S^T = K Q^T and O^T += V^T P^T are
//       small dense products done with mma.sync m16n8k16 (bf16 in, fp32 accumulate): 8 + 16
//       MMAs per warp and page, operands read with ldmatrix; mask, online softmax (exp2,
//       shuffles over the keys) in registers.  Each warp keeps (m, l, O) for
//       its quarter of every page of a segment and drops it into one of two shared-memory
//       buffers at the segment's end, then carries straight on with the next segment.
//   epilogue  merges the eight warps' results of a finished segment, writes the output (or
//       the partial + arrival count + last-arriver merge) while the consumers stream on.
//
// Why tensor cores in a bandwidth-bound kernel: per 512 B pair the group needs 2*G*128
// multiply-adds.  On the CUDA cores that is, with bf16 unpacking and the reductions, several
// hundred issue slots per pair and SM (174 warp instructions per pair at G = 4 in an earlier
// CUDA-core version of this kernel), and the issue rate, not HBM, limits the kernel from G = 4 on.  As MMA tiles it is 24 instructions per page and
// warp, and the page stream alone sets the pace.
//
// Every wait is bounded (about a second).  A consumer warp whose page never lands records
// SPKV_E_TIMEOUT and leaves its loop -- all four warps wait on the same barrier, so they
// leave at the same page; a producer whose stage is never released records the error and
// stops issuing, after which the consumers run into their own limit.  Before the block
// exits the producer waits (bounded again) for the copies it still has in flight.
#include <atomic>

#include "spkv_decode_common.cuh"
#include "spkv_mma.cuh"

namespace spkv {

struct TcSmem {  // offsets into dynamic shared memory, computed on host and device alike
  int n_stages, red_bufs, stage_bytes, off_bar, off_meta, off_np, off_pre, off_unit, off_len, off_ring, off_row,
      off_tmp, off_cut, off_red, off_mrg, off_flags, total;
};
__host__ __device__ inline TcSmem tc_smem_layout(int n_items, int GP, int n_stages, int red_bufs) {
  TcSmem L;
  L.n_stages = n_stages;
  L.red_bufs = red_bufs;
  L.stage_bytes = kPageBytes + GP * kRowBytes;  // page + the segment's query rows
  int o = n_stages * L.stage_bytes;
  o = (o + 15) / 16 * 16;
  L.off_bar = o;   o += (2 * kMaxStages + 4) * 8;  // full[], empty[], red_full[2], red_empty[2]
  L.off_meta = o;  o += kMaxStages * (int)sizeof(StageMeta);
  L.off_np = o;    o += n_items * 4;
  L.off_pre = o;   o += (n_items + 1) * 4;
  L.off_unit = o;  o += n_items * 4;
  L.off_len = o;   o += n_items * 4;
  L.off_ring = o;  o += n_items * 4;
  L.off_row = o;   o += n_items * 4;
  L.off_tmp = o;   o += 64 * 4;
  L.off_cut = o;   o += (kMaxGrid + 1) * 4;
  o = (o + 15) / 16 * 16;
  L.off_red = o;   o += red_bufs * kConsumerWarps * GP * 132 * 4;
  L.off_mrg = o;   o += kMergeCap * 8;
  L.off_flags = o; o += 16;
  L.total = o;
  return L;
}

#ifdef SPKV_PHASE_TIMING
__device__ inline unsigned long long gtimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define SPKV_STAMP_T(i, cond) do { if (cond) reinterpret_cast<unsigned long long *>(a.part_acc + (size_t)(148 + a.n_items) * a.G * kD)[blockIdx.x * 16 + (i)] = gtimer(); } while (0)
#else
#define SPKV_STAMP_T(i, cond)
#endif

template <int NH>  // 8-head tiles on the N side: 1 for G <= 8, 2 for G <= 16
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(DecodeArgs a, int GP, int n_stages, int red_bufs) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const CacheView &c = a.c;
  const int n = a.n_items;
  const TcSmem L = tc_smem_layout(n, GP, n_stages, red_bufs);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + L.off_bar);
  uint64_t *empty = full + kMaxStages;
  volatile StageMeta *s_meta = reinterpret_cast<volatile StageMeta *>(smem + L.off_meta);
  int *s_np = reinterpret_cast<int *>(smem + L.off_np);
  int *s_pre = reinterpret_cast<int *>(smem + L.off_pre);
  int *s_unit = reinterpret_cast<int *>(smem + L.off_unit);
  int *s_len = reinterpret_cast<int *>(smem + L.off_len);
  int *s_ring = reinterpret_cast<int *>(smem + L.off_ring);
  int *s_row = reinterpret_cast<int *>(smem + L.off_row);   // the unit's page-table row (-1: a local-only head)
  int *s_tmp = reinterpret_cast<int *>(smem + L.off_tmp);
  int *s_cut = reinterpret_cast<int *>(smem + L.off_cut);
  float *s_red = reinterpret_cast<float *>(smem + L.off_red);
  uint64_t *red_full = empty + kMaxStages, *red_empty = red_full + 2;
  float2 *s_mrg = reinterpret_cast<float2 *>(smem + L.off_mrg);
  volatile int *s_redmeta = reinterpret_cast<volatile int *>(smem + L.off_flags);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  SPKV_STAMP_T(0, tid == 0);
#ifdef SPKV_PHASE_TIMING
  int dbg_pages = 0, dbg_segs = 0;
  long long dbg_c[5] = {0, 0, 0, 0, 0};
#endif

  // counted in by a thread that has nothing else to do here (see sync_count_start)
  if (tid == 32) sync_count_start(c, a.layer, kSyncDecStart);
  if (tid == 0) {
    for (int i = 0; i < n_stages; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], kConsumerWarps);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&red_full[i], kConsumerWarps);
      mbar_init(&red_empty[i], 1);
    }
    mbar_fence_init();
  }
  // query rows past the group size are never written by a copy: zero them once
  for (int i = tid; i < n_stages * (GP - a.G) * (kRowBytes / 16); i += kTcThreads) {
    const int per = (GP - a.G) * (kRowBytes / 16);
    const int st = i / per, r = i % per;
    reinterpret_cast<uint4 *>(smem + (size_t)st * L.stage_bytes + kPageBytes + a.G * kRowBytes)[r] =
        make_uint4(0, 0, 0, 0);
  }
  // Everything above touched only this block's shared memory and may overlap the tail of the
  // previous kernel of the stream; from here on its results (lengths, pages) are read.
  // Overlap mode (wait_mode 1): the kernels before this one may still be running.  It shares data
  // with the appends of its own layer (lengths, ring, pages) and with the decode launch that
  // last used this half of the workspace, and waits for exactly those.
  // The sequence ids are an input of the call, complete by contract in this mode: fetched now,
  // beside the counter reads below.
  int seq_first = -1;
  if (a.wait_mode == 1 && tid < n) seq_first = a.seq_ids[tid / c.Hkv];
  if (a.wait_mode == 0) pdl_wait();
  // (the counter reads run beside thread 32's count-in: one trip to L2 for both)
  if (a.wait_mode == 1 && tid == 0 &&
      !sync_wait_finished(c, a.layer, kSyncAppStart, a.prev_half_layer, kSyncDecStart))
    set_status(c, SPKV_E_ORDER_DECODE);
  __syncthreads();  // the block is counted in before any of its threads lets dependents launch
  pdl_trigger();
  if (a.wait_mode == 1)
    asm volatile("fence.proxy.async;" ::: "memory");  // the appends wrote the pages the bulk copies read
  for (int i = tid; i < n; i += kTcThreads) {
    const int b = i / c.Hkv, kvh = i % c.Hkv;
    const int seq = (a.wait_mode == 1 && i == tid) ? seq_first : a.seq_ids[b];
    int np = 0, u = 0, len = 0, n_ring = 0, trow = -1;
    if (seq >= 0 && seq < c.S) {
      u = unit_index(c, a.layer, seq, kvh);
      trow = unit_table_row(c, u);
      // (L2 loads: in overlap mode the writer may be a kernel that ended after this block began,
      // and an SM's L1 is not coherent with other SMs' stores)
      len = ldcg_keep(&c.len[u]);
      n_ring = min(ldcg_keep(&c.t[u]), c.w);
      np = (len + kP - 1) / kP + (n_ring + kP - 1) / kP;
    } else if (blockIdx.x == 0) {
      set_status(c, SPKV_E_BOUNDS);
    }
    s_np[i] = np > 0 ? np + 1 : 0;  // + the marker position
    s_unit[i] = u; s_len[i] = len; s_ring[i] = n_ring; s_row[i] = trow;
    if (np == 0 && blockIdx.x == 0) {  // nothing to attend to: defined output
      for (int g = 0; g < a.G; ++g) {
        __nv_bfloat16 *o = a.out + ((size_t)b * c.Hq + kvh * a.G + g) * kD;
        for (int d = 0; d < kD; ++d) o[d] = __float2bfloat16(0.f);
        if (a.out_f32)
          for (int d = 0; d < kD; ++d) a.out_f32[((size_t)b * c.Hq + kvh * a.G + g) * kD + d] = 0.f;
        if (a.lse) a.lse[(size_t)b * c.Hq + kvh * a.G + g] = -INFINITY;
      }
    }
  }
  __syncthreads();
  block_exclusive_scan(s_np, s_pre, n, s_tmp);
  const int VP = s_pre[n];
  // Blocks per launch.  A small launch is latency-bound: as many blocks as have four positions
  // each (tiny calls would otherwise be cut into single pages and spend their time merging).
  // A launch with at least half a grid of a.min_pos-position ranges gives every block at least
  // that many: consecutive launches overlap, the SMs this one leaves idle work for its
  // neighbours, and a block's fixed cost (start-up, merge) is spread over more pages.
  const int nb_eff = VP >= a.min_pos * ((int)gridDim.x / 2) ? min((int)gridDim.x, (VP + a.min_pos - 1) / a.min_pos)
                                                            : max(1, min((int)gridDim.x, (VP + 3) / 4));
  // snapping distance: a.snap positions, less for short ranges
  for (int cc = tid; cc <= nb_eff; cc += kTcThreads)
    s_cut[cc] = range_cut(cc, nb_eff, VP, min(a.snap, VP / nb_eff / 4), s_pre, n);
  __syncthreads();
  const Ranges rg = {nb_eff, s_cut};
  SPKV_STAMP_T(1, tid == 0);

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer warp
    // Pages are resolved in groups of up to 32 (one per lane) of the block's range.
    // The next group is resolved before the current
    // group is issued, so the page-table loads overlap with the copies.
    struct Group { int gpage, valid, flags, item, count; };
    const int cidx = blockIdx.x;
    const bool active = VP > 0 && cidx < rg.nb;
    const int r_ps = active ? rg.start(cidx) : 0, r_pe = active ? rg.start(cidx + 1) : 0;
    int cur_base = r_ps;
    // resolves the next (up to) 32 positions of the range; markers come out with valid = 0
    auto resolve = [&]() {
      Group gq = {0, 0, 0, 0, 0};
      if (cur_base >= r_pe) return gq;
      gq.count = min(32, r_pe - cur_base);
      const int pp = cur_base + lane;
      if (pp < r_pe) {
        int lo = 0, hi = n;
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (s_pre[mid] <= pp) lo = mid; else hi = mid;
        }
        const int item = lo, j = pp - s_pre[item] - 1;  // j = -1: the unit's marker
        if (j >= 0) {
          const int u = s_unit[item], len = s_len[item], nk = (len + kP - 1) / kP;
          if (j < nk) {
            // (debug bounds: a table entry that names no pool page is read from the unit's ring instead)
            gq.gpage = checked_page(c, ldcg_keep(&unit_table(c, s_row[item])[j]), (int)ring_page(c, u, 0));
            gq.valid = min(kP, len - j * kP);
          } else {
            gq.gpage = (int)ring_page(c, u, j - nk);
            gq.valid = min(kP, s_ring[item] - (j - nk) * kP);
          }
          gq.item = item;
          gq.flags = ((pp == r_ps || j == 0) ? F_BEGIN : 0) |
                     ((pp == r_pe - 1 || pp == s_pre[item + 1] - 1) ? F_END : 0);
        }
      }
      cur_base += 32;
      return gq;
    };

    int k = 0;  // pages issued by this block
    int gave_up = 0;
    // keys and values are read once per step: their lines leave L2 first, so that what every step
    // reads again (lengths, page tables: loaded with the opposite hint) stays there (+1 % in step)
    const uint64_t l2pol = l2_evict_first_policy();
    Group cur = resolve();
    while (cur.count > 0 && !gave_up) {
      const Group nxt = resolve();
      for (int i = 0; i < cur.count; ++i) {
        const int gp = __shfl_sync(0xffffffffu, cur.gpage, i), va = __shfl_sync(0xffffffffu, cur.valid, i);
        const int fl = __shfl_sync(0xffffffffu, cur.flags, i), it = __shfl_sync(0xffffffffu, cur.item, i);
        if (va == 0) continue;  // marker
        const int stage = k % n_stages, use = k / n_stages;
        int ok = 1;
        if (lane == 0 && use > 0) ok = wait_or_flag(&empty[stage], (use - 1) & 1, c);
        if (!__shfl_sync(0xffffffffu, ok, 0)) {
          gave_up = 1;
          break;
        }
        if (lane == 0) {
          s_meta[stage].packed = va | (fl << 8) | (it << 12);
          unsigned char *dst = smem + (size_t)stage * L.stage_bytes;
          const uint32_t qbytes = (fl & F_BEGIN) ? (uint32_t)(a.G * kRowBytes) : 0u;
          mbar_arrive_expect_tx(&full[stage], kPageBytes + qbytes);
          bulk_load_hint(dst, c.pages + (int64_t)gp * kPageElems, kPageBytes, &full[stage], l2pol);
          if (qbytes)
            bulk_load(dst + kPageBytes,
                      a.q + ((size_t)(it / c.Hkv) * c.Hq + (size_t)(it % c.Hkv) * a.G) * kD, qbytes,
                      &full[stage]);
        }
        ++k;
      }
      cur = nxt;
    }
    if (lane == 0 && !gave_up) {  // tell the consumers that nothing follows
      const int stage = k % n_stages, use = k / n_stages;
      if (use == 0 || wait_or_flag(&empty[stage], (use - 1) & 1, c)) {
        s_meta[stage].packed = F_STOP << 8;
        mbar_arrive(&full[stage]);
      } else {
        gave_up = 1;
      }
    }
    if (lane == 0 && gave_up) {
      // do not leave while copies may still be landing in shared memory
      for (int kk = max(0, k - n_stages); kk < k; ++kk)
        mbar_wait_bounded(&full[kk % n_stages], (kk / n_stages) & 1);
    }
  } else if (warp < kConsumerWarps) {
    // ----------------------------------------------------------------- consumer warps
    uint32_t qb[NH][8][2];
    float m[NH][2], l[NH][2], o[NH][8][4];
    int seg_k = 0;  // pages of the current segment so far: group g takes those with seg_k % 2 == g, so that a
                    // segment's sums do not depend on what the block streamed before it
    int n_seg = 0;
    for (int k = 0;; ++k) {
      const int stage = k % n_stages, use = k / n_stages;
#ifdef SPKV_PHASE_TIMING
      const long long c0 = clock64();
#endif
      if (!wait_or_flag(&full[stage], use & 1, c)) break;
#ifdef SPKV_PHASE_TIMING
      const long long c1 = clock64();
#endif
      SPKV_STAMP_T(3, tid == 0 && k == 0);
      const int meta = s_meta[stage].packed;
      const int flags = (meta >> 8) & 15;
      if (flags & F_STOP) break;
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
#ifdef SPKV_PHASE_TIMING
        const long long c2 = clock64();
#endif
        qk_tile_t<NH>(s, qb, sK, tok0, lane);
#ifdef SPKV_PHASE_TIMING
        const long long c3 = clock64();
        dbg_c[1] += c2 - c1; dbg_c[2] += c3 - c2;
#endif
        softmax_pv_tile_t<NH>(s, valid, a.scale_log2, m, l, o, sV, tok0, lane);
#ifdef SPKV_PHASE_TIMING
        dbg_c[3] += clock64() - c3;
#endif
      }
      ++seg_k;
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);
#ifdef SPKV_PHASE_TIMING
      dbg_c[0] += c1 - c0; dbg_c[4] += clock64() - c0;
      dbg_pages++;
      if (flags & F_END) dbg_segs++;
#endif
      if (!(flags & F_END)) continue;

      // last page of the segment: hand this warp's (m, l, O) to the epilogue warp
      const int rb = n_seg & 1, ruse = n_seg >> 1;
      ++n_seg;
      if (ruse > 0 && !wait_or_flag(&red_empty[rb], (ruse - 1) & 1, c)) break;
      segment_hand_over<NH>(s_red + (size_t)rb * kConsumerWarps * GP * 132, warp, GP, a.G, m, l, o, lane);
      if (tid == 0) s_redmeta[rb] = item;
      __syncwarp();
      if (lane == 0) mbar_arrive(&red_full[rb]);
    }
    // tell the epilogue warp that nothing follows
    {
      const int rb = n_seg & 1, ruse = n_seg >> 1;
      if (ruse == 0 || wait_or_flag(&red_empty[rb], (ruse - 1) & 1, c)) {
        if (tid == 0) s_redmeta[rb] = -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(&red_full[rb]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warp
    // Merges the four consumer warps of a finished segment (lane l owns dims 4l..4l+3),
    // writes the output or the partial, and, for a unit split over several blocks, takes
    // part in the last-arriver merge -- all off the consumers' critical path.
    const int cidx = blockIdx.x;
    for (int e = 0;; ++e) {
      const int rb = e & 1;
      if (!wait_or_flag(&red_full[rb], (e >> 1) & 1, c)) break;
      const int item = s_redmeta[rb];
      if (item < 0) break;
      const SegOut so = {a.out, a.out_f32, a.lse, a.counters, a.group_counters, a.part_ml, a.part_acc};
      finish_segment(c, a.G, GP, so, rg, s_pre, s_red + (size_t)rb * kConsumerWarps * GP * 132, s_mrg, &red_empty[rb],
                     item, cidx, lane);
    }
  }
  SPKV_STAMP_T(4, tid == 0);
#ifdef SPKV_PHASE_TIMING
  if (tid == 0) {
    unsigned long long *dbg = reinterpret_cast<unsigned long long *>(a.part_acc + (size_t)(148 + a.n_items) * a.G * kD);
    { unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); dbg[blockIdx.x * 16 + 15] = smid; }
  }
#endif
  __syncthreads();
  if (tid == 0) sync_count_finish(c, a.layer, kSyncDecFin);
  SPKV_STAMP_T(5, tid == 0);
}

}  // namespace spkv

using namespace spkv;

extern "C" size_t spkv_decode_workspace_bytes(const spkv_config_t *cfg, int32_t B) {
  if (!cfg || B < 0 || cfg->n_kv_heads < 1) return 0;
  return 2 * decode_ws_layout(B * cfg->n_kv_heads, cfg->n_q_heads / cfg->n_kv_heads).total;
}

// Argument checks of a decode call that need no workspace (B > 0 on SPKV_OK with *empty = false).
static int decode_check_args(const spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids, int32_t B,
                             const void *d_q, const void *d_out, const float *d_out_f32, bool *empty) {
  *empty = false;
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || B < 0 || B > cache->cfg.max_seqs)
    return SPKV_E_INVALID;
  if (B == 0) { *empty = true; return SPKV_OK; }
  if (!d_seq_ids || !d_q || !d_out) return SPKV_E_INVALID;
  if (((uintptr_t)d_q | (uintptr_t)d_out | (uintptr_t)d_out_f32) & 15) return SPKV_E_INVALID;
  if (B * cache->view.Hkv > 1024) return SPKV_E_UNSUPPORTED;
  return SPKV_OK;
}

static int decode_attention_impl(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids, int32_t B,
                                 const void *d_q, void *d_out, float *d_out_f32, float *d_lse_opt, float sm_scale,
                                 void *d_workspace, size_t workspace_bytes, spkv_stream_t stream) {
  bool empty;
  const int rc_args = decode_check_args(cache, layer, d_seq_ids, B, d_q, d_out, d_out_f32, &empty);
  if (rc_args || empty) return rc_args;
  const CacheView &v = cache->view;
  const int n_items = B * v.Hkv;
  const DecodeWs wl = decode_ws_layout(n_items, v.G);
  if (!d_workspace || ((uintptr_t)d_workspace & 255) || workspace_bytes < 2 * wl.total) return SPKV_E_WORKSPACE;

  DecodeArgs a;
  a.c = v; a.layer = layer; a.B = B; a.n_items = n_items; a.G = v.G;
  a.seq_ids = d_seq_ids;
  a.q = static_cast<const __nv_bfloat16 *>(d_q);
  a.out = static_cast<__nv_bfloat16 *>(d_out);
  a.out_f32 = d_out_f32;
  a.lse = d_lse_opt;
  a.scale_log2 = sm_scale * kLog2e;
  a.snap = 6;       // measured best on the 32 K and 128 K workloads (0, 2, 4, 6, 8, 12 tried)
  // likewise (32 ... 96 tried) where launches overlap: the SMs a launch leaves idle work for its
  // neighbours.  A stream-ordered launch has no neighbours to share with and takes every SM.
  a.min_pos = (cache->cfg.flags & SPKV_FLAG_OVERLAP) ? 56 : 4;
  // Two consecutive decode launches may overlap (the next one starts on the SMs this one
  // has left): they alternate between the two halves of the workspace.  A third cannot
  // join: it needs every block of the second resident, i.e. every SM left by the first.
  const int half = cache->ws_toggle;
  char *ws = static_cast<char *>(d_workspace) + (size_t)half * wl.total;
  cache->ws_toggle ^= 1;
  // Overlap mode: directly after this layer's append on the same stream the kernel need not wait
  // for the whole stream, only for that append and for the previous user of its workspace half.
  // When that user was a decode launch of this same layer (one- and two-layer stacks), the wait
  // for the append covers it: the append, launched after that decode, itself waited for every
  // decode launch of its layer before it touched the cache.  (The kernel could not wait for it
  // directly: a block cannot tell its own launch's count from older ones.)
  a.wait_mode = ((cache->cfg.flags & SPKV_FLAG_OVERLAP) && cache->last_kind == kLastAppend &&
                 cache->last_layer == layer && cache->last_stream == as_stream(stream) &&
                 // same workspace, cut into the same halves, as the launch it may run beside
                 cache->last_decode_items == n_items && cache->last_decode_ws == d_workspace)
                    ? 1 : 0;
  cache->last_decode_items = n_items;
  cache->last_decode_ws = d_workspace;
  a.prev_half_layer = cache->half_last_layer[half] == layer ? -1 : cache->half_last_layer[half];
  cache->half_last_layer[half] = layer;
  cache->appends_pending[layer] = 0;
  cache->last_kind = kLastDecode;
  cache->last_layer = layer;
  cache->last_stream = as_stream(stream);
  a.counters = reinterpret_cast<int32_t *>(ws);
  a.group_counters = reinterpret_cast<int32_t *>(ws + wl.off_gcnt);
  a.part_ml = reinterpret_cast<float *>(ws + wl.off_ml);
  a.part_acc = reinterpret_cast<float *>(ws + wl.off_acc);

  cudaStream_t s = as_stream(stream);
  int GP = 1;
  while (GP < v.G) GP <<= 1;
  // as many page stages as fit beside the two merge buffers
  const int limit = 227 * 1024;
  int n_stages = 6;
  const int red_bufs = 2;
  TcSmem L = tc_smem_layout(n_items, GP, n_stages, red_bufs);
  while (L.total > limit && n_stages > 2) L = tc_smem_layout(n_items, GP, --n_stages, red_bufs);
  if (L.total > limit) return SPKV_E_UNSUPPORTED;
  void (*kernel)(DecodeArgs, int, int, int) = GP > 8 ? decode_tc_kernel<2> : decode_tc_kernel<1>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total) != cudaSuccess)
    return SPKV_E_CUDA;
  const int grid = min(kMaxGrid, cache->sm_count);
  // (a programmatic dependent launch in every mode: with wait_mode 0 the kernel runs only its
  // block-local prologue before griddepcontrol.wait orders it after everything earlier on the stream)
  return check_stream_error(
      launch_overlapped(kernel, dim3(grid), dim3(kTcThreads), (size_t)L.total, s, a, GP, n_stages, red_bufs));
}

extern "C" int spkv_decode_attention(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                                     int32_t B, const void *d_q, void *d_out, float *d_lse_opt,
                                     float sm_scale, void *d_workspace, size_t workspace_bytes,
                                     spkv_stream_t stream) {
  return decode_attention_impl(cache, layer, d_seq_ids, B, d_q, d_out, nullptr, d_lse_opt, sm_scale, d_workspace,
                               workspace_bytes, stream);
}

extern "C" int spkv_decode_attention_f32(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                                         int32_t B, const void *d_q, void *d_out, float *d_out_f32,
                                         float *d_lse_opt, float sm_scale, void *d_workspace,
                                         size_t workspace_bytes, spkv_stream_t stream) {
  if (!d_out_f32) return SPKV_E_INVALID;
  return decode_attention_impl(cache, layer, d_seq_ids, B, d_q, d_out, d_out_f32, d_lse_opt, sm_scale, d_workspace,
                               workspace_bytes, stream);
}

// ---- decode attention for callers that cannot allocate device memory ---------------------
//
// The split-K scratch (arrival counters and partial results) of this variant lives in a
// fixed array inside the library's device image instead of a caller-supplied workspace.
// Every GPU that loads the library carries these 6 MiB until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SPKV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// device address of g_static_scratch per device; non-null = looked up (published with release
// order, so a thread that reads it non-null reads the address the lookup returned)
std::atomic<void *> g_scratch_ptr[kMaxDevices];
}  // namespace

extern "C" int spkv_decode_attention_static(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                                            int32_t B, const void *d_q, void *d_out, float *d_lse_opt,
                                            float sm_scale, spkv_stream_t stream) {
  // every refusal comes before anything touches the shared array
  bool empty;
  const int rc_args = decode_check_args(cache, layer, d_seq_ids, B, d_q, d_out, nullptr, &empty);
  if (rc_args || empty) return rc_args;
  const size_t need = spkv_decode_workspace_bytes(&cache->cfg, B);
  if (need > (size_t)SPKV_STATIC_SCRATCH_BYTES) return SPKV_E_SCRATCH_LIMIT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPKV_E_CUDA;
  void *scratch = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // In host code `g_static_scratch` names a host-side stand-in, not device memory: the
    // address a kernel may use has to be asked for, once per device, with that device current.
    if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) return SPKV_E_CUDA;
    g_scratch_ptr[dev].store(scratch, std::memory_order_release);
  }
  // the array keeps whatever the previous call left: the arrival counters must start at zero
  const size_t counters =
      decode_ws_layout(B * cache->cfg.n_kv_heads, cache->cfg.n_q_heads / cache->cfg.n_kv_heads).off_ml;
  for (int half = 0; half < 2; ++half)
    if (cudaMemsetAsync(static_cast<char *>(scratch) + half * (need / 2), 0, counters,
                        as_stream(stream)) != cudaSuccess)
      return SPKV_E_CUDA;
  return spkv_decode_attention(cache, layer, d_seq_ids, B, d_q, d_out, d_lse_opt, sm_scale, scratch,
                               SPKV_STATIC_SCRATCH_BYTES, stream);
}

static size_t a256(size_t x) { return (x + 255) / 256 * 256; }

// ---- decode step from host buffers: a two-slot pipeline over three streams ----------------
//   copy_in : [wait kernels of call i-2]  x, q, k, v -> slot            record ev_in[slot]
//   stream  : [wait ev_in[slot], ev_out[slot] of call i-2] score+append, decode   record ev_k[slot]
//             [wait ev_out of call i-1]
//   copy_out: [wait ev_k[slot]]  out -> host                            record ev_out[slot]
// so the copies of one layer run under the kernels of its neighbours.  After call i the
// caller's stream has waited for the output of call i-1; spkv_decode_step_host_flush makes it
// wait for the last one.
static size_t host_slot_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in) {
  const size_t q = a256((size_t)B * cfg->n_q_heads * kD * 2), kv = a256((size_t)B * cfg->n_kv_heads * kD * 2);
  return a256((size_t)B * d_in * 2) + 2 * q + 2 * kv + a256((size_t)B * cfg->n_kv_heads * 4);
}

extern "C" size_t spkv_decode_step_staging_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in) {
  if (!cfg || B < 0 || d_in < 0) return 0;
  return 2 * host_slot_bytes(cfg, B, d_in) + spkv_decode_workspace_bytes(cfg, B);
}

static int host_pipeline_init(spkv_cache *c) {
  if (c->host_ready) return SPKV_OK;
  if (cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking) != cudaSuccess) return SPKV_E_CUDA;
  if (cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking) != cudaSuccess) return SPKV_E_CUDA;
  for (int i = 0; i < 2; ++i)
    if (cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_k[i], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming) != cudaSuccess)
      return SPKV_E_CUDA;
  c->host_calls = 0;
  c->host_ready = true;
  return SPKV_OK;
}

extern "C" int spkv_decode_step_host(spkv_cache_t *cache, int32_t layer, const spkv_predictor_t *pred,
                                     const int32_t *d_seq_ids, int32_t B, const void *h_x,
                                     const void *h_q, const void *h_k, const void *h_v, void *h_out,
                                     float sm_scale, void *d_staging, size_t staging_bytes,
                                     spkv_stream_t stream) {
  if (!cache || !pred || !h_x || !h_q || !h_k || !h_v || !h_out || B < 1) return SPKV_E_INVALID;
  if (!d_staging || ((uintptr_t)d_staging & 255) ||
      staging_bytes < spkv_decode_step_staging_bytes(&cache->cfg, B, pred->d_in))
    return SPKV_E_WORKSPACE;
  int rc = host_pipeline_init(cache);
  if (rc) return rc;
  const spkv_config_t &cfg = cache->cfg;
  const size_t xb = (size_t)B * pred->d_in * 2, qb = (size_t)B * cfg.n_q_heads * kD * 2,
               kvb = (size_t)B * cfg.n_kv_heads * kD * 2, slot_bytes = host_slot_bytes(&cfg, B, pred->d_in);
  const long long call = cache->host_calls++;
  const int slot = (int)(call & 1);
  char *p = static_cast<char *>(d_staging) + slot * slot_bytes;
  char *d_x = p; p += a256(xb);
  char *d_q = p; p += a256(qb);
  char *d_o = p; p += a256(qb);
  char *d_k = p; p += a256(kvb);
  char *d_v = p; p += a256(kvb);
  float *d_lg = reinterpret_cast<float *>(p);
  void *d_ws = static_cast<char *>(d_staging) + 2 * slot_bytes;
  cudaStream_t s = as_stream(stream);
  // inputs: this slot was last read by the kernels of call - 2
  if (call >= 2 && cudaStreamWaitEvent(cache->copy_in, cache->ev_k[slot], 0) != cudaSuccess) return SPKV_E_CUDA;
  if (cudaMemcpyAsync(d_x, h_x, xb, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
      cudaMemcpyAsync(d_q, h_q, qb, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
      cudaMemcpyAsync(d_k, h_k, kvb, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
      cudaMemcpyAsync(d_v, h_v, kvb, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
      cudaEventRecord(cache->ev_in[slot], cache->copy_in) != cudaSuccess)
    return SPKV_E_CUDA;
  // kernels: after the inputs have landed and the slot's previous output has left
  if (cudaStreamWaitEvent(s, cache->ev_in[slot], 0) != cudaSuccess) return SPKV_E_CUDA;
  if (call >= 2 && cudaStreamWaitEvent(s, cache->ev_out[slot], 0) != cudaSuccess) return SPKV_E_CUDA;
  rc = spkv_score_append_evict(cache, layer, pred, d_seq_ids, B, d_x, d_k, d_v, d_lg, stream);
  if (rc) return rc;
  rc = spkv_decode_attention(cache, layer, d_seq_ids, B, d_q, d_o, nullptr, sm_scale, d_ws,
                             spkv_decode_workspace_bytes(&cfg, B), stream);
  if (rc) return rc;
  if (cudaEventRecord(cache->ev_k[slot], s) != cudaSuccess) return SPKV_E_CUDA;
  // output
  if (cudaStreamWaitEvent(cache->copy_out, cache->ev_k[slot], 0) != cudaSuccess ||
      cudaMemcpyAsync(h_out, d_o, qb, cudaMemcpyDeviceToHost, cache->copy_out) != cudaSuccess ||
      cudaEventRecord(cache->ev_out[slot], cache->copy_out) != cudaSuccess)
    return SPKV_E_CUDA;
  // the caller's stream answers for the output of the call before this one
  if (call >= 1 && cudaStreamWaitEvent(s, cache->ev_out[slot ^ 1], 0) != cudaSuccess) return SPKV_E_CUDA;
  return check_stream_error(cudaGetLastError());
}

extern "C" int spkv_decode_step_host_flush(spkv_cache_t *cache, spkv_stream_t stream) {
  if (!cache) return SPKV_E_INVALID;
  if (!cache->host_ready || cache->host_calls == 0) return SPKV_OK;
  const int last = (int)((cache->host_calls - 1) & 1);
  return check_stream_error(cudaStreamWaitEvent(as_stream(stream), cache->ev_out[last], 0));
}

// ---- one decode step of the WHOLE layer stack from host buffers ------------------------------
// For an attention-only stack every layer's inputs exist before the step starts.  The layers go
// in three chunks -- a short head (a sixteenth of the stack), the bulk, a short tail: each chunk's
// inputs travel in four copies on the cache's input stream, its two launches (the appends of its
// layers, one persistent decode kernel over its layers: spkv_decode_stack's) follow on the
// caller's stream once they have landed, and its outputs leave on the output stream while the
// next chunk computes.  Only the head's inputs and the tail's outputs travel with nothing running
// beside them, so those two are small; the bulk's inputs land under the head's kernels and its
// outputs leave under the tail's.  (Measured with per-layer launches, 32 layers, batch 16:
// 2 + 28 + 2 layers 7440 tokens/s; four chunks of 8 7150; 2 + 14 + 14 + 2 7340; 1 + 30 + 1 7290;
// one chunk 6920.)  The caller's stream ends up waiting for the last output copy: synchronising it
// means the outputs are on the host.
static int stack_pipeline_init(spkv_cache *c) {
  int rc = host_pipeline_init(c);
  if (rc) return rc;
  if (c->stack_ready) return SPKV_OK;
  for (int i = 0; i < kStackChunks; ++i)
    if (cudaEventCreateWithFlags(&c->ev_st_in[i], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_st_k[i], cudaEventDisableTiming) != cudaSuccess)
      return SPKV_E_CUDA;
  if (cudaEventCreateWithFlags(&c->ev_st_start, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_st_done, cudaEventDisableTiming) != cudaSuccess)
    return SPKV_E_CUDA;
  c->stack_ready = true;
  return SPKV_OK;
}

static size_t stack_inputs_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in, size_t *x, size_t *q, size_t *kv,
                                 size_t *lg) {
  *x = a256((size_t)cfg->n_layers * B * d_in * 2);
  *q = a256((size_t)cfg->n_layers * B * cfg->n_q_heads * kD * 2);
  *kv = a256((size_t)cfg->n_layers * B * cfg->n_kv_heads * kD * 2);
  *lg = a256((size_t)cfg->n_layers * B * cfg->n_kv_heads * 4);
  return *x + 2 * *q + 2 * *kv + *lg;
}

extern "C" size_t spkv_decode_stack_staging_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in) {
  if (!cfg || B < 0 || d_in < 0) return 0;
  size_t x, q, kv, lg;
  return stack_inputs_bytes(cfg, B, d_in, &x, &q, &kv, &lg) + spkv_decode_stack_workspace_bytes(cfg, B);
}

extern "C" int spkv_decode_stack_host(spkv_cache_t *cache, const spkv_predictor_t *preds, const int32_t *d_seq_ids,
                                      int32_t B, const void *h_x, const void *h_q, const void *h_k, const void *h_v,
                                      void *h_out, float sm_scale, void *d_staging, size_t staging_bytes,
                                      spkv_stream_t stream) {
  if (!cache || !preds || !h_x || !h_q || !h_k || !h_v || !h_out || B < 1) return SPKV_E_INVALID;
  const spkv_config_t &cfg = cache->cfg;
  const int L = cfg.n_layers, d_in = preds[0].d_in;
  for (int l = 0; l < L; ++l)
    if (preds[l].d_in != d_in) return SPKV_E_INVALID;
  if (!d_staging || ((uintptr_t)d_staging & 255) || staging_bytes < spkv_decode_stack_staging_bytes(&cfg, B, d_in))
    return SPKV_E_WORKSPACE;
  size_t xb, qb, kvb, lgb;
  stack_inputs_bytes(&cfg, B, d_in, &xb, &qb, &kvb, &lgb);
  char *p = static_cast<char *>(d_staging);
  char *d_x = p; p += xb;
  char *d_q = p; p += qb;
  char *d_o = p; p += qb;
  char *d_k = p; p += kvb;
  char *d_v = p; p += kvb;
  float *d_lg = reinterpret_cast<float *>(p); p += lgb;
  const size_t x_l = (size_t)B * d_in * 2, q_l = (size_t)B * cfg.n_q_heads * kD * 2,
               kv_l = (size_t)B * cfg.n_kv_heads * kD * 2;
  cudaStream_t s = as_stream(stream);
  int rc = stack_pipeline_init(cache);
  if (rc) return rc;
  // chunks of layers: a short head, the bulk, a short tail (fewer chunks for a short stack)
  int bounds[kStackChunks + 1];
  int nc;
  {
    const int h = L / 16 > 1 ? L / 16 : 1;
    bounds[0] = 0;
    if (L >= 4 * h) {
      nc = 3;
      bounds[1] = h; bounds[2] = L - h; bounds[3] = L;
    } else {
      nc = L < kStackChunks ? L : kStackChunks;
      for (int ci = 1; ci <= nc; ++ci) bounds[ci] = (int)((size_t)ci * L / nc);
    }
  }
  const char *hx = static_cast<const char *>(h_x), *hq = static_cast<const char *>(h_q),
             *hk = static_cast<const char *>(h_k), *hv = static_cast<const char *>(h_v);
  // the staging buffers are free once everything enqueued on the caller's stream so far has run
  if (cudaEventRecord(cache->ev_st_start, s) != cudaSuccess ||
      cudaStreamWaitEvent(cache->copy_in, cache->ev_st_start, 0) != cudaSuccess)
    return SPKV_E_CUDA;
  for (int ci = 0; ci < nc; ++ci) {
    const size_t l0 = (size_t)bounds[ci], n = (size_t)bounds[ci + 1] - l0;
    if (cudaMemcpyAsync(d_x + l0 * x_l, hx + l0 * x_l, n * x_l, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
        cudaMemcpyAsync(d_q + l0 * q_l, hq + l0 * q_l, n * q_l, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
        cudaMemcpyAsync(d_k + l0 * kv_l, hk + l0 * kv_l, n * kv_l, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
        cudaMemcpyAsync(d_v + l0 * kv_l, hv + l0 * kv_l, n * kv_l, cudaMemcpyHostToDevice, cache->copy_in) != cudaSuccess ||
        cudaEventRecord(cache->ev_st_in[ci], cache->copy_in) != cudaSuccess)
      return SPKV_E_CUDA;
  }
  for (int ci = 0; ci < nc; ++ci) {
    const int l0 = bounds[ci], l1 = bounds[ci + 1];
    if (cudaStreamWaitEvent(s, cache->ev_st_in[ci], 0) != cudaSuccess) return SPKV_E_CUDA;
    // the chunk's layers: their appends in one launch, their decode attention in one persistent launch
    rc = decode_stack_layers(cache, l0, l1, preds, d_seq_ids, B, d_x, d_q, d_k, d_v, d_o, d_lg, nullptr, sm_scale, p,
                             spkv_decode_stack_workspace_bytes(&cfg, B), stream);
    if (rc) return rc;
    if (cudaEventRecord(cache->ev_st_k[ci], s) != cudaSuccess ||
        cudaStreamWaitEvent(cache->copy_out, cache->ev_st_k[ci], 0) != cudaSuccess ||
        cudaMemcpyAsync(static_cast<char *>(h_out) + l0 * q_l, d_o + l0 * q_l, (size_t)(l1 - l0) * q_l,
                        cudaMemcpyDeviceToHost, cache->copy_out) != cudaSuccess)
      return SPKV_E_CUDA;
  }
  cache->last_kind = kLastOther;
  if (cudaEventRecord(cache->ev_st_done, cache->copy_out) != cudaSuccess ||
      cudaStreamWaitEvent(s, cache->ev_st_done, 0) != cudaSuccess)
    return SPKV_E_CUDA;
  return check_stream_error(cudaGetLastError());
}
