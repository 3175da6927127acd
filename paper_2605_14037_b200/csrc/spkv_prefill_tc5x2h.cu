// Chunk attention of spkv_prefill on tcgen05 (Eq. 3-5 for every query of a chunk), two query heads
// per block, P.V in fp16 -- or, for a unit whose values span too wide a range for that, in two
// bf16 terms.
//
// One block = two 128-row slots that walk the same pages -- two query heads that share a KV head
// on one tile of 128 consecutive queries (Eq. 5: head j reads KV head j / G), or, for the last head
// of an odd group (G = 1: every head), two consecutive query tiles of that head; every 32 KB page
// is fetched once and feeds both slots; one softmax group of 128 threads per slot, thread = query
// row = TMEM lane.  ("Head h" below means slot h.)  Per page and slot: S = Q K^T (8 MMAs M128 N64
// K16, S in tensor memory), softmax in registers, O += P V with P taken from tensor memory.
//
// * P is ONE fp16 term (11 significant bits).  The tensor cores want both operands in the same
//   type, so warps 2-3 rewrite the value block of every page from bf16 to fp16 in shared memory,
//   multiplied by a power of two that brings the largest |v| a query of this call can see (the
//   unit's kept pairs, the old ring, the chunk: H_VMAX of the plan header) into [2^14, 2^15); the
//   epilogue undoes the factor exactly.  A bf16 value converts to fp16 without loss unless it is
//   more than 2^28 below that maximum, where fp16 goes subnormal: such a value is off by at most
//   2^-39 of the maximum.  P carries a bias of 2^7 (p <= 2^8 under the lazy rescale), which
//   cancels between O and the row sum.
//
// * "Wide" units: an fp16 P also drops weights below 2^-32 of the row's reference maximum, which
//   is harmless unless such a key carries a value many orders above the others: at max|v| = 2^20
//   a dropped key is worth at most 2^-12 in the output, the value flush above 2^-19.  When the
//   maximum is 2^20 or more the blocks of
//   such a unit -- and every block when the cache was created with SPKV_FLAG_PREFILL_PV_BF16 --
//   leave the values in bf16 and split P into hi + lo bf16 terms (16 significant bits, bf16's
//   exponent range): 8 P.V MMAs per page instead of 4.  The branch is uniform per block.
//
// Two pipelines, chosen at compile time (kDeep = !kSoft): the hard-gated kernel runs the deep one,
// the soft-gated kernel -- whose softmax groups do more per page (gate biases) and set the pace by
// themselves -- the flat one; each measured 3-8 % faster than the other in its place.
//
// * Deep (hard-gated).  Two score buffers per head, and P written back over the scores it came
//   from.  A group copies its row of S(j) into registers, and when the exponentials are done
//   stores P(j) into the first columns of the same buffer; Q.K^T(j+2) goes into that buffer after
//   P.V(j) has read it (the tensor pipe runs a thread's MMAs in order), Q.K^T(j+1) went into the
//   other one a page earlier.  So a group always finds its next scores waiting.  One MMA-issuing
//   warp per head: the tensor pipe takes only a few instructions ahead, the issuing thread blocks
//   until the pipe accepts an MMA, and whatever else that warp does -- wait for a P, commit, turn
//   its loop -- is time in which it feeds the pipe nothing (measured: every 100 cycles of delay put
//   into a single issuing warp's loop lengthened the page period by 75-83).  With a warp per
//   head, each running  wait P(j) | PV(j) | QK(j+2) | commit  for its own head, one head's MMAs
//   fill the gaps of the other's.
//   Tensor memory (512 columns): score buffer b = j & 1 of head h at [64 (2h + b), +64), P(j) in
//   its first 32 columns (two fp16 per column; a wide unit: hi in the first 32, lo in the other
//   32); O of head h at [256 + 128 h, +128).
//
// * Flat (soft-gated).  One score buffer per head and P in columns of its own; a group copies its
//   row of S into registers and hands the buffer back at once (S_FREE), so Q.K^T of the next page
//   runs under the softmax of this one and only P.V waits for P.  One MMA warp, order per page j:
//   QK0(j+1) | PV0(j) | QK1(j+1) | PV1(j): the two heads' scores become ready half a page apart,
//   which keeps the two groups out of step.
//   Tensor memory: S of head h at [64 h, +64); P buffer b of head h at [128 + 32 (2h + b), +32)
//   (a wide unit: hi at [128 + 64 h, +32), lo in the 32 columns after it, one buffer per head:
//   a group then waits for P.V of the previous page before it overwrites P); O as above.
//
// A launch with fewer page walks than SMs (a chunk of a few hundred tokens) cuts every walk into
// up to 16 shares of consecutive pages, one block each; a share writes its unnormalised rows and
// their (m, l), and prefill_merge_kernel combines the shares by their log-sum-exp weights.
//
// What sets the pace of the deep pipeline is the softmax groups: with their scores always waiting
// they are busy ~85 % of the page period, each slowed by the other (alone a group needs ~1060
// cycles per page, side by side ~1550), and no unit is saturated (special-function unit ~60 %,
// issue slots ~55 %); in the flat pipeline it is the chain scores -> softmax -> P -> MMA warp ->
// next scores.
// Shared memory: Q of both heads (64 KB) + 5 page stages (deep: pages j .. j+2 in use).
// Warps: 0 MMA issue (deep: head 0), 1 page loader + TMEM allocation, 2-3 value conversion,
// 4-7 group 0, 8-11 group 1, 12 MMA issue head 1 (deep only).  All waits are bounded.
#include <algorithm>

#include "spkv_prefill_common.cuh"
#include "spkv_tc5.cuh"

namespace spkv {

namespace tc5x2h {
constexpr int kThreads = 416;
// Warp roles.  Both MMA-issuing warps sit on scheduler 0 (warp % 4), the loader on 1, the value
// converters on 2 and 3; every scheduler also runs one warp of each softmax group.  (Measured:
// the MMA warps on different schedulers, or the conversion spread over four warps, lose 1-4 %.)
constexpr int kMmaWarp0 = 0, kMmaWarp1 = 12, kLoaderWarp = 1;
__host__ __device__ constexpr bool is_conv(int w) { return w == 2 || w == 3; }
constexpr int kTmemCols = 512;
constexpr int kSQ = 0;                     // 2 x 32 KB: Q of head 0, head 1 (two slabs of 128 rows x 128 B each)
constexpr int kStages = 5;
constexpr int kSKV = 65536;                // kStages x 32 KB
constexpr int kSBar = kSKV + kStages * kPageBytes;
constexpr int kSGate = kSBar + 512;        // kStages x 64 floats: gate bias of a stage's keys (soft-gated forward)
constexpr int kSmemBytes = kSGate + kStages * kP * 4;
enum { B_KV_FULL = 0, B_KV_EMPTY = 8, B_V_READY = 16 /* [stage] */, B_S_FULL = 24 /* [2h+b] */,
       B_P_FULL = 28 /* [2h+b] */, B_O_DONE = 32 /* [2h+b] */, B_S_FREE = 36 /* [h], flat pipeline only */, B_COUNT = 38 };
constexpr int kConvThreads = 64;           // warps 2-3
constexpr float kPBias = 7.f;              // P is stored as 2^7 p
constexpr int kPartFloats = 128 * 128 + 128 * 2;   // one partial result: O of 128 rows, then (m, l) per row
constexpr int kMaxSplit = 16;
constexpr int kMinSharePages = 16;          // a walk is not cut into shares shorter than this
}  // namespace tc5x2h

#ifdef SPKV_TC5_TRACE
__device__ long long g_tc5h_trace[16][2048];
#ifndef SPKV_TC5_TRACE_MASK
#define SPKV_TC5_TRACE_MASK 0xffff
#endif
#define TC5H_STAMP(cond, who, j) do { if (((SPKV_TC5_TRACE_MASK >> (who)) & 1) && (cond) && (j) < 2048) g_tc5h_trace[who][j] = clock64(); } while (0)
#else
#define TC5H_STAMP(cond, who, j) do { } while (0)
#endif

// A page walk serves two 128-row slots: two query heads of a KV head on one query tile, or -- for
// the last head of an odd group (G = 1: every head) -- two consecutive query tiles of that one
// head (one tile and an idle slot when the launch would otherwise have too few blocks to fill
// the GPU: a.pair_tiles = 0).  Work order: KV heads by keys per query, heaviest first; inside a
// head the head pairs tile by tile from the end of the chunk backwards, then the single head's
// tile pairs likewise.  Called by whole warps.
struct WalkSlots {
  int kvh, hq0, hq1, i00, i01;   // slot h: query head hq<h>, first query row i0<h>
  bool two;                      // is slot 1 in use
};
template <bool kEvenG>
__device__ inline WalkSlots walk_slots(const PrefillArgs &a, int walk) {
  const CacheView &c = a.c;
  const int n_xtiles = (a.C + 127) / 128, n_xpairs = a.pair_tiles ? (n_xtiles + 1) / 2 : n_xtiles;
  const int per_kvh = (c.G >> 1) * n_xtiles + (c.G & 1) * n_xpairs;
  WalkSlots w;
  w.kvh = prefill_kvh_by_rank(a, walk / per_kvh);
  const int rem = walk % per_kvh;
  if (kEvenG || rem < (c.G >> 1) * n_xtiles) {
    const int pair = rem / n_xtiles, xtile = n_xtiles - 1 - rem % n_xtiles;
    w.hq0 = w.kvh * c.G + pair * 2; w.hq1 = w.hq0 + 1;
    w.i00 = w.i01 = xtile * 128;
    w.two = true;
  } else {
    const int xp = n_xpairs - 1 - (rem - (c.G >> 1) * n_xtiles);
    w.hq0 = w.hq1 = w.kvh * c.G + c.G - 1;
    w.i00 = a.pair_tiles ? xp * 256 : xp * 128;
    w.i01 = w.i00 + 128;
    w.two = a.pair_tiles && w.i01 < a.C;
  }
  return w;
}
// Is the unit "wide" (two-term bf16 P.V), and otherwise the power of two that brings the largest
// visible |v| into [2^14, 2^15), with its inverse.  vm: fp32 bit pattern of that largest |v|.
constexpr uint32_t kWideFrom = 0x49800000u;   // 2^20
__device__ inline bool value_scale(uint32_t vm, int force_wide, float &v_scale, float &v_unscale) {
  v_scale = v_unscale = 1.f;
  if (force_wide || vm >= kWideFrom) return true;
  if (vm) {
    const int k = min(14 - ((int)(vm >> 23) - 127), 126);
    v_scale = __int_as_float((127 + k) << 23);
    v_unscale = __int_as_float((127 - k) << 23);
  }
  return false;
}

// Pages of a walk: the compact-cache pages its last query sees (*n_ptiles), then the band pages
// sp_lo ... of the staging area; the soft-gated forward walks every page from the start.
template <bool kSoft>
__device__ inline int walk_pages(const PrefillArgs &a, const WalkSlots &w, int *n_ptiles, int *sp_lo) {
  const int32_t *hdr = unit_ws(a, w.kvh);
  const int32_t *E = hdr + kHdrInts;
  const int len0 = hdr[H_LEN0], n_old = hdr[H_NOLD], N = hdr[H_N];
  // the last query of the block (slot 1 never starts before slot 0) sees the most kept pairs
  const int i_first = w.i00, i_last = min((w.two ? w.i01 : w.i00) + 127, a.C - 1);
  const int nv = kSoft ? 0 : len0 + E[min(max(i_last + n_old - a.c.w + 1, 0), N)];
  *n_ptiles = (nv + kP - 1) / kP;
  *sp_lo = kSoft ? 0 : max(0, i_first + n_old - a.c.w + 1) / kP;
  return *n_ptiles + ((i_last + n_old) / kP - *sp_lo + 1);
}
// Shares a walk of n_pages pages is cut into, one block each, when the launch has a.n_split
// blocks per walk.  A launch with fewer walks than SMs cuts every walk into runs of 16 pages.
// A launch of one to two and a half waves of walks cuts a walk only when it is long against the
// launch's fair share per SM (all pages of all walks / SMs, estimated from the plan headers: a KV
// head's walks see its kept pairs from before the call plus, on average, half of those the chunk
// adds, and ~3 band pages): a share costs a block's start-up, its partial result (128 KB) and the
// merge, which only pays where a walk would otherwise outlast the rest of the launch -- a KV
// head that keeps far more than the others.  Walks that stay whole write their output directly.
// (Measured, TFLOP/s useful, 32 k past: 32 query / 8 KV heads with keep rates 0 - 0.9, chunk 1536:
// 660 against 630 with every walk cut in four and 414 uncut; 8 / 2 heads, rates 0.15 / 0.6, chunk
// 8192: 941 against 861 and 973.)
constexpr float kSplitThr = 1.25f, kSplitFrac = 0.6f;
template <bool kSoft>
__device__ inline int walk_shares(const PrefillArgs &a, int n_pages) {
  if (a.n_split <= 1) return 1;   // (uniform over the block)
  // fewer walks than SMs: as many shares as there are runs of kMinSharePages pages
  if (a.split_unit == 0.f) return max(1, min(a.n_split, n_pages / tc5x2h::kMinSharePages));
  // (called by whole warps: one lane per KV head, so that the headers are fetched side by side)
  float total = 0.f;
  for (int k = threadIdx.x & 31; k < a.c.Hkv; k += 32) {
    const int32_t *hd = unit_ws(a, k);
    const float kept = kSoft ? 0.5f * a.C : hd[H_LEN0] + 0.5f * (hd + kHdrInts)[hd[H_N]];
    total += kept * (1.f / kP) + 3.f;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
  const float fair = total * a.walks_per_kvh / a.split_unit;
  if (n_pages <= kSplitThr * fair || n_pages < 2 * tc5x2h::kMinSharePages) return 1;
  const float share = fmaxf((float)tc5x2h::kMinSharePages, kSplitFrac * fair);
  return max(1, min(a.n_split, (int)ceilf(n_pages / share)));
}

// kEvenG: every block is a head pair on one tile (the branches for single heads compile away).
// kSoft: the soft-gated whole-sequence forward (Eq. 6): no compact-cache pages, the walk covers
// every causal page of the sequence, and a key beyond a query's window is not masked but biased
// by the logarithm of its gate.  The gate biases of a page's 64 keys travel with the page into
// shared memory (one 256-byte bulk copy on the same barrier), once per page for all 256 rows.
template <bool kEvenG, bool kSoft>
__global__ void __launch_bounds__(tc5x2h::kThreads, 1) prefill_attn_tc5x2h_kernel(PrefillArgs a) {
  using namespace tc5;
  using namespace tc5x2h;
  constexpr bool kDeep = !kSoft;   // which of the two pipelines (see the head of the file)
  extern __shared__ __align__(1024) unsigned char smem[];
  pdl_chain_link();
  const CacheView &c = a.c;
  uint64_t *bar = reinterpret_cast<uint64_t *>(smem + kSBar);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kSBar + B_COUNT * 8);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // a.n_split blocks share one page walk (small launches: see the launcher)
  const int walk = blockIdx.x / a.n_split, split = blockIdx.x % a.n_split;
  const WalkSlots ws = walk_slots<kEvenG>(a, walk);
  const int kvh = ws.kvh, hq_s0 = ws.hq0, hq_s1 = ws.hq1, i0_s0 = ws.i00, i0_s1 = ws.i01;
  bool two = ws.two;
  const int32_t *hdr = unit_ws(a, kvh);
  const int32_t *E = hdr + kHdrInts;
  const int len0 = hdr[H_LEN0], n_old = hdr[H_NOLD], N = hdr[H_N];
  const int u = unit_index(c, a.layer, a.seq, kvh);
  // fp16 P.V: the values are multiplied by 2^k with the largest visible |v| brought into
  // [2^14, 2^15); the epilogue multiplies by 2^-k.  A wide unit keeps bf16 values (factor 1).
  float v_scale, v_unscale;
  const bool wide = value_scale((uint32_t)hdr[H_VMAX], a.force_wide, v_scale, v_unscale);
  // kept pairs visible to chunk query i: the first nvis(i) pairs of the compact cache
  auto nvis = [&](int i) { return kSoft ? 0 : len0 + E[min(max(i + n_old - c.w + 1, 0), N)]; };
  if (kEvenG) two = true;
  // band of both slots together, in staging indices (query i is staging pair n_old + i)
  int n_ptiles, sp_lo;
  const int n_tiles_all = walk_pages<kSoft>(a, ws, &n_ptiles, &sp_lo);
  // this block's share of the walk: pages [j_begin, j_begin + n_tiles) of the list (compact-cache
  // pages, then band pages); page numbers below are local, j_begin + j is the page's place in the
  // list.  The blocks of a walk beyond its number of shares leave at once.
  const int n_shares = walk_shares<kSoft>(a, n_tiles_all);
  if (split >= n_shares) return;
  const int j_begin = (int)((long long)n_tiles_all * split / n_shares);
  const int n_tiles = (int)((long long)n_tiles_all * (split + 1) / n_shares) - j_begin;

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&bar[B_KV_FULL + i], 1);
      mbar_init(&bar[B_KV_EMPTY + i], (kDeep && (kEvenG || ws.two)) ? 2 : 1);   // one commit per MMA warp at work
      mbar_init(&bar[B_V_READY + i], kConvThreads);
    }
    // Deep pipeline.  S_FULL / P_FULL / O_DONE: one barrier per head and page parity b = j & 1 (the
    // score buffer the page uses), one phase per two pages.  The scores of page j+2 go into the
    // buffer of page j and are issued after P.V(j), which needs P(j): a barrier is never more than
    // one phase ahead of the group that waits on it.  O_DONE is committed for the last two pages.
    // Flat pipeline.  S_FULL / S_FREE: one barrier per head (index 2h), one phase per page -- the
    // MMA thread commits the scores of page j+1 only after the group has freed the buffer of page
    // j, and the group frees it only after seeing it full, so the two are never more than one
    // phase apart.  P_FULL / O_DONE per head and page parity: a group may hand over P(j+1) before
    // the MMA thread has looked at P(j); P(j+2) cannot follow before that, it needs the scores of
    // page j+2, whose Q.K^T is issued after P.V(j).
    for (int i = 0; i < 4; ++i) {
      mbar_init(&bar[B_S_FULL + i], 1);
      mbar_init(&bar[B_P_FULL + i], 128);
      mbar_init(&bar[B_O_DONE + i], 1);
    }
    mbar_init(&bar[B_S_FREE + 0], 128);
    mbar_init(&bar[B_S_FREE + 1], 128);
    mbar_fence_init();
  }
  // Q tiles -> per head two slabs of 128 rows x 128 B, 128-byte swizzle (rows past the chunk are zero)
  for (int x = tid; x < 2 * 128 * 16; x += kThreads) {
    const int h = x >> 11, r = (x >> 4) & 127, ch = x & 15;
    uint4 val = make_uint4(0, 0, 0, 0);
    const int i0h = h ? i0_s1 : i0_s0, hqh = h ? hq_s1 : hq_s0;
    if (i0h + r < a.C && (h == 0 || two))
      val = *reinterpret_cast<const uint4 *>(a.q + ((size_t)(i0h + r) * c.Hq + hqh) * kD + ch * 8);
    *reinterpret_cast<uint4 *>(smem + kSQ + h * 32768 + (ch >> 3) * 16384 + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = val;
  }
  fence_async_smem();
  if (warp == kLoaderWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tbase = *tmem_slot;
  bool failed = false;
#ifdef SPKV_TC5_TRACE
  const bool traced = blockIdx.x == 0;
#endif

  if (warp == kLoaderWarp) {
    // ---------------------------------------------------------------- page loader
    int j = 0;
    for (int base = 0; base < n_tiles && !failed; base += 32) {
      const int jl = j_begin + base + lane;
      int64_t src_off = 0;
      if (jl < n_ptiles)   // (debug bounds: an entry that names no pool page is read from the unit's ring instead)
        src_off = (int64_t)checked_page(c, unit_table(c, c.table_row[u])[jl], (int)ring_page(c, u, 0)) * kPageElems;
      const int cnt = min(32, n_tiles - base);
      for (int x = 0; x < cnt; ++x, ++j) {
        const int64_t off = __shfl_sync(0xffffffffu, src_off, x);
        if (lane == 0) {
          const int s = j % kStages;
          if (j >= kStages && !mbar_wait_bounded(&bar[B_KV_EMPTY + s], ((j / kStages) - 1) & 1)) failed = true;
          if (!failed) {
            const __nv_bfloat16 *src =
                j_begin + j < n_ptiles
                    ? c.pages + off
                    : a.stage_pages + ((size_t)kvh * a.n_stage_pages + sp_lo + (j_begin + j - n_ptiles)) * kPageElems;
            mbar_arrive_expect_tx(&bar[B_KV_FULL + s], kPageBytes + (kSoft ? kP * 4 : 0));
            bulk_load(smem + kSKV + s * kPageBytes, src, kPageBytes, &bar[B_KV_FULL + s]);
            if (kSoft)   // the gate biases of the page's 64 keys
              bulk_load(smem + kSGate + s * kP * 4,
                        a.gate2 + ((size_t)kvh * a.n_stage_pages + (j_begin + j)) * kP, kP * 4, &bar[B_KV_FULL + s]);
          }
        }
        failed = __shfl_sync(0xffffffffu, (int)failed, 0) != 0;
        if (failed) break;
      }
    }
    if (failed && lane == 0)  // do not leave while copies may still be landing
      for (int k = max(0, j - kStages); k < j; ++k)
        mbar_wait_bounded(&bar[B_KV_FULL + (k % kStages)], (k / kStages) & 1);
  } else if (kDeep && (warp == kMmaWarp0 || warp == kMmaWarp1)) {
    // ---------------------------------------------------------------- MMA issue (whole warp, one elected lane issues)
    // Deep pipeline: one warp per head.  Issuing blocks while the tensor pipe's short queue is
    // full, and everything else the warp does (barrier waits, commits, its loop) is time in which
    // it feeds the pipe nothing; the other head's warp fills those gaps.
    const int h_first = warp == kMmaWarp0 ? 0 : 1;
    const int h_count = (h_first == 0 || two) ? 1 : 0;
    constexpr uint32_t idesc_qk = instr_desc(128, 64, false), idesc_pv = instr_desc(128, 128, true, true),
                       idesc_pv_bf16 = instr_desc(128, 128, true, false);
    constexpr uint32_t kStageUnits = kPageBytes >> 4;   // a page stage in descriptor address units
    const uint32_t kv0 = smem_u32(smem + kSKV);
    const uint64_t dQ0 = smem_desc(smem_u32(smem + kSQ), 16, 1024);   // head 1: 32 KB = 2048 units later
    const uint64_t dK = smem_desc(kv0, 16, 1024), dV = smem_desc(kv0 + kBlockElems * 2, 8192, 1024);
    // S_h = Q_h . K^T of the page in `stage` into score buffer b, committed at once
    auto issue_qk = [&](int h, uint32_t stage, uint32_t ph, uint32_t b) {
      if (!mbar_wait_bounded(&bar[B_KV_FULL + stage], ph)) { failed = true; return; }
      fence_after();
      umma_qk_page<16384 / 16, 8192 / 16>(tbase + (2 * h + b) * 64, dQ0 + h * 2048, dK + stage * kStageUnits, idesc_qk);
      umma_commit(&bar[B_S_FULL + 2 * h + b]);
    };
    const int n_mine = h_count ? n_tiles : 0;
    for (int jj = 0; jj < min(2, n_mine) && !failed; ++jj)   // the scores of the first two pages
      for (int h = h_first; h < h_first + h_count && !failed; ++h) issue_qk(h, jj, 0, jj);
    uint32_t st = 0, ph = 0, st2 = 2, ph2 = 0;   // stage and phase parity of pages j and j + 2
    for (int j = 0; j < n_mine && !failed; ++j) {
      const uint32_t b = j & 1;
      TC5H_STAMP(traced && lane == 0, 15 - h_first, j);
      if (!mbar_wait_bounded(&bar[B_V_READY + st], ph)) { failed = true; break; }
      for (int h = h_first; h < h_first + h_count && !failed; ++h) {
        // O_h += P_h(j) . V(j): A = P from tensor memory (it lies where the page's scores lay), B =
        // the page's value block (fp16 by now), MN-major
        if (!mbar_wait_bounded(&bar[B_P_FULL + 2 * h + b], (j >> 1) & 1)) { failed = true; break; }
        TC5H_STAMP(traced && lane == 0, 8 + h, j);
        fence_after();
        const uint32_t t_p = tbase + (2 * h + b) * 64, t_o = tbase + 256 + h * 128;
        if (wide)
          umma_pv_page(t_o, t_p, dV + st * kStageUnits, idesc_pv_bf16, j > 0 ? 1u : 0u);
        else
          umma_pv_page_f16(t_o, t_p, dV + st * kStageUnits, idesc_pv, j > 0 ? 1u : 0u);
        TC5H_STAMP(traced && lane == 0, 13 - h, j);
        if (j + 2 < n_tiles) {
          // the tensor pipe runs a thread's instructions in order: Q.K^T(j+2) overwrites the buffer
          // only after P.V(j) has read P from it, and its S_FULL vouches for that P.V
          issue_qk(h, st2, ph2, b);
        } else {
          umma_commit(&bar[B_O_DONE + 2 * h + b]);   // the last two P.V have no later Q.K^T
        }
        TC5H_STAMP(traced && lane == 0, 11 - h, j);
      }
      if (failed) break;
      umma_commit(&bar[B_KV_EMPTY + st]);  // this warp's head(s) have no use for page j any more
      if (++st == kStages) { st = 0; ph ^= 1; }
      if (++st2 == kStages) { st2 = 0; ph2 ^= 1; }
    }
  } else if (!kDeep && warp == kMmaWarp0) {
    // ---------------------------------------------------------------- MMA issue, flat pipeline (whole warp, one elected lane issues)
    // Order per page j:  QK0(j+1) | PV0(j) | QK1(j+1) | PV1(j).  The two heads' scores become ready
    // half a page apart, which keeps the two groups out of step.
    constexpr uint32_t idesc_qk = instr_desc(128, 64, false), idesc_pv = instr_desc(128, 128, true, true),
                       idesc_pv_bf16 = instr_desc(128, 128, true, false);
    const uint32_t sQ = smem_u32(smem + kSQ);
    auto wait_page = [&](int jj) {
      if (!mbar_wait_bounded(&bar[B_KV_FULL + jj % kStages], (jj / kStages) & 1)) failed = true;
      fence_after();
    };
    auto issue_qk = [&](int h, int jj) {  // S_h = Q_h . K(jj)^T, committed at once
      const uint32_t sK = smem_u32(smem + kSKV + (jj % kStages) * kPageBytes);
      umma_qk_page<16384 / 16, 8192 / 16>(tbase + h * 64, smem_desc(sQ + h * 32768, 16, 1024), smem_desc(sK, 16, 1024),
                                          idesc_qk);
      umma_commit(&bar[B_S_FULL + h]);
    };
    // the group has copied the scores of page jj out of the S buffer
    auto wait_s_free = [&](int h, int jj) {
      if (!mbar_wait_bounded(&bar[B_S_FREE + h], jj & 1)) failed = true;
      fence_after();
    };
    // O_h += P_h(jj) . V(jj): A from tensor memory, B = the page's value block (fp16 by now), MN-major
    auto issue_pv = [&](int h, int jj) {
      if (!mbar_wait_bounded(&bar[B_P_FULL + 2 * h + (jj & 1)], (jj >> 1) & 1)) failed = true;
      fence_after();
      if (failed) return;
      const uint32_t sV = smem_u32(smem + kSKV + (jj % kStages) * kPageBytes) + kBlockElems * 2;
      if (wide)
        umma_pv_page(tbase + 256 + h * 128, tbase + 128 + h * 64, smem_desc(sV, 8192, 1024), idesc_pv_bf16,
                     jj > 0 ? 1u : 0u);
      else
        umma_pv_page_f16(tbase + 256 + h * 128, tbase + 128 + (2 * h + (jj & 1)) * 32, smem_desc(sV, 8192, 1024),
                         idesc_pv, jj > 0 ? 1u : 0u);
      // the last two P.V have no later Q.K^T whose S_FULL would vouch for their completion
      if (jj + 2 >= n_tiles) umma_commit(&bar[B_O_DONE + 2 * h + (jj & 1)]);
    };
    wait_page(0);
    if (!failed) {
      issue_qk(0, 0);
      if (two) issue_qk(1, 0);
    }
    for (int j = 0; j < n_tiles && !failed; ++j) {
      const bool more = j + 1 < n_tiles;
      if (more) {
        wait_page(j + 1);
        wait_s_free(0, j);
        if (failed) break;
        issue_qk(0, j + 1);
      }
      if (!mbar_wait_bounded(&bar[B_V_READY + j % kStages], (j / kStages) & 1)) failed = true;
      if (failed) break;
      issue_pv(0, j);
      if (failed) break;
      if (more && two) {
        wait_s_free(1, j);
        if (failed) break;
        issue_qk(1, j + 1);
      }
      if (two) issue_pv(1, j);
      if (failed) break;
      umma_commit(&bar[B_KV_EMPTY + (j % kStages)]);  // page j has no reader left
    }
  } else if (is_conv(warp)) {
    // ---------------------------------------------------------------- value converter (warps 2-3)
    // bf16 -> fp16 in place, in the swizzled layout the copy left (element positions do not move);
    // a wide unit's values stay as they are
    const int ct = tid - 64;
    for (int j = 0; j < n_tiles; ++j) {
      const int s = j % kStages;
      if (!mbar_wait_bounded(&bar[B_KV_FULL + s], (j / kStages) & 1)) { failed = true; break; }
      uint4 *vb = reinterpret_cast<uint4 *>(smem + kSKV + s * kPageBytes + kBlockElems * 2) + ct;
#pragma unroll
      for (int x = 0; x < (wide ? 0 : 1024 / kConvThreads); ++x) {
        uint4 r = vb[x * kConvThreads];
        r.x = bf16x2_to_f16x2(r.x, v_scale); r.y = bf16x2_to_f16x2(r.y, v_scale);
        r.z = bf16x2_to_f16x2(r.z, v_scale); r.w = bf16x2_to_f16x2(r.w, v_scale);
        vb[x * kConvThreads] = r;
      }
      fence_async_smem();
      mbar_arrive(&bar[B_V_READY + s]);
    }
  } else if (warp >= 4 && warp < 12) {
    // ---------------------------------------------------------------- softmax groups
    const int h = (warp >> 2) - 1, row = tid & 127, i = (h ? i0_s1 : i0_s0) + row, hq = h ? hq_s1 : hq_s0;
    const bool row_ok = i < a.C;
    const int nv = row_ok ? nvis(i) : 0;
    const int jq = n_old + i;  // staging index of this row's own pair
    const uint32_t t_lane = tbase + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t t_o = t_lane + 256 + h * 128;
    float m_ref = -INFINITY, l = 0.f;
    const int n_mine = (h == 0 || two) ? n_tiles : 0;   // the idle group of a one-head block has no pages
    // the scores of page jj are complete (waiting does not consume the phase)
    auto s_full_wait = [&](int jj) {
      return kDeep ? mbar_wait_bounded(&bar[B_S_FULL + 2 * h + (jj & 1)], (jj >> 1) & 1)
                   : mbar_wait_bounded(&bar[B_S_FULL + h], jj & 1);
    };
    for (int j = 0; j < n_mine; ++j) {
      if (!s_full_wait(j)) { failed = true; break; }
      TC5H_STAMP(traced && row == 0, h * 4 + 0, j);
      fence_after();
      // deep: the page's score buffer, and P goes back into it; flat: the head's one score buffer
      const uint32_t t_s = t_lane + (kDeep ? (2 * h + (j & 1)) * 64 : h * 64);
      float v[64];
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        float t16[16];
        tmem_ld16(t_s + q4 * 16, t16);
#pragma unroll
        for (int x = 0; x < 16; ++x) v[q4 * 16 + x] = t16[x];
      }
      tmem_ld_wait();
      if (!kDeep) {   // the scores are in registers: Q.K^T of the next page may overwrite the buffer
        fence_before();
        mbar_arrive(&bar[B_S_FREE + h]);
      }
      TC5H_STAMP(traced && row == 0, h * 4 + 1, j);
      // visibility: compact-cache page j -> first nv pairs; staging page -> the band of this row.
      // v keeps the raw scores (masked ones become -inf); the scale is folded into the exponent,
      // and pages that every row of the warp sees in full skip the masking altogether.
      const int jg = j_begin + j;   // the page's place in the list
      float mx;
      if (kSoft) {
        // Eq. 6: score * scale + bias, bias = 0 inside the window, log2 of the key's gate before
        // it, -inf for the future.  v becomes the biased score in the log2 domain.
        const int base = jg * kP;
        // the copy that brought the page also brought its gate biases (completed before the scores
        // were committed; observing the barrier here makes the bytes visible to this thread)
        if (!mbar_wait_bounded(&bar[B_KV_FULL + j % kStages], (j / kStages) & 1)) { failed = true; break; }
        const float4 *gs = reinterpret_cast<const float4 *>(smem + kSGate + (j % kStages) * kP * 4);
        if (__all_sync(0xffffffffu, row_ok && base + kP - 1 <= jq - c.w)) {
          // the whole page lies before the window of every row of this warp: gate bias everywhere
#pragma unroll
          for (int x4 = 0; x4 < 16; ++x4) {
            const float4 g4 = gs[x4];
            v[4 * x4] = fmaf(v[4 * x4], a.scale_log2, g4.x);
            v[4 * x4 + 1] = fmaf(v[4 * x4 + 1], a.scale_log2, g4.y);
            v[4 * x4 + 2] = fmaf(v[4 * x4 + 2], a.scale_log2, g4.z);
            v[4 * x4 + 3] = fmaf(v[4 * x4 + 3], a.scale_log2, g4.w);
          }
        } else {
#pragma unroll
          for (int x4 = 0; x4 < 16; ++x4) {
            const float4 g4 = gs[x4];
            const float gg[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
            for (int y = 0; y < 4; ++y) {
              const int jj = base + 4 * x4 + y;
              const float sc = fmaf(v[4 * x4 + y], a.scale_log2, jj > jq - c.w ? 0.f : gg[y]);
              v[4 * x4 + y] = (row_ok && jj <= jq) ? sc : -INFINITY;
            }
          }
        }
      } else if (jg < n_ptiles) {
        const int base = jg * kP;
        if (!__all_sync(0xffffffffu, base + kP <= nv)) {
#pragma unroll
          for (int x = 0; x < 64; ++x) v[x] = (base + x < nv) ? v[x] : -INFINITY;
        }
      } else {
        const int base = (sp_lo + jg - n_ptiles) * kP;
#pragma unroll
        for (int x = 0; x < 64; ++x) {
          const int jj = base + x;
          v[x] = (row_ok && jj <= jq && jj > jq - c.w) ? v[x] : -INFINITY;
        }
      }
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int x = 0; x < 64; x += 8) {
        mx0 = max3(mx0, v[x], v[x + 1]);
        mx1 = max3(mx1, v[x + 2], v[x + 3]);
        mx2 = max3(mx2, v[x + 4], v[x + 5]);
        mx3 = max3(mx3, v[x + 6], v[x + 7]);
      }
      // (the hard-gated path keeps raw scores in v and folds the scale, > 0, into the exponent)
      mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * (kSoft ? 1.f : a.scale_log2);
      // the reference maximum moves only when the row maximum outgrows it by 2^8
      const bool grow = mx > m_ref + 8.f;
      const float m_new = grow ? mx : m_ref;
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
        // O is stable between the completion of PV(j-1) and the hand-over of P(j).  QK(j+1) is
        // issued after PV(j-1) and needs nothing more from this group, so S_FULL(j+1) vouches for
        // it (waiting on it here does not consume the phase); the last page has its own barrier.
        if (!(j + 1 < n_tiles ? s_full_wait(j + 1) : mbar_wait_bounded(&bar[B_O_DONE + 2 * h + ((j - 1) & 1)], 0))) {
          failed = true;
          break;
        }
        fence_after();
        const float f = grow ? fast_exp2(m_ref - m_new) : 1.f;  // m_ref = -inf -> 0
#pragma unroll
        for (int q8 = 0; q8 < 8; ++q8) {
          float t16[16];
          tmem_ld16(t_o + q8 * 16, t16);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 16; ++x) t16[x] *= f;
          tmem_st16(t_o + q8 * 16, t16);
        }
        l *= f;
      }
      m_ref = m_new;
      TC5H_STAMP(traced && row == 0, h * 4 + 2, j);
      const float ms = m_ref == -INFINITY ? 0.f : m_ref;
      // two elements per instruction where the hardware has a packed form (fma, add, sub)
      const float bias = wide ? 0.f : kPBias;
      const uint64_t sc2 = pack2(a.scale_log2, a.scale_log2), nms2 = pack2(bias - ms, bias - ms);
      uint64_t l2a = pack2(0.f, 0.f), l2b = l2a;
      if (wide) {
        // deep: hi in the first 32 columns of the page's score buffer, lo in the other 32.
        // flat: one P buffer per head (hi, then lo): P.V of the previous page must have read it;
        // Q.K^T(j+1) is issued after P.V(j-1), so S_FULL(j+1) vouches for it; the last page has its
        // own barrier.
        if (!kDeep && j > 0 &&
            !(j + 1 < n_tiles ? s_full_wait(j + 1) : mbar_wait_bounded(&bar[B_O_DONE + 2 * h + ((j - 1) & 1)], 0))) {
          failed = true;
          break;
        }
        if (!kDeep) fence_after();
        const uint32_t t_p = kDeep ? t_s : t_lane + 128 + h * 64;
#pragma unroll
        for (int q2 = 0; q2 < 2; ++q2) {  // 32 keys -> 16 columns of hi, 16 of lo
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            float e0, e1, r0, r1;
            const uint64_t v2 = pack2(v[q2 * 32 + 2 * x], v[q2 * 32 + 2 * x + 1]);
            unpack2(kSoft ? add2(v2, nms2) : fma2(v2, sc2, nms2), e0, e1);
            const float p0 = fast_exp2(e0), p1 = fast_exp2(e1);
            const uint64_t p2 = pack2(p0, p1);
            if (x & 1) l2b = add2(l2b, p2); else l2a = add2(l2a, p2);
            const __nv_bfloat162 hb = __floats2bfloat162_rn(p0, p1);
            hi[x] = *reinterpret_cast<const uint32_t *>(&hb);
            unpack2(sub2(p2, pack2(__uint_as_float(hi[x] << 16), __uint_as_float(hi[x] & 0xffff0000u))), r0, r1);
            lo[x] = pack_bf16(r0, r1);
          }
          tmem_st16u(t_p + q2 * 16, hi);
          tmem_st16u(t_p + 32 + q2 * 16, lo);
        }
      } else {
        // deep: the first 32 columns of the page's score buffer; flat: P buffer j & 1 of the head
        // (free: S_FULL(j) completed after P.V(j-2))
        const uint32_t t_p = kDeep ? t_s : t_lane + 128 + (2 * h + (j & 1)) * 32;
#pragma unroll
        for (int q2 = 0; q2 < 2; ++q2) {  // 32 keys -> 16 columns of fp16 pairs
          uint32_t ph[16];
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            float e0, e1;
            const uint64_t v2 = pack2(v[q2 * 32 + 2 * x], v[q2 * 32 + 2 * x + 1]);
            unpack2(kSoft ? add2(v2, nms2) : fma2(v2, sc2, nms2), e0, e1);
            const float p0 = fast_exp2(e0), p1 = fast_exp2(e1);
            const uint64_t p2 = pack2(p0, p1);
            if (x & 1) l2b = add2(l2b, p2); else l2a = add2(l2a, p2);
            ph[x] = pack_f16(p0, p1);
          }
          tmem_st16u(t_p + q2 * 16, ph);
        }
      }
      {
        float la, lb;
        unpack2(add2(l2a, l2b), la, lb);
        l += la + lb;
      }
      tmem_st_wait();
      fence_before();
      mbar_arrive(&bar[B_P_FULL + 2 * h + (j & 1)]);
      TC5H_STAMP(traced && row == 0, h * 4 + 3, j);
    }
    if (h == 1 && !two) {
      // idle slot: nothing to write
    } else if (n_shares > 1) {
      // a share of a split walk: the unnormalised row (fp32, in the scaled units) and its (m, l)
      // go to the partial results; prefill_merge_kernel puts the shares together
      float *part = a.partials + ((size_t)(walk * 2 + h) * a.n_split + split) * kPartFloats;
      if (!failed && mbar_wait_bounded(&bar[B_O_DONE + 2 * h + ((n_tiles - 1) & 1)], 0)) {
        fence_after();
#pragma unroll
        for (int q8 = 0; q8 < 8; ++q8) {
          float t16[16];
          tmem_ld16(t_o + q8 * 16, t16);
          tmem_ld_wait();
          float4 *dst = reinterpret_cast<float4 *>(part + row * 128 + q8 * 16);
          dst[0] = make_float4(t16[0], t16[1], t16[2], t16[3]);
          dst[1] = make_float4(t16[4], t16[5], t16[6], t16[7]);
          dst[2] = make_float4(t16[8], t16[9], t16[10], t16[11]);
          dst[3] = make_float4(t16[12], t16[13], t16[14], t16[15]);
        }
        part[128 * 128 + row * 2] = m_ref;
        part[128 * 128 + row * 2 + 1] = l;
      } else {
        failed = true;
      }
    } else if (!failed && mbar_wait_bounded(&bar[B_O_DONE + 2 * h + ((n_tiles - 1) & 1)], 0)) {
      fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;  // the bias of P cancels between O and l
      __nv_bfloat16 *orow = a.out + ((size_t)i * c.Hq + hq) * kD;
      if (a.lse && row_ok)   // l = sum 2^(s - m_ref + bias)
        a.lse[(size_t)i * c.Hq + hq] = (m_ref - (wide ? 0.f : kPBias) + log2f(l)) * 0.6931471805599453f;
#pragma unroll
      for (int q8 = 0; q8 < 8; ++q8) {
        float t16[16];
        tmem_ld16(t_o + q8 * 16, t16);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 16; ++x) t16[x] = t16[x] * inv * v_unscale;  // |O| / l < 2^15 in the scaled units, then <= max |v|
        if (row_ok) {
          uint4 w0, w1;
          w0.x = pack_bf16(t16[0], t16[1]);   w0.y = pack_bf16(t16[2], t16[3]);
          w0.z = pack_bf16(t16[4], t16[5]);   w0.w = pack_bf16(t16[6], t16[7]);
          w1.x = pack_bf16(t16[8], t16[9]);   w1.y = pack_bf16(t16[10], t16[11]);
          w1.z = pack_bf16(t16[12], t16[13]); w1.w = pack_bf16(t16[14], t16[15]);
          *reinterpret_cast<uint4 *>(orow + q8 * 16) = w0;
          *reinterpret_cast<uint4 *>(orow + q8 * 16 + 8) = w1;
        }
      }
    } else {
      failed = true;
    }
  }
  if (failed) set_status(c, SPKV_E_TIMEOUT);
  fence_before();
  __syncthreads();
  if (warp == kLoaderWarp)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "n"(tc5x2h::kTmemCols) : "memory");
}

#ifdef SPKV_TC5_TRACE
extern "C" int spkv_debug_tc5h_trace(long long *host_out) {
  return cudaMemcpyFromSymbol(host_out, g_tc5h_trace, sizeof(g_tc5h_trace)) == cudaSuccess ? 0 : -1;
}
#endif

// Puts the shares of a split page walk together: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s
// (M = max_s m_s; the m are log2-domain reference maxima, the O and l carry the same bias and value
// scale in every share).  grid (walks, 2 slots, 4 row quarters), 256 threads: 32 rows per block,
// thread = (row, 16-dim group).
template <bool kEvenG, bool kSoft>
__global__ void __launch_bounds__(256) prefill_merge_kernel(PrefillArgs a) {
  using namespace tc5x2h;
  pdl_chain_link();
  const CacheView &c = a.c;
  const int walk = blockIdx.x, h = blockIdx.y, row0 = blockIdx.z * 32;
  const WalkSlots ws = walk_slots<kEvenG>(a, walk);
  if (h == 1 && !ws.two) return;
  int n_ptiles, sp_lo;
  const int S = walk_shares<kSoft>(a, walk_pages<kSoft>(a, ws, &n_ptiles, &sp_lo));
  if (S == 1) return;   // the walk stayed whole and wrote its output itself
  const int hq = h ? ws.hq1 : ws.hq0, i0 = h ? ws.i01 : ws.i00;
  if (i0 + row0 >= a.C) return;
  float v_scale, v_unscale;
  const bool wide = value_scale((uint32_t)unit_ws(a, ws.kvh)[H_VMAX], a.force_wide, v_scale, v_unscale);
  const float *part = a.partials + (size_t)(walk * 2 + h) * a.n_split * kPartFloats;
  __shared__ float s_w[kMaxSplit][32];   // weight of share s for a row, already divided by the row sum
  if (threadIdx.x < 32) {
    const int row = row0 + threadIdx.x;
    float ms[kMaxSplit], M = -INFINITY;
#pragma unroll
    for (int s = 0; s < kMaxSplit; ++s) {
      ms[s] = s < S ? part[(size_t)s * kPartFloats + 128 * 128 + row * 2] : -INFINITY;
      M = fmaxf(M, ms[s]);
    }
    float L = 0.f, wg[kMaxSplit];
#pragma unroll
    for (int s = 0; s < kMaxSplit; ++s) {
      wg[s] = ms[s] == -INFINITY ? 0.f : exp2f(ms[s] - M);
      if (s < S) L += wg[s] * part[(size_t)s * kPartFloats + 128 * 128 + row * 2 + 1];
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int s = 0; s < kMaxSplit; ++s) s_w[s][threadIdx.x] = wg[s] * inv;
    if (a.lse && i0 + row < a.C)   // the shares' l carry the same bias of P as the unsplit kernel's
      a.lse[(size_t)(i0 + row) * c.Hq + hq] = (M - (wide ? 0.f : kPBias) + log2f(L)) * 0.6931471805599453f;
  }
  __syncthreads();
  const int r = threadIdx.x >> 3, g = threadIdx.x & 7, row = row0 + r, i = i0 + row;
  if (i >= a.C) return;
  float acc[16];
#pragma unroll
  for (int d = 0; d < 16; ++d) acc[d] = 0.f;
  for (int s = 0; s < S; ++s) {
    const float wgt = s_w[s][r];
    const float4 *src = reinterpret_cast<const float4 *>(part + (size_t)s * kPartFloats + row * 128 + g * 16);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 v = src[q];
      acc[4 * q] += wgt * v.x; acc[4 * q + 1] += wgt * v.y; acc[4 * q + 2] += wgt * v.z; acc[4 * q + 3] += wgt * v.w;
    }
  }
  uint4 w0, w1;
  w0.x = pack_bf16(acc[0] * v_unscale, acc[1] * v_unscale);   w0.y = pack_bf16(acc[2] * v_unscale, acc[3] * v_unscale);
  w0.z = pack_bf16(acc[4] * v_unscale, acc[5] * v_unscale);   w0.w = pack_bf16(acc[6] * v_unscale, acc[7] * v_unscale);
  w1.x = pack_bf16(acc[8] * v_unscale, acc[9] * v_unscale);   w1.y = pack_bf16(acc[10] * v_unscale, acc[11] * v_unscale);
  w1.z = pack_bf16(acc[12] * v_unscale, acc[13] * v_unscale); w1.w = pack_bf16(acc[14] * v_unscale, acc[15] * v_unscale);
  __nv_bfloat16 *orow = a.out + ((size_t)i * c.Hq + hq) * kD + g * 16;
  *reinterpret_cast<uint4 *>(orow) = w0;
  *reinterpret_cast<uint4 *>(orow + 8) = w1;
}

// Number of blocks that share a page walk.  A chunk of a few hundred tokens has only a handful of
// walks (tiles x KV heads x head pairs) however long the context is; cutting each walk into
// shares, as the decode kernel cuts a unit into page ranges, puts the other SMs to work.
// Measured on a 32 k past, 32 query / 8 KV heads (TFLOP/s useful, whole call): with fewer walks
// than SMs two waves of shares are best; a launch of one to two and a half waves of whole walks
// is as slow as its longest walk (the heaviest head: ~0.5 ms) and gains from about six waves of
// shares (chunk 1536: 460 -> 670, 2048: 600 -> 730); from there on whole walks win.
int prefill_split_count(int n_walks, int sms) {
  if (2 * n_walks >= 5 * sms) return 1;
  const int target = n_walks < sms ? 2 * sms : 6 * sms;
  return std::min(tc5x2h::kMaxSplit, (target + n_walks - 1) / n_walks);
}
// partial results the workspace holds: walks (one query tile per single head) x shares, for a GPU
// of up to 192 SMs; the launcher never uses more (fewer walks or fewer SMs mean fewer blocks)
static long long split_slots(int C, int G, int Hkv) {
  const int n_xtiles = (C + 127) / 128;
  const int n_walks = ((G / 2) * n_xtiles + (G & 1) * n_xtiles) * Hkv;
  const int S = prefill_split_count(n_walks, 192);
  return S > 1 ? (long long)n_walks * S : 0;
}
size_t prefill_split_bytes(const spkv_config_t *cfg, int C) {
  return (size_t)split_slots(C, cfg->n_q_heads / cfg->n_kv_heads, cfg->n_kv_heads) * 2 * tc5x2h::kPartFloats * 4;
}

int launch_prefill_attn_tc5x2h(const PrefillArgs &a_in, cudaStream_t s) {
  PrefillArgs a = a_in;
  auto kernel = a.soft ? ((a.c.G & 1) ? prefill_attn_tc5x2h_kernel<false, true> : prefill_attn_tc5x2h_kernel<true, true>)
                       : ((a.c.G & 1) ? prefill_attn_tc5x2h_kernel<false, false> : prefill_attn_tc5x2h_kernel<true, false>);
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc5x2h::kSmemBytes) != cudaSuccess)
    return SPKV_E_CUDA;
  const int n_xtiles = (a.C + 127) / 128;
  // A single head's blocks take two query tiles each (the page walk then feeds 256 rows, as with
  // a head pair) when that still leaves two waves of blocks; a small launch keeps one tile per
  // block, whose finer grain balances better over the SMs.
  static const int sms = [] {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n;
  }();
  a.pair_tiles = ((a.c.G / 2) * n_xtiles + (a.c.G & 1) * ((n_xtiles + 1) / 2)) * a.c.Hkv >= 2 * sms;
  const int per_kvh = (a.c.G / 2) * n_xtiles + (a.c.G & 1) * (a.pair_tiles ? (n_xtiles + 1) / 2 : n_xtiles);
  const int n_walks = per_kvh * a.c.Hkv;
  a.n_split = a.partials ? prefill_split_count(n_walks, std::min(sms, 192)) : 1;
  a.n_split = (int)std::max(1LL, std::min<long long>(a.n_split, split_slots(a.C, a.c.G, a.c.Hkv) / n_walks));
  a.walks_per_kvh = per_kvh;
  a.split_unit = n_walks < sms ? 0.f : (float)sms;
  if (launch_link(a.chained != 0, kernel, dim3(n_walks * a.n_split), dim3(tc5x2h::kThreads), (size_t)tc5x2h::kSmemBytes, s,
                  a) != cudaSuccess)
    return SPKV_E_CUDA;
  if (a.n_split > 1) {
    auto merge = a.soft ? ((a.c.G & 1) ? prefill_merge_kernel<false, true> : prefill_merge_kernel<true, true>)
                        : ((a.c.G & 1) ? prefill_merge_kernel<false, false> : prefill_merge_kernel<true, false>);
    if (launch_link(a.chained != 0, merge, dim3(n_walks, 2, 4), dim3(256), 0, s, a) != cudaSuccess) return SPKV_E_CUDA;
  }
  return check_stream_error(cudaGetLastError());
}

}  // namespace spkv
