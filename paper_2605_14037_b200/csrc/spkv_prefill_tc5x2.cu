// Chunk attention of spkv_prefill on tcgen05, two query heads per block, P.V in two bf16 terms.
// (The comparison kernel, SPKV_PREFILL_PV=bf16; the default is the fp16 P.V kernel in
// spkv_prefill_tc5x2h.cu, which does a third less tensor work per page.)
//
// One block = 128 consecutive queries of TWO query heads that share a KV head (GQA, Eq. 5:
// head j reads KV head j / G).  Both heads walk the same page list, so each 32 KB page is
// fetched once and feeds both.  Each head owns one "softmax group" of 128 threads (thread =
// query row = TMEM lane), two S buffers and one O accumulator in tensor memory.  The single MMA
// thread runs two pages ahead with Q.K^T, so a group finds the scores of its next page ready
// when it finishes the current one, and the issue-to-completion latency of the MMAs of one head
// hides under the softmax of both:
//
//   MMA warp, per page j  :  wait P0(j), P1(j) | PV0(j) PV1(j) | wait page j+2 | QK0(j+2) QK1(j+2)
//   group h               :  softmax_h(j) softmax_h(j+1) softmax_h(j+2) ...
//
// P = exp2(S - m) is split into hi + lo bf16 terms and written back into the tensor-memory
// columns S came from (two bf16 per 32-bit column); the P.V MMAs take it from there as their A
// operand, so P never touches shared memory.  tcgen05.mma instructions execute in issue order:
// QK(j+2) of a head cannot overwrite P(j) before PV(j) has read it.  O is rescaled only when a
// row's maximum grows by more than 2^8; a group that has to rescale first waits for PV(j-1).
//
// Tensor memory (512 columns): S/P buffer b of head h at [(2h+b) 64, +64); O of head h at
// [256 + 128 h, +128).  Shared memory: Q of both heads (64 KB) + 5 page stages.
// Warps: 0 MMA issue, 1 page loader + TMEM allocation, 2-3 idle, 4-7 group 0, 8-11 group 1
// (a warp reaches the TMEM lanes 32 (warp % 4) ...).  The MMA warp comes first because the
// warp schedulers favour lower-numbered warps when several are ready: as warp 9, behind two
// always-ready softmax warps on its scheduler, it got an issue slot every ~9 cycles and the
// tensor pipe starved.  All waits are bounded.
#include "spkv_prefill_common.cuh"
#include "spkv_tc5.cuh"

namespace spkv {

namespace tc5x2 {
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;
constexpr int kSQ = 0;                     // 2 x 32 KB: Q of head 0, head 1 (two slabs of 128 rows x 128 B each)
constexpr int kStages = 5;
constexpr int kSKV = 65536;                // kStages x 32 KB
constexpr int kSBar = kSKV + kStages * kPageBytes;
constexpr int kSmemBytes = kSBar + 256;
enum { B_KV_FULL = 0, B_KV_EMPTY = 8, B_S_FULL = 16 /* [2h+b] */, B_P_FULL = 20 /* [2h+b] */, B_O_DONE = 24 /* [2h+b] */, B_COUNT = 28 };
}  // namespace tc5x2

#ifdef SPKV_TC5_TRACE
__device__ long long g_tc5_trace[16][2048];
#define TC5_STAMP(cond, who, j) do { if ((cond) && (j) < 2048) g_tc5_trace[who][j] = clock64(); } while (0)
#else
#define TC5_STAMP(cond, who, j) do { } while (0)
#endif

__global__ void __launch_bounds__(tc5x2::kThreads, 1) prefill_attn_tc5x2_kernel(PrefillArgs a) {
  using namespace tc5;
  using namespace tc5x2;
  extern __shared__ __align__(1024) unsigned char smem[];
  const CacheView &c = a.c;
  uint64_t *bar = reinterpret_cast<uint64_t *>(smem + kSBar);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kSBar + B_COUNT * 8);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int kvh, pair, xtile;
  prefill_work_item(a, blockIdx.x, (a.C + 127) / 128, c.G >> 1, kvh, pair, xtile);
  const int hq0 = kvh * c.G + pair * 2, i0 = xtile * 128;
  const int32_t *hdr = unit_ws(a, kvh);
  const int32_t *E = hdr + kHdrInts;
  const int len0 = hdr[H_LEN0], n_old = hdr[H_NOLD], N = hdr[H_N];
  const int u = unit_index(c, a.layer, a.seq, kvh);
  // kept pairs visible to chunk query i: the first nvis(i) pairs of the compact cache
  auto nvis = [&](int i) { return len0 + E[min(max(i + n_old - c.w + 1, 0), N)]; };
  const int i_last = min(i0 + 127, a.C - 1);
  const int n_ptiles = (nvis(i_last) + kP - 1) / kP;
  // band, in staging indices (query i is staging pair n_old + i)
  const int sp_lo = max(0, i0 + n_old - c.w + 1) / kP, sp_hi = (i_last + n_old) / kP;
  const int n_tiles = n_ptiles + (sp_hi - sp_lo + 1);

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&bar[B_KV_FULL + i], 1);
      mbar_init(&bar[B_KV_EMPTY + i], 1);
    }
    // One barrier per head and page parity: a parity wait only tells adjacent phases apart, and
    // producer and waiter of S, P and O can be two pages apart (a group may finish page j+1
    // before the MMA thread has looked at P(j); PV(j-1) and PV(j) can both be in flight).
    // Per parity they are at most one phase apart: S_FULL(j) completes after every MMA issued
    // before it, PV(j-2) included.  O_DONE is committed for the last two pages only (one use
    // per barrier).
    for (int i = 0; i < 4; ++i) {
      mbar_init(&bar[B_S_FULL + i], 1);
      mbar_init(&bar[B_P_FULL + i], 128);
      mbar_init(&bar[B_O_DONE + i], 1);
    }
    mbar_fence_init();
  }
  // Q tiles -> per head two slabs of 128 rows x 128 B, 128-byte swizzle (rows past the chunk are zero)
  for (int x = tid; x < 2 * 128 * 16; x += kThreads) {
    const int h = x >> 11, r = (x >> 4) & 127, ch = x & 15;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (i0 + r < a.C) val = *reinterpret_cast<const uint4 *>(a.q + ((size_t)(i0 + r) * c.Hq + hq0 + h) * kD + ch * 8);
    *reinterpret_cast<uint4 *>(smem + kSQ + h * 32768 + (ch >> 3) * 16384 + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = val;
  }
  fence_async_smem();
  if (warp == 1) {
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

  if (warp == 1) {
    // ---------------------------------------------------------------- page loader
    int j = 0;
    for (int base = 0; base < n_tiles && !failed; base += 32) {
      const int jl = base + lane;
      int64_t src_off = 0;
      if (jl < n_ptiles) src_off = (int64_t)c.table[(size_t)u * c.max_pages + jl] * kPageElems;
      const int cnt = min(32, n_tiles - base);
      for (int x = 0; x < cnt; ++x, ++j) {
        const int64_t off = __shfl_sync(0xffffffffu, src_off, x);
        if (lane == 0) {
          const int s = j % kStages;
          if (j >= kStages && !mbar_wait_bounded(&bar[B_KV_EMPTY + s], ((j / kStages) - 1) & 1)) failed = true;
          if (!failed) {
            const __nv_bfloat16 *src =
                j < n_ptiles ? c.pages + off
                             : a.stage_pages + ((size_t)kvh * a.n_stage_pages + sp_lo + (j - n_ptiles)) * kPageElems;
            mbar_arrive_expect_tx(&bar[B_KV_FULL + s], kPageBytes);
            bulk_load(smem + kSKV + s * kPageBytes, src, kPageBytes, &bar[B_KV_FULL + s]);
          }
        }
        failed = __shfl_sync(0xffffffffu, (int)failed, 0) != 0;
        if (failed) break;
      }
    }
    if (failed && lane == 0)  // do not leave while copies may still be landing
      for (int k = max(0, j - kStages); k < j; ++k)
        mbar_wait_bounded(&bar[B_KV_FULL + (k % kStages)], (k / kStages) & 1);
  } else if (warp == 0) {
    // ---------------------------------------------------------------- MMA issue (whole warp, one elected lane issues)
    {
      constexpr uint32_t idesc_qk = instr_desc(128, 64, false), idesc_pv = instr_desc(128, 128, true);
      const uint32_t sQ = smem_u32(smem + kSQ);
      auto issue_qk = [&](int h, int jj) {  // S_h[jj & 1] = Q_h . K(jj)^T
        const uint32_t sK = smem_u32(smem + kSKV + (jj % kStages) * kPageBytes);
        umma_qk_page<16384 / 16, 8192 / 16>(tbase + (2 * h + (jj & 1)) * 64, smem_desc(sQ + h * 32768, 16, 1024),
                                            smem_desc(sK, 16, 1024), idesc_qk);
      };
      auto commit_s = [&](int jj) {  // both heads' scores of page jj (each also covers the P.V before it)
        umma_commit(&bar[B_S_FULL + 0 + (jj & 1)]);
        umma_commit(&bar[B_S_FULL + 2 + (jj & 1)]);
      };
      // O_h += P_h(jj) . V(jj): A from tensor memory (hi in columns [0,32) of the S buffer the
      // scores came from, lo in [32,64)), B = the page's value block, MN-major
      auto wait_p = [&](int h, int jj) {
        if (!mbar_wait_bounded(&bar[B_P_FULL + 2 * h + (jj & 1)], (jj >> 1) & 1)) failed = true;
        TC5_STAMP(traced && lane == 0, 8 + h, jj);
        fence_after();
      };
      auto issue_pv = [&](int h, int jj) {
        const uint32_t sV = smem_u32(smem + kSKV + (jj % kStages) * kPageBytes) + kBlockElems * 2;
        const uint32_t tP = tbase + (2 * h + (jj & 1)) * 64;
        umma_pv_page(tbase + 256 + h * 128, tP, smem_desc(sV, 8192, 1024), idesc_pv, jj > 0 ? 1u : 0u);
        // the last two PVs have no later QK whose S_FULL would vouch for their completion
        if (jj + 2 >= n_tiles) umma_commit(&bar[B_O_DONE + 2 * h + (jj & 1)]);
        TC5_STAMP(traced && lane == 0, 11 + 2 * h, jj);
      };
      auto wait_page = [&](int jj) {
        if (!mbar_wait_bounded(&bar[B_KV_FULL + jj % kStages], (jj / kStages) & 1)) failed = true;
        TC5_STAMP(traced && lane == 0, 10, jj);
        fence_after();
      };
      for (int jj = 0; jj < 2 && jj < n_tiles && !failed; ++jj) {
        wait_page(jj);
        if (failed) break;
        issue_qk(0, jj);
        issue_qk(1, jj);
        commit_s(jj);
      }
      // Both heads' P.V of a page, then both heads' Q.K^T of the page after next: one cluster of
      // waits and commits per page instead of one per head and page (every wait or commit
      // between two runs of MMAs lets the tensor pipe run dry for a few dozen clocks).
      for (int j = 0; j < n_tiles && !failed; ++j) {
        wait_p(0, j);
        wait_p(1, j);
        if (failed) break;
        issue_pv(0, j);
        issue_pv(1, j);
        umma_commit(&bar[B_KV_EMPTY + (j % kStages)]);  // page j has no reader left
        if (j + 2 < n_tiles) {
          wait_page(j + 2);
          if (failed) break;
          issue_qk(0, j + 2);
          issue_qk(1, j + 2);
          commit_s(j + 2);
        }
      }
    }
  } else if (warp >= 4) {
    // ---------------------------------------------------------------- softmax groups
    const int h = (warp >> 2) - 1, row = tid & 127, i = i0 + row, hq = hq0 + h;
    const bool row_ok = i < a.C;
    const int nv = row_ok ? nvis(i) : 0;
    const int jq = n_old + i;  // staging index of this row's own pair
    const uint32_t t_lane = tbase + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t t_o = t_lane + 256 + h * 128;
    float m_ref = -INFINITY, l = 0.f;
    for (int j = 0; j < n_tiles; ++j) {
      const uint32_t t_s = t_lane + (2 * h + (j & 1)) * 64;
      if (!mbar_wait_bounded(&bar[B_S_FULL + 2 * h + (j & 1)], (j >> 1) & 1)) { failed = true; break; }
      TC5_STAMP(traced && row == 0, h * 4 + 0, j);
      fence_after();
      float v[64];
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        float t16[16];
        tmem_ld16(t_s + q4 * 16, t16);
#pragma unroll
        for (int x = 0; x < 16; ++x) v[q4 * 16 + x] = t16[x];
      }
      tmem_ld_wait();
      
      // visibility: compact-cache page j -> first nv pairs; staging page -> the band of this row.
      // v keeps the raw scores (masked ones become -inf); the scale is folded into the exponent,
      // and pages that every row of the warp sees in full skip the masking altogether.
      if (j < n_ptiles) {
        const int base = j * kP;
        if (!__all_sync(0xffffffffu, base + kP <= nv)) {
#pragma unroll
          for (int x = 0; x < 64; ++x) v[x] = (base + x < nv) ? v[x] : -INFINITY;
        }
      } else {
        const int base = (sp_lo + j - n_ptiles) * kP;
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
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * a.scale_log2;  // scale > 0 (host-checked)
      // the reference maximum moves only when the row maximum outgrows it by 2^8
      const bool grow = mx > m_ref + 8.f;
      const float m_new = grow ? mx : m_ref;
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
        // O is stable between the completion of PV(j-1) and the hand-over of P(j).  QK(j+1) was
        // issued right after PV(j-1), so S_FULL(j+1) vouches for it (waiting on it here does not
        // consume the phase); the last page has its own barrier.
        if (!(j + 1 < n_tiles ? mbar_wait_bounded(&bar[B_S_FULL + 2 * h + ((j + 1) & 1)], ((j + 1) >> 1) & 1)
                              : mbar_wait_bounded(&bar[B_O_DONE + 2 * h + ((j - 1) & 1)], 0))) {
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
      
      const float ms = m_ref == -INFINITY ? 0.f : m_ref;
      // two elements per instruction where the hardware has a packed form (fma, add, sub)
      const uint64_t sc2 = pack2(a.scale_log2, a.scale_log2), nms2 = pack2(-ms, -ms);
      uint64_t l2a = pack2(0.f, 0.f), l2b = l2a;
#pragma unroll
      for (int q2 = 0; q2 < 2; ++q2) {  // 32 keys -> 16 columns of hi, 16 of lo
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int x = 0; x < 16; ++x) {
          float e0, e1, r0, r1;
          unpack2(fma2(pack2(v[q2 * 32 + 2 * x], v[q2 * 32 + 2 * x + 1]), sc2, nms2), e0, e1);
          const float p0 = fast_exp2(e0), p1 = fast_exp2(e1);
          const uint64_t p2 = pack2(p0, p1);
          if (x & 1) l2b = add2(l2b, p2); else l2a = add2(l2a, p2);
          const __nv_bfloat162 hb = __floats2bfloat162_rn(p0, p1);
          hi[x] = *reinterpret_cast<const uint32_t *>(&hb);
          unpack2(sub2(p2, pack2(__uint_as_float(hi[x] << 16), __uint_as_float(hi[x] & 0xffff0000u))), r0, r1);
          lo[x] = pack_bf16(r0, r1);
        }
        tmem_st16u(t_s + q2 * 16, hi);
        tmem_st16u(t_s + 32 + q2 * 16, lo);
      }
      {
        float la, lb;
        unpack2(add2(l2a, l2b), la, lb);
        l += la + lb;
      }
      tmem_st_wait();
      fence_before();
      mbar_arrive(&bar[B_P_FULL + 2 * h + (j & 1)]);
      TC5_STAMP(traced && row == 0, h * 4 + 3, j);
      TC5_STAMP(traced && h == 0 && lane == 0 && warp > 4, warp - 4, j);  // rows 1-3: P arrival of warps 1-3 (trace only)
    }
    if (!failed && mbar_wait_bounded(&bar[B_O_DONE + 2 * h + ((n_tiles - 1) & 1)], 0)) {
      fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16 *orow = a.out + ((size_t)i * c.Hq + hq) * kD;
#pragma unroll
      for (int q8 = 0; q8 < 8; ++q8) {
        float t16[16];
        tmem_ld16(t_o + q8 * 16, t16);
        tmem_ld_wait();
        if (row_ok) {
          uint4 w0, w1;
          w0.x = pack_bf16(t16[0] * inv, t16[1] * inv);   w0.y = pack_bf16(t16[2] * inv, t16[3] * inv);
          w0.z = pack_bf16(t16[4] * inv, t16[5] * inv);   w0.w = pack_bf16(t16[6] * inv, t16[7] * inv);
          w1.x = pack_bf16(t16[8] * inv, t16[9] * inv);   w1.y = pack_bf16(t16[10] * inv, t16[11] * inv);
          w1.z = pack_bf16(t16[12] * inv, t16[13] * inv); w1.w = pack_bf16(t16[14] * inv, t16[15] * inv);
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
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "n"(tc5x2::kTmemCols) : "memory");
}

#ifdef SPKV_TC5_TRACE
extern "C" int spkv_debug_tc5_trace(long long *host_out) {
  return cudaMemcpyFromSymbol(host_out, g_tc5_trace, sizeof(g_tc5_trace)) == cudaSuccess ? 0 : -1;
}
#endif

int launch_prefill_attn_tc5x2(const PrefillArgs &a, cudaStream_t s) {
  if (cudaFuncSetAttribute(prefill_attn_tc5x2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           tc5x2::kSmemBytes) != cudaSuccess)
    return SPKV_E_CUDA;
  prefill_attn_tc5x2_kernel<<<dim3(((a.C + 127) / 128) * a.c.Hkv * (a.c.G / 2)), tc5x2::kThreads, tc5x2::kSmemBytes, s>>>(a);
  return check_stream_error(cudaGetLastError());
}

}  // namespace spkv
