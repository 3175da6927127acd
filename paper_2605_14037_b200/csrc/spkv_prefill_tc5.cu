// Chunk attention of spkv_prefill on the 5th-generation tensor cores (tcgen05.mma, TMEM): the
// one-head kernel, the first tcgen05 version, kept for comparison (SPKV_PREFILL_KERNEL=tc5x1; the
// default is the two-head fp16 kernel in spkv_prefill_tc5x2h.cu), and the staging kernel that
// every tcgen05 attention kernel runs behind.
//
// One block = 128 consecutive queries of one query head.  Keys/values arrive as 64-pair pages
// -- first the compact-cache pages that hold the kept pairs visible to the tile (a prefix of the
// cache, see spkv_prefill.cu), then the "staging" pages that hold the old ring pairs and the
// chunk's own pairs in position order (the dense band t-w < s <= t).  Every page, cached or
// staged, is the same 32 KB image, so one cp.async.bulk brings it in and its slabs are valid
// tcgen05.mma operands as they are: keys K-major, values MN-major, 128-byte swizzle.
//
// Per page:  S (128 x 64, fp32, TMEM)  = Q (128 x 128, smem) . K^T        8 MMAs  M128 N64  K16
//            softmax threads (one per query row): tcgen05.ld their row of S, mask, running
//            max / sum, P = exp2(S - m) split into two bf16 terms (hi + lo), written to
//            shared memory in operand layout
//            O (128 x 128, fp32, TMEM) += P_hi . V + P_lo . V             8 MMAs  M128 N128 K16
// S is double-buffered in TMEM, so Q.K^T of the next page runs under the softmax of this one.
// O is rescaled only when a row's maximum grows by more than 2^8 (the final O / l is exact
// whatever reference maximum the row carries).
//
// Warps: 0-3 softmax/correction/epilogue (thread = query row = TMEM lane), 4 page loader (one
// lane) and TMEM allocation, 5 MMA issue (one elected lane).  All waits are bounded.
#include <stdlib.h>

#include "spkv_prefill_common.cuh"
#include "spkv_tc5.cuh"

namespace spkv {

namespace tc5 {

constexpr int kThreads = 192;
constexpr int kTmemCols = 256;  // S0 [0,64) S1 [64,128) O [128,256)
constexpr int kSQ = 0;                       // 32 KB: Q, two slabs of 128 rows x 128 B
constexpr int kStages = 4;                   // page stages in flight
constexpr int kSKV = 32768;                  // kStages x 32 KB
constexpr int kSP = kSKV + kStages * kPageBytes;  // 16 KB P_hi + 16 KB P_lo (128 rows x 128 B each)
constexpr int kSBar = kSP + 32768;           // barriers
constexpr int kSmemBytes = kSBar + 256;

enum { B_KV_FULL = 0, B_KV_EMPTY = 4, B_S_FULL = 8, B_S_FREE = 10, B_P_FULL = 12, B_O_DONE = 13, B_COUNT = 14 };

}  // namespace tc5

// ------------------------------------------------------------------ staging pages
// Old ring pairs and chunk pairs, in position order, rewritten as pages (workspace).
// grid (n_stage_pages, Hkv), 256 threads: 8 warps x 8 rows.
__global__ void __launch_bounds__(256) prefill_stage_kernel(PrefillArgs a) {
  const CacheView &c = a.c;
  const int kvh = blockIdx.y, sp = blockIdx.x;
  const int32_t *hdr = unit_ws(a, kvh);
  const int t0 = hdr[H_T0], n_old = hdr[H_NOLD], N = hdr[H_N];
  const int u = unit_index(c, a.layer, a.seq, kvh);
  __nv_bfloat16 *page = a.stage_pages + ((size_t)kvh * a.n_stage_pages + sp) * kPageElems;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = lane & 15, blk = (lane >> 4) * kBlockElems;
  uint32_t vm = 0;  // largest |v| among the chunk's values this lane moves (old ring pairs are accounted for already)
  for (int r = warp * 8; r < warp * 8 + 8; ++r) {
    const int j = sp * kP + r;
    uint4 val = make_uint4(0, 0, 0, 0);  // rows past the last pair read as zeros
    if (j < N) {
      if (j < n_old) {
        const int slot = (t0 - n_old + j) % c.w;
        const __nv_bfloat16 *pg = c.pages + ring_page(c, u, slot / kP) * kPageElems;
        val = *reinterpret_cast<const uint4 *>(pg + blk + swz_off(slot % kP, chunk));
      } else {
        const __nv_bfloat16 *src = (lane < 16 ? a.k : a.v) + ((size_t)(j - n_old) * c.Hkv + kvh) * kD;
        val = *reinterpret_cast<const uint4 *>(src + chunk * 8);
        if (lane >= 16) vm = max(vm, chunk_abs_max_bf16(val));
      }
    }
    *reinterpret_cast<uint4 *>(page + blk + swz_off(r, chunk)) = val;
  }
  vm = __reduce_max_sync(0xffffffffu, vm);
  if (lane == 0 && vm) note_vmax(c, u, vm);
}

// ------------------------------------------------------------------ chunk attention
__global__ void __launch_bounds__(tc5::kThreads, 1) prefill_attn_tc5_kernel(PrefillArgs a) {
  using namespace tc5;
  extern __shared__ __align__(1024) unsigned char smem[];
  const CacheView &c = a.c;
  uint64_t *bar = reinterpret_cast<uint64_t *>(smem + kSBar);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kSBar + B_COUNT * 8);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int kvh, sub, xtile;
  prefill_work_item(a, blockIdx.x, (a.C + 127) / 128, c.G, kvh, sub, xtile);
  const int hq = kvh * c.G + sub, i0 = xtile * 128;
  const int32_t *hdr = unit_ws(a, kvh);
  const int32_t *E = hdr + kHdrInts;
  const int len0 = hdr[H_LEN0], n_old = hdr[H_NOLD], N = hdr[H_N];
  const int u = unit_index(c, a.layer, a.seq, kvh);
  // kept pairs visible to chunk query i: the first nvis(i) pairs of the compact cache
  auto nvis = [&](int i) { return len0 + E[min(max(i + n_old - c.w + 1, 0), N)]; };
  const int i_last = min(i0 + 127, a.C - 1);
  const int n_ptiles = (nvis(i_last) + kP - 1) / kP;
  // band, in staging indices (pair j of the staging sequence has position p0 + j; query i is j = n_old + i)
  const int sp_lo = max(0, i0 + n_old - c.w + 1) / kP, sp_hi = (i_last + n_old) / kP;
  const int n_tiles = n_ptiles + (sp_hi - sp_lo + 1);

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&bar[B_KV_FULL + i], 1);
      mbar_init(&bar[B_KV_EMPTY + i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar[B_S_FULL + i], 1);
      mbar_init(&bar[B_S_FREE + i], 128);
    }
    mbar_init(&bar[B_P_FULL], 128);
    mbar_init(&bar[B_O_DONE], 1);
    mbar_fence_init();
  }
  // Q tile -> two slabs of 128 rows x 128 B, 128-byte swizzle (rows past the chunk are zero)
  for (int x = tid; x < 128 * 16; x += kThreads) {
    const int r = x >> 4, ch = x & 15;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (i0 + r < a.C) val = *reinterpret_cast<const uint4 *>(a.q + ((size_t)(i0 + r) * c.Hq + hq) * kD + ch * 8);
    *reinterpret_cast<uint4 *>(smem + kSQ + (ch >> 3) * 16384 + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = val;
  }
  fence_async_smem();
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "n"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tbase = *tmem_slot;
  bool failed = false;

  if (warp == 4) {
    // ---------------------------------------------------------------- page loader
    // the warp fetches 32 page-table entries at a time; lane 0 issues the copies
    int j = 0;
    for (int base = 0; base < n_tiles && !failed; base += 32) {
      const int jl = base + lane;
      int64_t src_off = 0;  // element offset from c.pages, or from the staging pages (negative tag)
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
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issue (whole warp, one elected lane issues)
    {
      constexpr uint32_t idesc_qk = instr_desc(128, 64, false), idesc_pv = instr_desc(128, 128, true);
      const uint32_t sQ = smem_u32(smem + kSQ), sP = smem_u32(smem + kSP);
      auto issue_pv = [&](int jj) {
        if (!mbar_wait_bounded(&bar[B_P_FULL], jj & 1)) { failed = true; return; }
        fence_after();
        const uint32_t sV = smem_u32(smem + kSKV + (jj % kStages) * kPageBytes) + kBlockElems * 2;
#pragma unroll
        for (int part = 0; part < 2; ++part)  // P_hi, then P_lo
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma(tbase + 128, smem_desc(sP + part * 16384 + kk * 32, 16, 1024),
                 smem_desc(sV + kk * 2048, 8192, 1024), idesc_pv, (jj > 0 || part > 0 || kk > 0) ? 1u : 0u);
        umma_commit(&bar[B_KV_EMPTY + (jj % kStages)]);
        umma_commit(&bar[B_O_DONE]);
      };
      for (int j = 0; j < n_tiles && !failed; ++j) {
        const int s = j & 1, ks = j % kStages;
        if (!mbar_wait_bounded(&bar[B_KV_FULL + ks], (j / kStages) & 1)) { failed = true; break; }
        if (j >= 2 && !mbar_wait_bounded(&bar[B_S_FREE + s], ((j >> 1) - 1) & 1)) { failed = true; break; }
        fence_after();
        const uint32_t sK = smem_u32(smem + kSKV + ks * kPageBytes);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma(tbase + s * 64, smem_desc(sQ + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024),
               smem_desc(sK + (kk >> 2) * 8192 + (kk & 3) * 32, 16, 1024), idesc_qk, kk > 0 ? 1u : 0u);
        umma_commit(&bar[B_S_FULL + s]);
        if (j >= 1) issue_pv(j - 1);
      }
      if (!failed) issue_pv(n_tiles - 1);
    }
  } else {
    // ---------------------------------------------------------------- softmax threads
    const int row = tid, i = i0 + row;
    const bool row_ok = i < a.C;
    const int nv = row_ok ? nvis(i) : 0;
    const int jq = n_old + i;  // staging index of this row's own pair
    const uint32_t t_lane = tbase + ((uint32_t)(warp * 32) << 16);
    float m_ref = -INFINITY, l = 0.f;
    for (int j = 0; j < n_tiles; ++j) {
      const int s = j & 1;
      if (!mbar_wait_bounded(&bar[B_S_FULL + s], (j >> 1) & 1)) { failed = true; break; }
      fence_after();
      float v[64];
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        float t16[16];
        tmem_ld16(t_lane + s * 64 + q4 * 16, t16);
#pragma unroll
        for (int x = 0; x < 16; ++x) v[q4 * 16 + x] = t16[x];
      }
      tmem_ld_wait();
      fence_before();
      mbar_arrive(&bar[B_S_FREE + s]);
      // visibility: compact-cache page j -> first nv pairs; staging page -> the band of this row.
      // v keeps the raw scores (masked ones become -inf); the scale is folded into the exponent
      // below, and pages that every row of the warp sees in full skip the masking altogether.
      float mx = -INFINITY;
      if (j < n_ptiles) {
        const int base = j * kP;
        const bool all_visible = __all_sync(0xffffffffu, base + kP <= nv);
        if (!all_visible) {
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
#pragma unroll
      for (int x = 0; x < 64; ++x) mx = fmaxf(mx, v[x]);
      mx *= a.scale_log2;  // scale > 0 (checked on the host): the maximum commutes with it
      // the reference maximum moves only when the row maximum outgrows it by 2^8
      const bool grow = mx > m_ref + 8.f;
      const float m_new = grow ? mx : m_ref;
      if (j > 0) {
        if (!mbar_wait_bounded(&bar[B_O_DONE], (j - 1) & 1)) { failed = true; break; }
        fence_after();
        if (__any_sync(0xffffffffu, grow)) {
          const float f = grow ? fast_exp2(m_ref - m_new) : 1.f;  // m_ref = -inf -> 0
#pragma unroll
          for (int q8 = 0; q8 < 8; ++q8) {
            float t16[16];
            tmem_ld16(t_lane + 128 + q8 * 16, t16);
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 16; ++x) t16[x] *= f;
            tmem_st16(t_lane + 128 + q8 * 16, t16);
          }
          tmem_st_wait();
          l *= f;
        }
      }
      m_ref = m_new;
      const float ms = m_ref == -INFINITY ? 0.f : m_ref;
      unsigned char *p_hi = smem + kSP + row * 128, *p_lo = p_hi + 16384;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float p0 = fast_exp2(fmaf(v[ch * 8 + 2 * x], a.scale_log2, -ms));
          const float p1 = fast_exp2(fmaf(v[ch * 8 + 2 * x + 1], a.scale_log2, -ms));
          l += p0 + p1;
          const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
          const float2 hf = __bfloat1622float2(h);
          hi[x] = *reinterpret_cast<const uint32_t *>(&h);
          lo[x] = pack_bf16(p0 - hf.x, p1 - hf.y);
        }
        const int off = (ch ^ (row & 7)) << 4;
        *reinterpret_cast<uint4 *>(p_hi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4 *>(p_lo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
      fence_async_smem();
      fence_before();
      mbar_arrive(&bar[B_P_FULL]);
    }
    if (!failed && mbar_wait_bounded(&bar[B_O_DONE], (n_tiles - 1) & 1)) {
      fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16 *orow = a.out + ((size_t)i * c.Hq + hq) * kD;
#pragma unroll
      for (int q8 = 0; q8 < 8; ++q8) {
        float t16[16];
        tmem_ld16(t_lane + 128 + q8 * 16, t16);
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
  if (warp == 4)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "n"(tc5::kTmemCols) : "memory");
}

int launch_prefill_attn_tc5(const PrefillArgs &a, cudaStream_t s) {
  if (cudaFuncSetAttribute(prefill_attn_tc5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           tc5::kSmemBytes) != cudaSuccess)
    return SPKV_E_CUDA;
  static const bool one_head = [] {
    const char *e = getenv("SPKV_PREFILL_KERNEL");  // "tc5x1": one query head per block
    return e && e[0] == 't' && e[1] == 'c' && e[2] == '5' && e[3] == 'x' && e[4] == '1';
  }();
  static const bool bf16_pv = [] {
    const char *e = getenv("SPKV_PREFILL_PV");  // "bf16": the two-term bf16 P.V kernel (comparison)
    return e && e[0] == 'b';
  }();
  prefill_stage_kernel<<<dim3(a.n_stage_pages, a.c.Hkv), 256, 0, s>>>(a);
  if (!one_head && !bf16_pv) return launch_prefill_attn_tc5x2h(a, s);   // any G: an odd group's last block has one head
  if (!one_head && a.c.G % 2 == 0) return launch_prefill_attn_tc5x2(a, s);
  prefill_attn_tc5_kernel<<<dim3(((a.C + 127) / 128) * a.c.Hq), tc5::kThreads, tc5::kSmemBytes, s>>>(a);
  return check_stream_error(cudaGetLastError());
}

}  // namespace spkv
