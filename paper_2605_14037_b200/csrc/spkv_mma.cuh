// Warp-level building blocks of the attention kernels: the bf16 tensor-core tiles of the decode
// kernel (mma.sync m16n8k16, operands fetched with ldmatrix from swizzled shared memory) with
// their online-softmax update, and the mbarrier / bulk-copy primitives of the page pipelines.
//
// Shared-memory image of a key or value block (identical to its image in HBM): two slabs
// (dims 0-63 | 64-127) of 64 rows x 128 B; 16-byte chunk c (0-7) of a slab row r is stored at
// chunk position c ^ (r & 7).  Eight consecutive rows at a fixed logical chunk therefore hit
// eight different 16-byte bank groups: every ldmatrix phase is conflict-free.
//
// Fragment conventions (g = lane >> 2, t = lane & 3), m16n8k16, A row-major, B col-major:
//   A: a0 (row g,   k 2t..2t+1)  a1 (row g+8, k 2t..2t+1)  a2 (row g, k 2t+8..)  a3 (row g+8, k 2t+8..)
//   B: b0 (k 2t..2t+1, n g)      b1 (k 2t+8.., n g)
//   C: c0,c1 (row g, n 2t..2t+1) c2,c3 (row g+8, n 2t..2t+1)
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace spkv {

__device__ inline uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ inline void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ inline void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ inline void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Byte offset of (row, logical 16-byte chunk) inside a swizzled key/value block.
__device__ inline uint32_t blk_off(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * 8192 + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// ---- "keys as rows" tiles for decode --------------------------------------------------------
// In decode the query side has only G <= 16 rows (the heads of one group), the key side 64 per
// page.  Putting the 16 keys of a warp on the M side and the heads on the N side (8 per tile)
// wastes nothing for G = 8 and half for G = 4, and needs 8 + 16 MMAs per warp and page instead
// of 16 + 32:
//   S^T (16 keys x 8 heads)  = K (16 x 128) . Q^T          A = K rows (ldmatrix), B = Q
//   O^T (128 dims x 8 heads) += V^T (128 x 16) . P^T        A = V (ldmatrix.trans), B = P^T
// P^T is obtained from the S^T accumulator layout with movmatrix (8x8 transpose in registers).
// Accumulator layout of a 16 x 8 tile (g = lane >> 2, t = lane & 3):
//   e=0: (row g, col 2t)  e=1: (row g, col 2t+1)  e=2: (row g+8, col 2t)  e=3: (row g+8, col 2t+1)

__device__ inline uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// B fragments of Q^T for head tile hn: qb[hn][kk][0..1].  q_row(h) -> address of head h's 128
// bf16 (shared or global memory) or nullptr for a padding head.
template <int NH, class RowPtr>
__device__ inline void load_q_frags_t(uint32_t (&qb)[NH][8][2], RowPtr q_row, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int hn = 0; hn < NH; ++hn) {
    const __nv_bfloat16 *r = q_row(hn * 8 + g);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      qb[hn][kk][0] = r ? *reinterpret_cast<const uint32_t *>(r + kk * 16 + t * 2) : 0u;
      qb[hn][kk][1] = r ? *reinterpret_cast<const uint32_t *>(r + kk * 16 + 8 + t * 2) : 0u;
    }
  }
}

// s[hn][.] = scores of keys tok0..tok0+15 (rows) against heads 8hn..8hn+7 (cols), unscaled.
// mma.sync results come back after a long pipeline, and a warp issues in order: a chain of MMAs
// on one accumulator stalls for that latency at every link.  The eight k-steps therefore go to
// four accumulators (chains of two) that are summed at the end.
template <int NH>
__device__ inline void qk_tile_t(float (&s)[NH][4], const uint32_t (&qb)[NH][8][2], uint32_t sK, int tok0,
                                 int lane) {
  float acc[4][NH][4];
#pragma unroll
  for (int c4 = 0; c4 < 4; ++c4)
#pragma unroll
    for (int hn = 0; hn < NH; ++hn)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[c4][hn][e] = 0.f;
  const int mi = lane >> 3, ri = lane & 7;
  const int row = tok0 + (mi & 1) * 8 + ri;
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    uint32_t a[4];
    ldsm_x4(a, sK + blk_off(row, 2 * kk + (mi >> 1)));
#pragma unroll
    for (int hn = 0; hn < NH; ++hn) mma_bf16_16816(acc[kk & 3][hn], a, qb[hn][kk][0], qb[hn][kk][1]);
  }
#pragma unroll
  for (int hn = 0; hn < NH; ++hn)
#pragma unroll
    for (int e = 0; e < 4; ++e)
      s[hn][e] = (acc[0][hn][e] + acc[1][hn][e]) + (acc[2][hn][e] + acc[3][hn][e]);
}

// Online softmax over the 16 keys of this warp + O^T += V^T P^T.  n_valid: keys tok0.. that are
// < n_valid (page-local index) are visible.  m, l: per head (2 per thread and head tile: heads
// 8hn+2t, 8hn+2t+1); l is a per-thread partial (reduce over lanes with equal t at the end).
// o[hn][mt][e]: dims 16mt + g + 8(e>>1), head 8hn + 2t + (e&1).
template <int NH>
__device__ inline void softmax_pv_tile_t(float (&s)[NH][4], int n_valid, float scale_log2, float (&m)[NH][2],
                                         float (&l)[NH][2], float (&o)[NH][8][4], uint32_t sV, int tok0,
                                         int lane) {
  const int g = lane >> 2;
  const bool vis0 = tok0 + g < n_valid, vis1 = tok0 + g + 8 < n_valid;
  uint32_t bhi[NH][2], blo[NH][2];
#pragma unroll
  for (int hn = 0; hn < NH; ++hn) {
    float v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = ((e >> 1) ? vis1 : vis0) ? s[hn][e] * scale_log2 : -INFINITY;
    float corr[2], ms[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float mx = fmaxf(v[j], v[j + 2]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      const float mn = fmaxf(m[hn][j], mx);
      ms[j] = mn == -INFINITY ? 0.f : mn;
      corr[j] = fast_exp2(m[hn][j] - ms[j]);
      m[hn][j] = mn;
      l[hn][j] *= corr[j];
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[hn][mt][e] *= corr[e & 1];
    float p[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      p[e] = fast_exp2(v[e] - ms[e & 1]);
      l[hn][e & 1] += p[e];
    }
    // P is split into two bf16 terms, P = hi + lo (lo = P - bf16(P)), each multiplied into V: the
    // weights then carry ~16 mantissa bits, so that the result keeps float32-accumulation accuracy
    // even when large value terms cancel (a single bf16 P would err by 2^-9 sum p|v|).
    // Transposed into B-fragment layout.
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(p[0], p[1]), h1 = __floats2bfloat162_rn(p[2], p[3]);
    const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
    bhi[hn][0] = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&h0));
    bhi[hn][1] = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&h1));
    blo[hn][0] = movmatrix_trans(pack_bf16(p[0] - f0.x, p[1] - f0.y));
    blo[hn][1] = movmatrix_trans(pack_bf16(p[2] - f1.x, p[3] - f1.y));
  }
  // all "hi" products first, then all "lo" products: no MMA waits for its predecessor
  const int mi = lane >> 3, ri = lane & 7;
  const int row = tok0 + (mi >> 1) * 8 + ri;
  uint32_t a[8][4];
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    ldsm_x4_trans(a[mt], sV + blk_off(row, 2 * mt + (mi & 1)));
#pragma unroll
    for (int hn = 0; hn < NH; ++hn) mma_bf16_16816(o[hn][mt], a[mt], bhi[hn][0], bhi[hn][1]);
  }
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int hn = 0; hn < NH; ++hn) mma_bf16_16816(o[hn][mt], a[mt], blo[hn][0], blo[hn][1]);
}

// ---- mbarrier + bulk copy (global -> shared, completion counted in bytes) -------------

__device__ inline void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ inline void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ inline bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` clock cycles (default ~2^31, about a second) and returns false.
constexpr long long kWaitClocks = 1LL << 31;
__device__ inline bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, long long limit = kWaitClocks) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) return false;
  }
  return true;
}
// Counts `bytes` as arrived on the barrier's current phase without any copy (used to close a
// phase that was armed for more bytes than were ever sent).
__device__ inline void mbar_complete_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// 1-D bulk copy; src, dst 16-byte aligned, bytes a multiple of 16.
__device__ inline void bulk_load(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// The same copy with an L2 eviction hint for data that is read once: the lines go first when L2
// needs room, so what is read again every step (lengths, page tables, ring metadata) stays.
__device__ inline uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ inline void bulk_load_hint(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar,
                                      uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}

}  // namespace spkv
