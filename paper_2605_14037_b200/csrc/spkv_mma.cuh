// Warp-level building blocks of the attention kernels: bf16 tensor-core tiles
// (mma.sync m16n8k16, operands fetched with ldmatrix from swizzled shared memory),
// the online-softmax update, and the mbarrier / bulk-copy primitives of the page pipeline.
//
// Shared-memory image of a key or value block (identical to its image in HBM):
// 64 rows of 256 B, 16-byte chunk c of row r stored at chunk position c ^ (r & 7).
// Eight consecutive rows at a fixed logical chunk therefore hit eight different
// 16-byte bank groups: every ldmatrix phase is conflict-free.
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
  return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4));
}

// Loads the A fragments of a 16 x 128 query tile straight from global memory.
// row_ptr(r) returns the address of row r's 128 bf16 (or nullptr for a padding row).
template <class RowPtr>
__device__ inline void load_q_frags(uint32_t (&qf)[8][4], RowPtr row_ptr, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const __nv_bfloat16 *r0 = row_ptr(g), *r1 = row_ptr(g + 8);
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    const int c = kk * 16 + t * 2;
    qf[kk][0] = r0 ? *reinterpret_cast<const uint32_t *>(r0 + c) : 0u;
    qf[kk][1] = r1 ? *reinterpret_cast<const uint32_t *>(r1 + c) : 0u;
    qf[kk][2] = r0 ? *reinterpret_cast<const uint32_t *>(r0 + c + 8) : 0u;
    qf[kk][3] = r1 ? *reinterpret_cast<const uint32_t *>(r1 + c + 8) : 0u;
  }
}

// s[n][.] = Q (16 x 128) . K^T for keys tok0 + 8n .. tok0 + 8n + 7, n < NT/8.
template <int NT>
__device__ inline void qk_tile(float (&s)[NT / 8][4], const uint32_t (&qf)[8][4], uint32_t sK,
                               int tok0, int lane) {
#pragma unroll
  for (int n = 0; n < NT / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
  const int mi = lane >> 3, ri = lane & 7;
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
    for (int jp = 0; jp < NT / 16; ++jp) {
      uint32_t b[4];
      const int tok = tok0 + jp * 16 + (mi >> 1) * 8 + ri;
      ldsm_x4(b, sK + blk_off(tok, 2 * kk + (mi & 1)));
      mma_bf16_16816(s[2 * jp], qf[kk], b[0], b[1]);
      mma_bf16_16816(s[2 * jp + 1], qf[kk], b[2], b[3]);
    }
  }
}

// Online-softmax update with the NT keys of this tile, then O += P . V.
// visible(h, col): is key `col` (tile-local index tok0-based: col in [tok0, tok0+NT))
// visible to row (g + 8h)?  m/l/o are per-thread state for rows g and g+8; l is a
// per-thread partial sum (reduce over the 4 lanes of a quad at the end).
template <int NT, class Visible>
__device__ inline void softmax_pv_tile(float (&s)[NT / 8][4], Visible visible, float scale_log2,
                                       float (&m)[2], float (&l)[2], float (&o)[16][4], uint32_t sV,
                                       int tok0, int lane) {
  const int t = lane & 3;
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int n = 0; n < NT / 8; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int h = e >> 1;
      const int col = tok0 + n * 8 + t * 2 + (e & 1);
      const float v = visible(h, col) ? s[n][e] * scale_log2 : -INFINITY;
      s[n][e] = v;
      mx[h] = fmaxf(mx[h], v);
    }
  float ms[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
    const float mn = fmaxf(m[h], mx[h]);
    ms[h] = mn == -INFINITY ? 0.f : mn;  // a row that has seen no key yet
    const float corr = fast_exp2(m[h] - ms[h]);
    m[h] = mn;
    l[h] *= corr;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      o[n][2 * h] *= corr;
      o[n][2 * h + 1] *= corr;
    }
  }
#pragma unroll
  for (int n = 0; n < NT / 8; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float p = fast_exp2(s[n][e] - ms[e >> 1]);
      s[n][e] = p;
      l[e >> 1] += p;
    }
  // P is split into two bf16 terms, P = hi + lo (lo = P - bf16(P)), each multiplied into V:
  // the weights then carry ~16 mantissa bits, so that the result keeps float32-accumulation
  // accuracy even when large value terms cancel (a single bf16 P would err by 2^-9 sum p|v|).
  const int mi = lane >> 3, ri = lane & 7;
#pragma unroll
  for (int kk = 0; kk < NT / 16; ++kk) {
    uint32_t a[4], alo[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float p0 = s[2 * kk + (x >> 1)][(x & 1) * 2], p1 = s[2 * kk + (x >> 1)][(x & 1) * 2 + 1];
      const __nv_bfloat162 hi = __floats2bfloat162_rn(p0, p1);
      const float2 hf = __bfloat1622float2(hi);
      a[x] = *reinterpret_cast<const uint32_t *>(&hi);
      alo[x] = pack_bf16(p0 - hf.x, p1 - hf.y);
    }
    const int tok = tok0 + kk * 16 + (mi & 1) * 8 + ri;
#pragma unroll
    for (int jn = 0; jn < 8; ++jn) {
      uint32_t b[4];
      ldsm_x4_trans(b, sV + blk_off(tok, 2 * jn + (mi >> 1)));
      mma_bf16_16816(o[2 * jn], a, b[0], b[1]);
      mma_bf16_16816(o[2 * jn + 1], a, b[2], b[3]);
      mma_bf16_16816(o[2 * jn], alo, b[0], b[1]);
      mma_bf16_16816(o[2 * jn + 1], alo, b[2], b[3]);
    }
  }
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
// Bounded wait: gives up after ~2^31 clock cycles (about a second) and returns false.
__device__ inline bool mbar_wait_bounded(uint64_t *bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > (1LL << 31)) return false;
  }
  return true;
}
// 1-D bulk copy; src, dst 16-byte aligned, bytes a multiple of 16.
__device__ inline void bulk_load(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ---- cp.async (16-byte) for gathered tiles ---------------------------------------------
__device__ inline void cp_async16(uint32_t smem_dst, const void *gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ inline void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

}  // namespace spkv
