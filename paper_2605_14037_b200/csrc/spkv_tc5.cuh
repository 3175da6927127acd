// tcgen05 / tensor-memory helpers shared by the prefill attention kernels.
#pragma once
#include "spkv_mma.cuh"

namespace spkv {
namespace tc5 {

__device__ inline uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // shared-memory matrix descriptor: start address, leading / stride byte offsets (in 16-byte
  // units), descriptor version 1, 128-byte swizzle
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// instruction descriptor, kind::f16: fp32 accumulate, A K-major, A and B both bf16 (format 1)
// or both fp16 (format 0)
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major, bool fp16 = false) {
  return (1u << 4) | ((fp16 ? 0u : 1u) << 7) | ((fp16 ? 0u : 1u) << 10) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// The MMA warp runs its loops with all 32 lanes (convergent control flow lets the compiler keep
// descriptors and addresses in uniform registers: issuing from inside an `if (lane == 0)` branch
// costs about 185 cycles per instruction, issuing this way 48-64, the rate of the tensor pipe
// itself); one elected lane -- the same one every time -- executes each tcgen05 instruction.
__device__ inline void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ inline void umma_commit(uint64_t *bar) {
  asm volatile(
      "{\n .reg .pred e;\n elect.sync _|e, 0xffffffff;\n"
      " @e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}\n"
      ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 16 consecutive fp32 columns of this thread's TMEM lane
__device__ inline void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ inline void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ inline void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
      "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
      "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
      "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
      "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ inline void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D (TMEM) (+)= A (TMEM, bf16 pairs packed in 32-bit columns, lane = row) . B (smem descriptor)
__device__ inline void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// One page of scores: D (128 x 64) = Q (128 x 128) . K^T, eight K=16 steps in one asm block with a
// single election.  adesc/bdesc are the descriptors of k-step 0; a step advances both by 32 bytes
// (2 descriptor units) inside a 64-dim slab, the second slab starts a_slab / b_slab units later.
template <int kASlabUnits, int kBSlabUnits>
__device__ inline void umma_qk_page(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  asm volatile(
      "{\n .reg .pred e;\n .reg .b64 a1, a2, a3, a4, a5, a6, a7, b1, b2, b3, b4, b5, b6, b7;\n"
      " elect.sync _|e, 0xffffffff;\n"
      " add.u64 a1, %1, 2; add.u64 a2, %1, 4; add.u64 a3, %1, 6;\n"
      " add.u64 a4, %1, %4; add.u64 a5, a4, 2; add.u64 a6, a4, 4; add.u64 a7, a4, 6;\n"
      " add.u64 b1, %2, 2; add.u64 b2, %2, 4; add.u64 b3, %2, 6;\n"
      " add.u64 b4, %2, %5; add.u64 b5, b4, 2; add.u64 b6, b4, 4; add.u64 b7, b4, 6;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, 0;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a2, b2, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a3, b3, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a4, b4, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a5, b5, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a6, b6, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], a7, b7, %3, 1;\n}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "n"(kASlabUnits), "n"(kBSlabUnits) : "memory");
}
// One page of P.V: D (128 x 128) (+)= P_hi . V + P_lo . V with P in tensor memory (hi at a_tmem,
// lo 32 columns later, 8 columns per K=16 step) and V MN-major (a k-step = 16 value rows =
// 2048 bytes = 128 descriptor units).  `first` = 0 overwrites D with the first product.
__device__ inline void umma_pv_page(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t first) {
  asm volatile(
      "{\n .reg .pred e, p;\n .reg .b64 b1, b2, b3;\n .reg .b32 t1, t2, t3, t4, t5, t6, t7;\n"
      " elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n"
      " add.u64 b1, %2, 128; add.u64 b2, %2, 256; add.u64 b3, %2, 384;\n"
      " add.u32 t1, %1, 8; add.u32 t2, %1, 16; add.u32 t3, %1, 24; add.u32 t4, %1, 32;\n"
      " add.u32 t5, %1, 40; add.u32 t6, %1, 48; add.u32 t7, %1, 56;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t1], b1, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t2], b2, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t3], b3, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t4], %2, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t5], b1, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t6], b2, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t7], b3, %3, 1;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(first) : "memory");
}
// One page of P.V with a single fp16 P (64 keys = 32 columns at a_tmem): four K=16 steps.
__device__ inline void umma_pv_page_f16(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                        uint32_t first) {
  asm volatile(
      "{\n .reg .pred e, p;\n .reg .b64 b1, b2, b3;\n .reg .b32 t1, t2, t3;\n"
      " elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n"
      " add.u64 b1, %2, 128; add.u64 b2, %2, 256; add.u64 b3, %2, 384;\n"
      " add.u32 t1, %1, 8; add.u32 t2, %1, 16; add.u32 t3, %1, 24;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t1], b1, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t2], b2, %3, 1;\n"
      " @e tcgen05.mma.cta_group::1.kind::f16 [%0], [t3], b3, %3, 1;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(first) : "memory");
}
// two bf16 (one 32-bit word) -> two fp16, each multiplied by `scale` first (a power of two)
__device__ inline uint32_t bf16x2_to_f16x2(uint32_t x, float scale) {
  uint32_t d;
  const float lo = __uint_as_float(x << 16) * scale, hi = __uint_as_float(x & 0xffff0000u) * scale;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ inline uint32_t pack_f16(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// ---- packed fp32 pairs (two lanes per instruction on sm_100) and the three-input maximum
__device__ inline uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ inline void unpack2(uint64_t r, float &a, float &b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r)); }
__device__ inline uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ inline uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ inline uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ inline float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ inline void tmem_st16u(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

}  // namespace tc5
}  // namespace spkv
