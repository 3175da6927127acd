// Two-layer utility predictor (Eq. 1 with f a 2-layer perceptron) on the tensor cores, for
// whole chunks of tokens at model width:
//
//   Z = X W1^T          [n_tok, hidden]   tcgen05.mma, bf16 x bf16 -> fp32 in tensor memory
//   A = SiLU(Z + b1)                      epilogue threads (thread = token = TMEM lane)
//   logit = A W2^T + b2 [n_tok, n_kv_heads], flag = logit >= tau_logit (Eq. 2)
//
// One block = 128 tokens x all hidden units (hidden <= 256 = one accumulator tile), or -- when
// the chunk has fewer token tiles than the GPU has SMs -- a cluster of two blocks that share the
// tokens and take half of the hidden units each (see the kernel).  X and W1
// are row-major with the contraction dimension innermost, i.e. K-major operands as they are: a
// TMA tile load (64 dims x rows, 128-byte swizzle) puts them in shared memory in operand layout.
// Rows past n_tok and dims past d_in are zero-filled by the TMA unit.  192 KB mbarrier
// pipeline (4 stages of 48 KB, or 6 of 32 KB): warp 4 = TMA producer, warp 5 = MMA issue (whole
// warp, one elected lane), warps 0-3 = epilogue.  Traffic: n_tok * d_in * 2 B of activations from HBM once; W1 (hidden * d_in * 2 B)
// is re-read per block from L2.  All waits are bounded.
#include <cuda.h>
#include <stdlib.h>

#include "spkv_internal.cuh"
#include "spkv_tc5.cuh"

namespace spkv {

namespace sctc {
constexpr int kThreads = 192;
constexpr int kTok = 128;      // tokens per block (MMA M)
constexpr int kKC = 64;        // dims per pipeline stage (one 128-byte swizzle row)
constexpr int kMaxHidden = 256;
constexpr int kABytes = kTok * kKC * 2;            // 16 KB
constexpr int kBBytesMax = kMaxHidden * kKC * 2;   // 32 KB (16 KB when the hidden units are split over two blocks)
constexpr int kPipeBytes = 4 * (kABytes + kBBytesMax);  // 192 KB: 4 stages of 48 KB, or 6 of 32 KB
constexpr int kMaxStages = 6;
constexpr int kMaxW2Floats = 4096;                 // hidden x (n_kv_heads rounded up to 8)
constexpr int kSW2 = kPipeBytes;                   // [hidden][heads8] fp32
constexpr int kSB1 = kSW2 + kMaxW2Floats * 4;      // [hidden] fp32
constexpr int kSPart = kSB1 + kMaxHidden * 4;      // split only: [2][128][heads8 <= 16] fp32 partial logits
constexpr int kSBar = kSPart + 2 * kTok * 16 * 4;
constexpr int kSmemBytes = kSBar + 128;
enum { B_FULL = 0, B_EMPTY = kMaxStages, B_ACC = 2 * kMaxStages, B_COUNT = 2 * kMaxStages + 1 };

__device__ inline void tma_load_2d(void *smem_dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ inline uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// float store into the same shared-memory location of another block of the cluster
__device__ inline void st_cluster_f32(const float *local_addr, uint32_t rank, float v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local_addr)), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}
__device__ inline void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
}  // namespace sctc

// kSplit = 1: one block computes all hidden units of its 128 tokens.  kSplit = 2: a cluster of two
// blocks shares the tokens, each takes half of the hidden units (its own half of W1, the same X
// tile -- the second read comes from L2), and block 1 hands its partial logits to block 0 through
// distributed shared memory.  Twice the blocks, two thirds of the bytes per block and six
// stages in flight instead of four: the kernel is bound by load latency x bytes in flight per
// SM and by the number of blocks (a chunk of 8192 tokens is only 64 token tiles on 148 SMs).
template <int kSplit>
__global__ void __launch_bounds__(sctc::kThreads, 1)
score_mlp_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w1, int n_tok,
                    int d_in, int hidden, const float *__restrict__ b1, const __nv_bfloat16 *__restrict__ W2,
                    const float *__restrict__ b2, int Hkv, float tau_logit, float *__restrict__ logits,
                    uint8_t *__restrict__ flags, int32_t *status) {
  using namespace tc5;
  using namespace sctc;
  constexpr int kStages = kSplit == 2 ? 6 : 4;
  constexpr int kStageBytes = kPipeBytes / kStages;
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t *bar = reinterpret_cast<uint64_t *>(smem + kSBar);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kSBar + B_COUNT * 8);
  float *w2s = reinterpret_cast<float *>(smem + kSW2), *b1s = reinterpret_cast<float *>(smem + kSB1);
  float *part = reinterpret_cast<float *>(smem + kSPart);  // [0]: this block's, [1]: the partner's partial logits
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = kSplit == 2 ? (int)cluster_rank() : 0;
  const int hl = hidden / kSplit, j_off = rank * hl;  // this block's hidden units
  const int tok0 = (blockIdx.x / kSplit) * kTok, n_kc = (d_in + kKC - 1) / kKC, heads8 = (Hkv + 7) & ~7;

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&bar[B_FULL + i], 1);
      mbar_init(&bar[B_EMPTY + i], 1);
    }
    mbar_init(&bar[B_ACC], 1);
    mbar_fence_init();
  }
  // second layer, transposed and padded: w2s[j][h] (zero for h >= Hkv), and the first bias
  for (int x = tid; x < hl * heads8; x += kThreads) {
    const int j = x / heads8, h = x % heads8;
    w2s[x] = h < Hkv ? __bfloat162float(W2[(size_t)h * hidden + j_off + j]) : 0.f;
  }
  for (int x = tid; x < hl; x += kThreads) b1s[x] = b1[j_off + x];
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tbase = *tmem_slot;
  bool failed = false;

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      const uint32_t stage_tx = kABytes + (uint32_t)hl * kKC * 2;
      int kc = 0;
      for (; kc < n_kc; ++kc) {
        const int s = kc % kStages;
        if (kc >= kStages && !mbar_wait_bounded(&bar[B_EMPTY + s], ((kc / kStages) - 1) & 1)) { failed = true; break; }
        mbar_arrive_expect_tx(&bar[B_FULL + s], stage_tx);
        tma_load_2d(smem + s * kStageBytes, &map_x, kc * kKC, tok0, &bar[B_FULL + s]);
        tma_load_2d(smem + s * kStageBytes + kABytes, &map_w1, kc * kKC, j_off, &bar[B_FULL + s]);
      }
      if (failed)  // do not leave while copies may still be landing
        for (int k = max(0, kc - kStages); k < kc; ++k) mbar_wait_bounded(&bar[B_FULL + (k % kStages)], (k / kStages) & 1);
    }
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issue
    const uint32_t idesc = instr_desc(kTok, hl, false);
    for (int kc = 0; kc < n_kc && !failed; ++kc) {
      const int s = kc % kStages;
      if (!mbar_wait_bounded(&bar[B_FULL + s], (kc / kStages) & 1)) { failed = true; break; }
      fence_after();
      const uint32_t sA = smem_u32(smem + s * kStageBytes), sB = sA + kABytes;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
        umma(tbase, smem_desc(sA + kk * 32, 16, 1024), smem_desc(sB + kk * 32, 16, 1024), idesc, (kc > 0 || kk > 0) ? 1u : 0u);
      umma_commit(&bar[B_EMPTY + s]);
    }
    if (!failed) umma_commit(&bar[B_ACC]);
  } else {
    // ---------------------------------------------------------------- epilogue (thread = token)
    const int tok = tok0 + tid;
    const uint32_t t_lane = tbase + ((uint32_t)(warp * 32) << 16);
    if (mbar_wait_bounded(&bar[B_ACC], 0)) {
      fence_after();
      for (int h0 = 0; h0 < Hkv; h0 += 8) {
        float acc[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) acc[h] = 0.f;
        for (int j0 = 0; j0 < hl; j0 += 16) {
          float z[16];
          tmem_ld16(t_lane + j0, z);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            const float zz = z[x] + b1s[j0 + x];
            const float act = zz / (1.f + __expf(-zz));  // SiLU
            const float4 wa = *reinterpret_cast<const float4 *>(w2s + (size_t)(j0 + x) * heads8 + h0);
            const float4 wb = *reinterpret_cast<const float4 *>(w2s + (size_t)(j0 + x) * heads8 + h0 + 4);
            acc[0] = fmaf(wa.x, act, acc[0]); acc[1] = fmaf(wa.y, act, acc[1]);
            acc[2] = fmaf(wa.z, act, acc[2]); acc[3] = fmaf(wa.w, act, acc[3]);
            acc[4] = fmaf(wb.x, act, acc[4]); acc[5] = fmaf(wb.y, act, acc[5]);
            acc[6] = fmaf(wb.z, act, acc[6]); acc[7] = fmaf(wb.w, act, acc[7]);
          }
        }
        if (kSplit == 2) {
          // block 0 parks its half, block 1 sends its half to block 0; summed after the cluster barrier
#pragma unroll
          for (int h = 0; h < 8; ++h) {
            if (rank == 0) part[(size_t)tid * heads8 + h0 + h] = acc[h];
            else st_cluster_f32(part + (size_t)kTok * heads8 + (size_t)tid * heads8 + h0 + h, 0, acc[h]);
          }
        } else if (tok < n_tok) {
#pragma unroll
          for (int h = 0; h < 8; ++h)
            if (h0 + h < Hkv) {
              const float v = acc[h] + b2[h0 + h];
              logits[(size_t)tok * Hkv + h0 + h] = v;
              if (flags) flags[(size_t)tok * Hkv + h0 + h] = v >= tau_logit ? 1 : 0;
            }
        }
      }
    } else {
      failed = true;
    }
  }
  if (kSplit == 2) {
    cluster_sync_all();  // every thread of both blocks; block 1's stores are visible to block 0 after it
    if (rank == 0 && warp < 4) {
      const int tok = tok0 + tid;
      if (tok < n_tok)
        for (int h = 0; h < Hkv; ++h) {
          const float v = part[(size_t)tid * heads8 + h] + part[(size_t)kTok * heads8 + (size_t)tid * heads8 + h] + b2[h];
          logits[(size_t)tok * Hkv + h] = v;
          if (flags) flags[(size_t)tok * Hkv + h] = v >= tau_logit ? 1 : 0;
        }
    }
  }
  if (failed) atomicCAS(status, 0, SPKV_E_TIMEOUT);
  fence_before();
  __syncthreads();
  if (warp == 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tbase) : "memory");
}

}  // namespace spkv

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// the driver's tensor-map encoder, looked up through the runtime (the library does not link libcuda)
EncodeTiledFn encode_tiled() {
  static const EncodeTiledFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// row-major [rows, cols] bf16 matrix, tile = box_rows x 64 columns, 128-byte swizzle, zero fill outside
bool make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)spkv::sctc::kKC, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return encode_tiled()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace spkv {

// Returns SPKV_OK when the tensor-core kernel was launched, 1 when the shape is outside what it
// covers (the caller then uses the CUDA-core kernel), < 0 on error.
int launch_score_mlp_tc(spkv_cache *cache, const spkv_predictor_t *p, const void *d_x, int n_tok, float *d_logits,
                        uint8_t *d_flags, cudaStream_t s) {
  const int Hkv = cache->view.Hkv, heads8 = (Hkv + 7) & ~7;
  if (n_tok < 64 || p->hidden < 16 || p->hidden > sctc::kMaxHidden || (p->hidden & 15) ||
      p->hidden * heads8 > sctc::kMaxW2Floats || (p->d_in & 7) || ((uintptr_t)d_x & 15) || ((uintptr_t)p->d_W1 & 15) ||
      !encode_tiled())
    return 1;
  // two blocks per token tile when that gives more blocks than one wave would otherwise hold
  const int tiles = (n_tok + sctc::kTok - 1) / sctc::kTok;
  const bool split = (p->hidden % 32) == 0 && heads8 <= 16 && tiles < cache->sm_count;
  const int hl = split ? p->hidden / 2 : p->hidden;
  CUtensorMap map_x, map_w1;
  if (!make_map(&map_x, d_x, n_tok, p->d_in, sctc::kTok) || !make_map(&map_w1, p->d_W1, p->hidden, p->d_in, hl))
    return 1;
  auto kernel = split ? score_mlp_tc_kernel<2> : score_mlp_tc_kernel<1>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sctc::kSmemBytes) != cudaSuccess)
    return SPKV_E_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles * (split ? 2 : 1));
  cfg.blockDim = dim3(sctc::kThreads);
  cfg.dynamicSmemBytes = sctc::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = split ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kernel, map_x, map_w1, n_tok, (int)p->d_in, (int)p->hidden, p->d_b1,
                         static_cast<const __nv_bfloat16 *>(p->d_W2), p->d_b2, Hkv, cache->tau_logit, d_logits,
                         d_flags, cache->view.status) != cudaSuccess)
    return SPKV_E_CUDA;
  return check_stream_error(cudaGetLastError());
}

}  // namespace spkv
