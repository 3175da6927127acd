// Decode attention, comparison kernel on the CUDA cores (warp-shuffle dot products, direct
// global loads).  Selected with SPKV_DECODE_KERNEL=simt; same results as the main kernel.
//
// Schedule: the NP pages of the call are cut into min(gridDim.x, NP) equal contiguous
// ranges, one per block; a (block, unit) intersection is a segment; partial results go to
// workspace slot (block + item) and the block that arrives last at a unit merges them.
#include "spkv_decode_common.cuh"

namespace spkv {

// First page of block c's range when NP pages are cut into n_blocks ranges.
__device__ inline int range_start(int c, int NP, int n_blocks) {
  return (int)(((long long)c * NP) / n_blocks);
}
// Block whose range contains page p.
__device__ inline int block_of_page(int p, int NP, int n_blocks) {
  return (int)((((long long)p + 1) * n_blocks - 1) / NP);
}

__device__ inline float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// 4 warps; warp w of a block takes pages j0+w, j0+w+4, ... of a segment; lane l owns dims
// 4l..4l+3 of every row.
template <int GP>
__global__ void __launch_bounds__(128) decode_simt_kernel(DecodeArgs a) {
  extern __shared__ int s_int[];
  const CacheView &c = a.c;
  const int n = a.n_items;
  int *s_np = s_int;                   // [n]
  int *s_pre = s_np + n;               // [n+1]
  int *s_tmp = s_pre + n + 1;          // [64]
  ItemInfo *s_item = reinterpret_cast<ItemInfo *>(s_tmp + 64);  // [n]
  float *s_red = reinterpret_cast<float *>(s_item + n);         // [4][GP][130]
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int i = tid; i < n; i += blockDim.x) {
    const int b = i / c.Hkv, kvh = i % c.Hkv;
    const int seq = a.seq_ids[b];
    ItemInfo it = {0, 0, 0, 0};
    if (seq >= 0 && seq < c.S) {
      it.unit = unit_index(c, a.layer, seq, kvh);
      it.len = c.len[it.unit];
      it.n_ring = min(c.t[it.unit], c.w);
      it.nk = (it.len + kP - 1) / kP;
    } else if (blockIdx.x == 0) {
      set_status(c, SPKV_E_BOUNDS);
    }
    const int np = it.nk + (it.n_ring + kP - 1) / kP;
    s_item[i] = it;
    s_np[i] = np;
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
  const int NP = s_pre[n];
  if (NP == 0) return;
  // with fewer pages than blocks only the first NP blocks work (every range non-empty,
  // so the segments of a unit sit in consecutive blocks)
  const int nb = min((int)gridDim.x, NP);
  if ((int)blockIdx.x >= nb) return;
  int p = range_start(blockIdx.x, NP, nb);
  const int p_end = range_start(blockIdx.x + 1, NP, nb);
  if (p >= p_end) return;

  // item containing page p: last i with s_pre[i] <= p
  int lo = 0, hi = n;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_pre[mid] <= p) lo = mid; else hi = mid;
  }
  int item = lo;

  while (p < p_end) {
    while (s_pre[item + 1] <= p) ++item;
    const ItemInfo it = s_item[item];
    const int j0 = p - s_pre[item];
    const int j1 = min(s_np[item], j0 + (p_end - p));
    const int b = item / c.Hkv, kvh = item % c.Hkv;

    // query fragment: this lane's 4 dims of every head of the group
    float q[GP][4];
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      if (g < a.G) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(
            a.q + ((size_t)b * c.Hq + kvh * a.G + g) * kD + lane * 4);
        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.x));
        const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.y));
        q[g][0] = x.x; q[g][1] = x.y; q[g][2] = y.x; q[g][3] = y.y;
      } else {
        q[g][0] = q[g][1] = q[g][2] = q[g][3] = 0.f;
      }
    }
    float m[GP], l[GP], acc[GP][4];
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      m[g] = -INFINITY; l[g] = 0.f;
      acc[g][0] = acc[g][1] = acc[g][2] = acc[g][3] = 0.f;
    }
    const int chunk = lane >> 1, sub = (lane & 1) * 4;
    for (int j = j0 + warp; j < j1; j += 4) {
      int64_t gpage;
      int valid;
      if (j < it.nk) {
        gpage = c.table[(size_t)it.unit * c.max_pages + j];
        valid = min(kP, it.len - j * kP);
      } else {
        gpage = ring_page(c, it.unit, j - it.nk);
        valid = min(kP, it.n_ring - (j - it.nk) * kP);
      }
      const __nv_bfloat16 *kb = c.pages + gpage * kPageElems;
      const __nv_bfloat16 *vb = kb + kBlockElems;
      for (int r = 0; r < valid; ++r) {
        const int off = swz_off(r, chunk) + sub;
        const uint2 kr = *reinterpret_cast<const uint2 *>(kb + off);
        const uint2 vr = *reinterpret_cast<const uint2 *>(vb + off);
        const float2 k0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&kr.x));
        const float2 k1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&kr.y));
        const float2 v0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&vr.x));
        const float2 v1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&vr.y));
#pragma unroll
        for (int g = 0; g < GP; ++g) {
          float s = q[g][0] * k0.x + q[g][1] * k0.y + q[g][2] * k1.x + q[g][3] * k1.y;
          s = warp_sum_f(s) * a.scale_log2;
          const float mn = fmaxf(m[g], s);
          const float corr = exp2f(m[g] - mn), pw = exp2f(s - mn);
          m[g] = mn;
          l[g] = l[g] * corr + pw;
          acc[g][0] = acc[g][0] * corr + pw * v0.x;
          acc[g][1] = acc[g][1] * corr + pw * v0.y;
          acc[g][2] = acc[g][2] * corr + pw * v1.x;
          acc[g][3] = acc[g][3] * corr + pw * v1.y;
        }
      }
    }
    // combine the 4 warps through shared memory
    __syncthreads();
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      float *dst = s_red + ((size_t)warp * GP + g) * 130;
      dst[lane * 4 + 0] = acc[g][0]; dst[lane * 4 + 1] = acc[g][1];
      dst[lane * 4 + 2] = acc[g][2]; dst[lane * 4 + 3] = acc[g][3];
      if (lane == 0) { dst[128] = m[g]; dst[129] = l[g]; }
    }
    __syncthreads();
    const int c_first = block_of_page(s_pre[item], NP, nb);
    const int c_last = block_of_page(s_pre[item + 1] - 1, NP, nb);
    const int nseg = c_last - c_first + 1;
    const int slot = blockIdx.x + item;
    // thread d owns output dim d
    float M[GP], Lsum[GP], O[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      M[g] = -INFINITY;
      for (int w4 = 0; w4 < 4; ++w4) M[g] = fmaxf(M[g], s_red[((size_t)w4 * GP + g) * 130 + 128]);
      Lsum[g] = 0.f; O[g] = 0.f;
      for (int w4 = 0; w4 < 4; ++w4) {
        const float *src = s_red + ((size_t)w4 * GP + g) * 130;
        const float f = src[128] == -INFINITY ? 0.f : exp2f(src[128] - M[g]);
        Lsum[g] += src[129] * f;
        O[g] += src[tid] * f;
      }
    }
    if (nseg > 1) {
#pragma unroll
      for (int g = 0; g < GP; ++g)
        if (g < a.G) {
          a.part_acc[((size_t)slot * a.G + g) * kD + tid] = O[g];
          if (tid == 0) {
            a.part_ml[((size_t)slot * a.G + g) * 2 + 0] = M[g];
            a.part_ml[((size_t)slot * a.G + g) * 2 + 1] = Lsum[g];
          }
        }
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        const int old = atomicAdd(&a.counters[item], 1);
        s_last = (old == nseg - 1);
        if (s_last) a.counters[item] = 0;
      }
      __syncthreads();
      if (s_last) {
        __threadfence();
#pragma unroll
        for (int g = 0; g < GP; ++g)
          if (g < a.G) {
            float Mx = -INFINITY;
            for (int sidx = c_first; sidx <= c_last; ++sidx)
              Mx = fmaxf(Mx, __ldcg(&a.part_ml[((size_t)(sidx + item) * a.G + g) * 2]));
            float Ls = 0.f, Os = 0.f;
            for (int sidx = c_first; sidx <= c_last; ++sidx) {
              const size_t base = (size_t)(sidx + item) * a.G + g;
              const float f = exp2f(__ldcg(&a.part_ml[base * 2]) - Mx);
              Ls += __ldcg(&a.part_ml[base * 2 + 1]) * f;
              Os += __ldcg(&a.part_acc[base * kD + tid]) * f;
            }
            M[g] = Mx; Lsum[g] = Ls; O[g] = Os;
          }
      }
    }
    if (nseg == 1 || s_last) {
#pragma unroll
      for (int g = 0; g < GP; ++g)
        if (g < a.G) {
          const size_t row = (size_t)b * c.Hq + kvh * a.G + g;
          a.out[row * kD + tid] = __float2bfloat16(O[g] / Lsum[g]);
          if (a.out_f32) a.out_f32[row * kD + tid] = O[g] / Lsum[g];
          if (a.lse && tid == 0) a.lse[row] = (M[g] + log2f(Lsum[g])) * kLn2;
        }
    }
    __syncthreads();
    p += j1 - j0;
  }
}


template <int GP>
static int launch_simt(const DecodeArgs &a, int grid, size_t smem, cudaStream_t s) {
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(decode_simt_kernel<GP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return SPKV_E_CUDA;
  decode_simt_kernel<GP><<<grid, 128, smem, s>>>(a);
  return check_stream_error(cudaGetLastError());
}


int launch_decode_simt(const DecodeArgs &a, int sm_count, cudaStream_t s) {
  int GP = 1;
  while (GP < a.G) GP <<= 1;
  const int n_items = a.n_items;
  const int grid = min(kMaxGrid, sm_count * 4);
  const size_t smem = (size_t)(n_items + n_items + 1 + 64) * 4 + (size_t)n_items * sizeof(ItemInfo) +
                      (size_t)4 * GP * 130 * 4;
  switch (GP) {
    case 1: return launch_simt<1>(a, grid, smem, s);
    case 2: return launch_simt<2>(a, grid, smem, s);
    case 4: return launch_simt<4>(a, grid, smem, s);
    case 8: return launch_simt<8>(a, grid, smem, s);
    case 16: return launch_simt<16>(a, grid, smem, s);
    default: return SPKV_E_UNSUPPORTED;
  }
}

}  // namespace spkv
