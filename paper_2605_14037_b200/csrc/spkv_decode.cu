// Step 3 of the hot path: ragged split-K decode attention (Eq. 3-5) over
// ring window U compact cache, with the log-sum-exp merge fused in.
//
// Schedule.  The call covers n_items = B * n_kv_heads units.  Unit i owns a list of
// np_i pages (its kept pages followed by its ring pages).  All lists are laid end to
// end into one sequence of NP pages and cut into `gridDim.x` contiguous ranges of equal
// size (+-1 page), one per thread block, whatever the keep rates of the heads are.  A
// range may cover the tail of one unit, several whole units and the head of another;
// each (block, unit) intersection is a "segment".  Every block recomputes the prefix
// sums of np_i itself (lengths live on the device and change every step), so no extra
// launch and no host synchronisation is needed.
//
// Merge.  A segment that covers its whole unit writes the output directly.  Otherwise
// the block stores (m, l, acc) for the segment in workspace slot (block + item) -- unique
// because consecutive segments differ in block or item -- and bumps the unit's arrival
// counter; the block that arrives last merges all slots of the unit by their
// log-sum-exp weights and resets the counter.  Nobody ever waits.
#include <stdlib.h>

#include "spkv_internal.cuh"
#include "spkv_mma.cuh"

namespace spkv {

constexpr int kMaxGrid = 1024;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecodeArgs {
  CacheView c;
  int layer, B, n_items, G;
  const int32_t *seq_ids;
  const __nv_bfloat16 *q;  // [B][Hq][128]
  __nv_bfloat16 *out;      // [B][Hq][128]
  float *lse;              // [B][Hq] or null
  float scale_log2;        // sm_scale * log2(e)
  int32_t *counters;       // [n_items]
  float *part_ml;          // [slots][G][2]
  float *part_acc;         // [slots][G][128]
};

struct ItemInfo {  // per item, in shared memory
  int unit, len, n_ring, nk;
};

// Exclusive prefix sum over s_np[0..n) -> s_pre[0..n], s_pre[n] = total.  All threads call.
__device__ inline void block_exclusive_scan(const int *s_np, int *s_pre, int n, int *s_tmp) {
  const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (n + nt - 1) / nt;
  const int a = min(tid * per, n), b = min(a + per, n);
  int sum = 0;
  for (int i = a; i < b; ++i) sum += s_np[i];
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_tmp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int v = lane < (nt >> 5) ? s_tmp[lane] : 0;
    int inc2 = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int x = __shfl_up_sync(0xffffffffu, inc2, o);
      if (lane >= o) inc2 += x;
    }
    s_tmp[32 + lane] = inc2 - v;  // exclusive offset of each warp
  }
  __syncthreads();
  int run = s_tmp[32 + warp] + incl - sum;
  for (int i = a; i < b; ++i) {
    s_pre[i] = run;
    run += s_np[i];
  }
  if (tid == nt - 1) s_pre[n] = run;
  __syncthreads();
}

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

// ------------------------------------------------------------------------------------
// Baseline kernel (CUDA cores, warp-shuffle dot products, direct global loads).
// 4 warps; warp w of a block takes pages j0+w, j0+w+4, ... of a segment; lane l owns
// dims 4l..4l+3 of every row.  Kept as the simple comparison point for the tensor-core
// kernel below: same schedule, same merge.
// ------------------------------------------------------------------------------------
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
          if (a.lse && tid == 0) a.lse[row] = (M[g] + log2f(Lsum[g])) * kLn2;
        }
    }
    __syncthreads();
    p += j1 - j0;
  }
}


// ------------------------------------------------------------------------------------
// Main kernel: one persistent block per SM, a pipeline of whole pages.
//
//   warp 4, lane 0 (producer): for every page of the block's range, one 32 KB linear bulk
//       copy HBM -> shared memory (cp.async.bulk, completion counted on an mbarrier).
//       The page in HBM already is the swizzled shared-memory image, so nothing is
//       rearranged on the way.  n_stages pages (5-6, i.e. 160-192 KB per SM) are in flight.
//   warps 0-3 (consumers): each takes 16 of the page's 64 pairs.  The group's G query
//       heads form the rows of a 16-row tile (padded), so S = Q K^T and O += P V are small
//       dense products done with mma.sync m16n8k16 (bf16 in, fp32 accumulate), operands
//       read with ldmatrix; masking, online softmax (exp2, quad shuffles) in registers.
//       A warp keeps its own (m, l, O) for its quarter of every page of a segment; the
//       four are merged through shared memory once per segment.
//
// Why tensor cores in a bandwidth-bound kernel: per 512 B pair the group needs 2*G*128
// multiply-adds.  On the CUDA cores (kernel above) that is, with bf16 unpacking and the
// reductions, several hundred issue slots per pair and SM -- the issue rate, not HBM, then
// limits the kernel at G >= 4.  As MMA tiles the same arithmetic is 2 x 16 instructions per
// page and warp, and the kernel is limited by the page stream alone.
//
// Every wait is bounded: if a copy never lands the waiting thread records
// SPKV_E_TIMEOUT, raises the block's abort flag, and all threads run to the end without
// waiting again (control flow stays uniform, outputs are then meaningless).
// ------------------------------------------------------------------------------------
constexpr int kListCap = 512;
constexpr int kTcThreads = 160;

struct TcSmem {  // offsets into dynamic shared memory, computed on host and device alike
  int n_stages, off_bar, off_np, off_pre, off_tmp, off_list, off_meta, off_red, off_flags, total;
};
__host__ __device__ inline TcSmem tc_smem_layout(int n_items, int GP, int n_stages) {
  TcSmem L;
  L.n_stages = n_stages;
  int o = n_stages * kPageBytes;
  L.off_bar = o;   o += 2 * 8 * 8;  // up to 8 stages: full[8], empty[8]
  L.off_np = o;    o += n_items * 4;
  L.off_pre = o;   o += (n_items + 1) * 4;
  L.off_tmp = o;   o += 64 * 4;
  L.off_list = o;  o += kListCap * 4;
  L.off_meta = o;  o += kListCap * 4;
  o = (o + 15) / 16 * 16;
  L.off_red = o;   o += 4 * GP * 132 * 4;
  L.off_flags = o; o += 16;
  L.total = o;
  return L;
}

__device__ inline void consumer_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ inline void wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                     const CacheView &c) {
  if (*abort_flag) return;
  if (!mbar_wait_bounded(bar, parity)) {
    *abort_flag = 1;
    set_status(c, SPKV_E_TIMEOUT);
  }
}

__global__ void __launch_bounds__(kTcThreads, 1) decode_tc_kernel(DecodeArgs a, int GP, int n_stages) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const CacheView &c = a.c;
  const int n = a.n_items;
  const TcSmem L = tc_smem_layout(n, GP, n_stages);
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + L.off_bar);
  uint64_t *empty = full + 8;
  int *s_np = reinterpret_cast<int *>(smem + L.off_np);
  int *s_pre = reinterpret_cast<int *>(smem + L.off_pre);
  int *s_tmp = reinterpret_cast<int *>(smem + L.off_tmp);
  int *s_list = reinterpret_cast<int *>(smem + L.off_list);
  int *s_meta = reinterpret_cast<int *>(smem + L.off_meta);
  float *s_red = reinterpret_cast<float *>(smem + L.off_red);
  volatile int *s_abort = reinterpret_cast<volatile int *>(smem + L.off_flags);
  volatile int *s_last = s_abort + 1;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int i = 0; i < n_stages; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 4);
    }
    mbar_fence_init();
    *s_abort = 0;
    *s_last = 0;
  }
  for (int i = tid; i < n; i += kTcThreads) {
    const int b = i / c.Hkv, kvh = i % c.Hkv;
    const int seq = a.seq_ids[b];
    int np = 0;
    if (seq >= 0 && seq < c.S) {
      const int u = unit_index(c, a.layer, seq, kvh);
      np = (c.len[u] + kP - 1) / kP + (min(c.t[u], c.w) + kP - 1) / kP;
    } else if (blockIdx.x == 0) {
      set_status(c, SPKV_E_BOUNDS);
    }
    s_np[i] = np;
    if (np == 0 && blockIdx.x == 0) {
      for (int g = 0; g < a.G; ++g) {
        __nv_bfloat16 *o = a.out + ((size_t)b * c.Hq + kvh * a.G + g) * kD;
        for (int d = 0; d < kD; ++d) o[d] = __float2bfloat16(0.f);
        if (a.lse) a.lse[(size_t)b * c.Hq + kvh * a.G + g] = -INFINITY;
      }
    }
  }
  __syncthreads();
  block_exclusive_scan(s_np, s_pre, n, s_tmp);
  const int NP = s_pre[n];
  if (NP == 0) return;
  const int nb = min((int)gridDim.x, NP);
  if ((int)blockIdx.x >= nb) return;
  const int p_begin = range_start(blockIdx.x, NP, nb);
  const int p_end = range_start(blockIdx.x + 1, NP, nb);

  // consumer state
  uint32_t qf[8][4];
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f}, o[16][4];
  int k_page = 0;  // pages handled so far by this block (same count in producer and consumers)

  for (int round = p_begin; round < p_end; round += kListCap) {
    const int cnt = min(kListCap, p_end - round);
    __syncthreads();  // the previous round's list is no longer in use
    for (int i = tid; i < cnt; i += kTcThreads) {
      const int pp = round + i;
      int lo = 0, hi = n;
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (s_pre[mid] <= pp) lo = mid; else hi = mid;
      }
      const int item = lo, j = pp - s_pre[item];
      const int u = unit_index(c, a.layer, a.seq_ids[item / c.Hkv], item % c.Hkv);
      const int len = c.len[u], nk = (len + kP - 1) / kP;
      int gpage, valid;
      if (j < nk) {
        gpage = c.table[(size_t)u * c.max_pages + j];
        valid = min(kP, len - j * kP);
      } else {
        gpage = (int)ring_page(c, u, j - nk);
        valid = min(kP, min(c.t[u], c.w) - (j - nk) * kP);
      }
      const int seg_begin = (pp == p_begin) || (j == 0);
      const int seg_end = (pp == p_end - 1) || (j == s_np[item] - 1);
      s_list[i] = gpage;
      s_meta[i] = valid | (seg_end << 8) | (seg_begin << 9) | (item << 10);
    }
    __syncthreads();

    if (warp == 4) {
      if (lane == 0) {
        for (int i = 0; i < cnt; ++i) {
          const int k = k_page + i, stage = k % n_stages, use = k / n_stages;
          if (use > 0) wait_or_abort(&empty[stage], (use - 1) & 1, s_abort, c);
          mbar_arrive_expect_tx(&full[stage], kPageBytes);
          bulk_load(smem + (size_t)stage * kPageBytes, c.pages + (int64_t)s_list[i] * kPageElems,
                    kPageBytes, &full[stage]);
        }
      }
    } else {
      for (int i = 0; i < cnt; ++i) {
        const int k = k_page + i, stage = k % n_stages, use = k / n_stages;
        const int meta = s_meta[i];
        const int valid = meta & 255, item = meta >> 10;
        const int b = item / c.Hkv, kvh = item % c.Hkv;
        if (meta & 512) {  // first page of a segment
          load_q_frags(qf, [&](int r) -> const __nv_bfloat16 * {
            return r < a.G ? a.q + ((size_t)b * c.Hq + kvh * a.G + r) * kD : nullptr;
          }, lane);
          m[0] = m[1] = -INFINITY;
          l[0] = l[1] = 0.f;
#pragma unroll
          for (int x = 0; x < 16; ++x) o[x][0] = o[x][1] = o[x][2] = o[x][3] = 0.f;
        }
        wait_or_abort(&full[stage], use & 1, s_abort, c);
        const int tok0 = warp * 16;
        if (tok0 < valid) {
          const uint32_t sK = smem_u32(smem + (size_t)stage * kPageBytes), sV = sK + kBlockElems * 2;
          float s[2][4];
          qk_tile<16>(s, qf, sK, tok0, lane);
          softmax_pv_tile<16>(s, [&](int, int col) { return col < valid; }, a.scale_log2, m, l, o, sV,
                              tok0, lane);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);

        if (meta & 256) {  // last page of the segment: merge the four warps, emit
          const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            l[h] += __shfl_xor_sync(0xffffffffu, l[h], 1);
            l[h] += __shfl_xor_sync(0xffffffffu, l[h], 2);
            const int row = g + 8 * h;
            if (row < a.G) {
              float *dst = s_red + ((size_t)warp * GP + row) * 132;
#pragma unroll
              for (int x = 0; x < 16; ++x) {
                dst[x * 8 + t4 * 2] = o[x][2 * h];
                dst[x * 8 + t4 * 2 + 1] = o[x][2 * h + 1];
              }
              if (t4 == 0) { dst[128] = m[h]; dst[129] = l[h]; }
            }
          }
          consumer_bar();
          const int c_first = block_of_page(s_pre[item], NP, nb);
          const int c_last = block_of_page(s_pre[item + 1] - 1, NP, nb);
          const int nseg = c_last - c_first + 1;
          const int slot = blockIdx.x + item;
          for (int gh = 0; gh < a.G; ++gh) {
            float M = -INFINITY;
#pragma unroll
            for (int w4 = 0; w4 < 4; ++w4) M = fmaxf(M, s_red[((size_t)w4 * GP + gh) * 132 + 128]);
            float Ls = 0.f, Os = 0.f;
#pragma unroll
            for (int w4 = 0; w4 < 4; ++w4) {
              const float *src = s_red + ((size_t)w4 * GP + gh) * 132;
              const float f = src[128] == -INFINITY ? 0.f : exp2f(src[128] - M);
              Ls += src[129] * f;
              Os += src[tid] * f;
            }
            const size_t row = (size_t)b * c.Hq + kvh * a.G + gh;
            if (nseg == 1) {
              a.out[row * kD + tid] = __float2bfloat16(Os / Ls);
              if (a.lse && tid == 0) a.lse[row] = (M + log2f(Ls)) * kLn2;
            } else {
              a.part_acc[((size_t)slot * a.G + gh) * kD + tid] = Os;
              if (tid == 0) {
                a.part_ml[((size_t)slot * a.G + gh) * 2 + 0] = M;
                a.part_ml[((size_t)slot * a.G + gh) * 2 + 1] = Ls;
              }
            }
          }
          if (nseg > 1) {
            __threadfence();
            consumer_bar();
            if (tid == 0) {
              const int old = atomicAdd(&a.counters[item], 1);
              const int last = old == nseg - 1;
              if (last) a.counters[item] = 0;
              *s_last = last;
            }
            consumer_bar();
            if (*s_last) {
              __threadfence();
              for (int gh = 0; gh < a.G; ++gh) {
                float Mx = -INFINITY;
                for (int sidx = c_first; sidx <= c_last; ++sidx)
                  Mx = fmaxf(Mx, __ldcg(&a.part_ml[((size_t)(sidx + item) * a.G + gh) * 2]));
                float Ls = 0.f, Os = 0.f;
                for (int sidx = c_first; sidx <= c_last; ++sidx) {
                  const size_t base = (size_t)(sidx + item) * a.G + gh;
                  const float f = exp2f(__ldcg(&a.part_ml[base * 2]) - Mx);
                  Ls += __ldcg(&a.part_ml[base * 2 + 1]) * f;
                  Os += __ldcg(&a.part_acc[base * kD + tid]) * f;
                }
                const size_t row = (size_t)b * c.Hq + kvh * a.G + gh;
                a.out[row * kD + tid] = __float2bfloat16(Os / Ls);
                if (a.lse && tid == 0) a.lse[row] = (Mx + log2f(Ls)) * kLn2;
              }
            }
          }
          consumer_bar();  // s_red and s_last are free again
        }
      }
    }
    k_page += cnt;
  }
  // after an abort, do not leave while copies may still be landing in shared memory
  __syncthreads();
  if (*s_abort && tid == 0) {
    const int first = max(0, k_page - n_stages);
    for (int k = first; k < k_page; ++k) mbar_wait_bounded(&full[k % n_stages], (k / n_stages) & 1);
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

size_t decode_ws_bytes(int n_items, int G) {
  size_t counters = ((size_t)n_items * 4 + 255) / 256 * 256;
  size_t slots = (size_t)kMaxGrid + n_items;
  size_t ml = (slots * G * 2 * 4 + 255) / 256 * 256;
  size_t acc = slots * G * kD * 4;
  return counters + ml + acc;
}

}  // namespace spkv

using namespace spkv;

extern "C" size_t spkv_decode_workspace_bytes(const spkv_config_t *cfg, int32_t B) {
  if (!cfg || B < 0 || cfg->n_kv_heads < 1) return 0;
  return decode_ws_bytes(B * cfg->n_kv_heads, cfg->n_q_heads / cfg->n_kv_heads);
}

extern "C" int spkv_decode_attention(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                                     int32_t B, const void *d_q, void *d_out, float *d_lse_opt,
                                     float sm_scale, void *d_workspace, size_t workspace_bytes,
                                     spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || B < 0 || B > cache->cfg.max_seqs)
    return SPKV_E_INVALID;
  if (B == 0) return SPKV_OK;
  if (!d_seq_ids || !d_q || !d_out) return SPKV_E_INVALID;
  if (((uintptr_t)d_q | (uintptr_t)d_out) & 15) return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  const int n_items = B * v.Hkv;
  if (n_items > 4096) return SPKV_E_UNSUPPORTED;
  if (!d_workspace || ((uintptr_t)d_workspace & 255) || workspace_bytes < decode_ws_bytes(n_items, v.G))
    return SPKV_E_WORKSPACE;

  DecodeArgs a;
  a.c = v; a.layer = layer; a.B = B; a.n_items = n_items; a.G = v.G;
  a.seq_ids = d_seq_ids;
  a.q = static_cast<const __nv_bfloat16 *>(d_q);
  a.out = static_cast<__nv_bfloat16 *>(d_out);
  a.lse = d_lse_opt;
  a.scale_log2 = sm_scale * kLog2e;
  char *ws = static_cast<char *>(d_workspace);
  a.counters = reinterpret_cast<int32_t *>(ws);
  size_t off = ((size_t)n_items * 4 + 255) / 256 * 256;
  a.part_ml = reinterpret_cast<float *>(ws + off);
  off += (((size_t)kMaxGrid + n_items) * v.G * 2 * 4 + 255) / 256 * 256;
  a.part_acc = reinterpret_cast<float *>(ws + off);

  int GP = 1;
  while (GP < v.G) GP <<= 1;
  cudaStream_t s = as_stream(stream);
  static const bool use_simt = [] {
    const char *e = getenv("SPKV_DECODE_KERNEL");  // "simt": the CUDA-core comparison kernel
    return e && e[0] == 's';
  }();
  if (!use_simt) {
    if (n_items > 1024) return SPKV_E_UNSUPPORTED;
    int n_stages = 6;
    TcSmem L = tc_smem_layout(n_items, GP, n_stages);
    while (L.total > 227 * 1024 && n_stages > 2) L = tc_smem_layout(n_items, GP, --n_stages);
    if (cudaFuncSetAttribute(decode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total) !=
        cudaSuccess)
      return SPKV_E_CUDA;
    decode_tc_kernel<<<min(kMaxGrid, cache->sm_count), kTcThreads, L.total, s>>>(a, GP, n_stages);
    return check_stream_error(cudaGetLastError());
  }
  const int grid = min(kMaxGrid, cache->sm_count * 4);
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

static size_t a256(size_t x) { return (x + 255) / 256 * 256; }

extern "C" size_t spkv_decode_step_staging_bytes(const spkv_config_t *cfg, int32_t B, int32_t d_in) {
  if (!cfg || B < 0 || d_in < 0) return 0;
  const size_t q = a256((size_t)B * cfg->n_q_heads * kD * 2), kv = a256((size_t)B * cfg->n_kv_heads * kD * 2);
  return a256((size_t)B * d_in * 2) + 2 * q + 2 * kv + a256((size_t)B * cfg->n_kv_heads * 4) +
         spkv_decode_workspace_bytes(cfg, B);
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
  const spkv_config_t &cfg = cache->cfg;
  const size_t xb = (size_t)B * pred->d_in * 2, qb = (size_t)B * cfg.n_q_heads * kD * 2,
               kvb = (size_t)B * cfg.n_kv_heads * kD * 2;
  char *p = static_cast<char *>(d_staging);
  char *d_x = p; p += a256(xb);
  char *d_q = p; p += a256(qb);
  char *d_o = p; p += a256(qb);
  char *d_k = p; p += a256(kvb);
  char *d_v = p; p += a256(kvb);
  float *d_lg = reinterpret_cast<float *>(p); p += a256((size_t)B * cfg.n_kv_heads * 4);
  cudaStream_t s = as_stream(stream);
  if (cudaMemcpyAsync(d_x, h_x, xb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(d_q, h_q, qb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(d_k, h_k, kvb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(d_v, h_v, kvb, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return SPKV_E_CUDA;
  int rc = spkv_score(cache, pred, d_x, B, d_lg, nullptr, stream);
  if (rc) return rc;
  rc = spkv_append_evict(cache, layer, d_seq_ids, B, d_k, d_v, d_lg, stream);
  if (rc) return rc;
  rc = spkv_decode_attention(cache, layer, d_seq_ids, B, d_q, d_o, nullptr, sm_scale, p,
                             spkv_decode_workspace_bytes(&cfg, B), stream);
  if (rc) return rc;
  return check_stream_error(cudaMemcpyAsync(h_out, d_o, qb, cudaMemcpyDeviceToHost, s));
}
