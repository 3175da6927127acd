// Companion path: chunked prefill of C pairs for one (layer, sequence).
//
// By definition the result equals C x (append/evict, decode attention) -- the paper's
// chunked-prefill protocol, cache compressed after every chunk (Section "Sparse decoding
// approximation"), attention per Eq. 3-5.  It is computed in five launches:
//
//  A  plan     one block per KV head: thresholds the old ring pairs and the chunk pairs in
//              position order ("staging" sequence of N = min(t0,w) + C pairs), exclusive
//              prefix sum of the flags (warp ballot + popc, block carry), pops the pages
//              the unit will need and extends its page table.
//  B  scatter  stream compaction proper: every flagged staging pair whose position is
//              <= t_last - w is copied to compact-cache index len0 + E[j] (ascending
//              position, so order and indices are unique and bit-exact).
//  STG stage    the old ring pairs and the chunk's pairs, in position order, rewritten as pages
//              in the workspace ("staging pages"), so that every key/value tile of the
//              attention -- compact-cache page or band page -- is the same 32 KB image.
//  ATT attention of every query of the chunk (tcgen05 tensor cores, fp32 accumulation, online
//              softmax; spkv_prefill_tc5x2h.cu) over
//                (a) the first nvis(t) = len0 + E[t - w - p0 + 1] pairs of the compact cache
//                    (the kept pairs with position <= t - w: a prefix, because the cache is in
//                    ascending position order), and
//                (b) the dense band t-w < s <= t, read from the not-yet-updated ring and the
//                    chunk's own K/V.
//              A kept pair inside the band is counted once: the prefix (a) stops at t - w.
//  C  ring     the last min(C, w) pairs of the chunk overwrite their ring slots; t and len
//              are advanced.
//
// Workspace per KV head: a 64-int header followed by E[0..N] (int32).
#include "spkv_prefill_common.cuh"

namespace spkv {

// ---------------------------------------------------------------- A: plan (flags + scan)
__global__ void __launch_bounds__(1024) prefill_plan_kernel(PrefillArgs a) {
  pdl_chain_link();
  const CacheView &c = a.c;
  const int kvh = blockIdx.x;
  const int u = unit_index(c, a.layer, a.seq, kvh);
  int32_t *hdr = unit_ws(a, kvh);
  int32_t *E = hdr + kHdrInts;
  const int t0 = c.t[u], len0 = c.len[u];
  const float thr = head_threshold(c, a.layer, kvh, a.tau_logit);
  const int trow = c.table_row[u];   // -1: a head declared local-only keeps nothing, sinks included
  const int n_old = min(t0, c.w), p0 = t0 - n_old;
  const int N = n_old + a.C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __shared__ int s_warp[32];
  __shared__ int s_carry, s_pages_base, s_fail;
  if (tid == 0) { s_carry = 0; s_fail = 0; }
  __syncthreads();
  for (int base = 0; base < N; base += 1024) {
    const int j = base + tid;
    bool flag = false;
    if (j < N) {
      const float lg = j < n_old ? c.ring_logit[(size_t)u * c.w + (p0 + j) % c.w]
                                 : a.logits[(size_t)(j - n_old) * c.Hkv + kvh];
      flag = trow >= 0 && (lg >= thr || p0 + j < c.n_sink);  // Eq. 2 on the float32 logit; sink positions always
    }
    const unsigned ballot = __ballot_sync(0xffffffffu, flag);
    const int before = __popc(ballot & ((1u << lane) - 1u));
    if (lane == 31) s_warp[warp] = __popc(ballot);
    __syncthreads();
    if (warp == 0) {
      int v = s_warp[lane], incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
      }
      s_warp[lane] = incl - v;
      if (lane == 31) s_pages_base = incl;  // tile total (reusing the slot)
    }
    __syncthreads();
    if (j < N) E[j] = s_carry + s_warp[warp] + before;
    __syncthreads();
    if (tid == 0) s_carry += s_pages_base;
    __syncthreads();
  }
  if (tid == 0) E[N] = s_carry;
  __syncthreads();
  // pairs leaving the window in this call: staging index j < N - w
  const int n_leave = max(N - c.w, 0);
  const int n_commit = E[n_leave];  // written by this block above
  const int len1 = len0 + n_commit;
  const int pages0 = (len0 + kP - 1) / kP, pages1 = (len1 + kP - 1) / kP;
  const int n_new = pages1 - pages0;
  if (tid == 0) {
    int fail = 0;
    if (pages1 > c.max_pages) {
      fail = SPKV_E_CONTEXT_OVERFLOW;
    } else if (n_new > 0) {
      // all n_new pages or none: the counter only ever moves by what is really taken, so the
      // blocks of the other KV heads never see a number lower than the pool holds
      int top = atomicAdd(&c.status[1], 0);
      for (;;) {
        if (top < n_new) { fail = SPKV_E_POOL_EXHAUSTED; break; }
        const int seen = atomicCAS(&c.status[1], top, top - n_new);
        if (seen == top) { s_pages_base = top; break; }
        top = seen;
      }
    }
    if (fail) set_status(c, fail);
    s_fail = fail;
    hdr[H_T0] = t0; hdr[H_LEN0] = len0; hdr[H_NOLD] = n_old; hdr[H_N] = N;
    hdr[H_NCOMMIT] = fail ? 0 : n_commit;
    hdr[H_LEN1] = fail ? len0 : len1;
    hdr[H_FAIL] = fail;
    hdr[H_VMAX] = (int32_t)c.vmax[u];   // the kept pairs so far; the stage kernel adds ring and chunk
  }
  __syncthreads();
  if (s_fail || n_new == 0) return;
  // (debug bounds: an index from the stack that names no pool page is recorded; the scatter kernel
  // skips what would go there)
  int32_t *table = unit_table(c, trow);   // n_new > 0: the unit keeps pairs, so it has a table
  for (int i = tid; i < n_new; i += blockDim.x)
    table[pages0 + i] = checked_page(c, c.free_stack[s_pages_base - 1 - i], -1);
  __syncthreads();
  // rows past the final length of a freshly popped last page must read as zeros
  if (len1 % kP && table[pages1 - 1] >= 0) {
    const int last = table[pages1 - 1];
    uint4 *vb = reinterpret_cast<uint4 *>(c.pages + (int64_t)last * kPageElems + kBlockElems);
    for (int i = tid; i < kBlockElems * 2 / 16; i += blockDim.x) vb[i] = make_uint4(0, 0, 0, 0);
  }
}

// Source row of staging pair j: old ring slot (swizzled page) or chunk input (linear).
struct SrcRow {
  const __nv_bfloat16 *k, *v;  // row >= 0: base of the key / value block; row < 0: the row itself
  int row;                     // >= 0: row of a swizzled block; -1: linear row
};
__device__ inline SrcRow staging_row(const PrefillArgs &a, int u, int kvh, int t0, int n_old, int j) {
  SrcRow r;
  if (j < n_old) {
    const int slot = (t0 - n_old + j) % a.c.w;
    const __nv_bfloat16 *pg = a.c.pages + ring_page(a.c, u, slot / kP) * kPageElems;
    r.row = slot % kP;
    r.k = pg;
    r.v = pg + kBlockElems;
  } else {
    const size_t off = ((size_t)(j - n_old) * a.c.Hkv + kvh) * kD;
    r.row = -1;
    r.k = a.k + off;
    r.v = a.v + off;
  }
  return r;
}
__device__ inline uint4 load_chunk(const __nv_bfloat16 *rowbase, int row, int chunk) {
  return *reinterpret_cast<const uint4 *>(rowbase + (row >= 0 ? swz_off(row, chunk) : chunk * 8));
}

// ------------------------------------------------------------------ B: scatter (compact)
// grid (ceil(n_leave_max / 64), Hkv); each warp moves 8 consecutive staging pairs.
__global__ void __launch_bounds__(256) prefill_scatter_kernel(PrefillArgs a) {
  pdl_chain_link();
  const CacheView &c = a.c;
  const int kvh = blockIdx.y;
  const int32_t *hdr = unit_ws(a, kvh);
  const int32_t *E = hdr + kHdrInts;
  if (hdr[H_FAIL]) return;
  const int t0 = hdr[H_T0], len0 = hdr[H_LEN0], n_old = hdr[H_NOLD], N = hdr[H_N];
  const int n_leave = max(N - c.w, 0);
  const int u = unit_index(c, a.layer, a.seq, kvh);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = lane & 15, blk = (lane >> 4) * kBlockElems;
  const int j0 = (blockIdx.x * 8 + warp) * 8;
  const int trow = c.table_row[u];
  uint32_t vm = 0;  // largest |v| among the pairs this warp appends to the compact cache
  for (int j = j0; j < min(j0 + 8, n_leave); ++j) {
    const int e = E[j];
    if (E[j + 1] == e) continue;  // not flagged
    const int idx = len0 + e;
    const int page = checked_page(c, unit_table(c, trow)[idx / kP], -1);
    if (page < 0) continue;   // debug bounds: recorded, the pair is not written
    const int drow = idx % kP;
    const SrcRow s = staging_row(a, u, kvh, t0, n_old, j);
    const uint4 val = load_chunk(lane < 16 ? s.k : s.v, s.row, chunk);
    *reinterpret_cast<uint4 *>(c.pages + (int64_t)page * kPageElems + blk + swz_off(drow, chunk)) = val;
    if (lane >= 16) vm = max(vm, chunk_abs_max_bf16(val));
    if (lane == 0) c.pos_pool[((int64_t)page - c.n_ring_pages_total) * kP + drow] = t0 - n_old + j;
  }
  vm = __reduce_max_sync(0xffffffffu, vm);
  if (lane == 0 && vm) note_vmax(c, u, vm);
}

// --------------------------------------------------------------------- C: ring update
// grid (ceil(min(C,w) / 8), Hkv); one warp per pair.
__global__ void __launch_bounds__(256) prefill_ring_kernel(PrefillArgs a) {
  pdl_chain_link();
  const CacheView &c = a.c;
  const int kvh = blockIdx.y;
  const int32_t *hdr = unit_ws(a, kvh);
  const int t0 = hdr[H_T0];
  const int u = unit_index(c, a.layer, a.seq, kvh);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int first = max(a.C - c.w, 0);
  const int i = first + blockIdx.x * 8 + warp;
  if (i < a.C) {
    const int slot = (t0 + i) % c.w, row = slot % kP;
    __nv_bfloat16 *pg = c.pages + ring_page(c, u, slot / kP) * kPageElems;
    const int chunk = lane & 15, blk = (lane >> 4) * kBlockElems;
    const size_t off = ((size_t)i * c.Hkv + kvh) * kD;
    const uint4 val = *reinterpret_cast<const uint4 *>((lane < 16 ? a.k : a.v) + off + chunk * 8);
    *reinterpret_cast<uint4 *>(pg + blk + swz_off(row, chunk)) = val;
    if (lane == 0) c.ring_logit[(size_t)u * c.w + slot] = a.logits[(size_t)i * c.Hkv + kvh];
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    c.t[u] = t0 + a.C;
    c.len[u] = hdr[H_LEN1];
  }
}

// ------------------------------------------------------------------ STG: staging pages
// Old ring pairs and chunk pairs, in position order, rewritten as pages (workspace).
// grid (n_stage_pages, Hkv), 256 threads: 8 warps x 8 rows.
__global__ void __launch_bounds__(256) prefill_stage_kernel(PrefillArgs a) {
  pdl_chain_link();
  const CacheView &c = a.c;
  const int kvh = blockIdx.y, sp = blockIdx.x;
  int32_t *hdr = unit_ws(a, kvh);
  const int t0 = hdr[H_T0], n_old = hdr[H_NOLD], N = hdr[H_N];
  const int u = unit_index(c, a.layer, a.seq, kvh);
  __nv_bfloat16 *page = a.stage_pages + ((size_t)kvh * a.n_stage_pages + sp) * kPageElems;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = lane & 15, blk = (lane >> 4) * kBlockElems;
  uint32_t vm = 0;  // largest |v| among the values this lane moves
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
      }
      if (lane >= 16) vm = max(vm, chunk_abs_max_bf16(val));
    }
    *reinterpret_cast<uint4 *>(page + blk + swz_off(r, chunk)) = val;
  }
  vm = __reduce_max_sync(0xffffffffu, vm);
  if (lane == 0 && vm) atomicMax(reinterpret_cast<uint32_t *>(&hdr[H_VMAX]), vm);
}

int launch_prefill_stage(const PrefillArgs &a, cudaStream_t s) {
  return check_stream_error(launch_link(a.chained != 0, prefill_stage_kernel, dim3(a.n_stage_pages, a.c.Hkv), dim3(256), 0, s, a));
}

static size_t prefill_ws_stride_ints(int C, int w) {
  size_t ints = kHdrInts + (size_t)C + w + 2;
  return (ints + 63) / 64 * 64;
}

}  // namespace spkv

using namespace spkv;

static size_t prefill_plan_bytes(const spkv_config_t *cfg, int C) {
  size_t b = prefill_ws_stride_ints(C, cfg->window) * 4 * (size_t)cfg->n_kv_heads;
  return (b + 1023) / 1024 * 1024;
}
static int prefill_stage_pages(const spkv_config_t *cfg, int C) { return (C + cfg->window + kP - 1) / kP; }

extern "C" size_t spkv_prefill_workspace_bytes(const spkv_config_t *cfg, int32_t C) {
  if (!cfg || C < 0) return 0;
  // plan (header + prefix sums per KV head), then the staging pages of the chunk attention, then
  // (small chunks only) the partial results of split page walks
  return prefill_plan_bytes(cfg, C) + (size_t)cfg->n_kv_heads * prefill_stage_pages(cfg, C) * kPageBytes +
         prefill_split_bytes(cfg, C);
}

extern "C" int spkv_prefill(spkv_cache_t *cache, int32_t layer, int32_t seq, int32_t C,
                            const void *d_q, const void *d_k, const void *d_v,
                            const float *d_logits, void *d_out, float sm_scale, void *d_workspace,
                            size_t workspace_bytes, spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || seq < 0 || seq >= cache->cfg.max_seqs || C < 0)
    return SPKV_E_INVALID;
  if (C == 0) return SPKV_OK;
  if (!d_k || !d_v || !d_logits || ((d_q == nullptr) != (d_out == nullptr))) return SPKV_E_INVALID;
  // the attention kernel folds the scale into the exponent and takes row maxima before scaling
  if (d_q && !(sm_scale > 0.f && sm_scale < INFINITY)) return SPKV_E_INVALID;
  if (((uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_q | (uintptr_t)d_out) & 15) return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  if (!d_workspace || ((uintptr_t)d_workspace & 255) ||
      workspace_bytes < spkv_prefill_workspace_bytes(&cache->cfg, C))
    return SPKV_E_WORKSPACE;
  PrefillArgs a;
  a.c = v; a.layer = layer; a.seq = seq; a.C = C;
  a.q = static_cast<const __nv_bfloat16 *>(d_q);
  a.k = static_cast<const __nv_bfloat16 *>(d_k);
  a.v = static_cast<const __nv_bfloat16 *>(d_v);
  a.logits = d_logits;
  a.out = static_cast<__nv_bfloat16 *>(d_out);
  a.tau_logit = cache->tau_logit;
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.ws = static_cast<int32_t *>(d_workspace);
  a.ws_stride = (int)prefill_ws_stride_ints(C, v.w);
  a.stage_pages = reinterpret_cast<__nv_bfloat16 *>(static_cast<char *>(d_workspace) +
                                                    prefill_plan_bytes(&cache->cfg, C));
  a.n_stage_pages = prefill_stage_pages(&cache->cfg, C);
  a.pair_tiles = 0;
  a.n_split = 1;
  a.force_wide = (cache->cfg.flags & SPKV_FLAG_PREFILL_PV_BF16) ? 1 : 0;
  a.soft = 0;
  a.gate2 = nullptr;
  a.lse = nullptr;
  a.chained = C < 64;   // measured: see pdl_chain_link
  a.partials = prefill_split_bytes(&cache->cfg, C)
                   ? reinterpret_cast<float *>(reinterpret_cast<char *>(a.stage_pages) +
                                               (size_t)v.Hkv * a.n_stage_pages * kPageBytes)
                   : nullptr;
  cudaStream_t s = as_stream(stream);
  cache->last_kind = kLastOther;

  if (launch_link(a.chained != 0, prefill_plan_kernel, dim3(v.Hkv), dim3(1024), 0, s, a) != cudaSuccess) return SPKV_E_CUDA;
  // at most max(min(t0,w) + C - w, 0) <= C pairs leave the window
  if (launch_link(a.chained != 0, prefill_scatter_kernel, dim3((C + 63) / 64, v.Hkv), dim3(256), 0, s, a) != cudaSuccess)
    return SPKV_E_CUDA;
  if (d_q) {
    int rc = launch_prefill_stage(a, s);
    if (!rc) rc = launch_prefill_attn_tc5x2h(a, s);
    if (rc) return rc;
  }
  const int n_ring = C < v.w ? C : v.w;
  return check_stream_error(launch_link(a.chained != 0, prefill_ring_kernel, dim3((n_ring + 7) / 8, v.Hkv), dim3(256), 0, s, a));
}
