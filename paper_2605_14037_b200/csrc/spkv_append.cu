// Step 2 of the hot path: fused append + evict (paper, Appendix "Inference Kernels").
//
// One warp owns one unit (layer, sequence, KV head) for the duration of the call, so a
// unit's ring, length, page table and pages have a single writer and no locks are
// needed.  The only atomic is the pop from the shared free-page stack.
//
// Bytes per unit and step: 512 B read (new k, v) + 512 B written to the ring slot, and,
// when the pair leaving the ring is kept, 512 B read back + 512 B written to its page.
#include "spkv_internal.cuh"

namespace spkv {

// Pops a free page (lane 0) and clears its value block, so that rows past a page's
// valid count always hold zeros (the attention kernels multiply them by weight 0).
// Returns the global page index, -1 when the pool is empty, -2 when the index popped from the stack
// failed the debug bounds check (status set already).
__device__ inline int alloc_page(const CacheView &c, int lane) {
  int page = -1;
  if (lane == 0) {
    int top = atomicSub(&c.status[1], 1);
    if (top <= 0) {
      atomicAdd(&c.status[1], 1);
    } else {
      page = checked_page(c, __ldcg(&c.free_stack[top - 1]), -2);
    }
  }
  page = __shfl_sync(0xffffffffu, page, 0);
  if (page >= 0) {
    uint4 *vb = reinterpret_cast<uint4 *>(c.pages + (int64_t)page * kPageElems + kBlockElems);
    for (int i = lane; i < kBlockElems * 2 / 16; i += 32) vb[i] = make_uint4(0, 0, 0, 0);
  }
  return page;
}

// One warp: the append + evict of one unit.
__device__ inline void append_unit(const CacheView &c, int layer, int item, const int32_t *__restrict__ seq_ids, int B,
                                   const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                                   const float *__restrict__ logits, float tau_logit,
                                   const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ W,
                                   const float *__restrict__ bias, int d_in, float *__restrict__ logits_out,
                                   unsigned long long local_mask) {
  const int lane = threadIdx.x & 31;
  if (item >= B * c.Hkv) return;
  const int b = item / c.Hkv, kvh = item % c.Hkv;
  const int seq = seq_ids[b];
  if (seq < 0 || seq >= c.S) {
    if (lane == 0) set_status(c, SPKV_E_BOUNDS);
    return;
  }
  const int u = unit_index(c, layer, seq, kvh);
  // a head declared local-only keeps nothing and has no page table: its utility is never looked
  // at, so it is not computed either (its logit is written as 0)
  const bool local_only = kvh < 64 && ((local_mask >> kvh) & 1ULL);
  // The kernel is a chain of dependent trips to memory, so the loads are issued in three rounds
  // rather than where the control flow first needs them.  Round 1 (above): the sequence id.
  // Round 2, everything that depends on the unit alone: pairs received, kept length, page-table
  // row, the head's own threshold, and the new pair itself.  Metadata is read from L2 (in overlap
  // mode this kernel does not start at a stream-wide synchronisation point, and an SM's L1 is not
  // coherent with other SMs' stores).
  const int t = ldcg_keep(&c.t[u]);
  const int n = ldcg_keep(&c.len[u]);
  const int trow = local_only ? -1 : unit_table_row(c, u);
  const float thr = head_threshold(c, layer, kvh, tau_logit);
  // lanes 0-15 move the key row, lanes 16-31 the value row, one 16-byte chunk each
  const int chunk = lane & 15;
  const int blk = (lane >> 4) * kBlockElems;
  const uint4 new_cell = ((lane < 16 ? k_new : v_new) + (size_t)item * 16)[chunk];
  // fused scoring (Eq. 1, linear predictor): this unit's logit for the new pair
  float new_logit;
  if (local_only) {
    new_logit = 0.f;
    if (x && logits_out && lane == 0) logits_out[item] = 0.f;
  } else if (x) {
    new_logit = warp_dot_bf16(x + (size_t)b * d_in, W + (size_t)kvh * d_in, d_in, lane) + bias[kvh];
    if (logits_out && lane == 0) logits_out[item] = new_logit;
  } else {
    new_logit = logits[item];
  }
  const int slot = t % c.w;
  const int row = slot % kP;
  __nv_bfloat16 *ring = c.pages + ring_page(c, u, slot / kP) * kPageElems;
  uint4 *ring_cell = reinterpret_cast<uint4 *>(ring + blk + swz_off(row, chunk));
  // Round 3, what depends on t and the length: the stored logit of the pair that leaves the window,
  // the pair itself and the page-table entry it would go to (read whether or not it is kept).
  const bool leaves = t >= c.w && trow >= 0;
  const int pj = n / kP, prow = n % kP;
  int32_t *table = unit_table(c, trow >= 0 ? trow : 0);
  const float lg = __ldcg(&c.ring_logit[(size_t)u * c.w + slot]);
  const uint4 evictee = __ldcg(ring_cell);
  const int page_at_tail = (leaves && prow != 0 && pj < c.max_pages) ? ldcg_keep(&table[pj]) : -1;

  if (leaves && (lg >= thr || t - c.w < c.n_sink)) {
    // the pair of position t - w leaves the window and passes the threshold on its stored logit
    // (sink positions are kept regardless)
    int page = -1, err = 0;
    if (pj >= c.max_pages) {
      err = SPKV_E_CONTEXT_OVERFLOW;
    } else if (prow == 0) {
      page = alloc_page(c, lane);
      if (page == -1) err = SPKV_E_POOL_EXHAUSTED;
      else if (page < 0) err = SPKV_E_BOUNDS_PAGE;
      else if (lane == 0) table[pj] = page;
    } else {
      page = checked_page(c, page_at_tail, -2);
      if (page < 0) err = SPKV_E_BOUNDS_PAGE;   // the evicted pair is dropped, as on exhaustion
    }
    if (err) {
      if (lane == 0) set_status(c, err);
    } else {
      __syncwarp();
      __nv_bfloat16 *dst = c.pages + (int64_t)page * kPageElems;
      *reinterpret_cast<uint4 *>(dst + blk + swz_off(prow, chunk)) = evictee;
      // the compact cache's largest |value| (the prefill attention picks its value scale by it)
      const uint32_t vm = __reduce_max_sync(0xffffffffu, lane < 16 ? 0u : chunk_abs_max_bf16(evictee));
      if (lane == 0) {
        c.pos_pool[((int64_t)page - c.n_ring_pages_total) * kP + prow] = t - c.w;
        c.len[u] = n + 1;
        note_vmax(c, u, vm);
      }
    }
  }
  *ring_cell = new_cell;
  if (lane == 0) {
    c.ring_logit[(size_t)u * c.w + slot] = new_logit;
    c.t[u] = t + 1;
  }
}

__global__ void __launch_bounds__(128)
append_evict_kernel(CacheView c, int layer, const int32_t *__restrict__ seq_ids, int B,
                    const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                    const float *__restrict__ logits, float tau_logit,
                    const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ W,
                    const float *__restrict__ bias, int d_in, float *__restrict__ logits_out,
                    int wait_prev, unsigned long long local_mask) {
  // Every block counts itself in before dependents may launch and out when it is done: that is
  // what later kernels that skip griddepcontrol.wait order themselves by.
  if (threadIdx.x == 0) sync_count_start(c, layer, kSyncAppStart);
  // wait_prev = 1: wait for everything earlier on the stream.  wait_prev = 0 (overlap mode; the
  // host passes it only when the launches since the last full wait were hot-path kernels of
  // this cache on other layers): the earlier kernels may still be running, and the only ones
  // this launch shares data with are the decode launches of its own layer, which it waits out.
  // The "started" counter is read BEFORE the block lets dependents launch: the decode launch
  // that follows counts itself into the same counter and waits for this append, so reading it
  // later would make the two wait for each other.
  if (wait_prev) pdl_wait();
  else if (threadIdx.x == 0 && !sync_wait_finished(c, layer, kSyncDecStart)) set_status(c, SPKV_E_ORDER_APPEND);
  __syncthreads();
  pdl_trigger();
  append_unit(c, layer, blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), seq_ids, B, k_new, v_new, logits, tau_logit,
              x, W, bias, d_in, logits_out, local_mask);
  __syncthreads();
  if (threadIdx.x == 0) sync_count_finish(c, layer, kSyncAppFin);
}

// The appends of every layer of a stack step in one launch (spkv_decode_stack): warp g owns unit
// g % items of layer layer0 + g / items.  Inputs and logits are laid out layer after layer, layer0's first.  A plain
// stream-ordered launch: no overlap bookkeeping.
__global__ void __launch_bounds__(128)
append_stack_kernel(CacheView c, StackPreds sp, int layer0, int n_layers, const int32_t *__restrict__ seq_ids, int B,
                    const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                    const __nv_bfloat16 *__restrict__ x, int d_in, float *__restrict__ logits_out, float tau_logit) {
  // the decode launch behind this one is a programmatic dependent launch: let its blocks become
  // resident and run their block-local set-up now (they wait for this grid to complete before they
  // read the cache)
  pdl_trigger();
  const int items = B * c.Hkv;
  const long long g = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int layer = (int)(g / items), item = (int)(g % items);
  if (layer >= n_layers) return;
  append_unit(c, layer0 + layer, item, seq_ids, B, k_new + (size_t)layer * items * 16, v_new + (size_t)layer * items * 16,
              nullptr, tau_logit, x + (size_t)layer * B * d_in, sp.W[layer], sp.bias[layer], d_in,
              logits_out ? logits_out + (size_t)layer * items : nullptr, sp.local_mask[layer]);
}

int launch_append_stack(spkv_cache *cache, const StackPreds &sp, int layer0, int n_layers, const int32_t *d_seq_ids, int B,
                        const void *d_k, const void *d_v, const void *d_x, int d_in, float *d_logits_out,
                        cudaStream_t s) {
  const long long warps = (long long)n_layers * B * cache->view.Hkv;
  const int grid = (int)((warps + 3) / 4);
  append_stack_kernel<<<grid, 128, 0, s>>>(cache->view, sp, layer0, n_layers, d_seq_ids, B, static_cast<const uint4 *>(d_k),
                                           static_cast<const uint4 *>(d_v), static_cast<const __nv_bfloat16 *>(d_x), d_in,
                                           d_logits_out, cache->tau_logit);
  return check_stream_error(cudaGetLastError());
}

}  // namespace spkv

using namespace spkv;

// Records this append as the cache's latest launch and tells whether it has to wait for
// everything before it on the stream.  It need not (overlap mode only) when the previous launch
// was a decode/append of a different layer of this cache on the same stream and no other append
// of this layer is outstanding: the kernel then waits for its own layer's decode launches only.
static int append_must_wait(spkv_cache *cache, int layer, cudaStream_t s) {
  const bool independent = (cache->cfg.flags & SPKV_FLAG_OVERLAP) &&
                           (cache->last_kind == kLastDecode || cache->last_kind == kLastAppend) &&
                           cache->last_layer != layer && cache->last_stream == s &&
                           cache->appends_pending[layer] == 0;
  cache->last_kind = kLastAppend;
  cache->last_layer = layer;
  cache->last_stream = s;
  cache->appends_pending[layer]++;
  return independent ? 0 : 1;
}

// Every launch is a programmatic dependent launch: the blocks may become resident and run their
// block-local prologue while the previous kernel of the stream is still finishing.  Without
// SPKV_FLAG_OVERLAP (and in overlap mode whenever the host cannot vouch for the preceding launches)
// the kernel then executes griddepcontrol.wait before it touches any input or the cache, i.e. it
// is ordered after everything earlier on the stream exactly as a plain launch would be; only the
// launch latency is hidden.  Blocks of two warps: small enough to fit on an SM beside a resident
// decode block (320 threads x 168 registers leave 11.7 K registers), which is what lets the
// append of the next layer run under the decode in overlap mode.
constexpr int kAppendThreads = 64;
template <class... Args>
static int launch_append(spkv_cache *cache, int items, cudaStream_t s, Args... args) {
  const int per = kAppendThreads / 32, grid = (items + per - 1) / per;
  (void)cache;
  return check_stream_error(launch_overlapped(append_evict_kernel, dim3(grid), dim3(kAppendThreads), 0, s, args...));
}

extern "C" int spkv_append_evict(spkv_cache_t *cache, int32_t layer, const int32_t *d_seq_ids,
                                 int32_t B, const void *d_k, const void *d_v,
                                 const float *d_logits, spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || B < 0 || B > cache->cfg.max_seqs)
    return SPKV_E_INVALID;
  if (B == 0) return SPKV_OK;
  if (!d_seq_ids || !d_k || !d_v || !d_logits) return SPKV_E_INVALID;
  if (((uintptr_t)d_k | (uintptr_t)d_v) & 15) return SPKV_E_INVALID;
  const int items = B * cache->view.Hkv;
  const int wait_prev = append_must_wait(cache, layer, as_stream(stream));
  return launch_append(cache, items, as_stream(stream), cache->view, layer, d_seq_ids, B,
                       static_cast<const uint4 *>(d_k), static_cast<const uint4 *>(d_v), d_logits,
                       cache->tau_logit, (const __nv_bfloat16 *)nullptr, (const __nv_bfloat16 *)nullptr,
                       (const float *)nullptr, 0, (float *)nullptr, wait_prev, cache->local_mask[layer]);
}

extern "C" int spkv_score_append_evict(spkv_cache_t *cache, int32_t layer, const spkv_predictor_t *pred,
                                       const int32_t *d_seq_ids, int32_t B, const void *d_x,
                                       const void *d_k, const void *d_v, float *d_logits_out,
                                       spkv_stream_t stream) {
  if (!cache || !pred || layer < 0 || layer >= cache->cfg.n_layers || B < 0 || B > cache->cfg.max_seqs)
    return SPKV_E_INVALID;
  if (B == 0) return SPKV_OK;
  if (!d_seq_ids || !d_x || !d_k || !d_v) return SPKV_E_INVALID;
  if (pred->kind != 0) {
    // two-layer predictor: the hidden layer is shared by the KV heads, so it is scored by
    // its own kernel first
    if (!d_logits_out) return SPKV_E_INVALID;
    int rc = spkv_score(cache, pred, d_x, B, d_logits_out, nullptr, stream);
    if (rc) return rc;
    cache->last_kind = kLastOther;
    return spkv_append_evict(cache, layer, d_seq_ids, B, d_k, d_v, d_logits_out, stream);
  }
  if (!pred->d_W1 || !pred->d_b1 || pred->d_in < 8 || (pred->d_in & 7)) return SPKV_E_INVALID;
  if (((uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_x | (uintptr_t)pred->d_W1) & 15) return SPKV_E_INVALID;
  const int items = B * cache->view.Hkv;
  const int wait_prev = append_must_wait(cache, layer, as_stream(stream));
  return launch_append(cache, items, as_stream(stream), cache->view, layer, d_seq_ids, B,
                       static_cast<const uint4 *>(d_k), static_cast<const uint4 *>(d_v), (const float *)nullptr,
                       cache->tau_logit, static_cast<const __nv_bfloat16 *>(d_x),
                       static_cast<const __nv_bfloat16 *>(pred->d_W1), pred->d_b1, pred->d_in, d_logits_out,
                       wait_prev, cache->local_mask[layer]);
}
