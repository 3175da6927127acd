// Cache lifetime, bookkeeping and read-back (host side + small maintenance kernels).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "spkv_internal.cuh"

namespace spkv {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_stream_error(cudaError_t e) { return e == cudaSuccess ? SPKV_OK : SPKV_E_CUDA; }

// Eq. 2 moved to logit space: u >= tau  <=>  logit >= log(tau / (1 - tau)).
float tau_to_logit(float tau) {
  if (!(tau > 0.0f)) return -INFINITY;
  if (!(tau < 1.0f)) return INFINITY;
  return (float)log((double)tau / (1.0 - (double)tau));
}

static int validate(const spkv_config_t *c) {
  if (!c) return SPKV_E_INVALID;
  if (c->n_layers < 1 || c->max_seqs < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return SPKV_E_INVALID;
  if (c->n_q_heads % c->n_kv_heads) return SPKV_E_INVALID;
  if (c->window < 1 || c->max_context < 1 || c->pool_pages < 0) return SPKV_E_INVALID;
  if (c->head_dim != kD || c->page_tokens != kP) return SPKV_E_UNSUPPORTED;
  if (c->n_q_heads / c->n_kv_heads > kMaxGroup) return SPKV_E_UNSUPPORTED;
  if (c->tau != c->tau || c->sink_tokens < 0) return SPKV_E_INVALID;
  int64_t units = (int64_t)c->n_layers * c->max_seqs * c->n_kv_heads;
  int64_t ring_pages = (c->window + kP - 1) / kP;
  if (units > (1 << 24)) return SPKV_E_INVALID;
  if (units * ring_pages + c->pool_pages > 0x7fffffffLL) return SPKV_E_INVALID;
  if (c->h_local_only && c->n_kv_heads > 64) return SPKV_E_UNSUPPORTED;   // one bit per KV head of a layer
  return SPKV_OK;
}

static void make_layout(const spkv_config_t *c, Layout *l) {
  size_t units = (size_t)c->n_layers * c->max_seqs * c->n_kv_heads;
  size_t ring_pages = (c->window + kP - 1) / kP;
  size_t max_pages = ((size_t)c->max_context + kP - 1) / kP;
  // units of a head declared local-only have no page table
  size_t global_heads = (size_t)c->n_layers * c->n_kv_heads;
  if (c->h_local_only)
    for (size_t i = 0, n = global_heads; i < n; ++i) global_heads -= c->h_local_only[i] ? 1 : 0;
  l->n_table_rows = global_heads * c->max_seqs;
  size_t o = 0;
  int n_can = 0;
  // a region of `bytes` bytes at the current offset, followed by its canary block
  auto region = [&](size_t bytes) {
    const size_t at = o;
    o = align_up(o + bytes, 256);
    l->canary[n_can++] = o;
    o += kCanaryBytes;
    return at;
  };
  l->off_header = region(256);
  l->off_t = region(units * 4);
  l->off_len = region(units * 4);
  l->off_table = region(l->n_table_rows * max_pages * 4);
  l->off_free = region((size_t)c->pool_pages * 4);
  l->off_pos = region((size_t)c->pool_pages * kP * 4);
  l->off_rlogit = region(units * (size_t)c->window * 4);
  l->off_htau = region((size_t)c->n_layers * c->n_kv_heads * 4);
  l->off_sync = region((size_t)c->n_layers * 4 * 8);
  l->off_vmax = region(units * 4);
  l->off_trow = region(units * 4);
  o = align_up(o, 1024);
  l->off_pages = o;  o += (units * ring_pages + (size_t)c->pool_pages) * kPageBytes;
  l->total = o;
}

// What an arena must agree on with a configuration to be attached to: everything that fixes the
// layout (FNV-1a over the fields; tau and flags are run-time settings and may differ).
static uint64_t layout_hash(const spkv_config_t *c) {
  const int64_t f[] = {c->n_layers, c->max_seqs, c->n_q_heads, c->n_kv_heads, c->head_dim, c->window,
                       c->page_tokens, c->max_context, c->pool_pages, c->sink_tokens};
  uint64_t h = 1469598103934665603ULL;
  for (int64_t v : f)
    for (int b = 0; b < 8; ++b) { h ^= (uint64_t)(v >> (8 * b)) & 0xff; h *= 1099511628211ULL; }
  if (c->h_local_only)   // which heads have no page table is part of the layout
    for (int i = 0; i < c->n_layers * c->n_kv_heads; ++i) { h ^= c->h_local_only[i] ? 1 : 0; h *= 1099511628211ULL; }
  return h;
}
constexpr uint32_t kMagic = 0x564B5053u;   // "SPKV"
constexpr uint32_t kLayoutVersion = 3;
constexpr int kHdrMagicWord = 8;            // int32 index of {magic, version, hash lo, hash hi} in the header

// value = NaN clears the override
__global__ void set_head_tau_kernel(float *head_tau, int first, int count, float value) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) head_tau[first + i] = value;
}

// Page-table rows of one layer's units: row = base_row + seq * (global heads of the layer) + rank of
// the head among them; -1 for the units of a local-only head, whose threshold becomes +inf.
__global__ void init_table_rows_kernel(int32_t *table_row, float *head_tau, int layer, int S, int Hkv,
                                       unsigned long long local_mask, int32_t base_row) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= S * Hkv) return;
  const int seq = i / Hkv, h = i % Hkv;
  const bool local = Hkv <= 64 && ((local_mask >> h) & 1ULL);
  const unsigned long long all = Hkv >= 64 ? ~0ULL : ((1ULL << Hkv) - 1ULL);
  const int n_global = Hkv <= 64 ? __popcll(~local_mask & all) : Hkv;
  const int rank = Hkv <= 64 ? __popcll(~local_mask & ((1ULL << h) - 1ULL)) : h;
  table_row[((size_t)layer * S + seq) * Hkv + h] = local ? -1 : base_row + seq * n_global + rank;
  if (local && seq == 0) head_tau[layer * Hkv + h] = INFINITY;
}

__global__ void init_free_stack_kernel(int32_t *stack, int32_t *free_top, int64_t pool_pages,
                                       int64_t first) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0) *free_top = (int32_t)pool_pages;
  // popped from the top: ascending page order for a fresh cache
  if (i < pool_pages) stack[i] = (int32_t)(first + (pool_pages - 1 - i));
}

// One block per (layer, kvh) of the sequence being reset.
__global__ void reset_seq_kernel(CacheView c, int seq) {
  const int layer = blockIdx.x / c.Hkv, kvh = blockIdx.x % c.Hkv;
  const int u = unit_index(c, layer, seq, kvh);
  const int n_pages = (c.len[u] + kP - 1) / kP;
  __shared__ int base;
  if (threadIdx.x == 0) base = n_pages ? atomicAdd(&c.status[1], n_pages) : 0;
  __syncthreads();
  for (int j = threadIdx.x; j < n_pages; j += blockDim.x)   // (n_pages > 0: the unit has a page table)
    c.free_stack[base + j] = unit_table(c, c.table_row[u])[j];
  uint4 *ring = reinterpret_cast<uint4 *>(c.pages + ring_page(c, u, 0) * kPageElems);
  const int n16 = c.ring_pages * (kPageBytes / 16);
  for (int i = threadIdx.x; i < n16; i += blockDim.x) ring[i] = make_uint4(0, 0, 0, 0);
  for (int i = threadIdx.x; i < c.w; i += blockDim.x) c.ring_logit[(size_t)u * c.w + i] = 0.f;
  __syncthreads();
  if (threadIdx.x == 0) { c.len[u] = 0; c.t[u] = 0; c.vmax[u] = 0; }
}

}  // namespace spkv

using namespace spkv;

extern "C" int spkv_arena_bytes(const spkv_config_t *cfg, size_t *out_bytes) {
  int rc = validate(cfg);
  if (rc) return rc;
  if (!out_bytes) return SPKV_E_INVALID;
  Layout l;
  make_layout(cfg, &l);
  *out_bytes = l.total;
  return SPKV_OK;
}

// Host handle over an arena laid out for `cfg` (nothing is enqueued).
static int make_handle(const spkv_config_t *cfg, void *d_arena, const Layout &l, spkv_cache **out) {
  spkv_cache *c = new (std::nothrow) spkv_cache();
  if (!c) return SPKV_E_INVALID;
  c->cfg = *cfg;
  c->layout = l;
  c->arena = d_arena;
  c->tau_logit = tau_to_logit(cfg->tau);
  c->last_kind = kLastOther;
  c->last_layer = -1;
  c->last_stream = nullptr;
  c->ws_toggle = 0;
  c->half_last_layer[0] = c->half_last_layer[1] = -1;
  c->last_decode_items = -1;
  c->last_decode_ws = nullptr;
  c->appends_pending = new (std::nothrow) int[cfg->n_layers]();
  c->local_mask = new (std::nothrow) unsigned long long[cfg->n_layers]();
  if (!c->appends_pending || !c->local_mask) {
    delete[] c->appends_pending; delete[] c->local_mask; delete c;
    return SPKV_E_INVALID;
  }
  if (cfg->h_local_only)
    for (int l2 = 0; l2 < cfg->n_layers; ++l2)
      for (int h = 0; h < cfg->n_kv_heads; ++h)
        if (cfg->h_local_only[l2 * cfg->n_kv_heads + h]) c->local_mask[l2] |= 1ULL << h;
  c->cfg.h_local_only = nullptr;   // the caller's array is read during this call only
  c->host_ready = false;
  c->stack_ready = false;
  c->host_calls = 0;
  char *base = static_cast<char *>(d_arena);
  CacheView &v = c->view;
  v.L = cfg->n_layers; v.S = cfg->max_seqs; v.Hq = cfg->n_q_heads; v.Hkv = cfg->n_kv_heads;
  v.G = cfg->n_q_heads / cfg->n_kv_heads;
  v.w = cfg->window;
  v.n_sink = cfg->sink_tokens;
  v.debug_bounds = (cfg->flags & SPKV_FLAG_DEBUG_BOUNDS) ? 1 : 0;
  v.ring_pages = (cfg->window + kP - 1) / kP;
  v.max_pages = (cfg->max_context + kP - 1) / kP;
  v.n_units = cfg->n_layers * cfg->max_seqs * cfg->n_kv_heads;
  v.pool_pages = cfg->pool_pages;
  v.n_ring_pages_total = (int64_t)v.n_units * v.ring_pages;
  v.status = reinterpret_cast<int32_t *>(base + l.off_header);
  v.t = reinterpret_cast<int32_t *>(base + l.off_t);
  v.len = reinterpret_cast<int32_t *>(base + l.off_len);
  v.table = reinterpret_cast<int32_t *>(base + l.off_table);
  v.free_stack = reinterpret_cast<int32_t *>(base + l.off_free);
  v.pos_pool = reinterpret_cast<int32_t *>(base + l.off_pos);
  v.ring_logit = reinterpret_cast<float *>(base + l.off_rlogit);
  v.head_tau = reinterpret_cast<float *>(base + l.off_htau);
  v.sync_ctr = reinterpret_cast<unsigned long long *>(base + l.off_sync);
  v.vmax = reinterpret_cast<uint32_t *>(base + l.off_vmax);
  v.table_row = reinterpret_cast<int32_t *>(base + l.off_trow);
  v.pages = reinterpret_cast<__nv_bfloat16 *>(base + l.off_pages);
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    delete[] c->appends_pending;
    delete[] c->local_mask;
    delete c;
    return SPKV_E_CUDA;
  }
  c->sm_count = prop.multiProcessorCount;
  *out = c;
  return SPKV_OK;
}

static void free_handle(spkv_cache *c) {
  delete[] c->appends_pending;
  delete[] c->local_mask;
  delete c;
}

extern "C" int spkv_cache_create(const spkv_config_t *cfg, void *d_arena, size_t arena_bytes,
                                 spkv_stream_t stream, spkv_cache_t **out) {
  int rc = validate(cfg);
  if (rc) return rc;
  if (!d_arena || !out || ((uintptr_t)d_arena & 255)) return SPKV_E_INVALID;
  Layout l;
  make_layout(cfg, &l);
  if (arena_bytes < l.total) return SPKV_E_ARENA_TOO_SMALL;
  spkv_cache *c = nullptr;
  rc = make_handle(cfg, d_arena, l, &c);
  if (rc) return rc;
  char *base = static_cast<char *>(d_arena);
  const CacheView &v = c->view;
  cudaStream_t s = as_stream(stream);
  // metadata and ring pages start at zero; pool pages are zeroed when first allocated
  cudaError_t e = cudaMemsetAsync(base, 0, l.off_pages + (size_t)v.n_ring_pages_total * kPageBytes, s);
  for (int i = 0; i < kCanaries && e == cudaSuccess; ++i)
    e = cudaMemsetAsync(base + l.canary[i], kCanaryByte, kCanaryBytes, s);
  if (e == cudaSuccess) {
    // what spkv_cache_attach recognises the arena by (pageable host source: copied before the call returns)
    const uint64_t h = layout_hash(cfg);
    const uint32_t id[4] = {kMagic, kLayoutVersion, (uint32_t)h, (uint32_t)(h >> 32)};
    e = cudaMemcpyAsync(v.status + kHdrMagicWord, id, sizeof id, cudaMemcpyHostToDevice, s);
  }
  if (e == cudaSuccess) {
    const int nh = v.L * v.Hkv;
    set_head_tau_kernel<<<(nh + 255) / 256, 256, 0, s>>>(v.head_tau, 0, nh, NAN);
    // page-table rows in (layer, sequence, KV head) order, local-only heads skipped; such a head
    // also carries the keep-nothing threshold for good
    int32_t base_row = 0;
    for (int l2 = 0; l2 < v.L; ++l2) {
      const unsigned long long m = c->local_mask[l2];
      init_table_rows_kernel<<<(v.S * v.Hkv + 255) / 256, 256, 0, s>>>(v.table_row, v.head_tau, l2, v.S, v.Hkv, m, base_row);
      int n_global = 0;
      for (int h = 0; h < v.Hkv; ++h) n_global += (h < 64 && ((m >> h) & 1ULL)) ? 0 : 1;
      base_row += n_global * v.S;
    }
    e = cudaGetLastError();
  }
  if (e == cudaSuccess && v.pool_pages > 0) {
    int64_t n = v.pool_pages;
    init_free_stack_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(v.free_stack, &c->view.status[1], n,
                                                                      v.n_ring_pages_total);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    free_handle(c);
    return SPKV_E_CUDA;
  }
  *out = c;
  return SPKV_OK;
}

extern "C" int spkv_cache_attach(const spkv_config_t *cfg, void *d_arena, size_t arena_bytes,
                                 spkv_stream_t stream, spkv_cache_t **out) {
  int rc = validate(cfg);
  if (rc) return rc;
  if (!d_arena || !out || ((uintptr_t)d_arena & 255)) return SPKV_E_INVALID;
  Layout l;
  make_layout(cfg, &l);
  if (arena_bytes < l.total) return SPKV_E_ARENA_TOO_SMALL;
  uint32_t id[4] = {0, 0, 0, 0};
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess ||
      cudaMemcpy(id, static_cast<char *>(d_arena) + l.off_header + kHdrMagicWord * 4, sizeof id,
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPKV_E_CUDA;
  const uint64_t h = layout_hash(cfg);
  if (id[0] != kMagic || id[1] != kLayoutVersion || id[2] != (uint32_t)h || id[3] != (uint32_t)(h >> 32))
    return SPKV_E_ATTACH;
  spkv_cache *c = nullptr;
  rc = make_handle(cfg, d_arena, l, &c);
  if (rc) return rc;
  *out = c;
  return SPKV_OK;
}

// ---- checkpoint / rollback of everything a decode or prefill call can change in place ---------
static size_t checkpoint_bytes(const spkv_cache *c) {
  return c->layout.off_pages + (size_t)c->view.n_ring_pages_total * kPageBytes;
}
extern "C" size_t spkv_cache_checkpoint_bytes(const spkv_cache_t *cache) { return cache ? checkpoint_bytes(cache) : 0; }

extern "C" int spkv_cache_checkpoint(spkv_cache_t *cache, void *d_buf, size_t bytes, spkv_stream_t stream) {
  if (!cache || !d_buf) return SPKV_E_INVALID;
  if (bytes < checkpoint_bytes(cache)) return SPKV_E_WORKSPACE;
  cache->last_kind = kLastOther;
  return check_stream_error(
      cudaMemcpyAsync(d_buf, cache->arena, checkpoint_bytes(cache), cudaMemcpyDeviceToDevice, as_stream(stream)));
}

extern "C" int spkv_cache_rollback(spkv_cache_t *cache, const void *d_buf, size_t bytes, spkv_stream_t stream) {
  if (!cache || !d_buf) return SPKV_E_INVALID;
  if (bytes < checkpoint_bytes(cache)) return SPKV_E_WORKSPACE;
  cache->last_kind = kLastOther;
  return check_stream_error(
      cudaMemcpyAsync(cache->arena, d_buf, checkpoint_bytes(cache), cudaMemcpyDeviceToDevice, as_stream(stream)));
}

extern "C" int spkv_note_foreign_work(spkv_cache_t *cache) {
  if (!cache) return SPKV_E_INVALID;
  cache->last_kind = kLastOther;
  return SPKV_OK;
}

extern "C" int spkv_arena_canaries(const spkv_config_t *cfg, size_t *h_offsets, int32_t cap, int32_t *n_out) {
  int rc = validate(cfg);
  if (rc) return rc;
  Layout l;
  make_layout(cfg, &l);
  if (n_out) *n_out = kCanaries;
  for (int i = 0; h_offsets && i < kCanaries && i < cap; ++i) h_offsets[i] = l.canary[i];
  return SPKV_OK;
}

// ---- safe-step budget -----------------------------------------------------------------------
// Worst case over n further steps: every pair that leaves a unit's window is kept.  A unit that has
// received t pairs and keeps len then holds len + e(n) pairs, e(n) = max(t + n - w, 0) - max(t - w, 0),
// and needs ceil((len + e(n)) / 64) - ceil(len / 64) new pages; it must also stay within its page table.
static bool steps_fit(const spkv_config_t *cfg, const int32_t *len, const int32_t *t, int64_t n_units,
                      int64_t pages_free, int64_t n) {
  const int64_t w = cfg->window, max_pages = ((int64_t)cfg->max_context + kP - 1) / kP;
  int64_t need = 0;
  for (int64_t u = 0; u < n_units; ++u) {
    const int64_t ev = std::max<int64_t>(t[u] + n - w, 0) - std::max<int64_t>(t[u] - w, 0);
    const int64_t p0 = ((int64_t)len[u] + kP - 1) / kP, p1 = ((int64_t)len[u] + ev + kP - 1) / kP;
    if (p1 > max_pages) return false;
    need += p1 - p0;
    if (need > pages_free) return false;
  }
  return true;
}

extern "C" int spkv_safe_steps_from_lengths(const spkv_config_t *cfg, const int32_t *h_len, const int32_t *h_t,
                                            int64_t n_units, int64_t pages_free, int64_t *out_steps) {
  int rc = validate(cfg);
  if (rc) return rc;
  if (!h_len || !h_t || !out_steps || n_units < 0 || pages_free < 0) return SPKV_E_INVALID;
  int64_t lo = 0, hi = (int64_t)1 << 31;   // steps_fit(lo) holds (no step needs nothing); find the last n that fits
  if (steps_fit(cfg, h_len, h_t, n_units, pages_free, hi)) { *out_steps = hi; return SPKV_OK; }
  while (hi - lo > 1) {
    const int64_t mid = lo + (hi - lo) / 2;
    if (steps_fit(cfg, h_len, h_t, n_units, pages_free, mid)) lo = mid; else hi = mid;
  }
  *out_steps = lo;
  return SPKV_OK;
}

extern "C" int spkv_safe_steps(spkv_cache_t *cache, const int32_t *h_seq_ids, int32_t B, spkv_stream_t stream,
                               int64_t *out_steps) {
  if (!cache || !out_steps || B < 0 || (B > 0 && !h_seq_ids)) return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  for (int b = 0; b < B; ++b)
    if (h_seq_ids[b] < 0 || h_seq_ids[b] >= v.S) return SPKV_E_INVALID;
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return SPKV_E_CUDA;
  std::vector<int32_t> t(v.n_units), len(v.n_units);
  int32_t hdr[2];
  if (cudaMemcpy(t.data(), v.t, (size_t)v.n_units * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(len.data(), v.len, (size_t)v.n_units * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(hdr, v.status, 8, cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPKV_E_CUDA;
  // the units of the listed sequences (every layer and KV head); B = 0: all sequences
  std::vector<int32_t> sl, st;
  for (int l = 0; l < v.L; ++l)
    for (int b = 0; b < (B ? B : v.S); ++b)
      for (int h = 0; h < v.Hkv; ++h) {
        if (h < 64 && ((cache->local_mask[l] >> h) & 1ULL)) continue;   // a local-only head never needs a page
        const int u = (l * v.S + (B ? h_seq_ids[b] : b)) * v.Hkv + h;
        sl.push_back(len[u]);
        st.push_back(t[u]);
      }
  return spkv_safe_steps_from_lengths(&cache->cfg, sl.data(), st.data(), (int64_t)sl.size(),
                                      hdr[1] > 0 ? hdr[1] : 0, out_steps);
}

extern "C" int spkv_cache_destroy(spkv_cache_t *cache) {
  if (!cache) return SPKV_E_INVALID;
  if (cache->stack_ready) {
    for (int i = 0; i < kStackChunks; ++i) {
      cudaEventDestroy(cache->ev_st_in[i]);
      cudaEventDestroy(cache->ev_st_k[i]);
    }
    cudaEventDestroy(cache->ev_st_start);
    cudaEventDestroy(cache->ev_st_done);
  }
  if (cache->host_ready) {  // host-side objects of the host-buffer pipeline
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(cache->ev_in[i]);
      cudaEventDestroy(cache->ev_k[i]);
      cudaEventDestroy(cache->ev_out[i]);
    }
    cudaStreamDestroy(cache->copy_in);
    cudaStreamDestroy(cache->copy_out);
  }
  free_handle(cache);
  return SPKV_OK;
}

extern "C" int spkv_cache_reset_seq(spkv_cache_t *cache, int32_t seq, spkv_stream_t stream) {
  if (!cache || seq < 0 || seq >= cache->cfg.max_seqs) return SPKV_E_INVALID;
  cache->last_kind = kLastOther;
  reset_seq_kernel<<<cache->view.L * cache->view.Hkv, 256, 0, as_stream(stream)>>>(cache->view, seq);
  return check_stream_error(cudaGetLastError());
}

extern "C" int spkv_set_tau(spkv_cache_t *cache, float tau) {
  if (!cache || tau != tau) return SPKV_E_INVALID;
  cache->cfg.tau = tau;
  cache->tau_logit = tau_to_logit(tau);
  return SPKV_OK;
}

extern "C" int spkv_set_head_tau(spkv_cache_t *cache, int32_t layer, int32_t kv_head, float tau,
                                 spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->view.L || kv_head < -1 || kv_head >= cache->view.Hkv)
    return SPKV_E_INVALID;
  // a head declared local-only at creation has no page table: it stays local-only
  const unsigned long long target = kv_head < 0 ? ~0ULL : (kv_head < 64 ? 1ULL << kv_head : 0ULL);
  if (cache->local_mask[layer] & target) return SPKV_E_INVALID;
  const float value = tau != tau ? NAN : tau_to_logit(tau);
  const int first = layer * cache->view.Hkv + (kv_head < 0 ? 0 : kv_head);
  const int count = kv_head < 0 ? cache->view.Hkv : 1;
  cache->last_kind = kLastOther;
  set_head_tau_kernel<<<1, 256, 0, as_stream(stream)>>>(cache->view.head_tau, first, count, value);
  return check_stream_error(cudaGetLastError());
}

extern "C" float spkv_tau_logit(const spkv_cache_t *cache) { return cache ? cache->tau_logit : NAN; }

extern "C" int spkv_status(spkv_cache_t *cache, spkv_stream_t stream) {
  if (!cache) return SPKV_E_INVALID;
  int32_t st = 0;
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return SPKV_E_CUDA;
  if (cudaMemcpy(&st, cache->view.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPKV_E_CUDA;
  if (st == SPKV_OK && (cache->cfg.flags & SPKV_FLAG_DEBUG_BOUNDS)) {
    // the canary blocks between the metadata regions must still hold their pattern
    unsigned char blk[kCanaryBytes];
    for (int i = 0; i < kCanaries; ++i) {
      if (cudaMemcpy(blk, static_cast<char *>(cache->arena) + cache->layout.canary[i], kCanaryBytes,
                     cudaMemcpyDeviceToHost) != cudaSuccess)
        return SPKV_E_CUDA;
      for (int b = 0; b < kCanaryBytes; ++b)
        if (blk[b] != kCanaryByte) return SPKV_E_CANARY;
    }
  }
  return st;
}

extern "C" int spkv_clear_status(spkv_cache_t *cache, spkv_stream_t stream) {
  if (!cache) return SPKV_E_INVALID;
  return check_stream_error(cudaMemsetAsync(cache->view.status, 0, 4, as_stream(stream)));
}

extern "C" int spkv_read_lengths(spkv_cache_t *cache, int32_t layer, int32_t *h_len, int32_t *h_t,
                                 spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers) return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return SPKV_E_CUDA;
  size_t n = (size_t)v.S * v.Hkv, off = (size_t)layer * n;
  if (h_len && cudaMemcpy(h_len, v.len + off, n * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPKV_E_CUDA;
  if (h_t && cudaMemcpy(h_t, v.t + off, n * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPKV_E_CUDA;
  return SPKV_OK;
}

// Copies one page to the host and undoes the row swizzle for rows [0, n_rows).
static int fetch_page(const CacheView &v, int64_t gpage, int n_rows, uint16_t *tmp, uint16_t *h_k,
                      uint16_t *h_v) {
  if (cudaMemcpy(tmp, v.pages + gpage * kPageElems, kPageBytes, cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPKV_E_CUDA;
  for (int r = 0; r < n_rows; ++r)
    for (int ch = 0; ch < 16; ++ch) {
      if (h_k) memcpy(h_k + (size_t)r * kD + ch * 8, tmp + swz_off(r, ch), 16);
      if (h_v) memcpy(h_v + (size_t)r * kD + ch * 8, tmp + kBlockElems + swz_off(r, ch), 16);
    }
  return SPKV_OK;
}

extern "C" int spkv_read_kept(spkv_cache_t *cache, int32_t layer, int32_t seq, int32_t kvh,
                              int32_t *h_pos, void *h_k, void *h_v, int32_t cap, int32_t *n_out,
                              spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || seq < 0 || seq >= cache->cfg.max_seqs ||
      kvh < 0 || kvh >= cache->cfg.n_kv_heads || cap < 0)
    return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return SPKV_E_CUDA;
  const int u = (layer * v.S + seq) * v.Hkv + kvh;
  int32_t len = 0;
  if (cudaMemcpy(&len, v.len + u, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPKV_E_CUDA;
  if (n_out) *n_out = len;
  int n = len < cap ? len : cap;
  int n_pages = (n + kP - 1) / kP;
  if (n_pages == 0) return SPKV_OK;
  std::vector<int32_t> table(n_pages);
  int32_t trow = -1;
  if (cudaMemcpy(&trow, v.table_row + u, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPKV_E_CUDA;
  if (trow < 0 || (size_t)trow >= cache->layout.n_table_rows) return SPKV_E_INVALID;
  if (cudaMemcpy(table.data(), v.table + (size_t)trow * v.max_pages, (size_t)n_pages * 4,
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPKV_E_CUDA;
  std::vector<uint16_t> tmp(kPageElems);
  for (int j = 0; j < n_pages; ++j) {
    int rows = n - j * kP < kP ? n - j * kP : kP;
    int64_t g = table[j];
    if (g < v.n_ring_pages_total || g >= v.n_ring_pages_total + v.pool_pages) return SPKV_E_INVALID;
    int rc = fetch_page(v, g, rows, tmp.data(),
                        h_k ? (uint16_t *)h_k + (size_t)j * kP * kD : nullptr,
                        h_v ? (uint16_t *)h_v + (size_t)j * kP * kD : nullptr);
    if (rc) return rc;
    if (h_pos && cudaMemcpy(h_pos + (size_t)j * kP, v.pos_pool + (g - v.n_ring_pages_total) * kP,
                            (size_t)rows * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
      return SPKV_E_CUDA;
  }
  return SPKV_OK;
}

extern "C" int spkv_read_window(spkv_cache_t *cache, int32_t layer, int32_t seq, int32_t kvh,
                                int32_t *h_pos, void *h_k, void *h_v, float *h_logits,
                                int32_t *n_out, spkv_stream_t stream) {
  if (!cache || layer < 0 || layer >= cache->cfg.n_layers || seq < 0 || seq >= cache->cfg.max_seqs ||
      kvh < 0 || kvh >= cache->cfg.n_kv_heads)
    return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return SPKV_E_CUDA;
  const int u = (layer * v.S + seq) * v.Hkv + kvh;
  int32_t t = 0;
  if (cudaMemcpy(&t, v.t + u, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPKV_E_CUDA;
  const int n = t < v.w ? t : v.w;
  if (n_out) *n_out = n;
  std::vector<uint16_t> ring((size_t)v.ring_pages * kPageElems);
  std::vector<float> lg(v.w);
  if (cudaMemcpy(ring.data(), v.pages + (int64_t)u * v.ring_pages * kPageElems,
                 ring.size() * 2, cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPKV_E_CUDA;
  if (cudaMemcpy(lg.data(), v.ring_logit + (size_t)u * v.w, (size_t)v.w * 4, cudaMemcpyDeviceToHost) !=
      cudaSuccess)
    return SPKV_E_CUDA;
  for (int j = 0; j < n; ++j) {
    const int s = t - n + j, slot = s % v.w, pg = slot / kP, r = slot % kP;
    const uint16_t *page = ring.data() + (size_t)pg * kPageElems;
    if (h_pos) h_pos[j] = s;
    if (h_logits) h_logits[j] = lg[slot];
    for (int ch = 0; ch < 16; ++ch) {
      if (h_k) memcpy((uint16_t *)h_k + (size_t)j * kD + ch * 8, page + swz_off(r, ch), 16);
      if (h_v) memcpy((uint16_t *)h_v + (size_t)j * kD + ch * 8, page + kBlockElems + swz_off(r, ch), 16);
    }
  }
  return SPKV_OK;
}

extern "C" int spkv_cache_stats(spkv_cache_t *cache, spkv_stream_t stream, spkv_stats_t *out) {
  if (!cache || !out) return SPKV_E_INVALID;
  const CacheView &v = cache->view;
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return SPKV_E_CUDA;
  std::vector<int32_t> t(v.n_units), len(v.n_units);
  std::vector<float> lg((size_t)v.n_units * v.w), htau((size_t)v.L * v.Hkv);
  int32_t hdr[2];
  if (cudaMemcpy(htau.data(), v.head_tau, htau.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(t.data(), v.t, (size_t)v.n_units * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(len.data(), v.len, (size_t)v.n_units * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(lg.data(), v.ring_logit, lg.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(hdr, v.status, 8, cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPKV_E_CUDA;
  memset(out, 0, sizeof *out);
  out->units = v.n_units;
  for (int u = 0; u < v.n_units; ++u) {
    const int nw = t[u] < v.w ? t[u] : v.w;
    out->pairs_seen += t[u];
    out->pairs_kept += len[u];
    out->pairs_in_window += nw;
    out->pairs_evicted += t[u] > v.w ? t[u] - v.w : 0;
    out->pages_in_use += (len[u] + kP - 1) / kP;
    out->gates_open += len[u];
    const float own = htau[(size_t)(u / (v.S * v.Hkv)) * v.Hkv + u % v.Hkv];  // unit = (layer * S + seq) * Hkv + kvh
    const float thr = own != own ? cache->tau_logit : own;
    for (int s = 0; s < nw; ++s)
      if (lg[(size_t)u * v.w + s] >= thr) out->gates_open++;
  }
  out->pages_free = hdr[1];
  out->bytes_resident = (out->pairs_kept + out->pairs_in_window) * 2 * kRowBytes;
  out->density_all = out->pairs_seen ? (double)out->gates_open / (double)out->pairs_seen : 0.0;
  out->density_cache = out->pairs_evicted ? (double)out->pairs_kept / (double)out->pairs_evicted : 0.0;
  return SPKV_OK;
}

extern "C" const char *spkv_error_string(int code) {
  switch (code) {
    case SPKV_OK: return "ok";
    case SPKV_E_INVALID: return "invalid argument";
    case SPKV_E_ARENA_TOO_SMALL: return "arena too small";
    case SPKV_E_UNSUPPORTED: return "unsupported configuration";
    case SPKV_E_CUDA: return "CUDA runtime error";
    case SPKV_E_POOL_EXHAUSTED: return "page pool exhausted";
    case SPKV_E_CONTEXT_OVERFLOW: return "unit page table full";
    case SPKV_E_WORKSPACE: return "workspace missing or too small";
    case SPKV_E_TIMEOUT: return "bounded device wait ran out";
    case SPKV_E_BOUNDS: return "sequence id out of range";
    case SPKV_E_SCRATCH_LIMIT: return "request exceeds the built-in scratch area";
    case SPKV_E_ORDER_DECODE: return "overlap mode: decode launch gave up waiting for its append / workspace";
    case SPKV_E_ORDER_APPEND: return "overlap mode: append gave up waiting for its layer's decode launches";
    case SPKV_E_BOUNDS_PAGE: return "debug bounds: page index outside the pool";
    case SPKV_E_CANARY: return "debug bounds: a canary block between arena regions was overwritten";
    case SPKV_E_ATTACH: return "arena does not hold a cache of this configuration";
    default: return "unknown error";
  }
}
