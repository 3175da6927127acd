// Internal declarations shared by the translation units of libspkv.so.
//
// Arena layout (all offsets 256-byte aligned, computed by spkv_layout()):
//   header      : status word, free-page counter, magic + layout version + configuration hash
//   (every metadata region is followed by a 256-byte canary block of 0xC5 bytes)
//   t[]         : pairs received per unit                       int32 [n_units]
//   len[]       : kept pairs per unit                           int32 [n_units]
//   table[]     : page table per unit that can keep pairs        int32 [rows][max_pages]
//                 (units of heads declared local-only at creation have none)
//   free_stack[]: LIFO of free pool pages (global page indices) int32 [pool_pages]
//   pos_pool[]  : position of every kept pair, by pool page     int32 [pool_pages][P]
//   ring_logit[]: stored logit per ring slot                    f32   [n_units][w]
//   head_tau[]  : per-(layer, KV head) threshold override       f32   [L][Hkv]  (NaN: none)
//   vmax[]      : largest finite |value| in a unit's compact cache u32 [n_units] (fp32 bit pattern)
//   sync_ctr[]  : blocks started / finished per layer and kernel u64   [L][4]    (launch overlap)
//   table_row[] : row of a unit in table[], -1 = none            int32 [n_units]
//   pages       : ring pages of every unit ([n_units][ring_pages]) followed by the pool
//
// A page holds P = 64 pairs: a 16 KB key block followed by a 16 KB value block.  Each
// block is two 8 KB slabs (dims 0-63, dims 64-127) of 64 rows x 128 B, one row per pair;
// inside a row the eight 16-byte chunks are XOR-swizzled by the row number,
// chunk' = chunk ^ (row & 7) -- the 128-byte-swizzle operand layout of the tensor cores.
// The page in HBM is exactly the shared-memory image the attention kernels want: one
// linear bulk copy brings it in, `ldmatrix` reads it without bank conflicts, and
// tcgen05.mma can take a slab as a K-major (keys) or MN-major (values) operand as it is.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/spkv.h"

namespace spkv {

constexpr int kD = 128;            // head_dim
constexpr int kP = 64;             // pairs per page
constexpr int kRowBytes = kD * 2;  // 256
constexpr int kBlockElems = kP * kD;        // bf16 elements in a key (or value) block
constexpr int kPageElems = 2 * kBlockElems; // 16384 elements = 32 KB
constexpr int kPageBytes = kPageElems * 2;
constexpr int kMaxGroup = 16;      // query heads per KV head supported by the kernels
constexpr int kStackChunks = 4;    // most chunks spkv_decode_stack_host cuts the layer stack into

struct CacheView {
  int32_t L, S, Hq, Hkv, G, w, ring_pages, max_pages, n_units;
  int32_t n_sink;       // positions < n_sink are kept whatever their logit (sink tokens)
  int32_t debug_bounds; // SPKV_FLAG_DEBUG_BOUNDS: page indices read from tables are range-checked
  int64_t pool_pages, n_ring_pages_total;
  int32_t *status;      // [0] sticky status, [1] free_top
  int32_t *t;
  int32_t *len;
  int32_t *table;       // [table rows][max_pages]: a row per unit that can keep pairs
  int32_t *table_row;   // [n_units]: the unit's row in `table`, -1 for a unit of a local-only head
  int32_t *free_stack;
  int32_t *pos_pool;
  float *ring_logit;
  float *head_tau;      // [L][Hkv] logit-space threshold of a (layer, KV head); NaN = the cache-wide one
  unsigned long long *sync_ctr;  // [L][4]: append blocks started, finished; decode blocks started, finished
  // [n_units] bit pattern of the largest finite |v| among the pairs the unit's compact cache holds
  // (raised when a pair is kept, cleared when the sequence is reset).  The prefill attention
  // multiplies P.V in fp16 after scaling the values by a power of two; it takes that factor from
  // the largest |v| its queries can see: this word, the ring and the chunk.
  uint32_t *vmax;
  __nv_bfloat16 *pages;
};

constexpr int kCanaries = 11;          // one 256-byte block after each metadata region
constexpr int kCanaryBytes = 256;
constexpr unsigned char kCanaryByte = 0xC5;
struct Layout {
  size_t off_header, off_t, off_len, off_table, off_free, off_pos, off_rlogit, off_htau, off_sync, off_vmax, off_trow,
      off_pages, total;
  size_t n_table_rows;
  size_t canary[kCanaries];
};

// largest finite |x| among the eight bf16 of a 16-byte chunk, as the upper half of an fp32 bit
// pattern (infinities and NaNs do not count: they come out of the attention as they went in)
__device__ inline uint32_t chunk_abs_max_bf16(const uint4 &v) {
  uint32_t m = 0;
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t a = w[i] & 0x7fffu, b = (w[i] >> 16) & 0x7fffu;
    m = max(m, a < 0x7f80u ? a : 0u);
    m = max(m, b < 0x7f80u ? b : 0u);
  }
  return m << 16;
}
// one thread; the result is not used, so this is a fire-and-forget reduction
__device__ inline void note_vmax(const CacheView &c, int u, uint32_t m) {
  if (m) atomicMax(&c.vmax[u], m);
}

// element offset of (row, 16-byte chunk) inside a key or value block
__host__ __device__ inline int swz_off(int row, int chunk) {
  return (chunk >> 3) * (kP * 64) + row * 64 + (((chunk & 7) ^ (row & 7)) << 3);
}

__device__ inline int unit_index(const CacheView &c, int layer, int seq, int kvh) {
  return (layer * c.S + seq) * c.Hkv + kvh;
}

__device__ inline void set_status(const CacheView &c, int code) { atomicCAS(c.status, 0, code); }

// ---- SPKV_FLAG_DEBUG_BOUNDS: page indices that come out of memory (page tables, free stack) ----
__device__ inline bool pool_page_ok(const CacheView &c, int page) {
  return (int64_t)page >= c.n_ring_pages_total && (int64_t)page < c.n_ring_pages_total + c.pool_pages;
}
// `page` if the check is off or the index names a pool page; otherwise the violation is recorded
// in the status word and `fallback` is returned (a page that is safe to read, or -1 = skip)
__device__ inline int checked_page(const CacheView &c, int page, int fallback) {
  if (!c.debug_bounds || pool_page_ok(c, page)) return page;
  set_status(c, SPKV_E_BOUNDS_PAGE);
  return fallback;
}

// threshold in force for a (layer, KV head): its own if one was set, else the cache-wide one
__device__ inline float head_threshold(const CacheView &c, int layer, int kvh, float tau_logit) {
  const float own = __ldcg(&c.head_tau[layer * c.Hkv + kvh]);
  return own != own ? tau_logit : own;
}

// page table of a unit (the caller knows the unit has one: row >= 0)
__device__ inline int32_t *unit_table(const CacheView &c, int row) { return c.table + (size_t)row * c.max_pages; }
// 32-bit load that bypasses L1 (an SM's L1 is not coherent with other SMs' stores) and asks L2 to
// keep the line: for the metadata every step reads again (lengths, page tables), which the
// streaming reads of keys and values -- issued with the opposite hint -- would otherwise push out.
__device__ inline int ldcg_keep(const int *p) {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  int v;
  asm volatile("ld.global.cg.L2::cache_hint.b32 %0, [%1], %2;" : "=r"(v) : "l"(p), "l"(pol) : "memory");
  return v;
}
__device__ inline int unit_table_row(const CacheView &c, int u) { return ldcg_keep(&c.table_row[u]); }

// global page index of ring page j of a unit
__device__ inline int64_t ring_page(const CacheView &c, int unit, int j) {
  return (int64_t)unit * c.ring_pages + j;
}

// ---- dot product used by the utility predictor (fixed summation order: the logit of a
// token is bit-identical whichever kernel computes it) -------------------------------------
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// <a, b> over d elements (d % 8 == 0), a and b bf16, one warp, 16-byte loads.
__device__ inline float warp_dot_bf16(const __nv_bfloat16 *a, const __nv_bfloat16 *b, int d, int lane) {
  float acc = 0.f;
  for (int i = lane * 8; i < d; i += 256) {
    const uint4 av = *reinterpret_cast<const uint4 *>(a + i);
    const uint4 bv = *reinterpret_cast<const uint4 *>(b + i);
    const __nv_bfloat162 *a2 = reinterpret_cast<const __nv_bfloat162 *>(&av);
    const __nv_bfloat162 *b2 = reinterpret_cast<const __nv_bfloat162 *>(&bv);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 fa = __bfloat1622float2(a2[j]), fb = __bfloat1622float2(b2[j]);
      acc = fmaf(fa.x, fb.x, acc);
      acc = fmaf(fa.y, fb.y, acc);
    }
  }
  return warp_sum(acc);
}

// ---- programmatic dependent launch ---------------------------------------------------------
// Kernels launched with launch_overlapped() may begin while the previous kernel of the stream
// is still running, once all of its blocks have executed pdl_trigger() (or exited).
// pdl_wait() blocks until that previous kernel has completed and its writes are visible.
__device__ inline void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ inline void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <class... KArgs, class... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// First statement of a kernel that is one link of a chain of dependent launches (the prefill
// call's kernels): lets the next kernel of the stream be scheduled as soon as every block of
// this one has started, and then waits until the previous kernel has completed and its writes
// are visible.  Ordering is that of plain launches; what is gained is the launch latency of every
// link: a chunk of 1-16 tokens on a 32 K past takes 71-78 us instead of 80-88.  Chunks of 128
// tokens and more measured 7-8 % SLOWER chained (their kernels run long enough to hide the launch
// latency by themselves), so the host chains small chunks only.
__device__ inline void pdl_chain_link() {
  pdl_trigger();
  pdl_wait();
}

// A link of such a chain when `chained`, a plain launch otherwise (pdl_chain_link is then a no-op).
template <class... KArgs, class... Args>
inline cudaError_t launch_link(bool chained, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                               cudaStream_t stream, Args... args) {
  if (chained) return launch_overlapped(kernel, grid, block, smem, stream, args...);
  kernel<<<grid, block, smem, stream>>>(KArgs(args)...);
  return cudaGetLastError();
}

enum { kLastOther = 0, kLastAppend = 1, kLastDecode = 2 };

// ---- launch overlap without griddepcontrol.wait ---------------------------------------------
// griddepcontrol.wait returns only when EVERY earlier kernel of the stream has completed, so a
// kernel that calls it cannot begin its real work under the tail of its predecessor.  In overlap
// mode (SPKV_FLAG_OVERLAP) the hot-path kernels skip it where the host knows what the preceding
// launches were, and order themselves by the data they actually share: every block counts
// itself into "started" before it lets dependents launch and into "finished" (release) when it
// is done.  A later kernel is launched only after all blocks of all earlier kernels of the
// stream have started (each launch needs its predecessor's blocks to have triggered), so when
// it reads "started" that number is final, and "finished >= started" (acquire) means those
// kernels are done.  A block must read "started" BEFORE it lets dependents launch: a dependent
// may count itself into the very counter being read and wait for this kernel in turn, and the
// two would then wait for each other.  Nothing here depends on values the host passes per
// launch: a captured CUDA graph replays correctly.  The spin is bounded; on expiry the status
// word is set.
enum { kSyncAppStart = 0, kSyncAppFin = 1, kSyncDecStart = 2, kSyncDecFin = 3 };

__device__ inline void sync_count_start(const CacheView &c, int layer, int which) {  // one thread per block
  atomicAdd(&c.sync_ctr[layer * 4 + which], 1ULL);
  __threadfence();
}
__device__ inline void sync_count_finish(const CacheView &c, int layer, int which) {  // one thread, after a block barrier
  asm volatile("red.release.gpu.global.add.u64 [%0], 1;" ::"l"(&c.sync_ctr[layer * 4 + which]) : "memory");
}
// true when every block counted in "started" has also finished, for up to two (layer, kernel)
// pairs at once (layer_b < 0: only the first).  One thread per block calls; all four counters
// are fetched together (relaxed loads, one fence at the end), so the common case -- already
// satisfied -- costs one trip to L2.
__device__ inline unsigned long long sync_load(const unsigned long long *p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ inline bool sync_wait_finished(const CacheView &c, int layer_a, int which_a, int layer_b = -1,
                                          int which_b = 0) {
  const unsigned long long *pa = &c.sync_ctr[layer_a * 4 + which_a];
  const unsigned long long *pb = layer_b >= 0 ? &c.sync_ctr[layer_b * 4 + which_b] : pa;
  const unsigned long long sa = sync_load(pa), sb = sync_load(pb);
  unsigned long long fa = sync_load(pa + 1), fb = sync_load(pb + 1);
  const long long t0 = clock64();
  while (fa < sa || fb < sb) {
    if (clock64() - t0 > (1LL << 31)) return false;
    __nanosleep(64);
    fa = sync_load(pa + 1);
    fb = sync_load(pb + 1);
  }
  __threadfence();  // acquire: what those blocks wrote before counting themselves out is visible now
  return true;
}

}  // namespace spkv

struct spkv_cache {
  spkv_config_t cfg;
  spkv::CacheView view;
  spkv::Layout layout;
  void *arena;
  float tau_logit;
  int sm_count;
  // what the previous launch on this cache was (decides whether an append may overlap it)
  int last_kind;        // 0 other, 1 append, 2 decode
  int last_layer;
  cudaStream_t last_stream;
  int ws_toggle;        // decode workspace half used by the next decode launch
  int half_last_layer[2];   // layer of the decode launch that last used each workspace half (-1: none)
  int last_decode_items;    // units of the previous decode launch (the workspace halves depend on it)
  void *last_decode_ws;     // and its workspace
  int *appends_pending;     // [n_layers] appends since the layer's last decode launch
  unsigned long long *local_mask;   // [n_layers] bit h set: KV head h of the layer was declared local-only
  // spkv_decode_step_host: copy streams and events of its two-slot pipeline (made on first use)
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_in[2], ev_k[2], ev_out[2];   // per slot: inputs landed, kernels done, output landed
  long long host_calls;                        // calls so far; slot = call & 1
  bool host_ready;
  // spkv_decode_stack_host: per chunk of layers, inputs landed / kernels done; start and end of a call
  cudaEvent_t ev_st_in[spkv::kStackChunks], ev_st_k[spkv::kStackChunks], ev_st_start, ev_st_done;
  bool stack_ready;
};

namespace spkv {
int check_stream_error(cudaError_t e);
inline cudaStream_t as_stream(spkv_stream_t s) { return reinterpret_cast<cudaStream_t>(s); }
float tau_to_logit(float tau);
// per-layer linear predictors and local-only masks of a stack step, passed to kernels by value
constexpr int kMaxStackLayers = 128;
struct StackPreds {
  const __nv_bfloat16 *W[kMaxStackLayers];
  const float *bias[kMaxStackLayers];
  unsigned long long local_mask[kMaxStackLayers];
};
int launch_append_stack(spkv_cache *cache, const StackPreds &sp, int layer0, int n_layers, const int32_t *d_seq_ids, int B,
                        const void *d_k, const void *d_v, const void *d_x, int d_in, float *d_logits_out,
                        cudaStream_t s);
int decode_stack_layers(spkv_cache *cache, int l0, int l1, const spkv_predictor_t *preds, const int32_t *d_seq_ids,
                        int32_t B, const void *d_x, const void *d_q, const void *d_k, const void *d_v, void *d_out,
                        float *d_logits_out, float *d_lse_opt, float sm_scale, void *d_workspace, size_t workspace_bytes,
                        spkv_stream_t stream);
int launch_score_mlp_tc(spkv_cache *cache, const spkv_predictor_t *p, const void *d_x, int n_tok, float *d_logits,
                        uint8_t *d_flags, cudaStream_t s);
}  // namespace spkv
