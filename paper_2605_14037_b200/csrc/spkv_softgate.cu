// Soft-gated whole-sequence forward (the paper's training-time attention; Section "Training",
// Eq. 6, the annealed gate of Eq. 7, and the paragraph "Training Efficiency"): causal attention of
// T queries over T keys in which a key inside the query's window has bias 0 and an earlier key the
// bias log u~_s, u~_s = (1 - alpha) sigma(logit_s) + alpha 1[logit_s >= tau_logit].
//
// No cache is involved.  The call rewrites K and V as 64-key pages in the workspace (the page
// image every attention kernel of this library reads), turns the logits into gate biases in the
// log2 domain once per key, and runs the chunk-attention kernel of spkv_prefill in its soft mode:
// tcgen05 tensor cores, two query heads of a KV head per block, the gate biases of a page's 64
// keys fetched once per page for all 256 query rows of the block and added to the scaled scores
// before the row maximum (the paper's kernel prefetches them once per KV-block column; same idea).
#include "spkv_prefill_common.cuh"

namespace spkv {

// log2 of the (annealed) gate of one key; -inf when the gate is 0.
__device__ inline float gate_log2(float logit, float alpha, float tau_logit) {
  if (alpha == 0.f) {
    // log sigma(l) = -log(1 + e^-l), without forming the sigmoid (finite for every finite l)
    const float ln = logit >= 0.f ? -log1pf(expf(-logit)) : logit - log1pf(expf(logit));
    return ln * 1.4426950408889634f;
  }
  const float u = 1.f / (1.f + expf(-logit));
  const float z = logit >= tau_logit ? 1.f : 0.f;          // Eq. 2, on the float32 logit
  return log2f((1.f - alpha) * u + alpha * z);             // Eq. 7, then Eq. 6
}

// grid (n_stage_pages, Hkv), 64 threads: the gate biases of one page of keys; block (0, kvh) also
// writes the plan header the attention kernel reads (an empty cache, a "chunk" of T pairs).
__global__ void __launch_bounds__(64) softgate_prepare_kernel(PrefillArgs a, float *gate2, float alpha) {
  pdl_chain_link();
  const int kvh = blockIdx.y, s = blockIdx.x * kP + threadIdx.x;
  gate2[((size_t)kvh * a.n_stage_pages + blockIdx.x) * kP + threadIdx.x] =
      s < a.C ? gate_log2(a.logits[(size_t)s * a.c.Hkv + kvh], alpha, a.tau_logit) : 0.f;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    int32_t *hdr = unit_ws(a, kvh);
    hdr[H_T0] = 0; hdr[H_LEN0] = 0; hdr[H_NOLD] = 0; hdr[H_N] = a.C;
    hdr[H_NCOMMIT] = 0; hdr[H_LEN1] = 0; hdr[H_FAIL] = 0; hdr[H_VMAX] = 0;
  }
}

}  // namespace spkv

using namespace spkv;

namespace {
struct SoftWs { size_t off_gate, off_pages, off_split, total; int n_pages; };
bool soft_layout(int T, int Hq, int Hkv, SoftWs *w) {
  if (T < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq / Hkv > kMaxGroup) return false;
  spkv_config_t cfg = {};
  cfg.n_q_heads = Hq;
  cfg.n_kv_heads = Hkv;
  w->n_pages = (T + kP - 1) / kP;
  size_t o = ((size_t)Hkv * kHdrInts * 4 + 1023) / 1024 * 1024;
  w->off_gate = o;  o += ((size_t)Hkv * w->n_pages * kP * 4 + 1023) / 1024 * 1024;
  w->off_pages = o; o += (size_t)Hkv * w->n_pages * kPageBytes;
  w->off_split = o; o += prefill_split_bytes(&cfg, T);
  w->total = o;
  return true;
}
}  // namespace

extern "C" size_t spkv_softgate_workspace_bytes(int32_t T, int32_t n_q_heads, int32_t n_kv_heads) {
  SoftWs w;
  return soft_layout(T, n_q_heads, n_kv_heads, &w) ? w.total : 0;
}

extern "C" int spkv_softgate_forward(int32_t T, int32_t n_q_heads, int32_t n_kv_heads, int32_t window,
                                     const void *d_q, const void *d_k, const void *d_v, const float *d_logits,
                                     float alpha, float tau, float sm_scale, int32_t flags, void *d_out,
                                     float *d_lse_opt, void *d_workspace, size_t workspace_bytes,
                                     int32_t *d_status, spkv_stream_t stream) {
  if (T < 0 || window < 1 || !(alpha >= 0.f && alpha <= 1.f) || tau != tau) return SPKV_E_INVALID;
  if (!(sm_scale > 0.f && sm_scale < INFINITY)) return SPKV_E_INVALID;
  SoftWs w;
  if (T > 0 && !soft_layout(T, n_q_heads, n_kv_heads, &w))
    return (n_q_heads >= 1 && n_kv_heads >= 1 && n_q_heads % n_kv_heads == 0) ? SPKV_E_UNSUPPORTED : SPKV_E_INVALID;
  if (T == 0) return SPKV_OK;
  if (!d_q || !d_k || !d_v || !d_logits || !d_out || !d_status) return SPKV_E_INVALID;
  if (((uintptr_t)d_q | (uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_out) & 15) return SPKV_E_INVALID;
  if (!d_workspace || ((uintptr_t)d_workspace & 255) || workspace_bytes < w.total) return SPKV_E_WORKSPACE;
  char *ws = static_cast<char *>(d_workspace);
  PrefillArgs a = {};
  a.c.L = 1; a.c.S = 1; a.c.Hq = n_q_heads; a.c.Hkv = n_kv_heads; a.c.G = n_q_heads / n_kv_heads;
  a.c.w = window;
  a.c.n_units = n_kv_heads;
  a.c.status = d_status;     // a bounded wait that runs out is recorded here
  a.layer = 0; a.seq = 0; a.C = T;
  a.q = static_cast<const __nv_bfloat16 *>(d_q);
  a.k = static_cast<const __nv_bfloat16 *>(d_k);
  a.v = static_cast<const __nv_bfloat16 *>(d_v);
  a.logits = d_logits;
  a.out = static_cast<__nv_bfloat16 *>(d_out);
  a.tau_logit = tau_to_logit(tau);
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.ws = reinterpret_cast<int32_t *>(ws);
  a.ws_stride = kHdrInts;
  a.stage_pages = reinterpret_cast<__nv_bfloat16 *>(ws + w.off_pages);
  a.n_stage_pages = w.n_pages;
  a.pair_tiles = 0;
  a.n_split = 1;
  a.partials = w.total > w.off_split ? reinterpret_cast<float *>(ws + w.off_split) : nullptr;
  a.force_wide = (flags & SPKV_FLAG_PREFILL_PV_BF16) ? 1 : 0;
  a.soft = 1;
  a.gate2 = reinterpret_cast<const float *>(ws + w.off_gate);
  a.lse = d_lse_opt;
  cudaStream_t s = as_stream(stream);
  a.chained = T < 64;
  int rc = check_stream_error(launch_link(a.chained != 0, softgate_prepare_kernel, dim3(w.n_pages, n_kv_heads), dim3(64), 0, s,
                                          a, reinterpret_cast<float *>(ws + w.off_gate), alpha));
  if (!rc) rc = launch_prefill_stage(a, s);
  if (!rc) rc = launch_prefill_attn_tc5x2h(a, s);
  return rc;
}
