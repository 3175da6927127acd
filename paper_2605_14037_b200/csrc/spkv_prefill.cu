// Companion path: chunked prefill (placeholder until the kernels land).
#include "spkv_internal.cuh"

extern "C" size_t spkv_prefill_workspace_bytes(const spkv_config_t *cfg, int32_t C) {
  (void)cfg; (void)C;
  return 256;
}

extern "C" int spkv_prefill(spkv_cache_t *, int32_t, int32_t, int32_t, const void *, const void *,
                            const void *, const float *, void *, float, void *, size_t,
                            spkv_stream_t) {
  return SPKV_E_UNSUPPORTED;
}
