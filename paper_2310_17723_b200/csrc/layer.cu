// hero_layer_forward (Sec. 2.2.2-2.2.3, Table 1) -- under construction.
#include "common.cuh"
extern "C" hero_status hero_layer_workspace_bytes(const hero_layer_desc* d, int64_t M, size_t* bytes) {
  (void)d; (void)M; (void)bytes;
  hero::set_error("hero_layer_workspace_bytes: not built yet");
  return HERO_ERR_UNSUPPORTED;
}
extern "C" hero_status hero_layer_forward(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in,
                                          const hero_tensor* pending, const hero_tensor* out, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  (void)h; (void)d; (void)in; (void)pending; (void)out; (void)workspace; (void)workspace_bytes; (void)stream;
  hero::set_error("hero_layer_forward: not built yet");
  return HERO_ERR_UNSUPPORTED;
}
