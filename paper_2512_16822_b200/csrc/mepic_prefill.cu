// Prefill (selective recompute) entry points: placeholder translation unit until the kernel lands.
#include "mepic.h"
#include "mepic_internal.h"

extern "C" size_t mepic_attn_prefill_workspace(const mepic_config_t* cfg, int32_t batch, const int32_t* row_offsets_host) {
  (void)cfg; (void)batch; (void)row_offsets_host;
  mepic_set_error("prefill: not built yet");
  return 0;
}

extern "C" int32_t mepic_attn_prefill(const mepic_config_t* cfg, const mepic_prefill_args_t* args, void* cuda_stream) {
  (void)cfg; (void)args; (void)cuda_stream;
  mepic_set_error("prefill: not built yet");
  return MEPIC_E_INVAL;
}
