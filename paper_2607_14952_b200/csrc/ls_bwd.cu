// Replay backward (placeholder until the kernels land).
#include "ls_internal.h"

extern "C" ls_status_t ls_replay_attn_bwd(const ls_pages_t*, const ls_attn_params_t*, const void*, const void*,
                                          const void*, const float*, const float*, const void*, void*, void*,
                                          void*, void*, size_t, int32_t*, void*) {
  return LS_ERR_UNSUPPORTED_SHAPE;
}
