// MLP population objective: host orchestration.
#include "mlp.h"

namespace lsgd {

static inline int64_t up32(int64_t n) { return (n + 31) / 32 * 32; }

lsgd_status mlp_validate(const lsgd_config&, const lsgd_mlp_desc&) { return LSGD_ERR_UNSUPPORTED; }
lsgd_status mlp_create(lsgd_ctx*) { return LSGD_ERR_UNSUPPORTED; }
lsgd_status mlp_grad(lsgd_ctx*, const int32_t*) { return LSGD_ERR_UNSUPPORTED; }
lsgd_status mlp_heldout_loss(lsgd_ctx*, float*) { return LSGD_ERR_UNSUPPORTED; }
uint16_t* mlp_weight_shadow(lsgd_ctx*) { return nullptr; }
void mlp_destroy(lsgd_ctx*) {}

}  // namespace lsgd

extern "C" {

lsgd_status lsgd_mlp_param_offsets(const int32_t* dims, int64_t* w_off, int64_t* b_off, int64_t* d_out) {
  if (!dims || !w_off || !b_off || !d_out) return LSGD_ERR_INVALID_ARG;
  int64_t off = 0;
  for (int l = 0; l < LSGD_MLP_MAX_LAYERS; ++l) {
    if (dims[l] < 1 || dims[l + 1] < 1) return LSGD_ERR_INVALID_ARG;
    w_off[l] = off;
    off = lsgd::up32(off + (int64_t)dims[l] * dims[l + 1]);
    b_off[l] = off;
    off = lsgd::up32(off + dims[l + 1]);
  }
  *d_out = off;
  return LSGD_OK;
}

uint64_t lsgd_mlp_scratch_bytes(const int32_t*, int32_t, int32_t, int32_t) { return 0; }

}  // extern "C"
