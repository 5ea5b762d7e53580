// MLP population pipeline (forward, backward, held-out loss) -- host-side interface used by the API.
#pragma once
#include "internal.h"

namespace lsgd {

lsgd_status mlp_validate(const lsgd_config& c, const lsgd_mlp_desc& m);
lsgd_status mlp_create(lsgd_ctx* h);
// fuse_sgd: apply the plain step for W1, W2 inside the weight-gradient products (g not written there)
lsgd_status mlp_grad(lsgd_ctx* h, const int32_t* batch_idx, bool fuse_sgd);
// the parameter ranges lsgd_step still has to update after a fused lsgd_grad: {offset, length} pairs
int mlp_unfused_ranges(lsgd_ctx* h, int64_t (*ranges)[2]);
lsgd_status mlp_heldout_loss(lsgd_ctx* h, float* loss);
lsgd_status mlp_window_loss(lsgd_ctx* h, float* loss);  // mean of the recorded minibatch losses (loss_window)
lsgd_status mlp_train_loss(lsgd_ctx* h, float* loss);   // mean minibatch loss of the last lsgd_grad
// stored hidden activations of the last mlp_grad as bf16 bit patterns, HOST [P][B][d1] and [P][B][d2]
lsgd_status mlp_get_activations(lsgd_ctx* h, uint16_t* h1, uint16_t* h2);
lsgd_status mlp_refresh_shadow(lsgd_ctx* h);             // bf16 copy of the weights <- x
uint16_t* mlp_weight_shadow(lsgd_ctx* h);
void mlp_destroy(lsgd_ctx* h);

}  // namespace lsgd
