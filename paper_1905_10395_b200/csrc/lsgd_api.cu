// Host side of the C ABI: validation, group tables, device state, and the dispatch of each entry
// point to its kernels.  See include/lsgd.h for the contract of every function.
#include <cmath>
#include <cstring>
#include <new>

#include "internal.h"
#include "mlp.h"

using namespace lsgd;

namespace {

constexpr int32_t kMaxWorkers = 4096;  // group tables live in shared memory of the update kernel

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t up256(size_t n) { return (n + 255) & ~size_t(255); }

#define LSGD_CUDA(expr)                          \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return LSGD_ERR_CUDA; \
  } while (0)

lsgd_status validate(const lsgd_config* c) {
  if (!c) return LSGD_ERR_INVALID_ARG;
  if (c->struct_size != sizeof(lsgd_config)) return LSGD_ERR_INVALID_ARG;
  if (c->P < 1 || c->d < 1 || c->ld < c->d || c->tau < 1) return LSGD_ERR_INVALID_ARG;
  if (!std::isfinite(c->eta) || !std::isfinite(c->lambda_l) || !std::isfinite(c->lambda_g)) return LSGD_ERR_INVALID_ARG;
  if (c->G < 1 || c->G > c->P) return LSGD_ERR_BAD_GROUPS;
  if (!c->group_of) return LSGD_ERR_INVALID_ARG;
  {
    std::vector<int32_t> cnt(c->G, 0);
    for (int i = 0; i < c->P; ++i) {
      if (c->group_of[i] < 0 || c->group_of[i] >= c->G) return LSGD_ERR_BAD_GROUPS;
      cnt[c->group_of[i]]++;
    }
    for (int j = 0; j < c->G; ++j)
      if (cnt[j] == 0) return LSGD_ERR_BAD_GROUPS;
  }
  if (c->arithmetic < LSGD_ARITH_FP64 || c->arithmetic > LSGD_ARITH_FP32) return LSGD_ERR_INVALID_ARG;
  if (c->flags & LSGD_FLAG_ALGORITHM1) {
    if (c->tau_g < 1 || !std::isfinite(c->gamma_l) || !std::isfinite(c->gamma_g)) return LSGD_ERR_INVALID_ARG;
    if (!c->leader_copies) return LSGD_ERR_INVALID_ARG;
    if (!aligned16(c->leader_copies)) return LSGD_ERR_ALIGNMENT;
  }
  if (c->flags & LSGD_FLAG_EAGD) {
    if (!c->leader_copies) return LSGD_ERR_INVALID_ARG;
    if (!aligned16(c->leader_copies)) return LSGD_ERR_ALIGNMENT;
    if (c->lambda_g != 0.f) return LSGD_ERR_INVALID_ARG;
    if ((c->flags & (LSGD_FLAG_ALGORITHM1 | LSGD_FLAG_MLP_FUSED_STEP | LSGD_FLAG_MATCOMP_FUSED_STEP)) || c->v)
      return LSGD_ERR_UNSUPPORTED;
  }
  if (c->v) {
    if (!std::isfinite(c->momentum) || !std::isfinite(c->weight_decay)) return LSGD_ERR_INVALID_ARG;
    if (!c->g) return LSGD_ERR_INVALID_ARG;
    if (!aligned16(c->v)) return LSGD_ERR_ALIGNMENT;
    if (c->flags & (LSGD_FLAG_MLP_FUSED_STEP | LSGD_FLAG_ALGORITHM1)) return LSGD_ERR_UNSUPPORTED;
  }
  if (c->P > kMaxWorkers) return LSGD_ERR_UNSUPPORTED;
  // the register-staged pull kernel keeps P + 2 G + 1 table words in shared memory below the 48 KiB default
  if ((int64_t)c->P + 2 * (int64_t)c->G + 2 > 12288) return LSGD_ERR_UNSUPPORTED;
  if (c->ld % 32 != 0) return LSGD_ERR_ALIGNMENT;
  if (!c->x) return LSGD_ERR_INVALID_ARG;
  if (!aligned16(c->x) || !aligned16(c->g)) return LSGD_ERR_ALIGNMENT;
  switch (c->objective) {
    case LSGD_OBJ_EXTERNAL:
      if (!c->g) return LSGD_ERR_INVALID_ARG;
      break;
    case LSGD_OBJ_QUADRATIC: {
      const auto* q = static_cast<const lsgd_quadratic_desc*>(c->objective_desc);
      if (!q || !q->a || !q->b || !std::isfinite(q->sigma)) return LSGD_ERR_INVALID_ARG;
      if (!aligned16(q->a) || !aligned16(q->b)) return LSGD_ERR_ALIGNMENT;
      break;
    }
    case LSGD_OBJ_MATCOMP: {
      const auto* m = static_cast<const lsgd_matcomp_desc*>(c->objective_desc);
      if (!m || !c->g) return LSGD_ERR_INVALID_ARG;
      if (m->n_rows < 1 || m->n_cols < 1 || m->rank < 1 || m->n_obs < 1 || m->batch < 1 || m->n_heldout < 1)
        return LSGD_ERR_INVALID_ARG;
      if (!m->obs_r || !m->obs_c || !m->obs_v || !m->heldout_pos) return LSGD_ERR_INVALID_ARG;
      if ((int64_t)(m->n_rows + (int64_t)m->n_cols) * m->rank != c->d) return LSGD_ERR_INVALID_ARG;
      if (m->rank > 32) return LSGD_ERR_UNSUPPORTED;
      if (m->batch > (1 << 15)) return LSGD_ERR_UNSUPPORTED;   // range of the fixed-point gradient accumulator
      if (m->scratch) {
        if (reinterpret_cast<uintptr_t>(m->scratch) & 255u) return LSGD_ERR_ALIGNMENT;
        if (m->scratch_bytes < lsgd_matcomp_scratch_bytes(c->P, c->ld)) return LSGD_ERR_INVALID_ARG;
      }
      break;
    }
    case LSGD_OBJ_PSD_COMPLETION: {
      const auto* m = static_cast<const lsgd_psd_desc*>(c->objective_desc);
      if (!m || !c->g || !m->M || m->n < 1 || m->r < 1) return LSGD_ERR_INVALID_ARG;
      if ((int64_t)m->n * m->r != c->d) return LSGD_ERR_INVALID_ARG;
      if (m->r > 128) return LSGD_ERR_UNSUPPORTED;
      if (m->scratch) {
        if (reinterpret_cast<uintptr_t>(m->scratch) & 255u) return LSGD_ERR_ALIGNMENT;
        if (m->scratch_bytes < lsgd_psd_scratch_bytes(m->r, c->P, c->ld)) return LSGD_ERR_INVALID_ARG;
      }
      break;
    }
    case LSGD_OBJ_MLP: {
      const auto* m = static_cast<const lsgd_mlp_desc*>(c->objective_desc);
      if (!m || !c->g) return LSGD_ERR_INVALID_ARG;
      lsgd_status st = mlp_validate(*c, *m);
      if (st != LSGD_OK) return st;
      break;
    }
    default:
      return LSGD_ERR_INVALID_ARG;
  }
  return LSGD_OK;
}

lsgd_status algorithm1_pulls(lsgd_ctx* h, bool local, bool glob);

// The handle's buffers, stream and kernel attributes belong to the device that was current at creation.
inline bool on_own_device(const lsgd_ctx* h) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

GroupTables tables(const lsgd_ctx* h) { return GroupTables{h->d_rows_by_group, h->d_group_start, h->d_group_of}; }

}  // namespace

extern "C" {

lsgd_status lsgd_create(const lsgd_config* cfg, lsgd_handle* out) {
  if (out) *out = nullptr;
  if (!out) return LSGD_ERR_INVALID_ARG;
  lsgd_status st = validate(cfg);
  if (st != LSGD_OK) return st;

  lsgd_ctx* h = new (std::nothrow) lsgd_ctx();
  if (!h) return LSGD_ERR_INVALID_ARG;
  h->cfg = *cfg;
  h->group_of.assign(cfg->group_of, cfg->group_of + cfg->P);
  h->cfg.group_of = h->group_of.data();
  h->stream = static_cast<cudaStream_t>(cfg->stream);
  h->t = 0;
  h->n_elections = 0;
  h->grad_ready = false;
  h->eagd_center_ready = false;
  h->fused_applied = false;
  h->mc_step_pending = false;
  h->armed_noise = nullptr;
  h->slab = nullptr;
  h->mlp_state = nullptr;
  h->d_acc64 = nullptr;
  h->d_psd_part = nullptr;
  h->owns_acc64 = false;
  h->owns_psd_part = false;
  std::memset(&h->quad, 0, sizeof(h->quad));
  std::memset(&h->mc, 0, sizeof(h->mc));
  std::memset(&h->mlp, 0, sizeof(h->mlp));
  std::memset(&h->psd, 0, sizeof(h->psd));
  h->loss_partials_valid = false;
  h->n_partials = 0;
  if (cfg->objective == LSGD_OBJ_QUADRATIC) {
    h->quad = *static_cast<const lsgd_quadratic_desc*>(cfg->objective_desc);
    h->n_partials = quadratic_loss_blocks(cfg->d);
  } else if (cfg->objective == LSGD_OBJ_MATCOMP) {
    h->mc = *static_cast<const lsgd_matcomp_desc*>(cfg->objective_desc);
    h->n_partials = matcomp_loss_blocks(h->mc.n_heldout);
  } else if (cfg->objective == LSGD_OBJ_MLP) {
    h->mlp = *static_cast<const lsgd_mlp_desc*>(cfg->objective_desc);
  } else if (cfg->objective == LSGD_OBJ_PSD_COMPLETION) {
    h->psd = *static_cast<const lsgd_psd_desc*>(cfg->objective_desc);
    h->n_partials = psd_loss_blocks(h->psd.n, h->psd.r);
  }
  h->cfg.objective_desc = nullptr;

  if (cudaGetDevice(&h->device) != cudaSuccess) {
    delete h;
    return LSGD_ERR_CUDA;
  }

  // Workers sorted by group (counting sort keeps index order inside a group).
  const int P = cfg->P, G = cfg->G;
  std::vector<int32_t> start(G + 1, 0), rows(P);
  for (int i = 0; i < P; ++i) start[h->group_of[i] + 1]++;
  for (int j = 0; j < G; ++j) start[j + 1] += start[j];
  {
    std::vector<int32_t> fill(start.begin(), start.end() - 1);
    for (int i = 0; i < P; ++i) rows[fill[h->group_of[i]]++] = i;
  }

  // One slab: rows_by_group[P] group_start[G+1] group_of[P] ll[G] gl[1] count_g[P] count_l[P]
  //           status[1] loss[P] group_keys[G] partials[P*n_partials]
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += up256(bytes); return o; };
  const size_t o_rows = take(sizeof(int32_t) * P), o_start = take(sizeof(int32_t) * (G + 1));
  const size_t o_gof = take(sizeof(int32_t) * P), o_ll = take(sizeof(int32_t) * G), o_gl = take(sizeof(int32_t));
  const size_t o_cg = take(sizeof(int32_t) * P), o_cl = take(sizeof(int32_t) * P), o_status = take(sizeof(uint32_t));
  const size_t o_loss = take(sizeof(float) * P), o_keys = take(sizeof(unsigned long long) * G);
  const size_t o_part = take(sizeof(double) * (size_t)P * (size_t)(h->n_partials > 0 ? h->n_partials : 1));
  const size_t o_self = take(sizeof(int32_t));
  const size_t o_shard = take(sizeof(int32_t) * 4);
  if (cudaMalloc(&h->slab, off) != cudaSuccess) {
    delete h;
    return LSGD_ERR_CUDA;
  }
  char* base = static_cast<char*>(h->slab);
  h->d_rows_by_group = reinterpret_cast<int32_t*>(base + o_rows);
  h->d_group_start = reinterpret_cast<int32_t*>(base + o_start);
  h->d_group_of = reinterpret_cast<int32_t*>(base + o_gof);
  h->d_ll = reinterpret_cast<int32_t*>(base + o_ll);
  h->d_gl = reinterpret_cast<int32_t*>(base + o_gl);
  h->d_count_g = reinterpret_cast<int32_t*>(base + o_cg);
  h->d_count_l = reinterpret_cast<int32_t*>(base + o_cl);
  h->d_status = reinterpret_cast<uint32_t*>(base + o_status);
  h->d_loss = reinterpret_cast<float*>(base + o_loss);
  h->d_group_keys = reinterpret_cast<unsigned long long*>(base + o_keys);
  h->d_partials = reinterpret_cast<double*>(base + o_part);
  h->d_selftest = reinterpret_cast<int32_t*>(base + o_self);
  h->d_shard = reinterpret_cast<int32_t*>(base + o_shard);

  bool ok = cudaMemsetAsync(h->slab, 0, off, h->stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(h->d_rows_by_group, rows.data(), sizeof(int32_t) * P, cudaMemcpyHostToDevice, h->stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(h->d_group_start, start.data(), sizeof(int32_t) * (G + 1), cudaMemcpyHostToDevice, h->stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(h->d_group_of, h->group_of.data(), sizeof(int32_t) * P, cudaMemcpyHostToDevice, h->stream) == cudaSuccess;
  // the host vectors die at return: drain the copies now (creation is not on the hot path)
  ok = ok && cudaStreamSynchronize(h->stream) == cudaSuccess;
  if (ok && cfg->objective == LSGD_OBJ_MLP) ok = (mlp_create(h) == LSGD_OK);
  if (ok && cfg->objective == LSGD_OBJ_MATCOMP) {
    const size_t bytes = (size_t)lsgd_matcomp_scratch_bytes(P, cfg->ld);
    if (h->mc.scratch) {
      h->d_acc64 = static_cast<unsigned long long*>(h->mc.scratch);           // the caller's buffer
    } else {
      ok = cudaMalloc(reinterpret_cast<void**>(&h->d_acc64), bytes) == cudaSuccess;
      h->owns_acc64 = ok;
    }
    ok = ok && cudaMemsetAsync(h->d_acc64, 0, bytes, h->stream) == cudaSuccess;
  }
  if (ok && cfg->objective == LSGD_OBJ_PSD_COMPLETION && psd_split(h->psd.r) > 1) {
    if (h->psd.scratch) {
      h->d_psd_part = static_cast<double*>(h->psd.scratch);
    } else {
      ok = cudaMalloc(reinterpret_cast<void**>(&h->d_psd_part), (size_t)lsgd_psd_scratch_bytes(h->psd.r, P, cfg->ld)) == cudaSuccess;
      h->owns_psd_part = ok;
    }
  }
  // EAGD: rows 0 .. G-1 of leader_copies are read (with a zero coefficient) before the library writes them all
  if (ok && (cfg->flags & LSGD_FLAG_EAGD))
    ok = cudaMemsetAsync(cfg->leader_copies, 0, sizeof(float) * (size_t)(G + 1) * (size_t)cfg->ld, h->stream) == cudaSuccess;
  // the gradient kernel of this objective writes columns < d only: clear the padding of g once
  if (ok && cfg->objective == LSGD_OBJ_PSD_COMPLETION && cfg->ld > cfg->d)
    ok = cudaMemsetAsync(cfg->g, 0, sizeof(float) * (size_t)P * (size_t)cfg->ld, h->stream) == cudaSuccess;
  if (!ok) {
    if (h->mlp_state) mlp_destroy(h);
    if (h->owns_acc64) cudaFree(h->d_acc64);
    if (h->owns_psd_part) cudaFree(h->d_psd_part);
    cudaFree(h->slab);
    delete h;
    return LSGD_ERR_CUDA;
  }
  *out = h;
  return LSGD_OK;
}

lsgd_status lsgd_grad(lsgd_handle h, const void* batch) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  if (!on_own_device(h)) return LSGD_ERR_STATE;
  const lsgd_config& c = h->cfg;
  switch (c.objective) {
    case LSGD_OBJ_EXTERNAL:
      break;
    case LSGD_OBJ_QUADRATIC:
      if (batch && !aligned16(batch)) return LSGD_ERR_ALIGNMENT;
      if (c.g) {
        LSGD_CUDA(launch_quadratic_grad(c.x, c.g, h->quad.a, h->quad.b, static_cast<const float*>(batch),
                                        h->quad.sigma, c.P, c.d, c.ld, c.arithmetic != LSGD_ARITH_FP32,
                                        h->stream));
      } else {
        h->armed_noise = static_cast<const float*>(batch);
      }
      break;
    case LSGD_OBJ_MATCOMP: {
      if (!batch) return LSGD_ERR_INVALID_ARG;
      if (h->mc_step_pending) return LSGD_ERR_STATE;   // the previous gradient still waits for its lsgd_step
      MatcompArgs a{h->mc, c.x, c.g, c.ld, c.P, h->d_status};
      const bool fuse = (c.flags & LSGD_FLAG_MATCOMP_FUSED_STEP) && !(c.flags & LSGD_FLAG_ALGORITHM1) && !c.v &&
                        (h->t % c.tau) != 0;
      LSGD_CUDA(launch_matcomp_grad(a, static_cast<const int32_t*>(batch), h->d_acc64, !fuse, h->stream));
      h->mc_step_pending = fuse;
      break;
    }
    case LSGD_OBJ_PSD_COMPLETION:
      LSGD_CUDA(launch_psd_grad(c.x, c.g, h->psd.M, h->psd.n, h->psd.r, c.P, c.ld, h->d_partials, h->n_partials, true,
                                h->d_psd_part, h->stream));
      h->loss_partials_valid = true;
      break;
    case LSGD_OBJ_MLP: {
      if (!batch) return LSGD_ERR_INVALID_ARG;
      if (h->fused_applied) return LSGD_ERR_STATE;   // the pending gradient has already moved W1, W2
      const bool fuse = (h->t % c.tau) != 0 && (c.flags & LSGD_FLAG_MLP_FUSED_STEP) && !(c.flags & LSGD_FLAG_ALGORITHM1);
      lsgd_status st = mlp_grad(h, static_cast<const int32_t*>(batch), fuse);
      if (st != LSGD_OK) return st;
      h->fused_applied = fuse;
      break;
    }
    default:
      return LSGD_ERR_INVALID_ARG;
  }
  h->grad_ready = true;
  return LSGD_OK;
}

// Evaluates the objective's own election loss at the current x and points the election at it.
static lsgd_status own_election_loss(lsgd_ctx* h, ElectArgs& e) {
  const lsgd_config& c = h->cfg;
  e.loss_in = nullptr;
  switch (c.objective) {
    case LSGD_OBJ_QUADRATIC:
      LSGD_CUDA(launch_quadratic_loss_partials(c.x, h->quad.a, h->quad.b, c.P, c.d, c.ld, h->d_partials,
                                               h->n_partials, h->stream));
      e.partials = h->d_partials;
      e.n_partials = h->n_partials;
      e.partial_scale = 0.5;
      return LSGD_OK;
    case LSGD_OBJ_MATCOMP: {
      MatcompArgs a{h->mc, c.x, c.g, c.ld, c.P, h->d_status};
      LSGD_CUDA(launch_matcomp_loss_partials(a, h->d_partials, h->n_partials, h->stream));
      e.partials = h->d_partials;
      e.n_partials = h->n_partials;
      e.partial_scale = 1.0 / (double)h->mc.n_heldout;
      return LSGD_OK;
    }
    case LSGD_OBJ_PSD_COMPLETION:
      if (!h->loss_partials_valid)   // otherwise lsgd_grad has just summed F at this x
        LSGD_CUDA(launch_psd_grad(c.x, c.g, h->psd.M, h->psd.n, h->psd.r, c.P, c.ld, h->d_partials, h->n_partials,
                                  false, h->d_psd_part, h->stream));
      h->loss_partials_valid = true;
      e.partials = h->d_partials;
      e.n_partials = h->n_partials;
      e.partial_scale = 0.25;
      return LSGD_OK;
    case LSGD_OBJ_MLP: {
      lsgd_status st;
      if (h->mlp.loss_window > 0) {
        st = mlp_window_loss(h, h->d_loss);            // running mean of the training losses
      } else {
        if (h->fused_applied) return LSGD_ERR_STATE;   // x is between two steps: no loss at x_t any more
        st = mlp_heldout_loss(h, h->d_loss);
      }
      if (st != LSGD_OK) return st;
      e.loss_in = h->d_loss;
      e.partials = nullptr;
      e.n_partials = 0;
      return LSGD_OK;
    }
    default:
      return LSGD_ERR_INVALID_ARG;  // EXTERNAL has no loss of its own
  }
}

lsgd_status lsgd_elect(lsgd_handle h, const float* loss) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  if (!on_own_device(h)) return LSGD_ERR_STATE;
  const lsgd_config& c = h->cfg;
  ElectArgs e{};
  e.loss_in = loss;
  e.partials = nullptr;
  e.n_partials = 0;
  e.partial_scale = 1.0;
  e.loss_out = h->d_loss;
  e.P = c.P;
  e.G = c.G;
  e.tab = tables(h);
  e.ll = h->d_ll;
  e.gl = h->d_gl;
  e.group_keys = h->d_group_keys;
  e.count_global = h->d_count_g;
  e.count_local = h->d_count_l;
  e.update_local = true;
  e.update_global = true;
  const bool alg1 = (c.flags & LSGD_FLAG_ALGORITHM1) != 0;
  const bool alg1_init = alg1 && h->n_elections == 0;
  if (alg1 && !alg1_init) {
    if (h->t == 0) return LSGD_ERR_STATE;                     // initialisation was already done
    e.update_local = (h->t % c.tau) == 0;
    e.update_global = (h->t % c.tau_g) == 0;
    if (!e.update_local && !e.update_global) return LSGD_ERR_STATE;   // not a communication step
  }
  if (!loss) {
    lsgd_status st = own_election_loss(h, e);
    if (st != LSGD_OK) return st;
  }
  if (alg1 && !alg1_init && !loss && e.update_local && e.update_global) {
    // Algorithm 1, both periods due: the listing determines the global best worker after the local pull,
    // so the objective's loss is evaluated a second time on the pulled parameters.
    e.update_global = false;
    LSGD_CUDA(launch_elect(e, h->stream));
    lsgd_status st = algorithm1_pulls(h, true, false);
    if (st != LSGD_OK) return st;
    st = own_election_loss(h, e);
    if (st != LSGD_OK) return st;
    e.update_local = false;
    e.update_global = true;
    LSGD_CUDA(launch_elect(e, h->stream));
    h->n_elections++;
    return algorithm1_pulls(h, false, true);
  }
  LSGD_CUDA(launch_elect(e, h->stream));
  h->n_elections++;
  if (alg1_init) {
    LSGD_CUDA(launch_leader_copies(c.x, c.leader_copies, h->d_ll, h->d_gl, c.G, 0, c.G + 1, c.d, c.ld, h->stream));
  } else if (alg1) {
    return algorithm1_pulls(h, e.update_local, e.update_global);
  }
  return LSGD_OK;
}

}  // extern "C"

namespace {

UpdateArgs base_update_args(lsgd_ctx* h) {
  const lsgd_config& c = h->cfg;
  UpdateArgs a{};
  a.x = c.x;
  a.g = c.g;
  a.quad = QuadInline{h->quad.a, h->quad.b, h->armed_noise, h->quad.sigma};
  a.x_bf16 = (c.objective == LSGD_OBJ_MLP) ? mlp_weight_shadow(h) : nullptr;
  a.snap = nullptr;
  a.use_g = true;
  a.d = c.d;
  a.ld = c.ld;
  a.P = c.P;
  a.G = c.G;
  a.tab = tables(h);
  a.ll = h->d_ll;
  a.gl = h->d_gl;
  a.k.eta = (double)c.eta;
  a.k.cl = (double)c.eta * (double)c.lambda_l;
  a.k.cg = (double)c.eta * (double)c.lambda_g;
  a.k.sigma = (double)h->quad.sigma;
  a.k.eta_f = c.eta;
  a.k.cl_f = (float)a.k.cl;
  a.k.cg_f = (float)a.k.cg;
  a.k.sigma_f = h->quad.sigma;
  a.k.mu = (double)c.momentum;
  a.k.wd = (double)c.weight_decay;
  a.k.mu_f = c.momentum;
  a.k.wd_f = c.weight_decay;
  a.arith = c.arithmetic;
  a.status = h->d_status;
  a.pull = false;
  a.v = c.v;
  return a;
}

void set_pull_coefficients(UpdateArgs& a, double cl, double cg) {
  a.k.cl = cl;
  a.k.cg = cg;
  a.k.cl_f = (float)cl;
  a.k.cg_f = (float)cg;
}

// Algorithm 1, communication part: pure pulls towards freshly elected leaders, in place.  A leader's
// own pull is zero, so reading the leader rows of x while x is rewritten is exact.
lsgd_status algorithm1_pulls(lsgd_ctx* h, bool local, bool glob) {
  const lsgd_config& c = h->cfg;
  h->loss_partials_valid = false;   // x moves
  if (local) {
    UpdateArgs a = base_update_args(h);
    a.pull = true;
    a.use_g = false;
    set_pull_coefficients(a, (double)c.eta * (double)c.lambda_l, 0.0);
    LSGD_CUDA(launch_update(a, h->stream));
    LSGD_CUDA(launch_leader_copies(c.x, c.leader_copies, h->d_ll, h->d_gl, c.G, 0, c.G, c.d, c.ld, h->stream));
  }
  if (glob) {
    UpdateArgs a = base_update_args(h);
    a.pull = true;
    a.use_g = false;
    set_pull_coefficients(a, 0.0, (double)c.eta * (double)c.lambda_g);
    LSGD_CUDA(launch_update(a, h->stream));
    LSGD_CUDA(launch_leader_copies(c.x, c.leader_copies, h->d_ll, h->d_gl, c.G, c.G, c.G + 1, c.d, c.ld, h->stream));
  }
  return LSGD_OK;
}

}  // namespace

extern "C" lsgd_status lsgd_step(lsgd_handle h) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  if (!on_own_device(h)) return LSGD_ERR_STATE;
  const lsgd_config& c = h->cfg;
  const bool alg1 = (c.flags & LSGD_FLAG_ALGORITHM1) != 0;
  const bool eagd = (c.flags & LSGD_FLAG_EAGD) != 0;
  const bool pull = alg1 ? (c.gamma_l != 0.f || c.gamma_g != 0.f) : (h->t % c.tau) == 0;
  if ((pull || alg1) && !eagd && h->n_elections == 0) return LSGD_ERR_STATE;
  if (c.objective != LSGD_OBJ_EXTERNAL && !h->grad_ready) return LSGD_ERR_STATE;
  UpdateArgs a = base_update_args(h);
  a.pull = pull;
  float* const center = eagd ? c.leader_copies + (size_t)c.G * (size_t)c.ld : nullptr;
  if (eagd && pull) {
    // elastic averaging: the guide point of every worker is the center variable (row G of leader_copies).  The
    // new center is formed from x_t and the old center into row 0 first, the workers then step towards the OLD
    // center, and the new one replaces it afterwards: every right-hand side is taken at time t.
    if (!h->eagd_center_ready) {
      LSGD_CUDA(launch_center(c.x, center, c.P, c.d, c.ld, h->stream));
      h->eagd_center_ready = true;
    }
    const double kk = ((double)c.P * (double)c.eta) * (double)c.lambda_l;
    LSGD_CUDA(launch_eagd_center(c.x, center, c.leader_copies, c.P, c.ld, kk, h->stream));
    a.snap = c.leader_copies;
    set_pull_coefficients(a, 0.0, (double)c.eta * (double)c.lambda_l);
  }
  if (alg1 && pull) {
    // small pulls towards the (stale) copies of the leaders' parameters
    a.snap = c.leader_copies;
    set_pull_coefficients(a, (double)c.eta * ((double)c.gamma_l / (double)c.tau),
                          (double)c.eta * ((double)c.gamma_g / (double)c.tau_g));
  }
  if (h->fused_applied) {
    // W1 and W2 were stepped inside lsgd_grad; finish the biases and the last layer
    int64_t ranges[4][2];
    const int nr = mlp_unfused_ranges(h, ranges);
    for (int r = 0; r < nr; ++r) {
      UpdateArgs b = a;
      b.x = a.x + ranges[r][0];
      b.g = a.g + ranges[r][0];
      b.x_bf16 = a.x_bf16 + ranges[r][0];
      b.d = ranges[r][1];
      LSGD_CUDA(launch_update(b, h->stream));
    }
  } else if (h->mc_step_pending) {
    // plain step straight from the fixed-point gradient sums (only the entries the batch touched move)
    LSGD_CUDA(launch_matcomp_finish_step(h->d_acc64, c.x, c.P, c.ld, (double)c.eta, (int)c.arithmetic, h->stream));
  } else if (a.v) {
    LSGD_CUDA(launch_momentum_update(a, h->stream));
  } else {
    LSGD_CUDA(launch_update(a, h->stream));
  }
  if (eagd && pull)
    LSGD_CUDA(cudaMemcpyAsync(center, c.leader_copies, sizeof(float) * (size_t)c.ld, cudaMemcpyDeviceToDevice, h->stream));
  h->t++;
  h->loss_partials_valid = false;
  h->fused_applied = false;
  h->mc_step_pending = false;
  h->grad_ready = false;
  h->armed_noise = nullptr;
  return LSGD_OK;
}

extern "C" {

lsgd_status lsgd_destroy(lsgd_handle h) {
  if (!h) return LSGD_OK;
  cudaStreamSynchronize(h->stream);
  if (h->mlp_state) mlp_destroy(h);
  if (h->owns_acc64) cudaFree(h->d_acc64);
  if (h->owns_psd_part) cudaFree(h->d_psd_part);
  cudaError_t e = cudaFree(h->slab);
  delete h;
  return e == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}

lsgd_status lsgd_get_leaders(lsgd_handle h, int32_t* local_leaders, int32_t* global_leader) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  if (h->n_elections == 0) return LSGD_ERR_STATE;
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  if (local_leaders) LSGD_CUDA(cudaMemcpy(local_leaders, h->d_ll, sizeof(int32_t) * h->cfg.G, cudaMemcpyDeviceToHost));
  if (global_leader) LSGD_CUDA(cudaMemcpy(global_leader, h->d_gl, sizeof(int32_t), cudaMemcpyDeviceToHost));
  return LSGD_OK;
}

lsgd_status lsgd_set_leaders(lsgd_handle h, const int32_t* local_leaders, int32_t global_leader) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  const lsgd_config& c = h->cfg;
  if (global_leader < -1 || global_leader >= c.P) return LSGD_ERR_BAD_GROUPS;
  if (local_leaders)
    for (int j = 0; j < c.G; ++j)
      if (local_leaders[j] < 0 || local_leaders[j] >= c.P || h->group_of[local_leaders[j]] != j) return LSGD_ERR_BAD_GROUPS;
  if ((!local_leaders || global_leader < 0) && h->n_elections == 0) return LSGD_ERR_STATE;   // nothing to keep yet
  // pageable host memory: the copies are staged before the calls return, so the caller's array may go away
  if (local_leaders)
    LSGD_CUDA(cudaMemcpyAsync(h->d_ll, local_leaders, sizeof(int32_t) * c.G, cudaMemcpyHostToDevice, h->stream));
  if (global_leader >= 0)
    LSGD_CUDA(cudaMemcpyAsync(h->d_gl, &global_leader, sizeof(int32_t), cudaMemcpyHostToDevice, h->stream));
  h->n_elections++;
  return LSGD_OK;
}

lsgd_status lsgd_shard_best_key(lsgd_handle h, int32_t n_own, const int32_t* global_index, int64_t* key_out) {
  if (!h || !global_index || !key_out) return LSGD_ERR_INVALID_ARG;
  if (n_own < 1 || n_own > h->cfg.P) return LSGD_ERR_INVALID_ARG;
  if (h->n_elections == 0) return LSGD_ERR_STATE;                  // no loss vector yet
  if (!on_own_device(h)) return LSGD_ERR_STATE;
  LSGD_CUDA(launch_shard_best_key(h->d_loss, global_index, n_own, reinterpret_cast<unsigned long long*>(key_out), h->d_shard,
                                  h->stream));
  return LSGD_OK;
}

lsgd_status lsgd_shard_pick_global(lsgd_handle h, const int64_t* keys, int32_t world, int32_t my_rank, int32_t guest_row,
                                   int32_t* result) {
  if (!h || !keys || !result) return LSGD_ERR_INVALID_ARG;
  if (world < 1 || my_rank < 0 || my_rank >= world) return LSGD_ERR_INVALID_ARG;
  if (guest_row < 0 || guest_row >= h->cfg.P) return LSGD_ERR_BAD_GROUPS;
  if (h->n_elections == 0) return LSGD_ERR_STATE;
  if (!on_own_device(h)) return LSGD_ERR_STATE;
  LSGD_CUDA(launch_shard_pick_global(reinterpret_cast<const unsigned long long*>(keys), world, my_rank, guest_row, h->d_shard,
                                     h->d_gl, h->d_shard + 1, h->stream));
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  LSGD_CUDA(cudaMemcpy(result, h->d_shard + 1, sizeof(int32_t) * 3, cudaMemcpyDeviceToHost));
  return LSGD_OK;
}

lsgd_status lsgd_get_loss(lsgd_handle h, float* loss) {
  if (!h || !loss) return LSGD_ERR_INVALID_ARG;
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  LSGD_CUDA(cudaMemcpy(loss, h->d_loss, sizeof(float) * h->cfg.P, cudaMemcpyDeviceToHost));
  return LSGD_OK;
}

lsgd_status lsgd_get_train_loss(lsgd_handle h, float* loss) {
  if (!h || !loss) return LSGD_ERR_INVALID_ARG;
  if (h->cfg.objective != LSGD_OBJ_MLP) return LSGD_ERR_UNSUPPORTED;
  // the reduction-partials area (at least P doubles, unused by this objective) receives the P means
  float* tmp = reinterpret_cast<float*>(h->d_partials);
  lsgd_status st = mlp_train_loss(h, tmp);
  if (st != LSGD_OK) return st;
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  LSGD_CUDA(cudaMemcpy(loss, tmp, sizeof(float) * h->cfg.P, cudaMemcpyDeviceToHost));
  return LSGD_OK;
}

lsgd_status lsgd_mlp_get_activations(lsgd_handle h, uint16_t* h1, uint16_t* h2) {
  if (!h || (!h1 && !h2)) return LSGD_ERR_INVALID_ARG;
  if (h->cfg.objective != LSGD_OBJ_MLP) return LSGD_ERR_UNSUPPORTED;
  return mlp_get_activations(h, h1, h2);
}

lsgd_status lsgd_get_step(lsgd_handle h, int64_t* t) {
  if (!h || !t) return LSGD_ERR_INVALID_ARG;
  *t = h->t;
  return LSGD_OK;
}

lsgd_status lsgd_get_leader_counts(lsgd_handle h, int32_t* global_counts, int32_t* local_counts) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  if (global_counts) LSGD_CUDA(cudaMemcpy(global_counts, h->d_count_g, sizeof(int32_t) * h->cfg.P, cudaMemcpyDeviceToHost));
  if (local_counts) LSGD_CUDA(cudaMemcpy(local_counts, h->d_count_l, sizeof(int32_t) * h->cfg.P, cudaMemcpyDeviceToHost));
  return LSGD_OK;
}

lsgd_status lsgd_check_device(lsgd_handle h, uint32_t* flag_out) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  uint32_t f = 0;
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  LSGD_CUDA(cudaMemcpy(&f, h->d_status, sizeof(f), cudaMemcpyDeviceToHost));
  if (f) LSGD_CUDA(cudaMemset(h->d_status, 0, sizeof(f)));
  if (flag_out) *flag_out = f;
  return f ? LSGD_ERR_DEVICE_FLAG : LSGD_OK;
}

lsgd_status lsgd_selftest_wait_timeout(lsgd_handle h, int32_t which, int64_t budget_cycles, int32_t* gave_up) {
  if (!h || !gave_up) return LSGD_ERR_INVALID_ARG;
  if (which < 0 || which > 1) return LSGD_ERR_INVALID_ARG;
  if (budget_cycles < 1 || budget_cycles > 100000000) return LSGD_ERR_INVALID_ARG;   // at most ~50 ms
  if (!on_own_device(h)) return LSGD_ERR_STATE;
  if (which == 0)
    LSGD_CUDA(launch_wait_timeout_selftest(h->d_status, (long long)budget_cycles, h->d_selftest, h->stream));
  else
    LSGD_CUDA(launch_gemm_wait_timeout_selftest(h->d_status, (long long)budget_cycles, h->d_selftest, h->stream));
  LSGD_CUDA(cudaStreamSynchronize(h->stream));
  LSGD_CUDA(cudaMemcpy(gave_up, h->d_selftest, sizeof(int32_t), cudaMemcpyDeviceToHost));
  return LSGD_OK;
}

uint64_t lsgd_matcomp_scratch_bytes(int32_t P, int64_t ld) {
  if (P < 1 || ld < 1) return 0;
  return sizeof(unsigned long long) * (uint64_t)P * (uint64_t)ld;
}

uint64_t lsgd_psd_scratch_bytes(int32_t r, int32_t P, int64_t ld) {
  if (r < 1 || P < 1 || ld < 1 || psd_split(r) <= 1) return 0;
  return sizeof(double) * (uint64_t)psd_split(r) * (uint64_t)P * (uint64_t)ld;
}

lsgd_status lsgd_center(lsgd_handle h, float* center) {
  if (!h || !center) return LSGD_ERR_INVALID_ARG;
  if (!aligned16(center)) return LSGD_ERR_ALIGNMENT;
  LSGD_CUDA(launch_center(h->cfg.x, center, h->cfg.P, h->cfg.d, h->cfg.ld, h->stream));
  return LSGD_OK;
}

lsgd_status lsgd_sync_parameters(lsgd_handle h) {
  if (!h) return LSGD_ERR_INVALID_ARG;
  h->loss_partials_valid = false;
  if (h->cfg.objective == LSGD_OBJ_MLP) return mlp_refresh_shadow(h);
  return LSGD_OK;
}

lsgd_status lsgd_advance_step(lsgd_handle h, int64_t n_steps) {
  if (!h || n_steps < 0) return LSGD_ERR_INVALID_ARG;
  h->t += n_steps;
  h->loss_partials_valid = false;
  return LSGD_OK;
}

lsgd_status lsgd_set_eta(lsgd_handle h, float eta) {
  if (!h || !std::isfinite(eta)) return LSGD_ERR_INVALID_ARG;
  h->cfg.eta = eta;
  return LSGD_OK;
}

const char* lsgd_status_string(lsgd_status s) {
  switch (s) {
    case LSGD_OK: return "ok";
    case LSGD_ERR_INVALID_ARG: return "invalid argument";
    case LSGD_ERR_BAD_GROUPS: return "bad group assignment";
    case LSGD_ERR_ALIGNMENT: return "misaligned pointer or row stride";
    case LSGD_ERR_STATE: return "call order violates the step protocol";
    case LSGD_ERR_CUDA: return "CUDA runtime error";
    case LSGD_ERR_UNSUPPORTED: return "unsupported configuration";
    case LSGD_ERR_DEVICE_FLAG: return "a kernel reported a device-side failure";
    case LSGD_ERR_TOO_LARGE: return "problem exceeds the fixed capacity of this entry point";
  }
  return "unknown status";
}

}  // extern "C"
