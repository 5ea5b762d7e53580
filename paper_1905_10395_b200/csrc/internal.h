// Internal declarations shared by the host API and the kernel launchers.  Not installed.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>
#include <vector>

#include "lsgd.h"

namespace lsgd {

// Status-word bits set by kernels (reported as LSGD_ERR_DEVICE_FLAG).
enum : uint32_t {
  FLAG_BAD_LEADER = LSGD_DEVFLAG_BAD_LEADER,     // a leader index outside [0, P) reached the update kernel
  FLAG_WAIT_TIMEOUT = LSGD_DEVFLAG_WAIT_TIMEOUT, // a bounded mbarrier / tensor-pipe wait ran out
  FLAG_BAD_INDEX = LSGD_DEVFLAG_BAD_INDEX,       // a batch position / sample index out of range (entry skipped)
  FLAG_OVERFLOW = LSGD_DEVFLAG_OVERFLOW,         // a contribution outside the fixed-point accumulator's range (skipped)
};

// One-time launch state is per DEVICE, not per process: a kernel's dynamic-shared-memory attribute applies to
// the device that was current when it was set, and devices need not have the same number of SMs.
constexpr int kMaxDevices = 64;
inline int device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  return dev;
}
struct OncePerDevice {
  bool done[kMaxDevices] = {};
  bool& here() { return done[device_slot()]; }
};
inline int sm_count() {
  static int sms[kMaxDevices] = {};
  const int dev = device_slot();
  if (sms[dev] == 0) {
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    sms[dev] = n > 0 ? n : 148;
  }
  return sms[dev];
}

struct GroupTables {
  // Workers sorted by group: members of group j are rows_by_group[group_start[j] .. group_start[j+1]).
  const int32_t* rows_by_group;  // DEVICE int32[P]
  const int32_t* group_start;    // DEVICE int32[G+1]
  const int32_t* group_of;       // DEVICE int32[P]
};

// Inline gradient of the diagonal quadratic inside the update kernel (g never touches memory).
struct QuadInline {
  const float* a;      // DEVICE [ld]
  const float* b;      // DEVICE [ld]
  const float* noise;  // DEVICE [P*ld] or nullptr
  float sigma;
};

// Step coefficients in both precisions: eta, eta*lambda_l, eta*lambda_g, sigma.
struct Coef {
  double eta, cl, cg, sigma;
  float eta_f, cl_f, cg_f, sigma_f;
  double mu, wd;            // Nesterov momentum and weight decay (momentum kernel only)
  float mu_f, wd_f;
};

struct UpdateArgs {
  float* x;
  const float* g;           // nullptr => use quad
  QuadInline quad;
  uint16_t* x_bf16;         // optional bf16 shadow of x, same [P][ld] layout (nullptr = none)
  int64_t d, ld;
  int32_t P, G;
  GroupTables tab;
  const int32_t* ll;        // DEVICE int32[G]
  const int32_t* gl;        // DEVICE int32[1]
  const float* snap;        // leaders' parameters as copies [(G+1)][ld] (rows 0..G-1 local, G global), or
                            // nullptr = read the leader rows of x itself (staged before anything is written)
  bool use_g;               // false: pure pull, the gradient term is dropped (g / noise are not read)
  Coef k;
  int arith;                // 0 fp64 unfused, 1 fp64 fma, 2 fp32 fma (see update.cu)
  uint32_t* status;
  bool pull;
  float* v;                 // momentum buffers [P][ld], or nullptr = the step of Eq. (1)
};
cudaError_t launch_update(const UpdateArgs& a, cudaStream_t s);
// Section 4.1 optimiser (a.v != nullptr): Nesterov momentum + weight decay around the same step.
cudaError_t launch_momentum_update(const UpdateArgs& a, cudaStream_t s);
cudaError_t launch_momentum_update_chunked(const UpdateArgs& a, cudaStream_t s);   // cudaErrorNotSupported: shape does not fit
// One warp runs the update pipeline's bounded barrier wait on a barrier nothing completes: *gave_up (DEVICE) <- 1
// and FLAG_WAIT_TIMEOUT in *status after about budget_cycles clock cycles.
cudaError_t launch_wait_timeout_selftest(uint32_t* status, long long budget_cycles, int* gave_up, cudaStream_t s);
// the same for the bounded wait of the tensor-core product kernels (gemm_tc.cu)
cudaError_t launch_gemm_wait_timeout_selftest(uint32_t* status, long long budget_cycles, int* gave_up, cudaStream_t s);
cudaError_t launch_center(const float* x, float* center, int32_t P, int64_t d, int64_t ld, cudaStream_t s);

// out[k] <- (1 - kk) center[k] + kk * mean_i x[i][k] over all ld columns (EAGD center rule, kk = P eta lambda)
cudaError_t launch_eagd_center(const float* x, const float* center, float* out, int32_t P, int64_t ld, double kk,
                               cudaStream_t s);

struct ElectArgs {
  const float* loss_in;     // DEVICE float[P] or nullptr when partials are given
  const double* partials;   // DEVICE double[P][n_partials] (row sums in fixed order) or nullptr
  int32_t n_partials;
  double partial_scale;     // loss_i = partial_scale * sum_b partials[i][b]
  float* loss_out;          // DEVICE float[P]: the loss vector the election used
  int32_t P, G;
  GroupTables tab;
  int32_t* ll;
  int32_t* gl;
  unsigned long long* group_keys;  // DEVICE u64[G] scratch
  int32_t* count_global;    // DEVICE int32[P]
  int32_t* count_local;     // DEVICE int32[P]
  bool update_local;        // write ll (and count)
  bool update_global;       // write gl (and count)
};
cudaError_t launch_elect(const ElectArgs& a, cudaStream_t s);
// cross-device election (groups spread over devices), see elect.cu
cudaError_t launch_shard_best_key(const float* loss, const int32_t* global_index, int32_t n_own, unsigned long long* key_out,
                                  int32_t* best_local, cudaStream_t s);
cudaError_t launch_shard_pick_global(const unsigned long long* keys, int32_t world, int32_t my_rank, int32_t guest_row,
                                     const int32_t* best_local, int32_t* gl, int32_t* result, cudaStream_t s);
// copies[r] <- x[ll[r]] for r in [r0, min(r1, G)), and copies[G] <- x[gl] if r1 > G
cudaError_t launch_leader_copies(const float* x, float* copies, const int32_t* ll, const int32_t* gl, int32_t G,
                                 int32_t r0, int32_t r1, int64_t d, int64_t ld, cudaStream_t s);

// Quadratic objective.
cudaError_t launch_quadratic_grad(const float* x, float* g, const float* a, const float* b,
                                  const float* noise, float sigma, int32_t P, int64_t d, int64_t ld,
                                  bool fp64, cudaStream_t s);
int32_t quadratic_loss_blocks(int64_t d);
cudaError_t launch_quadratic_loss_partials(const float* x, const float* a, const float* b, int32_t P,
                                           int64_t d, int64_t ld, double* partials, int32_t n_partials,
                                           cudaStream_t s);

// Matrix completion objective.
struct MatcompArgs {
  lsgd_matcomp_desc m;
  const float* x;
  float* g;
  int64_t ld;
  int32_t P;
  uint32_t* status;
};
// acc: DEVICE u64[P*ld] fixed-point accumulator, all zero on entry and again on exit
// finish: also convert the sums to fp32 in a.g and clear acc; otherwise the sums stay in acc for
// launch_matcomp_finish_step, which takes the plain step x <- x - eta g from them and clears acc
cudaError_t launch_matcomp_grad(const MatcompArgs& a, const int32_t* pos, unsigned long long* acc, bool finish, cudaStream_t s);
cudaError_t launch_matcomp_finish_step(unsigned long long* acc, float* x, int32_t P, int64_t ld, double eta, int arith,
                                       cudaStream_t s);
int32_t matcomp_loss_blocks(int32_t n_heldout);
cudaError_t launch_matcomp_loss_partials(const MatcompArgs& a, double* partials, int32_t n_partials,
                                         cudaStream_t s);

// Dense PSD completion objective.
int32_t psd_split(int32_t r);                     // CTAs per row block (partial gradients to combine), 1 = none
int32_t psd_loss_blocks(int32_t n, int32_t r);
// gpart: DEVICE double[psd_split(r) * P * ld] scratch when psd_split(r) > 1, else unused
cudaError_t launch_psd_grad(const float* x, float* g, const float* M, int32_t n, int32_t r, int32_t P, int64_t ld,
                            double* partials, int32_t n_partials, bool write_g, double* gpart, cudaStream_t s);

// Programmatic dependent launch.  A kernel started with launch_pdl() may become resident, and run its
// prologue (barrier and tensor-memory set-up, descriptor prefetch), while the kernel before it in the stream
// is still draining.  Such a kernel calls pdl_wait() before its first access to global memory that an earlier
// kernel may have written or may still read: the wait returns once every earlier kernel has completed and its
// writes are visible.  pdl_launch_dependents() lets the NEXT kernel in the stream become resident as soon as
// resources free up; it says nothing about this kernel's data, which the next kernel obtains through its own
// pdl_wait().  Building with -DLSGD_NO_PDL=1 turns every such launch into a plain one.
#ifndef LSGD_NO_PDL
#define LSGD_NO_PDL 0
#endif
#if defined(__CUDACC__)
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Sum of n doubles by one warp in a fixed order (lane-strided partial sums, then a butterfly), so the value
// does not depend on timing.  All 32 lanes call it and all get the result.
__device__ __forceinline__ double warp_sum_fixed(const double* __restrict__ v, int n) {
  double acc = 0.0;
  for (int b = threadIdx.x & 31; b < n; b += 32) acc += v[b];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  return acc;
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = LSGD_NO_PDL ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif

}  // namespace lsgd

struct lsgd_ctx {
  lsgd_config cfg;
  lsgd_quadratic_desc quad;
  lsgd_matcomp_desc mc;
  lsgd_mlp_desc mlp;
  lsgd_psd_desc psd;
  bool loss_partials_valid;  // PSD: the partial sums of F in d_partials belong to the current x
  cudaStream_t stream;
  int device;
  std::vector<int32_t> group_of;
  // one device slab holding all small state
  void* slab;
  int32_t *d_rows_by_group, *d_group_start, *d_group_of, *d_ll, *d_gl, *d_count_g, *d_count_l;
  uint32_t* d_status;
  float* d_loss;
  unsigned long long* d_group_keys;
  double* d_partials;
  int32_t* d_selftest;          // one word written by lsgd_selftest_wait_timeout
  int32_t* d_shard;             // cross-device election: [0] this device's best own worker, [1..3] the result triple
  int32_t n_partials;
  int64_t t;
  int64_t n_elections;
  bool grad_ready;
  bool eagd_center_ready;    // EAGD: the center row has been initialised to the workers' mean
  bool fused_applied;        // MLP: the pending gradient has already stepped W1, W2 (plain step)
  const float* armed_noise;  // QUADRATIC with g == NULL: noise pointer for the next step
  void* mlp_state;           // opaque MLP pipeline state
  unsigned long long* d_acc64;  // MATCOMP: fixed-point gradient accumulator [P*ld], kept all-zero between steps
  bool mc_step_pending;         // MATCOMP fused step: the gradient sums wait in d_acc64 for lsgd_step
  double* d_psd_part;           // PSD, small ranks: partial gradients of the CTAs that share a row block
  bool owns_acc64, owns_psd_part;   // false: the buffer is the caller's (descriptor scratch field)
};
