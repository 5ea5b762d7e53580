// lsgd_quadratic_loss_noalloc: the quadratic election loss for callers that must not allocate.
//
// Who needs this: code that runs where device allocation is forbidden or unsafe -- inside a region a
// framework has fenced off against allocator calls (a memory-pool-managed training loop whose pool
// owns all device memory, a real-time or safety-certified loop with a "no allocation after start-up"
// rule, a plugin running under someone else's CUDA context with a fixed memory budget).  Such callers
// cannot use lsgd_create, which allocates its state with cudaMalloc.
//
// The two-stage reduction needs P x ceil(d / 8192) doubles of scratch for the per-chunk partial sums.
// Here that scratch is a fixed array in the library's device image instead of an allocation:
// kNoAllocMaxPartials doubles (512 KiB), resident on every GPU that loads the library until the process
// exits.  Larger problems are rejected with LSGD_ERR_TOO_LARGE.
//
// Host code cannot pass the array's name to a kernel: on the host the name is only a stand-in for the
// symbol, not a device address.  The device address is looked up once per device with
// cudaGetSymbolAddress (first call on that device, with that device current) and cached.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int kNoAllocMaxPartials = 65536;   // doubles: 512 KiB per GPU
constexpr int kMaxDevices = 64;

static __device__ __align__(256) double g_noalloc_partials[kNoAllocMaxPartials];

// loss[i] = 1/2 * (partials[i][0] + partials[i][1] + ...), one warp per worker, added in fp64 in the same
// fixed order and with the same rounding as the election kernel's own second stage.  Device code names the
// array directly.
__global__ void __launch_bounds__(128) noalloc_finish_kernel(float* __restrict__ loss, int32_t P, int32_t n_partials) {
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= P) return;      // whole warps leave together
  const double acc = warp_sum_fixed(g_noalloc_partials + (int64_t)i * n_partials, n_partials);
  if ((threadIdx.x & 31) == 0) loss[i] = (float)(acc * 0.5);
}

double* scratch_address_for_current_device(cudaError_t* err) {
  static double* cache[kMaxDevices] = {nullptr};
  int dev = -1;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= kMaxDevices) {
    *err = cudaErrorInvalidDevice;
    return nullptr;
  }
  if (!cache[dev]) {
    double* p = nullptr;
    *err = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_partials);
    if (*err != cudaSuccess) return nullptr;
    cache[dev] = p;
  }
  return cache[dev];
}

}  // namespace
}  // namespace lsgd

extern "C" lsgd_status lsgd_quadratic_loss_noalloc(const float* x, const float* a, const float* b, int32_t P, int64_t d,
                                                   int64_t ld, float* loss, void* stream) {
  using namespace lsgd;
  if (!x || !a || !b || !loss) return LSGD_ERR_INVALID_ARG;
  if (P < 1 || P > 65535 || d < 1 || ld < d) return LSGD_ERR_INVALID_ARG;
  if (ld % 32 != 0) return LSGD_ERR_ALIGNMENT;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) & 15u)
    return LSGD_ERR_ALIGNMENT;
  const int64_t n_partials = quadratic_loss_blocks(d);
  if ((int64_t)P * n_partials > kNoAllocMaxPartials) return LSGD_ERR_TOO_LARGE;
  cudaError_t err = cudaSuccess;
  double* scratch = scratch_address_for_current_device(&err);
  if (!scratch) return LSGD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Every partial [i][blk] is written by exactly one CTA before it is read, so nothing has to be
  // cleared although the array still holds the previous call's values.
  if (launch_quadratic_loss_partials(x, a, b, P, d, ld, scratch, (int32_t)n_partials, s) != cudaSuccess) return LSGD_ERR_CUDA;
  noalloc_finish_kernel<<<(P + 3) / 4, 128, 0, s>>>(loss, P, (int32_t)n_partials);
  return cudaGetLastError() == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}
