// Positive semi-definite low-rank matrix completion, the paper's motivating example (Section 2.1 and the
// supplement's "Low-Rank Matrix Completion Experiments"):
//     F(X) = 1/4 || M - X X^T ||_F^2,   X in R^{n x r},   grad F(X) = (X X^T - M) X.
// A worker's parameter row is X, row-major.  One pass computes the exact (batch) gradient of every worker
// and the partial sums of F, so the election loss costs nothing extra on the step that also needs g.
//
// CTA (tile, worker) owns 32 rows I of X.  For every 32-row block J it forms the residual tile
// R = X_I X_J^T - M_IJ (thread (a, b) one entry), adds R^2 to the loss, and accumulates G_I += R X_J.
// R is never written to memory.  Products and sums are fp64 (the experiment is about reaching high
// accuracy; fp64 runs at half the fp32 rate on this part and the problem is small), results are
// rounded once to fp32.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int T = 32;
constexpr int kMaxRank = 128;

__global__ void __launch_bounds__(T * T)
psd_grad_kernel(const float* __restrict__ x, float* __restrict__ g, const float* __restrict__ M, int32_t n, int32_t r,
                int64_t ld, double* __restrict__ partials, int32_t n_partials, int write_g) {
  extern __shared__ double s_psd[];
  const int pitch = r | 1;                      // odd pitch: conflict-free column walks
  double* XI = s_psd;                           // [T][pitch]
  double* XJ = XI + T * pitch;                  // [T][pitch]
  double* Rt = XJ + T * pitch;                  // [T][T + 1]
  const int i = blockIdx.y, I0 = blockIdx.x * T;
  const int a = threadIdx.y, b = threadIdx.x, tid = a * T + b;
  const float* xi = x + (int64_t)i * ld;
  for (int idx = tid; idx < T * r; idx += T * T) {
    const int row = idx / r, k = idx - row * r;
    XI[row * pitch + k] = (I0 + row < n) ? (double)xi[(int64_t)(I0 + row) * r + k] : 0.0;
  }
  double acc[kMaxRank / T];
#pragma unroll
  for (int m = 0; m < kMaxRank / T; ++m) acc[m] = 0.0;
  double lsum = 0.0;
  for (int J0 = 0; J0 < n; J0 += T) {
    for (int idx = tid; idx < T * r; idx += T * T) {
      const int row = idx / r, k = idx - row * r;
      XJ[row * pitch + k] = (J0 + row < n) ? (double)xi[(int64_t)(J0 + row) * r + k] : 0.0;
    }
    __syncthreads();
    double s = 0.0;
    for (int k = 0; k < r; ++k) s = fma(XI[a * pitch + k], XJ[b * pitch + k], s);
    const double rab = (I0 + a < n && J0 + b < n) ? s - (double)M[(int64_t)(I0 + a) * n + J0 + b] : 0.0;
    lsum = fma(rab, rab, lsum);
    Rt[a * (T + 1) + b] = rab;
    __syncthreads();
#pragma unroll
    for (int m = 0; m < kMaxRank / T; ++m) {
      const int k = b + T * m;
      if (k < r) {
        double t = acc[m];
#pragma unroll 8
        for (int bb = 0; bb < T; ++bb) t = fma(Rt[a * (T + 1) + bb], XJ[bb * pitch + k], t);
        acc[m] = t;
      }
    }
    __syncthreads();
  }
  if (write_g && I0 + a < n) {
    float* gi = g + (int64_t)i * ld + (int64_t)(I0 + a) * r;
#pragma unroll
    for (int m = 0; m < kMaxRank / T; ++m) {
      const int k = b + T * m;
      if (k < r) gi[k] = (float)acc[m];
    }
  }
  // block sum of R^2 in a fixed order: warp shuffles, then the 32 warp sums in index order
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, o);
  __shared__ double s_w[T];
  if (b == 0) s_w[a] = lsum;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < T; ++w) t += s_w[w];
    partials[(int64_t)i * n_partials + blockIdx.x] = t;
  }
}

}  // namespace

int32_t psd_loss_blocks(int32_t n) { return (n + T - 1) / T; }

cudaError_t launch_psd_grad(const float* x, float* g, const float* M, int32_t n, int32_t r, int32_t P, int64_t ld,
                            double* partials, int32_t n_partials, bool write_g, cudaStream_t s) {
  const int pitch = r | 1;
  const size_t smem = sizeof(double) * (size_t)(2 * T * pitch + T * (T + 1));
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(psd_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid((unsigned)n_partials, (unsigned)P), block(T, T);
  psd_grad_kernel<<<grid, block, smem, s>>>(x, g, M, n, r, ld, partials, n_partials, write_g ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace lsgd
