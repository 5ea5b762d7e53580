// Diagonal quadratic objective f(x) = 1/2 sum_k a_k (x_k - b_k)^2 (the quadratic model of
// Section 3.3 with a diagonal Hessian): materialised stochastic gradient g = a (x - b) + sigma eps
// and the first stage of the exact election loss f(x_i).
//
// Loss: CTA (blk, row group) sums the terms of up to 4 workers over a fixed chunk of columns, every term
// evaluated and accumulated in fp64, and writes one partial per worker; the election kernel adds the
// partials in index order.
// Chunking and tree shape depend only on d, so the result is reproducible run to run.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 8;                               // float4 per thread per chunk
constexpr int64_t kChunkCols = (int64_t)kThreads * 4 * kVecPerThread;  // 8192 columns per CTA

// fp64: one IEEE operation per printed operation, rounded once to fp32.
template <bool F64>
__device__ __forceinline__ float grad1(float x, float a, float b, float n, float sigma, bool noise) {
  if (F64) {
    double r = __dmul_rn((double)a, __dsub_rn((double)x, (double)b));
    if (noise) r = __dadd_rn(r, __dmul_rn((double)sigma, (double)n));
    return (float)r;
  }
  return fmaf(a, x - b, noise ? sigma * n : 0.f);
}

template <bool F64>
__global__ void __launch_bounds__(kThreads)
quadratic_grad_kernel(const float* __restrict__ x, float* __restrict__ g, const float* __restrict__ a,
                      const float* __restrict__ b, const float* __restrict__ noise, float sigma, int32_t P,
                      int64_t n4, int64_t ld) {
  const int64_t total = (int64_t)P * n4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    const int64_t row = e / n4, c = (e - row * n4) * 4;
    const int64_t off = row * ld + c;
    const float4 xv = __ldg(reinterpret_cast<const float4*>(x + off));
    const float4 av = __ldg(reinterpret_cast<const float4*>(a + c));
    const float4 bv = __ldg(reinterpret_cast<const float4*>(b + c));
    float4 nv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (noise) nv = __ldcs(reinterpret_cast<const float4*>(noise + off));
    float4 r;
    const bool hn = noise != nullptr;
    r.x = grad1<F64>(xv.x, av.x, bv.x, nv.x, sigma, hn);
    r.y = grad1<F64>(xv.y, av.y, bv.y, nv.y, sigma, hn);
    r.z = grad1<F64>(xv.z, av.z, bv.z, nv.z, sigma, hn);
    r.w = grad1<F64>(xv.w, av.w, bv.w, nv.w, sigma, hn);
    *reinterpret_cast<float4*>(g + off) = r;
  }
}

// Workers per CTA: a and b are loaded and converted once for all of them.  4 rather than 8: the CTAs of the
// 64 x 2^20 problem then fill 2.8 waves instead of 1.4, and the partial sums stay the same bit for bit.
constexpr int kLossRows = 4;

__device__ __forceinline__ double term(double x, double a, double b) {
  const double r = x - b;
  return a * r * r;
}

// CTA (chunk, row group): partial sums of f over 8192 columns for up to kLossRows workers.
__global__ void __launch_bounds__(kThreads)
quadratic_loss_kernel(const float* __restrict__ x, const float* __restrict__ a, const float* __restrict__ b, int32_t P,
                      int64_t d, int64_t ld, double* __restrict__ partials, int32_t n_partials) {
  pdl_wait();
  pdl_launch_dependents();
  const int i0 = blockIdx.y * kLossRows;
  const int rows = min(kLossRows, P - i0);
  const int64_t c0 = (int64_t)blockIdx.x * kChunkCols;
  double acc[kLossRows];
#pragma unroll
  for (int r = 0; r < kLossRows; ++r) acc[r] = 0.0;
#pragma unroll 2
  for (int v = 0; v < kVecPerThread; ++v) {
    const int64_t c = c0 + ((int64_t)v * kThreads + threadIdx.x) * 4;
    if (c + 3 < d) {
      const float4 af = __ldg(reinterpret_cast<const float4*>(a + c));
      const float4 bf = __ldg(reinterpret_cast<const float4*>(b + c));
      const double a0 = af.x, a1 = af.y, a2 = af.z, a3 = af.w;
      const double b0 = bf.x, b1 = bf.y, b2 = bf.z, b3 = bf.w;
      float4 xv[kLossRows];
#pragma unroll
      for (int r = 0; r < kLossRows; ++r)
        if (r < rows) xv[r] = __ldcs(reinterpret_cast<const float4*>(x + (int64_t)(i0 + r) * ld + c));
#pragma unroll
      for (int r = 0; r < kLossRows; ++r)
        if (r < rows)
          acc[r] += term((double)xv[r].x, a0, b0) + term((double)xv[r].y, a1, b1) + term((double)xv[r].z, a2, b2) +
                    term((double)xv[r].w, a3, b3);
    } else {
      for (int64_t k = c; k < d; ++k)
        for (int r = 0; r < rows; ++r) acc[r] += term((double)x[(int64_t)(i0 + r) * ld + k], (double)a[k], (double)b[k]);
    }
  }
  __shared__ double s_w[kLossRows][kThreads / 32];
#pragma unroll
  for (int r = 0; r < kLossRows; ++r) {
    double t = acc[r];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    if ((threadIdx.x & 31) == 0) s_w[r][threadIdx.x >> 5] = t;
  }
  __syncthreads();
  if (threadIdx.x < rows) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) t += s_w[threadIdx.x][w];
    partials[(int64_t)(i0 + threadIdx.x) * n_partials + blockIdx.x] = t;
  }
}

}  // namespace

cudaError_t launch_quadratic_grad(const float* x, float* g, const float* a, const float* b, const float* noise,
                                  float sigma, int32_t P, int64_t d, int64_t ld, bool fp64, cudaStream_t s) {
  const int64_t n4 = (d + 3) / 4;
  const int64_t total = (int64_t)P * n4;
  int64_t blocks = (total + kThreads - 1) / kThreads;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  if (fp64)
    quadratic_grad_kernel<true><<<(unsigned)blocks, kThreads, 0, s>>>(x, g, a, b, noise, sigma, P, n4, ld);
  else
    quadratic_grad_kernel<false><<<(unsigned)blocks, kThreads, 0, s>>>(x, g, a, b, noise, sigma, P, n4, ld);
  return cudaGetLastError();
}

int32_t quadratic_loss_blocks(int64_t d) { return (int32_t)((d + kChunkCols - 1) / kChunkCols); }

cudaError_t launch_quadratic_loss_partials(const float* x, const float* a, const float* b, int32_t P, int64_t d,
                                           int64_t ld, double* partials, int32_t n_partials, cudaStream_t s) {
  dim3 grid((unsigned)n_partials, (unsigned)((P + kLossRows - 1) / kLossRows));
  return launch_pdl(quadratic_loss_kernel, grid, dim3(kThreads), 0, s, x, a, b, P, d, ld, partials, n_partials);
}

}  // namespace lsgd
