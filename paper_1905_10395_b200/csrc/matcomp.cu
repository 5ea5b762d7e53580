// Factorised matrix completion on observed entries (low-rank completion is the paper's motivating
// example, Section 2.1; here with two factors and a sampled set of observed cells).
// Worker row = [X (n_rows x rank) | Y (n_cols x rank)], both row-major.
//
//   gradient of (1/(2B)) sum_{(r,c,v) in batch} (<X_r, Y_c> - v)^2 :
//     dX_r += e Y_c / B,  dY_c += e X_r / B,  e = <X_r, Y_c> - v     (duplicates in a batch add up)
//   election loss: (1/N) sum over the held-out list of e^2, fp64 partial sums in a fixed order.
//
// The whole state of this workload (a few MB per worker) lives in L2; the kernels are gather /
// scatter bound, not HBM bound.  Duplicated rows and columns of a batch make the gradient a scatter-ADD.
// To keep it independent of the order in which the adds land, every contribution e * y / B is evaluated
// in fp64, converted to 2^-44 fixed point and added with 64-bit integer atomics (integer addition is
// associative, so the sum is exact and the same on every run); a second kernel converts the sums to fp32
// and clears the accumulator for the next step.  The resolution is 5.7e-14.  Range: a contribution must be
// finite and below 2^4 in magnitude, and at most 2^15 of them can meet in one entry (the batch size is capped
// there at creation), so the 64-bit sum stays below 2^63.  A contribution outside that range -- a diverging
// worker -- is not added; the kernel raises FLAG_OVERFLOW in the status word instead of saturating silently.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxRank = 32;
constexpr int kLossPerThread = 4;

constexpr double kFixScale = 17592186044416.0;        // 2^44
constexpr double kFixInv = 1.0 / 17592186044416.0;
constexpr double kFixLimit = 16.0 * 17592186044416.0;  // 2^48: |contribution| < 2^4 in fixed-point units

// A group of GROUP lanes (8, 16 or 32: the smallest that holds the rank) works on one observed entry, lane k
// on component k of its two factor rows, so a row is fetched and its sums are updated as one contiguous piece.
// dot = sum_k x_k y_k is added in component order by every lane of the group (each product of two floats is
// exact in fp64, so this is the same value a sequential fused-multiply-add loop gives).
template <int GROUP>
__device__ __forceinline__ double group_dot(float xk, float yk, int rank, int base) {
  const double p = (double)xk * (double)yk;
  double dot = 0.0;
  for (int k = 0; k < rank; ++k) dot += __shfl_sync(0xFFFFFFFFu, p, base + k);
  return dot;
}

template <int GROUP>
__global__ void __launch_bounds__(kThreads)
matcomp_grad_kernel(MatcompArgs a, const int32_t* __restrict__ pos, unsigned long long* __restrict__ acc) {
  const int i = blockIdx.y;
  const int lane = threadIdx.x & 31, k = lane % GROUP, base = lane - k;
  const int p = (blockIdx.x * kThreads + threadIdx.x) / GROUP;       // this group's entry of the batch
  const int rank = a.m.rank;
  bool ok = p < a.m.batch;
  int r = 0, c = 0;
  float v = 0.f;
  if (ok) {
    const int q = pos[(int64_t)i * a.m.batch + p];
    if (q < 0 || q >= a.m.n_obs) {
      if (k == 0) atomicOr(a.status, FLAG_BAD_INDEX);
      ok = false;
    } else {
      r = a.m.obs_r[q];
      c = a.m.obs_c[q];
      v = a.m.obs_v[q];
      if (r < 0 || r >= a.m.n_rows || c < 0 || c >= a.m.n_cols) {
        if (k == 0) atomicOr(a.status, FLAG_BAD_INDEX);
        ok = false;
      }
    }
  }
  const int64_t xo = (int64_t)i * a.ld + (int64_t)r * rank;
  const int64_t yo = (int64_t)i * a.ld + ((int64_t)a.m.n_rows + c) * rank;
  const bool mine = ok && k < rank;
  const float xk = mine ? a.x[xo + k] : 0.f, yk = mine ? a.x[yo + k] : 0.f;
  const double dot = group_dot<GROUP>(xk, yk, rank, base);          // all 32 lanes take part in the shuffles
  if (mine) {
    const double e = (dot - (double)v) / (double)a.m.batch * kFixScale;
    const double cx = e * (double)yk, cy = e * (double)xk;
    if (fabs(cx) < kFixLimit && fabs(cy) < kFixLimit) {          // false for NaN and infinities too
      atomicAdd(acc + xo + k, (unsigned long long)__double2ll_rn(cx));
      atomicAdd(acc + yo + k, (unsigned long long)__double2ll_rn(cy));
    } else {
      atomicOr(a.status, FLAG_OVERFLOW);
    }
  }
}

// g <- fixed-point sums as fp32; the accumulator is cleared on the way
__global__ void __launch_bounds__(kThreads)
matcomp_finish_kernel(unsigned long long* __restrict__ acc, float* __restrict__ g, int64_t total) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    const long long v = (long long)acc[e];
    if (v != 0) acc[e] = 0ull;
    g[e] = (float)((double)v * kFixInv);
  }
}

// x <- x - eta g for the entries the batch touched, g as above, without storing g: the plain step taken straight
// from the fixed-point sums (x - eta * 0 = x exactly, so untouched entries need no work).  A thread scans four
// consecutive sums (two 16-byte loads); nearly all are zero.
__global__ void __launch_bounds__(kThreads)
matcomp_finish_step_kernel(unsigned long long* __restrict__ acc, float* __restrict__ x, int64_t total, double eta, int arith) {
  const int64_t e0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;     // total is a multiple of 32
  if (e0 >= total) return;
  const ulonglong2 lo = *reinterpret_cast<const ulonglong2*>(acc + e0);
  const ulonglong2 hi = *reinterpret_cast<const ulonglong2*>(acc + e0 + 2);
  const unsigned long long raw[4] = {lo.x, lo.y, hi.x, hi.y};
  if ((lo.x | lo.y | hi.x | hi.y) == 0ull) return;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const long long v = (long long)raw[j];
    if (v != 0) {
      acc[e0 + j] = 0ull;
      const float g = (float)((double)v * kFixInv);
      const float xv = x[e0 + j];
      float xn;
      if (arith == 0) xn = (float)__dsub_rn((double)xv, __dmul_rn(eta, (double)g));
      else if (arith == 1) xn = (float)fma(-eta, (double)g, (double)xv);
      else xn = fmaf(-(float)eta, g, xv);
      x[e0 + j] = xn;
    }
  }
}

// Held-out loss: one thread per entry (the kernel is bound by the L2 gathers of the factor rows, 2 sectors per
// row whoever fetches them; one entry per thread keeps the most of them in flight), fp64 residuals, partial sums
// per CTA in a fixed order.
__global__ void __launch_bounds__(kThreads)
matcomp_loss_kernel(MatcompArgs a, double* __restrict__ partials, int32_t n_partials) {
  const int i = blockIdx.y;
  const int rank = a.m.rank;
  const float* xi = a.x + (int64_t)i * a.ld;
  double acc = 0.0;
#pragma unroll
  for (int u = 0; u < kLossPerThread; ++u) {
    const int p = (blockIdx.x * kLossPerThread + u) * kThreads + threadIdx.x;
    if (p < a.m.n_heldout) {
      const int q = a.m.heldout_pos[p];
      if (q < 0 || q >= a.m.n_obs) {
        atomicOr(a.status, FLAG_BAD_INDEX);
        continue;
      }
      const int r = a.m.obs_r[q], c = a.m.obs_c[q];
      if (r < 0 || r >= a.m.n_rows || c < 0 || c >= a.m.n_cols) {
        atomicOr(a.status, FLAG_BAD_INDEX);
        continue;
      }
      const float* xr = xi + (int64_t)r * rank;
      const float* yc = xi + ((int64_t)a.m.n_rows + c) * rank;
      double dot = 0.0;
      for (int k = 0; k < rank; ++k) dot += (double)xr[k] * (double)yc[k];
      const double e = dot - (double)a.m.obs_v[q];
      acc += e * e;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  __shared__ double s_w[kThreads / 32];
  if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) t += s_w[w];
    partials[(int64_t)i * n_partials + blockIdx.x] = t;
  }
}

}  // namespace

cudaError_t launch_matcomp_grad(const MatcompArgs& a, const int32_t* pos, unsigned long long* acc, bool finish, cudaStream_t s) {
  const int rank = a.m.rank;
  const int group = rank <= 8 ? 8 : (rank <= 16 ? 16 : 32);
  const int per_cta = kThreads / group;
  dim3 grid((unsigned)((a.m.batch + per_cta - 1) / per_cta), (unsigned)a.P);
  if (group == 8) matcomp_grad_kernel<8><<<grid, kThreads, 0, s>>>(a, pos, acc);
  else if (group == 16) matcomp_grad_kernel<16><<<grid, kThreads, 0, s>>>(a, pos, acc);
  else matcomp_grad_kernel<32><<<grid, kThreads, 0, s>>>(a, pos, acc);
  if (finish) {
    const int64_t total = (int64_t)a.P * a.ld;
    int64_t blocks = (total + kThreads - 1) / kThreads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    matcomp_finish_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(acc, a.g, total);
  }
  return cudaGetLastError();
}

cudaError_t launch_matcomp_finish_step(unsigned long long* acc, float* x, int32_t P, int64_t ld, double eta, int arith,
                                       cudaStream_t s) {
  const int64_t total = (int64_t)P * ld;                    // ld is a multiple of 32
  const int64_t blocks = (total / 4 + kThreads - 1) / kThreads;
  matcomp_finish_step_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(acc, x, total, eta, arith);
  return cudaGetLastError();
}

int32_t matcomp_loss_blocks(int32_t n_heldout) {
  const int per = kThreads * kLossPerThread;
  return (n_heldout + per - 1) / per;
}

cudaError_t launch_matcomp_loss_partials(const MatcompArgs& a, double* partials, int32_t n_partials, cudaStream_t s) {
  dim3 grid((unsigned)n_partials, (unsigned)a.P);
  matcomp_loss_kernel<<<grid, kThreads, 0, s>>>(a, partials, n_partials);
  return cudaGetLastError();
}

}  // namespace lsgd
