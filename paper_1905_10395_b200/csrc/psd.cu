// Positive semi-definite low-rank matrix completion, the paper's motivating example (Section 2.1 and the
// supplement's "Low-Rank Matrix Completion Experiments"):
//     F(X) = 1/4 || M - X X^T ||_F^2,   X in R^{n x r},   grad F(X) = (X X^T - M) X.
// A worker's parameter row is X, row-major.  One pass computes the exact (batch) gradient of every worker
// and the partial sums of F, so the election loss costs nothing extra on the step that also needs g.
//
// CTA (tile, worker) owns 64 rows I of X.  For every 64-row block J it forms the residual tile
// R = X_I X_J^T - M_IJ, adds R^2 to the loss, and accumulates G_I += R X_J.  R is never written to
// memory.  Products and sums are fp64 (the experiment is about reaching high accuracy; fp64 runs at half
// the fp32 rate on this part and the problem is small), results are rounded once to fp32.
//
// 256 threads as 16 x 16; each thread holds a 4 x 4 micro-tile of R (rows ty + 16 i, columns tx + 16 j)
// and 4 x (r / 16) outputs of G, so one shared-memory load feeds four fused multiply-adds; the X tiles
// are converted to fp64 once when they are staged.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int T = 64;            // tile edge
constexpr int TH = 16;           // threads per tile edge
constexpr int MT = T / TH;       // micro-tile edge (4)

// KM = output columns of G per thread = ceil(r / 16) rounded up to 1, 2, 4 or 8: a compile-time bound, so a
// small rank neither issues the fp64 operations of absent columns (predicated off, they still occupy the pipe:
// at r = 10 they were seven eighths of its work) nor holds their accumulators in registers.
// Z = CTAs that share one row block (gridDim.z): CTA z takes the column blocks z, z + Z, ...  At small rank the
// time is the dependent chain over the column blocks, which only a shorter chain shortens; the Z partial
// gradients go to gpart[z][P][ld] in fp64 and psd_combine_kernel adds them in z order.  Z = 1 writes g itself.
template <int KM, int Z>
__global__ void __launch_bounds__(TH * TH, Z > 1 ? 2 : 1)
psd_grad_kernel(const float* __restrict__ x, float* __restrict__ g, const float* __restrict__ M, int32_t n, int32_t r,
                int64_t ld, double* __restrict__ partials, int32_t n_partials, int write_g, double* __restrict__ gpart,
                int32_t P) {
  extern __shared__ double s_psd[];
  const int pitch = r | 1;                      // odd pitch: conflict-free column walks
  double* XI = s_psd;                           // [T][pitch]
  double* XJ = XI + T * pitch;                  // [T][pitch]
  double* Rt = XJ + T * pitch;                  // [T][T + 1]
  const int i = blockIdx.y, I0 = blockIdx.x * T;
  const int ty = threadIdx.y, tx = threadIdx.x, tid = ty * TH + tx;
  const float* xi = x + (int64_t)i * ld;
  for (int idx = tid; idx < T * r; idx += TH * TH) {
    const int row = idx / r, k = idx - row * r;
    XI[row * pitch + k] = (I0 + row < n) ? (double)xi[(int64_t)(I0 + row) * r + k] : 0.0;
  }
  double acc[MT][KM];
#pragma unroll
  for (int a = 0; a < MT; ++a)
#pragma unroll
    for (int m = 0; m < KM; ++m) acc[a][m] = 0.0;
  double lsum = 0.0;
  // The next block's operands -- this thread's 16 entries of M and its share of X_J -- are fetched into
  // registers while the current block is being worked on, so their latency is off the critical path.
  constexpr int NX = (T * 16 * KM + TH * TH - 1) / (TH * TH);   // X_J values per thread (r <= 16 KM)
  float m_next[MT][MT], xj_next[NX];
  auto fetch = [&](int J0) {
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int b = 0; b < MT; ++b) {
        const int ri = I0 + ty + TH * a, cj = J0 + tx + TH * b;
        m_next[a][b] = (ri < n && cj < n) ? M[(int64_t)ri * n + cj] : 0.f;
      }
#pragma unroll
    for (int q = 0; q < NX; ++q) {
      const int idx = tid + q * TH * TH;
      const int row = idx / r, k = idx - row * r;
      xj_next[q] = (idx < T * r && J0 + row < n) ? xi[(int64_t)(J0 + row) * r + k] : 0.f;
    }
  };
  const int Jstep = T * Z;
  fetch((int)blockIdx.z * T);
  for (int J0 = (int)blockIdx.z * T; J0 < n; J0 += Jstep) {
    float m_cur[MT][MT];
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int b = 0; b < MT; ++b) m_cur[a][b] = m_next[a][b];
#pragma unroll
    for (int q = 0; q < NX; ++q) {
      const int idx = tid + q * TH * TH;
      const int row = idx / r, k = idx - row * r;
      if (idx < T * r) XJ[row * pitch + k] = (double)xj_next[q];
    }
    __syncthreads();
    if (J0 + Jstep < n) fetch(J0 + Jstep);
    // R micro-tile: rows ty + 16 a, columns tx + 16 b
    double s[MT][MT];
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int b = 0; b < MT; ++b) s[a][b] = 0.0;
    for (int k = 0; k < r; ++k) {
      double xa[MT], xb[MT];
#pragma unroll
      for (int a = 0; a < MT; ++a) xa[a] = XI[(ty + TH * a) * pitch + k];
#pragma unroll
      for (int b = 0; b < MT; ++b) xb[b] = XJ[(tx + TH * b) * pitch + k];
#pragma unroll
      for (int a = 0; a < MT; ++a)
#pragma unroll
        for (int b = 0; b < MT; ++b) s[a][b] = fma(xa[a], xb[b], s[a][b]);
    }
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int b = 0; b < MT; ++b) {
        const int ri = I0 + ty + TH * a, cj = J0 + tx + TH * b;
        const double rab = (ri < n && cj < n) ? s[a][b] - (double)m_cur[a][b] : 0.0;
        lsum = fma(rab, rab, lsum);
        Rt[(ty + TH * a) * (T + 1) + tx + TH * b] = rab;
      }
    __syncthreads();
    // G rows ty + 16 a, columns tx + 16 m
    for (int bb = 0; bb < T; ++bb) {
      double ra[MT];
#pragma unroll
      for (int a = 0; a < MT; ++a) ra[a] = Rt[(ty + TH * a) * (T + 1) + bb];
#pragma unroll
      for (int m = 0; m < KM; ++m) {
        const int k = tx + TH * m;
        if (k < r) {
          const double xj = XJ[bb * pitch + k];
#pragma unroll
          for (int a = 0; a < MT; ++a) acc[a][m] = fma(ra[a], xj, acc[a][m]);
        }
      }
    }
    __syncthreads();
  }
  if (write_g) {
#pragma unroll
    for (int a = 0; a < MT; ++a) {
      const int ri = I0 + ty + TH * a;
      if (ri < n) {
        const int64_t row = (int64_t)i * ld + (int64_t)ri * r;
#pragma unroll
        for (int m = 0; m < KM; ++m) {
          const int k = tx + TH * m;
          if (k < r) {
            if (Z == 1) g[row + k] = (float)acc[a][m];
            else gpart[((int64_t)blockIdx.z * P) * ld + row + k] = acc[a][m];
          }
        }
      }
    }
  }
  // block sum of R^2 in a fixed order: warp shuffles, then the 8 warp sums in index order
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, o);
  __shared__ double s_w[TH * TH / 32];
  if ((tid & 31) == 0) s_w[tid >> 5] = lsum;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < TH * TH / 32; ++w) t += s_w[w];
    partials[(int64_t)i * n_partials + blockIdx.x * Z + blockIdx.z] = t;
  }
}

// g = the Z partial gradients added in z order in fp64, rounded once
__global__ void __launch_bounds__(256)
psd_combine_kernel(const double* __restrict__ gpart, float* __restrict__ g, int64_t total, int32_t Z, int64_t cols, int64_t ld) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    if (e % ld >= cols) continue;                 // padding columns of g are not this objective's
    double t = 0.0;
    for (int z = 0; z < Z; ++z) t += gpart[(int64_t)z * total + e];
    g[e] = (float)t;
  }
}

}  // namespace

#ifndef LSGD_PSD_SPLIT
#define LSGD_PSD_SPLIT 2
#endif
// CTAs per row block: small ranks are latency-bound and split the column blocks (see psd_grad_kernel)
int32_t psd_split(int32_t r) { return r <= 32 ? LSGD_PSD_SPLIT : 1; }

int32_t psd_loss_blocks(int32_t n, int32_t r) { return ((n + T - 1) / T) * psd_split(r); }

template <int KM, int Z>
cudaError_t launch_psd_t(const float* x, float* g, const float* M, int32_t n, int32_t r, int32_t P, int64_t ld, double* partials,
                         int32_t n_partials, int wg, double* gpart, cudaStream_t s) {
  const int pitch = r | 1;
  const size_t smem = sizeof(double) * (size_t)(2 * T * pitch + T * (T + 1));
  static OncePerDevice attr;
  if (!attr.here()) {
    cudaError_t e = cudaFuncSetAttribute(psd_grad_kernel<KM, Z>, cudaFuncAttributeMaxDynamicSharedMemorySize, 180 * 1024);
    if (e == cudaSuccess && Z > 1)   // two CTAs per SM: ask for the largest shared-memory carve-out
      e = cudaFuncSetAttribute(psd_grad_kernel<KM, Z>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr.here() = true;
  }
  dim3 grid((unsigned)(n_partials / Z), (unsigned)P, (unsigned)Z), block(TH, TH);
  psd_grad_kernel<KM, Z><<<grid, block, smem, s>>>(x, g, M, n, r, ld, partials, n_partials, wg, gpart, P);
  if (Z > 1 && wg) {
    const int64_t total = (int64_t)P * ld;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    psd_combine_kernel<<<(unsigned)blocks, 256, 0, s>>>(gpart, g, total, Z, (int64_t)n * r, ld);
  }
  return cudaGetLastError();
}

// gpart: DEVICE double[psd_split(r) * P * ld] when psd_split(r) > 1 (unused otherwise)
cudaError_t launch_psd_grad(const float* x, float* g, const float* M, int32_t n, int32_t r, int32_t P, int64_t ld,
                            double* partials, int32_t n_partials, bool write_g, double* gpart, cudaStream_t s) {
  if (n_partials != psd_loss_blocks(n, r)) return cudaErrorInvalidValue;
  const int wg = write_g ? 1 : 0;
  constexpr int ZS = LSGD_PSD_SPLIT;
  if (psd_split(r) > 1 && !gpart) return cudaErrorInvalidValue;
  if (r <= 16) return launch_psd_t<1, ZS>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
  if (r <= 32) return launch_psd_t<2, ZS>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
  if (r <= 64) return launch_psd_t<4, 1>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
  return launch_psd_t<8, 1>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
}

}  // namespace lsgd
