// Positive semi-definite low-rank matrix completion, the paper's motivating example (Section 2.1 and the
// supplement's "Low-Rank Matrix Completion Experiments"):
//     F(X) = 1/4 || M - X X^T ||_F^2,   X in R^{n x r},   grad F(X) = (X X^T - M) X.
// A worker's parameter row is X, row-major.  One pass computes the exact (batch) gradient of every worker
// and the partial sums of F, so the election loss costs nothing extra on the step that also needs g.
//
// CTA (tile, worker) owns 64 rows I of X.  For every 64-row block J it forms the residual tile
// R = X_I X_J^T - M_IJ, adds R^2 to the loss, and accumulates G_I += R X_J.  R is never written to
// memory.  Products and sums are fp64 (the experiment is about reaching high accuracy and the problem is
// small), results are rounded once to fp32.
//
// Both products run on the fp64 matrix instruction (mma.sync m8n8k4, 256 fused multiply-adds per warp
// instruction; on this part it has the same peak as scalar fp64 arithmetic, 64 FMA per clock per SM, but needs
// one shared-memory operand per 8 FMAs of a thread instead of one per 2-4, which is what bounded the scalar
// version).  Fragment layout of the instruction, lane t: A[t/4][t%4], B[t%4][t/4], C[t/4][2(t%4) + {0,1}].
// 8 warps.  Product 1: warp w owns R's row blocks 2(w%4), 2(w%4)+1 and column blocks 4(w/4) .. +3 (blocks of 8);
// its C fragments start at -M, so R needs no separate subtraction, and rows or columns beyond n are zero in X
// and in M, hence zero in R.  Product 2: warp w owns G's row blocks 2(w%4), +1 and one half of G's column
// blocks.  The X tiles are converted to fp64 once when they are staged, zero-padded to the row pitch; the pitch
// of every shared array is 4 mod 8 doubles, which makes all fragment loads bank-conflict free.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int T = 64;            // tile edge
constexpr int NT = 256;          // threads per CTA
constexpr int RP = T + 4;        // pitch of the residual tile (doubles)

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1]) : "d"(a), "d"(b));
}

// NH = column blocks of G per warp (half of ceil(r / 8), rounded up to 1, 2, 4, 7 or 8): a compile-time bound
// on the accumulators a thread holds.
// Z = CTAs that share one row block (gridDim.z): CTA z takes the column blocks z, z + Z, ...  At small rank the
// time is the dependent chain over the column blocks, which only a shorter chain shortens; the Z partial
// gradients go to gpart[z][P][ld] in fp64 and psd_combine_kernel adds them in z order.  Z = 1 writes g itself.
template <int NH, int Z>
__global__ void __launch_bounds__(NT, Z > 1 ? 2 : 1)
psd_grad_kernel(const float* __restrict__ x, float* __restrict__ g, const float* __restrict__ M, int32_t n, int32_t r,
                int32_t pitch, int64_t ld, double* __restrict__ partials, int32_t n_partials, int write_g,
                double* __restrict__ gpart, int32_t P) {
  extern __shared__ double s_psd[];
  double* XI = s_psd;                           // [T][pitch]
  double* XJ = XI + T * pitch;                  // [T][pitch]
  double* Rt = XJ + T * pitch;                  // [T][RP]
  const int i = blockIdx.y, I0 = blockIdx.x * T;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, lr = lane >> 2, lc = lane & 3;
  const float* xi = x + (int64_t)i * ld;
  for (int idx = tid; idx < T * pitch; idx += NT) {
    const int row = idx / pitch, k = idx - row * pitch;
    XI[idx] = (k < r && I0 + row < n) ? (double)xi[(int64_t)(I0 + row) * r + k] : 0.0;
    XJ[idx] = 0.0;                              // the padding columns stay zero for the whole kernel
  }
  __syncthreads();                              // the zeros are in place before anybody stores a tile over them
  const int rb0 = (warp & 3) * 2;               // this warp's two row blocks (both products)
  const int cb0 = (warp >> 2) * 4;              // product 1: its four column blocks of R
  const int ncb = (r + 7) >> 3;                 // product 2: column blocks of G, split in two halves
  const int nhalf = (ncb + 1) >> 1;
  const int gcb0 = (warp >> 2) * nhalf;
  const int nmine = min(nhalf, ncb - gcb0);     // may be <= 0 for the second half at very small rank
  double acc[2][NH][2];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int m = 0; m < NH; ++m) acc[a][m][0] = acc[a][m][1] = 0.0;
  double lsum = 0.0;
  // The next block's operands -- this thread's 16 entries of M and its share of X_J -- are fetched into
  // registers while the current block is being worked on, so their latency is off the critical path.
  constexpr int NX = (T * 16 * NH + NT - 1) / NT;   // X_J values per thread (r <= 16 NH)
  float m_next[2][4][2], xj_next[NX];
  const int row0 = tid / r, col0 = tid - row0 * r;   // where element tid of a block sits, and the stride of NT elements
  const int drow = NT / r, dk = NT - drow * r;
  auto fetch = [&](int J0) {
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int ri = I0 + (rb0 + a) * 8 + lr, cj = J0 + (cb0 + b) * 8 + lc * 2 + q;
          m_next[a][b][q] = (ri < n && cj < n) ? M[(int64_t)ri * n + cj] : 0.f;
        }
    // the block is T * r consecutive floats of the worker's row; element tid + q NT sits in row (tid + q NT) / r
    const float* src = xi + (int64_t)J0 * r;
    int row = row0, k = col0;
#pragma unroll
    for (int q = 0; q < NX; ++q) {
      const int idx = tid + q * NT;
      xj_next[q] = (idx < T * r && J0 + row < n) ? src[idx] : 0.f;
      row += drow;
      k += dk;
      if (k >= r) {
        k -= r;
        ++row;
      }
    }
  };
  const int Jstep = T * Z;
  const int r4 = (r + 3) & ~3;
  fetch((int)blockIdx.z * T);
  for (int J0 = (int)blockIdx.z * T; J0 < n; J0 += Jstep) {
    double c[2][4][2];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        c[a][b][0] = -(double)m_next[a][b][0];
        c[a][b][1] = -(double)m_next[a][b][1];
      }
    {
      int row = row0, k = col0;
#pragma unroll
      for (int q = 0; q < NX; ++q) {
        if (tid + q * NT < T * r) XJ[row * pitch + k] = (double)xj_next[q];
        row += drow;
        k += dk;
        if (k >= r) {
          k -= r;
          ++row;
        }
      }
    }
    __syncthreads();
    if (J0 + Jstep < n) fetch(J0 + Jstep);
    // product 1: R = X_I X_J^T - M on this warp's 16 x 32 piece
    {
      const double* pa = XI + (rb0 * 8 + lr) * pitch + lc;
      const double* pb = XJ + (cb0 * 8 + lr) * pitch + lc;
      for (int k0 = 0; k0 < r4; k0 += 4) {
        double fa[2], fb[4];
#pragma unroll
        for (int a = 0; a < 2; ++a) fa[a] = pa[a * 8 * pitch + k0];
#pragma unroll
        for (int b = 0; b < 4; ++b) fb[b] = pb[b * 8 * pitch + k0];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) dmma(c[a][b], fa[a], fb[b]);
      }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        lsum = fma(c[a][b][0], c[a][b][0], lsum);
        lsum = fma(c[a][b][1], c[a][b][1], lsum);
        *reinterpret_cast<double2*>(Rt + ((rb0 + a) * 8 + lr) * RP + (cb0 + b) * 8 + lc * 2) = make_double2(c[a][b][0], c[a][b][1]);
      }
    asm volatile("bar.sync %0, 64;" ::"r"(1 + (warp & 3)) : "memory");   // warps w and w ^ 4: their rows of R are written
    // product 2: G_I += R X_J on this warp's 16 rows and its half of the columns
    if (nmine > 0) {
      const double* pa = Rt + (rb0 * 8 + lr) * RP + lc;
      const double* pb = XJ + lc * pitch + gcb0 * 8 + lr;
      for (int k0 = 0; k0 < T; k0 += 4) {
        double fa[2];
#pragma unroll
        for (int a = 0; a < 2; ++a) fa[a] = pa[a * 8 * RP + k0];
#pragma unroll
        for (int m = 0; m < NH; ++m) {
          if (m < nmine) {
            const double fb = pb[k0 * pitch + m * 8];
#pragma unroll
            for (int a = 0; a < 2; ++a) dmma(acc[a][m], fa[a], fb);
          }
        }
      }
    }
    __syncthreads();
  }
  if (write_g) {
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      const int ri = I0 + (rb0 + a) * 8 + lr;
      if (ri < n) {
        const int64_t row = (int64_t)i * ld + (int64_t)ri * r;
#pragma unroll
        for (int m = 0; m < NH; ++m)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int k = (gcb0 + m) * 8 + lc * 2 + q;
            if (m < nmine && k < r) {
              if (Z == 1) g[row + k] = (float)acc[a][m][q];
              else gpart[((int64_t)blockIdx.z * P) * ld + row + k] = acc[a][m][q];
            }
          }
      }
    }
  }
  // block sum of R^2 in a fixed order: warp shuffles, then the 8 warp sums in index order
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, o);
  __shared__ double s_w[NT / 32];
  if (lane == 0) s_w[warp] = lsum;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < NT / 32; ++w) t += s_w[w];
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
#ifndef LSGD_PSD_SPLIT_MAX_RANK
#define LSGD_PSD_SPLIT_MAX_RANK 32
#endif
// CTAs per row block: small ranks are latency-bound and split the column blocks (see psd_grad_kernel)
int32_t psd_split(int32_t r) { return r <= LSGD_PSD_SPLIT_MAX_RANK ? LSGD_PSD_SPLIT : 1; }

int32_t psd_loss_blocks(int32_t n, int32_t r) { return ((n + T - 1) / T) * psd_split(r); }

// Row pitch (doubles) of the staged X tiles: room for whole column blocks of 8, and 4 mod 8 so that the eight
// rows of an A / B fragment and the four rows of product 2's B fragment fall on distinct banks.
inline int psd_pitch(int r) {
  int p = ((r + 7) / 8) * 8;
  while (p % 8 != 4) p += 4;
  return p;
}

template <int NH, int Z>
cudaError_t launch_psd_t(const float* x, float* g, const float* M, int32_t n, int32_t r, int32_t P, int64_t ld, double* partials,
                         int32_t n_partials, int wg, double* gpart, cudaStream_t s) {
  const int pitch = psd_pitch(r);
  const size_t smem = sizeof(double) * (size_t)(2 * T * pitch + T * RP);
  static OncePerDevice attr;
  if (!attr.here()) {
    cudaError_t e = cudaFuncSetAttribute(psd_grad_kernel<NH, Z>, cudaFuncAttributeMaxDynamicSharedMemorySize, 180 * 1024);
    if (e == cudaSuccess && Z > 1)   // two CTAs per SM: ask for the largest shared-memory carve-out
      e = cudaFuncSetAttribute(psd_grad_kernel<NH, Z>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr.here() = true;
  }
  dim3 grid((unsigned)(n_partials / Z), (unsigned)P, (unsigned)Z);
  psd_grad_kernel<NH, Z><<<grid, NT, smem, s>>>(x, g, M, n, r, pitch, ld, partials, n_partials, wg, gpart, P);
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
  static_assert(LSGD_PSD_SPLIT_MAX_RANK >= 32, "ranks up to 32 always split");
  if (r <= 64) {
    if (psd_split(r) > 1) return launch_psd_t<4, ZS>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
    return launch_psd_t<4, 1>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
  }
  if (r <= 112) return launch_psd_t<7, 1>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
  return launch_psd_t<8, 1>(x, g, M, n, r, P, ld, partials, n_partials, wg, gpart, s);
}

}  // namespace lsgd
