// MLP population objective: a population of P three-layer ReLU classifiers trained with mean softmax
// cross-entropy, each worker on its own minibatch (the paper's deep-network setting, Section 4: every
// worker runs its own SGD on its own batches; here the networks are small dense MLPs).
//
// Parameter row = [W1 | b1 | W2 | b2 | W3 | b3], W_l stored [n_out][n_in].  All matrix products take
// bf16 operands and accumulate in fp32:
//   forward   H1 = relu(X W1^T + b1), H2 = relu(H1 W2^T + b2)            tensor cores (gemm_tc.cu)
//   head      Z = H2 W3^T + b3, loss, dZ, dH2; dW3, db3, db2, db1        CUDA cores (n_classes is tiny)
//   backward  dH1 = (dH2 W2) * [H1 > 0], dW2 = dH2^T H1, dW1 = dH1^T X   tensor cores
// Stored activations and back-propagated deltas are rounded to bf16 once, when they are written.
// The bf16 copy of the weights is refreshed by the update kernel itself when it writes x.
#include <cuda_bf16.h>

#include <cmath>
#include <new>

#include "gemm_tc.h"
#include "mlp.h"

namespace lsgd {
namespace {

constexpr int kMaxClasses = 16;
constexpr int kMaxLossWindow = 64;

inline int64_t up32(int64_t n) { return (n + 31) / 32 * 32; }
inline size_t up1k(size_t n) { return (n + 1023) & ~size_t(1023); }

struct Layout {
  int64_t w[3], b[3], d;
};
Layout param_layout(const int32_t* dims) {
  Layout L{};
  int64_t off = 0;
  for (int l = 0; l < 3; ++l) {
    L.w[l] = off;
    off = up32(off + (int64_t)dims[l] * dims[l + 1]);
    L.b[l] = off;
    off = up32(off + dims[l + 1]);
  }
  L.d = off;
  return L;
}

struct Scratch {
  size_t wb, xb, h1, h2, dh2, dh1, dz, loss_b, xh, hh1, hh2, loss_h, ring, logits, total;
};
Scratch scratch_layout(const int32_t* dims, int64_t ld, int32_t P, int32_t B, int32_t nH) {
  Scratch s{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += up1k(bytes); return o; };
  s.wb = take((size_t)P * ld * 2);
  s.xb = take((size_t)P * B * dims[0] * 2);
  s.h1 = take((size_t)P * B * dims[1] * 2);
  s.h2 = take((size_t)P * B * dims[2] * 2);
  s.dh2 = take((size_t)P * B * dims[2] * 2);
  s.dh1 = take((size_t)P * B * dims[1] * 2);
  s.dz = take((size_t)P * B * dims[3] * 4);
  s.loss_b = take((size_t)P * B * 4);
  s.xh = take((size_t)nH * dims[0] * 2);
  s.hh1 = take((size_t)P * nH * dims[1] * 2);
  s.hh2 = take((size_t)P * nH * dims[2] * 2);
  s.loss_h = take((size_t)P * nH * 4);
  s.ring = take((size_t)kMaxLossWindow * P * 4);
  s.logits = take((size_t)P * nH * kMaxClasses * 4);
  s.total = off;
  return s;
}

struct MlpState {
  Layout L;
  Scratch S;
  int32_t dims[4];
  int32_t B, nH, P;
  int64_t ld;
  __nv_bfloat16 *wb, *xb, *h1, *h2, *dh2, *dh1, *xh, *hh1, *hh2;
  float* logits;                         // held-out logits [P][nH][kMaxClasses] (fp32)
  float *dz, *loss_b, *loss_h, *ring;   // ring[slot][P]: mean minibatch loss of the last grads
  int64_t n_grads;
  CUtensorMap m_xb, m_w1, m_w2, m_w3, m_h1, m_dh2, m_dh1, m_xh, m_hh1, m_hh2;
};

// ------------------------------------------------------------------------------------ small kernels
__global__ void f32_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t n) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) dst[i] = __float2bfloat16_rn(src[i]);
}

// xb[row][:] = bf16(pool[idx[row]][:]); 16-byte loads, 8-byte stores (d0 is a multiple of 8)
__global__ void __launch_bounds__(128)
gather_rows_kernel(const float* __restrict__ pool, const int32_t* __restrict__ idx, __nv_bfloat16* __restrict__ xb,
                   int32_t rows_total, int32_t d0, int32_t pool_rows, uint32_t* status) {
  pdl_wait();
  pdl_launch_dependents();
  const int row = blockIdx.x;
  if (row >= rows_total) return;
  int src = idx[row];
  const bool bad = src < 0 || src >= pool_rows;
  if (bad) {
    if (threadIdx.x == 0) atomicOr(status, FLAG_BAD_INDEX);
    src = 0;
  }
  const float4* s4 = reinterpret_cast<const float4*>(pool + (int64_t)src * d0);
  uint2* o2 = reinterpret_cast<uint2*>(xb + (int64_t)row * d0);
  for (int k = threadIdx.x; k < (d0 >> 2); k += blockDim.x) {
    float4 v = __ldg(s4 + k);
    if (bad) v = make_float4(0.f, 0.f, 0.f, 0.f);
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    o2[k] = u;
  }
}

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 t = __bfloat1622float2(h[j]);
    f[2 * j] = t.x;
    f[2 * j + 1] = t.y;
  }
}

// A CTA stages W3 once in shared memory.  A warp takes S samples at a time, so each unpacked 16-byte piece
// of W3 is used S times: S = 1 for a training batch (most parallelism), S = 4 for the large held-out batch
// (the kernel is bound by unpacking W3, not by reading H2).
constexpr int kHeadWarps = 8;

// Last layer forward: logits Z = H2 W3^T + b3 from 16-byte (8 x bf16) loads, the softmax cross-entropy of
// each sample, and (training) dZ = (p - onehot) / n rounded to bf16.
template <int S>
__global__ void __launch_bounds__(kHeadWarps * 32)
head_forward_kernel(const __nv_bfloat16* __restrict__ h2, const __nv_bfloat16* __restrict__ wb, const float* __restrict__ x,
                    const int32_t* __restrict__ labels, const int32_t* __restrict__ label_idx, float* __restrict__ dz,
                    __nv_bfloat16* __restrict__ dh2, float* __restrict__ loss_b, int32_t n, int32_t d2, int32_t C, int64_t ld,
                    int64_t w3_off, int64_t b3_off, int32_t label_rows, int32_t groups_per_warp, uint32_t* status) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ uint4 s_w3[];   // [C][d2 / 8]
  const int i = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = d2 >> 3;
  const uint4* w3 = reinterpret_cast<const uint4*>(wb + (int64_t)i * ld + w3_off);
  for (int t = threadIdx.x; t < C * chunks; t += blockDim.x) s_w3[t] = w3[t];
  __syncthreads();
  const float* b3 = x + (int64_t)i * ld + b3_off;
  for (int grp = 0; grp < groups_per_warp; ++grp) {
    const int b0 = ((blockIdx.x * kHeadWarps + warp) * groups_per_warp + grp) * S;
    if (b0 >= n) break;
    float acc[S][kMaxClasses];
#pragma unroll
    for (int sx = 0; sx < S; ++sx)
#pragma unroll
      for (int c = 0; c < kMaxClasses; ++c) acc[sx][c] = 0.f;
    for (int ch = lane; ch < chunks; ch += 32) {
      float hv[S][8];
#pragma unroll
      for (int sx = 0; sx < S; ++sx) {
        const int b = b0 + sx < n ? b0 + sx : n - 1;
        unpack8(reinterpret_cast<const uint4*>(h2 + ((int64_t)i * n + b) * d2)[ch], hv[sx]);
      }
#pragma unroll
      for (int c = 0; c < kMaxClasses; ++c)
        if (c < C) {
          float wv[8];
          unpack8(s_w3[c * chunks + ch], wv);
#pragma unroll
          for (int sx = 0; sx < S; ++sx)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[sx][c] = fmaf(hv[sx][j], wv[j], acc[sx][c]);
        }
    }
#pragma unroll
    for (int sx = 0; sx < S; ++sx)
#pragma unroll
      for (int c = 0; c < kMaxClasses; ++c)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[sx][c] += __shfl_xor_sync(0xFFFFFFFFu, acc[sx][c], o);
    // Every lane holds all the reduced sums.  Held-out batch: lane sx finishes sample b0 + sx.  Training batch:
    // all lanes finish the sample together (the same arithmetic in every lane), lane sx stores the loss and dZ,
    // and the warp goes on to this sample's row of dH2 = [H2 > 0] * (dZ W3) while W3 is still in shared memory.
#pragma unroll
    for (int sx = 0; sx < S; ++sx) {
      const int b = b0 + sx;
      const bool writer = lane == sx;
      if ((writer || dh2 != nullptr) && b < n) {
        int y = label_idx ? label_idx[(int64_t)i * n + b] : b;   // training: pool row of this sample
        if (y < 0 || y >= label_rows) {
          if (writer) atomicOr(status, FLAG_BAD_INDEX);
          y = 0;
        }
        int cls = labels[y];
        if (cls < 0 || cls >= C) {
          if (writer) atomicOr(status, FLAG_BAD_INDEX);
          cls = 0;
        }
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < kMaxClasses; ++c)
          if (c < C) {
            acc[sx][c] += b3[c];
            zmax = fmaxf(zmax, acc[sx][c]);
          }
        float sum = 0.f, zy = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxClasses; ++c)
          if (c < C) {
            sum += expf(acc[sx][c] - zmax);
            if (c == cls) zy = acc[sx][c];
          }
        const float lse = zmax + logf(sum);
        if (writer) loss_b[(int64_t)i * n + b] = lse - zy;
        if (dz) {
          const float inv_n = 1.f / (float)n;
          float zr[kMaxClasses];          // dZ of this sample, rounded to bf16 as every back-propagated delta is
#pragma unroll
          for (int c = 0; c < kMaxClasses; ++c) {
            zr[c] = 0.f;
            if (c < C) {
              const float pc = expf(acc[sx][c] - lse);
              const float v = (pc - (c == cls ? 1.f : 0.f)) * inv_n;
              zr[c] = __bfloat162float(__float2bfloat16_rn(v));
              if (writer) dz[((int64_t)i * n + b) * C + c] = zr[c];
            }
          }
          if (dh2) {
            const uint4* hrow = reinterpret_cast<const uint4*>(h2 + ((int64_t)i * n + b) * d2);
            uint4* drow = reinterpret_cast<uint4*>(dh2 + ((int64_t)i * n + b) * d2);
            for (int ch = lane; ch < chunks; ch += 32) {
              float hv[8], dh[8];
              unpack8(hrow[ch], hv);
#pragma unroll
              for (int j = 0; j < 8; ++j) dh[j] = 0.f;
#pragma unroll
              for (int c = 0; c < kMaxClasses; ++c)
                if (c < C) {
                  float wv[8];
                  unpack8(s_w3[c * chunks + ch], wv);
#pragma unroll
                  for (int j = 0; j < 8; ++j) dh[j] = fmaf(zr[c], wv[j], dh[j]);
                }
              uint4 o;
              uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 r = __floats2bfloat162_rn(hv[2 * j] > 0.f ? dh[2 * j] : 0.f, hv[2 * j + 1] > 0.f ? dh[2 * j + 1] : 0.f);
                ow[j] = *reinterpret_cast<const uint32_t*>(&r);
              }
              drow[ch] = o;
            }
          }
        }
      }
    }
  }
}

constexpr int kDzPitch = kMaxClasses;

// Plain step of one parameter, the arithmetic of the update kernels (fp64 unfused / fp64 fused / fp32 fused).
__device__ __forceinline__ float sgd1(float x, float g, double eta, int arith) {
  if (arith == 0) return (float)__dsub_rn((double)x, __dmul_rn(eta, (double)g));
  if (arith == 1) return (float)fma(-eta, (double)g, (double)x);
  return fmaf(-(float)eta, g, x);
}

// Every gradient that is a sum over the batch of stored quantities, in one launch.  A CTA takes 128 columns of
// one worker and one of three jobs:
//   blocks [0, nb2)              : dW3[c][k] = sum_b dZ[b][c] H2[b][k]; block 0 also db3[c] = sum_b dZ[b][c];
//   blocks [nb2, 2 nb2)          : db2[k] = sum_b dH2[b][k];
//   blocks [2 nb2, 2 nb2 + nb1)  : db1[k] = sum_b dH1[b][k].
// Thread (k, s) owns columns 2k, 2k + 1 and the samples b = s, s + 8, ...; the slices are added in slice order.
// The kernel is all memory latency; two CTAs per SM with four loads in flight per thread measured best (more
// loads in flight cost registers, and spills or a single CTA per SM cost more than they gain).
// With sgd set the plain step x <- x - eta g of these parameters is taken here as well (x and its bf16 copy),
// so that nothing is left for a separate update launch.
constexpr int kBwdThreadsX = 64;   // each thread owns two adjacent columns (one bf16x2)
constexpr int kBwdCols = 2 * kBwdThreadsX;
constexpr int kBwdSlices = 8;      // batch slices per CTA (blockDim.y), combined in a fixed order
constexpr int kSumBatch = 4;       // samples whose loads a thread has in flight
__global__ void __launch_bounds__(kBwdThreadsX * kBwdSlices, 2)
batch_sums_kernel(const __nv_bfloat16* __restrict__ h2, const __nv_bfloat16* __restrict__ dh2, const __nv_bfloat16* __restrict__ dh1,
                  const float* __restrict__ dz, float* __restrict__ g, float* __restrict__ x, __nv_bfloat16* __restrict__ wb,
                  int32_t n, int32_t d1, int32_t d2, int32_t C, int64_t ld, int64_t w3_off, int64_t b3_off, int64_t b2_off,
                  int64_t b1_off, int32_t nb2, bool sgd, double eta, int arith) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(16) float s_mem[];
  float* s_dz = s_mem;                              // [n][kDzPitch], zero beyond C (job 0 only)
  float* s_red = s_mem + (size_t)n * kDzPitch;      // [kBwdSlices][rows][kBwdCols]
  const int i = blockIdx.y;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int tid = ty * kBwdThreadsX + tx;
  constexpr int kThreads = kBwdThreadsX * kBwdSlices;
  float* gi = g + (int64_t)i * ld;
  float* xi = x + (int64_t)i * ld;
  __nv_bfloat16* wi = wb + (int64_t)i * ld;
  const int job = (int)blockIdx.x < nb2 ? 0 : ((int)blockIdx.x < 2 * nb2 ? 1 : 2);
  const int blk = blockIdx.x - (job == 0 ? 0 : (job == 1 ? nb2 : 2 * nb2));
  const int dcols = job == 2 ? d1 : d2;
  const int rows = job == 0 ? C : 1;                // accumulator rows per column
  const __nv_bfloat16* src = (job == 0 ? h2 : (job == 1 ? dh2 : dh1)) + (int64_t)i * n * dcols;
  // where output (row c, column kcol) lives in the parameter row
  auto out_off = [&](int c, int kcol) -> int64_t {
    return job == 0 ? w3_off + (int64_t)c * d2 + kcol : (job == 1 ? b2_off : b1_off) + kcol;
  };
  // the x values the plain step will need: fetched now, used at the very end
  constexpr int kMaxOut = (kMaxClasses * kBwdCols + kThreads - 1) / kThreads;
  float x_old[kMaxOut];
#pragma unroll
  for (int u = 0; u < kMaxOut; ++u) {
    const int t = tid + u * kThreads;
    const int c = t / kBwdCols, kcol = blk * kBwdCols + (t - c * kBwdCols);
    x_old[u] = (sgd && c < rows && kcol < dcols) ? xi[out_off(c, kcol)] : 0.f;
  }
  if (job == 0) {
    const float* dzi = dz + (int64_t)i * n * C;
    for (int t = tid; t < n * kDzPitch; t += kThreads) {
      const int b = t / kDzPitch, c = t - b * kDzPitch;
      s_dz[t] = c < C ? dzi[b * C + c] : 0.f;
    }
    __syncthreads();
    if (blk == 0 && tid < C) {
      float sum = 0.f;
      for (int b = 0; b < n; ++b) sum += s_dz[b * kDzPitch + tid];
      gi[b3_off + tid] = sum;
      if (sgd) {
        const float xn = sgd1(xi[b3_off + tid], sum, eta, arith);
        xi[b3_off + tid] = xn;
        wi[b3_off + tid] = __float2bfloat16_rn(xn);
      }
    }
  }
  const int k = blk * kBwdCols + 2 * tx;            // layer widths are even: k and k + 1 are both valid or both not
  const bool live = k < dcols;
  float a0[kMaxClasses], a1[kMaxClasses];
#pragma unroll
  for (int c = 0; c < kMaxClasses; ++c) {
    a0[c] = 0.f;
    a1[c] = 0.f;
  }
  if (live) {
    const __nv_bfloat16* col = src + k;
    for (int b0 = ty; b0 < n; b0 += kSumBatch * kBwdSlices) {
      uint32_t raw[kSumBatch];
#pragma unroll
      for (int u = 0; u < kSumBatch; ++u) {
        const int b = b0 + u * kBwdSlices;
        raw[u] = b < n ? *reinterpret_cast<const uint32_t*>(col + (int64_t)b * dcols) : 0u;
      }
#pragma unroll
      for (int u = 0; u < kSumBatch; ++u) {
        const int b = b0 + u * kBwdSlices;
        if (b < n) {
          const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw[u]));
          if (job == 0) {
#pragma unroll
            for (int q = 0; q < kMaxClasses / 4; ++q) {
              if (4 * q < C) {      // entries beyond C are zero in s_dz
                const float4 t = *reinterpret_cast<const float4*>(s_dz + b * kDzPitch + 4 * q);
                a0[4 * q] = fmaf(t.x, v.x, a0[4 * q]);         a1[4 * q] = fmaf(t.x, v.y, a1[4 * q]);
                a0[4 * q + 1] = fmaf(t.y, v.x, a0[4 * q + 1]); a1[4 * q + 1] = fmaf(t.y, v.y, a1[4 * q + 1]);
                a0[4 * q + 2] = fmaf(t.z, v.x, a0[4 * q + 2]); a1[4 * q + 2] = fmaf(t.z, v.y, a1[4 * q + 2]);
                a0[4 * q + 3] = fmaf(t.w, v.x, a0[4 * q + 3]); a1[4 * q + 3] = fmaf(t.w, v.y, a1[4 * q + 3]);
              }
            }
          } else {
            a0[0] += v.x;
            a1[0] += v.y;
          }
        }
      }
    }
  }
  float* red = s_red + (size_t)ty * rows * kBwdCols;
#pragma unroll
  for (int c = 0; c < kMaxClasses; ++c)
    if (c < rows) {
      red[c * kBwdCols + 2 * tx] = a0[c];
      red[c * kBwdCols + 2 * tx + 1] = a1[c];
    }
  __syncthreads();
  // rows x kBwdCols sums over the slices, in slice order
#pragma unroll
  for (int u = 0; u < kMaxOut; ++u) {
    const int t = tid + u * kThreads;
    const int c = t / kBwdCols, kk = t - c * kBwdCols;
    const int kcol = blk * kBwdCols + kk;
    if (c >= rows || kcol >= dcols) continue;
    float acc = 0.f;
    for (int sl = 0; sl < kBwdSlices; ++sl) acc += s_red[((size_t)sl * rows + c) * kBwdCols + kk];
    const int64_t off = out_off(c, kcol);
    gi[off] = acc;
    if (sgd) {
      const float xn = sgd1(x_old[u], acc, eta, arith);
      xi[off] = xn;
      wi[off] = __float2bfloat16_rn(xn);
    }
  }
}

// Per-sample softmax cross-entropy from stored logits (+ bias): one thread per sample.
__global__ void __launch_bounds__(256)
logits_loss_kernel(const float* __restrict__ logits, const float* __restrict__ x, const int32_t* __restrict__ labels,
                   float* __restrict__ loss_b, int32_t n, int32_t C, int64_t ld, int64_t b3_off, uint32_t* status) {
  const int i = blockIdx.y;
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= n) return;
  const float* z = logits + ((int64_t)i * n + b) * kMaxClasses;
  const float* b3 = x + (int64_t)i * ld + b3_off;
  int cls = labels[b];
  if (cls < 0 || cls >= C) {
    atomicOr(status, FLAG_BAD_INDEX);
    cls = 0;
  }
  float v[kMaxClasses];
  float zmax = -INFINITY;
#pragma unroll
  for (int c = 0; c < kMaxClasses; ++c)
    if (c < C) {
      v[c] = z[c] + b3[c];
      zmax = fmaxf(zmax, v[c]);
    }
  float sum = 0.f, zy = 0.f;
#pragma unroll
  for (int c = 0; c < kMaxClasses; ++c)
    if (c < C) {
      sum += expf(v[c] - zmax);
      if (c == cls) zy = v[c];
    }
  loss_b[(int64_t)i * n + b] = zmax + logf(sum) - zy;
}

// out[i] = mean over the first n_slots rows of ring[slot][i], added in slot order in fp64
__global__ void window_mean_kernel(const float* __restrict__ ring, float* __restrict__ out, int32_t P, int32_t n_slots) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= P) return;
  double acc = 0.0;
  for (int sl = 0; sl < n_slots; ++sl) acc += (double)ring[(int64_t)sl * P + i];
  out[i] = (float)(acc / (double)n_slots);
}

// out[i] = mean_b v[i][b], summed in a fixed order by one warp per worker.
__global__ void __launch_bounds__(32) row_mean_kernel(const float* __restrict__ v, float* __restrict__ out, int32_t n) {
  pdl_wait();
  pdl_launch_dependents();
  const int i = blockIdx.x, lane = threadIdx.x;
  double acc = 0.0;
  for (int b = lane; b < n; b += 32) acc += (double)v[(int64_t)i * n + b];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (lane == 0) out[i] = (float)(acc / (double)n);
}

MlpState* state(lsgd_ctx* h) { return static_cast<MlpState*>(h->mlp_state); }

GemmShape shape(int M, int N, int K, int batch, int a_mn, int b_mn, int a_batched, int epi, void* c, int64_t ldc,
                int64_t stride_c, uint32_t* status) {
  GemmShape g{};
  g.M = M; g.N = N; g.K = K; g.batch = batch;
  g.a_mn = a_mn; g.b_mn = b_mn; g.a_batched = a_batched; g.b_batched = 1;
  g.epilogue = epi; g.c = c; g.ldc = ldc; g.stride_c = stride_c; g.status = status;
  return g;
}

lsgd_status forward_hidden(lsgd_ctx* h, const CUtensorMap& m_in, int a_batched, int n, __nv_bfloat16* o1, const CUtensorMap& m_o1,
                           __nv_bfloat16* o2) {
  MlpState* st = state(h);
  const lsgd_config& c = h->cfg;
  const int32_t* d = st->dims;
  GemmShape g1 = shape(n, d[1], d[0], st->P, 0, 0, a_batched, GEMM_EPI_BIAS_RELU_BF16, o1, d[1], (int64_t)n * d[1], h->d_status);
  g1.bias = c.x + st->L.b[0];
  g1.stride_bias = st->ld;
  if (launch_bgemm(m_in, st->m_w1, g1, h->stream) != cudaSuccess) return LSGD_ERR_CUDA;
  GemmShape g2 = shape(n, d[2], d[1], st->P, 0, 0, 1, GEMM_EPI_BIAS_RELU_BF16, o2, d[2], (int64_t)n * d[2], h->d_status);
  g2.bias = c.x + st->L.b[1];
  g2.stride_bias = st->ld;
  if (launch_bgemm(m_o1, st->m_w2, g2, h->stream) != cudaSuccess) return LSGD_ERR_CUDA;
  return LSGD_OK;
}

}  // namespace

lsgd_status mlp_validate(const lsgd_config& c, const lsgd_mlp_desc& m) {
  for (int l = 0; l < 4; ++l)
    if (m.dims[l] < 1) return LSGD_ERR_INVALID_ARG;
  if (m.batch < 1 || m.pool < 1 || m.n_heldout < 1) return LSGD_ERR_INVALID_ARG;
  if (m.loss_window < 0 || m.loss_window > kMaxLossWindow) return LSGD_ERR_INVALID_ARG;
  if (!m.pool_x || !m.pool_y || !m.held_x || !m.held_y || !m.scratch) return LSGD_ERR_INVALID_ARG;
  // TMA rows must be 16-byte multiples (8 bf16); the head kernels keep the class scores in registers
  if (m.dims[0] % 8 || m.dims[1] % 8 || m.dims[2] % 8 || m.dims[3] > kMaxClasses) return LSGD_ERR_UNSUPPORTED;
  if (m.batch % 8 || m.n_heldout % 8 || m.batch > 1024) return LSGD_ERR_UNSUPPORTED;
  // shared-memory budgets of the last-layer kernels (48 KB without opting in)
  if ((size_t)m.dims[3] * m.dims[2] * 2 > 48 * 1024) return LSGD_ERR_UNSUPPORTED;
  if (sizeof(float) * ((size_t)m.batch * kDzPitch + (size_t)8 * m.dims[3] * 128) > 160 * 1024) return LSGD_ERR_UNSUPPORTED;
  const Layout L = param_layout(m.dims);
  if (L.d != c.d || c.ld != c.d) return LSGD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(m.scratch) & 1023u) return LSGD_ERR_ALIGNMENT;
  if (m.scratch_bytes < lsgd_mlp_scratch_bytes(m.dims, c.P, m.batch, m.n_heldout)) return LSGD_ERR_INVALID_ARG;
  return LSGD_OK;
}

lsgd_status mlp_create(lsgd_ctx* h) {
  const lsgd_config& c = h->cfg;
  const lsgd_mlp_desc& m = h->mlp;
  MlpState* st = new (std::nothrow) MlpState();
  if (!st) return LSGD_ERR_INVALID_ARG;
  h->mlp_state = st;
  for (int l = 0; l < 4; ++l) st->dims[l] = m.dims[l];
  st->L = param_layout(m.dims);
  st->B = m.batch;
  st->nH = m.n_heldout;
  st->P = c.P;
  st->ld = c.ld;
  st->S = scratch_layout(m.dims, c.ld, c.P, m.batch, m.n_heldout);
  char* base = static_cast<char*>(m.scratch);
  st->wb = reinterpret_cast<__nv_bfloat16*>(base + st->S.wb);
  st->xb = reinterpret_cast<__nv_bfloat16*>(base + st->S.xb);
  st->h1 = reinterpret_cast<__nv_bfloat16*>(base + st->S.h1);
  st->h2 = reinterpret_cast<__nv_bfloat16*>(base + st->S.h2);
  st->dh2 = reinterpret_cast<__nv_bfloat16*>(base + st->S.dh2);
  st->dh1 = reinterpret_cast<__nv_bfloat16*>(base + st->S.dh1);
  st->dz = reinterpret_cast<float*>(base + st->S.dz);
  st->loss_b = reinterpret_cast<float*>(base + st->S.loss_b);
  st->xh = reinterpret_cast<__nv_bfloat16*>(base + st->S.xh);
  st->hh1 = reinterpret_cast<__nv_bfloat16*>(base + st->S.hh1);
  st->hh2 = reinterpret_cast<__nv_bfloat16*>(base + st->S.hh2);
  st->loss_h = reinterpret_cast<float*>(base + st->S.loss_h);
  st->ring = reinterpret_cast<float*>(base + st->S.ring);
  st->logits = reinterpret_cast<float*>(base + st->S.logits);
  st->n_grads = 0;

  const int32_t* d = st->dims;
  const int64_t B = st->B, nH = st->nH, P = st->P, ld = st->ld;
  bool ok = true;
  ok = ok && make_operand_map(&st->m_xb, st->xb, d[0], B, d[0], P, B * d[0]);
  ok = ok && make_operand_map(&st->m_w1, st->wb + st->L.w[0], d[0], d[1], d[0], P, ld);
  ok = ok && make_operand_map(&st->m_w2, st->wb + st->L.w[1], d[1], d[2], d[1], P, ld);
  ok = ok && make_operand_map(&st->m_h1, st->h1, d[1], B, d[1], P, B * d[1]);
  ok = ok && make_operand_map(&st->m_dh2, st->dh2, d[2], B, d[2], P, B * d[2]);
  ok = ok && make_operand_map(&st->m_dh1, st->dh1, d[1], B, d[1], P, B * d[1]);
  ok = ok && make_operand_map(&st->m_xh, st->xh, d[0], nH, d[0], 1, 0);
  ok = ok && make_operand_map(&st->m_hh1, st->hh1, d[1], nH, d[1], P, nH * d[1]);
  ok = ok && make_operand_map(&st->m_hh2, st->hh2, d[2], nH, d[2], P, nH * d[2]);
  ok = ok && make_operand_map(&st->m_w3, st->wb + st->L.w[2], d[2], d[3], d[2], P, ld);
  if (!ok) return LSGD_ERR_CUDA;

  // bf16 copies of the weights and of the held-out inputs; gradient padding cleared once
  f32_to_bf16_kernel<<<148 * 8, 256, 0, h->stream>>>(c.x, st->wb, (int64_t)P * ld);
  f32_to_bf16_kernel<<<148 * 2, 256, 0, h->stream>>>(m.held_x, st->xh, (int64_t)nH * d[0]);
  if (cudaGetLastError() != cudaSuccess) return LSGD_ERR_CUDA;
  if (cudaMemsetAsync(c.g, 0, sizeof(float) * (size_t)P * (size_t)ld, h->stream) != cudaSuccess) return LSGD_ERR_CUDA;
  return LSGD_OK;
}

lsgd_status mlp_grad(lsgd_ctx* h, const int32_t* batch_idx, bool fuse_sgd) {
  MlpState* st = state(h);
  const lsgd_config& c = h->cfg;
  const lsgd_mlp_desc& m = h->mlp;
  const int32_t* d = st->dims;
  const int B = st->B, P = st->P;
  const int64_t ld = st->ld;
  cudaStream_t s = h->stream;

  if (launch_pdl(gather_rows_kernel, dim3(P * B), dim3(128), 0, s, m.pool_x, batch_idx, st->xb, P * B, d[0], m.pool,
                 h->d_status) != cudaSuccess)
    return LSGD_ERR_CUDA;
  lsgd_status fs = forward_hidden(h, st->m_xb, 1, B, st->h1, st->m_h1, st->h2);
  if (fs != LSGD_OK) return fs;

  const size_t w3_smem = (size_t)d[3] * d[2] * 2;
  if (launch_pdl(head_forward_kernel<1>, dim3((B + kHeadWarps - 1) / kHeadWarps, P), dim3(kHeadWarps * 32), w3_smem, s,
                 st->h2, st->wb, c.x, m.pool_y, batch_idx, st->dz, st->dh2, st->loss_b, B, d[2], d[3], ld, st->L.w[2],
                 st->L.b[2], m.pool, 1, h->d_status) != cudaSuccess)
    return LSGD_ERR_CUDA;
  if (m.loss_window > 0) {   // remember this step's mean minibatch losses for the running-mean election
    if (launch_pdl(row_mean_kernel, dim3(P), dim3(32), 0, s, st->loss_b, st->ring + (st->n_grads % m.loss_window) * P,
                   B) != cudaSuccess)
      return LSGD_ERR_CUDA;
    st->n_grads++;
  }

  // dH1 = (dH2 . W2) masked by H1 > 0        [B x d1] = [B x d2] . [d2 x d1]
  GemmShape gd = shape(B, d[1], d[2], P, 0, 1, 1, GEMM_EPI_MASK_BF16, st->dh1, d[1], (int64_t)B * d[1], h->d_status);
  gd.mask = st->h1;
  gd.ld_mask = d[1];
  gd.stride_mask = (int64_t)B * d[1];
  if (launch_bgemm(st->m_dh2, st->m_w2, gd, s) != cudaSuccess) return LSGD_ERR_CUDA;
  // dW3, db3, db2, db1: the sums over the batch (and, fused, the plain step of those parameters)
  const size_t sums_smem = sizeof(float) * ((size_t)B * kDzPitch + (size_t)kBwdSlices * d[3] * kBwdCols);
  static OncePerDevice sums_attr;
  if (!sums_attr.here()) {
    if (cudaFuncSetAttribute(batch_sums_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024) != cudaSuccess)
      return LSGD_ERR_CUDA;
    // two CTAs per SM: ask for the largest shared-memory carve-out (the default fits one CTA only)
    if (cudaFuncSetAttribute(batch_sums_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) !=
        cudaSuccess)
      return LSGD_ERR_CUDA;
    sums_attr.here() = true;
  }
  const int nb2 = (d[2] + kBwdCols - 1) / kBwdCols, nb1 = (d[1] + kBwdCols - 1) / kBwdCols;
  if (launch_pdl(batch_sums_kernel, dim3(2 * nb2 + nb1, P), dim3(kBwdThreadsX, kBwdSlices), sums_smem, s, st->h2, st->dh2, st->dh1,
                 st->dz, c.g, c.x, st->wb, B, d[1], d[2], d[3], ld, st->L.w[2], st->L.b[2], st->L.b[1], st->L.b[0], nb2, fuse_sgd,
                 (double)c.eta, (int)c.arithmetic) != cudaSuccess)
    return LSGD_ERR_CUDA;
  // dW2 = dH2^T . H1                          [d2 x d1], contraction over the batch
  GemmShape g2 = shape(d[2], d[1], B, P, 1, 1, 1, fuse_sgd ? GEMM_EPI_SGD : GEMM_EPI_F32, c.g + st->L.w[1], d[1], ld, h->d_status);
  g2.x_upd = c.x + st->L.w[1];
  g2.x_shadow = reinterpret_cast<uint16_t*>(st->wb) + st->L.w[1];
  g2.eta = (double)c.eta;
  g2.arith = c.arithmetic;
  if (launch_bgemm(st->m_dh2, st->m_h1, g2, s) != cudaSuccess) return LSGD_ERR_CUDA;
  // dW1 = dH1^T . X                           [d1 x d0]
  GemmShape g1 = shape(d[1], d[0], B, P, 1, 1, 1, fuse_sgd ? GEMM_EPI_SGD : GEMM_EPI_F32, c.g + st->L.w[0], d[0], ld, h->d_status);
  g1.x_upd = c.x + st->L.w[0];
  g1.x_shadow = reinterpret_cast<uint16_t*>(st->wb) + st->L.w[0];
  g1.eta = (double)c.eta;
  g1.arith = c.arithmetic;
  if (launch_bgemm(st->m_dh1, st->m_xb, g1, s) != cudaSuccess) return LSGD_ERR_CUDA;
  return LSGD_OK;
}

lsgd_status mlp_heldout_loss(lsgd_ctx* h, float* loss) {
  MlpState* st = state(h);
  const lsgd_config& c = h->cfg;
  const lsgd_mlp_desc& m = h->mlp;
  const int32_t* d = st->dims;
  lsgd_status fs = forward_hidden(h, st->m_xh, 0, st->nH, st->hh1, st->m_hh1, st->hh2);
  if (fs != LSGD_OK) return fs;
  if (st->nH >= 512) {
    // large held-out batch: the logits are one more tensor-core product (N = n_classes, zero-filled to a
    // tile by TMA), followed by a per-sample softmax
    GemmShape g3 = shape(st->nH, d[3], d[2], st->P, 0, 0, 1, GEMM_EPI_F32, st->logits, kMaxClasses,
                         (int64_t)st->nH * kMaxClasses, h->d_status);
    if (launch_bgemm(st->m_hh2, st->m_w3, g3, h->stream) != cudaSuccess) return LSGD_ERR_CUDA;
    logits_loss_kernel<<<dim3((st->nH + 255) / 256, st->P), 256, 0, h->stream>>>(st->logits, c.x, m.held_y, st->loss_h, st->nH,
                                                                              d[3], st->ld, st->L.b[2], h->d_status);
  } else {
    constexpr int kS = 4, kGroups = 2;   // 8 warps x 2 groups x 4 samples = 64 samples per CTA
    const int per_cta = kHeadWarps * kGroups * kS;
    head_forward_kernel<kS><<<dim3((st->nH + per_cta - 1) / per_cta, st->P), kHeadWarps * 32, (size_t)d[3] * d[2] * 2, h->stream>>>(
        st->hh2, st->wb, c.x, m.held_y, nullptr, nullptr, nullptr, st->loss_h, st->nH, d[2], d[3], st->ld, st->L.w[2], st->L.b[2],
        st->nH, kGroups, h->d_status);
  }
  row_mean_kernel<<<st->P, 32, 0, h->stream>>>(st->loss_h, loss, st->nH);
  return cudaGetLastError() == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}

lsgd_status mlp_window_loss(lsgd_ctx* h, float* loss) {
  MlpState* st = state(h);
  const int K = h->mlp.loss_window;
  if (!st || K < 1 || st->n_grads < 1) return LSGD_ERR_STATE;   // nothing recorded yet
  const int n_slots = st->n_grads < K ? (int)st->n_grads : K;
  window_mean_kernel<<<(st->P + 127) / 128, 128, 0, h->stream>>>(st->ring, loss, st->P, n_slots);
  return cudaGetLastError() == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}

lsgd_status mlp_train_loss(lsgd_ctx* h, float* loss) {
  MlpState* st = state(h);
  if (!st) return LSGD_ERR_STATE;
  row_mean_kernel<<<st->P, 32, 0, h->stream>>>(st->loss_b, loss, st->B);
  return cudaGetLastError() == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}

lsgd_status mlp_get_activations(lsgd_ctx* h, uint16_t* h1, uint16_t* h2) {
  MlpState* st = state(h);
  if (!st) return LSGD_ERR_STATE;
  if (cudaStreamSynchronize(h->stream) != cudaSuccess) return LSGD_ERR_CUDA;
  const size_t n1 = (size_t)st->P * st->B * st->dims[1], n2 = (size_t)st->P * st->B * st->dims[2];
  if (h1 && cudaMemcpy(h1, st->h1, n1 * sizeof(uint16_t), cudaMemcpyDeviceToHost) != cudaSuccess) return LSGD_ERR_CUDA;
  if (h2 && cudaMemcpy(h2, st->h2, n2 * sizeof(uint16_t), cudaMemcpyDeviceToHost) != cudaSuccess) return LSGD_ERR_CUDA;
  return LSGD_OK;
}

int mlp_unfused_ranges(lsgd_ctx* h, int64_t (*ranges)[2]) {
  // none: W1, W2 are stepped in the weight-gradient products, the biases and W3 in the batch-sum kernel
  (void)h;
  (void)ranges;
  return 0;
}

lsgd_status mlp_refresh_shadow(lsgd_ctx* h) {
  MlpState* st = state(h);
  if (!st) return LSGD_ERR_STATE;
  f32_to_bf16_kernel<<<148 * 8, 256, 0, h->stream>>>(h->cfg.x, st->wb, (int64_t)st->P * st->ld);
  return cudaGetLastError() == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}

uint16_t* mlp_weight_shadow(lsgd_ctx* h) { return h->mlp_state ? reinterpret_cast<uint16_t*>(state(h)->wb) : nullptr; }

void mlp_destroy(lsgd_ctx* h) {
  delete state(h);
  h->mlp_state = nullptr;
}

}  // namespace lsgd

extern "C" {

lsgd_status lsgd_mlp_param_offsets(const int32_t* dims, int64_t* w_off, int64_t* b_off, int64_t* d_out) {
  if (!dims || !w_off || !b_off || !d_out) return LSGD_ERR_INVALID_ARG;
  for (int l = 0; l < 4; ++l)
    if (dims[l] < 1) return LSGD_ERR_INVALID_ARG;
  const lsgd::Layout L = lsgd::param_layout(dims);
  for (int l = 0; l < 3; ++l) {
    w_off[l] = L.w[l];
    b_off[l] = L.b[l];
  }
  *d_out = L.d;
  return LSGD_OK;
}

uint64_t lsgd_mlp_scratch_bytes(const int32_t* dims, int32_t P, int32_t batch, int32_t n_heldout) {
  if (!dims || P < 1 || batch < 1 || n_heldout < 1) return 0;
  for (int l = 0; l < 4; ++l)
    if (dims[l] < 1) return 0;
  const lsgd::Layout L = lsgd::param_layout(dims);
  return lsgd::scratch_layout(dims, L.d, P, batch, n_heldout).total;
}

// Status word of the stand-alone product, one per device, allocated on the first use on that device.
static uint32_t* bgemm_status_word() {
  static uint32_t* words[lsgd::kMaxDevices] = {};
  uint32_t*& w = words[lsgd::device_slot()];
  if (!w) {
    if (cudaMalloc(&w, sizeof(uint32_t)) != cudaSuccess) {
      w = nullptr;
      return nullptr;
    }
    cudaMemset(w, 0, sizeof(uint32_t));
  }
  return w;
}

lsgd_status lsgd_bgemm_check_device(uint32_t* flag_out) {
  uint32_t* status = bgemm_status_word();
  if (!status) return LSGD_ERR_CUDA;
  uint32_t f = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return LSGD_ERR_CUDA;
  if (cudaMemcpy(&f, status, sizeof(f), cudaMemcpyDeviceToHost) != cudaSuccess) return LSGD_ERR_CUDA;
  if (f && cudaMemset(status, 0, sizeof(f)) != cudaSuccess) return LSGD_ERR_CUDA;
  if (flag_out) *flag_out = f;
  return f ? LSGD_ERR_DEVICE_FLAG : LSGD_OK;
}

lsgd_status lsgd_bgemm_bf16(const lsgd_bgemm_desc* g, void* stream) {
  using namespace lsgd;
  if (!g || !g->a || !g->b || !g->c) return LSGD_ERR_INVALID_ARG;
  if (g->M < 1 || g->N < 1 || g->K < 1 || g->batch < 1 || g->epilogue < 0 || g->epilogue > 3) return LSGD_ERR_INVALID_ARG;
  if (g->epilogue == GEMM_EPI_BIAS_RELU_BF16 && !g->bias) return LSGD_ERR_INVALID_ARG;
  if (g->epilogue == GEMM_EPI_MASK_BF16 && !g->mask) return LSGD_ERR_INVALID_ARG;
  uint32_t* status = bgemm_status_word();   // status word of the stand-alone entry point (per device)
  if (!status) return LSGD_ERR_CUDA;
  CUtensorMap ma, mb;
  const int64_t a_inner = g->a_mn_major ? g->M : g->K, a_outer = g->a_mn_major ? g->K : g->M;
  const int64_t b_inner = g->b_mn_major ? g->N : g->K, b_outer = g->b_mn_major ? g->K : g->N;
  if (!make_operand_map(&ma, g->a, a_inner, a_outer, g->lda, g->stride_a ? g->batch : 1, g->stride_a)) return LSGD_ERR_ALIGNMENT;
  if (!make_operand_map(&mb, g->b, b_inner, b_outer, g->ldb, g->stride_b ? g->batch : 1, g->stride_b)) return LSGD_ERR_ALIGNMENT;
  GemmShape p{};
  p.M = g->M; p.N = g->N; p.K = g->K; p.batch = g->batch;
  p.a_mn = g->a_mn_major ? 1 : 0; p.b_mn = g->b_mn_major ? 1 : 0;
  p.a_batched = g->stride_a ? 1 : 0; p.b_batched = g->stride_b ? 1 : 0;
  p.epilogue = g->epilogue; p.c = g->c; p.ldc = g->ldc; p.stride_c = g->stride_c;
  p.bias = g->bias; p.stride_bias = g->stride_bias;
  p.mask = g->mask; p.ld_mask = g->ld_mask; p.stride_mask = g->stride_mask;
  p.status = status;
  if (launch_bgemm(ma, mb, p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return LSGD_ERR_CUDA;
  return LSGD_OK;
}

}  // extern "C"
