// The LSGD step with the optimiser of the paper's deep-network runs (Section 4.1: Nesterov momentum and
// weight decay for every method), on top of Eq. (1):
//
//     d  = g + wd x,    v+ = mu v + d,    u = d + mu v+,
//     x+ = x - eta u  [ - eta lambda_l (x - x_ll) - eta lambda_g (x - x_gl)   on a pull step ].
//
// The pulls stay outside the momentum buffer, so mu = wd = 0 is Eq. (1) again.  Same ownership rule as
// the plain kernels: a thread owns one 16-byte column (4 parameters) for ALL P workers; on a pull step it
// reads the global leader's and each group's local leader's values into registers before any row of the
// column is rewritten, so every right-hand side is x at time t.  Per worker-parameter the kernel reads
// x, g, v and writes x, v: 20 bytes.
#include <cuda_bf16.h>

#include "internal.h"

namespace lsgd {
namespace {

constexpr int kThreads = 256;
constexpr int kRows = 2;   // rows whose loads are issued before the first is consumed

__device__ __forceinline__ float4 ld4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }
__device__ __forceinline__ void st4_bf16(uint16_t* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

// One parameter.  MODE 0: fp64, one IEEE operation per written operation, one rounding per stored value
// (what a plain double-precision restatement produces); 1: fp64 with fused multiply-adds; 2: fp32 FMAs.
template <int MODE, bool PULL>
__device__ __forceinline__ void step1(float x, float g, float v, float xl, float xg, const Coef& k, float& x_new, float& v_new) {
  if (MODE == 0) {
    const double X = (double)x;
    const double D = __dadd_rn((double)g, __dmul_rn(k.wd, X));
    const double VN = __dadd_rn(__dmul_rn(k.mu, (double)v), D);
    const double U = __dadd_rn(D, __dmul_rn(k.mu, VN));
    double acc = __dsub_rn(X, __dmul_rn(k.eta, U));
    if (PULL) {
      acc = __dsub_rn(acc, __dmul_rn(k.cl, __dsub_rn(X, (double)xl)));
      acc = __dsub_rn(acc, __dmul_rn(k.cg, __dsub_rn(X, (double)xg)));
    }
    x_new = (float)acc;
    v_new = (float)VN;
  } else if (MODE == 1) {
    const double X = (double)x;
    const double D = fma(k.wd, X, (double)g);
    const double VN = fma(k.mu, (double)v, D);
    const double U = fma(k.mu, VN, D);
    double acc = fma(-k.eta, U, X);
    if (PULL) {
      acc = fma(-k.cl, X - (double)xl, acc);
      acc = fma(-k.cg, X - (double)xg, acc);
    }
    x_new = (float)acc;
    v_new = (float)VN;
  } else {
    const float D = fmaf(k.wd_f, x, g);
    const float VN = fmaf(k.mu_f, v, D);
    const float U = fmaf(k.mu_f, VN, D);
    float acc = fmaf(-k.eta_f, U, x);
    if (PULL) {
      acc = fmaf(-k.cl_f, x - xl, acc);
      acc = fmaf(-k.cg_f, x - xg, acc);
    }
    x_new = acc;
    v_new = VN;
  }
}

template <int MODE, bool PULL, bool SHADOW>
__global__ void __launch_bounds__(kThreads, 4)
momentum_update_kernel(UpdateArgs p, int64_t n4) {
  extern __shared__ int32_t s_tab[];
  int32_t* s_ll = s_tab;                 // [G]
  int32_t* s_start = s_ll + p.G;         // [G+1]
  int32_t* s_rows = s_start + p.G + 1;   // [P]
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  int gl = 0;
  if (PULL) {
    for (int k = threadIdx.x; k < p.G; k += blockDim.x) {
      const int l = p.ll[k];
      if (l < 0 || l >= p.P) s_bad = 1;
      s_ll[k] = l;
    }
    gl = *p.gl;
    if (threadIdx.x == 0 && (gl < 0 || gl >= p.P)) s_bad = 1;
  }
  for (int k = threadIdx.x; k <= p.G; k += blockDim.x) s_start[k] = p.tab.group_start[k];
  for (int k = threadIdx.x; k < p.P; k += blockDim.x) s_rows[k] = p.tab.rows_by_group[k];
  __syncthreads();
  if (s_bad) {  // never dereference a leader index that is out of range
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(p.status, FLAG_BAD_LEADER);
    return;
  }
  const Coef k = p.k;
  const int64_t ld = p.ld;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n4; c += stride) {
    const int64_t col = c * 4;
    float* xc = p.x + col;
    float* vc = p.v + col;
    const float* gc = p.g + col;
    float4 xg = make_float4(0.f, 0.f, 0.f, 0.f);
    if (PULL) xg = ld4(xc + (int64_t)gl * ld);
    for (int j = 0; j < p.G; ++j) {
      int l = -1;
      float4 xl = xg;
      if (PULL) {
        l = s_ll[j];
        if (l != gl) xl = ld4(xc + (int64_t)l * ld);
      }
      const int m1 = s_start[j + 1];
      for (int m = s_start[j]; m < m1; m += kRows) {
        float4 xs[kRows], gs[kRows], vs[kRows];
        int rows[kRows];
#pragma unroll
        for (int u = 0; u < kRows; ++u) {
          if (m + u < m1) {
            const int i = s_rows[m + u];
            rows[u] = i;
            xs[u] = (PULL && i == l) ? xl : ld4(xc + (int64_t)i * ld);
            gs[u] = ld4(gc + (int64_t)i * ld);
            vs[u] = ld4(vc + (int64_t)i * ld);
          }
        }
#pragma unroll
        for (int u = 0; u < kRows; ++u) {
          if (m + u < m1) {
            const float4 x = xs[u], g = gs[u], v = vs[u];
            float4 r, w;
            step1<MODE, PULL>(x.x, g.x, v.x, xl.x, xg.x, k, r.x, w.x);
            step1<MODE, PULL>(x.y, g.y, v.y, xl.y, xg.y, k, r.y, w.y);
            step1<MODE, PULL>(x.z, g.z, v.z, xl.z, xg.z, k, r.z, w.z);
            step1<MODE, PULL>(x.w, g.w, v.w, xl.w, xg.w, k, r.w, w.w);
            st4(xc + (int64_t)rows[u] * ld, r);
            st4(vc + (int64_t)rows[u] * ld, w);
            if (SHADOW) st4_bf16(p.x_bf16 + col + (int64_t)rows[u] * ld, r);
          }
        }
      }
    }
  }
}

template <int MODE, bool PULL, bool SHADOW>
cudaError_t launch_k(const UpdateArgs& a, cudaStream_t s) {
  const int sms = sm_count();
  const int64_t n4 = (a.d + 3) / 4;
  int64_t blocks = (n4 + kThreads - 1) / kThreads;
  const int64_t cap = (int64_t)sms * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const size_t smem = sizeof(int32_t) * (size_t)(a.P + 2 * a.G + 1);
  momentum_update_kernel<MODE, PULL, SHADOW><<<(unsigned)blocks, kThreads, smem, s>>>(a, n4);
  return cudaGetLastError();
}

template <int MODE>
cudaError_t launch_m(const UpdateArgs& a, cudaStream_t s) {
  const bool shadow = a.x_bf16 != nullptr;
  if (a.pull) return shadow ? launch_k<MODE, true, true>(a, s) : launch_k<MODE, true, false>(a, s);
  return shadow ? launch_k<MODE, false, true>(a, s) : launch_k<MODE, false, false>(a, s);
}

}  // namespace

cudaError_t launch_momentum_update(const UpdateArgs& a, cudaStream_t s) {
  if (!a.v || !a.g || a.snap || !a.use_g) return cudaErrorInvalidValue;
  // first choice: the chunked staged pipeline of update.cu with the momentum buffer as a third row per worker
  const cudaError_t e = launch_momentum_update_chunked(a, s);
  if (e != cudaErrorNotSupported) return e;
  switch (a.arith) {
    case 0: return launch_m<0>(a, s);
    case 1: return launch_m<1>(a, s);
    default: return launch_m<2>(a, s);
  }
}

}  // namespace lsgd
