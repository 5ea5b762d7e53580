// Fused LSGD update (Eq. (1) with eta-scaled pulls, Section 3.1.1) and the plain (S)GD step used
// between communications (Section 3.1.2).
//
// Ownership rule of every form below: a CTA owns a column tile for ALL P workers, so whoever reads a leader's
// values does so before anyone rewrites them, and every right-hand side is x at time t although x is updated
// in place.  Three realisations, chosen in launch_t() / launch_momentum_update_chunked():
//   staged   (pull_update_staged_kernel): all rows of a 3 KiB-wide tile brought into shared memory by bulk
//            copies, for populations small enough that they fit twice (P <= 25 with a gradient row per worker);
//   chunked  (update_chunked_kernel): a leader block, then the rows streamed through a ring of chunks of 8
//            workers -- any P whose leader block fits, the inline quadratic gradient, the momentum step;
//   register-staged (pull_update_kernel, described next): the fallback for everything else.
//
// Register-staged pull form.  A thread owns one 16-byte column (4 consecutive parameters) for ALL P workers.  It
// reads the global leader's 4 values once, then walks the workers group by group: the group's local
// leader is read once into registers, after which each member row is read, updated and written.
// A leader row is taken from the registers it was staged in instead of being read again, so every
// byte of x and g is read exactly once and every byte of x written exactly once (12 B per
// worker-parameter, leaders cost nothing extra).  Because the same thread reads a leader's column
// before it (or anyone) writes it, all right-hand sides are x at time t although x is updated in
// place -- the simultaneous update of all workers at a communication (Section 2.2).
//
// A leader's own pull term is (x - x) = 0 exactly, and fmaf(-c, 0, acc) == acc, so the leader's
// step is bit-identical to the plain step without a branch (supplement, "Definitions and Notation":
// the update reduces to an (S)GD step for the leader).
#include <cuda_bf16.h>

#include "internal.h"

namespace lsgd {
namespace {

// Launch shapes, chosen by timing sweeps on the 16 x 2^26 stress shape (fp64 arithmetic):
//   pull form : 256 threads, 2 rows of loads in flight, registers capped for 4 CTAs per SM, 8 grid-stride
//               CTAs per SM (more rows in flight cost occupancy and lose; 5+ CTAs per SM spill);
//   plain form: 256 threads, 4 elements in flight, one CTA per 1024 columns up to 64 CTAs per SM.
#ifndef LSGD_K1_NO_STAGED
#define LSGD_K1_NO_STAGED 0     // 1: never use the shared-memory-staged pull kernel
#endif
#ifndef LSGD_K1_THREADS
#define LSGD_K1_THREADS 256
#endif
#ifndef LSGD_K1_PULL_ROWS
#define LSGD_K1_PULL_ROWS 2
#endif
#ifndef LSGD_K1_PULL_MIN_BLOCKS
#define LSGD_K1_PULL_MIN_BLOCKS 4
#endif
#ifndef LSGD_K1_PULL_CTAS_PER_SM
#define LSGD_K1_PULL_CTAS_PER_SM 8
#endif
#ifndef LSGD_K1_PLAIN_ROWS
#define LSGD_K1_PLAIN_ROWS 4
#endif
#ifndef LSGD_K1_PLAIN_CTAS_PER_SM
#define LSGD_K1_PLAIN_CTAS_PER_SM 64
#endif
constexpr int kThreads = LSGD_K1_THREADS;
constexpr int kPullRows = LSGD_K1_PULL_ROWS;     // rows whose loads are issued before the first is consumed
constexpr int kPlainRows = LSGD_K1_PLAIN_ROWS;

__device__ __forceinline__ float4 ld4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 ld4_cached(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

__device__ __forceinline__ void st4_bf16(uint16_t* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

// Arithmetic modes (UpdateArgs::arith).  The stored types are always fp32.
//   0: fp64 evaluation, one IEEE operation per printed operation (no contraction), one rounding to
//      fp32 at the end -- the same value a plain double-precision restatement of Eq. (1) produces;
//   1: fp64 evaluation with fused multiply-adds;
//   2: fp32 fused multiply-adds.
template <int MODE>
__device__ __forceinline__ float quad_g(float x, float a, float b, float n, const Coef& k, bool noise) {
  if (MODE == 0) {
    double r = __dmul_rn((double)a, __dsub_rn((double)x, (double)b));
    if (noise) r = __dadd_rn(r, __dmul_rn(k.sigma, (double)n));
    return (float)r;
  } else if (MODE == 1) {
    double r = (double)a * ((double)x - (double)b);
    if (noise) r = fma(k.sigma, (double)n, r);
    return (float)r;
  } else {
    return fmaf(a, x - b, noise ? k.sigma_f * n : 0.f);
  }
}

template <int MODE>
__device__ __forceinline__ float plain1(float x, float g, const Coef& k) {
  if (MODE == 0) return (float)__dsub_rn((double)x, __dmul_rn(k.eta, (double)g));
  if (MODE == 1) return (float)fma(-k.eta, (double)g, (double)x);
  return fmaf(-k.eta_f, g, x);
}

template <int MODE>
__device__ __forceinline__ float pull1(float x, float g, float xl, float xg, const Coef& k) {
  if (MODE == 0) {
    const double X = (double)x;
    double acc = __dsub_rn(X, __dmul_rn(k.eta, (double)g));
    acc = __dsub_rn(acc, __dmul_rn(k.cl, __dsub_rn(X, (double)xl)));
    acc = __dsub_rn(acc, __dmul_rn(k.cg, __dsub_rn(X, (double)xg)));
    return (float)acc;
  } else if (MODE == 1) {
    const double X = (double)x;
    double acc = fma(-k.eta, (double)g, X);
    acc = fma(-k.cl, X - (double)xl, acc);
    acc = fma(-k.cg, X - (double)xg, acc);
    return (float)acc;
  } else {
    float acc = fmaf(-k.eta_f, g, x);
    acc = fmaf(-k.cl_f, x - xl, acc);
    acc = fmaf(-k.cg_f, x - xg, acc);
    return acc;
  }
}

// The same three formulas on operands already held in the evaluation precision (double for modes 0 and 1,
// float for mode 2).  float -> double is exact, so converting an operand once and reusing it gives the same
// bits as converting it at every use.
template <int MODE> struct Eval { using T = double; };
template <> struct Eval<2> { using T = float; };

template <int MODE>
__device__ __forceinline__ float quad_g_t(typename Eval<MODE>::T X, typename Eval<MODE>::T A, typename Eval<MODE>::T B,
                                          float n, const Coef& k, bool noise) {
  if (MODE == 0) {
    double r = __dmul_rn((double)A, __dsub_rn((double)X, (double)B));
    if (noise) r = __dadd_rn(r, __dmul_rn(k.sigma, (double)n));
    return (float)r;
  } else if (MODE == 1) {
    double r = (double)A * ((double)X - (double)B);
    if (noise) r = fma(k.sigma, (double)n, r);
    return (float)r;
  } else {
    return fmaf((float)A, (float)X - (float)B, noise ? k.sigma_f * n : 0.f);
  }
}

template <int MODE>
__device__ __forceinline__ float plain1_t(typename Eval<MODE>::T X, float g, const Coef& k) {
  if (MODE == 0) return (float)__dsub_rn((double)X, __dmul_rn(k.eta, (double)g));
  if (MODE == 1) return (float)fma(-k.eta, (double)g, (double)X);
  return fmaf(-k.eta_f, g, (float)X);
}

template <int MODE>
__device__ __forceinline__ float pull1_t(typename Eval<MODE>::T X, float g, typename Eval<MODE>::T XL,
                                         typename Eval<MODE>::T XG, const Coef& k) {
  if (MODE == 0) {
    double acc = __dsub_rn((double)X, __dmul_rn(k.eta, (double)g));
    acc = __dsub_rn(acc, __dmul_rn(k.cl, __dsub_rn((double)X, (double)XL)));
    acc = __dsub_rn(acc, __dmul_rn(k.cg, __dsub_rn((double)X, (double)XG)));
    return (float)acc;
  } else if (MODE == 1) {
    double acc = fma(-k.eta, (double)g, (double)X);
    acc = fma(-k.cl, (double)X - (double)XL, acc);
    acc = fma(-k.cg, (double)X - (double)XG, acc);
    return (float)acc;
  } else {
    float acc = fmaf(-k.eta_f, g, (float)X);
    acc = fmaf(-k.cl_f, (float)X - (float)XL, acc);
    acc = fmaf(-k.cg_f, (float)X - (float)XG, acc);
    return acc;
  }
}

// The step with the Section 4.1 optimiser around it (the formulas of momentum.cu, same operation order):
//   d = g + wd x,  v+ = mu v + d,  u = d + mu v+,  x+ = x - eta u [- pulls].
template <int MODE, bool PULL>
__device__ __forceinline__ void momentum1_t(typename Eval<MODE>::T X, float g, float v, typename Eval<MODE>::T XL,
                                            typename Eval<MODE>::T XG, const Coef& k, float& x_new, float& v_new) {
  if (MODE == 0) {
    const double D = __dadd_rn((double)g, __dmul_rn(k.wd, (double)X));
    const double VN = __dadd_rn(__dmul_rn(k.mu, (double)v), D);
    const double U = __dadd_rn(D, __dmul_rn(k.mu, VN));
    double acc = __dsub_rn((double)X, __dmul_rn(k.eta, U));
    if (PULL) {
      acc = __dsub_rn(acc, __dmul_rn(k.cl, __dsub_rn((double)X, (double)XL)));
      acc = __dsub_rn(acc, __dmul_rn(k.cg, __dsub_rn((double)X, (double)XG)));
    }
    x_new = (float)acc;
    v_new = (float)VN;
  } else if (MODE == 1) {
    const double D = fma(k.wd, (double)X, (double)g);
    const double VN = fma(k.mu, (double)v, D);
    const double U = fma(k.mu, VN, D);
    double acc = fma(-k.eta, U, (double)X);
    if (PULL) {
      acc = fma(-k.cl, (double)X - (double)XL, acc);
      acc = fma(-k.cg, (double)X - (double)XG, acc);
    }
    x_new = (float)acc;
    v_new = (float)VN;
  } else {
    const float D = fmaf(k.wd_f, (float)X, g);
    const float VN = fmaf(k.mu_f, v, D);
    const float U = fmaf(k.mu_f, VN, D);
    float acc = fmaf(-k.eta_f, U, (float)X);
    if (PULL) {
      acc = fmaf(-k.cl_f, (float)X - (float)XL, acc);
      acc = fmaf(-k.cg_f, (float)X - (float)XG, acc);
    }
    x_new = acc;
    v_new = VN;
  }
}

template <int MODE, bool QUAD, bool NOISE, bool SHADOW>
__global__ void __launch_bounds__(kThreads, LSGD_K1_PULL_MIN_BLOCKS)
pull_update_kernel(UpdateArgs p, int64_t n4) {
  extern __shared__ int32_t s_tab[];
  int32_t* s_ll = s_tab;                 // [G]
  int32_t* s_start = s_ll + p.G;         // [G+1]
  int32_t* s_rows = s_start + p.G + 1;   // [P]
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  for (int k = threadIdx.x; k < p.G; k += blockDim.x) {
    int l = p.ll[k];
    if (l < 0 || l >= p.P) s_bad = 1;
    s_ll[k] = l;
  }
  for (int k = threadIdx.x; k <= p.G; k += blockDim.x) s_start[k] = p.tab.group_start[k];
  for (int k = threadIdx.x; k < p.P; k += blockDim.x) s_rows[k] = p.tab.rows_by_group[k];
  const int gl = *p.gl;
  if (threadIdx.x == 0 && (gl < 0 || gl >= p.P)) s_bad = 1;
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
    const float* gc = (QUAD ? p.quad.noise : p.g) + col;
    const float* snap = p.snap;
    const float4 xg = snap ? ld4_cached(snap + (int64_t)p.G * ld + col) : ld4(xc + (int64_t)gl * ld);
    float4 av, bv;
    if (QUAD) {
      av = ld4_cached(p.quad.a + col);
      bv = ld4_cached(p.quad.b + col);
    }
    for (int j = 0; j < p.G; ++j) {
      const int l = s_ll[j];
      const float4 xl = snap ? ld4_cached(snap + (int64_t)j * ld + col) : ((l == gl) ? xg : ld4(xc + (int64_t)l * ld));
      const int m1 = s_start[j + 1];
      for (int m = s_start[j]; m < m1; m += kPullRows) {
        float4 xs[kPullRows], gs[kPullRows];
        int rows[kPullRows];
#pragma unroll
        for (int u = 0; u < kPullRows; ++u) {
          if (m + u < m1) {
            const int i = s_rows[m + u];
            rows[u] = i;
            xs[u] = (!snap && i == l) ? xl : ld4(xc + (int64_t)i * ld);
            if ((!QUAD || NOISE) && p.use_g) gs[u] = ld4(gc + (int64_t)i * ld);
          }
        }
#pragma unroll
        for (int u = 0; u < kPullRows; ++u) {
          if (m + u < m1) {
            float4 x = xs[u], g = gs[u];
            if (QUAD) {
              g.x = quad_g<MODE>(x.x, av.x, bv.x, g.x, k, NOISE);
              g.y = quad_g<MODE>(x.y, av.y, bv.y, g.y, k, NOISE);
              g.z = quad_g<MODE>(x.z, av.z, bv.z, g.z, k, NOISE);
              g.w = quad_g<MODE>(x.w, av.w, bv.w, g.w, k, NOISE);
            }
            if (!p.use_g) g = make_float4(0.f, 0.f, 0.f, 0.f);   // pure pull: x - eta * 0 = x exactly
            float4 r;
            r.x = pull1<MODE>(x.x, g.x, xl.x, xg.x, k);
            r.y = pull1<MODE>(x.y, g.y, xl.y, xg.y, k);
            r.z = pull1<MODE>(x.z, g.z, xl.z, xg.z, k);
            r.w = pull1<MODE>(x.w, g.w, xl.w, xg.w, k);
            st4(xc + (int64_t)rows[u] * ld, r);
            if (SHADOW) st4_bf16(p.x_bf16 + col + (int64_t)rows[u] * ld, r);
          }
        }
      }
    }
  }
}

// Plain step with the quadratic gradient evaluated inline: a thread owns a 16-byte column for all P
// rows, so a and b (and their conversions to the evaluation precision) are paid once per column.
template <int MODE, bool NOISE>
__global__ void __launch_bounds__(kThreads, LSGD_K1_PULL_MIN_BLOCKS)
quad_plain_column_kernel(UpdateArgs p, int64_t n4) {
  const Coef k = p.k;
  const int64_t ld = p.ld;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n4; c += stride) {
    const int64_t col = c * 4;
    float* xc = p.x + col;
    const float* nc = p.quad.noise + col;
    const float4 av = ld4_cached(p.quad.a + col);
    const float4 bv = ld4_cached(p.quad.b + col);
    for (int m = 0; m < p.P; m += kPullRows) {
      float4 xs[kPullRows], ns[kPullRows];
#pragma unroll
      for (int u = 0; u < kPullRows; ++u) {
        if (m + u < p.P) {
          xs[u] = ld4(xc + (int64_t)(m + u) * ld);
          if (NOISE) ns[u] = ld4(nc + (int64_t)(m + u) * ld);
        }
      }
#pragma unroll
      for (int u = 0; u < kPullRows; ++u) {
        if (m + u < p.P) {
          const float4 x = xs[u], n = ns[u];
          float4 r;
          r.x = plain1<MODE>(x.x, quad_g<MODE>(x.x, av.x, bv.x, n.x, k, NOISE), k);
          r.y = plain1<MODE>(x.y, quad_g<MODE>(x.y, av.y, bv.y, n.y, k, NOISE), k);
          r.z = plain1<MODE>(x.z, quad_g<MODE>(x.z, av.z, bv.z, n.z, k, NOISE), k);
          r.w = plain1<MODE>(x.w, quad_g<MODE>(x.w, av.w, bv.w, n.w, k, NOISE), k);
          st4(xc + (int64_t)(m + u) * ld, r);
        }
      }
    }
  }
}

// Plain step x <- x - eta g over the whole [P][n4] grid of 16-byte columns.
template <int MODE, bool QUAD, bool NOISE, bool SHADOW>
__global__ void __launch_bounds__(kThreads)
plain_update_kernel(UpdateArgs p, int64_t n4) {
  const int64_t total = (int64_t)p.P * n4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const Coef k = p.k;
  for (int64_t e0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e0 < total; e0 += stride * kPlainRows) {
    float4 xs[kPlainRows], gs[kPlainRows];
    int64_t off[kPlainRows], cols[kPlainRows];
#pragma unroll
    for (int u = 0; u < kPlainRows; ++u) {
      const int64_t e = e0 + u * stride;
      if (e < total) {
        const int64_t row = e / n4, c = e - row * n4;
        cols[u] = c * 4;
        off[u] = row * p.ld + c * 4;
        xs[u] = ld4(p.x + off[u]);
        if (!QUAD || NOISE) gs[u] = ld4((QUAD ? p.quad.noise : p.g) + off[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kPlainRows; ++u) {
      const int64_t e = e0 + u * stride;
      if (e < total) {
        float4 x = xs[u], g = gs[u];
        if (QUAD) {
          const float4 av = ld4_cached(p.quad.a + cols[u]);
          const float4 bv = ld4_cached(p.quad.b + cols[u]);
          g.x = quad_g<MODE>(x.x, av.x, bv.x, g.x, k, NOISE);
          g.y = quad_g<MODE>(x.y, av.y, bv.y, g.y, k, NOISE);
          g.z = quad_g<MODE>(x.z, av.z, bv.z, g.z, k, NOISE);
          g.w = quad_g<MODE>(x.w, av.w, bv.w, g.w, k, NOISE);
        }
        float4 r;
        r.x = plain1<MODE>(x.x, g.x, k);
        r.y = plain1<MODE>(x.y, g.y, k);
        r.z = plain1<MODE>(x.z, g.z, k);
        r.w = plain1<MODE>(x.w, g.w, k);
        st4(p.x + off[u], r);
        if (SHADOW) st4_bf16(p.x_bf16 + off[u], r);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// Pull form with the column tile staged in shared memory by the bulk-copy engine.
//
// A persistent CTA takes column tiles of W floats.  For a tile, one warp issues 2 P one-dimensional bulk
// copies (cp.async.bulk, row i of x and of g -> shared memory, completion on an mbarrier) into one of
// kTmaStages stages; eight consumer warps then read everything -- the row itself, its gradient and both
// leaders -- from that snapshot of x_t, and write the new x straight to global memory with 512-byte
// coalesced stores.  Leaders are therefore fetched once per tile together with the other rows, the
// in-place update cannot disturb them, and the loads in flight (stages x 2 P W x 4 bytes per SM) no longer
// depend on registers.  Waits are clock-bounded; on expiry the status word is flagged and the CTA leaves.
// Shape found by timing sweeps on the 16 x 2^26 stress shape: what matters most is the length of the
// contiguous piece fetched per row (3 KiB: 6.8 TB/s; 2 KiB: 6.4; 1 KiB: 5.5; 512 B: 2.9 -- DRAM pages are
// used best by long bursts), then enough consumer warps to keep up (24), and only two stages: more stages
// interleave more rows at the memory controllers and lose again.
#ifndef LSGD_K1_STAGED_STAGES
#define LSGD_K1_STAGED_STAGES 2
#endif
#ifndef LSGD_K1_STAGED_CONSUMERS
#define LSGD_K1_STAGED_CONSUMERS 768
#endif
#ifndef LSGD_K1_STAGED_W
#define LSGD_K1_STAGED_W 768
#endif
constexpr int kTmaStages = LSGD_K1_STAGED_STAGES;
constexpr int kTmaConsumers = LSGD_K1_STAGED_CONSUMERS;
constexpr int kTmaThreads = kTmaConsumers + 32;
constexpr int kTmaSmemBudget = 208 * 1024;
constexpr long long kTmaWaitCycles = 2000000000LL;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool bar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false once `budget` clock cycles have passed (the status word then carries FLAG_WAIT_TIMEOUT and
// the CTA-wide abort flag is raised) or when another role of the CTA has already given up.
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t* status,
                                         long long budget = kTmaWaitCycles) {
  if (bar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (bar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > budget) {
      *abort_flag = 1;
      atomicOr(status, FLAG_WAIT_TIMEOUT);
      return false;
    }
  }
}

// Self-test of the bounded wait: one warp waits, with a short budget, on a barrier that nothing will ever
// complete (no copy is in flight, nobody arrives), so the wait must run out, set the status bit and return.
__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(uint32_t* status, long long budget, int* gave_up) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bar)) : "memory");
  }
  __syncthreads();
  const bool ok = bar_wait(&bar, 0, &abort_flag, status, budget);
  __syncwarp();
  if (threadIdx.x == 0) {
    *gave_up = ok ? 0 : 1;
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_addr(&bar)) : "memory");
  }
}

template <int MODE, bool SHADOW>
__global__ void __launch_bounds__(kTmaThreads, 1)
pull_update_staged_kernel(UpdateArgs p, int64_t n_cols4, int W) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ __align__(128) uint8_t s_raw[];
  __shared__ uint64_t full_bar[kTmaStages], empty_bar[kTmaStages];
  __shared__ int s_abort, s_bad, s_gl;
  const int P = p.P;
  const bool use_g = p.use_g, snap = p.snap != nullptr;
  const int n_rows = P + (use_g ? P : 0) + (snap ? p.G + 1 : 0);  // x rows, g rows, leader copies
  const size_t stage_floats = (size_t)n_rows * W;
  float* stage0 = reinterpret_cast<float*>(s_raw);
  int32_t* s_lead = reinterpret_cast<int32_t*>(stage0 + kTmaStages * stage_floats);   // [P]: local leader row of worker i
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    s_abort = 0;
    s_bad = 0;
    for (int s = 0; s < kTmaStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&full_bar[s])), "r"(1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&empty_bar[s])), "r"(kTmaConsumers / 32) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const int gl = *p.gl;
    if (!snap && (gl < 0 || gl >= P)) s_bad = 1;
    s_gl = gl;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < P; i += blockDim.x) {
    // row of the stage that holds worker i's local leader: a row of x, or (with leader copies) a copy row
    const int grp = p.tab.group_of[i];
    const int l = snap ? grp : p.ll[grp];
    if (l < 0 || l >= P) s_bad = 1;
    s_lead[i] = l;
  }
  __syncthreads();
  if (s_bad) {   // never index shared memory with a leader that is out of range
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(p.status, FLAG_BAD_LEADER);
    return;
  }
  volatile int* abort_flag = &s_abort;
  const int64_t total_floats = n_cols4 * 4;
  const int64_t n_tiles = (total_floats + W - 1) / W;
  if (warp == kTmaConsumers / 32) {
    // ------------------------------------------------------------------ producer warp
    uint32_t it = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
      const int s = it % kTmaStages;
      ok = bar_wait(&empty_bar[s], ((it / kTmaStages) & 1) ^ 1, abort_flag, p.status);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      const int64_t c0 = t * W;
      const int wt = (int)((total_floats - c0) < W ? (total_floats - c0) : W);   // floats in this tile (multiple of 4)
      const uint32_t bytes = (uint32_t)wt * 4u;
      float* sx = stage0 + s * stage_floats;
      if (lane == 0)
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&full_bar[s])), "r"(bytes * (uint32_t)n_rows) : "memory");
      __syncwarp();
      for (int r = lane; r < n_rows; r += 32) {
        // stage row r: worker r's x, then worker (r - P)'s g, then the leader copies
        const float* src;
        if (r < P) src = p.x + (int64_t)r * p.ld;
        else if (use_g && r < 2 * P) src = p.g + (int64_t)(r - P) * p.ld;
        else src = p.snap + (int64_t)(r - P - (use_g ? P : 0)) * p.ld;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(sx + (size_t)r * W)), "l"(src + c0), "r"(bytes), "r"(smem_addr(&full_bar[s])) : "memory");
      }
    }
    if (*abort_flag && lane == 0) {
      // a wait ran out somewhere: let the copies already issued land before the CTA exits
      const uint32_t first = it > kTmaStages ? it - kTmaStages : 0;
      for (uint32_t j = first; j < it; ++j) {
        const long long t0 = clock64();
        while (!bar_try(&full_bar[j % kTmaStages], (j / kTmaStages) & 1) && clock64() - t0 < kTmaWaitCycles) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    const Coef k = p.k;
    const int gl = s_gl;
    const int w4 = W >> 2;                          // 16-byte columns per tile row
    const int c4 = threadIdx.x % w4;                // this thread's column
    const int r0 = threadIdx.x / w4, rstep = kTmaConsumers / w4;
    uint32_t it = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
      const int s = it % kTmaStages;
      ok = bar_wait(&full_bar[s], (it / kTmaStages) & 1, abort_flag, p.status);
      if (!ok) break;
      const int64_t c0 = t * W;
      const int wt4 = (int)(((total_floats - c0) < W ? (total_floats - c0) : W) >> 2);
      const float* sx = stage0 + s * stage_floats;
      const float* sg = sx + (size_t)P * W;
      const float* sl = snap ? sx + (size_t)(P + (use_g ? P : 0)) * W : sx;     // where the leaders' rows are
      // thread (column c4, row lane r0) walks rows r0, r0 + rstep, ...; the global leader's value stays in registers
      if (c4 < wt4) {
        const float4 xg = *reinterpret_cast<const float4*>(sl + (size_t)(snap ? p.G : gl) * W + c4 * 4);
        for (int i = r0; i < P; i += rstep) {
          const float4 x = *reinterpret_cast<const float4*>(sx + (size_t)i * W + c4 * 4);
          const float4 g = use_g ? *reinterpret_cast<const float4*>(sg + (size_t)i * W + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 xl = *reinterpret_cast<const float4*>(sl + (size_t)s_lead[i] * W + c4 * 4);
          float4 r;
          r.x = pull1<MODE>(x.x, g.x, xl.x, xg.x, k);
          r.y = pull1<MODE>(x.y, g.y, xl.y, xg.y, k);
          r.z = pull1<MODE>(x.z, g.z, xl.z, xg.z, k);
          r.w = pull1<MODE>(x.w, g.w, xl.w, xg.w, k);
          const int64_t off = (int64_t)i * p.ld + c0 + c4 * 4;
          st4(p.x + off, r);
          if (SHADOW) st4_bf16(p.x_bf16 + off, r);
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&empty_bar[s])) : "memory");
    }
  }
}

// Tile width (floats) for the staged kernel, 0 if the shape does not suit it: all P rows of a tile of at
// least 512 columns (2 KiB per row) must fit twice over in shared memory: 2 stages x 2 P rows x 2 KiB plus the
// P-entry leader table within 208 KiB, i.e. P <= 25 when every worker brings a gradient row; larger
// populations use the chunked or the register-staged kernel.
inline int staged_rows(const UpdateArgs& a) { return a.P + (a.use_g ? a.P : 0) + (a.snap ? a.G + 1 : 0); }
inline int staged_tile_width(const UpdateArgs& a) {
  if (!a.pull || (a.use_g && a.g == nullptr)) return 0;
  for (int W = LSGD_K1_STAGED_W; W >= 512; W -= 256) {
    const size_t bytes = (size_t)kTmaStages * staged_rows(a) * W * 4 + (size_t)a.P * 4;
    if (bytes <= (size_t)kTmaSmemBudget && (kTmaConsumers % (W / 4)) == 0) return W;
  }
  return 0;
}

// ---------------------------------------------------------------------------------------------------
// Chunked staged form: the same bulk-copy pipeline for any population size, and for the inline quadratic
// gradient.
//
// A tile's rows no longer have to fit in shared memory together.  What every row of the tile needs -- the
// leaders' pieces (one slot per group's local leader, one for the global leader when it is not among them, or
// the G + 1 leader copies) and, for the quadratic, the pieces of a and b -- goes into a double-buffered
// "leader block" first; the workers' rows (x and g / noise) then stream through a ring of chunks of R workers.
// The consumers start on a tile only after its leader block has landed, so every leader value is x at time t
// although the leader's own row is rewritten while the tile is processed.  A worker that is its group's
// leader takes its x from the leader block and its row is not fetched again: every byte of x and g is still
// read once.
#ifndef LSGD_K1_CHUNK_SHAPES
#define LSGD_K1_CHUNK_SHAPES {768, 8, 3}, {768, 8, 2}, {768, 4, 3}, {768, 4, 2}, {512, 12, 2}, {512, 6, 3}, {512, 6, 2}
#endif
#ifndef LSGD_K1_MOM_SHAPES
#define LSGD_K1_MOM_SHAPES {768, 8, 2}, {768, 4, 3}, {768, 4, 2}, {512, 12, 2}, {512, 6, 3}, {512, 6, 2}
#endif
constexpr int kChunkMaxStages = 4;
constexpr int kChunkSmemBudget = 224 * 1024;

struct ChunkShape {
  int W, R, S;      // tile width (floats), workers per chunk, ring stages; W == 0: the shape does not fit
  size_t smem;
};

template <int MODE, bool PULL, bool QUAD, bool NOISE, bool SHADOW, bool MOM>
__global__ void __launch_bounds__(kTmaThreads, 1)
update_chunked_kernel(UpdateArgs p, int64_t n_cols4, int W, int R, int S) {
  pdl_wait();                  // launched as a programmatic dependent: nothing is read before the earlier kernels end
  pdl_launch_dependents();
  extern __shared__ __align__(128) uint8_t s_raw[];
  __shared__ uint64_t full_bar[kChunkMaxStages], empty_bar[kChunkMaxStages], lfull_bar[2], lempty_bar[2];
  __shared__ int s_abort, s_bad, s_gslot;
  const int P = p.P, G = p.G;
  const bool snap = PULL && p.snap != nullptr;
  const bool has_g = (QUAD ? NOISE : true) && p.use_g;      // a pure pull drops the gradient term
  const int pull_slots = PULL ? G + 1 : 0;                  // slots 0..G-1: local leaders, slot G: global leader
  const int nlead = pull_slots + (QUAD ? 2 : 0);            // then a, b
  const int stage_rows = R * ((has_g ? 2 : 1) + (MOM ? 1 : 0));   // per worker: x, g / noise, momentum buffer
  float* lead0 = reinterpret_cast<float*>(s_raw);                                   // [2][nlead][W]
  float* ring0 = lead0 + (size_t)2 * nlead * W;                                     // [S][stage_rows][W]
  int32_t* s_lead = reinterpret_cast<int32_t*>(ring0 + (size_t)S * stage_rows * W); // [P] slot of worker i's local leader
  int32_t* s_self = s_lead + P;                                                     // [P] worker i is that leader: x comes from the slot
  int32_t* s_slot_row = s_self + P;                                                 // [G+1] row of x behind a slot
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    s_abort = 0;
    s_bad = 0;
    for (int s = 0; s < S; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&full_bar[s])), "r"(1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&empty_bar[s])), "r"(kTmaConsumers / 32) : "memory");
    }
    for (int b = 0; b < 2; ++b) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&lfull_bar[b])), "r"(1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&lempty_bar[b])), "r"(kTmaConsumers / 32) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_gslot = G;
    if (PULL && !snap) {
      const int gl = *p.gl;
      if (gl < 0 || gl >= P) {
        s_bad = 1;
      } else {
        const int grp = p.tab.group_of[gl];
        s_slot_row[G] = gl;
        if (p.ll[grp] == gl) s_gslot = grp;     // the global leader is its group's leader: one slot serves both
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < P; i += blockDim.x) {
    int slot = 0, self = 0;
    if (PULL) {
      slot = p.tab.group_of[i];
      if (!snap) {
        const int l = p.ll[slot];
        if (l < 0 || l >= P) s_bad = 1;
        self = (l == i);
      }
    }
    s_lead[i] = slot;
    s_self[i] = self;
  }
  if (PULL && !snap)
    for (int j = threadIdx.x; j < G; j += blockDim.x) s_slot_row[j] = p.ll[j];
  __syncthreads();
  if (s_bad) {   // never dereference a leader index that is out of range
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(p.status, FLAG_BAD_LEADER);
    return;
  }
  volatile int* abort_flag = &s_abort;
  const int gslot = s_gslot;
  const int64_t total_floats = n_cols4 * 4;
  const int64_t n_tiles = (total_floats + W - 1) / W;
  const int n_chunks = (P + R - 1) / R;
  const float* gsrc = QUAD ? p.quad.noise : p.g;
  if (warp == kTmaConsumers / 32) {
    // ------------------------------------------------------------------ producer warp
    uint32_t tit = 0, cit = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tit) {
      const int b = tit & 1;
      ok = bar_wait(&lempty_bar[b], ((tit >> 1) & 1) ^ 1, abort_flag, p.status);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      const int64_t c0 = t * W;
      const int wt = (int)((total_floats - c0) < W ? (total_floats - c0) : W);   // floats in this tile (multiple of 4)
      const uint32_t bytes = (uint32_t)wt * 4u;
      float* lead = lead0 + (size_t)b * nlead * W;
      // the leader block: leaders' pieces (slot G only when it is a row of its own), then a and b
      const int n_fetch = nlead - ((PULL && gslot != G) ? 1 : 0);
      if (lane == 0)
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&lfull_bar[b])), "r"(bytes * (uint32_t)n_fetch) : "memory");
      __syncwarp();
      for (int r = lane; r < nlead; r += 32) {
        const float* src;
        if (r < pull_slots) {
          if (r == G && gslot != G) continue;
          src = snap ? p.snap + (int64_t)r * p.ld : p.x + (int64_t)s_slot_row[r] * p.ld;
        } else {
          src = (r == pull_slots) ? p.quad.a : p.quad.b;
        }
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(lead + (size_t)r * W)), "l"(src + c0), "r"(bytes), "r"(smem_addr(&lfull_bar[b])) : "memory");
      }
      for (int c = 0; c < n_chunks && ok; ++c, ++cit) {
        const int s = cit % S;
        ok = bar_wait(&empty_bar[s], ((cit / S) & 1) ^ 1, abort_flag, p.status);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        const int i0 = c * R;
        const int nr = (P - i0) < R ? (P - i0) : R;
        float* sx = ring0 + (size_t)s * stage_rows * W;
        // rows q < nr: worker (i0 + q)'s x unless it sits in the leader block; rows R + q: its g / noise
        int mine = 0;
        for (int q = lane; q < nr; q += 32) mine += (s_self[i0 + q] ? 0 : 1) + (has_g ? 1 : 0) + (MOM ? 1 : 0);
        const int n_copies = __reduce_add_sync(0xFFFFFFFFu, mine);
        if (lane == 0)
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&full_bar[s])), "r"(bytes * (uint32_t)n_copies) : "memory");
        __syncwarp();
        for (int q = lane; q < nr; q += 32) {
          const int i = i0 + q;
          if (!s_self[i])
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sx + (size_t)q * W)), "l"(p.x + (int64_t)i * p.ld + c0), "r"(bytes), "r"(smem_addr(&full_bar[s])) : "memory");
          if (has_g)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sx + (size_t)(R + q) * W)), "l"(gsrc + (int64_t)i * p.ld + c0), "r"(bytes), "r"(smem_addr(&full_bar[s])) : "memory");
          if (MOM)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sx + (size_t)(2 * R + q) * W)), "l"(p.v + (int64_t)i * p.ld + c0), "r"(bytes), "r"(smem_addr(&full_bar[s])) : "memory");
        }
      }
    }
    if (*abort_flag && lane == 0) {
      // a wait ran out somewhere: let the copies already issued land before the CTA exits
      const uint32_t cfirst = cit > (uint32_t)S ? cit - S : 0;
      for (uint32_t j = cfirst; j < cit; ++j) {
        const long long t0 = clock64();
        while (!bar_try(&full_bar[j % S], (j / S) & 1) && clock64() - t0 < kTmaWaitCycles) {}
      }
      const uint32_t tfirst = tit > 1 ? tit - 1 : 0;
      for (uint32_t j = tfirst; j <= tit; ++j) {
        const long long t0 = clock64();
        while (!bar_try(&lfull_bar[j & 1], (j >> 1) & 1) && clock64() - t0 < kTmaWaitCycles) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    using T = typename Eval<MODE>::T;
    const Coef k = p.k;
    const int w4 = W >> 2;                          // 16-byte columns per tile row
    const int c4 = threadIdx.x % w4;                // this thread's column
    const int r0 = threadIdx.x / w4, rstep = kTmaConsumers / w4;
    uint32_t tit = 0, cit = 0;
    bool ok = true;
    for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tit) {
      const int b = tit & 1;
      ok = bar_wait(&lfull_bar[b], (tit >> 1) & 1, abort_flag, p.status);
      if (!ok) break;
      const int64_t c0 = t * W;
      const int wt4 = (int)(((total_floats - c0) < W ? (total_floats - c0) : W) >> 2);
      const bool live = c4 < wt4;
      const float* lead = lead0 + (size_t)b * nlead * W + c4 * 4;
      // a, b and the global leader's values are converted to the evaluation precision once per tile, a local
      // leader's once per run of rows that share it: with fp64 evaluation the float <-> double conversions
      // (16 per clock per SM) are what bounds this kernel, not the arithmetic or the memory system
      T XG[4] = {0, 0, 0, 0}, A[4] = {0, 0, 0, 0}, B[4] = {0, 0, 0, 0}, XL[4] = {0, 0, 0, 0};
      int cur_slot = -1;
      if (live) {
        if (PULL) {
          const float4 v = *reinterpret_cast<const float4*>(lead + (size_t)gslot * W);
          XG[0] = (T)v.x; XG[1] = (T)v.y; XG[2] = (T)v.z; XG[3] = (T)v.w;
        }
        if (QUAD) {
          const float4 av = *reinterpret_cast<const float4*>(lead + (size_t)pull_slots * W);
          const float4 bv = *reinterpret_cast<const float4*>(lead + (size_t)(pull_slots + 1) * W);
          A[0] = (T)av.x; A[1] = (T)av.y; A[2] = (T)av.z; A[3] = (T)av.w;
          B[0] = (T)bv.x; B[1] = (T)bv.y; B[2] = (T)bv.z; B[3] = (T)bv.w;
        }
      }
      for (int c = 0; c < n_chunks; ++c, ++cit) {
        const int s = cit % S;
        ok = bar_wait(&full_bar[s], (cit / S) & 1, abort_flag, p.status);
        if (!ok) break;
        const int i0 = c * R;
        const int nr = (P - i0) < R ? (P - i0) : R;
        const float* sx = ring0 + (size_t)s * stage_rows * W + c4 * 4;
        const float* sg = sx + (size_t)R * W;
        for (int q = r0; q < nr; q += rstep) {
          const int i = i0 + q;
          if (live) {
            if (PULL) {
              const int slot = s_lead[i];
              if (slot != cur_slot) {
                cur_slot = slot;
                const float4 v = *reinterpret_cast<const float4*>(lead + (size_t)slot * W);
                XL[0] = (T)v.x; XL[1] = (T)v.y; XL[2] = (T)v.z; XL[3] = (T)v.w;
              }
            }
            T X[4];
            if (PULL && s_self[i]) {
              X[0] = XL[0]; X[1] = XL[1]; X[2] = XL[2]; X[3] = XL[3];
            } else {
              const float4 v = *reinterpret_cast<const float4*>(sx + (size_t)q * W);
              X[0] = (T)v.x; X[1] = (T)v.y; X[2] = (T)v.z; X[3] = (T)v.w;
            }
            const float4 gv = has_g ? *reinterpret_cast<const float4*>(sg + (size_t)q * W) : make_float4(0.f, 0.f, 0.f, 0.f);
            float g[4] = {gv.x, gv.y, gv.z, gv.w}, r[4];
            const int64_t off = (int64_t)i * p.ld + c0 + c4 * 4;
            if (MOM) {
              const float4 vv = *reinterpret_cast<const float4*>(sx + (size_t)(2 * R + q) * W);
              const float vo[4] = {vv.x, vv.y, vv.z, vv.w};
              float vn[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) momentum1_t<MODE, PULL>(X[e], g[e], vo[e], XL[e], XG[e], k, r[e], vn[e]);
              st4(p.v + off, make_float4(vn[0], vn[1], vn[2], vn[3]));
            } else {
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                if (QUAD && p.use_g) g[e] = quad_g_t<MODE>(X[e], A[e], B[e], g[e], k, NOISE);
                r[e] = PULL ? pull1_t<MODE>(X[e], g[e], XL[e], XG[e], k) : plain1_t<MODE>(X[e], g[e], k);
              }
            }
            const float4 rv = make_float4(r[0], r[1], r[2], r[3]);
            st4(p.x + off, rv);
            if (SHADOW) st4_bf16(p.x_bf16 + off, rv);
          }
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&empty_bar[s])) : "memory");
      }
      if (!ok) break;
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&lempty_bar[b])) : "memory");
    }
  }
}

// Shape for the chunked kernel: the widest tile and deepest ring whose leader block (twice) and ring fit.
inline ChunkShape chunk_shape(const UpdateArgs& a, bool quad, bool noise, bool mom = false) {
  ChunkShape none{0, 0, 0, 0};
  if (!a.pull && !quad && !mom) return none;
  const bool has_g = (quad ? noise : true) && a.use_g;
  if (!quad && a.use_g && a.g == nullptr) return none;
  const int nlead = (a.pull ? a.G + 1 : 0) + (quad ? 2 : 0);
  // the momentum step streams three rows per worker over very long rows: two deep stages beat three there
  static const int shapes_plain[][3] = {LSGD_K1_CHUNK_SHAPES};
  static const int shapes_mom[][3] = {LSGD_K1_MOM_SHAPES};
  const int (*shapes)[3] = mom ? shapes_mom : shapes_plain;
  const int n_shapes = mom ? (int)(sizeof(shapes_mom) / sizeof(shapes_mom[0])) : (int)(sizeof(shapes_plain) / sizeof(shapes_plain[0]));
  for (int q = 0; q < n_shapes; ++q) {
    const int* sh = shapes[q];
    const int W = sh[0], R = sh[1], S = sh[2];
    if (S > kChunkMaxStages || (kTmaConsumers % (W / 4)) != 0) continue;
    const size_t bytes = ((size_t)2 * nlead + (size_t)S * R * ((has_g ? 2 : 1) + (mom ? 1 : 0))) * W * 4 +
                         (size_t)(2 * a.P + a.G + 1) * 4;
    if (bytes <= (size_t)kChunkSmemBudget) return ChunkShape{W, R, S, bytes};
  }
  return none;
}

template <int MODE, bool PULL, bool QUAD, bool NOISE, bool SHADOW, bool MOM = false>
cudaError_t launch_chunked(const UpdateArgs& a, const ChunkShape& cs, int64_t n4, int sms, cudaStream_t s) {
  static OncePerDevice attr;
  if (!attr.here()) {
    cudaError_t e = cudaFuncSetAttribute(update_chunked_kernel<MODE, PULL, QUAD, NOISE, SHADOW, MOM>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kChunkSmemBudget);
    if (e != cudaSuccess) return e;
    attr.here() = true;
  }
  const int64_t tiles = (n4 * 4 + cs.W - 1) / cs.W;
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  return launch_pdl(update_chunked_kernel<MODE, PULL, QUAD, NOISE, SHADOW, MOM>, dim3(grid), dim3(kTmaThreads), cs.smem, s, a, n4,
                    cs.W, cs.R, cs.S);
}

template <int MODE, bool QUAD, bool NOISE, bool SHADOW>
cudaError_t launch_t(const UpdateArgs& a, cudaStream_t s) {
  const int sms = sm_count();
  const int64_t n4 = (a.d + 3) / 4;
  const int64_t cap = (int64_t)sms * (a.pull ? LSGD_K1_PULL_CTAS_PER_SM : LSGD_K1_PLAIN_CTAS_PER_SM);
  const int W = (QUAD || LSGD_K1_NO_STAGED) ? 0 : staged_tile_width(a);
  if (W > 0) {
    static OncePerDevice attr;
    if (!attr.here()) {
      cudaError_t e = cudaFuncSetAttribute(pull_update_staged_kernel<MODE, SHADOW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kTmaSmemBudget + 1024);
      if (e != cudaSuccess) return e;
      attr.here() = true;
    }
    const size_t smem = (size_t)kTmaStages * staged_rows(a) * W * 4 + (size_t)a.P * 4;
    const int64_t tiles = (n4 * 4 + W - 1) / (W > 0 ? W : 1);
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    return launch_pdl(pull_update_staged_kernel<MODE, SHADOW>, dim3(grid), dim3(kTmaThreads), smem, s, a, n4, W);
  } else if (!LSGD_K1_NO_STAGED && (a.pull || (QUAD && !SHADOW)) && chunk_shape(a, QUAD, NOISE).W > 0) {
    const ChunkShape cs = chunk_shape(a, QUAD, NOISE);
    if (a.pull) return launch_chunked<MODE, true, QUAD, NOISE, SHADOW>(a, cs, n4, sms, s);
    if constexpr (QUAD && !SHADOW) return launch_chunked<MODE, false, QUAD, NOISE, false>(a, cs, n4, sms, s);
  } else if (a.pull) {
    int64_t blocks = (n4 + kThreads - 1) / kThreads;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const size_t smem = sizeof(int32_t) * (size_t)(a.P + 2 * a.G + 1);
    pull_update_kernel<MODE, QUAD, NOISE, SHADOW><<<(unsigned)blocks, kThreads, smem, s>>>(a, n4);
  } else if (QUAD && !SHADOW) {
    int64_t blocks = (n4 + kThreads - 1) / kThreads;
    const int64_t qcap = (int64_t)sms * LSGD_K1_PULL_CTAS_PER_SM;
    if (blocks > qcap) blocks = qcap;
    if (blocks < 1) blocks = 1;
    quad_plain_column_kernel<MODE, NOISE><<<(unsigned)blocks, kThreads, 0, s>>>(a, n4);
  } else {
    const int64_t total = (int64_t)a.P * n4;
    int64_t blocks = (total + (int64_t)kThreads * kPlainRows - 1) / ((int64_t)kThreads * kPlainRows);
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    plain_update_kernel<MODE, QUAD, NOISE, SHADOW><<<(unsigned)blocks, kThreads, 0, s>>>(a, n4);
  }
  return cudaGetLastError();
}

// center[k] = mean over the P workers of x[i][k] (fp64 accumulation in worker order, one rounding)
__global__ void __launch_bounds__(256)
center_kernel(const float* __restrict__ x, float* __restrict__ center, int32_t P, int64_t n4, int64_t ld) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const double inv = 1.0 / (double)P;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n4; c += stride) {
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    for (int i = 0; i < P; ++i) {
      const float4 v = ld4(x + (int64_t)i * ld + c * 4);
      s0 += (double)v.x;
      s1 += (double)v.y;
      s2 += (double)v.z;
      s3 += (double)v.w;
    }
    *reinterpret_cast<float4*>(center + c * 4) = make_float4((float)(s0 * inv), (float)(s1 * inv), (float)(s2 * inv), (float)(s3 * inv));
  }
}

// EAGD center rule (supplement, "Low-Rank Matrix Completion Experiments"):
//   out[k] = (1 - kk) center[k] + kk * ((sum_i x[i][k]) * (1 / P)),  kk = P eta lambda,
// one IEEE fp64 operation per printed operation (no contraction), worker-order sum, one rounding to fp32.
__global__ void __launch_bounds__(256)
eagd_center_kernel(const float* __restrict__ x, const float* __restrict__ center, float* __restrict__ out, int32_t P,
                   int64_t n4, int64_t ld, double kk) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const double inv = 1.0 / (double)P, keep = __dsub_rn(1.0, kk);
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n4; c += stride) {
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    for (int i = 0; i < P; ++i) {
      const float4 v = ld4(x + (int64_t)i * ld + c * 4);
      s0 += (double)v.x;
      s1 += (double)v.y;
      s2 += (double)v.z;
      s3 += (double)v.w;
    }
    const float4 z = ld4(center + c * 4);
    float4 o;
    o.x = (float)__dadd_rn(__dmul_rn(keep, (double)z.x), __dmul_rn(kk, __dmul_rn(s0, inv)));
    o.y = (float)__dadd_rn(__dmul_rn(keep, (double)z.y), __dmul_rn(kk, __dmul_rn(s1, inv)));
    o.z = (float)__dadd_rn(__dmul_rn(keep, (double)z.z), __dmul_rn(kk, __dmul_rn(s2, inv)));
    o.w = (float)__dadd_rn(__dmul_rn(keep, (double)z.w), __dmul_rn(kk, __dmul_rn(s3, inv)));
    *reinterpret_cast<float4*>(out + c * 4) = o;
  }
}

template <int MODE>
cudaError_t launch_m(const UpdateArgs& a, cudaStream_t s) {
  const bool quad = (a.g == nullptr);
  const bool noise = quad && a.quad.noise != nullptr;
  const bool shadow = a.x_bf16 != nullptr;
  if (!quad) return shadow ? launch_t<MODE, false, false, true>(a, s) : launch_t<MODE, false, false, false>(a, s);
  if (shadow) return cudaErrorNotSupported;
  return noise ? launch_t<MODE, true, true, false>(a, s) : launch_t<MODE, true, false, false>(a, s);
}

}  // namespace

cudaError_t launch_center(const float* x, float* center, int32_t P, int64_t d, int64_t ld, cudaStream_t s) {
  (void)d;
  const int64_t n4 = ld / 4;   // the padding columns are averaged too, so all ld outputs are defined
  int64_t blocks = (n4 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  center_kernel<<<(unsigned)blocks, 256, 0, s>>>(x, center, P, n4, ld);
  return cudaGetLastError();
}

cudaError_t launch_eagd_center(const float* x, const float* center, float* out, int32_t P, int64_t ld, double kk,
                               cudaStream_t s) {
  const int64_t n4 = ld / 4;
  int64_t blocks = (n4 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  eagd_center_kernel<<<(unsigned)blocks, 256, 0, s>>>(x, center, out, P, n4, ld, kk);
  return cudaGetLastError();
}

namespace {
template <int MODE>
cudaError_t launch_momentum_chunked_m(const UpdateArgs& a, const ChunkShape& cs, cudaStream_t s) {
  const int sms = sm_count();
  const int64_t n4 = (a.d + 3) / 4;
  const bool shadow = a.x_bf16 != nullptr;
  if (a.pull) return shadow ? launch_chunked<MODE, true, false, false, true, true>(a, cs, n4, sms, s)
                            : launch_chunked<MODE, true, false, false, false, true>(a, cs, n4, sms, s);
  return shadow ? launch_chunked<MODE, false, false, false, true, true>(a, cs, n4, sms, s)
                : launch_chunked<MODE, false, false, false, false, true>(a, cs, n4, sms, s);
}
}  // namespace

// The momentum step through the chunked staged pipeline (x, g and v rows in the ring).  cudaErrorNotSupported
// when the shape does not fit: the caller then uses the register-staged momentum kernel.
cudaError_t launch_momentum_update_chunked(const UpdateArgs& a, cudaStream_t s) {
  if (LSGD_K1_NO_STAGED || !a.v || !a.g || a.snap || !a.use_g) return cudaErrorNotSupported;
  const ChunkShape cs = chunk_shape(a, false, false, true);
  if (cs.W == 0) return cudaErrorNotSupported;
  switch (a.arith) {
    case 0: return launch_momentum_chunked_m<0>(a, cs, s);
    case 1: return launch_momentum_chunked_m<1>(a, cs, s);
    default: return launch_momentum_chunked_m<2>(a, cs, s);
  }
}

cudaError_t launch_wait_timeout_selftest(uint32_t* status, long long budget_cycles, int* gave_up, cudaStream_t s) {
  wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status, budget_cycles, gave_up);
  return cudaGetLastError();
}

cudaError_t launch_update(const UpdateArgs& a, cudaStream_t s) {
  switch (a.arith) {
    case 0: return launch_m<0>(a, s);
    case 1: return launch_m<1>(a, s);
    default: return launch_m<2>(a, s);
  }
}

}  // namespace lsgd
