// Batched bf16 x bf16 -> fp32 matrix product on the 5th-generation tensor cores (tcgen05), used by
// the MLP population objective.  C[z] = A[z] . B[z], C is M x N, the contraction length is K.
//
//   * operands are fetched by TMA (cp.async.bulk.tensor, 128-byte swizzle) into a 3-stage shared
//     memory ring guarded by mbarriers; each stage holds a 128 x 64 slice of A and of B;
//   * one elected thread issues tcgen05.mma (M = 128, N = 128, K = 16, cta_group::1) with the fp32
//     accumulator tile (128 lanes x 128 columns) in tensor memory;
//   * four epilogue warps read the accumulator back with tcgen05.ld and apply the fused epilogue
//     (bias + ReLU + bf16 store, ReLU-mask + bf16 store, or plain fp32 / bf16 store).
//
// Either operand may be "K-major" (the contraction index is contiguous in memory) or "MN-major"
// (the M resp. N index is contiguous): weights W[out][in], activations H[batch][feature] and their
// transposes are all consumed in place, nothing is transposed in memory.  In shared memory a
// 64-element-wide box is always 128 bytes per row, so both majors use 1024-byte swizzle atoms:
//   K-major : rows = M/N index, 8-row groups 1024 B apart (SBO); one K = 16 step is +32 B;
//   MN-major: rows = K index, 64-wide M/N blocks 8192 B apart (LBO), 8-row K groups 1024 B apart
//             (SBO); one K = 16 step is +2048 B.
//
// Every wait on an mbarrier is bounded by a clock budget; on expiry the kernel raises
// FLAG_WAIT_TIMEOUT in the status word, drains what it has in flight, frees its tensor memory and
// returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_tc.h"

namespace lsgd {
namespace {

constexpr int BM = 128, BN = 128, BK = 64;
constexpr int kStages = 3;
constexpr int kStageBytes = (BM * BK + BN * BK) * 2;       // 32 KiB
constexpr int kABytes = BM * BK * 2;                        // 16 KiB
constexpr int kThreads = 192;                               // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kSmemBytes = kStages * kStageBytes + 1024;    // + slack for 1024-byte alignment
constexpr uint32_t kTmemCols = 128;
constexpr int kStagePitch = BN + 4;                         // floats; 16-byte accesses stay conflict-free
static_assert((size_t)BM * kStagePitch * 4 <= (size_t)kStages * kStageBytes, "staging tile must fit in the ring");
constexpr long long kWaitBudgetCycles = 2000000000LL;       // about one second

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false after the clock budget (or when another role has aborted).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t* status) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitBudgetCycles) {
      *abort_flag = 1;
      atomicOr(status, FLAG_WAIT_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version for this architecture
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}

__device__ __forceinline__ void mma_bf16(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

__global__ void __launch_bounds__(kThreads)
bgemm_bf16_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, GemmShape p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_bar[kStages], empty_bar[kStages], acc_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM, z = blockIdx.z;
  const int nk = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&acc_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abort_flag = &abort_s;

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer
    const int za = p.a_batched ? z : 0, zb = p.b_batched ? z : 0;
    int issued = 0;
    for (int kt = 0; kt < nk; ++kt) {
      const int s = kt % kStages;
      if (kt >= kStages && !mbar_wait(&empty_bar[s], ((kt / kStages) - 1) & 1, abort_flag, p.status)) break;
      uint8_t* sa = smem + s * kStageBytes;
      uint8_t* sb = sa + kABytes;
      mbar_expect_tx(&full_bar[s], kStageBytes);
      const int k0 = kt * BK;
      // two 64-wide boxes per operand; a box is [64 rows][64 elements = 128 B]
      if (p.a_mn) {
        tma_load_3d(sa, &map_a, &full_bar[s], m0, k0, za);
        tma_load_3d(sa + 8192, &map_a, &full_bar[s], m0 + 64, k0, za);
      } else {
        tma_load_3d(sa, &map_a, &full_bar[s], k0, m0, za);
        tma_load_3d(sa + 8192, &map_a, &full_bar[s], k0, m0 + 64, za);
      }
      if (p.b_mn) {
        tma_load_3d(sb, &map_b, &full_bar[s], n0, k0, zb);
        tma_load_3d(sb + 8192, &map_b, &full_bar[s], n0 + 64, k0, zb);
      } else {
        tma_load_3d(sb, &map_b, &full_bar[s], k0, n0, zb);
        tma_load_3d(sb + 8192, &map_b, &full_bar[s], k0, n0 + 64, zb);
      }
      issued = kt + 1;
    }
    if (*abort_flag) {
      // drain: wait (bounded) for the copies already issued before the CTA may exit
      const int first = issued > kStages ? issued - kStages : 0;
      for (int kt = first; kt < issued; ++kt) {
        const long long t0 = clock64();
        while (!mbar_try(&full_bar[kt % kStages], (kt / kStages) & 1) && clock64() - t0 < kWaitBudgetCycles) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------------------------------------------------------- MMA issuer
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                           ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    bool ok = true;
    for (int kt = 0; kt < nk && ok; ++kt) {
      const int s = kt % kStages;
      ok = mbar_wait(&full_bar[s], (kt / kStages) & 1, abort_flag, p.status);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t sa = smem_u32(smem + s * kStageBytes), sb = sa + kABytes;
#pragma unroll
      for (int k = 0; k < BK / 16; ++k) {
        const uint64_t da = p.a_mn ? smem_desc(sa + k * 2048, 8192, 1024) : smem_desc(sa + k * 32, 16, 1024);
        const uint64_t db = p.b_mn ? smem_desc(sb + k * 2048, 8192, 1024) : smem_desc(sb + k * 32, 16, 1024);
        mma_bf16(tmem_base, da, db, idesc, (kt | k) != 0 ? 1u : 0u);
      }
      mma_commit(&empty_bar[s]);   // the stage is free once these MMAs have read it
    }
    if (ok) mma_commit(&acc_bar);  // accumulator complete
  } else if (warp >= 2) {
    // ---------------------------------------------------------------- epilogue
    if (p.epilogue == GEMM_EPI_SGD) {
      // while the products run, pull this tile of x towards L2 (each thread one 512-byte row)
      const int m = m0 + (warp & 3) * 32 + lane;
      if (m < p.M) {
        const float* xr = p.x_upd + (int64_t)z * p.stride_c + (int64_t)m * p.ldc + n0;
#pragma unroll
        for (int j = 0; j < BN; j += 32)
          if (n0 + j < p.N) asm volatile("prefetch.global.L2 [%0];" ::"l"(xr + j));
      }
    }
    if (mbar_wait(&acc_bar, 0, abort_flag, p.status)) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // All MMAs have completed, so the operand ring is free: it becomes a staging tile through which
      // the accumulator is transposed from "one row per thread" (tensor-memory order) to "one row per
      // warp instruction" (512 contiguous bytes per store).  A warp only touches its own 32 rows.
      float* stage = reinterpret_cast<float*>(smem);
      const int q = warp & 3;                 // TMEM lane quarter this warp may read
      float* my_row = stage + (size_t)(q * 32 + lane) * kStagePitch;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; j += 4)
          *reinterpret_cast<uint4*>(my_row + c * 32 + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
      }
      __syncwarp();
      const int n = n0 + lane * 4;            // this lane's 4 columns
      const int64_t zc = (int64_t)z * p.stride_c;
      float bias4[4] = {0.f, 0.f, 0.f, 0.f};
      if (p.epilogue == GEMM_EPI_BIAS_RELU_BF16) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (n + j < p.N) bias4[j] = p.bias[(int64_t)z * p.stride_bias + n + j];
      }
      const bool full = (n + 4 <= p.N) && p.vec_ok;
      if (p.epilogue == GEMM_EPI_SGD) {
        // The accumulator is this block of the gradient: take the plain step x <- x - eta g here, in
        // place, and refresh the bf16 copy; g is not stored.  Rows are processed 8 at a time so that 8
        // loads of x are in flight per lane.
        constexpr int kBatch = 8;
#pragma unroll 1
        for (int r0 = 0; r0 < 32; r0 += kBatch) {
          float4 xv[kBatch];
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const int m = m0 + q * 32 + r0 + u;
            xv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m < p.M && n < p.N) {
              const float* xo = p.x_upd + zc + (int64_t)m * p.ldc + n;
              if (full) {
                xv[u] = *reinterpret_cast<const float4*>(xo);
              } else {
                xv[u].x = xo[0];
                if (n + 1 < p.N) xv[u].y = xo[1];
                if (n + 2 < p.N) xv[u].z = xo[2];
                if (n + 3 < p.N) xv[u].w = xo[3];
              }
            }
          }
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const int m = m0 + q * 32 + r0 + u;
            if (m < p.M && n < p.N) {
              const float4 g4 = *reinterpret_cast<const float4*>(stage + (size_t)(q * 32 + r0 + u) * kStagePitch + lane * 4);
              float xs[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w};
              const float gs[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                if (p.arith == 0) xs[j] = (float)__dsub_rn((double)xs[j], __dmul_rn(p.eta, (double)gs[j]));
                else if (p.arith == 1) xs[j] = (float)fma(-p.eta, (double)gs[j], (double)xs[j]);
                else xs[j] = fmaf(-(float)p.eta, gs[j], xs[j]);
              }
              const int64_t off = zc + (int64_t)m * p.ldc + n;
              float* xo = p.x_upd + off;
              uint16_t* so = p.x_shadow + off;
              if (full) {
                *reinterpret_cast<float4*>(xo) = make_float4(xs[0], xs[1], xs[2], xs[3]);
                __nv_bfloat162 h0 = __floats2bfloat162_rn(xs[0], xs[1]), h1 = __floats2bfloat162_rn(xs[2], xs[3]);
                uint2 u2;
                u2.x = *reinterpret_cast<uint32_t*>(&h0);
                u2.y = *reinterpret_cast<uint32_t*>(&h1);
                *reinterpret_cast<uint2*>(so) = u2;
              } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  if (n + j < p.N) {
                    xo[j] = xs[j];
                    __nv_bfloat16 hb = __float2bfloat16_rn(xs[j]);
                    so[j] = *reinterpret_cast<uint16_t*>(&hb);
                  }
              }
            }
          }
        }
      } else
#pragma unroll 4
      for (int rr = 0; rr < 32; ++rr) {
        const int m = m0 + q * 32 + rr;
        if (m >= p.M || n >= p.N) break;
        const float4 a4 = *reinterpret_cast<const float4*>(stage + (size_t)(q * 32 + rr) * kStagePitch + lane * 4);
        float v[4] = {a4.x, a4.y, a4.z, a4.w};
        if (p.epilogue == GEMM_EPI_F32) {
          float* out = static_cast<float*>(p.c) + zc + (int64_t)m * p.ldc + n;
          if (full) {
            *reinterpret_cast<float4*>(out) = a4;
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (n + j < p.N) out[j] = v[j];
          }
        } else {
          if (p.epilogue == GEMM_EPI_BIAS_RELU_BF16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = fmaxf(v[j] + bias4[j], 0.f);
          } else if (p.epilogue == GEMM_EPI_MASK_BF16) {
            const __nv_bfloat16* mk = static_cast<const __nv_bfloat16*>(p.mask) + (int64_t)z * p.stride_mask + (int64_t)m * p.ld_mask + n;
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (n + j < p.N) v[j] = (__bfloat162float(mk[j]) > 0.f) ? v[j] : 0.f;
          }
          __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.c) + zc + (int64_t)m * p.ldc + n;
          if (full) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(v[0], v[1]), h1 = __floats2bfloat162_rn(v[2], v[3]);
            uint2 u;
            u.x = *reinterpret_cast<uint32_t*>(&h0);
            u.y = *reinterpret_cast<uint32_t*>(&h1);
            *reinterpret_cast<uint2*>(out) = u;
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (n + j < p.N) out[j] = __float2bfloat16_rn(v[j]);
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  }
  return fn;
}

}  // namespace

bool make_operand_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t pitch_elems, int64_t batch,
                      int64_t batch_stride_elems) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (pitch_elems * 2) % 16 != 0) return false;
  if (batch > 1 && (batch_stride_elems * 2) % 16 != 0) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)(batch < 1 ? 1 : batch)};
  cuuint64_t strides[2] = {(cuuint64_t)pitch_elems * 2,
                           (cuuint64_t)(batch > 1 ? batch_stride_elems : pitch_elems * outer) * 2};
  cuuint32_t box[3] = {64, 64, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

cudaError_t launch_bgemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmShape& p, cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(bgemm_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  GemmShape q = p;
  const int64_t esz = (p.epilogue == GEMM_EPI_F32 || p.epilogue == GEMM_EPI_SGD) ? 4 : 2;
  const void* cbase = p.epilogue == GEMM_EPI_SGD ? static_cast<const void*>(p.x_upd) : p.c;
  q.vec_ok = ((reinterpret_cast<uintptr_t>(cbase) & 15u) == 0 && (p.ldc * esz) % 16 == 0 && (p.stride_c * esz) % 16 == 0) ? 1 : 0;
  dim3 grid((unsigned)((p.N + BN - 1) / BN), (unsigned)((p.M + BM - 1) / BM), (unsigned)p.batch);
  bgemm_bf16_kernel<<<grid, kThreads, kSmemBytes, s>>>(map_a, map_b, q);
  return cudaGetLastError();
}

}  // namespace lsgd
