// Batched bf16 x bf16 -> fp32 matrix product on the 5th-generation tensor cores (tcgen05), used by
// the MLP population objective.  C[z] = A[z] . B[z], C is M x N, the contraction length is K.
//
// Persistent kernel, one CTA per SM, tiles of 128 x 128 handed out round-robin (tile = CTA, CTA +
// grid, ...), three roles:
//   * warp 0 (one thread): TMA producer.  cp.async.bulk.tensor loads of the operands (128-byte swizzle)
//     into a shared-memory ring (2 to 6 stages, see kSmemBytes) guarded by mbarriers; each stage holds a
//     128 x 64 slice of A and of B.  For epilogues that read a tile (the parameters x for the fused SGD step, the ReLU
//     mask) it also loads that tile into the epilogue buffer.
//   * warp 1 (one thread): issues tcgen05.mma (M = 128, N = 128, K = 16, cta_group::1) into one of TWO
//     fp32 accumulator tiles in tensor memory (2 x 128 columns), so the products of tile i+1 overlap
//     the epilogue of tile i.
//   * warps 2..9: epilogue (two warps per tensor-memory lane quarter, each half of the columns).  tcgen05.ld of the accumulator (thread = row), fused arithmetic, swizzled
//     st.shared into the epilogue buffers, then ONE thread issues TMA stores of the whole tile
//     (cp.async.bulk.tensor shared -> global): all global traffic of the kernel goes through TMA, edge
//     tiles are clipped by the tensor maps.
//
// Either operand may be "K-major" (the contraction index is contiguous in memory) or "MN-major"
// (the M resp. N index is contiguous): weights W[out][in], activations H[batch][feature] and their
// transposes are all consumed in place.  In shared memory a 64-element-wide box is always 128 bytes
// per row, so both majors use 1024-byte swizzle atoms:
//   K-major : rows = M/N index, 8-row groups 1024 B apart (SBO); one K = 16 step is +32 B;
//   MN-major: rows = K index, 64-wide M/N blocks 8192 B apart (LBO), 8-row K groups 1024 B apart
//             (SBO); one K = 16 step is +2048 B.
//
// Every wait on an mbarrier is bounded by a clock budget; on expiry the kernel raises
// FLAG_WAIT_TIMEOUT in the status word, every role leaves its loop, outstanding bulk stores are
// drained, tensor memory is freed and the CTA returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_tc.h"

namespace lsgd {
namespace {

constexpr int BM = 128, BK = 64;                            // tile rows, k-slice; the tile width BN (128 or 256) is a template parameter
constexpr int kMaxStages = 6;
constexpr int kABytes = BM * BK * 2;                        // 16 KiB
#ifndef LSGD_GEMM_EPI_WARPS
#define LSGD_GEMM_EPI_WARPS 8
#endif
constexpr int kEpiWarps = LSGD_GEMM_EPI_WARPS;              // kEpiWarps / 4 warps per tensor-memory lane quarter, sharing the columns
constexpr int kThreads = 64 + 32 * kEpiWarps;               // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
// Shared memory is carved per epilogue kind (at most 224 KiB + alignment slack):
//   bf16 outputs, 128-wide tiles : 6 operand stages (32 KiB) + 1 bf16 tile (32 KiB)
//   bf16 outputs, 256-wide tiles : 3 operand stages (48 KiB) + 1 bf16 tile (64 KiB); used when the product has
//                                  enough tiles to fill the machine twice -- a quarter less operand traffic
//                                  from L2 per flop, which is what bounds the M = 1024 forward products
//   fp32 output                  : 5 operand stages + 1 fp32 tile (64 KiB)
//   fused SGD step               : 2 operand stages (these products have K <= 128) + 2 fp32 tiles (the x tile of
//                                  the next tile is loaded while the current one is updated) + 1 bf16 tile
constexpr int kSmemBytes = 224 * 1024 + 1024;
constexpr long long kWaitBudgetCycles = 2000000000LL;       // about one second

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t* status,
                                          long long budget = kWaitBudgetCycles) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > budget) {
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
__device__ __forceinline__ void tma_store_3d(const void* src, const CUtensorMap* map, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
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
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory"); }

// Byte offset of the 16-byte unit `u` (0..7) of row `r` inside a [rows][128 B] box written / read by TMA
// with the 128-byte swizzle: the unit index is XORed with the row index modulo 8.
__device__ __forceinline__ uint32_t swz(int r, int u) { return (uint32_t)(r * 128 + ((u ^ (r & 7)) << 4)); }

struct Tile {
  int z, m0, n0;
};
__device__ __forceinline__ Tile tile_of(int t, int mt, int nt, int bn) {
  Tile q;
  q.n0 = (t % nt) * bn;
  t /= nt;
  q.m0 = (t % mt) * BM;
  q.z = t / mt;
  return q;
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
bgemm_bf16_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_aux, GemmShape p) {
  constexpr int kStageBytes = (BM * BK + BN * BK) * 2;     // 32 or 48 KiB
  constexpr int kEpiF32Bytes = BM * BN * 4;                 // fp32 tile: BN / 32 boxes of [128][32 floats]
  constexpr int kEpiBf16Bytes = BM * BN * 2;                // bf16 tile: BN / 64 boxes of [128][64 bf16]
  constexpr uint32_t kTmemCols = 2 * BN;                    // two accumulator tiles
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const bool sgd = (p.epilogue == GEMM_EPI_SGD);
  const int kStages = BN == 256 ? 3 : (sgd ? 2 : (p.epilogue == GEMM_EPI_F32 ? 5 : 6));
  const int nx = sgd ? 2 : 1;                               // input-tile buffers (x is double-buffered)
  uint8_t* buf_f32_0 = smem + kStages * kStageBytes;        // fp32 tile(s): C out, or x in/out (SGD)
  uint8_t* buf_b16 = buf_f32_0 + (sgd ? 2 : (p.epilogue == GEMM_EPI_F32 ? 1 : 0)) * kEpiF32Bytes;   // bf16 tile: C out, mask in, bf16 x out
  __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_full[2], acc_empty[2], in_full[2], in_free[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mt = (p.M + BM - 1) / BM, nt = (p.N + BN - 1) / BN;
  const int n_tiles = mt * nt * p.batch;
  const int nk = (p.K + BK - 1) / BK;
  const bool reads_tile = (p.epilogue == GEMM_EPI_SGD) || (p.epilogue == GEMM_EPI_MASK_BF16);

  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], kEpiWarps);   // one arrival per epilogue warp
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&in_full[b], 1);
      mbar_init(&in_free[b], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_aux) : "memory");
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
  // everything above touched only this CTA's own state; the operands may come from the kernel before
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer
    uint32_t it = 0;        // operand stages issued so far (all tiles)
    int local = 0;          // tiles this CTA has started
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
      const Tile q = tile_of(t, mt, nt, BN);
      const int za = p.a_batched ? q.z : 0, zb = p.b_batched ? q.z : 0;
      for (int kt = 0; kt < nk; ++kt, ++it) {
        const int s = it % kStages;
        ok = mbar_wait(&empty_bar[s], ((it / kStages) & 1) ^ 1, abort_flag, p.status);
        if (!ok) break;
        uint8_t* sa = smem + s * kStageBytes;
        uint8_t* sb = sa + kABytes;
        mbar_expect_tx(&full_bar[s], kStageBytes);
        const int k0 = kt * BK;
        // two 64-wide boxes per operand; a box is [64 rows][64 elements = 128 B]
        if (p.a_mn) {
          tma_load_3d(sa, &map_a, &full_bar[s], q.m0, k0, za);
          tma_load_3d(sa + 8192, &map_a, &full_bar[s], q.m0 + 64, k0, za);
        } else {
          tma_load_3d(sa, &map_a, &full_bar[s], k0, q.m0, za);
          tma_load_3d(sa + 8192, &map_a, &full_bar[s], k0, q.m0 + 64, za);
        }
#pragma unroll
        for (int j = 0; j < BN / 64; ++j) {
          if (p.b_mn) tma_load_3d(sb + j * 8192, &map_b, &full_bar[s], q.n0 + 64 * j, k0, zb);
          else tma_load_3d(sb + j * 8192, &map_b, &full_bar[s], k0, q.n0 + 64 * j, zb);
        }
      }
      if (ok && reads_tile) {
        // the epilogue's input tile, once the previous tile's stores have finished reading the buffers
        const int xb = local % nx;
        const int use = local / nx;       // how often this buffer has been used before
        ok = mbar_wait(&in_free[xb], (use & 1) ^ 1, abort_flag, p.status);
        if (!ok) break;
        if (sgd) {
          uint8_t* dst = buf_f32_0 + xb * kEpiF32Bytes;
          mbar_expect_tx(&in_full[xb], kEpiF32Bytes);
#pragma unroll
          for (int c = 0; c < 4; ++c) tma_load_3d(dst + c * 16384, &map_c, &in_full[xb], q.n0 + c * 32, q.m0, q.z);
        } else {
          mbar_expect_tx(&in_full[xb], kEpiBf16Bytes);
#pragma unroll
          for (int c = 0; c < BN / 64; ++c) tma_load_3d(buf_b16 + c * 16384, &map_aux, &in_full[xb], q.n0 + c * 64, q.m0, q.z);
        }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------------------------------------------------------- MMA issuer
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                           ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    uint32_t it = 0;
    int local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
      const int b = local & 1;
      ok = mbar_wait(&acc_empty[b], ((local >> 1) & 1) ^ 1, abort_flag, p.status);   // epilogue has drained it
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tacc = tmem_base + (uint32_t)(b * BN);
      for (int kt = 0; kt < nk; ++kt, ++it) {
        const int s = it % kStages;
        ok = mbar_wait(&full_bar[s], (it / kStages) & 1, abort_flag, p.status);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem_u32(smem + s * kStageBytes), sb = sa + kABytes;
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          const uint64_t da = p.a_mn ? smem_desc(sa + k * 2048, 8192, 1024) : smem_desc(sa + k * 32, 16, 1024);
          const uint64_t db = p.b_mn ? smem_desc(sb + k * 2048, 8192, 1024) : smem_desc(sb + k * 32, 16, 1024);
          mma_bf16(tacc, da, db, idesc, (kt | k) != 0 ? 1u : 0u);
        }
        mma_commit(&empty_bar[s]);   // the stage is free once these MMAs have read it
      }
      if (ok) mma_commit(&acc_full[b]);  // accumulator complete
    }
  } else if (warp >= 2) {
    // ---------------------------------------------------------------- epilogue (8 warps)
    const int q4 = warp & 3;                  // TMEM lane quarter this warp may read
    const int part = (warp - 2) >> 2;         // which share of the tile's columns this warp handles
    constexpr int kChunksPerPart = (BN / 32) / (kEpiWarps / 4);
    const int row = q4 * 32 + lane;           // row of the tile owned by this thread
    const bool leader = (threadIdx.x == 64);  // issues the bulk stores
    int local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
      const Tile q = tile_of(t, mt, nt, BN);
      const int b = local & 1;
      ok = mbar_wait(&acc_full[b], (local >> 1) & 1, abort_flag, p.status);
      const int xb = local % nx;
      if (ok && reads_tile) ok = mbar_wait(&in_full[xb], (local / nx) & 1, abort_flag, p.status);
      if (!ok) break;
      uint8_t* buf_f32 = buf_f32_0 + xb * kEpiF32Bytes;
      if (nx == 2) {
        // double-buffered input: the previous tile's stores were left in flight; before the shared bf16
        // tile is overwritten they must have been read, and then the previous x buffer is free again
        if (leader) {
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          if (local > 0) mbar_arrive(&in_free[xb ^ 1]);
        }
        epi_barrier();
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tacc = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(b * BN);
#pragma unroll 1
      for (int c = part * kChunksPerPart; c < (part + 1) * kChunksPerPart; ++c) {
        if (q.n0 + c * 32 >= p.N) break;                        // ragged last tile: these columns do not exist
        uint32_t r[32];
        tmem_ld32(tacc + (uint32_t)(c * 32), r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        uint8_t* f32_box = buf_f32 + c * 16384;                 // [128 rows][32 floats]
        uint8_t* b16_box = buf_b16 + (c >> 1) * 16384;          // [128 rows][64 bf16]; this chunk is half a row
        const int b16_u0 = (c & 1) * 4;
        if (p.epilogue == GEMM_EPI_F32) {
#pragma unroll
          for (int u = 0; u < 8; ++u)
            *reinterpret_cast<uint4*>(f32_box + swz(row, u)) = make_uint4(r[4 * u], r[4 * u + 1], r[4 * u + 2], r[4 * u + 3]);
        } else if (p.epilogue == GEMM_EPI_SGD) {
          // the accumulator is this block of the gradient: plain step x <- x - eta g on the staged x tile
          float xn[32];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const float4 x4 = *reinterpret_cast<const float4*>(f32_box + swz(row, u));
            const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float g = __uint_as_float(r[4 * u + j]);
              if (p.arith == 0) xn[4 * u + j] = (float)__dsub_rn((double)xs[j], __dmul_rn(p.eta, (double)g));
              else if (p.arith == 1) xn[4 * u + j] = (float)fma(-p.eta, (double)g, (double)xs[j]);
              else xn[4 * u + j] = fmaf(-(float)p.eta, g, xs[j]);
            }
            *reinterpret_cast<float4*>(f32_box + swz(row, u)) = make_float4(xn[4 * u], xn[4 * u + 1], xn[4 * u + 2], xn[4 * u + 3]);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(xn[8 * u], xn[8 * u + 1]), h1 = __floats2bfloat162_rn(xn[8 * u + 2], xn[8 * u + 3]);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(xn[8 * u + 4], xn[8 * u + 5]), h3 = __floats2bfloat162_rn(xn[8 * u + 6], xn[8 * u + 7]);
            uint4 w;
            w.x = *reinterpret_cast<uint32_t*>(&h0);
            w.y = *reinterpret_cast<uint32_t*>(&h1);
            w.z = *reinterpret_cast<uint32_t*>(&h2);
            w.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(b16_box + swz(row, b16_u0 + u)) = w;
          }
        } else {
          // bf16 outputs: bias + ReLU, ReLU mask, or plain conversion
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
          if (p.epilogue == GEMM_EPI_BIAS_RELU_BF16) {
            const float* bias = p.bias + (int64_t)q.z * p.stride_bias + q.n0 + c * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float bj = (q.n0 + c * 32 + j < p.N) ? bias[j] : 0.f;
              v[j] = fmaxf(v[j] + bj, 0.f);
            }
          } else if (p.epilogue == GEMM_EPI_MASK_BF16) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const uint4 mk = *reinterpret_cast<const uint4*>(b16_box + swz(row, b16_u0 + u));
              const __nv_bfloat162* mh = reinterpret_cast<const __nv_bfloat162*>(&mk);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float2 mf = __bfloat1622float2(mh[j]);
                if (!(mf.x > 0.f)) v[8 * u + 2 * j] = 0.f;
                if (!(mf.y > 0.f)) v[8 * u + 2 * j + 1] = 0.f;
              }
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(v[8 * u], v[8 * u + 1]), h1 = __floats2bfloat162_rn(v[8 * u + 2], v[8 * u + 3]);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(v[8 * u + 4], v[8 * u + 5]), h3 = __floats2bfloat162_rn(v[8 * u + 6], v[8 * u + 7]);
            uint4 w;
            w.x = *reinterpret_cast<uint32_t*>(&h0);
            w.y = *reinterpret_cast<uint32_t*>(&h1);
            w.z = *reinterpret_cast<uint32_t*>(&h2);
            w.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(b16_box + swz(row, b16_u0 + u)) = w;
          }
        }
      }
      // the accumulator has been read: hand it back to the MMA issuer (one arrival per warp)
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[b]);
      // make the tile visible to the bulk-copy engine, then one thread stores it
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      epi_barrier();
      if (leader) {
        if (p.epilogue == GEMM_EPI_F32 || p.epilogue == GEMM_EPI_SGD) {
#pragma unroll
          for (int c = 0; c < BN / 32; ++c)
            if (q.n0 + c * 32 < p.N) tma_store_3d(buf_f32 + c * 16384, &map_c, q.n0 + c * 32, q.m0, q.z);
        }
        if (p.epilogue != GEMM_EPI_F32) {
          const CUtensorMap* mo = (p.epilogue == GEMM_EPI_SGD) ? &map_aux : &map_c;
#pragma unroll
          for (int c = 0; c < BN / 64; ++c)
            if (q.n0 + c * 64 < p.N) tma_store_3d(buf_b16 + c * 16384, mo, q.n0 + c * 64, q.m0, q.z);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        if (nx == 1) {
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the buffers may be overwritten again
          if (reads_tile) mbar_arrive(&in_free[0]);
        }
      }
      if (nx == 1) epi_barrier();
    }
    if (leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // stores complete before the CTA exits
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------
// CTA-pair form (cta_group::2) for large products with bf16 output: a cluster of two CTAs on neighbouring SMs
// computes one 256 x 256 tile.  Each CTA loads only ITS half of both operands per k-slice -- 128 rows of A (its
// half of the tile's rows) and 128 rows of B (its half of the tile's columns), 32 KiB instead of the 48 KiB a
// 128 x 256 tile needs -- and one thread of the leader CTA (cluster rank 0) issues tcgen05.mma.cta_group::2
// (M = 256, N = 256, K = 16), which reads both CTAs' shared memory and writes both CTAs' tensor memory (each
// holds its 128 rows x 256 columns of the accumulator).  A third less operand traffic from L2 per flop, which is
// what bounds these products.  Every CTA fetches its own operand halves with ordinary tiled loads; no load is shared between CTAs.
//
// Synchronisation (all barriers live at the same shared-memory offsets in both CTAs):
//   full[s]      leader only; one arrival (the leader's expect_tx) plus the bytes of BOTH CTAs' loads, which
//                the peer directs at the leader's barrier (cp.async.bulk.tensor ... .cta_group::2);
//   empty[s]     each CTA; the leader's tcgen05.commit arrives on its own and on the peer's barrier;
//   acc_full[b]  each CTA; likewise by commit after the tile's last product;
//   acc_empty[b] leader only; 2 x kEpiWarps arrivals, the peer's epilogue warps arrive remotely.
// The two CTAs meet at a cluster barrier after set-up (barriers initialised, tensor memory allocated in both)
// and before they free tensor memory and exit.  Every mbarrier wait is bounded as in the kernel above.
#ifndef LSGD_GEMM_CTA_PAIRS
#define LSGD_GEMM_CTA_PAIRS 1     // 0: never use the CTA-pair kernel
#endif
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * kABytes;                 // 128 x 64 of A and 128 x 64 of B per CTA
constexpr int kPairEpiBytes = BM * 128 * 2;                  // half of this CTA's 128 x 256 bf16 output rows at a time
constexpr int kPairSmemBytes = kPairStages * kPairStageBytes + kPairEpiBytes + 1024;

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in the CTA with the given rank of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t a;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_addr), "r"(rank));
  return a;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(leader_bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void mma_bf16_pair(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}"
      ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc), "r"(0u)
      : "memory");
}
// arrival on an mbarrier (cluster address: this CTA's or the peer's) once the MMAs issued so far have completed
__device__ __forceinline__ void mma_commit_pair(uint32_t bar_cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
bgemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_c, GemmShape p) {
  constexpr int BN = 256;
  constexpr uint32_t kTmemCols = 2 * BN;                    // two accumulator tiles: all of tensor memory
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* buf_b16 = smem + kPairStages * kPairStageBytes;
  __shared__ uint64_t full_bar[kPairStages], empty_bar[kPairStages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();                     // 0: leader (issues the products), 1: peer
  const int mt = (p.M + 2 * BM - 1) / (2 * BM), nt = (p.N + BN - 1) / BN;
  const int n_tiles = mt * nt * p.batch;
  const int nk = (p.K + BK - 1) / BK;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < kPairStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 2 * kEpiWarps);   // one arrival per epilogue warp of either CTA
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();                                       // both CTAs' barriers and tensor memory are ready
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abort_flag = &abort_s;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0 && lane == 0) {
    // ---------------------------------------------------------------- TMA producer (each CTA: its own halves)
    uint32_t it = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles && ok; t += n_pairs) {
      const Tile q = tile_of(t, mt, nt, BN);                // q.m0 is in units of BM: scale to the 256-row tile
      const int m0 = 2 * q.m0 + (int)rank * BM, n0 = q.n0 + (int)rank * BM;
      const int za = p.a_batched ? q.z : 0, zb = p.b_batched ? q.z : 0;
      for (int kt = 0; kt < nk; ++kt, ++it) {
        const int s = it % kPairStages;
        ok = mbar_wait(&empty_bar[s], ((it / kPairStages) & 1) ^ 1, abort_flag, p.status);
        if (!ok) break;
        uint8_t* sa = smem + s * kPairStageBytes;
        uint8_t* sb = sa + kABytes;
        if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * kPairStageBytes);     // both CTAs' bytes land on this barrier
        const uint32_t bar = map_to_rank(smem_u32(&full_bar[s]), 0);
        const int k0 = kt * BK;
        tma_load_3d_pair(sa, &map_a, bar, k0, m0, za);
        tma_load_3d_pair(sa + 8192, &map_a, bar, k0, m0 + 64, za);
        tma_load_3d_pair(sb, &map_b, bar, k0, n0, zb);
        tma_load_3d_pair(sb + 8192, &map_b, bar, k0, n0 + 64, zb);
      }
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
    uint32_t it = 0;
    int local = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles && ok; t += n_pairs, ++local) {
      const int b = local & 1;
      ok = mbar_wait(&acc_empty[b], ((local >> 1) & 1) ^ 1, abort_flag, p.status);   // both epilogues have drained it
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tacc = tmem_base + (uint32_t)(b * BN);
      for (int kt = 0; kt < nk; ++kt, ++it) {
        const int s = it % kPairStages;
        ok = mbar_wait(&full_bar[s], (it / kPairStages) & 1, abort_flag, p.status);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem_u32(smem + s * kPairStageBytes), sb = sa + kABytes;
#pragma unroll
        for (int k = 0; k < BK / 16; ++k)
          mma_bf16_pair(tacc, smem_desc(sa + k * 32, 16, 1024), smem_desc(sb + k * 32, 16, 1024), idesc, (kt | k) != 0 ? 1u : 0u);
        // the stage is free in both CTAs once these products have read it
        mma_commit_pair(map_to_rank(smem_u32(&empty_bar[s]), 0));
        mma_commit_pair(map_to_rank(smem_u32(&empty_bar[s]), 1));
      }
      if (ok) {
        mma_commit_pair(map_to_rank(smem_u32(&acc_full[b]), 0));
        mma_commit_pair(map_to_rank(smem_u32(&acc_full[b]), 1));
      }
    }
  } else if (warp >= 2) {
    // ---------------------------------------------------------------- epilogue (8 warps in each CTA: its 128 rows)
    const int q4 = warp & 3;
    const int part = (warp - 2) >> 2;
    static_assert(kEpiWarps == 8, "the pair kernel's epilogue is written for two warp groups");
    const int row = q4 * 32 + lane;
    const bool leader_thread = (threadIdx.x == 64);
    int local = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles && ok; t += n_pairs, ++local) {
      const Tile q = tile_of(t, mt, nt, BN);
      const int m0 = 2 * q.m0 + (int)rank * BM;
      const int b = local & 1;
      ok = mbar_wait(&acc_full[b], (local >> 1) & 1, abort_flag, p.status);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tacc = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(b * BN);
      // the 256 columns leave in two halves through one 128-column staging buffer (that leaves room for six
      // operand stages); within a half, each of the two warp groups converts 64 columns into its own box
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          const int c = 4 * half + 2 * part + cc;               // 32-column chunk of the tile
          if (q.n0 + c * 32 >= p.N) break;
          uint32_t r[32];
          tmem_ld32(tacc + (uint32_t)(c * 32), r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          uint8_t* b16_box = buf_b16 + part * 16384;
          const int b16_u0 = cc * 4;
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
          if (p.epilogue == GEMM_EPI_BIAS_RELU_BF16) {
            const float* bias = p.bias + (int64_t)q.z * p.stride_bias + q.n0 + c * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float bj = (q.n0 + c * 32 + j < p.N) ? bias[j] : 0.f;
              v[j] = fmaxf(v[j] + bj, 0.f);
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(v[8 * u], v[8 * u + 1]), h1 = __floats2bfloat162_rn(v[8 * u + 2], v[8 * u + 3]);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(v[8 * u + 4], v[8 * u + 5]), h3 = __floats2bfloat162_rn(v[8 * u + 6], v[8 * u + 7]);
            uint4 w;
            w.x = *reinterpret_cast<uint32_t*>(&h0);
            w.y = *reinterpret_cast<uint32_t*>(&h1);
            w.z = *reinterpret_cast<uint32_t*>(&h2);
            w.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(b16_box + swz(row, b16_u0 + u)) = w;
          }
        }
        if (half == 1) {
          // this CTA's half of the accumulator has been read: tell the leader's issuer (one arrival per warp)
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&acc_empty[b]), 0));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        epi_barrier();
        if (leader_thread) {
#pragma unroll
          for (int bx = 0; bx < 2; ++bx) {
            const int col = q.n0 + half * 128 + bx * 64;
            if (col < p.N && m0 < p.M) tma_store_3d(buf_b16 + bx * 16384, &map_c, col, m0, q.z);
          }
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the buffer may be overwritten again
        }
        epi_barrier();
      }
    }
    if (leader_thread) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();      // nobody frees tensor memory or leaves while the other CTA may still signal or be read
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Self-test of the bounded wait of the product kernels: one warp waits, with a short budget, on a barrier that
// nothing completes (no copy or product is in flight), so the wait runs out, sets the status bit and returns.
__global__ void __launch_bounds__(32) gemm_wait_timeout_selftest_kernel(uint32_t* status, long long budget, int* gave_up) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar, 1);
  }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0, &abort_flag, status, budget);
  __syncwarp();
  if (threadIdx.x == 0) {
    *gave_up = ok ? 0 : 1;
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&bar)) : "memory");
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

bool encode(CUtensorMap* map, CUtensorMapDataType dt, int esz, const void* base, int64_t inner, int64_t outer,
            int64_t pitch_elems, int64_t batch, int64_t batch_stride_elems, int box_inner, int box_outer) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) || (pitch_elems * esz) % 16 != 0) return false;
  if (batch > 1 && (batch_stride_elems * esz) % 16 != 0) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)(batch < 1 ? 1 : batch)};
  cuuint64_t strides[2] = {(cuuint64_t)pitch_elems * esz,
                           (cuuint64_t)(batch > 1 ? batch_stride_elems : pitch_elems * outer) * esz};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

bool make_operand_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t pitch_elems, int64_t batch,
                      int64_t batch_stride_elems) {
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, inner, outer, pitch_elems, batch, batch_stride_elems, 64, 64);
}

bool make_tile_map_f32(CUtensorMap* map, const void* base, int64_t N, int64_t M, int64_t pitch_elems, int64_t batch,
                       int64_t batch_stride_elems) {
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, N, M, pitch_elems, batch, batch_stride_elems, 32, 128);
}

bool make_tile_map_bf16(CUtensorMap* map, const void* base, int64_t N, int64_t M, int64_t pitch_elems, int64_t batch,
                        int64_t batch_stride_elems) {
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, N, M, pitch_elems, batch, batch_stride_elems, 64, 128);
}

cudaError_t launch_gemm_wait_timeout_selftest(uint32_t* status, long long budget_cycles, int* gave_up, cudaStream_t s) {
  gemm_wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status, budget_cycles, gave_up);
  return cudaGetLastError();
}

cudaError_t launch_bgemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmShape& p, cudaStream_t s) {
  static OncePerDevice attr;
  if (!attr.here()) {
    cudaError_t e = cudaFuncSetAttribute(bgemm_bf16_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(bgemm_bf16_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr.here() = true;
  }
  const int sms = sm_count();
  // Tensor maps of the epilogue: map_c is C (fp32 or bf16) -- for the fused SGD step the parameter block
  // itself, loaded and stored; map_aux is the ReLU mask (input) or the bf16 copy of the parameters (output).
  CUtensorMap map_c, map_aux;
  bool ok = true;
  const int64_t nb = p.batch;
  switch (p.epilogue) {
    case GEMM_EPI_F32:
      ok = make_tile_map_f32(&map_c, p.c, p.N, p.M, p.ldc, nb, p.stride_c);
      map_aux = map_c;
      break;
    case GEMM_EPI_SGD:
      ok = make_tile_map_f32(&map_c, p.x_upd, p.N, p.M, p.ldc, nb, p.stride_c) &&
           make_tile_map_bf16(&map_aux, p.x_shadow, p.N, p.M, p.ldc, nb, p.stride_c);
      break;
    case GEMM_EPI_MASK_BF16:
      ok = make_tile_map_bf16(&map_c, p.c, p.N, p.M, p.ldc, nb, p.stride_c) &&
           make_tile_map_bf16(&map_aux, p.mask, p.N, p.M, p.ld_mask, nb, p.stride_mask);
      break;
    default:
      ok = make_tile_map_bf16(&map_c, p.c, p.N, p.M, p.ldc, nb, p.stride_c);
      map_aux = map_c;
      break;
  }
  if (!ok) return cudaErrorInvalidValue;
  const int64_t mtiles = (p.M + BM - 1) / BM;
  const int64_t tiles256 = (int64_t)((p.N + 255) / 256) * mtiles * p.batch;
  const bool bf16_out = p.epilogue != GEMM_EPI_F32 && p.epilogue != GEMM_EPI_SGD;
#if LSGD_GEMM_CTA_PAIRS
  // CTA pairs on 256 x 256 tiles: K-major operands, plain or bias + ReLU bf16 output, at least two rounds of tiles
  const int64_t pair_tiles = (int64_t)((p.N + 255) / 256) * ((p.M + 255) / 256) * p.batch;
  const int n_pairs = sms / 2;
  if ((p.epilogue == GEMM_EPI_BIAS_RELU_BF16 || p.epilogue == GEMM_EPI_BF16) && !p.a_mn && !p.b_mn && p.M >= 256 && p.N >= 256 &&
      pair_tiles >= 2 * (int64_t)n_pairs) {
    static OncePerDevice pair_attr;
    if (!pair_attr.here()) {
      cudaError_t e = cudaFuncSetAttribute(bgemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
      if (e != cudaSuccess) return e;
      pair_attr.here() = true;
    }
    const unsigned grid = 2u * (unsigned)(pair_tiles < n_pairs ? pair_tiles : n_pairs);
    return launch_pdl(bgemm_pair_kernel, dim3(grid), dim3(kThreads), kPairSmemBytes, s, map_a, map_b, map_c, p);
  }
#endif
  if (bf16_out && p.N >= 256 && tiles256 >= 2 * (int64_t)sms) {
    const unsigned grid = (unsigned)(tiles256 < sms ? tiles256 : sms);
    return launch_pdl(bgemm_bf16_kernel<256>, dim3(grid), dim3(kThreads), kSmemBytes, s, map_a, map_b, map_c, map_aux, p);
  } else {
    const int64_t tiles = (int64_t)((p.N + 127) / 128) * mtiles * p.batch;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    return launch_pdl(bgemm_bf16_kernel<128>, dim3(grid), dim3(kThreads), kSmemBytes, s, map_a, map_b, map_c, map_aux, p);
  }
}

}  // namespace lsgd
