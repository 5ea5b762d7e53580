// Batched bf16 tensor-core matrix product: launcher interface (see gemm_tc.cu).
#pragma once
#include <cuda.h>

#include "internal.h"

namespace lsgd {

enum GemmEpilogue : int {
  GEMM_EPI_F32 = 0,             // C fp32 = acc
  GEMM_EPI_BIAS_RELU_BF16 = 1,  // C bf16 = relu(acc + bias[n])
  GEMM_EPI_MASK_BF16 = 2,       // C bf16 = mask[m][n] > 0 ? acc : 0
  GEMM_EPI_BF16 = 3,            // C bf16 = acc
  GEMM_EPI_SGD = 4,             // internal: x[m][n] <- x[m][n] - eta * acc (fp32, in place) and its bf16 copy
};

struct GemmShape {
  int M, N, K, batch;
  int a_mn, b_mn;               // 1: the M (resp. N) index is contiguous in memory, 0: the K index is
  int a_batched, b_batched;     // 0: every batch entry reads batch 0 of that operand
  int epilogue;
  void* c;                      // [batch][M][ldc]
  int64_t ldc, stride_c;        // in elements of C
  const float* bias;            // [batch][N] fp32 (stride_bias apart)
  int64_t stride_bias;
  const void* mask;             // bf16 [batch][M][ld_mask]
  int64_t ld_mask, stride_mask;
  float* x_upd;                 // GEMM_EPI_SGD: parameters, indexed like C (ldc, stride_c)
  uint16_t* x_shadow;           // GEMM_EPI_SGD: bf16 copy of the parameters, indexed like C
  double eta;                   // GEMM_EPI_SGD
  int arith;                    // GEMM_EPI_SGD: 0 fp64 unfused, 1 fp64 fma, 2 fp32 fma (as the update kernel)
  uint32_t* status;             // device status word (bounded-wait failures)
};

// 3-D tensor map {inner (contiguous), outer, batch} of bf16 with a 64 x 64 x 1 box and 128-byte swizzle.
// K-major operand: inner = K, outer = M or N.  MN-major operand: inner = M or N, outer = K.
bool make_operand_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t pitch_elems,
                      int64_t batch, int64_t batch_stride_elems);

// Tile maps of the epilogue (128-row boxes, 128 bytes wide): fp32 {32, 128, 1}, bf16 {64, 128, 1}.
bool make_tile_map_f32(CUtensorMap* map, const void* base, int64_t N, int64_t M, int64_t pitch_elems, int64_t batch,
                       int64_t batch_stride_elems);
bool make_tile_map_bf16(CUtensorMap* map, const void* base, int64_t N, int64_t M, int64_t pitch_elems, int64_t batch,
                        int64_t batch_stride_elems);

cudaError_t launch_bgemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmShape& p, cudaStream_t s);

}  // namespace lsgd
