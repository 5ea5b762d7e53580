// Leader election (Section 2.2): local leader = argmin of the election loss inside each group,
// global leader = argmin over all workers = best of the local leaders.
//
// Each loss is packed with its worker index into one 64-bit key, (orderable(loss) << 32) | index,
// so that an unsigned minimum is the argmin with ties resolved to the lowest index.  orderable()
// maps floats monotonically to uint32 with -0 and +0 equal and every NaN above +inf.  One warp
// handles one group at a time: lanes stride over the group's members and a shuffle tree takes the
// minimum; warp 0 then reduces the G group keys.  A single CTA does the whole election (P is the
// number of workers, at most a few thousand); the work is latency, not bandwidth.
//
// Optionally the kernel first finishes a two-stage loss reduction: loss_i = scale * sum_b
// partials[i][b], summed in fp64 by one warp per worker in a fixed order, so the value does not depend
// on scheduling.
#include "internal.h"

namespace lsgd {
namespace {

constexpr int kElectThreads = 1024;

__device__ __forceinline__ uint32_t orderable(float v) {
  if (v != v) return 0xFFFFFFFFu;            // NaN: after +inf
  uint32_t u = __float_as_uint(v + 0.0f);    // -0 + 0 = +0 in round-to-nearest
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ unsigned long long warp_min(unsigned long long k) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, k, o);
    k = other < k ? other : k;
  }
  return k;
}

__global__ void __launch_bounds__(kElectThreads) elect_kernel(ElectArgs p) {
  pdl_wait();
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  if (p.partials != nullptr) {
    for (int i = warp; i < p.P; i += nwarps) {
      const double acc = warp_sum_fixed(p.partials + (int64_t)i * p.n_partials, p.n_partials);
      if (lane == 0) p.loss_out[i] = (float)(acc * p.partial_scale);
    }
  } else if (p.loss_in != p.loss_out) {
    for (int i = threadIdx.x; i < p.P; i += blockDim.x) p.loss_out[i] = p.loss_in[i];
  }
  __syncthreads();
  for (int j = warp; j < p.G; j += nwarps) {
    const int m0 = p.tab.group_start[j], m1 = p.tab.group_start[j + 1];
    unsigned long long best = ~0ull;
    for (int m = m0 + lane; m < m1; m += 32) {
      const int i = p.tab.rows_by_group[m];
      const unsigned long long k = ((unsigned long long)orderable(p.loss_out[i]) << 32) | (uint32_t)i;
      best = k < best ? k : best;
    }
    best = warp_min(best);
    if (lane == 0) {
      p.group_keys[j] = best;
      if (p.update_local) {
        const int l = (int)(uint32_t)best;
        p.ll[j] = l;
        atomicAdd(p.count_local + l, 1);
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    unsigned long long best = ~0ull;
    for (int j = lane; j < p.G; j += 32) {
      const unsigned long long k = p.group_keys[j];
      best = k < best ? k : best;
    }
    best = warp_min(best);
    if (lane == 0 && p.update_global) {
      const int l = (int)(uint32_t)best;
      *p.gl = l;
      atomicAdd(p.count_global + l, 1);
    }
  }
}

// copies[r] <- the parameters of leader r (rows 0..G-1: local leaders, row G: the global leader)
__global__ void __launch_bounds__(256)
leader_copies_kernel(const float* __restrict__ x, float* __restrict__ copies, const int32_t* __restrict__ ll,
                     const int32_t* __restrict__ gl, int32_t G, int32_t r0, int64_t n4, int64_t ld) {
  const int r = r0 + blockIdx.y;
  const int src = r < G ? ll[r] : *gl;
  const float4* s4 = reinterpret_cast<const float4*>(x + (int64_t)src * ld);
  float4* d4 = reinterpret_cast<float4*>(copies + (int64_t)r * ld);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n4; c += stride) d4[c] = s4[c];
}

// Cross-device election, first half: the best of this device's OWN workers (the first n_own rows of the handle)
// as a key whose low word is the worker's GLOBAL index, so that keys of different devices compare by the rule of
// the single-device election (loss order, then lowest global index).  One warp.
__global__ void __launch_bounds__(32)
shard_best_key_kernel(const float* __restrict__ loss, const int32_t* __restrict__ global_index, int32_t n_own,
                      unsigned long long* __restrict__ key_out, int32_t* __restrict__ best_local) {
  const int lane = threadIdx.x;
  unsigned long long best = ~0ull;
  int arg = 0;
  for (int i = lane; i < n_own; i += 32) {
    const unsigned long long k = ((unsigned long long)orderable(loss[i]) << 32) | (uint32_t)global_index[i];
    if (k < best) {
      best = k;
      arg = i;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, best, o);
    const int oarg = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
    if (other < best) {
      best = other;
      arg = oarg;
    }
  }
  if (lane == 0) {
    *key_out = best;
    *best_local = arg;
  }
}

// Second half: the minimum of the gathered keys names the device that owns the global leader.  This device's
// global-leader index becomes its own best worker if it won, else the guest row that receives the winner's
// parameters.  result = {winning rank, winner's global worker index, this device's best local worker}.
__global__ void __launch_bounds__(32)
shard_pick_global_kernel(const unsigned long long* __restrict__ keys, int32_t world, int32_t my_rank, int32_t guest_row,
                         const int32_t* __restrict__ best_local, int32_t* __restrict__ gl, int32_t* __restrict__ result) {
  const int lane = threadIdx.x;
  unsigned long long best = ~0ull;
  int arg = 0;
  for (int r = lane; r < world; r += 32) {
    const unsigned long long k = keys[r];
    if (k < best || (k == best && r < arg)) {
      best = k;
      arg = r;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, best, o);
    const int oarg = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
    if (other < best || (other == best && oarg < arg)) {
      best = other;
      arg = oarg;
    }
  }
  if (lane == 0) {
    *gl = (arg == my_rank) ? *best_local : guest_row;
    result[0] = arg;
    result[1] = (int32_t)(uint32_t)best;
    result[2] = *best_local;
  }
}

}  // namespace

cudaError_t launch_shard_best_key(const float* loss, const int32_t* global_index, int32_t n_own, unsigned long long* key_out,
                                  int32_t* best_local, cudaStream_t s) {
  shard_best_key_kernel<<<1, 32, 0, s>>>(loss, global_index, n_own, key_out, best_local);
  return cudaGetLastError();
}

cudaError_t launch_shard_pick_global(const unsigned long long* keys, int32_t world, int32_t my_rank, int32_t guest_row,
                                     const int32_t* best_local, int32_t* gl, int32_t* result, cudaStream_t s) {
  shard_pick_global_kernel<<<1, 32, 0, s>>>(keys, world, my_rank, guest_row, best_local, gl, result);
  return cudaGetLastError();
}

cudaError_t launch_leader_copies(const float* x, float* copies, const int32_t* ll, const int32_t* gl, int32_t G, int32_t r0,
                                 int32_t r1, int64_t d, int64_t ld, cudaStream_t s) {
  if (r1 > G + 1) r1 = G + 1;
  if (r1 <= r0) return cudaSuccess;
  const int64_t n4 = (d + 3) / 4;
  int64_t bx = (n4 + 255) / 256;
  if (bx > 1184) bx = 1184;
  dim3 grid((unsigned)bx, (unsigned)(r1 - r0));
  leader_copies_kernel<<<grid, 256, 0, s>>>(x, copies, ll, gl, G, r0, n4, ld);
  return cudaGetLastError();
}

cudaError_t launch_elect(const ElectArgs& a, cudaStream_t s) {
  return launch_pdl(elect_kernel, dim3(1), dim3(kElectThreads), 0, s, a);
}

}  // namespace lsgd
