// Top-k gating: router logits -> routing indexes and weights (the step before dispatch).
//
//   topk_idx[t, 0..K-1] = the K largest logits of token t in descending order (equal logits: lower
//                         expert index first)
//   topk_w[t, j]        = exp(l_j - l_0) / sum_j' exp(l_j' - l_0)   (fp32, sum in ascending j)
//
// One warp per token: the row of E logits is cached in shared memory, then K rounds of
// "largest remaining logit" run as a strided scan per lane plus a shuffle arg-max; the lane that
// owns the winner retires it.  The same routine is the front end of the fused gate + plan kernel.
#pragma once

#include "common.cuh"

namespace moe {

// Gating of one token by one warp.  `row`: E floats of this warp's shared memory (overwritten).
// On return lane j < K holds the j-th selected expert and its weight.
__device__ __forceinline__ void warp_gate_token(const float* __restrict__ logits_row, float* row, int E, int K, int lane,
                                                int32_t& idx_lane, float& w_lane) {
  for (int e = lane; e < E; e += 32) row[e] = __ldg(logits_row + e);
  __syncwarp();
  float sel_val = 0.0f;
  int32_t sel_idx = -1;
  for (int j = 0; j < K; ++j) {
    float bv = -INFINITY;
    int32_t bi = 0x7fffffff;
    for (int e = lane; e < E; e += 32) {   // ascending e and a strict compare: the lowest index among equals
      const float v = row[e];
      if (v > bv) {
        bv = v;
        bi = e;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, d);
      const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, d);
      if (ov > bv || (ov == bv && oi < bi)) {
        bv = ov;
        bi = oi;
      }
    }
    if (lane == j) {
      sel_val = bv;
      sel_idx = bi;
    }
    if (bi != 0x7fffffff && (bi & 31) == lane) row[bi] = -INFINITY;   // retired (logits are finite)
    __syncwarp();
  }
  const float top = __shfl_sync(0xffffffffu, sel_val, 0);
  const float ex = lane < K ? expf(sel_val - top) : 0.0f;
  float sum = 0.0f;
  for (int j = 0; j < K; ++j) sum += __shfl_sync(0xffffffffu, ex, j);
  w_lane = __fdiv_rn(ex, sum);
  idx_lane = sel_idx;
}

// Stand-alone gate: grid-stride over tokens, one warp per token.  Dynamic shared memory: warps * E floats.
__global__ void __launch_bounds__(256)
gate_topk_kernel(const float* __restrict__ logits, int32_t T, int32_t E, int32_t K, int32_t* __restrict__ topk_idx,
                 float* __restrict__ topk_w) {
  extern __shared__ float gate_rows[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpc = blockDim.x >> 5;
  float* row = gate_rows + warp * E;
  for (int32_t t = blockIdx.x * wpc + warp; t < T; t += gridDim.x * wpc) {
    int32_t idx;
    float w;
    warp_gate_token(logits + (size_t)t * E, row, E, K, lane, idx, w);
    if (lane < K) {
      topk_idx[(size_t)t * K + lane] = idx;
      topk_w[(size_t)t * K + lane] = w;
    }
    __syncwarp();
  }
}

}  // namespace moe
