// Top-k gating: router logits -> routing indexes and weights (the step before dispatch).
//
//   topk_idx[t, 0..K-1] = the K largest logits of token t in descending order (equal logits: lower
//                         expert index first)
//   topk_w[t, j]        = exp(l_j - l_0) / sum_j' exp(l_j' - l_0)   (fp32, sum in ascending j)
//
// One warp per token, K rounds of "largest remaining logit"; the lane that owns the winner retires it.
// Rows of up to 1024 logits live in registers (warp_gate_token_regs); longer rows are cached in
// shared memory and scanned with a shuffle arg-max (warp_gate_token).
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

// Order-preserving map from fp32 to uint32 (larger float <=> larger key), so that the warp-wide
// arg-max can use the single-instruction integer reductions (redux.sync).
__device__ __forceinline__ uint32_t sortable_key(float f) {
  const uint32_t u = __float_as_uint(f + 0.0f);   // -0 becomes +0: the two compare equal as floats
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// The same for E <= 32 * VPT with the row in registers: lane l holds experts l, l + 32, ... (coalesced
// loads) as sortable keys; 0 marks "absent or retired" (no finite float maps to key 0).  A round is
// VPT-1 integer max, one redux.max for the winning value, one redux.min for the lowest expert
// index that holds it, and a predicated retire: about 45 instructions instead of about 110 with a
// shuffle tree on (value, index) pairs.
template <int VPT>
__device__ __forceinline__ void warp_gate_token_regs(const float* __restrict__ logits_row, int E, int K, int lane,
                                                     int32_t& idx_lane, float& w_lane) {
  uint32_t v[VPT];
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const int e = lane + 32 * i;
    v[i] = e < E ? sortable_key(__ldg(logits_row + e)) : 0u;
  }
  uint32_t sel_key = 0;
  int32_t sel_idx = -1;
  for (int j = 0; j < K; ++j) {
    uint32_t local = v[0];
#pragma unroll
    for (int i = 1; i < VPT; ++i) local = max(local, v[i]);
    const uint32_t best = __reduce_max_sync(0xffffffffu, local);
    int32_t first = 0x7fffffff;                      // lowest expert index of mine that holds `best`
#pragma unroll
    for (int i = VPT - 1; i >= 0; --i) first = (v[i] == best) ? lane + 32 * i : first;
    // (a vote for the holder plus a shuffle of its index instead of this second reduction measured
    // slower: 35.2 vs 33.1 us at T=32768, E=256, K=8)
    const int32_t be = (int32_t)__reduce_min_sync(0xffffffffu, (uint32_t)first);
    if (lane == j) {
      sel_key = best;
      sel_idx = be;
    }
    // Retire the winner: a select on every register, so the array is never indexed dynamically.
    const int32_t hit = (be & 31) == lane ? (be >> 5) : -1;
#pragma unroll
    for (int i = 0; i < VPT; ++i) v[i] = (i == hit) ? 0u : v[i];
  }
  const float sel_val = key_to_float(sel_key);
  const float top = __shfl_sync(0xffffffffu, sel_val, 0);
  const float ex = lane < K ? expf(sel_val - top) : 0.0f;
  float sum = 0.0f;
  for (int j = 0; j < K; ++j) sum += __shfl_sync(0xffffffffu, ex, j);
  w_lane = __fdiv_rn(ex, sum);
  idx_lane = sel_idx;
}

// Stand-alone gate: grid-stride over tokens, one warp per token.  VPT > 0: register form for rows of at
// most 32 * VPT logits (one instantiation per row length class, so that short rows keep few registers
// and many warps per SM: 80 registers for a kernel holding every form, 3 CTAs per SM, against 6-8 CTAs
// per SM for the 256-logit form on its own).  VPT == 0: shared-memory form for longer rows; dynamic shared
// memory: warps * E floats.
template <int VPT>
__global__ void __launch_bounds__(256)
gate_topk_kernel(const float* __restrict__ logits, int32_t T, int32_t E, int32_t K, int32_t* __restrict__ topk_idx,
                 float* __restrict__ topk_w) {
  extern __shared__ float gate_rows[];
  release_dependents();   // a planner launched behind the gate (moe_gate_plan) may be scheduled; it waits for this kernel
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpc = blockDim.x >> 5;
  for (int32_t t = blockIdx.x * wpc + warp; t < T; t += gridDim.x * wpc) {
    int32_t idx;
    float w;
    if constexpr (VPT > 0) warp_gate_token_regs<VPT>(logits + (size_t)t * E, E, K, lane, idx, w);
    else warp_gate_token(logits + (size_t)t * E, gate_rows + warp * E, E, K, lane, idx, w);
    if (lane < K) {
      topk_idx[(size_t)t * K + lane] = idx;
      topk_w[(size_t)t * K + lane] = w;
    }
    __syncwarp();
  }
}

}  // namespace moe
