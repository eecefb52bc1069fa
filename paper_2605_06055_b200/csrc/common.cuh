// Shared device-side definitions of libmoecomm (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moecomm.h"

namespace moe {

// Branch tiles of the planning pass: a tile is a run of consecutive branches
// (flat index t*K + j) of ONE source rank.  PLAN_WARPS warps each take ROUNDS
// rounds of 32 branches.
constexpr int PLAN_WARPS = 8;
constexpr int PLAN_THREADS = PLAN_WARPS * 32;
constexpr int ROUNDS_PREFILL = 4;  // 1024 branches per tile
constexpr int ROUNDS_DECODE = 1;   //  256 branches per tile

// Token ranges and tile ranges of the source ranks, passed by value as a
// __grid_constant__ kernel parameter so that it is ordered with the launch and
// needs no device copy.
struct RankMap {
  int32_t R;
  int32_t uniform_tokens;             // > 0: every rank owns this many tokens
  int32_t tile_shift;                 // log2(branches per tile)
  int32_t pad;
  int32_t tok_start[MOE_MAX_R + 1];   // first token of rank r
  int32_t tile_start[MOE_MAX_R + 1];  // first tile of rank r
};

// Control words at the head of the workspace.
struct Control {
  int32_t status;       // first device-detected error (moe_status_t), 0 = none
  int32_t scan_ticket;  // "last block done" counter of the offset scan
  int32_t work;         // work-item counter of the running row kernel (see row_kernels.cuh); zero between launches
  int32_t work_done;    // warps of the running row kernel that have finished; zero between launches
  int32_t pad[60];
};

__device__ __forceinline__ void raise_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ int32_t load_status(const int32_t* status) {
  return *reinterpret_cast<const volatile int32_t*>(status);
}

// Source rank of token t: the r with tok_start[r] <= t < tok_start[r+1].
__device__ __forceinline__ int32_t src_rank(const RankMap& map, int32_t t) {
  if (map.uniform_tokens > 0) return t / map.uniform_tokens;
  int32_t lo = 0, hi = map.R;  // invariant: tok_start[lo] <= t < tok_start[hi]
  while (hi - lo > 1) {
    int32_t mid = (lo + hi) >> 1;
    if (map.tok_start[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// Tile that holds flat branch b of a token owned by rank r.
__device__ __forceinline__ int32_t tile_of_branch(const RankMap& map, int32_t r, int32_t b, int32_t K) {
  return map.tile_start[r] + ((b - map.tok_start[r] * K) >> map.tile_shift);
}

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute may
// start while the previous kernel of the stream still runs; dependency_wait() returns once that kernel
// has completed and its writes are visible (at once when the launch carried no such attribute), and
// release_dependents() lets the NEXT kernel of the stream start early in the same way.  The row kernels
// release only after their own wait, so whatever completed before them has completed before any
// kernel that follows them starts.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

}  // namespace moe
