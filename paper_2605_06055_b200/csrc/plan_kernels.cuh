// Planning kernels: routing indexes -> counts, small offsets, large offsets.
//
// Section 5.2 (Prefill Layout, Prefill Notify) and the first step of Decode
// Dispatch (Section 5.3).  The small offset s[t,j] is a STABLE rank: the number
// of earlier branches (flat order t*K + j) of the same source rank that chose
// the same expert.  It is computed without atomics so that the result is the
// token-ordered one and is reproducible bit for bit:
//
//   plan_tile_kernel   one CTA per tile of consecutive branches of one source
//                      rank: in-warp rank by match_any + popc, per-warp running
//                      counters in shared memory, exclusive scan across warps
//                      -> in-tile rank of every branch, tile histogram [E]
//   plan_scan_kernel   one CTA per source rank: exclusive scan of the tile
//                      histograms over that rank's tiles ("per-block counting
//                      plus prefix accumulation over earlier blocks") -> tile
//                      bases, row r of M.  The CTA that finishes last turns M
//                      into n_exp, n_recv, c_rank and the large offsets o
//                      (exclusive scan in window order: expert, then source rank).
//   plan_finalize_kernel  PREFILL only: s = in-tile rank + tile base.
//                      (DECODE folds this step into the dispatch launch.)
//   plan_rank_kernel   few branches per rank (decode steps, small prefill chunks): the whole
//                      plan in one launch, small offsets final at once.
#pragma once

#include "common.cuh"

namespace moe {

template <int ROUNDS>
__global__ void __launch_bounds__(PLAN_THREADS)
plan_tile_kernel(const int32_t* __restrict__ topk_idx, const __grid_constant__ RankMap map, int32_t K, int32_t E,
                 int32_t* __restrict__ tile_rank, int32_t* __restrict__ tile_hist, int32_t* status) {
  extern __shared__ int32_t warp_hist[];  // [PLAN_WARPS][E]
  const int tile = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // Source rank of this tile (tile_start is nondecreasing; empty ranks own no tile).
  int r = 0;
  {
    int lo = 0, hi = map.R;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (map.tile_start[mid] <= tile) lo = mid; else hi = mid;
    }
    r = lo;
  }
  const int32_t b_begin = map.tok_start[r] * K + ((tile - map.tile_start[r]) << map.tile_shift);
  const int32_t b_end = min(b_begin + (ROUNDS * PLAN_THREADS), map.tok_start[r + 1] * K);

  for (int i = threadIdx.x; i < PLAN_WARPS * E; i += PLAN_THREADS) warp_hist[i] = 0;
  __syncthreads();

  int32_t* my_hist = warp_hist + warp * E;
  const int32_t warp_begin = b_begin + warp * (ROUNDS * 32);
  int32_t e_of[ROUNDS], rk[ROUNDS];
  const unsigned lt = lanemask_lt();
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = warp_begin + i * 32 + lane;
    int32_t e = -1;
    if (b < b_end) {
      e = __ldg(topk_idx + b);
      if (e < 0 || e >= E) {
        raise_status(status, MOE_ERR_BAD_INDEX);
        e = -1;
      }
    }
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int ahead = __popc(peers & lt);           // equal keys in lower lanes = earlier branches
    int32_t base = 0;
    if (e >= 0) base = my_hist[e];
    __syncwarp();
    if (e >= 0 && ahead == 0) my_hist[e] = base + __popc(peers);
    __syncwarp();
    e_of[i] = e;
    rk[i] = base + ahead;
  }
  __syncthreads();

  // Exclusive scan over the warps (warp w holds earlier branches than warp w+1).
  for (int e = threadIdx.x; e < E; e += PLAN_THREADS) {
    int32_t run = 0;
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) {
      const int32_t c = warp_hist[w * E + e];
      warp_hist[w * E + e] = run;
      run += c;
    }
    tile_hist[(size_t)tile * E + e] = run;
  }
  __syncthreads();

#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = warp_begin + i * 32 + lane;
    if (b < b_end) tile_rank[b] = (e_of[i] >= 0) ? rk[i] + my_hist[e_of[i]] : 0;
  }
}

// Exclusive scan of n (<= blockDim-independent) ints held in shared memory,
// done by warp 0: each lane owns a contiguous chunk.  out[i] = sum of in[0..i-1],
// out[n] = total.  `in` and `out` may not alias.
__device__ __forceinline__ void warp0_exclusive_scan(const int32_t* in, int32_t* out, int n) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    const int chunk = (n + 31) / 32;
    const int lo = min(lane * chunk, n), hi = min(lo + chunk, n);
    int32_t sum = 0;
    for (int i = lo; i < hi; ++i) sum += in[i];
    int32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t v = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += v;
    }
    int32_t run = incl - sum;
    for (int i = lo; i < hi; ++i) {
      out[i] = run;
      run += in[i];
    }
    if (lane == 31) out[n] = incl;
  }
}

// Notify step proper: turns the complete count matrix M into receive counts and large offsets.
// Run by ONE CTA (the last to finish counting).  sm: 2*E + 1 ints of shared memory.
__device__ __forceinline__ void build_large_offsets(const int32_t* __restrict__ M, int32_t E, int32_t R,
                                                    int32_t full_table, int32_t* __restrict__ c_rank,
                                                    int32_t* __restrict__ o, int32_t* __restrict__ n_exp,
                                                    int32_t* __restrict__ n_recv, int32_t* sm) {
  int32_t* nexp_s = sm;
  int32_t* pre_s = sm + E;
  const int E_r = E / R;
  for (int e = threadIdx.x; e < E; e += (int)blockDim.x) {
    int32_t acc = 0;
#pragma unroll 16
    for (int rr = 0; rr < R; ++rr) acc += __ldcg(M + (size_t)rr * E + e);   // independent loads: keep many in flight
    nexp_s[e] = acc;
    n_exp[e] = acc;
  }
  __syncthreads();
  warp0_exclusive_scan(nexp_s, pre_s, E);
  __syncthreads();
  // Window of rank d = experts d*E_r ..; offsets restart at 0 in every window.
  for (int e = threadIdx.x; e < E; e += (int)blockDim.x) {
    const int d = e / E_r;
    int32_t run = pre_s[e] - pre_s[d * E_r];
#pragma unroll 16
    for (int rr = 0; rr < R; ++rr) {
      o[(size_t)e * R + rr] = run;
      run += __ldcg(M + (size_t)rr * E + e);
    }
  }
  for (int d = threadIdx.x; d < R; d += (int)blockDim.x) n_recv[d] = pre_s[(d + 1) * E_r] - pre_s[d * E_r];
  if (full_table) {
    for (int i = threadIdx.x; i < R * R; i += (int)blockDim.x) {
      const int rr = i / R, d = i % R;
      int32_t acc = 0;
#pragma unroll 16
      for (int e = d * E_r; e < (d + 1) * E_r; ++e) acc += __ldcg(M + (size_t)rr * E + e);
      c_rank[i] = acc;
    }
  }
}

__global__ void __launch_bounds__(PLAN_THREADS)
plan_scan_kernel(int32_t* __restrict__ tile_hist /* in: histograms, out: exclusive bases */,
                 const __grid_constant__ RankMap map, int32_t E, int32_t full_table,
                 int32_t* __restrict__ M, int32_t* __restrict__ c_rank, int32_t* __restrict__ o,
                 int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv, Control* ctl) {
  extern __shared__ int32_t sm[];  // [E] n_exp, [E+1] prefix
  __shared__ int is_last;
  const int r = blockIdx.x;
  const int R = map.R;
  const int t0 = map.tile_start[r], t1 = map.tile_start[r + 1];

  for (int e = threadIdx.x; e < E; e += PLAN_THREADS) {
    int32_t run = 0;
#pragma unroll 16
    for (int t = t0; t < t1; ++t) {
      const size_t at = (size_t)t * E + e;
      const int32_t c = tile_hist[at];
      tile_hist[at] = run;
      run += c;
    }
    M[(size_t)r * E + e] = run;
  }

  // Last block done: the final CTA to arrive sees every row of M.
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(&ctl->scan_ticket, 1) == R - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  build_large_offsets(M, E, R, full_table, c_rank, o, n_exp, n_recv, sm);
  if (threadIdx.x == 0) ctl->scan_ticket = 0;  // ready for the next plan on this stream
}

// Compact planner for batches in which every source rank holds few branches (every decode step,
// small prefill chunks): ONE launch, one CTA per source rank.  The CTA walks its rank's branches in passes of WARPS*32, carrying the running
// per-expert count in shared memory, so the small offsets come out final (no tile bases), row r of M
// falls out at the end, and the last CTA to finish builds the large offsets.
template <int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
plan_rank_kernel(const int32_t* __restrict__ topk_idx, const __grid_constant__ RankMap map, int32_t K, int32_t E,
                 int32_t full_table, int32_t* __restrict__ s, int32_t* __restrict__ M, int32_t* __restrict__ c_rank,
                 int32_t* __restrict__ o, int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv, Control* ctl) {
  extern __shared__ int32_t sm[];   // [WARPS][E] per-warp counts, [E] running base  (reused: 2E+1 scan area)
  __shared__ int is_last;
  int32_t* warp_hist = sm;
  int32_t* rank_base = sm + WARPS * E;
  const int r = blockIdx.x, R = map.R;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int32_t b_begin = map.tok_start[r] * K, b_end = map.tok_start[r + 1] * K;
  const unsigned lt = lanemask_lt();

  for (int e = threadIdx.x; e < E; e += WARPS * 32) rank_base[e] = 0;
  for (int32_t pass = b_begin; pass < b_end; pass += WARPS * 32) {
    for (int i = threadIdx.x; i < WARPS * E; i += WARPS * 32) warp_hist[i] = 0;
    __syncthreads();
    const int32_t b = pass + warp * 32 + lane;
    int32_t e = -1;
    if (b < b_end) {
      e = __ldg(topk_idx + b);
      if (e < 0 || e >= E) {
        raise_status(&ctl->status, MOE_ERR_BAD_INDEX);
        e = -1;
      }
    }
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int ahead = __popc(peers & lt);
    if (e >= 0 && ahead == 0) warp_hist[warp * E + e] = __popc(peers);   // one round per pass: no carry inside a warp
    __syncthreads();
    for (int x = threadIdx.x; x < E; x += WARPS * 32) {
      int32_t run = rank_base[x];
#pragma unroll 8
      for (int w = 0; w < WARPS; ++w) {
        const int32_t c = warp_hist[w * E + x];
        warp_hist[w * E + x] = run;
        run += c;
      }
      rank_base[x] = run;
    }
    __syncthreads();
    if (b < b_end) s[b] = e >= 0 ? warp_hist[warp * E + e] + ahead : 0;
    __syncthreads();
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += WARPS * 32) M[(size_t)r * E + e] = rank_base[e];

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(&ctl->scan_ticket, 1) == R - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  build_large_offsets(M, E, R, full_table, c_rank, o, n_exp, n_recv, sm);
  if (threadIdx.x == 0) ctl->scan_ticket = 0;
}

template <int ROUNDS>
__global__ void __launch_bounds__(PLAN_THREADS)
plan_finalize_kernel(const int32_t* __restrict__ topk_idx, const __grid_constant__ RankMap map, int32_t K, int32_t E,
                     const int32_t* __restrict__ tile_rank, const int32_t* __restrict__ tile_base,
                     int32_t* __restrict__ s) {
  const int tile = blockIdx.x;
  int r = 0;
  {
    int lo = 0, hi = map.R;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (map.tile_start[mid] <= tile) lo = mid; else hi = mid;
    }
    r = lo;
  }
  const int32_t b_begin = map.tok_start[r] * K + ((tile - map.tile_start[r]) << map.tile_shift);
  const int32_t b_end = min(b_begin + (ROUNDS * PLAN_THREADS), map.tok_start[r + 1] * K);
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = b_begin + i * PLAN_THREADS + threadIdx.x;
    if (b < b_end) {
      const int32_t e = __ldg(topk_idx + b);
      s[b] = (e >= 0 && e < E) ? tile_rank[b] + tile_base[(size_t)tile * E + e] : 0;
    }
  }
}

}  // namespace moe
