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
//                      histograms over that rank's tiles (counts per tile, then a
//                      prefix over the earlier tiles of the same rank: Section 5.2,
//                      Prefill Layout) -> tile bases, row r of M.  Then M becomes n_exp, n_recv, c_rank and the
//                      large offsets o (exclusive scan in window order: expert, then
//                      source rank): by every CTA for its own window when the R CTAs
//                      run as one thread-block cluster (rows of M exchanged through
//                      distributed shared memory), else by the CTA that finishes last.
//   plan_finalize_kernel  PREFILL only: s = in-tile rank + tile base.
//                      (DECODE folds this step into the dispatch launch.)
//   plan_rank_kernel   few branches per rank (decode steps, small prefill chunks): the whole
//                      plan in one launch, small offsets final at once.
// The tile, scan and finalize kernels are chained by programmatic stream serialization: each lets
// the next be scheduled at its start, and each waits for the one in front before it touches that
// kernel's output.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace moe {

template <int ROUNDS>
__global__ void __launch_bounds__(PLAN_THREADS)
plan_tile_kernel(const int32_t* __restrict__ topk_idx, const __grid_constant__ RankMap map, int32_t K, int32_t E,
                 int32_t* __restrict__ tile_rank, int32_t* __restrict__ tile_hist, int32_t* status) {
  extern __shared__ int32_t warp_hist[];  // [PLAN_WARPS][E]
  dependency_wait();      // behind the gate kernel (moe_gate_plan): its indexes are complete; else returns at once
  release_dependents();   // the scan kernel may be scheduled now; it waits for this kernel before reading anything
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

  int32_t* my_hist = warp_hist + warp * E;
  const int32_t warp_begin = b_begin + warp * (ROUNDS * 32);
  int32_t e_of[ROUNDS], rk[ROUNDS];
  const unsigned lt = lanemask_lt();
  // All of the warp's routing indexes first (independent loads, one memory round trip that overlaps
  // the clearing of the counters), then the rounds.
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = warp_begin + i * 32 + lane;
    e_of[i] = b < b_end ? __ldg(topk_idx + b) : -1;
  }
  for (int i = threadIdx.x; i < PLAN_WARPS * E; i += PLAN_THREADS) warp_hist[i] = 0;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = warp_begin + i * 32 + lane;
    int32_t e = e_of[i];
    if (b < b_end && (e < 0 || e >= E)) {
      raise_status(status, MOE_ERR_BAD_INDEX);
      e = -1;
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
    int32_t c[PLAN_WARPS];
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) c[w] = warp_hist[w * E + e];   // all loads before the first store
    int32_t run = 0;
#pragma unroll
    for (int w = 0; w < PLAN_WARPS; ++w) {
      warp_hist[w * E + e] = run;
      run += c[w];
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

// Exclusive scan of n ints in shared memory by the whole CTA (blockDim.x a multiple of 32, <= 1024).
// out[i] = in[0] + .. + in[i-1], out[n] = total.  `in` and `out` may not alias; `warp_sums` holds 33 ints.
__device__ __forceinline__ void block_exclusive_scan(const int32_t* in, int32_t* out, int n, int32_t* warp_sums) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int32_t carry = 0;
  for (int base = 0; base < n; base += blockDim.x) {   // uniform trip count
    const int i = base + threadIdx.x;
    const int32_t v = i < n ? in[i] : 0;
    int32_t incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t u = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += u;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int32_t w = lane < nwarps ? warp_sums[lane] : 0;
      int32_t wi = w;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int32_t u = __shfl_up_sync(0xffffffffu, wi, d);
        if (lane >= d) wi += u;
      }
      warp_sums[lane] = wi - w;              // exclusive prefix of the warp totals
      if (lane == 31) warp_sums[32] = wi;    // chunk total
    }
    __syncthreads();
    if (i < n) out[i] = carry + warp_sums[warp] + incl - v;
    carry += warp_sums[32];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[n] = carry;
}

// Shared memory the Notify step needs: n_exp [E], prefix [E+1], warp sums [33], and, when the count
// matrix is small enough to stage, M transposed and padded as [E][R+1].
constexpr int NOTIFY_STAGE_MAX = 8192;   // entries of M staged in shared memory
__host__ __device__ constexpr int notify_smem_ints(int E, int R) {
  return 2 * E + 1 + 33 + (R * E <= NOTIFY_STAGE_MAX ? E * (R + 1) : 0);
}

// Notify step proper: turns the complete count matrix M into receive counts and large offsets.
// Run by ONE CTA (the last to finish counting).  sm: notify_smem_ints(E, R) ints of shared memory.
//
// Staged path (R*E <= NOTIFY_STAGE_MAX): M is read from L2 once, in one batch of independent
// coalesced loads, into a transposed [E][R+1] tile (the odd row pitch keeps both the column walk of
// one thread per expert and the final row-major copy free of bank conflicts); the prefix over source
// ranks is formed in place and o leaves the SM as one coalesced stream.  A thread that stored its own
// 16 offsets of 4 bytes at a 64-byte pitch would instead occupy the store path for one cycle per
// 32-byte sector, which measured 2.9 us for 4096 offsets.
// Direct path (large R*E): loads first and in batches; no store sits between two loads, because the
// compiler cannot know that o and M never overlap and would serialise them at one L2 round trip each.
__device__ __forceinline__ void build_large_offsets(const int32_t* __restrict__ M, int32_t E, int32_t R,
                                                    int32_t full_table, int32_t align, int32_t* __restrict__ c_rank,
                                                    int32_t* __restrict__ o, int32_t* __restrict__ n_exp,
                                                    int32_t* __restrict__ n_recv, int32_t* sm) {
  int32_t* nexp_s = sm;
  int32_t* pre_s = sm + E;
  int32_t* warp_sums = sm + 2 * E + 1;
  int32_t* tile = sm + 2 * E + 1 + 33;   // [E][R+1], staged path only
  const int E_r = E / R, P = R + 1;
  const bool staged = R * E <= NOTIFY_STAGE_MAX;
  if (staged) {
    for (int i0 = 0; i0 < R * E; i0 += 4 * (int)blockDim.x) {   // batches of independent loads
      int32_t v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + k * (int)blockDim.x + (int)threadIdx.x;
        v[k] = i < R * E ? __ldcg(M + i) : 0;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + k * (int)blockDim.x + (int)threadIdx.x;   // i = r*E + e
        if (i < R * E) tile[(i % E) * P + i / E] = v[k];
      }
    }
    __syncthreads();
  }
  for (int e = threadIdx.x; e < E; e += (int)blockDim.x) {
    int32_t acc = 0;
    if (staged) {
      for (int rr = 0; rr < R; ++rr) acc += tile[e * P + rr];
    } else {
#pragma unroll 16
      for (int rr = 0; rr < R; ++rr) acc += __ldcg(M + (size_t)rr * E + e);
    }
    nexp_s[e] = (acc + align - 1) / align * align;   // rows the expert's run occupies (align = 1: its count)
    n_exp[e] = acc;
  }
  __syncthreads();
  block_exclusive_scan(nexp_s, pre_s, E, warp_sums);
  __syncthreads();
  // Window of rank d = experts d*E_r ..; offsets restart at 0 in every window.
  if (full_table) {   // per-rank branch counts, before the staged tile is overwritten by the offsets
    for (int i = threadIdx.x; i < R * R; i += (int)blockDim.x) {
      const int rr = i / R, d = i % R;
      int32_t acc = 0;
#pragma unroll 16
      for (int e = d * E_r; e < (d + 1) * E_r; ++e) acc += staged ? tile[e * P + rr] : __ldcg(M + (size_t)rr * E + e);
      c_rank[i] = acc;
    }
    __syncthreads();
  }
  if (staged) {
    for (int e = threadIdx.x; e < E; e += (int)blockDim.x) {
      int32_t run = pre_s[e] - pre_s[(e / E_r) * E_r];
      for (int rr = 0; rr < R; ++rr) {
        const int32_t m = tile[e * P + rr];
        tile[e * P + rr] = run;
        run += m;
      }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < E * R; i += (int)blockDim.x) o[i] = tile[(i / R) * P + i % R];   // coalesced
  } else {
    for (int e = threadIdx.x; e < E; e += (int)blockDim.x) {
      int32_t run = pre_s[e] - pre_s[(e / E_r) * E_r];
      for (int r0 = 0; r0 < R; r0 += 16) {
        int32_t m[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) m[k] = r0 + k < R ? __ldcg(M + (size_t)(r0 + k) * E + e) : 0;
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if (r0 + k < R) {
            o[(size_t)e * R + r0 + k] = run;
            run += m[k];
          }
      }
    }
  }
  for (int d = threadIdx.x; d < R; d += (int)blockDim.x) n_recv[d] = pre_s[(d + 1) * E_r] - pre_s[d * E_r];
}

// Notify inside a thread-block cluster (the R CTAs of plan_rank_kernel or plan_scan_kernel launched as
// ONE cluster).
// Every CTA keeps its row of M in shared memory; after a cluster barrier CTA d builds the offsets
// of window d (its E/R experts x R source ranks) straight from the other CTAs' shared memory, so
// the count matrix makes no trip through global memory, no CTA waits on a ticket, and the R windows
// are scanned in parallel instead of by the last CTA alone.
// Shared memory behind the planner's own: gathered tile [E/R][R+1], padded totals [E/R], their
// prefix [E/R + 1], warp sums [33].
__host__ __device__ constexpr int cluster_notify_smem_ints(int E, int R) {
  return (E / R) * (R + 1) + 2 * (E / R) + 1 + 33;
}

// How the planners' Notify step runs: by the last CTA to finish (a ticket), by every CTA of a cluster for its own
// window, or not at all (one rank's local part of a multi-rank plan: moe_layout).
enum { PLAN_TICKET = 0, PLAN_CLUSTER = 1, PLAN_LOCAL = 2 };

// The two halves of a cluster barrier.  Between them a CTA does what needs nobody else's data (arrive has release,
// wait has acquire semantics: what a CTA wrote to its shared memory before arriving is visible to the others after
// their wait).  Every thread of every CTA of the cluster executes each of them once per phase.
__device__ __forceinline__ void cluster_arrive() { __cluster_barrier_arrive(); }
__device__ __forceinline__ void cluster_wait() { __cluster_barrier_wait(); }
// Arrival that publishes nothing: for a barrier whose only meaning is "I have finished READING your shared memory".
// (The releasing form waits until this thread's earlier global stores are visible, which is not wanted there.)
__device__ __forceinline__ void cluster_arrive_relaxed() { __cluster_barrier_arrive_relaxed(); }

// Offsets of ONE window (rank d: its E/R experts x R source ranks) from the gathered tile of counts; every thread
// of the CTA calls it after the tile is complete (a __syncthreads behind the gather).
// scratch: cluster_notify_smem_ints(E, R) ints: tile [E/R][R+1] with entry (el, rr) = M[rr][d*E/R + el], padded
// totals [E/R], their prefix [E/R + 1], warp sums [33].
__device__ __forceinline__ void window_offsets(int32_t* scratch, int32_t E, int32_t R, int32_t d, int32_t full_table,
                                               int32_t align, int32_t* __restrict__ c_rank, int32_t* __restrict__ o,
                                               int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv) {
  const int E_r = E / R, P = R + 1, nthreads = (int)blockDim.x, tid = (int)threadIdx.x;
  int32_t* tile = scratch;
  int32_t* tot = tile + E_r * P;      // [E_r] rows each expert's run occupies
  int32_t* pre = tot + E_r;           // [E_r + 1]
  int32_t* warp_sums = pre + E_r + 1;
  if (full_table) {
    for (int rr = tid; rr < R; rr += nthreads) {     // branches from source rank rr to this rank
      int32_t acc = 0;
      for (int el = 0; el < E_r; ++el) acc += tile[el * P + rr];
      c_rank[(size_t)rr * R + d] = acc;
    }
    __syncthreads();
  }
  if (E_r <= 32 && R <= 16) {
    // Few experts per window (every decode configuration): one warp does both prefixes from registers -- lane el
    // loads its expert's R counts at once, writes their running sums back, and the padded totals are scanned
    // across the lanes by shuffles.  (With a dependent load-store chain per source rank and a block-wide scan
    // behind it these two steps took 1.0 us.)
    if (tid < 32) {
      const int el = tid;
      const bool live = el < E_r;
      int32_t m[16];
#pragma unroll
      for (int rr = 0; rr < 16; ++rr) m[rr] = (live && rr < R) ? tile[el * P + rr] : 0;
      int32_t run = 0;
#pragma unroll
      for (int rr = 0; rr < 16; ++rr) {
        if (live && rr < R) tile[el * P + rr] = run;
        run += m[rr];
      }
      if (live) n_exp[d * E_r + el] = run;
      const int32_t padded = live ? (run + align - 1) / align * align : 0;
      int32_t incl = padded;
#pragma unroll
      for (int dd = 1; dd < 32; dd <<= 1) {
        const int32_t u = __shfl_up_sync(0xffffffffu, incl, dd);
        if (tid >= dd) incl += u;
      }
      if (live) pre[el] = incl - padded;
      if (tid == 31) pre[E_r] = incl;
    }
    __syncthreads();
  } else {
    for (int el = tid; el < E_r; el += nthreads) {     // exclusive prefix over source ranks, in place
      int32_t run = 0;
      for (int rr = 0; rr < R; ++rr) {
        const int32_t m = tile[el * P + rr];
        tile[el * P + rr] = run;
        run += m;
      }
      n_exp[d * E_r + el] = run;
      tot[el] = (run + align - 1) / align * align;
    }
    __syncthreads();
    block_exclusive_scan(tot, pre, E_r, warp_sums);
    __syncthreads();
  }
  for (int q = tid; q < E_r * R; q += nthreads)      // o[d*E_r + el][rr], one coalesced stream
    o[(size_t)d * E_r * R + q] = pre[q / R] + tile[(q / R) * P + q % R];
  if (tid == 0) n_recv[d] = pre[E_r];
}

// On entry every thread of the CTA has ARRIVED at the cluster barrier that says "my row of M is complete".
__device__ __forceinline__ void cluster_notify(const int32_t* my_row /* shared, [E] */, int32_t* scratch, int32_t E,
                                               int32_t R, int32_t d, int32_t full_table, int32_t align,
                                               int32_t* __restrict__ c_rank, int32_t* __restrict__ o,
                                               int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int E_r = E / R, P = R + 1, nthreads = (int)blockDim.x, tid = (int)threadIdx.x;
  int32_t* tile = scratch;            // [E_r][P]: entry (el, rr) = M[rr][d*E_r + el]
  cluster_wait();                     // every CTA's row of M is complete and visible
  for (int q = tid; q < E_r * R; q += nthreads) {   // consecutive threads: consecutive experts of one remote row
    const int el = q % E_r, rr = q / E_r;
    const int32_t* remote = cluster.map_shared_rank(my_row, rr);
    tile[el * P + rr] = remote[d * E_r + el];
  }
  // This thread reads no other CTA's shared memory from here on.  Its remote loads have returned -- the stores
  // above carry their values -- and the barrier orders nothing else, so the arrival need not release anything
  // (a releasing arrival here waits for the s and M stores to drain: 0.3 us).
  cluster_arrive_relaxed();
  __syncthreads();
  window_offsets(scratch, E, R, d, full_table, align, c_rank, o, n_exp, n_recv);
  cluster_wait();                     // no CTA leaves while its row may still be read
}

__global__ void __launch_bounds__(PLAN_THREADS)
plan_scan_kernel(int32_t* __restrict__ tile_hist /* in: histograms, out: exclusive bases */,
                 const __grid_constant__ RankMap map, int32_t E, int32_t full_table, int32_t align,
                 int32_t* __restrict__ M, int32_t* __restrict__ c_rank, int32_t* __restrict__ o,
                 int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv, Control* ctl,
                 int32_t mode /* PLAN_TICKET, PLAN_CLUSTER (the grid is one cluster of R CTAs) or PLAN_LOCAL */,
                 int32_t first_rank /* rank of CTA 0 (PLAN_LOCAL: the grid is the one CTA of the rank that owns tokens) */) {
  // notify_smem_ints(E, R) ints, or (as a cluster) this CTA's row of M [E] followed by cluster_notify_smem_ints(E, R)
  extern __shared__ int32_t sm[];
  __shared__ int is_last;
  release_dependents();   // lets the kernel behind (finalize, or a dispatch) be scheduled; it waits for this one
  dependency_wait();      // the tile histograms are complete (returns at once under a plain launch)
  const bool as_cluster = mode == PLAN_CLUSTER;
  const int r = blockIdx.x + first_rank;
  const int R = map.R;
  const int t0 = map.tile_start[r], t1 = map.tile_start[r + 1];

  for (int e = threadIdx.x; e < E; e += PLAN_THREADS) {
    int32_t run = 0;
    for (int tb = t0; tb < t1; tb += 16) {   // loads first, then the in-place stores (see build_large_offsets)
      int32_t c[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) c[k] = (tb + k < t1) ? tile_hist[(size_t)(tb + k) * E + e] : 0;
#pragma unroll
      for (int k = 0; k < 16; ++k)
        if (tb + k < t1) {
          tile_hist[(size_t)(tb + k) * E + e] = run;
          run += c[k];
        }
    }
    M[(size_t)r * E + e] = run;
    if (as_cluster) sm[e] = run;
  }
  if (as_cluster) {   // see cluster_notify: every CTA builds its own window's offsets from the rows in shared memory
    __syncthreads();
    cluster_arrive();   // this CTA's row is complete
    cluster_notify(sm, sm + E, E, R, r, full_table, align, c_rank, o, n_exp, n_recv);
    return;
  }
  if (mode == PLAN_LOCAL) return;   // this rank's row of M and its tile bases are all that was asked for

  // Last block done: the final CTA to arrive sees every row of M.
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(&ctl->scan_ticket, 1) == R - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  build_large_offsets(M, E, R, full_table, align, c_rank, o, n_exp, n_recv, sm);
  if (threadIdx.x == 0) ctl->scan_ticket = 0;  // ready for the next plan on this stream
}

// Count exchange through the pooled memory (Section 5.2, Notify: the ranks exchange count metadata only).  Behind
// the arrival flags of a rank's state region lies a mailbox of two buffers, each [R][E] counts and [R] epoch
// words; an exchange with epoch e uses buffer e & 1.
__host__ __device__ constexpr size_t counts_box_bytes(int E, int R) {
  return 2 * ((size_t)R * E + R) * sizeof(int32_t);
}
__device__ __forceinline__ int32_t* box_counts(unsigned char* box, int E, int R, uint32_t epoch) {
  return reinterpret_cast<int32_t*>(box) + (size_t)(epoch & 1u) * ((size_t)R * E + R);
}

// Compact planner for batches in which every source rank holds few branches (every decode step,
// small prefill chunks): ONE launch, one CTA per source rank.  The CTA walks its rank's branches in
// passes of WARPS*32, carrying the running per-expert count in shared memory, so the small offsets
// come out final (no tile bases), row r of M falls out at the end, and the last CTA to finish
// builds the large offsets.
// Shared memory: counts [E][WARPS+1] (expert-major with an odd pitch: neither the leaders' scattered
// writes -- same warp column, different experts -- nor the scanning warp's row reads collide on a
// bank), running base [E]; reused by the Notify step at the end.
__host__ __device__ constexpr int rank_plan_smem_ints(int E, int R, int warps) {
  return (warps + 2) * E > notify_smem_ints(E, R) ? (warps + 2) * E : notify_smem_ints(E, R);
}

template <int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
plan_rank_kernel(const int32_t* __restrict__ topk_idx, const __grid_constant__ RankMap map, int32_t K, int32_t E,
                 int32_t full_table, int32_t align, int32_t* __restrict__ s, int32_t* __restrict__ M,
                 int32_t* __restrict__ c_rank,
                 int32_t* __restrict__ o, int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv, Control* ctl,
                 int32_t mode /* PLAN_TICKET, PLAN_CLUSTER or PLAN_LOCAL, see plan_scan_kernel */, int32_t first_rank,
                 unsigned char* const* __restrict__ box_of_rank /* PLAN_LOCAL: the ranks' count mailboxes, or nullptr */,
                 uint32_t epoch) {
  extern __shared__ int32_t sm[];
  __shared__ int is_last;
  const bool as_cluster = mode == PLAN_CLUSTER;
  // Behind the gate kernel (moe_gate_plan) this kernel may have been scheduled early: the routing indexes
  // are complete once the wait returns (at once under a plain launch).
  dependency_wait();
  // A dispatch launched behind this kernel with programmatic serialization (moe_plan_dispatch) may start
  // now and move its first payload loads while the plan is computed; it waits for this kernel's
  // completion before it reads anything written here.  Without such a dependent this does nothing.
  release_dependents();
  constexpr int P = WARPS + 1;
  int32_t* counts = sm;             // [E][P]
  int32_t* rank_base = sm + P * E;  // [E]
  const int r = blockIdx.x + first_rank, R = map.R;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int32_t b_begin = map.tok_start[r] * K, b_end = map.tok_start[r + 1] * K;
  const unsigned lt = lanemask_lt();

  for (int e = threadIdx.x; e < E; e += WARPS * 32) rank_base[e] = 0;
  bool arrived = false;   // as_cluster: at the barrier that says "my row of M is complete"
  for (int32_t pass = b_begin; pass < b_end; pass += WARPS * 32) {
    const int32_t b = pass + warp * 32 + lane;
    int32_t e = -1;
    if (b < b_end) e = __ldg(topk_idx + b);   // on its way while the counters are cleared
    for (int i = threadIdx.x; i < P * E; i += WARPS * 32) counts[i] = 0;
    if (b < b_end && (e < 0 || e >= E)) {
      raise_status(&ctl->status, MOE_ERR_BAD_INDEX);
      e = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int ahead = __popc(peers & lt);           // equal keys in lower lanes = earlier branches
    __syncthreads();
    if (e >= 0 && ahead == 0) counts[e * P + warp] = __popc(peers);   // one round per pass: no carry inside a warp
    __syncthreads();
    // Exclusive scan across the warps of every expert's counts: one thread per expert walks its WARPS counters
    // (loads first, then the running sums from registers, then the stores).  The row stride WARPS + 1 makes the
    // threads of a warp hit different banks at every step.  (As 32-lane shuffle scans, one per expert, this step
    // took 1.5 us of the planner's 6.7: 32 warps, eight scans each.)
    for (int x = threadIdx.x; x < E; x += WARPS * 32) {
      int32_t c[WARPS];
#pragma unroll
      for (int w = 0; w < WARPS; ++w) c[w] = counts[x * P + w];
      int32_t run = rank_base[x];
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        counts[x * P + w] = run;
        run += c[w];
      }
      rank_base[x] = run;
    }
    __syncthreads();
    const bool last_pass = pass + WARPS * 32 >= b_end;
    if (as_cluster && last_pass) {   // rank_base is final: the other CTAs may read it while s and M go out
      cluster_arrive();
      arrived = true;
    }
    if (b < b_end) s[b] = e >= 0 ? counts[e * P + warp] + ahead : 0;
    if (!last_pass) __syncthreads();   // the next pass clears the counters
  }
  if (as_cluster && !arrived) {   // a rank without tokens
    __syncthreads();
    cluster_arrive();
  }
  for (int e = threadIdx.x; e < E; e += WARPS * 32) M[(size_t)r * E + e] = rank_base[e];
  if (as_cluster) {
    cluster_notify(rank_base, sm + (P + 1) * E, E, R, r, full_table, align, c_rank, o, n_exp, n_recv);
    return;
  }
  if (mode == PLAN_LOCAL) {   // s and this rank's row of M: the offsets come from moe_notify / moe_notify_peers
    if (box_of_rank != nullptr) {
      // moe_layout_push: the row goes straight from shared memory into every rank's mailbox (see push_counts_kernel)
      for (int q = threadIdx.x; q < R * E; q += WARPS * 32) {
        const int d = q / E, e = q - d * E;
        box_counts(box_of_rank[d], E, R, epoch)[(size_t)r * E + e] = rank_base[e];
      }
      __syncthreads();
      for (int d = threadIdx.x; d < R; d += WARPS * 32) {
        uint32_t* word = reinterpret_cast<uint32_t*>(box_counts(box_of_rank[d], E, R, epoch) + (size_t)R * E) + r;
        asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(word), "r"(epoch) : "memory");
      }
    }
    return;
  }

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(&ctl->scan_ticket, 1) == R - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  build_large_offsets(M, E, R, full_table, align, c_rank, o, n_exp, n_recv, sm);
  if (threadIdx.x == 0) ctl->scan_ticket = 0;
}

// Notify from a count matrix gathered elsewhere (multi-rank use: every rank contributed its row): installs it as M
// and rebuilds the large offsets and receive counts.  R CTAs, one per window: the gathered matrix is complete in
// global memory before the launch, so CTA d takes its E/R columns of every row straight from there (and copies
// row d into M) -- no CTA waits for another and the time does not grow with R (a single CTA building every window
// took 4.2 us at R = 8 and 16.5 us at R = 64).
// Dynamic shared memory: cluster_notify_smem_ints(E, R) ints.
__global__ void __launch_bounds__(256)
notify_rank_kernel(const int32_t* counts_all, int32_t E, int32_t R, int32_t full_table, int32_t align,
                   int32_t* M, int32_t* __restrict__ c_rank, int32_t* __restrict__ o,
                   int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv) {
  extern __shared__ int32_t sm[];
  const int d = blockIdx.x, E_r = E / R, P = R + 1;
  for (int q = threadIdx.x; q < E_r * R; q += (int)blockDim.x) {   // consecutive threads: consecutive experts of one row
    const int el = q % E_r, rr = q / E_r;
    sm[el * P + rr] = counts_all[(size_t)rr * E + d * E_r + el];
  }
  if (counts_all != M)   // (the planners of one GPU call this on M itself when R is too large for a cluster)
    for (int e = threadIdx.x; e < E; e += (int)blockDim.x) M[(size_t)d * E + e] = counts_all[(size_t)d * E + e];
  __syncthreads();
  window_offsets(sm, E, R, d, full_table, align, c_rank, o, n_exp, n_recv);
}

// push: a CTA stores this rank's row of counts into entry [my_rank] of the mailboxes of 16 ranks (plain peer stores),
// then thread d publishes the row in rank d's mailbox with the epoch word (a release store at system scope behind
// the CTA barrier, so the row is visible to whoever acquires the word).  Nothing waits here.  (One CTA per
// destination, each with its own release, took 5 us from R = 16 on; one CTA for all of 64 destinations 6 us.)
constexpr int PUSH_RANKS_PER_CTA = 16;
__global__ void __launch_bounds__(1024)
push_counts_kernel(unsigned char* const* __restrict__ box_of_rank, const int32_t* __restrict__ my_row, int32_t E,
                   int32_t R, int32_t my_rank, uint32_t epoch) {
  const int d0 = blockIdx.x * PUSH_RANKS_PER_CTA, d1 = min(R, d0 + PUSH_RANKS_PER_CTA);
  for (int q = threadIdx.x; q < (d1 - d0) * E; q += (int)blockDim.x) {
    const int d = d0 + q / E, e = q % E;
    box_counts(box_of_rank[d], E, R, epoch)[(size_t)my_rank * E + e] = my_row[e];
  }
  __syncthreads();
  for (int d = d0 + threadIdx.x; d < d1; d += (int)blockDim.x) {
    uint32_t* word = reinterpret_cast<uint32_t*>(box_counts(box_of_rank[d], E, R, epoch) + (size_t)R * E) + my_rank;
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(word), "r"(epoch) : "memory");
  }
}

// notify from the mailbox: CTA d waits until every rank's epoch word in THIS rank's mailbox has reached `epoch`
// (acquire, system scope; at most limit_ms milliseconds, then MOE_ERR_TIMEOUT and a normal end with nothing
// written), then builds window d's offsets from the gathered rows like notify_rank_kernel.
// Dynamic shared memory: cluster_notify_smem_ints(E, R) ints.
__global__ void __launch_bounds__(256)
notify_box_kernel(unsigned char* my_box, int32_t E, int32_t R, uint32_t epoch, int32_t limit_ms, int32_t full_table,
                  int32_t align, int32_t* M, int32_t* __restrict__ c_rank, int32_t* __restrict__ o,
                  int32_t* __restrict__ n_exp, int32_t* __restrict__ n_recv, int32_t* status) {
  extern __shared__ int32_t sm[];
  __shared__ int gave_up;
  if (threadIdx.x == 0) gave_up = 0;
  __syncthreads();
  const int32_t* buf = box_counts(my_box, E, R, epoch);
  const uint32_t* words = reinterpret_cast<const uint32_t*>(buf + (size_t)R * E);
  for (int r = threadIdx.x; r < R; r += (int)blockDim.x) {
    uint64_t t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const uint64_t limit = (uint64_t)limit_ms * 1000000ull;
    for (;;) {
      uint32_t seen;
      asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(seen) : "l"(words + r) : "memory");
      if ((int32_t)(seen - epoch) >= 0) break;
      uint64_t now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (now - t0 > limit) {
        raise_status(status, MOE_ERR_TIMEOUT);
        gave_up = 1;
        break;
      }
      __nanosleep(200);
    }
  }
  __syncthreads();   // every row this CTA reads was acquired by one of its threads in front of this barrier
  if (gave_up) return;
  const int d = blockIdx.x, E_r = E / R, P = R + 1;
  const volatile int32_t* rows = buf;   // written by other GPUs during this kernel's lifetime: no cached copies
  for (int q = threadIdx.x; q < E_r * R; q += (int)blockDim.x) {
    const int el = q % E_r, rr = q / E_r;
    sm[el * P + rr] = rows[(size_t)rr * E + d * E_r + el];
  }
  for (int e = threadIdx.x; e < E; e += (int)blockDim.x) M[(size_t)d * E + e] = rows[(size_t)d * E + e];
  __syncthreads();
  window_offsets(sm, E, R, d, full_table, align, c_rank, o, n_exp, n_recv);
}

template <int ROUNDS>
__global__ void __launch_bounds__(PLAN_THREADS)
plan_finalize_kernel(const int32_t* __restrict__ topk_idx, const __grid_constant__ RankMap map, int32_t K, int32_t E,
                     const int32_t* __restrict__ tile_rank, const int32_t* __restrict__ tile_base,
                     int32_t* __restrict__ s) {
  release_dependents();   // a dispatch launched behind the plan may be scheduled; it waits for this kernel
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
  // The routing indexes do not depend on the kernels in front: they travel while the scan kernel runs.
  int32_t e_of[ROUNDS];
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = b_begin + i * PLAN_THREADS + threadIdx.x;
    e_of[i] = b < b_end ? __ldg(topk_idx + b) : -1;
  }
  dependency_wait();   // tile ranks and tile bases are complete (returns at once under a plain launch)
#pragma unroll
  for (int i = 0; i < ROUNDS; ++i) {
    const int32_t b = b_begin + i * PLAN_THREADS + threadIdx.x;
    if (b < b_end) {
      const int32_t e = e_of[i];
      s[b] = (e >= 0 && e < E) ? tile_rank[b] + tile_base[(size_t)tile * E + e] : 0;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Synchronisation metadata across ranks (Section 5.4): epochs in the state region behind every rank's window.
// signal: thread d stores `epoch` into entry [slot][my_rank] of rank d's region with release semantics at system
// scope, so that everything this stream completed before the launch (rows stored into rank d's window, expert
// outputs) is visible to whoever acquires the entry.  Plain peer stores; nothing waits here.
__global__ void signal_peers_kernel(unsigned char* const* __restrict__ state_of_rank, int32_t R, int32_t my_rank,
                                    int32_t slot, uint32_t epoch) {
  for (int d = threadIdx.x; d < R; d += blockDim.x) {
    uint32_t* entry = reinterpret_cast<uint32_t*>(state_of_rank[d]) + (size_t)slot * R + my_rank;
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(entry), "r"(epoch) : "memory");
  }
}

// wait: thread r polls entry [slot][r] of THIS rank's region (acquire, system scope) until it has reached `epoch`,
// sleeping between polls, for at most limit_ms milliseconds; a wait that runs out raises MOE_ERR_TIMEOUT and the
// kernel ends normally.
__global__ void wait_peers_kernel(const unsigned char* __restrict__ my_state, int32_t R, int32_t slot, uint32_t epoch,
                                  int32_t limit_ms, int32_t* status) {
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const uint32_t* entry = reinterpret_cast<const uint32_t*>(my_state) + (size_t)slot * R + r;
    uint64_t t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const uint64_t limit = (uint64_t)limit_ms * 1000000ull;
    for (;;) {
      uint32_t seen;
      asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(seen) : "l"(entry) : "memory");
      if ((int32_t)(seen - epoch) >= 0) break;
      uint64_t now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (now - t0 > limit) {
        raise_status(status, MOE_ERR_TIMEOUT);
        break;
      }
      __nanosleep(200);
    }
  }
}

// Tile list over the experts' runs (work list of a grouped GEMM that reads the windows in place): tile k is
// (expert, first window row, valid rows <= tile_rows), in window order.  ONE CTA; shared memory: tiles
// per expert [E], their exclusive prefix [E + 1], warp sums [33].
__global__ void __launch_bounds__(1024)
expert_tiles_kernel(const int32_t* __restrict__ large_off, const int32_t* __restrict__ n_exp, int32_t E, int32_t R,
                    int64_t C, int32_t tile_rows, int64_t max_tiles, int32_t* __restrict__ tile_expert,
                    int64_t* __restrict__ tile_row, int32_t* __restrict__ tile_valid, int32_t* __restrict__ n_tiles) {
  extern __shared__ int32_t tile_sm[];
  int32_t* nt = tile_sm;
  int32_t* pre = tile_sm + E;
  int32_t* warp_sums = pre + E + 1;
  const int E_r = E / R;
  for (int e = threadIdx.x; e < E; e += blockDim.x) nt[e] = (n_exp[e] + tile_rows - 1) / tile_rows;
  __syncthreads();
  block_exclusive_scan(nt, pre, E, warp_sums);   // window order is expert order
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const int64_t start = (int64_t)(e / E_r) * C + large_off[(size_t)e * R];   // the block of source rank 0 starts the run
    const int32_t count = n_exp[e];
    for (int32_t i = 0; i < nt[e]; ++i) {
      const int64_t k = (int64_t)pre[e] + i;
      if (k < max_tiles) {
        tile_expert[k] = e;
        tile_row[k] = start + (int64_t)i * tile_rows;
        tile_valid[k] = min(tile_rows, count - i * tile_rows);
      }
    }
  }
  if (threadIdx.x == 0) *n_tiles = pre[E];
}

}  // namespace moe
