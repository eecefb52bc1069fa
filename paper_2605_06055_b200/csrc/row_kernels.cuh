// Payload kernels: dispatch (scatter rows into expert windows) and combine
// (gather rows from expert windows + fp32 weighted sum), both token-major.
//
// Algorithm 1 / Algorithm 2 of the paper.  A warp works on (part of) one token
// row at a time: lane j < K resolves branch (t, j) to its window row with the
// two-level offset rule slot = dst(e)*C + o[e, src(t)] + s[t,j]; then the whole
// warp moves its share of the row in 16-byte chunks.  Dispatch reads X[t,:] from
// HBM exactly once and stores it K times; combine issues the K loads of a chunk
// before its j-ordered fma chain.  There is no relay, permute or unpermute
// buffer.  (The default dispatch is the bulk-copy kernel in bulk_kernels.cuh;
// dispatch_rows_kernel here is the register path.)
#pragma once

#include "common.cuh"

namespace moe {

struct RowArgs {
  const int32_t* topk_idx;   // [T,K]
  const int32_t* small_off;  // final small offsets s [T,K]; tile-planned DECODE: in-tile rank [T,K]
  int32_t* small_out;        // tile-planned DECODE dispatch: where delta is recorded; else nullptr
  // Finished window rows (dst*C + row in window) of every branch: a dispatch over the whole batch records them
  // (slot_out), and a combine with the same plan and capacity reads them back (slot_in) instead of walking
  // routing index -> large offset: one dependent load less in front of its first payload loads.  Else nullptr.
  int32_t* slot_out;
  const int32_t* slot_in;
  const int32_t* tile_base;  // tile-planned DECODE: [tiles,E] exclusive tile bases; else nullptr
  const int32_t* large_off;  // o [E,R]
  const int32_t* n_recv;     // [R]
  int32_t* status;
  int64_t C;                 // rows per window segment
  int32_t T, K, E, R, E_r;
  int32_t H16;               // 16-byte chunks per row
  int32_t* work;             // work-item counter (zero on entry, zeroed again by the last warp to finish)
  int32_t* work_done;        // finished-warp counter (same)
  int32_t granule;           // units (512-byte slabs) per work item
  int32_t items_per_row;     // ceil(units per row / granule)
  int32_t n_items;           // head items + tail items
  // The rows left over after the last full round of whole-row items (fewer rows than warps) are cut
  // finer, tail_granule units per item, so that the launch does not end with a few warps each moving a
  // whole row while the others idle.  Items [0, n_head) cover the first head_rows rows; without a tail
  // n_head == n_items and head_rows == t_count.
  int32_t n_head, head_rows, tail_granule, tail_items_per_row;
  int32_t t_begin, t_count;  // token range this launch covers (the whole batch unless a *_range call)
  // Multi-rank use: window segment d starts at win_base[d] (device array of R device pointers, e.g. peer
  // mappings of every rank's window); nullptr = one allocation of R consecutive segments of C rows.
  const unsigned char* const* win_base;
  float* const* scale_base;  // quantised dispatch, multi-rank use: scales of segment d start at scale_base[d]; else nullptr
  int32_t static_first;      // work items per warp that are fixed (warp id + k * warps) before the counter is used
  int32_t prefetch_meta;     // combine: fetch the next item's branch metadata while reducing the current one
  int32_t pdl;               // dispatch launched behind the planner with programmatic stream serialization
  int32_t wait_limit_ms;     // bound of every device-side wait
  int32_t test_starve;       // test hook of the bulk-copy dispatch: make one wait run out
};

// Load of a word the planner wrote (small offsets, tile bases, large offsets).  A kernel chained behind the
// planner by programmatic stream serialization is already running while the planner writes these arrays, so
// they are not read-only for its lifetime and must not take the non-coherent path (ld.global.nc / __ldg);
// a plain load issued after dependency_wait() sees the planner's writes.  Routing indexes, weights and payload
// rows are inputs of the whole call and keep the non-coherent loads.
__device__ __forceinline__ int32_t ld_plan(const int32_t* p) {
  int32_t v;
  asm volatile("ld.global.b32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

// Window row of branch (t, lane) for lane < K, -1 otherwise.  Small offsets of
// the DECODE schedule are finished here (in-tile rank + tile base).
__device__ __forceinline__ int64_t resolve_slot(const RowArgs& a, const RankMap& map, int32_t t, int lane,
                                                bool record) {
  if (lane >= a.K) return -1;
  const int32_t b = t * a.K + lane;
  const int32_t e = __ldg(a.topk_idx + b);
  if (e < 0 || e >= a.E) return -1;  // flagged by the plan; never dereferenced
  const int32_t r = src_rank(map, t);
  int32_t so = ld_plan(a.small_off + b);
  if (a.tile_base != nullptr) {
    so += ld_plan(a.tile_base + (size_t)tile_of_branch(map, r, b, a.K) * a.E + e);
    if (record) a.small_out[b] = so;
  }
  const int64_t slot = (int64_t)(e / a.E_r) * a.C + ld_plan(a.large_off + (size_t)e * a.R + r) + so;
  if (record && a.slot_out != nullptr) a.slot_out[b] = (int32_t)slot;
  return slot;
}

// The same resolution in two phases, so that its memory latency can hide behind payload traffic:
// load_meta issues the loads that depend only on the branch index (routing index, small offset,
// weight) and finish_slot adds the large offset.  When a work item is a single batch of loads
// (short rows, small K) combine calls load_meta for the NEXT item before it reduces the current
// one; measured 274 -> 256 us at H=4096, K=2, and 618 -> 629 us at H=7168, K=8, where a row is seven
// batches and the launcher therefore leaves the prefetch off.
struct BranchMeta {
  int32_t e, so;
  float w;
};

__device__ __forceinline__ BranchMeta load_meta(const RowArgs& a, const float* __restrict__ topk_w, int32_t t,
                                                int lane) {
  BranchMeta m;
  m.e = -1;
  m.so = 0;
  m.w = 0.0f;
  if (lane < a.K) {
    const int32_t b = t * a.K + lane;
    if (a.slot_in != nullptr) {
      m.so = ld_plan(a.slot_in + b);   // the finished row; the routing index is not needed
    } else {
      m.e = __ldg(a.topk_idx + b);
      m.so = ld_plan(a.small_off + b);
    }
    if (topk_w != nullptr) m.w = __ldg(topk_w + b);
  }
  return m;
}

__device__ __forceinline__ int64_t finish_slot(const RowArgs& a, const RankMap& map, const BranchMeta& m, int32_t t,
                                               int lane, bool record) {
  if (a.slot_in != nullptr) {
    // A recorded row is trusted only inside the windows: a table that no dispatch has filled (calls recorded into a
    // graph that never ran) must not become an address.
    if (lane >= a.K) return -1;
    if ((uint32_t)m.so >= (uint32_t)(a.R * a.C)) {
      raise_status(a.status, MOE_ERR_NOT_PLANNED);
      return -1;
    }
    return (int64_t)m.so;
  }
  if (lane >= a.K || m.e < 0 || m.e >= a.E) return -1;   // bad indexes were flagged by the plan; never dereferenced
  const int32_t r = src_rank(map, t);
  int32_t so = m.so;
  if (a.tile_base != nullptr) {
    const int32_t b = t * a.K + lane;
    so += ld_plan(a.tile_base + (size_t)tile_of_branch(map, r, b, a.K) * a.E + m.e);
    if (record) a.small_out[b] = so;
  }
  return (int64_t)(m.e / a.E_r) * a.C + ld_plan(a.large_off + (size_t)m.e * a.R + r) + so;
}

// Pulls a word into the cache hierarchy ahead of its use; the value is discarded.
__device__ __forceinline__ void warm(const int32_t* p) {
  const int32_t v = __ldg(p);
  asm volatile("" ::"r"(v));
}

// Address of window row `row` (global numbering d*C + local row).
__device__ __forceinline__ unsigned char* window_row(const RowArgs& a, const void* windows, int64_t row,
                                                     size_t row_bytes) {
  if (a.win_base == nullptr) return (unsigned char*)windows + (size_t)row * row_bytes;
  // (rows below 2^32 -- every realistic window -- take the 32-bit division: the 64-bit one is a long subroutine)
  const int64_t d = (uint64_t)(row | a.C) >> 32 ? row / a.C : (int64_t)((uint32_t)row / (uint32_t)a.C);
  return (unsigned char*)a.win_base[d] + (size_t)(row - d * a.C) * row_bytes;
}

// True when the call must not touch payload memory: an earlier error is pending
// or a window is too small.  Evaluated identically by every CTA.
__device__ __forceinline__ bool must_abort(const RowArgs& a) {
  int bad = load_status(a.status) != 0;
  int over = 0;
  for (int d = threadIdx.x; d < a.R; d += blockDim.x) over |= (a.n_recv[d] > a.C);
  over = __syncthreads_or(over);
  if (over && blockIdx.x == 0 && threadIdx.x == 0) raise_status(a.status, MOE_ERR_CAPACITY);
  return bad || over;
}

// 16-byte load of window / input rows, in three forms.
// LD_STREAM, LD_L1: read-only (non-coherent) loads for rows of THIS GPU's memory, which nothing writes while the
// kernel runs.  LD_STREAM marks the line "no allocate" in L1, LD_L1 lets it allocate.  Neither data is ever
// re-read, but measured on B200 the allocating form is 3 % faster for combine at prefill sizes (617 vs 637 us)
// and 10 % slower at decode sizes (55 vs 49 us), so the launcher picks by job size.
// LD_PEER, LD_PEER_L1: ordinary (coherent) loads, for windows addressed through a table of bases -- other GPUs'
// memory that other GPUs' kernels write.  They are valid whenever the reading kernel is ordered after the writers'
// completion (a host barrier, or a preceding wait on arrival flags, followed by this launch), which the
// non-coherent path does not promise once such ordering is established on the device.  The same choice by job
// size: LD_PEER does not allocate in L1, LD_PEER_L1 does (one GPU, every window behind the table: 51.3 against
// 55.1 us at the decode shape, 637 against 613 us at 32768 tokens).
enum { LD_STREAM = 0, LD_L1 = 1, LD_PEER = 2, LD_PEER_L1 = 3 };
template <int MODE>
__device__ __forceinline__ uint4 ld_row(const uint4* p) {
  uint4 v;
  if constexpr (MODE == LD_L1)
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  else if constexpr (MODE == LD_PEER)
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  else if constexpr (MODE == LD_PEER_L1)
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  else
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return ld_row<LD_STREAM>(p); }

__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

// Work partition shared by dispatch and combine.  A "unit" is one 512-byte
// column slab of one token row (32 lanes x 16 bytes).  A row is cut into
// items_per_row work items of `granule` units (the last may be shorter); the job
// is T * items_per_row items.  Warps take items from an atomic counter (after two
// fixed first items), fetching the next one while the current one is processed, so a warp that the memory
// system serves slowly simply takes fewer items: no wave quantisation at prefill
// sizes, full-GPU parallelism at decode sizes, no static tail.  Which warp moves
// which bytes does not affect the result.  The last warp of a launch to finish
// puts the counters back to zero, so every launch (eager, or replayed from a
// CUDA graph any number of times) starts from a clean state with no memset.
struct WorkItem {
  int32_t t;       // token
  int32_t i0, i1;  // unit range inside the row
};

// Called by every warp on every exit path of a row kernel.
__device__ __forceinline__ void end_work(const RowArgs& a) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) {
    const int32_t nwarps = (int32_t)(gridDim.x * (blockDim.x >> 5));
    __threadfence();                                   // this warp's item fetches come before its sign-off
    if (atomicAdd(a.work_done, 1) == nwarps - 1) {     // everyone else has signed off: nobody fetches any more
      *a.work = 0;
      *a.work_done = 0;
    }
  }
}

// Hands a warp its work items.  In small jobs (a few items per warp: decode) the first two are fixed
// (warp id, warp id + number of warps), so no warp waits on an atomic before its first bytes move
// (2 us of a 48 us call); every later one comes from the counter.  Large jobs take every item from
// the counter: fixed first items measured up to 6 % slower there.
struct ItemFeed {
  int64_t gid, nwarps;
  int32_t taken;
};

__device__ __forceinline__ ItemFeed begin_feed() {
  ItemFeed f;
  f.nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  f.gid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  f.taken = 0;
  return f;
}

__device__ __forceinline__ int32_t fetch_item(const RowArgs& a, ItemFeed& f) {
  int64_t item;
  if (f.taken < a.static_first) {
    item = f.gid + f.taken * f.nwarps;
  } else {
    int32_t v = 0;
    if ((threadIdx.x & 31) == 0) v = atomicAdd(a.work, 1);
    item = a.static_first * f.nwarps + __shfl_sync(0xffffffffu, v, 0);
  }
  ++f.taken;
  return (int32_t)min(item, (int64_t)a.n_items);
}

// TAIL = false: the launch has no finer-cut tail (n_head == n_items); saves the selects in kernels whose
// registers are all spoken for (the large-job combine).
template <bool TAIL = true>
__device__ __forceinline__ WorkItem decode_item(const RowArgs& a, int32_t item) {
  WorkItem w;
  if constexpr (TAIL) {
    // head and tail items differ only in four launch constants: selects, then one division
    const bool tail = item >= a.n_head;
    const int32_t ipr = tail ? a.tail_items_per_row : a.items_per_row;
    const int32_t g = tail ? a.tail_granule : a.granule;
    const int32_t rem = tail ? item - a.n_head : item;
    const int32_t q = rem / ipr;
    w.t = a.t_begin + (tail ? a.head_rows : 0) + q;
    w.i0 = (rem - q * ipr) * g;
    w.i1 = min(w.i0 + g, (a.H16 + 31) >> 5);
  } else {
    const int32_t q = item / a.items_per_row;
    w.t = a.t_begin + q;
    w.i0 = (item - q * a.items_per_row) * a.granule;
    w.i1 = min(w.i0 + a.granule, (a.H16 + 31) >> 5);
  }
  return w;
}

// ---------------------------------------------------------------- dispatch
// KT > 0: K known at compile time (row pointers live in registers).
// KT == 0: any K <= 32 (row index fetched by shuffle per store).
// UNROLL 16-byte loads are in flight per lane before the K x UNROLL stores; few
// warps with deep unrolling beat many thin warps here, because each warp then
// writes long contiguous runs of every destination row.
template <int KT, int UNROLL>
__global__ void __launch_bounds__(256, 1)
dispatch_rows_kernel(const uint4* __restrict__ X, uint4* __restrict__ windows, const RowArgs a,
                     const __grid_constant__ RankMap map) {
  if (must_abort(a)) {
    end_work(a);
    return;
  }
  const int lane = threadIdx.x & 31;
  const int K = KT > 0 ? KT : a.K;
  const int H16 = a.H16;

  ItemFeed feed = begin_feed();
  int32_t item = fetch_item(a, feed);
  while (item < a.n_items) {
    const int32_t next_item = fetch_item(a, feed);   // in flight while this item is processed
    const WorkItem w = decode_item(a, item);
    item = next_item;
    const int64_t slot = resolve_slot(a, map, w.t, lane, w.i0 == 0);   // the owner of the row start records delta
    const uint4* src = X + (size_t)w.t * H16;
    if constexpr (KT > 0) {
      uint4* dst[KT];
#pragma unroll
      for (int j = 0; j < KT; ++j) {
        const int64_t row = __shfl_sync(0xffffffffu, slot, j);
        dst[j] = row >= 0 ? reinterpret_cast<uint4*>(window_row(a, windows, row, (size_t)H16 * 16)) : nullptr;
      }
      for (int i = w.i0; i < w.i1; i += UNROLL) {
        uint4 v[UNROLL];
        bool ok[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          const int c = (i + u) * 32 + lane;
          ok[u] = (i + u < w.i1) && (c < H16);
          if (ok[u]) v[u] = ld_stream(src + c);
        }
#pragma unroll
        for (int j = 0; j < KT; ++j)
          if (dst[j] != nullptr) {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u)
              if (ok[u]) st_stream(dst[j] + (i + u) * 32 + lane, v[u]);
          }
      }
    } else {
      for (int i = w.i0; i < w.i1; ++i) {   // warp-uniform trip count: shuffles stay convergent
        const int c = i * 32 + lane;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (c < H16) v = ld_stream(src + c);
        for (int j = 0; j < K; ++j) {
          const int64_t row = __shfl_sync(0xffffffffu, slot, j);
          if (row >= 0 && c < H16) st_stream(reinterpret_cast<uint4*>(window_row(a, windows, row, (size_t)H16 * 16)) + c, v);
        }
      }
    }
  }
  end_work(a);
}

// ---------------------------------------------------------------- combine
__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], float w, const uint4& v) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc[2 * i] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i]);
    acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xffff0000u), acc[2 * i + 1]);
  }
}

__device__ __forceinline__ uint4 pack_bf16x8(const float (&acc)[8]) {
  uint32_t u[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);  // round to nearest even
    u[i] = *reinterpret_cast<const uint32_t*>(&p);
  }
  return make_uint4(u[0], u[1], u[2], u[3]);
}

// MODE: how window rows are loaded (see ld_row).  LD_L1 is also the large-job form without finer-cut tail items.
template <int KT, int UNROLL, int MODE>
__global__ void __launch_bounds__(256, 1)
combine_rows_kernel(const uint4* __restrict__ windows, const float* __restrict__ topk_w, uint4* __restrict__ Y,
                    const RowArgs a, const __grid_constant__ RankMap map) {
  const int lane = threadIdx.x & 31;
  constexpr int KMAX = KT > 0 ? KT : -KT;
  const int K = KT > 0 ? KT : a.K;
  const int H16 = a.H16;
  ItemFeed feed = begin_feed();
  int32_t item = a.n_items;
  BranchMeta meta = {-1, 0, 0.0f};
  // Small jobs: the first item is fixed (no counter), and the plan it reads is complete before this launch, so its
  // routing index, small offset and weight are asked for before the status and capacity checks and travel
  // while those are evaluated -- one round trip to memory less in front of the first row.
  bool meta_ready = false;
  if constexpr (MODE != LD_L1) {
    if (a.static_first >= 2) {
      item = fetch_item(a, feed);
      if (item < a.n_items) meta = load_meta(a, topk_w, decode_item<true>(a, item).t, lane);
      meta_ready = true;
    }
  }
  if (must_abort(a)) {
    end_work(a);
    return;
  }
  if (!meta_ready) {
    item = fetch_item(a, feed);
    if (a.prefetch_meta && item < a.n_items) meta = load_meta(a, topk_w, decode_item<MODE != LD_L1>(a, item).t, lane);
    meta_ready = a.prefetch_meta != 0;
  }
  while (item < a.n_items) {
    const int32_t next_item = fetch_item(a, feed);
    const WorkItem wi = decode_item<MODE != LD_L1>(a, item);
    if (!meta_ready) meta = load_meta(a, topk_w, wi.t, lane);
    meta_ready = a.prefetch_meta != 0;   // from the second item on, only the prefetching form has it in hand
    const int64_t slot = finish_slot(a, map, meta, wi.t, lane, false);
    const float w_lane = meta.w;
    // Lane j turns its own branch's row into an address once (with a table of bases: one division and one table
    // entry per lane, side by side, instead of K of each one after the other in every lane); the addresses are
    // what the lanes exchange.
    // (lanes without a branch resolve row 0 and drop the result: no divergent path in front of the loads)
    const unsigned long long any_addr =
        reinterpret_cast<unsigned long long>(window_row(a, windows, slot >= 0 ? slot : 0, (size_t)H16 * 16));
    const unsigned long long row_addr = slot >= 0 ? any_addr : 0ull;
    // short rows: the next item's routing index, small offset and weight travel while this item is reduced
    if (a.prefetch_meta && next_item < a.n_items) meta = load_meta(a, topk_w, decode_item<MODE != LD_L1>(a, next_item).t, lane);
    item = next_item;
    uint4* out = Y + (size_t)wi.t * H16;
    {
      // KT > 0: exactly KT branches.  KT < 0: up to KMAX = -KT branches, K of them live (the degrees without a kernel
      // of their own); the others hold a null address and are skipped, loads and fma alike, so the chain of the
      // live ones is the same.  (A form that fetched addresses and weights by shuffles inside the row loop, eight
      // branches at a time, ran at 1.6-1.75 TB/s whatever K: 417 us against 110 us for K = 9 at 8192 rows of 8 KB.)
      const uint4* src[KMAX];
      float w[KMAX];
#pragma unroll
      for (int j = 0; j < KMAX; ++j) {
        if constexpr (KT > 0 && KT <= 2) {   // one or two rows: every lane resolving them itself measured 1-3 % faster
          const int64_t row = __shfl_sync(0xffffffffu, slot, j);
          src[j] = row >= 0 ? reinterpret_cast<const uint4*>(window_row(a, windows, row, (size_t)H16 * 16)) : nullptr;
        } else {
          src[j] = reinterpret_cast<const uint4*>(__shfl_sync(0xffffffffu, row_addr, j));
        }
        w[j] = __shfl_sync(0xffffffffu, w_lane, j);
        if (KT < 0 && j >= K) src[j] = nullptr;
      }
      for (int i = wi.i0; i < wi.i1; i += UNROLL) {
        uint4 v[UNROLL][KMAX];
        bool ok[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          const int c = (i + u) * 32 + lane;
          ok[u] = (i + u < wi.i1) && (c < H16);
#pragma unroll
          for (int j = 0; j < KMAX; ++j)
            v[u][j] = (ok[u] && src[j] != nullptr) ? ld_row<MODE>(src[j] + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int j = 0; j < KMAX; ++j)
            if (KT > 0 || j < K) fma_bf16x8(acc, w[j], v[u][j]);   // j ascending, one fma per term
          if (ok[u]) out[(i + u) * 32 + lane] = pack_bf16x8(acc);
        }
      }
    }
  }
  end_work(a);
}

// ---------------------------------------------------------------- slots
__global__ void __launch_bounds__(256)
slots_kernel(int32_t* __restrict__ slots, const RowArgs a, const __grid_constant__ RankMap map) {
  if (must_abort(a)) return;
  const int32_t B = a.T * a.K;
  for (int32_t b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
    const int32_t t = b / a.K;
    const int32_t e = __ldg(a.topk_idx + b);
    if (e < 0 || e >= a.E) {
      slots[b] = -1;
      continue;
    }
    const int32_t r = src_rank(map, t);
    int32_t so = ld_plan(a.small_off + b);
    if (a.tile_base != nullptr) so += ld_plan(a.tile_base + (size_t)tile_of_branch(map, r, b, a.K) * a.E + e);
    slots[b] = (int32_t)((int64_t)(e / a.E_r) * a.C + ld_plan(a.large_off + (size_t)e * a.R + r) + so);
  }
}

// ---------------------------------------------------------------- expert ranges
// Grouped-GEMM style descriptors for the expert side: expert e owns window rows
// [row_start[e], row_start[e] + row_count[e]) -- the block of source rank 0 starts the expert's run.
__global__ void __launch_bounds__(256)
expert_ranges_kernel(const int32_t* __restrict__ large_off, const int32_t* __restrict__ n_exp, int32_t E, int32_t R,
                     int64_t C, int64_t* __restrict__ row_start, int32_t* __restrict__ row_count) {
  const int E_r = E / R;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < E; e += gridDim.x * blockDim.x) {
    row_start[e] = (int64_t)(e / E_r) * C + large_off[(size_t)e * R];
    row_count[e] = n_exp[e];
  }
}

}  // namespace moe
