// Dispatch through the bulk-copy engine (TMA, 1-D cp.async.bulk, no tensor map,
// no multicast).
//
// Same work items and same result as dispatch_rows_kernel, but the bytes never
// pass through registers: every warp drives a small ring of shared-memory
// stages.  Lane 0 asks the copy engine to load one work item (up to a whole
// 14 KB row) into a stage, and when the stage's mbarrier completes, to store it
// to the K destination rows.  One request covers the whole contiguous span, so
// HBM sees long sequential bursts per row, and the number of bytes in flight is
// set by shared memory (up to about 170 KB per SM), not by registers.  How many
// warps a CTA gets is the launcher's choice: as many rings as fit for small jobs,
// for large ones only as many as keep about 2400 destination rows being written
// at once across the device, which is what HBM serves best.
//
// Every wait is bounded in time: an mbarrier that does not complete within the
// limit (2 s by default) raises MOE_ERR_TIMEOUT and the warp stops taking work;
// the kernel still ends normally and the context stays usable.
#pragma once

#include "row_kernels.cuh"

namespace moe {

constexpr int BULK_MAX_WARPS = 8;      // warps per CTA: as many 3-stage rings as fit in BULK_SMEM_BUDGET
constexpr int BULK_SMEM_BUDGET = 200 * 1024;
constexpr int BULK_STAGES = 3;
constexpr int BULK_MAX_GRANULE = 32;   // a stage holds at most 16 KB of one row
constexpr int32_t WAIT_LIMIT_MS_DEFAULT = 2000;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait; false if the barrier did not complete within limit_ms milliseconds.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t limit_ms) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns(), limit = (uint64_t)limit_ms * 1000000ull;
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > limit) return false;
  }
}

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Window rows are written once and not read again by this kernel: an evict-first L2 policy on the
// stores measured 1-8 % faster (653 vs 661 us at prefill size, 47 vs 51 us at decode size).  The same
// policy on the row loads measured slower (664 vs 662 us, and the combine behind it 51 vs 49 us at
// decode size), so they keep the default.
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes, uint64_t policy) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
               ::"l"(dst), "r"(src_smem), "r"(bytes), "l"(policy) : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Dynamic shared memory: [warps][BULK_STAGES][stage_bytes] payload, then
// [warps][BULK_STAGES] mbarriers.  stage_bytes = granule * 512; warps = blockDim.x / 32.
__global__ void __launch_bounds__(BULK_MAX_WARPS * 32, 1)
dispatch_bulk_kernel(const unsigned char* __restrict__ X, unsigned char* __restrict__ windows, const RowArgs a,
                     const __grid_constant__ RankMap map) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const uint32_t stage_bytes = (uint32_t)a.granule * 512u;
  const uint32_t row_bytes = (uint32_t)a.H16 * 16u;
  const uint32_t buf0 = smem_addr(smem) + warp * BULK_STAGES * stage_bytes;
  const uint32_t bar0 = smem_addr(smem) + n_warps * BULK_STAGES * stage_bytes + warp * BULK_STAGES * 8;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < BULK_STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // Asks the copy engine for work item `item` into stage `s` (lane 0 only).
  auto issue_load = [&](int32_t item, int s) {
    const WorkItem w = decode_item(a, item);
    const uint32_t off = (uint32_t)w.i0 * 512u;
    const uint32_t bytes = min((uint32_t)w.i1 * 512u, row_bytes) - off;
    // Test hook: one warp expects 16 bytes that never come, so its wait runs out (see MOE_OPT_TEST_STARVE_WAIT_MS).
    const uint32_t starve = (a.test_starve && blockIdx.x == 0 && warp == 0 && item == 0) ? 16u : 0u;
    mbar_expect_tx(bar0 + 8 * s, bytes + starve);
    bulk_load(buf0 + s * stage_bytes, X + (size_t)w.t * row_bytes + off, bytes, bar0 + 8 * s);
  };

  // Items in flight: q0 is consumed this iteration, q1 is loading, q2 is fetched now.
  ItemFeed feed = begin_feed();
  int32_t q0 = a.n_items, q1 = a.n_items;
  // The first two items of a small job are fixed and their payload depends on nothing a planner writes, so
  // their loads are issued before anything else: before the wait for a planner this launch was chained behind
  // (moe_plan_dispatch: they travel while it runs), and before the status and capacity checks, whose loads
  // otherwise stand in front of the first payload byte (1 us of a flushed call).  Nothing is taken from the
  // work counter and no planner output is read before the wait; a call that must abort lets them land first.
  const bool early = a.static_first >= 2;
  if (early) {
    q0 = fetch_item(a, feed);
    q1 = fetch_item(a, feed);
    if (lane == 0) {
      if (q0 < a.n_items) issue_load(q0, 0);
      if (q1 < a.n_items) issue_load(q1, 1);
    }
    if (q0 < a.n_items && lane < a.K) warm(a.topk_idx + (size_t)decode_item(a, q0).t * a.K + lane);
  }
  dependency_wait();      // returns at once unless this launch was allowed to start early
  release_dependents();   // after the wait: whatever follows starts no earlier than the previous kernel's end
  if (must_abort(a)) {
    // loads already in flight must land before this CTA's shared memory is handed back
    if (early && lane == 0) {
      if (q0 < a.n_items) mbar_wait(bar0, 0, a.wait_limit_ms);
      if (q1 < a.n_items) mbar_wait(bar0 + 8, 0, a.wait_limit_ms);
    }
    end_work(a);
    return;
  }
  if (!early) {
    q0 = fetch_item(a, feed);
    q1 = fetch_item(a, feed);
    if (lane == 0) {
      if (q0 < a.n_items) issue_load(q0, 0);
      if (q1 < a.n_items) issue_load(q1, 1);
    }
  }
  uint64_t evict_first;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));
  uint32_t it = 0;
  bool alive = true;
  while (q0 < a.n_items && alive) {
    const int32_t q2 = fetch_item(a, feed);
    const int s = it % BULK_STAGES;
    const uint32_t parity = (it / BULK_STAGES) & 1u;
    const WorkItem w = decode_item(a, q0);
    const int64_t slot = resolve_slot(a, map, w.t, lane, w.i0 == 0);   // overlaps the load in flight
    const uint32_t off = (uint32_t)w.i0 * 512u;
    const uint32_t bytes = min((uint32_t)w.i1 * 512u, row_bytes) - off;

    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar0 + 8 * s, parity, a.wait_limit_ms) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) {
      if (lane == 0) {
        raise_status(a.status, MOE_ERR_TIMEOUT);
        // the load of the next item is in flight: let it land (bounded) before the CTA's shared memory is handed back
        if (q1 < a.n_items) mbar_wait(bar0 + 8 * ((it + 1) % BULK_STAGES), ((it + 1) / BULK_STAGES) & 1u, a.wait_limit_ms);
      }
      alive = false;
      break;
    }
    for (int j = 0; j < a.K; ++j) {
      const int64_t row = __shfl_sync(0xffffffffu, slot, j);
      if (lane == 0 && row >= 0) bulk_store(window_row(a, windows, row, row_bytes) + off, buf0 + s * stage_bytes, bytes, evict_first);
    }
    if (lane == 0) {
      bulk_commit();
      // The stage that held the previous item is refilled next: its stores must have read it.
      bulk_wait_read<1>();
      if (q2 < a.n_items) issue_load(q2, (it + 2) % BULK_STAGES);
    }
    q0 = q1;
    q1 = q2;
    ++it;
  }
  if (lane == 0) bulk_wait_all();
  end_work(a);
}

}  // namespace moe
