// Quantised dispatch: bf16 rows in, fp8 e4m3 codes + fp32 scales out, written
// straight into the destination expert windows and a parallel scale tensor in
// the same row order (Section 5.2, Prefill Dispatch).
//
// Format (the paper names none; this is the library's definition):
//   amax  = max_h |x[h]|                         (inputs are finite)
//   scale = amax / 448, inv = 448 / amax         (fp32, round to nearest; 1 and 1 when amax == 0)
//   code[h] = e4m3( x[h] * inv )                 (fp32 product, round to nearest even, clamped to +-448)
// Each token is quantised once; its K branches receive the same code row and scale.
// Group-wise form (GROUPED): the same rule applied to every group of 128 consecutive elements of a row on its
// own -- H / 128 scales per row, [rows, H / 128] fp32 in the same row order.  A group is the 16 chunks of 16 bytes
// that one half-warp reads side by side.
//
// Two kernels.  Both load a whole row (needed for amax) into shared memory with one cp.async.bulk, store the code
// row K times with cp.async.bulk, read X from HBM once and write only H + 4 bytes (group-wise: H + H/32) per
// branch; what bounds them below the copy rate is the latency of one warp walking its row, so the number of rows
// in flight per SM -- the number of warps shared memory admits -- is what counts.
//   dispatch_quant_reg_kernel  rows of at most 16 KB, held in registers: a load buffer (2H bytes) and a code
//                              buffer (H bytes) per warp; the next row's load is issued as soon as the current
//                              row is in registers.  3H bytes per warp.
//   dispatch_quant_kernel      a ring of two or three whole-row stages per warp, the codes written IN PLACE over
//                              the first half of the row's stage (they are half as wide, so the code of chunk c
//                              lands on bytes that chunks <= c/2 occupied and have already been read).  4H or 6H
//                              bytes per warp.  Kept for large row-wise jobs of rows beyond 8 KB (two loads in
//                              flight per warp, five warps: the copy rate at 14 KB rows) and, in a two-pass form
//                              that needs no registers for the row, for rows beyond 16 KB.
#pragma once

#include <cuda_fp8.h>

#include "bulk_kernels.cuh"

namespace moe {

// Ring kernel, stages per warp: 3 for large jobs (two loads in flight per warp), 2 otherwise.
constexpr int QUANT_MAX_ROW_BYTES = 32 * 1024;
constexpr int QUANT_MAX_WARPS = 16;
constexpr int QUANT_REG_WARPS_LONG = 10;        // register kernel, rows beyond 8 KB: 204 registers per thread at most
constexpr int QUANT_REG_WARPS_SHORT = 14;       // register kernel, rows up to 8 KB (16 warps measured slower than 14)
constexpr int QUANT_REG_WARPS_SHORT_LARGE_JOB = 9;
constexpr int QUANT_SMEM_BUDGET = 220 * 1024;   // shared memory the warps' rings may fill
constexpr int QUANT_GROUP = 128;                 // elements per scale of the group-wise form
constexpr int QUANT_MAX_GROUPS = QUANT_MAX_ROW_BYTES / 2 / QUANT_GROUP;

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}

__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

__device__ __forceinline__ void sts64(uint32_t addr, uint32_t lo, uint32_t hi) {
  asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(addr), "r"(lo), "r"(hi) : "memory");
}

// Two bf16 values packed in one word -> two e4m3 codes (low half first).  The two fp32 products come from one
// packed multiply (mul.rn.f32x2, an sm_100 instruction: each half is the same round-to-nearest product as a
// scalar multiply).
__device__ __forceinline__ uint32_t quant_pair(uint32_t two_bf16, float inv) {
  float2 f;
  asm("{\n\t.reg .b64 a, b, d;\n\t"
      "mov.b64 a, {%2, %3};\n\t"
      "mov.b64 b, {%4, %4};\n\t"
      "mul.rn.f32x2 d, a, b;\n\t"
      "mov.b64 {%0, %1}, d;\n\t}"
      : "=f"(f.x), "=f"(f.y)
      : "r"(two_bf16 << 16), "r"(two_bf16 & 0xffff0000u), "f"(inv));
  return (uint32_t)__nv_cvt_float2_to_fp8x2(f, __NV_SATFINITE, __NV_E4M3);
}

// Dynamic shared memory: [warps][QUANT_STAGES] stages of in_stride bytes (row bytes rounded up to 128),
// then [warps][QUANT_STAGES] mbarriers.
// CPL > 0: rows of at most CPL * 512 bytes, held in registers between the two passes -- every lane reads its CPL
// 16-byte chunks from the stage once (independent loads), the maximum and the conversion run from the registers,
// and the codes are written after ONE warp barrier.  The two-pass form below it (CPL == 0, any row length) reads
// the stage twice and needs a warp barrier per chunk, which left a warp at about 0.15 instructions per cycle:
// 3.8 us per 8 KB row, the whole run time at 49 rows per warp.  Registers decide how many warps a CTA may have:
// 16 for CPL <= 16, 8 beyond.
// FULL: the row is a whole number of 512-byte slabs (H % 256 == 0), so a chunk is valid for all lanes or for none
// and the per-lane bounds checks (a possibly divergent branch per chunk) reduce to a warp-uniform one.
// GROUPED (two-pass form only; shorter rows take dispatch_quant_reg_kernel): one scale per 128 elements
// (H % 128 == 0); dynamic shared memory then ends with [warps][2][QUANT_MAX_GROUPS] floats, the scales and the
// reciprocals of the row a warp is working on.
template <int QUANT_STAGES, int CPL, bool FULL, bool GROUPED = false>
__global__ void __launch_bounds__((CPL > 16 ? 8 : QUANT_MAX_WARPS) * 32, 1)
dispatch_quant_kernel(const unsigned char* __restrict__ X, unsigned char* __restrict__ windows_q,
                      float* __restrict__ scales, const RowArgs a, const __grid_constant__ RankMap map) {
  static_assert(!GROUPED || CPL == 0, "group-wise scales of rows held in registers: dispatch_quant_reg_kernel");
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const uint32_t row_bytes = (uint32_t)a.H16 * 16u;          // bf16 row
  const uint32_t code_bytes = (uint32_t)a.H16 * 8u;          // e4m3 row
  const uint32_t stage_stride = (row_bytes + 127u) & ~127u;
  const uint32_t buf0 = smem_addr(smem) + warp * QUANT_STAGES * stage_stride;
  const uint32_t bar0 = smem_addr(smem) + n_warps * QUANT_STAGES * stage_stride + warp * QUANT_STAGES * 8;
  // GROUPED: the scales of the row in hand
  float* group_scale = reinterpret_cast<float*>(smem + (size_t)n_warps * QUANT_STAGES * (stage_stride + 8)) +
                       warp * 2 * QUANT_MAX_GROUPS;                     // [QUANT_MAX_GROUPS] scales, then reciprocals
  float* group_inv = group_scale + QUANT_MAX_GROUPS;
  const int n_groups = a.H16 >> 4;                                      // GROUPED: scales per row
  // Which half-warp, through an opaque instruction: with `lane >> 4` the compiler (12.9) simplified the byte
  // offset (lane >> 4) * 4 to lane >> 2 under the store's guard (lane & 15) == 0 and then reused that address
  // for the unguarded loads of every lane -- a misaligned address on the device.
  int half;
  asm("shr.u32 %0, %1, 4;" : "=r"(half) : "r"(lane));

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < QUANT_STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  auto issue_load = [&](int32_t token, int s) {   // lane 0 only
    mbar_expect_tx(bar0 + 8 * s, row_bytes);
    bulk_load(buf0 + s * stage_stride, X + (size_t)token * row_bytes, row_bytes, bar0 + 8 * s);
  };

  uint64_t evict_first;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));

  // One work item = one token row (items_per_row == 1).  q0 is consumed in this iteration; the load of
  // q1 is issued at its start, into the stage whose code row was stored QUANT_STAGES - 1 iterations ago.
  ItemFeed feed = begin_feed();
  int32_t q0 = a.n_items, q1 = a.n_items;
  // The first two rows of a small job are fixed and depend on nothing a planner writes, so the first load is
  // issued before the wait for a planner in front (moe_plan_dispatch_quant) and before the status checks.
  const bool early = a.static_first >= 2;
  if (early) {
    q0 = fetch_item(a, feed);
    q1 = fetch_item(a, feed);
    if (lane == 0 && q0 < a.n_items) issue_load(q0, 0);
  }
  dependency_wait();      // returns at once unless this launch was allowed to start early
  release_dependents();
  if (must_abort(a)) {
    // a load already in flight must land before this CTA's shared memory is handed back
    if (early && lane == 0 && q0 < a.n_items) mbar_wait(bar0, 0, a.wait_limit_ms);
    end_work(a);
    return;
  }
  if (!early) {
    q0 = fetch_item(a, feed);
    q1 = fetch_item(a, feed);
    if (lane == 0 && q0 < a.n_items) issue_load(q0, 0);
  }
  uint32_t it = 0;
  bool timed_out = false;
  while (q0 < a.n_items) {
    const int32_t q2 = fetch_item(a, feed);
    const int s = it % QUANT_STAGES;
    const uint32_t parity = (it / QUANT_STAGES) & 1u;
    if (lane == 0 && q1 < a.n_items) {
      // the next stage still holds the code row of iteration it + 1 - QUANT_STAGES until its stores have read it
      bulk_wait_read<QUANT_STAGES - 2>();
      issue_load(q1, (it + 1) % QUANT_STAGES);
    }
    const int64_t slot = resolve_slot(a, map, q0, lane, true);   // overlaps the loads in flight
    const uint32_t in = buf0 + s * stage_stride;

    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar0 + 8 * s, parity, a.wait_limit_ms) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) {
      timed_out = true;
      break;
    }

    // amax: |bf16| patterns order like the values, so a per-halfword unsigned max of the
    // sign-cleared words is the maximum magnitude.
    float scale = 1.0f, inv = 1.0f;
    auto scale_from = [&](uint32_t m2) {
      uint32_t mbits = max(m2 & 0xffffu, m2 >> 16);
      mbits = __reduce_max_sync(0xffffffffu, mbits);
      const float amax = __uint_as_float(mbits << 16);
      if (amax > 0.0f) {
        scale = __fdiv_rn(amax, 448.0f);
        inv = __fdiv_rn(448.0f, amax);
      }
    };
    if constexpr (CPL > 0) {
      uint4 v[CPL];
      uint32_t m[4] = {0u, 0u, 0u, 0u};
      const int slabs = a.H16 >> 5;   // FULL: chunks per lane
      auto mine = [&](int k) { return FULL ? k < slabs : lane + 32 * k < a.H16; };
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        if (mine(k)) v[k] = lds128(in + (lane + 32 * k) * 16);
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        if (mine(k)) {
          m[0] = __vmaxu2(m[0], v[k].x & 0x7fff7fffu);
          m[1] = __vmaxu2(m[1], v[k].y & 0x7fff7fffu);
          m[2] = __vmaxu2(m[2], v[k].z & 0x7fff7fffu);
          m[3] = __vmaxu2(m[3], v[k].w & 0x7fff7fffu);
        }
      scale_from(__vmaxu2(__vmaxu2(m[0], m[1]), __vmaxu2(m[2], m[3])));   // the shuffles inside order every lane's reads
      __syncwarp();                                                        // ... in front of every lane's writes
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        if (mine(k)) {
          const uint32_t lo = quant_pair(v[k].x, inv) | (quant_pair(v[k].y, inv) << 16);
          const uint32_t hi = quant_pair(v[k].z, inv) | (quant_pair(v[k].w, inv) << 16);
          sts64(in + (lane + 32 * k) * 8, lo, hi);
        }
    } else if constexpr (GROUPED) {
      // Any row length, in batches of 16 chunks per lane (8 KB of the row, 32 groups), in place like the row-wise
      // two-pass form below: a batch is read into registers, its group maxima come from the transposing butterfly
      // of dispatch_quant_reg_kernel (packed maxima of two chunks per word, 7 shuffles for the batch), one lane per
      // group turns them into scale and reciprocal, and the batch is converted.  (One chunk at a time with a
      // sub-warp reduction and two divisions per lane and chunk ran at 2.3 TB/s on 32 KB rows against 6.1 TB/s for
      // the row-wise form.)  Batch b writes bytes [4096 b, 4096 b + 4096) of the stage, which only batches <= b
      // have read.
      for (int c0 = 0; c0 < a.H16; c0 += 512) {   // warp-uniform trip count; a.H16 is a multiple of 16
        uint4 v[16];
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int c = c0 + lane + 32 * k;
          v[k] = c < a.H16 ? lds128(in + c * 16) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {   // per-halfword maxima of chunks 2i and 2i+1 share a word
          const uint32_t e = __vmaxu2(__vmaxu2(v[2 * i].x & 0x7fff7fffu, v[2 * i].y & 0x7fff7fffu),
                                      __vmaxu2(v[2 * i].z & 0x7fff7fffu, v[2 * i].w & 0x7fff7fffu));
          const uint32_t o = __vmaxu2(__vmaxu2(v[2 * i + 1].x & 0x7fff7fffu, v[2 * i + 1].y & 0x7fff7fffu),
                                      __vmaxu2(v[2 * i + 1].z & 0x7fff7fffu, v[2 * i + 1].w & 0x7fff7fffu));
          w[i] = __vmaxu2(__byte_perm(e, o, 0x5410), __byte_perm(e, o, 0x7632));
        }
        int held = 8;
#pragma unroll
        for (int bit = 8; bit >= 1; bit >>= 1) {
          const bool up = (lane & bit) != 0;
          if (held > 1) {
            held >>= 1;
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (j < held) {
                const uint32_t send = up ? w[j] : w[j + held];
                const uint32_t keep = up ? w[j + held] : w[j];
                w[j] = __vmaxu2(keep, __shfl_xor_sync(0xffffffffu, send, bit));
              }
          } else {   // one word left: both partners finish with the same word
            w[0] = __vmaxu2(w[0], __shfl_xor_sync(0xffffffffu, w[0], bit));
          }
        }
        {
          // lane l of a half-warp holds word l >> 1 (chunks 2 (l >> 1) and 2 (l >> 1) + 1) and takes chunk k = l
          const int l = lane & 15;
          const uint32_t bits = (l & 1) ? (w[0] >> 16) : (w[0] & 0xffffu);
          const int g = (c0 >> 4) + 2 * l + half;
          if (g < n_groups) {
            const float amax = __uint_as_float(bits << 16);
            const float den = amax > 0.0f ? amax : 448.0f;   // an all-zero group: scale and reciprocal 1
            group_scale[g] = __fdiv_rn(den, 448.0f);
            group_inv[g] = __fdiv_rn(448.0f, den);
          }
        }
        __syncwarp();   // the reciprocals are visible; every lane's reads of the batch are in registers
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int c = c0 + lane + 32 * k;
          if (c < a.H16) {
            const float g_inv = group_inv[(c0 >> 4) + 2 * k + half];
            const uint32_t lo = quant_pair(v[k].x, g_inv) | (quant_pair(v[k].y, g_inv) << 16);
            const uint32_t hi = quant_pair(v[k].z, g_inv) | (quant_pair(v[k].w, g_inv) << 16);
            sts64(in + c * 8, lo, hi);
          }
        }
      }
    } else {
      uint32_t m2 = 0;
      for (int c = lane; c < a.H16; c += 32) {
        const uint4 v = lds128(in + c * 16);
        m2 = __vmaxu2(m2, v.x & 0x7fff7fffu);
        m2 = __vmaxu2(m2, v.y & 0x7fff7fffu);
        m2 = __vmaxu2(m2, v.z & 0x7fff7fffu);
        m2 = __vmaxu2(m2, v.w & 0x7fff7fffu);
      }
      scale_from(m2);
      // In place: the pass over chunks c = 32 i + lane reads bytes [512 i, 512 i + 512) and writes bytes
      // [256 i, 256 i + 256), which only earlier passes (and, for i = 0, this pass) have read; the warp
      // barrier puts every lane's read of a pass in front of every lane's write of it.
      for (int c = lane; c - lane < a.H16; c += 32) {   // warp-uniform trip count
        uint4 v = make_uint4(0, 0, 0, 0);
        if (c < a.H16) v = lds128(in + c * 16);
        __syncwarp();
        if (c < a.H16) {
          const uint32_t lo = quant_pair(v.x, inv) | (quant_pair(v.y, inv) << 16);
          const uint32_t hi = quant_pair(v.z, inv) | (quant_pair(v.w, inv) << 16);
          sts64(in + c * 8, lo, hi);
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // code row: generic writes -> bulk-copy reads
    __syncwarp();

    for (int j = 0; j < a.K; ++j) {
      const int64_t row = __shfl_sync(0xffffffffu, slot, j);
      if (lane == 0 && row >= 0) bulk_store(window_row(a, windows_q, row, code_bytes), in, code_bytes, evict_first);
    }
    if constexpr (GROUPED) {   // group_scale was written in front of the warp barrier above
      for (int j = 0; j < a.K; ++j) {
        const int64_t row = __shfl_sync(0xffffffffu, slot, j);
        if (row < 0) continue;
        float* dst = a.scale_base == nullptr ? scales + row * n_groups : a.scale_base[row / a.C] + (row % a.C) * n_groups;
        for (int g = lane; g < n_groups; g += 32) dst[g] = group_scale[g];
      }
    } else if (lane < a.K && slot >= 0) {
      if (a.scale_base == nullptr) scales[slot] = scale;
      else a.scale_base[slot / a.C][slot % a.C] = scale;   // one scale tensor per rank, same row order as its window
    }
    if (lane == 0) bulk_commit();   // one group per iteration
    q0 = q1;
    q1 = q2;
    ++it;
  }
  if (lane == 0) {
    if (timed_out) {   // report, and let the other load in flight land (bounded) before the CTA leaves
      raise_status(a.status, MOE_ERR_TIMEOUT);
      if (q1 < a.n_items) mbar_wait(bar0 + 8 * ((it + 1) % QUANT_STAGES), ((it + 1) / QUANT_STAGES) & 1u, a.wait_limit_ms);
    }
    bulk_wait_all();
  }
  end_work(a);
}

// The register forms as a kernel of their own: once a row of at most CPL * 512 bytes sits in a warp's registers its
// load buffer is free again, so the NEXT row's load is issued right then and travels while this row is converted
// and stored; the codes go to a separate buffer half as wide.  A warp needs 3H bytes of shared memory (2H load
// buffer + H code buffer) instead of the 4H or 6H of a ring of whole-row stages, so more warps -- more rows in
// flight -- share an SM: 10 instead of 5-7 at 14 KB rows.  One load and one group of stores are in flight per warp.
// Dynamic shared memory: [warps] load buffers of l_stride bytes (row bytes rounded up to 128), [warps] code buffers
// of c_stride bytes (codes, then for GROUPED the row's scales and their reciprocals, rounded up to 128), [warps]
// mbarriers.
template <int CPL, bool FULL, bool GROUPED>
__global__ void __launch_bounds__((CPL > 16 ? QUANT_REG_WARPS_LONG : QUANT_REG_WARPS_SHORT) * 32, 1)
dispatch_quant_reg_kernel(const unsigned char* __restrict__ X, unsigned char* __restrict__ windows_q,
                          float* __restrict__ scales, const RowArgs a, const __grid_constant__ RankMap map) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const uint32_t row_bytes = (uint32_t)a.H16 * 16u;          // bf16 row
  const uint32_t code_bytes = (uint32_t)a.H16 * 8u;          // e4m3 row
  const int n_groups = a.H16 >> 4;                            // GROUPED: scales per row
  const uint32_t sc_bytes = GROUPED ? (((uint32_t)n_groups * 4u + 15u) & ~15u) : 0u;
  const uint32_t l_stride = (row_bytes + 127u) & ~127u;
  const uint32_t c_stride = (code_bytes + 2u * sc_bytes + 127u) & ~127u;
  const uint32_t in = smem_addr(smem) + warp * l_stride;
  const uint32_t out = smem_addr(smem) + n_warps * l_stride + warp * c_stride;
  const uint32_t bar = smem_addr(smem) + n_warps * (l_stride + c_stride) + warp * 8;
  int half;   // lane >> 4 through an opaque instruction (see dispatch_quant_kernel)
  asm("shr.u32 %0, %1, 4;" : "=r"(half) : "r"(lane));

  if (lane == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  auto issue_load = [&](int32_t token) {   // lane 0 only
    mbar_expect_tx(bar, row_bytes);
    bulk_load(in, X + (size_t)token * row_bytes, row_bytes, bar);
  };

  uint64_t evict_first;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));

  // One work item = one token row.  q0 is consumed in this iteration; the load of q1 is issued in the middle of
  // it, as soon as every lane holds its part of q0.
  ItemFeed feed = begin_feed();
  int32_t q0 = a.n_items, q1 = a.n_items;
  // The first rows of a small job are fixed and depend on nothing a planner writes, so the first load is issued
  // before the wait for a planner in front and before the status checks.
  const bool early = a.static_first >= 2;
  if (early) {
    q0 = fetch_item(a, feed);
    q1 = fetch_item(a, feed);
    if (lane == 0 && q0 < a.n_items) issue_load(q0);
  }
  dependency_wait();      // returns at once unless this launch was allowed to start early
  release_dependents();
  if (must_abort(a)) {
    // a load already in flight must land before this CTA's shared memory is handed back
    if (early && lane == 0 && q0 < a.n_items) mbar_wait(bar, 0, a.wait_limit_ms);
    end_work(a);
    return;
  }
  if (!early) {
    q0 = fetch_item(a, feed);
    q1 = fetch_item(a, feed);
    if (lane == 0 && q0 < a.n_items) issue_load(q0);
  }
  const int slabs = a.H16 >> 5;   // FULL: chunks per lane
  auto mine = [&](int k) { return FULL ? k < slabs : lane + 32 * k < a.H16; };
  uint32_t it = 0;
  bool timed_out = false;
  while (q0 < a.n_items) {
    const int32_t q2 = fetch_item(a, feed);
    const int64_t slot = resolve_slot(a, map, q0, lane, true);   // overlaps the load in flight
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, it & 1u, a.wait_limit_ms) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) {
      timed_out = true;   // the only load in flight is the one that did not land
      break;
    }
    uint4 v[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k)
      if (mine(k)) v[k] = lds128(in + (lane + 32 * k) * 16);

    float scale = 1.0f, inv = 1.0f;
    if constexpr (GROUPED) {
      const uint32_t sc = out + code_bytes, rc = sc + sc_bytes;
      // Group maxima.  Chunk k of a lane belongs to group 2k + half, whose other fifteen chunks sit in the other
      // lanes of the half-warp.  (A sub-warp redux per chunk compiles into a 35-instruction collective: 1000
      // instructions per 14 KB row.)  Instead the maxima of chunks 2i and 2i+1 share a word, and a transposing
      // butterfly -- at every step a lane hands half of its words to its partner and reduces the other half with
      // what it receives -- leaves lane l of each half-warp with the finished maxima of one word: 15 shuffles and
      // packed maxima for 32 chunks.  That lane turns them into scale and reciprocal, so the divisions of all the
      // row's groups run side by side.
      constexpr int P = CPL / 2;   // words per lane: 16 or 8
      uint32_t w[P];
#pragma unroll
      for (int i = 0; i < P; ++i) {
        uint32_t e = 0u, o = 0u;   // per-halfword maxima of chunk 2i and of chunk 2i+1
        if (mine(2 * i))
          e = __vmaxu2(__vmaxu2(v[2 * i].x & 0x7fff7fffu, v[2 * i].y & 0x7fff7fffu),
                       __vmaxu2(v[2 * i].z & 0x7fff7fffu, v[2 * i].w & 0x7fff7fffu));
        if (mine(2 * i + 1))
          o = __vmaxu2(__vmaxu2(v[2 * i + 1].x & 0x7fff7fffu, v[2 * i + 1].y & 0x7fff7fffu),
                       __vmaxu2(v[2 * i + 1].z & 0x7fff7fffu, v[2 * i + 1].w & 0x7fff7fffu));
        // (max of e's halves, max of o's halves)
        w[i] = __vmaxu2(__byte_perm(e, o, 0x5410), __byte_perm(e, o, 0x7632));
      }
      if (lane == 0) bulk_wait_read<0>();   // the previous row's stores have read the code buffer (the shuffles
                                            // below keep every other lane behind this wait)
      int held = P;
#pragma unroll
      for (int bit = 8; bit >= 1; bit >>= 1) {
        const bool up = (lane & bit) != 0;
        if (held > 1) {
          held >>= 1;
#pragma unroll
          for (int j = 0; j < P / 2; ++j)
            if (j < held) {
              const uint32_t send = up ? w[j] : w[j + held];
              const uint32_t keep = up ? w[j + held] : w[j];
              w[j] = __vmaxu2(keep, __shfl_xor_sync(0xffffffffu, send, bit));
            }
        } else {   // one word left (rows of at most 8 KB): both partners finish with the same word
          w[0] = __vmaxu2(w[0], __shfl_xor_sync(0xffffffffu, w[0], bit));
        }
      }
      // every lane has handed over all of its chunks' maxima: the load buffer is free
      if (lane == 0 && q1 < a.n_items) issue_load(q1);
      {
        // P == 16: lane l of a half-warp holds word l = chunks 2l and 2l+1; P == 8: word l >> 1, of which it takes
        // chunk 2 (l >> 1) + (l & 1)
        const int l = lane & 15;
#pragma unroll
        for (int part = 0; part < (P == 16 ? 2 : 1); ++part) {
          const int k = P == 16 ? 2 * l + part : l;
          const uint32_t bits = (P == 16 ? part : (l & 1)) ? (w[0] >> 16) : (w[0] & 0xffffu);
          const int g = 2 * k + half;
          if (g < n_groups) {
            const float amax = __uint_as_float(bits << 16);
            const float den = amax > 0.0f ? amax : 448.0f;   // an all-zero group: scale and reciprocal 1
            sts_f32(sc + 4 * g, __fdiv_rn(den, 448.0f));
            sts_f32(rc + 4 * g, __fdiv_rn(448.0f, den));
          }
        }
      }
      __syncwarp();
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        if (mine(k)) {
          const float g_inv = lds_f32(rc + 4 * (2 * k + half));
          const uint32_t lo = quant_pair(v[k].x, g_inv) | (quant_pair(v[k].y, g_inv) << 16);
          const uint32_t hi = quant_pair(v[k].z, g_inv) | (quant_pair(v[k].w, g_inv) << 16);
          sts64(out + (lane + 32 * k) * 8, lo, hi);
        }
    } else {
      // amax: |bf16| patterns order like the values, so a per-halfword unsigned max of the sign-cleared words is
      // the maximum magnitude.
      uint32_t m[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        if (mine(k)) {
          m[0] = __vmaxu2(m[0], v[k].x & 0x7fff7fffu);
          m[1] = __vmaxu2(m[1], v[k].y & 0x7fff7fffu);
          m[2] = __vmaxu2(m[2], v[k].z & 0x7fff7fffu);
          m[3] = __vmaxu2(m[3], v[k].w & 0x7fff7fffu);
        }
      const uint32_t m2 = __vmaxu2(__vmaxu2(m[0], m[1]), __vmaxu2(m[2], m[3]));
      const uint32_t mbits = __reduce_max_sync(0xffffffffu, max(m2 & 0xffffu, m2 >> 16));
      // the reduction has consumed every lane's chunks: the load buffer is free
      if (lane == 0) {
        if (q1 < a.n_items) issue_load(q1);
        bulk_wait_read<0>();   // the previous row's stores have read the code buffer
      }
      const float amax = __uint_as_float(mbits << 16);
      if (amax > 0.0f) {
        scale = __fdiv_rn(amax, 448.0f);
        inv = __fdiv_rn(448.0f, amax);
      }
      __syncwarp();
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        if (mine(k)) {
          const uint32_t lo = quant_pair(v[k].x, inv) | (quant_pair(v[k].y, inv) << 16);
          const uint32_t hi = quant_pair(v[k].z, inv) | (quant_pair(v[k].w, inv) << 16);
          sts64(out + (lane + 32 * k) * 8, lo, hi);
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> bulk-copy reads
    __syncwarp();

    for (int j = 0; j < a.K; ++j) {
      const int64_t row = __shfl_sync(0xffffffffu, slot, j);
      if (row < 0) continue;
      if (lane == 0) bulk_store(window_row(a, windows_q, row, code_bytes), out, code_bytes, evict_first);
      if constexpr (GROUPED) {
        // a bulk copy where the row of scales starts on a 16-byte boundary and is a multiple of 16 bytes long
        float* dst = a.scale_base == nullptr ? scales + row * n_groups : a.scale_base[row / a.C] + (row % a.C) * n_groups;
        if ((n_groups & 3) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
          if (lane == 0) bulk_store(dst, out + code_bytes, (uint32_t)n_groups * 4u, evict_first);
        } else {
          for (int g = lane; g < n_groups; g += 32) dst[g] = lds_f32(out + code_bytes + 4 * g);
        }
      }
    }
    if constexpr (!GROUPED) {
      if (lane < a.K && slot >= 0) {
        if (a.scale_base == nullptr) scales[slot] = scale;
        else a.scale_base[slot / a.C][slot % a.C] = scale;   // one scale tensor per rank, same row order as its window
      }
    }
    if (lane == 0) bulk_commit();   // one group per row
    q0 = q1;
    q1 = q2;
    ++it;
  }
  if (lane == 0) {
    if (timed_out) raise_status(a.status, MOE_ERR_TIMEOUT);
    bulk_wait_all();
  }
  end_work(a);
}

}  // namespace moe
