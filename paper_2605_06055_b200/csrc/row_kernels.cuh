// Payload kernels: dispatch (scatter rows into expert windows) and combine
// (gather rows from expert windows + fp32 weighted sum), both token-major.
//
// Algorithm 1 / Algorithm 2 of the paper.  One warp owns one token at a time:
// lane j < K resolves branch (t, j) to its window row with the two-level offset
// rule slot = dst(e)*C + o[e, src(t)] + s[t,j]; then the whole warp moves the
// row in 16-byte chunks.  Dispatch reads X[t,:] from HBM exactly once and
// stores it K times; combine issues the K loads of a chunk before its
// j-ordered fma chain.  There is no relay, permute or unpermute buffer.
#pragma once

#include "common.cuh"

namespace moe {

struct RowArgs {
  const int32_t* topk_idx;   // [T,K]
  const int32_t* small_off;  // PREFILL: s [T,K].  DECODE: in-tile rank [T,K]
  int32_t* small_out;        // DECODE dispatch: where delta is recorded; else nullptr
  const int32_t* tile_base;  // DECODE: [tiles,E] exclusive tile bases; PREFILL: nullptr
  const int32_t* large_off;  // o [E,R]
  const int32_t* n_recv;     // [R]
  int32_t* status;
  int64_t C;                 // rows per window segment
  int32_t T, K, E, R, E_r;
  int32_t H16;               // 16-byte chunks per row
};

// Window row of branch (t, lane) for lane < K, -1 otherwise.  Small offsets of
// the DECODE schedule are finished here (in-tile rank + tile base).
__device__ __forceinline__ int64_t resolve_slot(const RowArgs& a, const RankMap& map, int32_t t, int lane,
                                                bool record) {
  if (lane >= a.K) return -1;
  const int32_t b = t * a.K + lane;
  const int32_t e = __ldg(a.topk_idx + b);
  if (e < 0 || e >= a.E) return -1;  // flagged by the plan; never dereferenced
  const int32_t r = src_rank(map, t);
  int32_t so = __ldg(a.small_off + b);
  if (a.tile_base != nullptr) {
    so += __ldg(a.tile_base + (size_t)tile_of_branch(map, r, b, a.K) * a.E + e);
    if (record) a.small_out[b] = so;
  }
  return (int64_t)(e / a.E_r) * a.C + __ldg(a.large_off + (size_t)e * a.R + r) + so;
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

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

// ---------------------------------------------------------------- dispatch
// KT > 0: K known at compile time (row pointers live in registers).
// KT == 0: any K <= 32 (row index fetched by shuffle per store).
template <int KT, int UNROLL>
__global__ void __launch_bounds__(256)
dispatch_rows_kernel(const uint4* __restrict__ X, uint4* __restrict__ windows, const RowArgs a,
                     const __grid_constant__ RankMap map) {
  if (must_abort(a)) return;
  const int lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  const int32_t warp0 = blockIdx.x * warps_per_cta + (threadIdx.x >> 5);
  const int32_t nwarps = gridDim.x * warps_per_cta;
  const int K = KT > 0 ? KT : a.K;
  const int H16 = a.H16;

  for (int32_t t = warp0; t < a.T; t += nwarps) {
    const int64_t slot = resolve_slot(a, map, t, lane, true);
    const uint4* src = X + (size_t)t * H16;
    if constexpr (KT > 0) {
      uint4* dst[KT];
#pragma unroll
      for (int j = 0; j < KT; ++j) {
        const int64_t row = __shfl_sync(0xffffffffu, slot, j);
        dst[j] = row >= 0 ? windows + (size_t)row * H16 : nullptr;
      }
      int c = lane;
      for (; c + 32 * (UNROLL - 1) < H16; c += 32 * UNROLL) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream(src + c + 32 * u);
#pragma unroll
        for (int j = 0; j < KT; ++j)
          if (dst[j] != nullptr) {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) st_stream(dst[j] + c + 32 * u, v[u]);
          }
      }
      for (; c < H16; c += 32) {
        const uint4 v = ld_stream(src + c);
#pragma unroll
        for (int j = 0; j < KT; ++j)
          if (dst[j] != nullptr) st_stream(dst[j] + c, v);
      }
    } else {
      for (int c0 = 0; c0 < H16; c0 += 32) {   // warp-uniform trip count: shuffles stay convergent
        const int c = c0 + lane;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (c < H16) v = ld_stream(src + c);
        for (int j = 0; j < K; ++j) {
          const int64_t row = __shfl_sync(0xffffffffu, slot, j);
          if (row >= 0 && c < H16) st_stream(windows + (size_t)row * H16 + c, v);
        }
      }
    }
  }
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

template <int KT, int UNROLL>
__global__ void __launch_bounds__(256)
combine_rows_kernel(const uint4* __restrict__ windows, const float* __restrict__ topk_w, uint4* __restrict__ Y,
                    const RowArgs a, const __grid_constant__ RankMap map) {
  if (must_abort(a)) return;
  const int lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  const int32_t warp0 = blockIdx.x * warps_per_cta + (threadIdx.x >> 5);
  const int32_t nwarps = gridDim.x * warps_per_cta;
  const int K = KT > 0 ? KT : a.K;
  const int H16 = a.H16;

  for (int32_t t = warp0; t < a.T; t += nwarps) {
    const int64_t slot = resolve_slot(a, map, t, lane, false);
    const float w_lane = lane < K ? __ldg(topk_w + (size_t)t * K + lane) : 0.0f;
    uint4* out = Y + (size_t)t * H16;
    if constexpr (KT > 0) {
      const uint4* src[KT];
      float w[KT];
#pragma unroll
      for (int j = 0; j < KT; ++j) {
        const int64_t row = __shfl_sync(0xffffffffu, slot, j);
        src[j] = row >= 0 ? windows + (size_t)row * H16 : nullptr;
        w[j] = __shfl_sync(0xffffffffu, w_lane, j);
      }
      int c = lane;
      for (; c + 32 * (UNROLL - 1) < H16; c += 32 * UNROLL) {
        uint4 v[UNROLL][KT];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
#pragma unroll
          for (int j = 0; j < KT; ++j)
            v[u][j] = src[j] != nullptr ? ld_stream(src[j] + c + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int j = 0; j < KT; ++j) fma_bf16x8(acc, w[j], v[u][j]);   // j ascending, one fma per term
          out[c + 32 * u] = pack_bf16x8(acc);
        }
      }
      for (; c < H16; c += 32) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        uint4 v[KT];
#pragma unroll
        for (int j = 0; j < KT; ++j) v[j] = src[j] != nullptr ? ld_stream(src[j] + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < KT; ++j) fma_bf16x8(acc, w[j], v[j]);
        out[c] = pack_bf16x8(acc);
      }
    } else {
      for (int c0 = 0; c0 < H16; c0 += 32) {
        const int c = c0 + lane;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int j = 0; j < K; ++j) {
          const int64_t row = __shfl_sync(0xffffffffu, slot, j);
          const float w = __shfl_sync(0xffffffffu, w_lane, j);
          uint4 v = make_uint4(0, 0, 0, 0);
          if (row >= 0 && c < H16) v = ld_stream(windows + (size_t)row * H16 + c);
          fma_bf16x8(acc, w, v);
        }
        if (c < H16) out[c] = pack_bf16x8(acc);
      }
    }
  }
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
    int32_t so = __ldg(a.small_off + b);
    if (a.tile_base != nullptr) so += __ldg(a.tile_base + (size_t)tile_of_branch(map, r, b, a.K) * a.E + e);
    slots[b] = (int32_t)((int64_t)(e / a.E_r) * a.C + __ldg(a.large_off + (size_t)e * a.R + r) + so);
  }
}

}  // namespace moe
