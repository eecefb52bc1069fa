// Top-k gating: router logits -> routing indexes and weights (the step before dispatch).
//
//   topk_idx[t, 0..K-1] = the K largest logits of token t in descending order (equal logits: lower
//                         expert index first)
//   topk_w[t, j]        = exp(l_j - l_0) / sum_j' exp(l_j' - l_0)   (fp32, sum in ascending j)
//
// Rows of up to 1024 logits live in registers, a lane owning consecutive experts (warp_gate_load).  Rows of four
// logits per lane or more are selected by threshold and rank (warp_gate_rank; two tokens per warp for large
// batches: warp_gate_rank_pair); shorter rows, and tokens with too many equal logits for that, by K rounds of
// "largest remaining logit" over cached lane maxima (warp_gate_select).  Rows beyond 1024 logits are cached in
// shared memory and scanned with a shuffle arg-max, one warp per token (warp_gate_token).
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

// Warp-wide max of fp32 values / min of unsigned values in one instruction each (redux.sync; the fp32 form
// is an sm_100a instruction).  Inputs are finite or -inf, never NaN.
__device__ __forceinline__ float warp_max_f32(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}

// The two largest of a lane's VPT logits with their expert indexes, lower index first among equals
// (ascending walk, strict compares); i0, i1 are positions inside the lane.  `dead` bit i set: element i has been
// selected already.
template <int VPT>
__device__ __forceinline__ void lane_top2(const float (&v)[VPT], uint32_t dead, float& h0, int32_t& i0, float& h1,
                                          int32_t& i1) {
  h0 = -INFINITY;
  h1 = -INFINITY;
  i0 = 0x7fffffff;
  i1 = 0x7fffffff;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const float x = ((dead >> i) & 1u) ? -INFINITY : v[i];
    const bool p0 = x > h0, p1 = x > h1;
    h1 = p0 ? h0 : (p1 ? x : h1);
    i1 = p0 ? i0 : (p1 ? i : i1);
    h0 = p0 ? x : h0;
    i0 = p0 ? i : i0;
  }
}

// Rows of at most 32 * VPT logits, held in registers: lane l owns the VPT CONSECUTIVE experts l*VPT .. l*VPT+VPT-1
// (two 16-byte loads per lane at 256 experts), so "lowest expert index" is "lowest lane, then lowest position".
// Every lane keeps its two largest remaining logits cached.  A round is then: redux.max over the lane heads,
// redux.min over the expert indexes of the lanes whose head equals it, and a pop on the one winning lane --
// about a dozen instructions, none of which touches the VPT registers.  Only when a lane has been popped twice
// is its cache rebuilt from its registers (a warp-uniform branch, taken well under once per token at 256 experts,
// top-8).  -inf marks absent and selected entries (logits are finite); -0 and +0 compare equal in every
// comparison made here, so either may be reported as the value (the weights do not depend on the sign of zero).
template <int VPT>
__device__ __forceinline__ void warp_gate_select(const float (&v)[VPT], int K, int lane, int32_t& idx_lane,
                                                 float& w_lane) {
  const int base = lane * VPT;
  uint32_t dead = 0;
  float h0, h1;
  int32_t i0, i1;
  lane_top2<VPT>(v, 0u, h0, i0, h1, i1);
  float sel_val = 0.0f;
  int32_t sel_idx = -1;
  for (int j = 0; j < K; ++j) {
    const float best = warp_max_f32(h0);
    const uint32_t cand = (h0 == best) ? (uint32_t)(base + i0) : 0x7fffffffu;
    const uint32_t be = __reduce_min_sync(0xffffffffu, cand);   // lowest expert index that holds `best`
    if (lane == j) {
      sel_val = best;
      sel_idx = (int32_t)be;
    }
    const bool win = cand == be;          // exactly one lane: expert indexes are unique
    if (win) {
      dead |= 1u << i0;
      h0 = h1;
      i0 = i1;
      h1 = -INFINITY;
      i1 = 0x7fffffff;
    }
    if constexpr (VPT > 2) {
      // popped twice since the last rebuild: this lane's remaining logits are unknown to its cache
      if (__any_sync(0xffffffffu, win && h0 == -INFINITY) && j + 1 < K) {
        if (win) lane_top2<VPT>(v, dead, h0, i0, h1, i1);
      }
    }
  }
  w_lane = sel_val;
  idx_lane = sel_idx;
}

// -1 where a >= b (a > b), else 0.  Written as `set`: the compiler turns the plain conditional into a longer
// sequence (50 more instructions per pair of tokens when the candidate counts were written that way).
__device__ __forceinline__ int32_t ge_mask_f32(float a, float b) {
  int32_t m;
  asm("set.ge.s32.f32 %0, %1, %2;" : "=r"(m) : "f"(a), "f"(b));
  return m;
}
__device__ __forceinline__ int32_t gt_mask_f32(float a, float b) {
  int32_t m;
  asm("set.gt.s32.f32 %0, %1, %2;" : "=r"(m) : "f"(a), "f"(b));
  return m;
}

// Selection by threshold and rank, for the common case.  theta, the K-th largest DISTINCT value among the 32
// lane maxima (K rounds of "warp max, then drop the lanes that hold it": three instructions each, no index
// tracking), is a lower bound of the K-th largest logit, because at least K entries are >= theta; so every
// selected entry is >= theta, and only a few more are (about nine at 256 experts, top-8).  Those entries are
// compacted, in ascending expert order, into one candidate per lane through shared memory; a candidate's place in
// the output is the number of candidates with a larger logit plus the number of EARLIER candidates with an equal
// one (equal logits: lower expert index first), counted directly.  More than 32 candidates (many equal logits, K
// close to 32): the caller falls back to warp_gate_select.
// On success lane j < K holds the j-th selected logit (in w_lane) and its expert.
constexpr int GATE_RANK_WORDS = 136;

template <int VPT>
__device__ __forceinline__ bool warp_gate_rank(const float (&v)[VPT], int K, int lane, float* sm, int32_t& idx_lane,
                                               float& w_lane) {
  float2* cand = reinterpret_cast<float2*>(sm);                  // [36] (value, expert): 32 candidates + padding of the last four
  float* out_val = sm + 72;                                      // [32]
  int32_t* out_idx = reinterpret_cast<int32_t*>(sm + 104);       // [32]
  const int base = lane * VPT;
  float m = v[0];
#pragma unroll
  for (int i = 1; i < VPT; ++i) m = fmaxf(m, v[i]);
  float theta = 0.0f;
  if (K == 8) {   // the common top-k degree, without the loop
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      theta = warp_max_f32(m);
      m = (m == theta) ? -INFINITY : m;
    }
  } else {
    for (int j = 0; j < K; ++j) {
      theta = warp_max_f32(m);
      m = (m == theta) ? -INFINITY : m;
    }
  }
  // absent entries are -inf and must never qualify; logits are finite, so -FLT_MAX admits every real entry
  theta = fmaxf(theta, -3.402823466e+38f);
  int c = 0;
#pragma unroll
  for (int i = 0; i < VPT; ++i) c -= ge_mask_f32(v[i], theta);
  int incl = c;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, incl, d);
    incl += (lane >= d) ? u : 0;
  }
  const int C = __shfl_sync(0xffffffffu, incl, 31);
  if (C > 32) return false;
  if (lane < 3) cand[C + lane].x = -INFINITY;   // the counting loop reads four candidates at a time
  // predicated stores and address steps, no branches: one 8-byte (value, expert) store per candidate
  uint32_t slot = (uint32_t)__cvta_generic_to_shared(cand) + 8u * (uint32_t)(incl - c);
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ge.f32 p, %1, %2;\n\t"
        "@p st.shared.v2.b32 [%0], {%1, %3};\n\t"
        "@p add.u32 %0, %0, 8;\n\t}"
        : "+r"(slot) : "f"(v[i]), "f"(theta), "r"(base + i) : "memory");
  }
  __syncwarp();
  float x = -INFINITY;
  int32_t xi = -1;
  if (lane < C) {
    const float2 me = cand[lane];
    x = me.x + 0.0f;   // -0 becomes +0: equal logits get equal bit patterns
    xi = __float_as_int(me.y);
  }
  int rank = __popc(__match_any_sync(0xffffffffu, __float_as_uint(x)) & lanemask_lt());   // earlier equal candidates
  for (int q = 0; q < C; q += 4) {
    const float4 c01 = *reinterpret_cast<const float4*>(cand + q);   // broadcast reads
    const float4 c23 = *reinterpret_cast<const float4*>(cand + q + 2);
    rank -= gt_mask_f32(c01.x, x) + gt_mask_f32(c01.z, x) + gt_mask_f32(c23.x, x) + gt_mask_f32(c23.z, x);
  }
  if (lane < C && rank < K) {
    out_val[rank] = x;
    out_idx[rank] = xi;
  }
  __syncwarp();
  w_lane = lane < K ? out_val[lane] : 0.0f;
  idx_lane = lane < K ? out_idx[lane] : -1;
  __syncwarp();   // the next token of this warp reuses the buffers
  return true;
}

// Two tokens per warp.  Everything a token costs whatever its row length -- the scan of the candidate counts, the
// rank loop, the softmax and the stores -- is a good half of warp_gate_rank's instructions; here two tokens share
// those instruction streams: the thresholds and the compaction still run over the whole warp for each token (the
// two counts ride through ONE scan, packed in the halves of a word), then lanes 0-15 rank token A's candidates while
// lanes 16-31 rank token B's, and the caller's epilogue works on half-warps.  Needs K <= 16; fails (nothing
// written that matters) if a token has more than 16 candidates -- the caller then takes the tokens one by one.
// On success lane j < K of half h holds the j-th selected logit and expert of token h.
// sm: GATE_PAIR_WORDS words: candidates [2][20] as (value, expert) pairs, selected values [2][16], experts [2][16].
constexpr int GATE_PAIR_WORDS = 144;

template <int VPT>
__device__ __forceinline__ bool warp_gate_rank_pair(const float (&va)[VPT], const float (&vb)[VPT], int K, int lane,
                                                    float* sm, int32_t& idx_lane, float& w_lane) {
  float2* cand = reinterpret_cast<float2*>(sm);                  // [2][20]: 16 candidates + padding of the last four
  float* out_val = sm + 80;                                      // [2][16]
  int32_t* out_idx = reinterpret_cast<int32_t*>(sm + 112);       // [2][16]
  const int base = lane * VPT;
  float ma = va[0], mb = vb[0];
#pragma unroll
  for (int i = 1; i < VPT; ++i) {
    ma = fmaxf(ma, va[i]);
    mb = fmaxf(mb, vb[i]);
  }
  float ta = 0.0f, tb = 0.0f;
  auto round = [&]() {
    ta = warp_max_f32(ma);
    tb = warp_max_f32(mb);
    ma = (ma == ta) ? -INFINITY : ma;
    mb = (mb == tb) ? -INFINITY : mb;
  };
  if (K == 8) {
#pragma unroll
    for (int j = 0; j < 8; ++j) round();
  } else {
    for (int j = 0; j < K; ++j) round();
  }
  ta = fmaxf(ta, -3.402823466e+38f);   // absent entries (-inf) never qualify
  tb = fmaxf(tb, -3.402823466e+38f);
  int na = 0, nb = 0;   // minus this lane's candidate counts
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    na += ge_mask_f32(va[i], ta);
    nb += ge_mask_f32(vb[i], tb);
  }
  const int c = -(na + (nb << 16));   // token A's count in the low half of the word, token B's in the high half
  int incl = c;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, incl, d);
    incl += (lane >= d) ? u : 0;
  }
  const int total = __shfl_sync(0xffffffffu, incl, 31);
  const int Ca = total & 0xffff, Cb = total >> 16;
  if (Ca > 16 || Cb > 16) return false;
  const int half = lane >> 4, l = lane & 15;
  const int Ch = half ? Cb : Ca;
  if (l < 3) cand[half * 20 + Ch + l].x = -INFINITY;   // the counting loop reads four candidates at a time
  const int excl = incl - c;
  const uint32_t sm_addr = (uint32_t)__cvta_generic_to_shared(cand);
  uint32_t slot_a = sm_addr + 8u * (uint32_t)(excl & 0xffff), slot_b = sm_addr + 160u + 8u * (uint32_t)(excl >> 16);
#pragma unroll
  for (int i = 0; i < VPT; ++i) {   // predicated stores and address steps, no branches
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ge.f32 p, %2, %3;\n\t"
        "setp.ge.f32 q, %5, %6;\n\t"
        "@p st.shared.v2.b32 [%0], {%2, %4};\n\t"
        "@q st.shared.v2.b32 [%1], {%5, %4};\n\t"
        "@p add.u32 %0, %0, 8;\n\t"
        "@q add.u32 %1, %1, 8;\n\t}"
        : "+r"(slot_a), "+r"(slot_b)
        : "f"(va[i]), "f"(ta), "r"(base + i), "f"(vb[i]), "f"(tb)
        : "memory");
  }
  __syncwarp();
  const float2* mine = cand + half * 20;
  float x = -INFINITY;
  int32_t xi = -1;
  if (l < Ch) {
    const float2 me = mine[l];
    x = me.x + 0.0f;   // -0 becomes +0: equal logits get equal bit patterns
    xi = __float_as_int(me.y);
  }
  const unsigned same_half_before = lanemask_lt() & (half ? 0xffff0000u : 0x0000ffffu);
  int rank = __popc(__match_any_sync(0xffffffffu, __float_as_uint(x)) & same_half_before);   // earlier equal candidates
  for (int q = 0; q < Ch; q += 4) {
    const float4 c01 = *reinterpret_cast<const float4*>(mine + q);   // broadcast reads inside the half-warp
    const float4 c23 = *reinterpret_cast<const float4*>(mine + q + 2);
    rank -= gt_mask_f32(c01.x, x) + gt_mask_f32(c01.z, x) + gt_mask_f32(c23.x, x) + gt_mask_f32(c23.z, x);
  }
  if (l < Ch && rank < K) {
    out_val[half * 16 + rank] = x;
    out_idx[half * 16 + rank] = xi;
  }
  __syncwarp();
  w_lane = l < K ? out_val[half * 16 + l] : 0.0f;
  idx_lane = l < K ? out_idx[half * 16 + l] : -1;
  __syncwarp();   // the next tokens of this warp reuse the buffers
  return true;
}

// The softmax of warp_gate_softmax for two tokens at once: lane j < K of each half-warp holds its token's j-th logit.
__device__ __forceinline__ float halfwarp_gate_softmax(float sel_val, int K, int lane) {
  const int l = lane & 15;
  const float top = __shfl_sync(0xffffffffu, sel_val, 0, 16);
  const float ex = l < K ? expf(sel_val - top) : 0.0f;
  float sum = 0.0f;
  for (int j0 = 0; j0 < K; j0 += 8) {   // K <= 16: no index leaves the half-warp
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) sum += __shfl_sync(0xffffffffu, ex, j0 + jj, 16);
  }
  return __fdiv_rn(l < K ? ex : 1.0f, sum);
}

// fp32 softmax over the K selected logits (lane j < K holds the j-th), summed in ascending j.
__device__ __forceinline__ float warp_gate_softmax(float sel_val, int K, int lane) {
  const float top = __shfl_sync(0xffffffffu, sel_val, 0);
  const float ex = lane < K ? expf(sel_val - top) : 0.0f;
  float sum = 0.0f;
  // eight terms at a time; the lanes beyond K hold +0, which leaves the sum unchanged (K <= 32, so no index wraps)
  for (int j0 = 0; j0 < K; j0 += 8) {
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) sum += __shfl_sync(0xffffffffu, ex, j0 + jj);
  }
  // the lanes beyond K divide 1 by the sum: a zero numerator would take the division's special-case path
  return __fdiv_rn(lane < K ? ex : 1.0f, sum);
}

// Loads the row of one token into the lane-contiguous register layout.  `vec`: the row starts on a 16-byte
// boundary and E is a multiple of 4, so a lane's run is read with 16-byte loads.
template <int VPT>
__device__ __forceinline__ void warp_gate_load(const float* __restrict__ row, int E, int lane, bool vec,
                                               float (&v)[VPT]) {
  const int base = lane * VPT;
  if constexpr (VPT % 4 == 0) {
    if (vec) {
#pragma unroll
      for (int q = 0; q < VPT / 4; ++q) {
        float4 f = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (base + 4 * q < E) f = __ldg(reinterpret_cast<const float4*>(row + base) + q);
        v[4 * q] = f.x;
        v[4 * q + 1] = f.y;
        v[4 * q + 2] = f.z;
        v[4 * q + 3] = f.w;
      }
      return;
    }
  }
#pragma unroll
  for (int i = 0; i < VPT; ++i) v[i] = base + i < E ? __ldg(row + base + i) : -INFINITY;
}

// One token, start to finish: threshold-and-rank selection (long rows), the rounds when that gives up or for short
// rows, softmax, stores.  sm: GATE_RANK_WORDS words of this warp.
template <int VPT>
__device__ __forceinline__ void warp_gate_one(const float (&v)[VPT], int32_t tok, int K, int lane, float* sm,
                                              int32_t* __restrict__ topk_idx, float* __restrict__ topk_w) {
  int32_t idx;
  float w;
  // rows of one or two logits per lane: the rounds are already cheap (nothing to scan inside a lane)
  bool done = false;
  if constexpr (VPT >= 4) done = warp_gate_rank<VPT>(v, K, lane, sm, idx, w);
  if (!done) warp_gate_select<VPT>(v, K, lane, idx, w);
  w = warp_gate_softmax(w, K, lane);
  if (lane < K) {
    topk_idx[(size_t)tok * K + lane] = idx;
    topk_w[(size_t)tok * K + lane] = w;
  }
}

// Stand-alone gate: grid-stride over tokens.  VPT > 0: register form for rows of at most 32 * VPT logits (one
// instantiation per row length class, so that short rows keep few registers and many warps per SM).  PAIRS: two
// tokens per warp (tokens 2p and 2p+1; needs VPT >= 4 and K <= 16), else one.  VPT == 0: shared-memory form for
// longer rows; dynamic shared memory: warps * E floats.
// The pair form loads its rows when it needs them: 32 resident warps per SM cover the latency, and loading the
// next pair ahead cost 32 registers, moves and spills (13.2 against 12.3 us at 32768 tokens of 256 logits).  No
// kernel inlines a selection form more than twice: with more copies the code outgrew the instruction caches
// (231 KB) and a planner chained behind the gate started 2 us later.
template <int VPT, bool PAIRS>
__global__ void __launch_bounds__(256, VPT == 8 ? 4 : 1)
gate_topk_kernel(const float* __restrict__ logits, int32_t T, int32_t E, int32_t K, int32_t* __restrict__ topk_idx,
                 float* __restrict__ topk_w) {
  extern __shared__ float gate_rows[];
  __shared__ __align__(16) float gate_cand[8][GATE_PAIR_WORDS];   // warp_gate_rank(_pair)'s buffers, one set per warp
  release_dependents();   // a planner launched behind the gate (moe_gate_plan) may be scheduled; it waits for this kernel
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpc = blockDim.x >> 5;
  const int32_t stride = gridDim.x * wpc;
  int32_t t = blockIdx.x * wpc + warp;
  if constexpr (VPT > 0) {
    const bool vec = (E % 4 == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15u) == 0);
    auto process = [&](const float (&v)[VPT], int32_t tok) {
      warp_gate_one<VPT>(v, tok, K, lane, gate_cand[warp], topk_idx, topk_w);
    };
    if constexpr (PAIRS) {
      // t counts pairs here.  An odd T ends in a pair whose second token does not exist: its row is read from
      // the last token again and nothing is stored for it.
      const int32_t pairs = (T + 1) >> 1;
      auto load_pair = [&](int32_t pp, float (&ra)[VPT], float (&rb)[VPT]) {
        const int32_t second = min(2 * pp + 1, T - 1);
        warp_gate_load<VPT>(logits + (size_t)(2 * pp) * E, E, lane, vec, ra);
        warp_gate_load<VPT>(logits + (size_t)second * E, E, lane, vec, rb);
      };
      auto process_pair = [&](const float (&ra)[VPT], const float (&rb)[VPT], int32_t pp) {
        int32_t idx;
        float w;
        if (warp_gate_rank_pair<VPT>(ra, rb, K, lane, gate_cand[warp], idx, w)) {
          w = halfwarp_gate_softmax(w, K, lane);
          const int l = lane & 15;
          const int32_t tok = 2 * pp + (lane >> 4);
          if (l < K && tok < T) {
            topk_idx[(size_t)tok * K + l] = idx;
            topk_w[(size_t)tok * K + l] = w;
          }
        } else {   // too many candidates for a half-warp: one by one (a single copy of that code for both)
          for (int h = 0; h < 2 && 2 * pp + h < T; ++h) {
            float one[VPT];
#pragma unroll
            for (int i = 0; i < VPT; ++i) one[i] = h ? rb[i] : ra[i];
            process(one, 2 * pp + h);
          }
        }
      };
      float a[VPT], b[VPT];
      for (; t < pairs; t += stride) {
        load_pair(t, a, b);
        process_pair(a, b, t);
      }
    } else {
      // two row buffers used in turn, the next token's row travelling while the current one is selected: the short
      // rows' few instructions per token do not cover a load from DRAM (11.2 against 12.2 us, 32768 tokens of 64)
      float row_a[VPT], row_b[VPT];
      if (t < T) warp_gate_load<VPT>(logits + (size_t)t * E, E, lane, vec, row_a);
      while (t < T) {
        if (t + stride < T) warp_gate_load<VPT>(logits + (size_t)(t + stride) * E, E, lane, vec, row_b);
        process(row_a, t);
        t += stride;
        if (t >= T) break;
        if (t + stride < T) warp_gate_load<VPT>(logits + (size_t)(t + stride) * E, E, lane, vec, row_a);
        process(row_b, t);
        t += stride;
      }
    }
  } else {
    for (; t < T; t += stride) {
      int32_t idx;
      float w;
      warp_gate_token(logits + (size_t)t * E, gate_rows + warp * E, E, K, lane, idx, w);
      if (lane < K) {
        topk_idx[(size_t)t * K + lane] = idx;
        topk_w[(size_t)t * K + lane] = w;
      }
      __syncwarp();
    }
  }
}

}  // namespace moe
