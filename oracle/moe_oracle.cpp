// CPU oracle for relay-buffer-free MoE dispatch / combine.
//
// TEST INFRASTRUCTURE ONLY (see moe_oracle.h).  Plain sequential C++17; the
// definition written out, no blocking, no fusion.  Build:
//   g++ -std=c++17 -O2 -ffp-contract=off -fPIC -shared -pthread moe_oracle.cpp -o liboracle.so
//
// Pins (tests marked "not gpu"): histogram vs a library bincount; s vs the
// literal set-cardinality definition by O(B^2) counting; o vs a library
// cumulative sum; slots vs a library stable sort by expert; dispatch vs
// row-by-row lookup; combine vs exact rational arithmetic, vs an fp64 sum, and
// vs closed forms (identity experts, W = 1/K, one-hot W); bf16 conversion vs a
// library conversion; a hand-worked example.  No function here is unpinned.

#include "moe_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <thread>
#include <vector>

namespace {

// Source rank of token t: the r with rank_tok_start[r] <= t < rank_tok_start[r+1]
// (Algorithm 1: "source rank of token t").
int32_t src_rank(const int32_t* rank_tok_start, int32_t R, int32_t t) {
  for (int32_t r = 0; r < R; ++r)
    if (t < rank_tok_start[r + 1]) return r;
  return R - 1;
}

bool shape_ok(int32_t T, int32_t K, int32_t E, int32_t R, const int32_t* rank_tok_start) {
  if (T < 0 || K < 1 || E < 1 || R < 1 || E % R != 0 || rank_tok_start == nullptr) return false;
  if (rank_tok_start[0] != 0 || rank_tok_start[R] != T) return false;
  for (int32_t r = 0; r < R; ++r)
    if (rank_tok_start[r + 1] < rank_tok_start[r]) return false;
  return true;
}

template <class F>
void for_token_ranges(int32_t T, int32_t n_threads, F body) {
  if (n_threads <= 1 || T < 2) {
    body(0, T);
    return;
  }
  std::vector<std::thread> pool;
  for (int32_t i = 0; i < n_threads; ++i) {
    int32_t lo = (int32_t)((int64_t)T * i / n_threads);
    int32_t hi = (int32_t)((int64_t)T * (i + 1) / n_threads);
    pool.emplace_back([=] { body(lo, hi); });
  }
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

float oracle_bf16_to_float(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

uint16_t oracle_float_to_bf16(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u)          // NaN: keep sign, force a quiet NaN
    return (uint16_t)((u >> 16) | 0x0040u);
  uint32_t lsb = (u >> 16) & 1u;                // ties to even
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

float oracle_e4m3_to_float(uint8_t c) {
  const int sign = c >> 7, exp = (c >> 3) & 15, man = c & 7;
  float v;
  if (exp == 15 && man == 7) v = std::nanf("");
  else if (exp == 0) v = std::ldexp((float)man, -9);             // subnormal: man * 2^-9
  else v = std::ldexp(1.0f + (float)man / 8.0f, exp - 7);
  return sign ? -v : v;
}

uint8_t oracle_float_to_e4m3(float f) {
  if (std::isnan(f)) return 0x7f;
  const uint8_t sign = std::signbit(f) ? 0x80 : 0x00;
  const float a = std::fabs(f);
  if (a >= 448.0f) return sign | 0x7e;                            // clamp to the largest finite value
  if (a < std::ldexp(1.0f, -6)) {                                 // subnormal range: multiples of 2^-9
    const int q = (int)std::nearbyint(std::ldexp(a, 9));          // exact scaling, ties to even
    return sign | (uint8_t)q;                                     // q == 8 is the smallest normal
  }
  int e = std::ilogb(a);                                          // a = m * 2^e, m in [1,2)
  int q = (int)std::nearbyint(std::ldexp(a, 3 - e)) - 8;          // (m - 1) * 8, ties to even
  if (q == 8) { q = 0; ++e; }
  const int code = ((e + 7) << 3) | q;
  return sign | (uint8_t)(code > 0x7e ? 0x7e : code);
}

int oracle_dispatch_quant(const uint16_t* X, int32_t T, int32_t H, int32_t K, const int64_t* slots,
                          uint8_t* windows_q, float* scales, int32_t n_threads) {
  if (T < 0 || H < 1 || K < 1) return ORACLE_ERR_INVALID_ARG;
  for_token_ranges(T, n_threads, [=](int32_t lo, int32_t hi) {
    std::vector<uint8_t> code((size_t)H);
    for (int32_t t = lo; t < hi; ++t) {
      const uint16_t* x = X + (int64_t)t * H;
      float amax = 0.0f;
      for (int32_t h = 0; h < H; ++h) amax = std::fmax(amax, std::fabs(oracle_bf16_to_float(x[h])));
      float scale = 1.0f, inv = 1.0f;
      if (amax > 0.0f) {
        scale = amax / 448.0f;
        inv = 448.0f / amax;
      }
      for (int32_t h = 0; h < H; ++h) code[h] = oracle_float_to_e4m3(oracle_bf16_to_float(x[h]) * inv);
      for (int32_t j = 0; j < K; ++j) {
        const int64_t row = slots[(int64_t)t * K + j];
        std::memcpy(windows_q + row * H, code.data(), (size_t)H);
        scales[row] = scale;
      }
    }
  });
  return ORACLE_OK;
}

int oracle_dispatch_quant_group(const uint16_t* X, int32_t T, int32_t H, int32_t K, const int64_t* slots,
                                uint8_t* windows_q, float* scales, int32_t group, int32_t n_threads) {
  if (T < 0 || H < 1 || K < 1 || group < 1 || H % group != 0) return ORACLE_ERR_INVALID_ARG;
  const int32_t G = H / group;
  for_token_ranges(T, n_threads, [=](int32_t lo, int32_t hi) {
    std::vector<uint8_t> code((size_t)H);
    std::vector<float> scale((size_t)G);
    for (int32_t t = lo; t < hi; ++t) {
      const uint16_t* x = X + (int64_t)t * H;
      for (int32_t g = 0; g < G; ++g) {      // every group of `group` consecutive elements is a little row of its own
        float amax = 0.0f;
        for (int32_t h = g * group; h < (g + 1) * group; ++h) amax = std::fmax(amax, std::fabs(oracle_bf16_to_float(x[h])));
        float inv = 1.0f;
        scale[g] = 1.0f;
        if (amax > 0.0f) {
          scale[g] = amax / 448.0f;
          inv = 448.0f / amax;
        }
        for (int32_t h = g * group; h < (g + 1) * group; ++h) code[h] = oracle_float_to_e4m3(oracle_bf16_to_float(x[h]) * inv);
      }
      for (int32_t j = 0; j < K; ++j) {
        const int64_t row = slots[(int64_t)t * K + j];
        std::memcpy(windows_q + row * H, code.data(), (size_t)H);
        std::memcpy(scales + row * G, scale.data(), (size_t)G * sizeof(float));
      }
    }
  });
  return ORACLE_OK;
}

int oracle_gate_topk(const float* logits, int32_t T, int32_t E, int32_t K, int32_t* topk_idx, float* topk_w) {
  if (T < 0 || E < 1 || K < 1 || K > E) return ORACLE_ERR_INVALID_ARG;
  std::vector<char> taken((size_t)E);
  for (int32_t t = 0; t < T; ++t) {
    const float* l = logits + (int64_t)t * E;
    std::fill(taken.begin(), taken.end(), 0);
    for (int32_t j = 0; j < K; ++j) {          // K rounds of "largest remaining logit, lowest index on ties"
      int32_t best = -1;
      for (int32_t e = 0; e < E; ++e)
        if (!taken[e] && (best < 0 || l[e] > l[best])) best = e;
      taken[best] = 1;
      topk_idx[(int64_t)t * K + j] = best;
    }
    const float top = l[topk_idx[(int64_t)t * K]];
    float sum = 0.0f;
    for (int32_t j = 0; j < K; ++j) {
      const float ex = std::exp(l[topk_idx[(int64_t)t * K + j]] - top);   // float overload: fp32 exponential
      topk_w[(int64_t)t * K + j] = ex;
      sum += ex;
    }
    for (int32_t j = 0; j < K; ++j) topk_w[(int64_t)t * K + j] /= sum;
  }
  return ORACLE_OK;
}

// Smallest multiple of `align` that is >= rows.
static int64_t round_up_rows(int64_t rows, int32_t align) { return (rows + align - 1) / align * align; }

int oracle_notify(const int32_t* M, int32_t E, int32_t R, int32_t align, int32_t* c_rank, int32_t* o,
                  int32_t* n_exp, int32_t* n_recv) {
  if (E < 1 || R < 1 || E % R != 0 || align < 1) return ORACLE_ERR_INVALID_ARG;
  const int32_t E_r = E / R;
  // Per-rank branch counts: c_rank[r,d] = sum over experts of rank d of M[r,e].
  for (int32_t r = 0; r < R; ++r)
    for (int32_t d = 0; d < R; ++d) {
      int32_t acc = 0;
      for (int32_t e = d * E_r; e < (d + 1) * E_r; ++e) acc += M[(size_t)r * E + e];
      c_rank[(size_t)r * R + d] = acc;
    }

  // Notify: receive counts, then large offsets.  Inside the window of rank d
  // the blocks follow each other expert by expert (ascending), and inside an
  // expert source rank by source rank (ascending); o[e,r] is where block
  // (r -> e) begins, counted from the start of rank d's window.  With
  // align > 1 the run of every expert is padded to a whole number of
  // `align`-row groups, so every expert starts on a multiple of align.
  for (int32_t e = 0; e < E; ++e) {
    int32_t acc = 0;
    for (int32_t r = 0; r < R; ++r) acc += M[(size_t)r * E + e];
    n_exp[e] = acc;
  }
  for (int32_t d = 0; d < R; ++d) {
    int32_t acc = 0;
    for (int32_t e = d * E_r; e < (d + 1) * E_r; ++e) {
      for (int32_t r = 0; r < R; ++r) {
        o[(size_t)e * R + r] = acc;
        acc += M[(size_t)r * E + e];
      }
      acc = (int32_t)round_up_rows(acc, align);
    }
    n_recv[d] = acc;
  }
  return ORACLE_OK;
}

int oracle_plan(const int32_t* topk_idx, int32_t T, int32_t K, int32_t E, int32_t R,
                const int32_t* rank_tok_start, int32_t align,
                int32_t* M, int32_t* c_rank, int32_t* s, int32_t* o,
                int32_t* n_exp, int32_t* n_recv) {
  if (!shape_ok(T, K, E, R, rank_tok_start) || align < 1) return ORACLE_ERR_INVALID_ARG;
  if (T > 0 && topk_idx == nullptr) return ORACLE_ERR_INVALID_ARG;
  const int64_t B = (int64_t)T * K;

  // Routing indexes lie in {0..E-1} (Section 5.1); anything else is an error.
  for (int64_t b = 0; b < B; ++b)
    if (topk_idx[b] < 0 || topk_idx[b] >= E) return ORACLE_ERR_BAD_INDEX;

  // Layout: one pass over branches in flat order (t, j).  run[r][e] is the
  // number of branches of source rank r seen so far that chose expert e, so the
  // value read before the increment is s[t,j]; its final value is M[r,e].
  std::vector<int32_t> run((size_t)R * E, 0);
  for (int32_t t = 0; t < T; ++t) {
    const int32_t r = src_rank(rank_tok_start, R, t);
    for (int32_t j = 0; j < K; ++j) {
      const int32_t e = topk_idx[(int64_t)t * K + j];
      s[(int64_t)t * K + j] = run[(size_t)r * E + e]++;
    }
  }
  for (int32_t r = 0; r < R; ++r)
    for (int32_t e = 0; e < E; ++e) M[(size_t)r * E + e] = run[(size_t)r * E + e];

  return oracle_notify(M, E, R, align, c_rank, o, n_exp, n_recv);
}

int oracle_slots(const int32_t* topk_idx, int32_t T, int32_t K, int32_t E, int32_t R,
                 const int32_t* rank_tok_start, const int32_t* s, const int32_t* o,
                 const int32_t* n_recv, int64_t C, int64_t* slots) {
  if (!shape_ok(T, K, E, R, rank_tok_start) || C < 0) return ORACLE_ERR_INVALID_ARG;
  const int32_t E_r = E / R;
  for (int32_t d = 0; d < R; ++d)
    if (n_recv[d] > C) return ORACLE_ERR_CAPACITY;
  for (int64_t b = 0; b < (int64_t)T * K; ++b)
    if (topk_idx[b] < 0 || topk_idx[b] >= E) return ORACLE_ERR_BAD_INDEX;
  for (int32_t t = 0; t < T; ++t) {
    const int32_t r_src = src_rank(rank_tok_start, R, t);
    for (int32_t j = 0; j < K; ++j) {
      const int64_t b = (int64_t)t * K + j;
      const int32_t e = topk_idx[b];
      const int32_t r_dst = e / E_r;                       // destination rank of the branch
      slots[b] = (int64_t)r_dst * C + o[(size_t)e * R + r_src] + s[b];
    }
  }
  return ORACLE_OK;
}

int oracle_expert_ranges(int32_t E, int32_t R, int64_t C, int32_t align, const int32_t* n_exp,
                         int64_t* row_start, int32_t* row_count) {
  if (E < 1 || R < 1 || E % R != 0 || C < 0 || align < 1) return ORACLE_ERR_INVALID_ARG;
  const int32_t E_r = E / R;
  for (int32_t d = 0; d < R; ++d) {
    int64_t local = 0;   // row inside window d
    for (int32_t e = d * E_r; e < (d + 1) * E_r; ++e) {
      row_start[e] = (int64_t)d * C + local;
      row_count[e] = n_exp[e];
      local = round_up_rows(local + n_exp[e], align);
    }
  }
  return ORACLE_OK;
}

int oracle_expert_tiles(int32_t E, int32_t R, int64_t C, int32_t align, int32_t tile_rows, const int32_t* n_exp,
                        int64_t max_tiles, int32_t* tile_expert, int64_t* tile_row, int32_t* tile_valid,
                        int64_t* n_tiles) {
  if (E < 1 || R < 1 || E % R != 0 || C < 0 || align < 1 || tile_rows < 1 || max_tiles < 0) return ORACLE_ERR_INVALID_ARG;
  const int32_t E_r = E / R;
  int64_t k = 0;
  for (int32_t d = 0; d < R; ++d) {
    int64_t local = 0;   // row inside window d where the current expert's run starts
    for (int32_t e = d * E_r; e < (d + 1) * E_r; ++e) {
      for (int32_t r0 = 0; r0 < n_exp[e]; r0 += tile_rows) {   // the expert's run, tile_rows at a time
        if (k < max_tiles) {
          tile_expert[k] = e;
          tile_row[k] = (int64_t)d * C + local + r0;
          tile_valid[k] = n_exp[e] - r0 < tile_rows ? n_exp[e] - r0 : tile_rows;
        }
        ++k;
      }
      local = round_up_rows(local + n_exp[e], align);
    }
  }
  *n_tiles = k;
  return ORACLE_OK;
}

int oracle_dispatch(const uint16_t* X, int32_t T, int32_t H, int32_t K,
                    const int64_t* slots, uint16_t* windows, int32_t n_threads) {
  if (T < 0 || H < 1 || K < 1) return ORACLE_ERR_INVALID_ARG;
  for_token_ranges(T, n_threads, [=](int32_t lo, int32_t hi) {
    for (int32_t t = lo; t < hi; ++t)
      for (int32_t j = 0; j < K; ++j)
        std::memcpy(windows + slots[(int64_t)t * K + j] * H, X + (int64_t)t * H,
                    (size_t)H * sizeof(uint16_t));
  });
  return ORACLE_OK;
}

int oracle_expert_scale(uint16_t* windows, int32_t H, int32_t E, int32_t R, int64_t C, int32_t align,
                        const int32_t* n_exp, const uint16_t* scale) {
  if (H < 1 || E < 1 || R < 1 || E % R != 0 || align < 1) return ORACLE_ERR_INVALID_ARG;
  const int32_t E_r = E / R;
  for (int32_t d = 0; d < R; ++d) {
    int64_t local = 0;   // row inside window d
    for (int32_t e = d * E_r; e < (d + 1) * E_r; ++e) {
      const float sc = oracle_bf16_to_float(scale[e]);
      for (int32_t i = 0; i < n_exp[e]; ++i) {
        const int64_t row = (int64_t)d * C + local + i;
        for (int32_t h = 0; h < H; ++h) {
          uint16_t* p = windows + row * H + h;
          *p = oracle_float_to_bf16(oracle_bf16_to_float(*p) * sc);
        }
      }
      local = round_up_rows(local + n_exp[e], align);   // padding rows are not the expert's
    }
  }
  return ORACLE_OK;
}

int oracle_combine(const uint16_t* windows, int32_t T, int32_t H, int32_t K,
                   const int64_t* slots, const float* W, uint16_t* Y, int32_t n_threads) {
  if (T < 0 || H < 1 || K < 1) return ORACLE_ERR_INVALID_ARG;
  for_token_ranges(T, n_threads, [=](int32_t lo, int32_t hi) {
    for (int32_t t = lo; t < hi; ++t)
      for (int32_t h = 0; h < H; ++h) {
        float acc = 0.0f;
        for (int32_t j = 0; j < K; ++j) {
          const int64_t b = (int64_t)t * K + j;
          acc = std::fmaf(W[b], oracle_bf16_to_float(windows[slots[b] * H + h]), acc);
        }
        Y[(int64_t)t * H + h] = oracle_float_to_bf16(acc);
      }
  });
  return ORACLE_OK;
}

}  // extern "C"
