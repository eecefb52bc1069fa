/* CPU oracle for relay-buffer-free MoE dispatch / combine.
 *
 * TEST INFRASTRUCTURE ONLY.  This is the plain, slow, sequential definition of
 * what the path computes.  It shares no source, header, helper or constant with
 * the CUDA library, and the CUDA library never calls it.  Only the tests, the
 * smoke check and the benchmark's cpu-baseline leg may load it.
 *
 * All pointers are HOST pointers.  Integer tensors are int32 (slots: int64),
 * hidden states are bf16 stored as uint16_t, routing weights are fp32.
 *
 * Notation follows the paper (Section 5.1, Table 1):
 *   T tokens, H hidden size, K top-k degree, E experts, R ranks, E_r = E / R,
 *   K[t,j] routing index, W[t,j] routing weight, s small offset, o large
 *   offset, M gathered count matrix, n_exp / n_recv receive counts.
 * Tokens of all source ranks are concatenated in rank order; source rank r owns
 * tokens rank_tok_start[r] .. rank_tok_start[r+1]-1.
 *
 * Every function returns one of the ORACLE_* codes below and leaves its outputs
 * untouched when it returns an error.
 */
#ifndef MOE_ORACLE_H
#define MOE_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  ORACLE_OK = 0,
  ORACLE_ERR_INVALID_ARG = 1,
  ORACLE_ERR_BAD_INDEX = 2,
  ORACLE_ERR_CAPACITY = 3
};

/* Top-k gating (the step before dispatch: both workflow figures, Figures 1 and 4, start from a gate
 * that turns hidden states into routing indexes and routing weights).  The paper gives no formula; the reading taken is the common one that the
 * benchmark configurations describe: the K largest router logits of every token, in descending
 * order (equal logits: the lower expert index first), and the softmax over those K logits in fp32:
 *   w_j = exp(l_j - l_0) / sum_{j'=0..K-1} exp(l_j' - l_0),   sum accumulated in ascending j.
 *   logits [T,E] fp32 (finite)  ->  topk_idx [T,K] int32, topk_w [T,K] fp32. */
int oracle_gate_topk(const float* logits, int32_t T, int32_t E, int32_t K, int32_t* topk_idx, float* topk_w);

/* Planning state of the prefill schedule (Layout + Notify, Section 5.2):
 *   M      [R,E]  M[r,e]  = #branches from source rank r to expert e      (gathered count matrix)
 *   c_rank [R,R]  c_rank[r,d] = #branches from source rank r to rank d    (per-rank branch counts)
 *   s      [T,K]  small offset: #earlier branches (flat order t*K+j) of the
 *                 same source rank that chose the same expert             (Layout, definition of s)
 *   o      [E,R]  large offset: first row, local to the window of rank
 *                 dst(e) = e / E_r, of the block (source rank r -> expert e);
 *                 blocks are laid out expert-major, then source rank       (Notify, definition of o)
 *   n_exp  [E]    rows received by expert e;  n_recv [R] rows received by rank d.
 * The decode schedule keeps only (o, s); its values are these same ones (Section 5.3).
 *
 * align (>= 1) is this library's consumer-side extension; the paper has no counterpart and align = 1
 * is its layout.  With align = A > 1 the run of every expert is padded to a whole number of A-row
 * groups, so that every expert's first row is a multiple of A inside its window (a grouped GEMM
 * that reads the window in place in tiles of A rows never sees two experts in one tile):
 *   start_e = sum over earlier experts e' of the same rank of ceil(n_exp[e'] / A) * A,
 *   o[e,r]  = start_e + sum_{r' < r} M[r',e],
 *   n_recv[d] = sum over the experts of rank d of ceil(n_exp[e] / A) * A   (rows the window must hold);
 * n_exp stays the true count, and the padding rows are never written nor read. */
int oracle_plan(const int32_t* topk_idx, int32_t T, int32_t K, int32_t E, int32_t R,
                const int32_t* rank_tok_start, int32_t align,
                int32_t* M, int32_t* c_rank, int32_t* s, int32_t* o,
                int32_t* n_exp, int32_t* n_recv);

/* Notify on its own (Section 5.2, Prefill Notify): from the gathered count matrix M [R,E] -- in a
 * real expert-parallel group every rank contributes its row -- the large offsets o [E,R], the
 * receive counts n_exp [E], n_recv [R] and c_rank [R,R].  oracle_plan is Layout followed by this. */
int oracle_notify(const int32_t* M, int32_t E, int32_t R, int32_t align, int32_t* c_rank, int32_t* o,
                  int32_t* n_exp, int32_t* n_recv);

/* Expert-window row of every branch (two-level offset rule, Section 5.1; Algorithm 1):
 *   slot[t,j] = dst(e) * C + o[e, src(t)] + s[t,j],  e = K[t,j].
 * The windows of the R ranks are R equal segments of C rows of one allocation.
 * ORACLE_ERR_CAPACITY if some n_recv[d] > C. */
int oracle_slots(const int32_t* topk_idx, int32_t T, int32_t K, int32_t E, int32_t R,
                 const int32_t* rank_tok_start, const int32_t* s, const int32_t* o,
                 const int32_t* n_recv, int64_t C, int64_t* slots);

/* Row range of every expert inside the window allocation: the expert FFNs consume the windows in
 * place, without further reordering (Section 5.2, Expert computation), so each expert's rows are one
 * contiguous run:  row_start[e] = dst(e) * C + (rows, padded to groups of `align`, of earlier experts
 * of the same rank), row_count[e] = n_exp[e]. */
int oracle_expert_ranges(int32_t E, int32_t R, int64_t C, int32_t align, const int32_t* n_exp,
                         int64_t* row_start, int32_t* row_count);

/* The same runs cut into tiles of at most tile_rows rows, in window order (rank, expert, position in the
 * run): the work list of a grouped GEMM that reads the windows in place.  Tile k belongs to expert
 * tile_expert[k], starts at window row tile_row[k] and holds tile_valid[k] rows (only the last tile of an
 * expert can be short; an expert without rows has no tile).  At most max_tiles entries are written;
 * *n_tiles is the number of tiles there are.  Consumer-side convenience, no counterpart in the paper. */
int oracle_expert_tiles(int32_t E, int32_t R, int64_t C, int32_t align, int32_t tile_rows, const int32_t* n_exp,
                        int64_t max_tiles, int32_t* tile_expert, int64_t* tile_row, int32_t* tile_valid,
                        int64_t* n_tiles);

/* Dispatch (Algorithm 1, first loop): copy row X[t,:] to window row slot[t,j]
 * for every branch.  Rows no branch maps to are left as the caller set them.
 * n_threads > 1 splits the token range over std::thread workers (same result). */
int oracle_dispatch(const uint16_t* X, int32_t T, int32_t H, int32_t K,
                    const int64_t* slots, uint16_t* windows, int32_t n_threads);

/* Stand-in for the expert FFN (not part of the method): multiply, in place,
 * every received row of expert e by the bf16 scalar scale[e]:
 *   y = bf16_rne(float(x) * float(scale[e])).
 * Rows of expert e are rows start_e .. start_e + n_exp[e] - 1 of its rank's
 * segment, start_e = sum of n_exp (each padded to a multiple of `align`) over earlier experts of the
 * same rank. */
int oracle_expert_scale(uint16_t* windows, int32_t H, int32_t E, int32_t R, int64_t C, int32_t align,
                        const int32_t* n_exp, const uint16_t* scale);

/* Combine (Algorithm 1, second loop):
 *   acc = +0.0f; for j = 0..K-1: acc = fmaf(W[t,j], float(Yexp[slot[t,j], h]), acc);
 *   Y[t,h] = bf16_rne(acc).
 * Y is fully overwritten. */
int oracle_combine(const uint16_t* windows, int32_t T, int32_t H, int32_t K,
                   const int64_t* slots, const float* W, uint16_t* Y, int32_t n_threads);

/* Row-wise quantised dispatch (Section 5.2, Prefill Dispatch: with row-wise quantisation switched on,
 * the scales go to a second tensor laid out row for row like the expert window).
 * The paper fixes no format; the reading taken here is fp8 e4m3 (1-4-3, bias 7, largest finite value
 * 448, no infinities) with one fp32 scale per row:
 *   amax  = max_h |float(X[t,h])|
 *   scale = amax / 448.0f, inv = 448.0f / amax    (fp32, round to nearest; both 1.0f if amax == 0)
 *   code[t,h] = e4m3_rne_sat(float(X[t,h]) * inv) (fp32 product, then round to nearest even, clamped to +-448)
 * and every branch (t,j) gets the same code row and the same scale at window row slot[t,j]:
 *   windows_q [rows, H] uint8,  scales [rows] fp32.   A consumer reads x ~ e4m3_to_float(code) * scale. */
int oracle_dispatch_quant(const uint16_t* X, int32_t T, int32_t H, int32_t K, const int64_t* slots,
                          uint8_t* windows_q, float* scales, int32_t n_threads);

/* The same with one scale per GROUP of `group` consecutive elements of a row instead of one per row (the
 * paper names no granularity; 128 is the group the fp8 expert GEMMs of the benchmark's model family consume):
 * each group is quantised exactly like a row of its own by the rule above.  H % group == 0.
 *   windows_q [rows, H] uint8,  scales [rows, H / group] fp32 (group g of row r at scales[r * (H/group) + g]). */
int oracle_dispatch_quant_group(const uint16_t* X, int32_t T, int32_t H, int32_t K, const int64_t* slots,
                                uint8_t* windows_q, float* scales, int32_t group, int32_t n_threads);

/* e4m3 conversions used above, exported so that tests can pin them against a library conversion. */
uint8_t oracle_float_to_e4m3(float f);
float oracle_e4m3_to_float(uint8_t c);

/* bf16 <-> fp32 conversions used above, exported so that tests can pin them
 * against a library conversion.  Round to nearest, ties to even; NaN stays NaN. */
uint16_t oracle_float_to_bf16(float f);
float oracle_bf16_to_float(uint16_t b);

#ifdef __cplusplus
}
#endif
#endif
