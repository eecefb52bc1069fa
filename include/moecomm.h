/* libmoecomm -- relay-buffer-free MoE dispatch / combine on one NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only.  Every pointer parameter says whether
 * it is a HOST or a DEVICE pointer.  The library allocates no device memory:
 * payload tensors and the control-state workspace are caller-owned.  All work
 * is enqueued on the caller's CUDA stream (a cudaStream_t passed as void*; NULL
 * is the default stream) and nothing synchronises except moe_status().
 *
 * Model (paper Section 3.2, Section 5.1).  The pooled, symmetric HBM of an
 * expert-parallel group of R ranks is one allocation `windows` of R equal
 * segments of C rows of H bf16 values; segment d is the expert window of rank
 * d, which hosts experts d*E_r .. (d+1)*E_r-1, E_r = E / R.  Tokens of all
 * source ranks are concatenated in rank order; source rank r owns tokens
 * rank_tok_start[r] .. rank_tok_start[r+1]-1.  A routed branch (t, j) with
 * expert e = K[t,j] lives in window row
 *
 *     slot(t,j) = dst(e) * C + o[e, src(t)] + s[t,j],      dst(e) = e / E_r
 *
 * (two-level offset rule, Section 5.1): o is the large offset (start of the
 * block "source rank r -> expert e" inside rank dst(e)'s window; blocks are laid
 * out expert-major, then by source rank), s is the small offset (number of
 * earlier branches, in (t, j) order, of the same source rank to the same
 * expert).  Slots are therefore deterministic and stable in token order.
 *
 * Limits: 1 <= R <= MOE_MAX_R, E % R == 0, E <= MOE_MAX_E, 1 <= K <= MOE_MAX_K,
 * H % 8 == 0 (rows are whole 16-byte chunks), T_max * K < 2^31.
 * Thread safety: one context per stream; a context holds no global state.
 */
#ifndef MOECOMM_H
#define MOECOMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOE_MAX_R 256
#define MOE_MAX_E 4096
#define MOE_MAX_K 32

typedef enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = 1, /* host-detected: null/misaligned pointer, bad shape, T > T_max ...      */
  MOE_ERR_BAD_INDEX = 2,   /* device-detected by moe_plan: a routing index outside [0, E)           */
  MOE_ERR_CAPACITY = 3,    /* device-detected: some n_recv[d] > capacity_rows; nothing was written  */
  MOE_ERR_NOT_PLANNED = 4, /* dispatch / combine / slots / view before a successful moe_plan        */
  MOE_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired                                    */
  MOE_ERR_CUDA = 6,        /* a CUDA runtime call or kernel launch failed                           */
  MOE_ERR_STALE_PEERS = 7  /* host-detected: the installed window address table is missing or out of date   */
} moe_status_t;

/* The two schedules of Section 4.  PREFILL runs Layout + Notify as separate
 * planning passes (folded into one launch when every source rank holds at most
 * 4096 branches) and keeps the whole planning table readable.  DECODE keeps
 * only the compact state (o_dec, delta, n_recv); delta is produced inside the
 * dispatch launch (Section 5.3, Decode Dispatch), or already by the single
 * planning launch when every source rank holds at most 4096 branches. */
typedef enum { MOE_SCHED_PREFILL = 0, MOE_SCHED_DECODE = 1 } moe_schedule_t;

typedef struct {
  int32_t T_max; /* largest total token count a plan may be asked for */
  int32_t H;     /* hidden size, multiple of 8                        */
  int32_t E;     /* experts                                           */
  int32_t R;     /* virtual expert-parallel ranks                     */
  int32_t K;     /* top-k routing degree                              */
} moe_shape_t;

typedef struct moe_ctx moe_ctx_t; /* opaque, HOST-side handle */

/* Bytes of DEVICE workspace a context of this shape needs (control state only:
 * O(T_max*K + R*E) int32).  0 if the shape is invalid. */
size_t moe_workspace_bytes(const moe_shape_t* shape /*HOST*/);

/* Creates a context over a caller-owned DEVICE workspace (256-byte aligned, at
 * least moe_workspace_bytes(shape) bytes, must outlive the context).  Clears
 * the control words with a synchronous memset; call it outside stream capture.
 * The context is bound to the CUDA device that is current at this call. */
moe_status_t moe_create(const moe_shape_t* shape /*HOST*/, void* workspace /*DEVICE*/,
                        size_t workspace_bytes, moe_ctx_t** out /*HOST*/);
moe_status_t moe_destroy(moe_ctx_t* ctx);

/* Planning (Section 5.2 Prefill Layout + Prefill Notify; Section 5.3 first step
 * of Decode Dispatch): from the routing indexes computes the count matrix M,
 * the small offsets s and the large offsets o (exclusive scan of M in window
 * order), plus c_rank, n_exp, n_recv.
 *   topk_idx        DEVICE [T,K] int32, values in [0,E).  The library reads it again in every
 *                   dispatch / combine / slots call of this plan: keep it valid and unchanged.
 *   rank_tok_start  HOST   [R+1] int32, nondecreasing, [0]=0, [R]=T; NULL means
 *                   uniform T/R tokens per rank (T % R must be 0).  Read before
 *                   the call returns.
 * An index outside [0,E) sets the device status word to MOE_ERR_BAD_INDEX (the
 * paper defines routing indexes in {0..E-1} only; there is no "dropped branch"
 * value).  Calls enqueued behind such a plan write nothing, and when moe_status()
 * reports the error it also discards the plan: dispatch / combine / slots then
 * return MOE_ERR_NOT_PLANNED until a new plan has been made. */
moe_status_t moe_plan(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx /*DEVICE*/,
                      int32_t T, const int32_t* rank_tok_start /*HOST*/, void* stream);

/* Top-k gating, the step in front of the path (Figures 1 and 4: top-k gating produces routing indexes
 * and weights).  The paper gives no formula; this library's definition is the K largest router logits
 * of a token in descending order (equal logits: lower expert index first) and the fp32 softmax over
 * those K logits, summed in ascending j.  Logits must be finite.
 *   logits    DEVICE [T,E] fp32            topk_idx  DEVICE [T,K] int32, out
 *                                          topk_w    DEVICE [T,K] fp32, out
 * moe_gate_topk is the stand-alone kernel (no context).  moe_gate_plan is the gate followed by
 * moe_plan on the indexes it wrote, enqueued back to back and chained (see MOE_OPT_OVERLAP): the planner
 * is scheduled while the gate kernel runs and reads the indexes once that kernel has completed.  (A
 * variant that gated inside the one-CTA-per-rank planner measured slower: gating is instruction-bound
 * and wants every SM.)
 * topk_idx must stay valid like moe_plan's input. */
moe_status_t moe_gate_topk(const float* logits /*DEVICE*/, int32_t T, int32_t E, int32_t K,
                           int32_t* topk_idx /*DEVICE*/, float* topk_w /*DEVICE*/, void* stream);
moe_status_t moe_gate_plan(moe_ctx_t* ctx, moe_schedule_t schedule, const float* logits /*DEVICE*/, int32_t T,
                           const int32_t* rank_tok_start /*HOST*/, int32_t* topk_idx /*DEVICE*/,
                           float* topk_w /*DEVICE*/, void* stream);

/* DEVICE views into the workspace, valid until the next moe_plan on this
 * context.  Shapes: counts M [R,E], c_rank [R,R], small_off s|delta [T,K],
 * large_off o|o_dec [E,R] (window-local row), n_exp [E], n_recv [R].
 * PREFILL fills every field.  DECODE leaves counts, c_rank and n_exp NULL, and
 * small_off is guaranteed to hold delta only after moe_dispatch has run (small
 * decode batches, at most 4096 branches per source rank, are planned in a single
 * launch that already leaves it final after moe_plan).
 * rows [T,K] is what the last dispatch over the whole batch recorded for this plan (see MOE_OPT_SLOT_REUSE):
 * the window row d*capacity_rows + large_off + small_off of every branch, the same numbers moe_slots writes,
 * for the capacity_rows given in rows_capacity; NULL and -1 when nothing is recorded (no such dispatch since
 * the plan, or an error was reported since).  Its contents are final once that dispatch has completed. */
typedef struct {
  const int32_t* counts;
  const int32_t* c_rank;
  const int32_t* small_off;
  const int32_t* large_off;
  const int32_t* n_exp;
  const int32_t* n_recv;
  const int32_t* rows;
  int64_t rows_capacity;
} moe_plan_view_t;
moe_status_t moe_plan_view(const moe_ctx_t* ctx, moe_plan_view_t* out /*HOST*/);

/* Dispatch (Algorithm 1 / Algorithm 2, first loop; Section 5.2 Prefill Dispatch):
 * copies row X[t,:] to window row slot(t,j) for every branch.
 *   x        DEVICE [T,H] bf16, 16-byte aligned
 *   windows  DEVICE [R, capacity_rows, H] bf16, 16-byte aligned
 * Rows >= n_recv[d] of segment d are never written.  If some n_recv[d] exceeds
 * capacity_rows the status word becomes MOE_ERR_CAPACITY and nothing is written. */
moe_status_t moe_dispatch(moe_ctx_t* ctx, const void* x /*DEVICE*/, void* windows /*DEVICE*/,
                          int64_t capacity_rows, void* stream);

/* Planning folded into the dispatch call (Section 5.3, Decode Dispatch: the count and offset state is
 * produced inside the dispatch procedure instead of by a separate Layout -> Notify sequence).
 * Same result as moe_plan followed by moe_dispatch with the same arguments, for either schedule; the
 * plan stays valid for moe_combine, moe_slots and the other consumers.  The dispatch kernel is
 * launched with programmatic stream serialization behind the planner: it starts while the planner
 * runs, moves the first payload loads of every warp (they depend on nothing the planner writes),
 * and waits for the planner's completion before it reads any offset.  x and topk_idx need only be
 * ready in stream order, as for the separate calls. */
moe_status_t moe_plan_dispatch(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx /*DEVICE*/,
                               int32_t T, const int32_t* rank_tok_start /*HOST*/, const void* x /*DEVICE*/,
                               void* windows /*DEVICE*/, int64_t capacity_rows, void* stream);

/* The whole front of a layer in one call: moe_gate_topk, moe_plan and moe_dispatch enqueued back to
 * back and chained like moe_plan_dispatch (the planner is scheduled behind the gate kernel and reads the
 * indexes only after that kernel has completed; the dispatch kernel is scheduled behind the planner,
 * releases nothing and reads no index before the planner has passed that point).  Same result as the
 * three calls.  Arguments as in moe_gate_plan and moe_dispatch; topk_idx and topk_w are outputs. */
moe_status_t moe_gate_plan_dispatch(moe_ctx_t* ctx, moe_schedule_t schedule, const float* logits /*DEVICE*/,
                                    int32_t T, const int32_t* rank_tok_start /*HOST*/,
                                    int32_t* topk_idx /*DEVICE*/, float* topk_w /*DEVICE*/,
                                    const void* x /*DEVICE*/, void* windows /*DEVICE*/, int64_t capacity_rows,
                                    void* stream);

/* Row-wise quantised dispatch (Section 5.2, Prefill Dispatch: with row-wise quantisation the scale
 * values go to a parallel scale tensor in the same row order).  The paper names no format; this
 * library's definition is fp8 e4m3 (1-4-3, bias 7, largest finite 448, no infinities) with one fp32
 * scale per row:  amax = max_h |x[t,h]|,  scale = amax / 448,  inv = 448 / amax  (fp32, round to
 * nearest; both 1 when amax == 0),  code[h] = e4m3_round_nearest_even_saturating(x[t,h] * inv).
 * Every branch (t,j) receives the same code row and scale at window row slot(t,j); a consumer
 * reconstructs x ~ e4m3_to_float(code) * scale.  Inputs must be finite.
 *   x          DEVICE [T,H] bf16, 16-byte aligned; H % 16 == 0 and H <= 16384
 *   windows_q  DEVICE [R, capacity_rows, H] uint8 (e4m3 codes), 16-byte aligned
 *   scales     DEVICE [R, capacity_rows] fp32
 * Errors and untouched padding rows as in moe_dispatch. */
moe_status_t moe_dispatch_quant(moe_ctx_t* ctx, const void* x /*DEVICE*/, void* windows_q /*DEVICE*/,
                                float* scales /*DEVICE*/, int64_t capacity_rows, void* stream);

/* moe_plan followed by moe_dispatch_quant as one chained call, like moe_plan_dispatch: the quantising
 * dispatch kernel is scheduled while the planner runs and loads its first rows meanwhile.  Same result
 * as the two calls. */
moe_status_t moe_plan_dispatch_quant(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx /*DEVICE*/,
                                     int32_t T, const int32_t* rank_tok_start /*HOST*/, const void* x /*DEVICE*/,
                                     void* windows_q /*DEVICE*/, float* scales /*DEVICE*/, int64_t capacity_rows,
                                     void* stream);

/* The quantised dispatch with one scale per GROUP of group_size consecutive elements of a row instead of
 * one per row (same passage; the paper names no granularity either, and 128 is what fp8 expert GEMMs with
 * 1 x 128 activation scales consume).  Every group is quantised by the rule of moe_dispatch_quant as if it
 * were a row of its own.
 *   group_size must be 128 and H % 128 == 0 (else MOE_ERR_INVALID_ARG); H <= 16384
 *   windows_q  DEVICE [R, capacity_rows, H] uint8, 16-byte aligned
 *   scales     DEVICE [R, capacity_rows, H / 128] fp32: group g of window row r at scales[r * (H/128) + g]
 * Otherwise as moe_dispatch_quant. */
moe_status_t moe_dispatch_quant_group(moe_ctx_t* ctx, const void* x /*DEVICE*/, void* windows_q /*DEVICE*/,
                                      float* scales /*DEVICE*/, int64_t capacity_rows, int32_t group_size,
                                      void* stream);

/* moe_plan followed by moe_dispatch_quant_group as one chained call (see moe_plan_dispatch_quant). */
moe_status_t moe_plan_dispatch_quant_group(moe_ctx_t* ctx, moe_schedule_t schedule,
                                           const int32_t* topk_idx /*DEVICE*/, int32_t T,
                                           const int32_t* rank_tok_start /*HOST*/, const void* x /*DEVICE*/,
                                           void* windows_q /*DEVICE*/, float* scales /*DEVICE*/,
                                           int64_t capacity_rows, int32_t group_size, void* stream);

/* Combine (Algorithm 1 / Algorithm 2, second loop; Section 5.2 Prefill Combine):
 *   Y[t,h] = bf16_rne( sum_{j=0..K-1} W[t,j] * float(windows[slot(t,j), h]) )
 * accumulated in fp32 from +0 with one fused multiply-add per term, j ascending.
 *   windows  DEVICE expert outputs, same layout as in moe_dispatch
 *   topk_w   DEVICE [T,K] fp32
 *   y        DEVICE [T,H] bf16, 16-byte aligned, fully overwritten */
moe_status_t moe_combine(moe_ctx_t* ctx, const void* windows /*DEVICE*/, int64_t capacity_rows,
                         const float* topk_w /*DEVICE*/, void* y /*DEVICE*/, void* stream);

/* Token sub-ranges of a plan (a convenience of this library; the paper has no counterpart -- its kernels
 * take a whole batch): the same as moe_dispatch / moe_combine for tokens t_begin <= t < t_end
 * only (x and y are still the full [T,H] tensors).  Chunks of a prefill batch can so be dispatched as
 * they arrive and combined as their experts finish; any partition of [0,T) gives the same bytes. */
moe_status_t moe_dispatch_range(moe_ctx_t* ctx, const void* x /*DEVICE*/, void* windows /*DEVICE*/,
                                int64_t capacity_rows, int32_t t_begin, int32_t t_end, void* stream);
moe_status_t moe_combine_range(moe_ctx_t* ctx, const void* windows /*DEVICE*/, int64_t capacity_rows,
                               const float* topk_w /*DEVICE*/, void* y /*DEVICE*/, int32_t t_begin, int32_t t_end,
                               void* stream);

/* Multi-rank decomposition of the same path (one process and one context per expert-parallel rank,
 * Section 5.2: Layout is local, Notify exchanges count metadata only, Dispatch places rows directly
 * into the destination ranks' windows, Combine reads them directly from there).
 *   moe_layout   plans THIS rank's tokens only: small offsets s and the rank's row of the count matrix,
 *                copied to counts_row (DEVICE [E] int32) for the caller to all-gather over the group.
 *   moe_notify   takes the gathered matrix counts_all (DEVICE [R,E] int32, row r from rank r) and builds
 *                the large offsets and receive counts; the context is then planned.
 *   moe_dispatch_peers / moe_combine_peers
 *                as moe_dispatch / moe_combine for the local tokens, with the window of rank d at
 *                window_bases[d] (DEVICE array of R DEVICE pointers, each [capacity_rows, H] bf16,
 *                16-byte aligned): peer-mapped windows of the other GPUs, or separate allocations.
 * The library launches no collective and waits for no peer: the caller orders the phases (all-gather
 * of the counts between layout and notify; a barrier after dispatch and after the experts). */
moe_status_t moe_layout(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx /*DEVICE [T_local,K]*/,
                        int32_t T_local, int32_t my_rank, int32_t* counts_row /*DEVICE*/, void* stream);
moe_status_t moe_notify(moe_ctx_t* ctx, const int32_t* counts_all /*DEVICE*/, void* stream);
moe_status_t moe_dispatch_peers(moe_ctx_t* ctx, const void* x /*DEVICE*/, const void* const* window_bases /*DEVICE*/,
                                int64_t capacity_rows, void* stream);
moe_status_t moe_combine_peers(moe_ctx_t* ctx, const void* const* window_bases /*DEVICE*/, int64_t capacity_rows,
                               const float* topk_w /*DEVICE*/, void* y /*DEVICE*/, void* stream);
/* Row-wise quantised dispatch in the same decomposition: code window and scale tensor of rank d start at
 * window_q_bases[d] (uint8 [capacity_rows, H]) and scale_bases[d] (fp32 [capacity_rows]); both tables are
 * DEVICE arrays of R device pointers. */
moe_status_t moe_dispatch_quant_peers(moe_ctx_t* ctx, const void* x /*DEVICE*/,
                                      const void* const* window_q_bases /*DEVICE*/,
                                      float* const* scale_bases /*DEVICE*/, int64_t capacity_rows, void* stream);

/* Window addresses of the expert-parallel group (Section 3.2: every rank's slice of the pooled memory is
 * visible to every rank; Section 5.3, Decode Combine, and Section 6.1: remote window addresses are made
 * available by an address handshake, or, in the cached-address mode, taken from an earlier exchange while
 * that is still valid).  One process per rank; rank d's window is [capacity_rows, H] bf16 in its own GPU's
 * memory.
 *
 *   moe_window_export   describes a window of THIS process for the other ranks: an inter-process handle of
 *                       the allocation that holds it, the window's offset inside that allocation, the device,
 *                       and a generation number chosen by the exporter, which must change whenever the rank
 *                       exports a different window.  The result is plain bytes; the caller sends it to the
 *                       other ranks over whatever channel it has (the binding uses the process group).
 *   moe_peers_open      the address handshake: takes the R handles (entry my_rank is ignored; my_window is used
 *                       for it), maps every other rank's window into this process (peer access over NVLink /
 *                       PCIe is enabled by the mapping), and installs the R addresses and generations as the
 *                       context's address table.  Mappings of an earlier handshake are released first.
 *                       Synchronises `stream` before it releases or installs anything.  The handles must come
 *                       from OTHER processes (a process cannot map its own export); windows that live in this
 *                       process are installed with moe_peers_set.
 *   moe_peers_set       installs addresses the caller already has (separate allocations of one process, a
 *                       symmetric-memory mapping, an earlier handshake of its own) without mapping anything:
 *                       window_bases HOST [R] of DEVICE pointers, generations HOST [R] or NULL (all zero);
 *                       flags: MOE_WINDOW_* bits saying what follows the rows of EVERY window.
 *   moe_peers_check     the cached-address test: MOE_OK if a table is installed and its generations equal
 *                       `generations` (HOST [R], what the ranks announced for this call -- the binding sends each
 *                       rank's generation along with its count row, so the test costs no exchange of its own);
 *                       MOE_ERR_STALE_PEERS otherwise.
 *   moe_dispatch_cached / moe_combine_cached / moe_dispatch_quant_cached
 *                       as moe_dispatch_peers / moe_combine_peers / moe_dispatch_quant_peers with the installed
 *                       table and its capacity (the quantised forms need windows exported with MOE_WINDOW_QUANT
 *                       or MOE_WINDOW_QUANT_GROUP: codes and scales land in the parts of every rank's allocation
 *                       that flag reserves).
 *                       `generations` as in moe_peers_check (NULL: no test); with a stale or missing table they
 *                       return MOE_ERR_STALE_PEERS and enqueue nothing -- no stale address is ever dereferenced.
 *   moe_peers_close     synchronises `stream`, releases the mappings of moe_peers_open and forgets the table
 *                       (also done by moe_destroy).
 * Only this library's kernels touch the mapped windows: rows are stored to them with plain (non-multicast)
 * bulk copies and read from them with ordinary loads.  The library still waits for no peer: the caller orders
 * the phases (all ranks' dispatches complete before any expert reads; all experts complete before combine). */
typedef struct {
  unsigned char ipc[64]; /* inter-process memory handle of the allocation that holds the window */
  int64_t offset;        /* first byte of the window inside that allocation                    */
  int64_t bytes;         /* size of the window                                                 */
  int32_t device;        /* device ordinal of the exporter                                     */
  int32_t generation;    /* exporter's window generation                                       */
  int32_t flags;         /* MOE_WINDOW_*: what follows the rows inside the exported range      */
  int32_t reserved;
} moe_window_handle_t;
/* What a window allocation holds behind its [capacity_rows, H] bf16 rows (each part starts on a 256-byte boundary,
 * in this order; moe_window_bytes gives the total): */
#define MOE_WINDOW_STATE 1 /* the state region of the device-side phase order (moe_signal_peers), zeroed once   */
#define MOE_WINDOW_QUANT 2 /* the e4m3 code window [capacity_rows, H] uint8 and the scale tensor [capacity_rows]
                              fp32 of the row-wise quantised dispatch (moe_dispatch_quant_cached)               */
#define MOE_WINDOW_QUANT_GROUP 4 /* the code window and the scale tensor [capacity_rows, H / 128] fp32 of the
                              group-wise quantised dispatch (moe_dispatch_quant_group_cached); not together with
                              MOE_WINDOW_QUANT, and H % 128 == 0                                                */
#define MOE_WINDOW_COUNTS 8 /* the mailbox of the count exchange (moe_push_counts), directly behind the state region:
                              only together with MOE_WINDOW_STATE; zeroed once with it                        */
moe_status_t moe_window_export(const void* window /*DEVICE*/, int64_t bytes, int32_t generation, int32_t flags,
                               moe_window_handle_t* out /*HOST*/);
moe_status_t moe_peers_open(moe_ctx_t* ctx, const moe_window_handle_t* handles /*HOST [R]*/, int32_t my_rank,
                            void* my_window /*DEVICE*/, int64_t capacity_rows, void* stream);
moe_status_t moe_peers_set(moe_ctx_t* ctx, const void* const* window_bases /*HOST [R]*/,
                           const int32_t* generations /*HOST [R] or NULL*/, int32_t my_rank, int64_t capacity_rows,
                           int32_t flags, void* stream);
moe_status_t moe_peers_check(const moe_ctx_t* ctx, const int32_t* generations /*HOST [R]*/);
moe_status_t moe_dispatch_cached(moe_ctx_t* ctx, const void* x /*DEVICE*/, const int32_t* generations /*HOST or NULL*/,
                                 void* stream);
moe_status_t moe_combine_cached(moe_ctx_t* ctx, const int32_t* generations /*HOST or NULL*/,
                                const float* topk_w /*DEVICE*/, void* y /*DEVICE*/, void* stream);
moe_status_t moe_dispatch_quant_cached(moe_ctx_t* ctx, const void* x /*DEVICE*/,
                                       const int32_t* generations /*HOST or NULL*/, void* stream);
/* moe_dispatch_quant_group through the installed table: windows exported with MOE_WINDOW_QUANT_GROUP. */
moe_status_t moe_dispatch_quant_group_cached(moe_ctx_t* ctx, const void* x /*DEVICE*/,
                                             const int32_t* generations /*HOST or NULL*/, int32_t group_size,
                                             void* stream);
moe_status_t moe_peers_close(moe_ctx_t* ctx, void* stream);

/* Synchronisation metadata in the pooled memory (Section 3.2: every rank's slice carries communicator state
 * beside its payload; Section 5.4: status flags and wait symbols order producers and consumers across ranks).
 * A window allocation may be followed by a state region of moe_state_bytes(R) bytes -- allocate
 * moe_window_bytes(shape, capacity_rows, MOE_WINDOW_STATE), zero the state region once, export with that flag --
 * which the handshake maps together with the rows (every rank must export the same flags).  It holds
 * MOE_SYNC_SLOTS arrays of R 32-bit epochs.
 *   moe_signal_peers  enqueues, behind everything already on `stream`, a store of `epoch` into entry
 *                     [slot][my_rank] of EVERY rank's state region (release, system scope): "what I enqueued
 *                     before this -- my rows in your window, my experts' outputs -- is complete".
 *   moe_wait_peers    enqueues a kernel that waits until entries [slot][0..R-1] of THIS rank's own state region
 *                     have all reached `epoch` (acquire, system scope); whatever is enqueued behind it sees
 *                     what the signalling ranks wrote before their signals.  The wait is bounded (2 s, or the
 *                     MOE_OPT_TEST_STARVE_WAIT_MS value): when it runs out the status word becomes
 *                     MOE_ERR_TIMEOUT, the kernel ends normally and later calls write nothing until
 *                     moe_status() has reported it.
 * Epochs must grow from call to call (compared as signed differences, so they may wrap).  A layer step uses
 * three slots: rows dispatched (before the experts read their window), expert outputs ready (before combine
 * reads), combine done (before the next step's dispatch overwrites a window).  With these no host
 * synchronisation is needed between the phases.  MOE_ERR_STALE_PEERS if no table with state is installed.
 * NOTE: a wait kernel occupies its GPU until the signals arrive, so the ranks must run on different GPUs (or the
 * caller must know that the signals were sent before the wait is enqueued). */
#define MOE_SYNC_SLOTS 4
/* Count exchange through the pooled memory (Section 5.2, Notify: count metadata is the only thing the ranks exchange
 * before payload moves; here it moves by the library's own peer stores instead of a collective of the caller's).
 * Windows exported with MOE_WINDOW_STATE | MOE_WINDOW_COUNTS carry, behind the arrival flags, a mailbox of two
 * buffers of [R][E] counts and [R] epoch words, zeroed once together with the state region.
 *   moe_push_counts   after moe_layout: stores this rank's row of counts into entry [my_rank] of EVERY rank's
 *                     mailbox (buffer epoch & 1) and publishes it with the epoch word (release, system scope).
 *                     Waits for nobody.
 *   moe_notify_peers  moe_notify from this rank's own mailbox: enqueues a kernel that waits until all R epoch words
 *                     of buffer epoch & 1 have reached `epoch` (acquire, system scope; bounded like moe_wait_peers:
 *                     MOE_ERR_TIMEOUT in the status word, a normal end, and no plan once moe_status has reported
 *                     it) and then builds the large offsets and receive counts; the context is then planned.
 * Epochs of successive exchanges must grow by one (the two buffers alternate); a rank may run one exchange ahead
 * of the slowest rank, which the phase order of a layer step guarantees (nobody starts step e + 2 before every
 * rank has combined step e + 1, hence consumed the counts of step e).  The NOTE on moe_wait_peers applies:
 * with several ranks on one GPU every rank's push must have been enqueued before any rank's notify.
 * MOE_ERR_STALE_PEERS without an installed table whose windows have the mailbox; MOE_ERR_NOT_PLANNED before
 * moe_layout.  (No counterpart call in the paper: its Notify kernel does both halves.) */
moe_status_t moe_push_counts(moe_ctx_t* ctx, uint32_t epoch, void* stream);
/* moe_layout followed by moe_push_counts in one call (my_rank must be the rank of the installed table): for batches
 * the single-launch planner takes (at most 4096 branches on this rank) and up to 16 ranks the one CTA that lays the
 * tokens out also sends the row, straight from its shared memory -- a launch less in front of every multi-rank step; larger batches
 * enqueue the two calls one behind the other.  Same results and errors as the two calls. */
moe_status_t moe_layout_push(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx /*DEVICE [T_local,K]*/,
                             int32_t T_local, int32_t my_rank, uint32_t epoch, void* stream);
moe_status_t moe_notify_peers(moe_ctx_t* ctx, uint32_t epoch, void* stream);
size_t moe_state_bytes(int32_t R);
size_t moe_window_bytes(const moe_shape_t* shape /*HOST*/, int64_t capacity_rows, int32_t flags);
moe_status_t moe_signal_peers(moe_ctx_t* ctx, int32_t slot, uint32_t epoch, void* stream);
moe_status_t moe_wait_peers(moe_ctx_t* ctx, int32_t slot, uint32_t epoch, void* stream);

/* Materialises slot(t,j) into caller memory (parity checks, expert-side
 * consumers).  slots DEVICE [T,K] int32; needs R * capacity_rows < 2^31. */
moe_status_t moe_slots(moe_ctx_t* ctx, int64_t capacity_rows, int32_t* slots /*DEVICE*/, void* stream);

/* Row range of every expert in the window allocation, for the expert side (Section 5.2, Expert
 * computation: the FFNs consume the windows in place, with no further reordering, so the rows of one
 * expert are one contiguous run -- exactly a grouped-GEMM problem list).  Works under both schedules.
 *   row_start  DEVICE [E] int64   first window row of expert e ( = dst(e) * capacity_rows + o[e, 0] )
 *   row_count  DEVICE [E] int32   rows received by expert e */
moe_status_t moe_expert_ranges(moe_ctx_t* ctx, int64_t capacity_rows, int64_t* row_start /*DEVICE*/,
                               int32_t* row_count /*DEVICE*/, void* stream);

/* The same runs cut into tiles of at most tile_rows rows, in window order (rank, expert, position in the
 * run): the work list of a grouped GEMM that reads the windows in place.  (Consumer-side convenience, no
 * counterpart in the paper.)  With MOE_OPT_EXPERT_ALIGN equal to tile_rows every tile also starts on a
 * multiple of tile_rows inside its window.
 *   tile_expert DEVICE [max_tiles] int32   expert of tile k
 *   tile_row    DEVICE [max_tiles] int64   first window row of tile k
 *   tile_valid  DEVICE [max_tiles] int32   rows of tile k that hold tokens (only an expert's last tile is short)
 *   n_tiles     DEVICE [1] int32           number of tiles there are = sum over experts of ceil(n_exp / tile_rows);
 *                                          entries beyond max_tiles are not written
 * An upper bound for max_tiles that needs no device read: T*K / tile_rows + E. */
moe_status_t moe_expert_tiles(moe_ctx_t* ctx, int64_t capacity_rows, int32_t tile_rows, int64_t max_tiles,
                              int32_t* tile_expert /*DEVICE*/, int64_t* tile_row /*DEVICE*/,
                              int32_t* tile_valid /*DEVICE*/, int32_t* n_tiles /*DEVICE*/, void* stream);

/* One whole layer call from HOST buffers, enqueued on `stream` (no counterpart in the paper, which starts
 * and ends in device memory; this entry point exists so that an end-to-end number including the
 * host<->device copies can be measured through the C ABI):
 * host->device copies of topk_idx, topk_w; plan; then, in sixteen token chunks, host->device copy
 * of the chunk of x (upload stream), dispatch and combine reading the dispatched windows (identity
 * experts; caller's stream), and the device->host copy of the chunk of y (download stream), so both
 * copy directions and the kernels overlap.  The two extra streams belong to the context and are
 * created on first use.  `stream` finishes only after the last download.
 * The *_dev arguments are caller-owned DEVICE staging buffers of the shapes
 * given above.  Pass pinned host memory for the copies to be asynchronous.
 * rank_tok_start as in moe_plan.  Call moe_status() to wait for the result. */
moe_status_t moe_forward_host(moe_ctx_t* ctx, moe_schedule_t schedule, int32_t T,
                              const int32_t* rank_tok_start /*HOST*/,
                              const void* x_host, const int32_t* topk_idx_host, const float* topk_w_host,
                              void* x_dev, int32_t* topk_idx_dev, float* topk_w_dev,
                              void* windows_dev, int64_t capacity_rows, void* y_dev,
                              void* y_host, void* stream);

/* Tuning knobs of a context (no counterpart in the paper; tests use them to reach every kernel, defaults
 * are the measured best).
 *   MOE_OPT_DISPATCH_PATH  which dispatch kernel runs: AUTO (currently the bulk-copy kernel),
 *                          REGISTERS (16-byte ld/st through registers, K-specialised), or
 *                          BULK (cp.async.bulk through shared-memory stages).  Same result.
 *   MOE_OPT_GRANULE        512-byte units per work item of dispatch/combine; 0 = chosen from the
 *                          job size.  Any value gives the same result.
 *   MOE_OPT_TEST_STARVE_WAIT_MS  failure-path test hook, 0 = off.  With value v > 0 the bulk-copy
 *                          dispatch lets ONE warp wait for 16 bytes that are never sent and bounds
 *                          every device-side wait by v milliseconds: that warp gives up, the status
 *                          word becomes MOE_ERR_TIMEOUT, the kernel ends normally (no trap, nothing
 *                          left in flight) and the windows are incomplete.  Normal bound: 2 s.
 *   MOE_OPT_OVERLAP        1 (default): kernels that one call enqueues back to back are chained by programmatic
 *                          stream serialization -- moe_plan_dispatch starts its dispatch kernel while the
 *                          planner runs, the planner's own kernels and the planner behind the gate kernel
 *                          (moe_gate_plan) are scheduled while the kernel in front still runs -- and each
 *                          waits for the kernel in front before it reads anything that kernel writes.
 *                          0: every kernel starts after the previous one has ended.  Same result either way.
 *   MOE_OPT_EXPERT_ALIGN   A in [1, 4096], default 1 (the packed layout of Section 5.2).  With A > 1 later
 *                          plans pad the run of every expert to a whole number of A-row groups, so that
 *                          every expert's first row is a multiple of A inside its window and a grouped
 *                          GEMM can read the window in place in tiles of A rows without two experts in
 *                          one tile.  (No counterpart in the paper; an extension for the consumer of the
 *                          windows.)  n_exp stays the true count; large_off includes the padding of
 *                          earlier experts; n_recv[d] becomes the sum over the experts of rank d of
 *                          ceil(n_exp[e] / A) * A, which is what capacity_rows is checked against.
 *                          Padding rows are never written by dispatch nor read by combine.  Setting the
 *                          option invalidates the current plan.
 *   MOE_OPT_CLUSTER_PLAN   1 (default): the single-launch planner of small batches (at most 4096 branches
 *                          per source rank) runs its R CTAs as one thread-block cluster when R is 2, 4, 8 or
 *                          16 and the device can co-schedule them: the count rows are exchanged through
 *                          distributed shared memory and every CTA builds its own window's offsets.
 *                          0: the last CTA to finish builds all offsets from the matrix in global memory.
 *                          Same result.
 *   MOE_OPT_SLOT_REUSE     1 (default): a dispatch over the whole batch (any form, not the *_range calls) also
 *                          records every branch's window row (the sum of Section 5.2's two offsets and the
 *                          window start) in the workspace, and a combine of the same plan with the same
 *                          capacity_rows reads that row back instead of resolving routing index -> large
 *                          offset again: one dependent load less before its first payload loads.  The record
 *                          is dropped by every new plan, by MOE_OPT_EXPERT_ALIGN and by a moe_status that
 *                          reports an error; a recorded row outside [0, R * capacity_rows) is never used as
 *                          an address (the branch is skipped and the status becomes MOE_ERR_NOT_PLANNED).
 *                          It assumes that the kernels run in the order of the calls (calls recorded into
 *                          a graph count from when the graph runs).  0: combine always resolves the branch
 *                          from the plan.  Same result. */
typedef enum {
  MOE_OPT_DISPATCH_PATH = 0,
  MOE_OPT_GRANULE = 1,
  MOE_OPT_TEST_STARVE_WAIT_MS = 2,
  MOE_OPT_OVERLAP = 3,
  MOE_OPT_EXPERT_ALIGN = 4,
  MOE_OPT_CLUSTER_PLAN = 5,
  MOE_OPT_SLOT_REUSE = 6
} moe_option_t;
enum { MOE_DISPATCH_AUTO = 0, MOE_DISPATCH_REGISTERS = 1, MOE_DISPATCH_BULK = 2 };
moe_status_t moe_set_option(moe_ctx_t* ctx, moe_option_t option, int64_t value);

/* Window slots straight from the routing indexes, for callers that cannot give the library a
 * workspace.  (No counterpart in the paper: this is a packaging convenience of this library.)
 * Who needs it: code that runs inside an engine which claimed all device memory for its own pool
 * at start-up and offers no allocation hook, and decode loops in which nothing may allocate once
 * serving has begun because a device allocation can stall every stream.  The planning scratch is
 * a fixed array inside the library image (about 1.2 MB, resident on every GPU that loads the
 * library until the process exits); this call allocates and frees nothing.
 *   topk_idx        DEVICE [T,K] int32          rank_tok_start  HOST [R+1] or NULL, as in moe_plan
 *   slots           DEVICE [T,K] int32, out     slot(t,j) as moe_plan(DECODE) + moe_slots gives it
 *   n_recv          DEVICE [R] int32, out       rows received per window
 *   status          DEVICE [1] int32, out       0, MOE_ERR_BAD_INDEX (some index outside [0, E)) or
 *                                               MOE_ERR_CAPACITY (some n_recv[d] > capacity_rows); with
 *                                               either error NO slot is written: `slots` keeps what it held
 * Limits: T*K <= 65536, E <= 512, R <= 64, K <= MOE_MAX_K, R*capacity_rows < 2^31; larger problems
 * are rejected with MOE_ERR_INVALID_ARG and a message on stderr -- use moe_plan with a workspace.
 * The first call on each device looks up the array's device address; make that call with the
 * device current and before any stream capture begins.  Host threads may make that first call at
 * the same time (the address is kept in an atomic; every thread finds the same one).  All calls on one device share the array
 * (it keeps the previous call's contents; the words that must start at zero are cleared on the
 * stream each time), so two calls whose kernels may overlap on the GPU -- different streams with
 * no ordering between them -- race; order them on one stream or with events. */
moe_status_t moe_slots_noalloc(const int32_t* topk_idx /*DEVICE*/, int32_t T, int32_t K, int32_t E, int32_t R,
                               const int32_t* rank_tok_start /*HOST*/, int64_t capacity_rows,
                               int32_t* slots /*DEVICE*/, int32_t* n_recv /*DEVICE*/, int32_t* status /*DEVICE*/,
                               void* stream);

/* Synchronises `stream`, then returns and clears the device status word
 * (first device-detected error since the last call, or MOE_OK).  Reporting MOE_ERR_BAD_INDEX also
 * discards the context's plan (see moe_plan). */
moe_status_t moe_status(moe_ctx_t* ctx, void* stream);

const char* moe_status_string(moe_status_t status);

/* Number of kernel launches this context has enqueued so far (for benchmarks; no counterpart in the paper). */
int64_t moe_launch_count(const moe_ctx_t* ctx);

#ifdef __cplusplus
}
#endif
#endif
