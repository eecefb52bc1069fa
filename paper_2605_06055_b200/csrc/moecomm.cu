// libmoecomm: host side of the C ABI declared in include/moecomm.h.
// Argument validation, workspace layout, launch configuration.  Every step of
// the path runs in the kernels of plan_kernels.cuh (planning), gate_kernels.cuh
// (top-k gate), bulk_kernels.cuh / quant_kernels.cuh (bulk-copy dispatch, plain
// and quantised) and row_kernels.cuh (register-path dispatch, combine, slots).

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"
#include "plan_kernels.cuh"
#include "gate_kernels.cuh"
#include "row_kernels.cuh"
#include "bulk_kernels.cuh"
#include "quant_kernels.cuh"

using namespace moe;

struct moe_ctx {
  moe_shape_t shape;
  int device;
  int num_sms;
  char* ws;
  size_t ws_bytes;
  // workspace views (device)
  Control* ctl;
  int32_t *M, *c_rank, *o, *n_exp, *n_recv, *s, *tile_rank, *tile_hist;
  // plan state (host)
  bool planned;
  bool layout_done;   // moe_layout has run; moe_notify may complete the plan
  bool compact_plan;  // plan done in one launch by plan_rank_kernel: small offsets are final after moe_plan
  moe_schedule_t schedule;
  int32_t T;
  int32_t n_tiles;
  const int32_t* topk_idx;  // device; routing indexes of the current plan, read again by dispatch/combine
  RankMap map;
  int64_t launches;
  int32_t dispatch_path;    // MOE_OPT_DISPATCH_PATH
  int32_t granule_override; // MOE_OPT_GRANULE
  int32_t starve_wait_ms;   // MOE_OPT_TEST_STARVE_WAIT_MS
  int32_t overlap;          // MOE_OPT_OVERLAP
  int32_t cluster_plan;     // MOE_OPT_CLUSTER_PLAN
  int32_t slot_reuse;       // MOE_OPT_SLOT_REUSE
  bool plan_cluster_ok;     // the compact planner of this shape can be launched as one cluster of R CTAs
  bool scan_cluster_ok;     // the same for the scan kernel of the tile planner
  int32_t expert_align;     // MOE_OPT_EXPERT_ALIGN: every expert's run starts on a multiple of this many rows
  // Window rows of every branch as the last whole-batch dispatch of the current plan recorded them, and the capacity
  // they were computed for (-1: none); a combine with that capacity reads them instead of resolving the branch again.
  int32_t* slot_table;      // device, [T_max * K] (inside the workspace)
  int64_t slots_for_C;
  cudaStream_t out_stream;  // moe_forward_host: download and upload streams, created on first use (no device memory)
  cudaStream_t in_stream;
  cudaEvent_t fwd_events[2 * 16 + 2];
  // window address table of the expert-parallel group (moe_peers_open / moe_peers_set)
  const unsigned char** peer_table;   // device, [R] (inside the workspace)
  void* peer_ptr[MOE_MAX_R];          // host copy of the installed addresses
  void* peer_mapping[MOE_MAX_R];      // base of the inter-process mapping this context opened for rank d, or nullptr
  int32_t peer_gen[MOE_MAX_R];
  int64_t peer_capacity;
  bool peers_installed;
  bool peers_have_state;              // every installed window is followed by its state region
  bool peers_have_quant;              // ... and by a code window and a scale tensor (one scale per row)
  bool peers_have_quant_group;        // ... or by a code window and a tensor of group scales
  bool peers_have_counts;             // ... and the state region by the mailbox of the count exchange
  unsigned char** box_table;          // device, [R]: count mailbox of every rank
  bool notified_by_box;               // the current plan's offsets came from moe_notify_peers
  unsigned char** code_table;         // device, [R]: e4m3 code window of every rank
  float** scale_table;                // device, [R]: scale tensor of every rank
  int32_t my_rank;                    // this process's rank in the installed table
  unsigned char** state_table;        // device, [R]: state region of every rank (inside the workspace)
  // resident CTAs per SM of the row kernels this context has launched (occupancy calculator results)
  const void* occ_kernel[16];
  int occ_per_sm[16];
  int occ_n;
};

namespace {

// Plans (either schedule) whose ranks each hold at most this many branches take the single-launch planner.
constexpr int64_t RANK_PLAN_MAX_BRANCHES = 4096;
constexpr int RANK_PLAN_WIDE_MAX_E = 768;   // 32-warp CTAs while 33*E counters fit comfortably in shared memory

constexpr int FWD_CHUNKS = 16;  // token chunks of moe_forward_host's upload / compute / download pipeline
constexpr size_t ALIGN = 256;
size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

bool shape_valid(const moe_shape_t* s) {
  if (s == nullptr) return false;
  if (s->R < 1 || s->R > MOE_MAX_R || s->E < 1 || s->E > MOE_MAX_E || s->E % s->R != 0) return false;
  if (s->K < 1 || s->K > MOE_MAX_K || s->H < 8 || s->H % 8 != 0 || s->T_max < 0) return false;
  if ((int64_t)s->T_max * s->K >= (int64_t)1 << 31) return false;
  return true;
}

int64_t max_tiles(const moe_shape_t* s) {
  const int64_t B = (int64_t)s->T_max * s->K;
  const int64_t smallest_tile = ROUNDS_DECODE * PLAN_THREADS;
  return (B + smallest_tile - 1) / smallest_tile + s->R;  // every rank may end in a partial tile
}

struct Layout {
  size_t ctl, M, c_rank, o, n_exp, n_recv, peers, s, slot, tile_rank, tile_hist, total;
};

Layout layout_of(const moe_shape_t* s) {
  Layout L;
  size_t at = 0;
  auto take = [&](size_t bytes) {
    size_t here = at;
    at = align_up(at + bytes);
    return here;
  };
  const size_t B = (size_t)s->T_max * s->K;
  L.ctl = take(sizeof(Control));
  L.M = take(sizeof(int32_t) * s->R * s->E);
  L.c_rank = take(sizeof(int32_t) * s->R * s->R);
  L.o = take(sizeof(int32_t) * s->E * s->R);
  L.n_exp = take(sizeof(int32_t) * s->E);
  L.n_recv = take(sizeof(int32_t) * s->R);
  L.peers = take(sizeof(void*) * s->R * 5);   // window bases, state regions, code windows, scale tensors, count mailboxes
  L.s = take(sizeof(int32_t) * B);
  L.slot = take(sizeof(int32_t) * B);
  L.tile_rank = take(sizeof(int32_t) * B);
  L.tile_hist = take(sizeof(int32_t) * (size_t)max_tiles(s) * s->E);
  L.total = at;
  return L;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

moe_status_t launch_ok(moe_ctx* ctx, int n = 1) {
  ctx->launches += n;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

RowArgs row_args(const moe_ctx* ctx, int64_t C, bool dispatching) {
  RowArgs a;
  const moe_shape_t& sh = ctx->shape;
  a.topk_idx = nullptr;  // set by caller
  // DECODE: small offsets are finished on the fly (in-tile rank + tile base) by every consumer, so a
  // dispatch that aborted on the device can never leave a later call with half-written state; the
  // dispatch launch also records them, which is what moe_plan_view exposes as delta.
  const bool finish_delta = ctx->schedule == MOE_SCHED_DECODE && !ctx->compact_plan;
  a.small_off = finish_delta ? ctx->tile_rank : ctx->s;
  a.small_out = (finish_delta && dispatching) ? ctx->s : nullptr;
  a.slot_out = nullptr;
  a.slot_in = nullptr;
  a.tile_base = finish_delta ? ctx->tile_hist : nullptr;
  a.large_off = ctx->o;
  a.n_recv = ctx->n_recv;
  a.status = &ctx->ctl->status;
  a.C = C;
  a.T = ctx->T;
  a.K = sh.K;
  a.E = sh.E;
  a.R = sh.R;
  a.E_r = sh.E / sh.R;
  a.H16 = sh.H / 8;
  a.work = nullptr;
  a.work_done = nullptr;
  a.granule = 1;
  a.items_per_row = 0;
  a.n_items = 0;
  a.n_head = 0;
  a.head_rows = 0;
  a.tail_granule = 1;
  a.tail_items_per_row = 1;
  a.win_base = nullptr;
  a.scale_base = nullptr;
  a.prefetch_meta = 0;
  a.static_first = 0;
  a.pdl = 0;
  a.t_begin = 0;
  a.t_count = ctx->T;
  a.wait_limit_ms = ctx->starve_wait_ms > 0 ? ctx->starve_wait_ms : WAIT_LIMIT_MS_DEFAULT;
  a.test_starve = ctx->starve_wait_ms > 0;
  return a;
}

// Chooses the work-item size and hands the launch its counter.  An item is a whole row (at most
// max_granule units) whenever that still gives every warp an item -- whole rows measured best
// even at decode sizes -- and an even fraction of a row for tiny batches.
void set_work(moe_ctx* ctx, RowArgs& a, int64_t nwarps, int max_granule, bool may_split_tail = true) {
  const int upr = (a.H16 + 31) / 32;
  int64_t g = upr < max_granule ? upr : max_granule;
  int64_t pieces = (upr + g - 1) / g;
  const int64_t tokens = a.t_count;
  if (tokens * pieces < nwarps && tokens > 0) {
    // Fewer rows than warps: cut every row into as many pieces as still give every warp AT MOST one item.  An item
    // of this size costs a warp one chain of latencies whatever its length, so a second round for some warps is
    // what must be avoided: with one piece more (every warp at least one item) 16 tokens per rank left a third
    // of the dispatch warps two items, and the launch took 10.7 instead of 6.5 us from first to last instruction.
    pieces = nwarps / tokens;
    if (pieces > upr) pieces = upr;
    if (pieces < 1) pieces = 1;
    g = (upr + pieces - 1) / pieces;
  }
  if (ctx->granule_override > 0) g = ctx->granule_override;
  if (g > max_granule) g = max_granule;
  if (g > upr) g = upr;
  if (g < 1) g = 1;
  while ((tokens * ((upr + g - 1) / g)) > ((int64_t)1 << 30) && g < upr) ++g;   // n_items stays in int32
  a.granule = (int32_t)g;
  a.items_per_row = (int32_t)((upr + g - 1) / g);
  a.n_items = (int32_t)(tokens * a.items_per_row);
  a.n_head = a.n_items;
  a.head_rows = (int32_t)tokens;
  a.tail_granule = a.granule;
  a.tail_items_per_row = a.items_per_row;
  // Whole-row items: after the last full round (one row per warp) fewer rows than warps are left.  When
  // they would occupy at most a quarter of the warps, they are cut so that (nearly) every warp gets a
  // piece, but no finer than MIN_TAIL_UNITS.  Measured at H=7168, K=8, T=1280 (96 rows left over):
  // dispatch 38.5 -> 32.7 us, combine 45.0 -> 36.1 us.  Leftovers that fill more of the warps are not cut:
  // at T=2048 (272 rows left for 592 dispatch warps) halving them measured 1.3 us slower.
  constexpr int MIN_TAIL_UNITS = 4;
  const int64_t left = tokens % nwarps;
  if (may_split_tail && ctx->granule_override == 0 && a.items_per_row == 1 && tokens > nwarps && left > 0 &&
      4 * left <= nwarps && upr >= 2 * MIN_TAIL_UNITS) {
    int64_t pieces = nwarps / left;
    if (pieces > upr / MIN_TAIL_UNITS) pieces = upr / MIN_TAIL_UNITS;
    const int tg = (int)((upr + pieces - 1) / pieces);
    const int tipr = (upr + tg - 1) / tg;
    a.head_rows = (int32_t)(tokens - left);
    a.n_head = a.head_rows;
    a.tail_granule = tg;
    a.tail_items_per_row = tipr;
    a.n_items = (int32_t)(a.head_rows + left * tipr);
  }
  a.static_first = a.n_items <= 4 * nwarps ? 2 : 0;
  a.work = &ctx->ctl->work;
  a.work_done = &ctx->ctl->work_done;
}

// One persistent wave: as many CTAs as fit on the device at once (from the occupancy calculator),
// but no more warps than there are 512-byte units of work.
template <class Kernel>
int row_grid(moe_ctx* ctx, Kernel kernel, int64_t tokens) {
  int per_sm = 0;
  const void* key = reinterpret_cast<const void*>(kernel);
  for (int i = 0; i < ctx->occ_n; ++i)
    if (ctx->occ_kernel[i] == key) per_sm = ctx->occ_per_sm[i];
  if (per_sm == 0) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 256, 0) != cudaSuccess || per_sm < 1) {
      cudaGetLastError();
      per_sm = 1;
    }
    if (ctx->occ_n < 16) {
      ctx->occ_kernel[ctx->occ_n] = key;
      ctx->occ_per_sm[ctx->occ_n++] = per_sm;
    }
  }
  const int64_t units = tokens * ((ctx->shape.H / 8 + 31) / 32);
  const int64_t need = (units + 7) / 8;
  const int64_t cap = (int64_t)ctx->num_sms * per_sm;
  return (int)(need < cap ? (need < 1 ? 1 : need) : cap);
}

// Loads in flight per lane before the dependent stores / fma chain.  Few fat warps (one 256-thread
// CTA per SM with about 32 16-byte loads per lane) measured faster than many thin ones: every warp
// then streams long contiguous runs of each row, which HBM serves with far fewer page switches.
// More than 32 where it measured ahead: K=4 with 48 (a row of 10-12 units is then one phase of loads instead of
// a long and a short one: 179 -> 147 us at 32768 rows of 5760 bytes), K=9 and 10 with 36-40 (3-4 % at every size
// tried); 48 loads measured behind for K=1, 2, 8 and mixed for K=6.
constexpr int combine_unroll(int K) {
  return K >= 17 ? 1 : K >= 16 ? 2 : K >= 11 ? 3 : K >= 7 ? 4 : K >= 6 ? 5 : K == 5 ? 6 : K == 4 ? 12 : K == 3 ? 10 : 16;
}
constexpr int DISPATCH_UNROLL = 14;

template <int KT>
void launch_dispatch_regs(moe_ctx* ctx, const RowArgs& a, const uint4* x, uint4* win, cudaStream_t st) {
  auto kernel = dispatch_rows_kernel<KT, (KT > 0 ? DISPATCH_UNROLL : 1)>;
  const int grid = row_grid(ctx, kernel, a.t_count);
  RowArgs b = a;
  set_work(ctx, b, (int64_t)grid * 8, 1 << 20);
  kernel<<<grid, 256, 0, st>>>(x, win, b, ctx->map);
}

// Launch with optional attributes.  `pdl`: programmatic stream serialization, i.e. the kernel may start while
// the previous kernel of the stream is still running and orders itself with dependency_wait().
// `cluster` > 0: the grid runs as thread-block clusters of that many CTAs.
template <class... KArgs, class... Args>
void launch_kernel(void (*kernel)(KArgs...), int grid, int threads, int smem, cudaStream_t st, bool pdl, int cluster,
                   Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster > 0) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Dynamic shared memory to ask for when a one-CTA-per-SM kernel is launched behind a planner with programmatic
// stream serialization.  Its CTAs are placed while the planner's CTAs still hold their SMs, and CTAs that are small
// enough to fit two per SM then double up on some SMs and leave others without any for the whole launch: with
// the two-warp CTAs (86 KB) of a large job of 14 KB rows, plan + dispatch as one call took 870 us against 663 us
// as two calls at 32768 tokens (229 against 181 us at 8192, 79.7 against 72.4 us at 3072).  Asking for more
// than half an SM's shared memory keeps it at one CTA per SM (661, 179 and 71.6 us); the kernels take their layout
// from the warp count, not from the size of the allocation.
constexpr int SOLO_SMEM_BYTES = 120 * 1024;
int solo_smem(int smem, bool pdl) { return (pdl && smem < SOLO_SMEM_BYTES) ? SOLO_SMEM_BYTES : smem; }

// Bulk-copy path: one CTA per SM; each warp drives a ring of BULK_STAGES stages, and the CTA has as
// many warps (up to BULK_MAX_WARPS) as fit their rings into the shared-memory budget: 4 for 14 KB
// rows, 8 for rows of 8 KB or less (short rows need more requests in flight to cover the latency).
void launch_dispatch_bulk(moe_ctx* ctx, const RowArgs& a, const uint4* x, uint4* win, cudaStream_t st, bool pdl) {
  const int upr = (a.H16 + 31) / 32;
  const int g_max = upr < BULK_MAX_GRANULE ? upr : BULK_MAX_GRANULE;
  int warps = BULK_SMEM_BUDGET / (BULK_STAGES * (g_max * 512 + 8));
  if (warps > BULK_MAX_WARPS) warps = BULK_MAX_WARPS;
  if (warps < 1) warps = 1;
  const int grid = ctx->num_sms;
  constexpr int BULK_STREAMS_TARGET = 2400;
  // Large jobs: HBM serves the writes best when about 2400 destination rows are being written at once
  // (every warp writes K rows at a time), so fewer warps than fit are used when K is large -- but never so
  // few that less than 56 KB of loads are in flight per SM (two stages per warp are loading).  Measured at
  // 14 KB rows, K=8: 4 warps 661.5 us, 3 warps 659.5 us, 2 warps 656.4 us, 1 warp 816 us; at 8 KB rows, K=2:
  // 8 warps 252 us, 4 warps 272 us; at 4 KB rows, K=8: 8 warps 381 us, 2 warps 668 us.  Small jobs keep every
  // warp: there the number of rows in flight decides (decode step 102.7 us with 4 warps, 115 us with 2).
  // "Large" = four rows or more per warp (T=4096 at 14 KB rows: 95.2 -> 93.6 us; T=2048 is slower with the rule).
  if ((int64_t)a.t_count >= (int64_t)4 * grid * warps) {
    int want = (BULK_STREAMS_TARGET + grid * ctx->shape.K / 2) / (grid * ctx->shape.K);
    const int floor_warps = (56 * 1024 + 2 * g_max * 512 - 1) / (2 * g_max * 512);
    if (want < floor_warps) want = floor_warps;
    if (want < 1) want = 1;
    if (want < warps) warps = want;
  }
  RowArgs b = a;
  set_work(ctx, b, (int64_t)grid * warps, g_max);
  // Small and medium jobs: the fewest warps that still finish in the same number of rounds.  2048 rows of 8 KB are
  // 13.8 rows per SM: two rounds with eight warps, of which the second is only three quarters full, and two full
  // rounds with seven (32.1 -> 30.4 us flushed, 27.6 -> 25.6 us back to back; 1024 rows: 19.5 -> 18.4 us).
  if (b.static_first >= 2 && b.n_items > 0 && ctx->granule_override == 0) {
    const int64_t rounds = ((int64_t)b.n_items + (int64_t)grid * warps - 1) / ((int64_t)grid * warps);
    const int fewer = (int)(((int64_t)b.n_items + grid * rounds - 1) / (grid * rounds));
    if (fewer >= 1 && fewer < warps) {
      RowArgs c = a;
      set_work(ctx, c, (int64_t)grid * fewer, g_max);
      // (the cut of the rows changes with the warp count: taken only if the rounds come out at least nine tenths
      // full -- 1280 rows of 8 KB are better off with eight warps and their leftover rows cut finer)
      if ((int64_t)c.n_items <= rounds * grid * fewer && (int64_t)c.n_items * 10 >= rounds * grid * fewer * 9) {
        b = c;
        warps = fewer;
      }
    }
  }
  const int smem = solo_smem(warps * BULK_STAGES * (b.granule * 512 + 8), pdl);
  b.pdl = pdl;
  launch_kernel(dispatch_bulk_kernel, grid, warps * 32, smem, st, pdl, 0, reinterpret_cast<const unsigned char*>(x),
                reinterpret_cast<unsigned char*>(win), b, ctx->map);
}

template <int KT>
void launch_combine(moe_ctx* ctx, const RowArgs& a, const uint4* win, const float* w, uint4* y, cudaStream_t st) {
  // Jobs that read several times the L2 capacity take the L1-allocating loads (see ld_row).
  // Windows addressed through a table of bases (other GPUs' memory) are read with coherent loads.
  const bool peers = a.win_base != nullptr;
  const bool many_bytes = (int64_t)a.t_count * ctx->shape.K * ctx->shape.H * 2 >= ((int64_t)512 << 20);
  const bool large = !peers && many_bytes;
  auto kernel = peers ? (many_bytes ? combine_rows_kernel<KT, combine_unroll(KT > 0 ? KT : -KT), LD_PEER_L1>
                                    : combine_rows_kernel<KT, combine_unroll(KT > 0 ? KT : -KT), LD_PEER>)
                : large ? combine_rows_kernel<KT, combine_unroll(KT > 0 ? KT : -KT), LD_L1>
                        : combine_rows_kernel<KT, combine_unroll(KT > 0 ? KT : -KT), LD_STREAM>;
  const int grid = row_grid(ctx, kernel, a.t_count);
  RowArgs b = a;
  int warps = 8;
  set_work(ctx, b, (int64_t)grid * warps, 1 << 20, !large);   // the large-job form has no tail items
  // Small and medium jobs: the fewest warps that finish in the same number of (nearly full) rounds, as in
  // launch_dispatch_bulk.
  if (b.static_first >= 2 && b.n_items > 0 && ctx->granule_override == 0) {
    const int64_t rounds = ((int64_t)b.n_items + (int64_t)grid * warps - 1) / ((int64_t)grid * warps);
    const int fewer = (int)(((int64_t)b.n_items + grid * rounds - 1) / (grid * rounds));
    if (fewer >= 1 && fewer < warps) {
      RowArgs c = a;
      set_work(ctx, c, (int64_t)grid * fewer, 1 << 20, !large);
      if ((int64_t)c.n_items <= rounds * grid * fewer && (int64_t)c.n_items * 10 >= rounds * grid * fewer * 9) {
        b = c;
        warps = fewer;
      }
    }
  }
  // an item that is one or two batches of loads cannot hide its own metadata latency: prefetch it
  constexpr int unroll = combine_unroll(KT > 0 ? KT : -KT);
  b.prefetch_meta = (b.granule + unroll - 1) / unroll <= 2;
  kernel<<<grid, warps * 32, 0, st>>>(win, w, y, b, ctx->map);
}

}  // namespace

extern "C" {

size_t moe_workspace_bytes(const moe_shape_t* shape) {
  if (!shape_valid(shape)) return 0;
  return layout_of(shape).total;
}

moe_status_t moe_create(const moe_shape_t* shape, void* workspace, size_t workspace_bytes, moe_ctx_t** out) {
  if (out == nullptr) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  if (!shape_valid(shape) || workspace == nullptr) return MOE_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % ALIGN != 0) return MOE_ERR_INVALID_ARG;
  const Layout L = layout_of(shape);
  if (workspace_bytes < L.total) return MOE_ERR_INVALID_ARG;

  moe_ctx* ctx = new (std::nothrow) moe_ctx();
  if (ctx == nullptr) return MOE_ERR_CUDA;
  ctx->shape = *shape;
  if (cudaGetDevice(&ctx->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess) {
    delete ctx;
    return MOE_ERR_CUDA;
  }
  ctx->ws = static_cast<char*>(workspace);
  ctx->ws_bytes = workspace_bytes;
  ctx->ctl = reinterpret_cast<Control*>(ctx->ws + L.ctl);
  ctx->M = reinterpret_cast<int32_t*>(ctx->ws + L.M);
  ctx->c_rank = reinterpret_cast<int32_t*>(ctx->ws + L.c_rank);
  ctx->o = reinterpret_cast<int32_t*>(ctx->ws + L.o);
  ctx->n_exp = reinterpret_cast<int32_t*>(ctx->ws + L.n_exp);
  ctx->n_recv = reinterpret_cast<int32_t*>(ctx->ws + L.n_recv);
  ctx->peer_table = reinterpret_cast<const unsigned char**>(ctx->ws + L.peers);
  ctx->state_table = reinterpret_cast<unsigned char**>(ctx->ws + L.peers) + shape->R;
  ctx->peers_installed = false;
  ctx->code_table = ctx->state_table + shape->R;
  ctx->scale_table = reinterpret_cast<float**>(ctx->code_table + shape->R);
  ctx->box_table = ctx->code_table + 2 * shape->R;
  ctx->peers_have_counts = false;
  ctx->notified_by_box = false;
  ctx->peers_have_state = false;
  ctx->peers_have_quant = false;
  ctx->peers_have_quant_group = false;
  ctx->my_rank = 0;
  ctx->peer_capacity = 0;
  for (int d = 0; d < MOE_MAX_R; ++d) {
    ctx->peer_ptr[d] = nullptr;
    ctx->peer_mapping[d] = nullptr;
    ctx->peer_gen[d] = 0;
  }
  ctx->s = reinterpret_cast<int32_t*>(ctx->ws + L.s);
  ctx->slot_table = reinterpret_cast<int32_t*>(ctx->ws + L.slot);
  ctx->slots_for_C = -1;
  ctx->tile_rank = reinterpret_cast<int32_t*>(ctx->ws + L.tile_rank);
  ctx->tile_hist = reinterpret_cast<int32_t*>(ctx->ws + L.tile_hist);
  ctx->planned = false;
  ctx->slots_for_C = -1;
  ctx->layout_done = false;
  ctx->compact_plan = false;
  ctx->launches = 0;
  ctx->topk_idx = nullptr;
  ctx->dispatch_path = MOE_DISPATCH_AUTO;
  ctx->granule_override = 0;
  ctx->starve_wait_ms = 0;
  ctx->overlap = 1;
  ctx->cluster_plan = 1;
  ctx->slot_reuse = 1;
  ctx->plan_cluster_ok = false;
  ctx->scan_cluster_ok = false;
  ctx->expert_align = 1;
  ctx->out_stream = nullptr;
  ctx->in_stream = nullptr;
  ctx->occ_n = 0;

  // Kernels whose dynamic shared memory can exceed 48 KB opt in to the device maximum.  The attribute
  // belongs to the kernel, not to a context, so it is always set to the same (largest) value: contexts
  // of different shapes can then be created and used in any order.
  bool ok = cudaMemset(ctx->ctl, 0, sizeof(Control)) == cudaSuccess;
  int optin = 0;
  ok = ok && cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device) == cudaSuccess;
  const int big = optin - 2048;   // leave room for the kernels' few static words
  auto opt_in = [&](auto kernel) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big) == cudaSuccess;
  };
  ok = ok && opt_in(dispatch_bulk_kernel) && opt_in(dispatch_quant_kernel<3, 32, true>) &&
       opt_in(dispatch_quant_kernel<3, 32, false>) &&
       opt_in(dispatch_quant_kernel<2, 0, false>) && opt_in(dispatch_quant_kernel<3, 0, false>) &&
       opt_in(dispatch_quant_kernel<2, 0, false, true>) && opt_in(dispatch_quant_kernel<3, 0, false, true>) &&
       opt_in(dispatch_quant_reg_kernel<16, true, true>) && opt_in(dispatch_quant_reg_kernel<16, false, true>) &&
       opt_in(dispatch_quant_reg_kernel<16, true, false>) && opt_in(dispatch_quant_reg_kernel<16, false, false>) &&
       opt_in(dispatch_quant_reg_kernel<32, true, true>) && opt_in(dispatch_quant_reg_kernel<32, false, true>) &&
       opt_in(dispatch_quant_reg_kernel<32, true, false>) && opt_in(dispatch_quant_reg_kernel<32, false, false>) &&
       opt_in(plan_rank_kernel<32>) &&
       opt_in(plan_rank_kernel<8>) && opt_in(plan_scan_kernel) && opt_in(notify_rank_kernel) && opt_in(notify_box_kernel) &&
       opt_in(plan_tile_kernel<ROUNDS_PREFILL>) && opt_in(plan_tile_kernel<ROUNDS_DECODE>) && opt_in(gate_topk_kernel<0, false>);
  // The shape must fit: per-warp expert counters of the planners, the Notify scratch.
  const int rank_smem =
      rank_plan_smem_ints(shape->E, shape->R, shape->E <= RANK_PLAN_WIDE_MAX_E ? 32 : 8) * (int)sizeof(int32_t);
  ok = ok && PLAN_WARPS * shape->E * (int)sizeof(int32_t) <= big && rank_smem <= big &&
       notify_smem_ints(shape->E, shape->R) * (int)sizeof(int32_t) <= big;
  if (!ok) {
    cudaGetLastError();
    delete ctx;
    return MOE_ERR_CUDA;
  }
  // Can the compact planner run as ONE cluster of R CTAs?  Sizes up to 8 are portable, 16 needs the opt-in.
  if (shape->R == 2 || shape->R == 4 || shape->R == 8 || shape->R == 16) {
    const bool wide = shape->E <= RANK_PLAN_WIDE_MAX_E;
    const int smem = rank_smem + cluster_notify_smem_ints(shape->E, shape->R) * (int)sizeof(int32_t);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)shape->R);
    cfg.blockDim = dim3((unsigned)((wide ? 32 : 8) * 32));
    cfg.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)shape->R;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    bool fits = smem <= big;
    if (fits && shape->R > 8)
      fits = cudaFuncSetAttribute(plan_rank_kernel<32>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
             cudaFuncSetAttribute(plan_rank_kernel<8>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    if (fits)
      fits = (wide ? cudaOccupancyMaxActiveClusters(&clusters, plan_rank_kernel<32>, &cfg)
                   : cudaOccupancyMaxActiveClusters(&clusters, plan_rank_kernel<8>, &cfg)) == cudaSuccess && clusters >= 1;
    cudaGetLastError();
    ctx->plan_cluster_ok = fits;
    // the scan kernel of the tile planner, same cluster shape
    cfg.blockDim = dim3((unsigned)PLAN_THREADS);
    cfg.dynamicSmemBytes = (size_t)(shape->E + cluster_notify_smem_ints(shape->E, shape->R)) * sizeof(int32_t);
    clusters = 0;
    fits = (int)cfg.dynamicSmemBytes <= big;
    if (fits && shape->R > 8)
      fits = cudaFuncSetAttribute(plan_scan_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    if (fits) fits = cudaOccupancyMaxActiveClusters(&clusters, plan_scan_kernel, &cfg) == cudaSuccess && clusters >= 1;
    cudaGetLastError();
    ctx->scan_cluster_ok = fits;
  }
  *out = ctx;
  return MOE_OK;
}

moe_status_t moe_destroy(moe_ctx_t* ctx) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  for (int d = 0; d < ctx->shape.R; ++d)
    if (ctx->peer_mapping[d] != nullptr) {
      cudaIpcCloseMemHandle(ctx->peer_mapping[d]);
      cudaGetLastError();
    }
  if (ctx->out_stream != nullptr) {
    cudaStreamSynchronize(ctx->out_stream);
    cudaStreamSynchronize(ctx->in_stream);
    for (int i = 0; i < 2 * FWD_CHUNKS + 2; ++i) cudaEventDestroy(ctx->fwd_events[i]);
    cudaStreamDestroy(ctx->out_stream);
    cudaStreamDestroy(ctx->in_stream);
  }
  delete ctx;
  return MOE_OK;
}

}  // extern "C"

namespace {

constexpr int GATE_OCC_MAX_DEVICES = 64;

template <int VPT, bool PAIRS>
void launch_gate_kernel(const float* logits, int32_t T, int32_t E, int32_t K, int32_t* idx, float* w, int num_sms,
                        int dev, cudaStream_t st) {
  int warps = 8, smem = 0;
  if (VPT == 0) {   // rows cached in shared memory
    while (warps > 1 && warps * E * (int)sizeof(float) > 96 * 1024) warps >>= 1;
    smem = warps * E * (int)sizeof(float);
  }
  // Resident CTAs per SM.  The register forms' answer depends only on the device, so it is kept per device in
  // a table of atomics (any thread may fill an entry; every writer stores the same value); the shared-memory
  // form's answer depends on E and is asked every time.
  static std::atomic<int> cached[GATE_OCC_MAX_DEVICES];
  int per_sm = (VPT > 0 && dev >= 0 && dev < GATE_OCC_MAX_DEVICES) ? cached[dev].load(std::memory_order_relaxed) : 0;
  if (per_sm == 0) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gate_topk_kernel<VPT, PAIRS>, warps * 32, smem) !=
            cudaSuccess ||
        per_sm < 1) {
      cudaGetLastError();
      per_sm = 1;
    }
    if (VPT > 0 && dev >= 0 && dev < GATE_OCC_MAX_DEVICES) cached[dev].store(per_sm, std::memory_order_relaxed);
  }
  const int64_t units = PAIRS ? ((int64_t)T + 1) / 2 : (int64_t)T;
  int64_t grid = (units + warps - 1) / warps;
  if (grid > (int64_t)num_sms * per_sm) grid = (int64_t)num_sms * per_sm;   // one resident wave, grid-stride over tokens
  if (grid < 1) grid = 1;
  gate_topk_kernel<VPT, PAIRS><<<(int)grid, warps * 32, smem, st>>>(logits, T, E, K, idx, w);
}

template <int VPT>
void launch_gate_form(const float* logits, int32_t T, int32_t E, int32_t K, int32_t* idx, float* w, int num_sms,
                      int dev, cudaStream_t st) {
  // Two tokens per warp (they share the rank / softmax / store instructions) once that still leaves every SM a
  // full CTA of pairs; small batches keep one token per warp and so more warps.  3.0 against 2.7 us at T=2048,
  // 4.7 against 5.1 us at T=8192, 12.3 against 14.3 us at T=32768 (256 logits, top-8).
  // A pair needs at most 16 candidates per token, which from K = 12 on fails too often (both tokens are then
  // taken one by one after the attempt): 32768 tokens of 256 logits, K=11 16.2 against 18.0 us, K=12 19.6 against
  // 18.6, K=16 27.2 against 21.5.
  if constexpr (VPT >= 4) {
    if (K <= 11 && (int64_t)T / 2 >= (int64_t)num_sms * 8) {
      launch_gate_kernel<VPT, true>(logits, T, E, K, idx, w, num_sms, dev, st);
      return;
    }
  }
  launch_gate_kernel<VPT, false>(logits, T, E, K, idx, w, num_sms, dev, st);
}

void launch_gate(const float* logits, int32_t T, int32_t E, int32_t K, int32_t* idx, float* w, int num_sms,
                 int dev, cudaStream_t st) {
  if (E <= 32) launch_gate_form<1>(logits, T, E, K, idx, w, num_sms, dev, st);
  else if (E <= 64) launch_gate_form<2>(logits, T, E, K, idx, w, num_sms, dev, st);
  else if (E <= 128) launch_gate_form<4>(logits, T, E, K, idx, w, num_sms, dev, st);
  else if (E <= 256) launch_gate_form<8>(logits, T, E, K, idx, w, num_sms, dev, st);
  else if (E <= 512) launch_gate_form<16>(logits, T, E, K, idx, w, num_sms, dev, st);
  else if (E <= 1024) launch_gate_form<32>(logits, T, E, K, idx, w, num_sms, dev, st);
  else launch_gate_form<0>(logits, T, E, K, idx, w, num_sms, dev, st);
}

// Planning, optionally with the gate in front (logits != nullptr: topk_idx and topk_w are OUTPUTS).
// local_rank >= 0: only that rank owns tokens and only its local part is wanted (its small offsets and its row of
// M; moe_layout) -- one CTA instead of R and no Notify step.
moe_status_t plan_impl(moe_ctx* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T,
                       const int32_t* rank_tok_start, void* stream, const float* logits, int32_t* idx_out,
                       float* w_out, int32_t local_rank = -1, bool push = false, uint32_t epoch = 0,
                       bool* pushed = nullptr) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  const moe_shape_t& sh = ctx->shape;
  if (schedule != MOE_SCHED_PREFILL && schedule != MOE_SCHED_DECODE) return MOE_ERR_INVALID_ARG;
  if (T < 0 || T > sh.T_max) return MOE_ERR_INVALID_ARG;
  if (rank_tok_start == nullptr && T % sh.R != 0) return MOE_ERR_INVALID_ARG;
  if (rank_tok_start != nullptr) {
    if (rank_tok_start[0] != 0 || rank_tok_start[sh.R] != T) return MOE_ERR_INVALID_ARG;
    for (int r = 0; r < sh.R; ++r)
      if (rank_tok_start[r + 1] < rank_tok_start[r]) return MOE_ERR_INVALID_ARG;
  }
  ctx->planned = false;
  ctx->slots_for_C = -1;
  ctx->layout_done = false;
  ctx->notified_by_box = false;

  const int rounds = schedule == MOE_SCHED_PREFILL ? ROUNDS_PREFILL : ROUNDS_DECODE;
  const int tile_branches = rounds * PLAN_THREADS;
  RankMap& map = ctx->map;
  std::memset(&map, 0, sizeof(map));
  map.R = sh.R;
  map.uniform_tokens = (rank_tok_start == nullptr && T > 0) ? T / sh.R : 0;
  map.tile_shift = 0;
  while ((1 << map.tile_shift) < tile_branches) ++map.tile_shift;
  int32_t tiles = 0;
  for (int r = 0; r <= sh.R; ++r) {
    const int32_t tok = rank_tok_start != nullptr ? rank_tok_start[r] : (int32_t)((int64_t)T / sh.R * r);
    map.tok_start[r] = tok;
    map.tile_start[r] = tiles;
    if (r < sh.R) {
      const int32_t next = rank_tok_start != nullptr ? rank_tok_start[r + 1] : (int32_t)((int64_t)T / sh.R * (r + 1));
      const int64_t branches = (int64_t)(next - tok) * sh.K;
      tiles += (int32_t)((branches + tile_branches - 1) / tile_branches);
    }
  }
  ctx->n_tiles = tiles;
  ctx->T = T;
  ctx->schedule = schedule;
  ctx->topk_idx = topk_idx;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int tile_smem = PLAN_WARPS * sh.E * (int)sizeof(int32_t);
  const int scan_smem = notify_smem_ints(sh.E, sh.R) * (int)sizeof(int32_t);
  const int rank_smem =
      rank_plan_smem_ints(sh.E, sh.R, sh.E <= RANK_PLAN_WIDE_MAX_E ? 32 : 8) * (int)sizeof(int32_t);
  const int full = schedule == MOE_SCHED_PREFILL;
  int64_t max_rank_branches = 0;
  for (int r = 0; r < sh.R; ++r) {
    const int64_t br = (int64_t)(map.tok_start[r + 1] - map.tok_start[r]) * sh.K;
    if (br > max_rank_branches) max_rank_branches = br;
  }
  ctx->compact_plan = max_rank_branches <= RANK_PLAN_MAX_BRANCHES;
  const bool wide = sh.E <= RANK_PLAN_WIDE_MAX_E;
  bool split_notify = false;
  int n = 0;
  if (logits != nullptr) {   // gate first (its own launch, spread over all SMs), then plan from the indexes it wrote
    launch_gate(logits, T, sh.E, sh.K, idx_out, w_out, ctx->num_sms, ctx->device, st);
    ++n;
  }
  if (ctx->compact_plan) {
    // One CTA per source rank.  When the R CTAs can run as one thread-block cluster, the Notify step reads
    // the count rows from the CTAs' shared memory and every CTA builds its own window's offsets.
    const bool local = local_rank >= 0;
    const bool as_cluster = !local && ctx->cluster_plan && ctx->plan_cluster_ok;
    const int threads = (wide ? 32 : 8) * 32;
    const int smem = rank_smem + (as_cluster ? cluster_notify_smem_ints(sh.E, sh.R) * (int)sizeof(int32_t) : 0);
    // More ranks than a cluster holds: the last CTA alone would build E x R offsets (20 us at R = 64), so the
    // CTAs only count and a second launch builds every window's offsets side by side.
    split_notify = !local && !as_cluster && sh.R > 16;
    const int32_t mode = (local || split_notify) ? PLAN_LOCAL : as_cluster ? PLAN_CLUSTER : PLAN_TICKET;
    const int ctas = local ? 1 : sh.R;
    const int32_t first = local ? local_rank : 0;
    const bool behind_gate = logits != nullptr && ctx->overlap != 0;
    // moe_layout_push: the single CTA also sends its row (up to 16 ranks; beyond, the push kernel's CTAs of 16
    // destinations are ahead of one CTA storing R x E words: 12.7 against 12.6 us for the whole exchange at R = 64)
    unsigned char* const* box = (local && push && sh.R <= 16) ? ctx->box_table : nullptr;
    if (wide)
      launch_kernel(plan_rank_kernel<32>, ctas, threads, smem, st, behind_gate, as_cluster ? sh.R : 0, topk_idx, map, sh.K, sh.E,
                    (int32_t)full, ctx->expert_align, ctx->s, ctx->M, ctx->c_rank, ctx->o, ctx->n_exp, ctx->n_recv,
                    ctx->ctl, mode, first, box, epoch);
    else
      launch_kernel(plan_rank_kernel<8>, ctas, threads, smem, st, behind_gate, as_cluster ? sh.R : 0, topk_idx, map, sh.K, sh.E,
                    (int32_t)full, ctx->expert_align, ctx->s, ctx->M, ctx->c_rank, ctx->o, ctx->n_exp, ctx->n_recv,
                    ctx->ctl, mode, first, box, epoch);
    if (pushed != nullptr) *pushed = box != nullptr;
    ++n;
  } else {
    if (tiles > 0) {
      const bool behind_gate = logits != nullptr && ctx->overlap != 0;
      if (full)
        launch_kernel(plan_tile_kernel<ROUNDS_PREFILL>, tiles, PLAN_THREADS, tile_smem, st, behind_gate, 0, topk_idx, map,
                      sh.K, sh.E, ctx->tile_rank, ctx->tile_hist, &ctx->ctl->status);
      else
        launch_kernel(plan_tile_kernel<ROUNDS_DECODE>, tiles, PLAN_THREADS, tile_smem, st, behind_gate, 0, topk_idx, map,
                      sh.K, sh.E, ctx->tile_rank, ctx->tile_hist, &ctx->ctl->status);
      ++n;
    }
    // The three kernels are chained by programmatic stream serialization: each may be scheduled while the one
    // in front still runs and waits for it before touching its output, so launch latencies (and the finalize
    // kernel's index loads) overlap the kernel in front.  The scan kernel's R CTAs run as one cluster when
    // the device can co-schedule them (see cluster_notify).
    const bool chain = ctx->overlap != 0;
    const bool local = local_rank >= 0;
    const bool scan_cluster = !local && ctx->cluster_plan && ctx->scan_cluster_ok;
    split_notify = !local && !scan_cluster && sh.R > 16;
    const int scan_bytes =
        scan_cluster ? (sh.E + cluster_notify_smem_ints(sh.E, sh.R)) * (int)sizeof(int32_t) : scan_smem;
    launch_kernel(plan_scan_kernel, local ? 1 : sh.R, PLAN_THREADS, scan_bytes, st, chain && tiles > 0,
                  scan_cluster ? sh.R : 0, ctx->tile_hist, map, sh.E, (int32_t)full, ctx->expert_align, ctx->M,
                  ctx->c_rank, ctx->o, ctx->n_exp, ctx->n_recv, ctx->ctl,
                  (int32_t)((local || split_notify) ? PLAN_LOCAL : scan_cluster ? PLAN_CLUSTER : PLAN_TICKET),
                  (int32_t)(local ? local_rank : 0));
    ++n;
    if (full && tiles > 0) {
      launch_kernel(plan_finalize_kernel<ROUNDS_PREFILL>, tiles, PLAN_THREADS, 0, st, chain, 0, topk_idx, map, sh.K, sh.E,
                    ctx->tile_rank, ctx->tile_hist, ctx->s);
      ++n;
    }
  }
  if (split_notify) {
    notify_rank_kernel<<<sh.R, 256, cluster_notify_smem_ints(sh.E, sh.R) * (int)sizeof(int32_t), st>>>(
        ctx->M, sh.E, sh.R, (int32_t)full, ctx->expert_align, ctx->M, ctx->c_rank, ctx->o, ctx->n_exp, ctx->n_recv);
    ++n;
  }
  const moe_status_t rc = launch_ok(ctx, n);
  if (rc == MOE_OK) ctx->planned = true;
  return rc;
}

}  // namespace

extern "C" {

moe_status_t moe_plan(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T,
                      const int32_t* rank_tok_start, void* stream) {
  if (T > 0 && topk_idx == nullptr) return MOE_ERR_INVALID_ARG;
  return plan_impl(ctx, schedule, topk_idx, T, rank_tok_start, stream, nullptr, nullptr, nullptr);
}

moe_status_t moe_gate_plan(moe_ctx_t* ctx, moe_schedule_t schedule, const float* logits, int32_t T,
                           const int32_t* rank_tok_start, int32_t* topk_idx, float* topk_w, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (ctx->shape.K > ctx->shape.E) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (logits == nullptr || topk_idx == nullptr || topk_w == nullptr)) return MOE_ERR_INVALID_ARG;
  return plan_impl(ctx, schedule, topk_idx, T, rank_tok_start, stream, logits, topk_idx, topk_w);
}

moe_status_t moe_gate_topk(const float* logits, int32_t T, int32_t E, int32_t K, int32_t* topk_idx, float* topk_w,
                           void* stream) {
  if (T < 0 || E < 1 || E > MOE_MAX_E || K < 1 || K > MOE_MAX_K || K > E) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (logits == nullptr || topk_idx == nullptr || topk_w == nullptr)) return MOE_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (E > 1024) {   // the shared-memory form of the gate: opt in like moe_create does
    int optin = 0;
    if (cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaFuncSetAttribute(gate_topk_kernel<0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - 2048) != cudaSuccess)
      return MOE_ERR_CUDA;
  }
  if (T > 0) launch_gate(logits, T, E, K, topk_idx, topk_w, sms, dev, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status_t moe_plan_view(const moe_ctx_t* c, moe_plan_view_t* out) {
  if (c == nullptr || out == nullptr) return MOE_ERR_INVALID_ARG;
  if (!c->planned) return MOE_ERR_NOT_PLANNED;
  const bool full = c->schedule == MOE_SCHED_PREFILL;
  out->counts = full ? c->M : nullptr;
  out->c_rank = full ? c->c_rank : nullptr;
  out->small_off = c->s;
  out->large_off = c->o;
  out->n_exp = full ? c->n_exp : nullptr;
  out->n_recv = c->n_recv;
  out->rows = c->slots_for_C >= 0 ? c->slot_table : nullptr;
  out->rows_capacity = c->slots_for_C;
  return MOE_OK;
}

}  // extern "C"

namespace {

// A dispatch over the whole batch records every branch's window row for the combine that follows (rows are kept
// as 32-bit words: not for windows of 2^31 rows or more).
bool records_slots(const moe_ctx* ctx, const RowArgs& a) {
  return a.t_begin == 0 && a.t_count == ctx->T && ctx->T > 0 && (int64_t)ctx->shape.R * a.C < ((int64_t)1 << 31);
}

moe_status_t dispatch_impl(moe_ctx* ctx, const void* x, void* windows, const void* const* bases, int64_t capacity_rows,
                           void* stream, int32_t t_begin = 0, int32_t t_end = -1, bool behind_plan = false) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->planned) return MOE_ERR_NOT_PLANNED;
  if (capacity_rows < 0 || (ctx->T > 0 && (x == nullptr || (windows == nullptr && bases == nullptr))))
    return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(windows)) return MOE_ERR_INVALID_ARG;
  if (t_end < 0) t_end = ctx->T;
  if (t_begin < 0 || t_begin > t_end || t_end > ctx->T) return MOE_ERR_INVALID_ARG;
  RowArgs a = row_args(ctx, capacity_rows, true);
  a.win_base = reinterpret_cast<const unsigned char* const*>(bases);
  a.t_begin = t_begin;
  a.t_count = t_end - t_begin;
  a.topk_idx = ctx->topk_idx;
  const bool records = records_slots(ctx, a);
  if (records) a.slot_out = ctx->slot_table;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint4* xs = static_cast<const uint4*>(x);
  uint4* win = static_cast<uint4*>(windows);
  if (ctx->dispatch_path != MOE_DISPATCH_REGISTERS) {
    launch_dispatch_bulk(ctx, a, xs, win, st, behind_plan && ctx->overlap);
  } else {
    switch (ctx->shape.K) {
      case 1: launch_dispatch_regs<1>(ctx, a, xs, win, st); break;
      case 2: launch_dispatch_regs<2>(ctx, a, xs, win, st); break;
      case 4: launch_dispatch_regs<4>(ctx, a, xs, win, st); break;
      case 6: launch_dispatch_regs<6>(ctx, a, xs, win, st); break;
      case 8: launch_dispatch_regs<8>(ctx, a, xs, win, st); break;
      default: launch_dispatch_regs<0>(ctx, a, xs, win, st); break;
    }
  }
  const moe_status_t rc = launch_ok(ctx);
  if (records && rc == MOE_OK) ctx->slots_for_C = capacity_rows;
  return rc;
}

}  // namespace

extern "C" {

moe_status_t moe_dispatch(moe_ctx_t* ctx, const void* x, void* windows, int64_t capacity_rows, void* stream) {
  if (ctx != nullptr && ctx->T > 0 && windows == nullptr) return MOE_ERR_INVALID_ARG;
  return dispatch_impl(ctx, x, windows, nullptr, capacity_rows, stream);
}

moe_status_t moe_plan_dispatch(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T,
                               const int32_t* rank_tok_start, const void* x, void* windows, int64_t capacity_rows,
                               void* stream) {
  if (ctx == nullptr || (T > 0 && (topk_idx == nullptr || x == nullptr || windows == nullptr)))
    return MOE_ERR_INVALID_ARG;
  if (capacity_rows < 0 || !aligned16(x) || !aligned16(windows)) return MOE_ERR_INVALID_ARG;
  const moe_status_t rc = plan_impl(ctx, schedule, topk_idx, T, rank_tok_start, stream, nullptr, nullptr, nullptr);
  if (rc != MOE_OK) return rc;
  return dispatch_impl(ctx, x, windows, nullptr, capacity_rows, stream, 0, -1, true);
}

moe_status_t moe_gate_plan_dispatch(moe_ctx_t* ctx, moe_schedule_t schedule, const float* logits, int32_t T,
                                    const int32_t* rank_tok_start, int32_t* topk_idx, float* topk_w, const void* x,
                                    void* windows, int64_t capacity_rows, void* stream) {
  if (ctx == nullptr || ctx->shape.K > ctx->shape.E) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (logits == nullptr || topk_idx == nullptr || topk_w == nullptr || x == nullptr || windows == nullptr))
    return MOE_ERR_INVALID_ARG;
  if (capacity_rows < 0 || !aligned16(x) || !aligned16(windows)) return MOE_ERR_INVALID_ARG;
  const moe_status_t rc = plan_impl(ctx, schedule, topk_idx, T, rank_tok_start, stream, logits, topk_idx, topk_w);
  if (rc != MOE_OK) return rc;
  return dispatch_impl(ctx, x, windows, nullptr, capacity_rows, stream, 0, -1, true);
}

moe_status_t moe_dispatch_range(moe_ctx_t* ctx, const void* x, void* windows, int64_t capacity_rows, int32_t t_begin,
                                int32_t t_end, void* stream) {
  if (ctx != nullptr && ctx->T > 0 && windows == nullptr) return MOE_ERR_INVALID_ARG;
  if (t_end < 0) return MOE_ERR_INVALID_ARG;
  return dispatch_impl(ctx, x, windows, nullptr, capacity_rows, stream, t_begin, t_end);
}

moe_status_t moe_dispatch_peers(moe_ctx_t* ctx, const void* x, const void* const* window_bases, int64_t capacity_rows,
                                void* stream) {
  if (window_bases == nullptr) return MOE_ERR_INVALID_ARG;
  return dispatch_impl(ctx, x, nullptr, window_bases, capacity_rows, stream);
}

// group: 0 = one scale per row, QUANT_GROUP = one per 128 elements.
static bool quant_shape_ok(int H, int group) {
  if (H % 16 != 0 || H * 2 > QUANT_MAX_ROW_BYTES) return false;
  return group == 0 || (group == QUANT_GROUP && H % QUANT_GROUP == 0);
}

static moe_status_t dispatch_quant_impl(moe_ctx* ctx, const void* x, void* windows_q, float* scales,
                                        int64_t capacity_rows, void* stream, bool behind_plan,
                                        const void* const* q_bases = nullptr, float* const* s_bases = nullptr,
                                        int group = 0) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->planned) return MOE_ERR_NOT_PLANNED;
  const bool peers = q_bases != nullptr;   // one code window and one scale tensor per rank, addressed through tables
  const int H = ctx->shape.H;
  if (!quant_shape_ok(H, group)) return MOE_ERR_INVALID_ARG;
  const bool grouped = group != 0;
  const int sh_K = ctx->shape.K;
  if (capacity_rows < 0 || (peers && s_bases == nullptr)) return MOE_ERR_INVALID_ARG;
  if (ctx->T > 0 && (x == nullptr || (!peers && (windows_q == nullptr || scales == nullptr)))) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || (!peers && (!aligned16(windows_q) || (reinterpret_cast<uintptr_t>(scales) & 3u) != 0)))
    return MOE_ERR_INVALID_ARG;
  RowArgs a = row_args(ctx, capacity_rows, true);
  a.topk_idx = ctx->topk_idx;
  a.win_base = reinterpret_cast<const unsigned char* const*>(q_bases);
  a.scale_base = s_bases;
  const bool records = records_slots(ctx, a);
  if (records) a.slot_out = ctx->slot_table;
  auto launched = [&]() {
    const moe_status_t rc = launch_ok(ctx);
    if (records && rc == MOE_OK) ctx->slots_for_C = capacity_rows;
    return rc;
  };
  // One work item per token: the whole row is needed for its scale.
  const int upr = (a.H16 + 31) / 32;
  const int stage = (H * 2 + 127) / 128 * 128;
  const int grid = ctx->num_sms;
  // 16-byte chunks of a row per lane: rows of up to 16 (8 KB) or 32 (16 KB) are held in registers, longer ones
  // take the two-pass form; the 32-chunk form has registers for eight warps.
  const int cpl = upr <= 16 ? 16 : upr <= 32 ? 32 : 0;
  const int64_t rows_per_sm = ((int64_t)ctx->T + grid - 1) / grid;
  const bool pdl = behind_plan && ctx->overlap != 0;
  a.pdl = pdl;
  const bool whole_slabs = a.H16 % 32 == 0;   // every chunk of a row is valid for all lanes or for none
  const int32_t keep = ctx->granule_override;
  // The ring of whole-row stages: two or three stages per warp; the two-pass form also stages the row's group scales.
  const int ring_warps_max = cpl == 32 ? 8 : QUANT_MAX_WARPS;
  const int per_warp_extra = (grouped && cpl == 0) ? 2 * QUANT_MAX_GROUPS * (int)sizeof(float) : 0;   // scales, reciprocals
  auto ring_warps = [&](int stages) {
    int w = QUANT_SMEM_BUDGET / (stages * (stage + 8) + per_warp_extra);
    return w > ring_warps_max ? ring_warps_max : w;
  };
  // A large job: every warp of the two-stage ring would see eight rows or more.
  const bool large = ring_warps(3) >= 1 && (int64_t)ctx->T >= (int64_t)8 * grid * ring_warps(2);
  // Rows short enough for registers take the register kernel (a load buffer and a code buffer per warp, the group
  // scales and reciprocals behind the codes): more rows in flight per SM.  Only large row-wise jobs of rows beyond
  // 8 KB with five or more branches per token stay on the three-stage ring, which runs them at the copy rate with
  // five warps (32768 rows of 14 KB, K=8: 368 against 373 us); with fewer branches the job is read-dominated and the
  // register kernel's ten warps are ahead (K=1: 116 against 172 us, K=2: 150 against 182, K=3: 186 against 199).  Measured, register kernel against ring: decode shape 31.9 against 33.8 us row-wise and 33.8
  // against 44.1 us group-wise; 65536 rows of 4 KB 170 against 203 us; 65536 rows of 8 KB 179 against 176 us.
  // Warps per CTA: as many as fit, but for large jobs of short rows at most 9.  At 65536 rows of 8 KB ten or eleven
  // warps reach 169-172 us in one run and 237-240 us (the rate of six warps) in the next, and twelve or more are
  // always at 237-240: past about 2700 window rows being written at once HBM serves the writes badly (the bulk-copy
  // dispatch bounds its warps for the same reason), and where exactly that sets in changes from run to run.
  if (cpl == 16 || (cpl == 32 && (grouped || !large || sh_K < 5))) {
    const int sc_bytes = grouped ? ((H / QUANT_GROUP) * 4 + 15) / 16 * 16 : 0;
    const int per_warp = stage + (H + 2 * sc_bytes + 127) / 128 * 128 + 8;
    int warps = QUANT_SMEM_BUDGET / per_warp;
    const int cap = cpl == 32 ? QUANT_REG_WARPS_LONG : large ? QUANT_REG_WARPS_SHORT_LARGE_JOB : QUANT_REG_WARPS_SHORT;
    if (warps > cap) warps = cap;
    // the fewest warps that still finish in the same number of rounds (14 rows per SM: 7 warps, not 10)
    const int64_t rounds = rows_per_sm < 1 ? 1 : (rows_per_sm + warps - 1) / warps;
    warps = rows_per_sm < 1 ? 1 : (int)((rows_per_sm + rounds - 1) / rounds);
    ctx->granule_override = upr;
    set_work(ctx, a, (int64_t)grid * warps, upr, false);
    ctx->granule_override = keep;
    auto launch = [&](auto kernel) {
      launch_kernel(kernel, grid, warps * 32, solo_smem(warps * per_warp, pdl), static_cast<cudaStream_t>(stream), pdl, 0,
                    static_cast<const unsigned char*>(x), static_cast<unsigned char*>(windows_q), scales, a, ctx->map);
    };
    if (cpl == 16) {
      if (grouped) whole_slabs ? launch(dispatch_quant_reg_kernel<16, true, true>) : launch(dispatch_quant_reg_kernel<16, false, true>);
      else whole_slabs ? launch(dispatch_quant_reg_kernel<16, true, false>) : launch(dispatch_quant_reg_kernel<16, false, false>);
    } else {
      if (grouped) whole_slabs ? launch(dispatch_quant_reg_kernel<32, true, true>) : launch(dispatch_quant_reg_kernel<32, false, true>);
      else whole_slabs ? launch(dispatch_quant_reg_kernel<32, true, false>) : launch(dispatch_quant_reg_kernel<32, false, false>);
    }
    return launched();
  }
  const int stages = large ? 3 : 2;
  int warps = ring_warps(stages);
  if (warps < 1) return MOE_ERR_INVALID_ARG;
  if (warps > rows_per_sm) warps = rows_per_sm < 1 ? 1 : (int)rows_per_sm;   // no warps without a row
  ctx->granule_override = upr;
  set_work(ctx, a, (int64_t)grid * warps, upr, false);
  ctx->granule_override = keep;
  const int smem = solo_smem(warps * (stages * (stage + 8) + per_warp_extra), pdl);
  auto launch = [&](auto kernel) {
    launch_kernel(kernel, grid, warps * 32, smem, static_cast<cudaStream_t>(stream), pdl, 0,
                  static_cast<const unsigned char*>(x), static_cast<unsigned char*>(windows_q), scales, a, ctx->map);
  };
  if (grouped) {   // rows beyond 16 KB
    stages == 3 ? launch(dispatch_quant_kernel<3, 0, false, true>) : launch(dispatch_quant_kernel<2, 0, false, true>);
  } else if (stages == 3) {
    if (cpl == 32) whole_slabs ? launch(dispatch_quant_kernel<3, 32, true>) : launch(dispatch_quant_kernel<3, 32, false>);
    else launch(dispatch_quant_kernel<3, 0, false>);
  } else {   // (rows beyond 16 KB only: shorter rows of small jobs went to the register kernel)
    launch(dispatch_quant_kernel<2, 0, false>);
  }
  return launched();
}

// moe_plan followed by the quantising dispatch, chained; every host-side check comes before anything is enqueued.
static moe_status_t plan_dispatch_quant_impl(moe_ctx* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T,
                                             const int32_t* rank_tok_start, const void* x, void* windows_q,
                                             float* scales, int64_t capacity_rows, int group, void* stream) {
  if (!quant_shape_ok(ctx->shape.H, group) || capacity_rows < 0 || !aligned16(x) || !aligned16(windows_q) ||
      (reinterpret_cast<uintptr_t>(scales) & 3u) != 0)
    return MOE_ERR_INVALID_ARG;
  const moe_status_t rc = plan_impl(ctx, schedule, topk_idx, T, rank_tok_start, stream, nullptr, nullptr, nullptr);
  if (rc != MOE_OK) return rc;
  return dispatch_quant_impl(ctx, x, windows_q, scales, capacity_rows, stream, true, nullptr, nullptr, group);
}

moe_status_t moe_dispatch_quant(moe_ctx_t* ctx, const void* x, void* windows_q, float* scales, int64_t capacity_rows,
                                void* stream) {
  return dispatch_quant_impl(ctx, x, windows_q, scales, capacity_rows, stream, false);
}

moe_status_t moe_dispatch_quant_group(moe_ctx_t* ctx, const void* x, void* windows_q, float* scales,
                                      int64_t capacity_rows, int32_t group_size, void* stream) {
  if (group_size != QUANT_GROUP) return MOE_ERR_INVALID_ARG;
  return dispatch_quant_impl(ctx, x, windows_q, scales, capacity_rows, stream, false, nullptr, nullptr, group_size);
}

moe_status_t moe_dispatch_quant_peers(moe_ctx_t* ctx, const void* x, const void* const* window_q_bases,
                                      float* const* scale_bases, int64_t capacity_rows, void* stream) {
  if (window_q_bases == nullptr || scale_bases == nullptr) return MOE_ERR_INVALID_ARG;
  return dispatch_quant_impl(ctx, x, nullptr, nullptr, capacity_rows, stream, false, window_q_bases, scale_bases);
}

moe_status_t moe_plan_dispatch_quant(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T,
                                     const int32_t* rank_tok_start, const void* x, void* windows_q, float* scales,
                                     int64_t capacity_rows, void* stream) {
  if (ctx == nullptr || (T > 0 && (topk_idx == nullptr || x == nullptr || windows_q == nullptr || scales == nullptr)))
    return MOE_ERR_INVALID_ARG;
  return plan_dispatch_quant_impl(ctx, schedule, topk_idx, T, rank_tok_start, x, windows_q, scales, capacity_rows, 0, stream);
}

moe_status_t moe_plan_dispatch_quant_group(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T,
                                           const int32_t* rank_tok_start, const void* x, void* windows_q,
                                           float* scales, int64_t capacity_rows, int32_t group_size, void* stream) {
  if (ctx == nullptr || group_size != QUANT_GROUP ||
      (T > 0 && (topk_idx == nullptr || x == nullptr || windows_q == nullptr || scales == nullptr)))
    return MOE_ERR_INVALID_ARG;
  return plan_dispatch_quant_impl(ctx, schedule, topk_idx, T, rank_tok_start, x, windows_q, scales, capacity_rows,
                                  group_size, stream);
}

}  // extern "C"

namespace {

moe_status_t combine_impl(moe_ctx* ctx, const void* windows, const void* const* bases, int64_t capacity_rows,
                          const float* topk_w, void* y, void* stream, int32_t t_begin = 0, int32_t t_end = -1) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->planned) return MOE_ERR_NOT_PLANNED;
  if (capacity_rows < 0 ||
      (ctx->T > 0 && ((windows == nullptr && bases == nullptr) || topk_w == nullptr || y == nullptr)))
    return MOE_ERR_INVALID_ARG;
  if (!aligned16(windows) || !aligned16(y)) return MOE_ERR_INVALID_ARG;
  if (t_end < 0) t_end = ctx->T;
  if (t_begin < 0 || t_begin > t_end || t_end > ctx->T) return MOE_ERR_INVALID_ARG;
  RowArgs a = row_args(ctx, capacity_rows, false);
  a.win_base = reinterpret_cast<const unsigned char* const*>(bases);
  a.t_begin = t_begin;
  a.t_count = t_end - t_begin;
  a.topk_idx = ctx->topk_idx;
  if (ctx->slots_for_C == capacity_rows && ctx->slot_reuse) a.slot_in = ctx->slot_table;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint4* win = static_cast<const uint4*>(windows);
  uint4* ys = static_cast<uint4*>(y);
  switch (ctx->shape.K) {
    case 1: launch_combine<1>(ctx, a, win, topk_w, ys, st); break;
    case 2: launch_combine<2>(ctx, a, win, topk_w, ys, st); break;
    case 4: launch_combine<4>(ctx, a, win, topk_w, ys, st); break;
    case 3: launch_combine<3>(ctx, a, win, topk_w, ys, st); break;
    case 5: launch_combine<5>(ctx, a, win, topk_w, ys, st); break;
    case 6: launch_combine<6>(ctx, a, win, topk_w, ys, st); break;
    case 7: launch_combine<7>(ctx, a, win, topk_w, ys, st); break;
    case 8: launch_combine<8>(ctx, a, win, topk_w, ys, st); break;
    case 9: launch_combine<9>(ctx, a, win, topk_w, ys, st); break;   // eight routed experts and a shared one
    case 10: launch_combine<10>(ctx, a, win, topk_w, ys, st); break;
    case 12: launch_combine<12>(ctx, a, win, topk_w, ys, st); break;
    case 16: launch_combine<16>(ctx, a, win, topk_w, ys, st); break;
    default:   // the other degrees share three kernels: up to 16, 24 or 32 branches, K of them live
      if (ctx->shape.K <= 16) launch_combine<-16>(ctx, a, win, topk_w, ys, st);
      else if (ctx->shape.K <= 24) launch_combine<-24>(ctx, a, win, topk_w, ys, st);
      else launch_combine<-32>(ctx, a, win, topk_w, ys, st);
      break;
  }
  return launch_ok(ctx);
}

}  // namespace

extern "C" {

moe_status_t moe_combine(moe_ctx_t* ctx, const void* windows, int64_t capacity_rows, const float* topk_w, void* y,
                         void* stream) {
  if (ctx != nullptr && ctx->T > 0 && windows == nullptr) return MOE_ERR_INVALID_ARG;
  return combine_impl(ctx, windows, nullptr, capacity_rows, topk_w, y, stream);
}

moe_status_t moe_combine_range(moe_ctx_t* ctx, const void* windows, int64_t capacity_rows, const float* topk_w, void* y,
                               int32_t t_begin, int32_t t_end, void* stream) {
  if (ctx != nullptr && ctx->T > 0 && windows == nullptr) return MOE_ERR_INVALID_ARG;
  if (t_end < 0) return MOE_ERR_INVALID_ARG;
  return combine_impl(ctx, windows, nullptr, capacity_rows, topk_w, y, stream, t_begin, t_end);
}

moe_status_t moe_combine_peers(moe_ctx_t* ctx, const void* const* window_bases, int64_t capacity_rows,
                               const float* topk_w, void* y, void* stream) {
  if (window_bases == nullptr) return MOE_ERR_INVALID_ARG;
  return combine_impl(ctx, nullptr, window_bases, capacity_rows, topk_w, y, stream);
}

/* Multi-rank decomposition: Layout for one rank's tokens, Notify from the gathered counts. */
moe_status_t moe_layout(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T_local,
                        int32_t my_rank, int32_t* counts_row, void* stream) {
  if (ctx == nullptr || my_rank < 0 || my_rank >= ctx->shape.R || counts_row == nullptr) return MOE_ERR_INVALID_ARG;
  if (T_local > 0 && topk_idx == nullptr) return MOE_ERR_INVALID_ARG;
  int32_t starts[MOE_MAX_R + 1];
  for (int r = 0; r <= ctx->shape.R; ++r) starts[r] = r <= my_rank ? 0 : T_local;   // only my_rank owns tokens
  const moe_status_t rc = plan_impl(ctx, schedule, topk_idx, T_local, starts, stream, nullptr, nullptr, nullptr, my_rank);
  if (rc != MOE_OK) return rc;
  ctx->planned = false;   // the offsets are not valid until moe_notify has seen every rank's counts
  ctx->slots_for_C = -1;
  if (cudaMemcpyAsync(counts_row, ctx->M + (size_t)my_rank * ctx->shape.E, sizeof(int32_t) * ctx->shape.E,
                      cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return MOE_ERR_CUDA;
  ctx->layout_done = true;
  return MOE_OK;
}

moe_status_t moe_layout_push(moe_ctx_t* ctx, moe_schedule_t schedule, const int32_t* topk_idx, int32_t T_local,
                             int32_t my_rank, uint32_t epoch, void* stream) {
  if (ctx == nullptr || my_rank < 0 || my_rank >= ctx->shape.R) return MOE_ERR_INVALID_ARG;
  if (T_local > 0 && topk_idx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->peers_installed || !ctx->peers_have_counts || my_rank != ctx->my_rank) return MOE_ERR_STALE_PEERS;
  int32_t starts[MOE_MAX_R + 1];
  for (int r = 0; r <= ctx->shape.R; ++r) starts[r] = r <= my_rank ? 0 : T_local;
  bool pushed = false;
  const moe_status_t rc =
      plan_impl(ctx, schedule, topk_idx, T_local, starts, stream, nullptr, nullptr, nullptr, my_rank, true, epoch, &pushed);
  if (rc != MOE_OK) return rc;
  ctx->planned = false;
  ctx->slots_for_C = -1;
  ctx->layout_done = true;
  return pushed ? MOE_OK : moe_push_counts(ctx, epoch, stream);   // (large batches: the tile planner, then the push)
}

moe_status_t moe_notify(moe_ctx_t* ctx, const int32_t* counts_all, void* stream) {
  if (ctx == nullptr || counts_all == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->layout_done) return MOE_ERR_NOT_PLANNED;
  const moe_shape_t& sh = ctx->shape;
  notify_rank_kernel<<<sh.R, 256, cluster_notify_smem_ints(sh.E, sh.R) * (int)sizeof(int32_t),
                       static_cast<cudaStream_t>(stream)>>>(
      counts_all, sh.E, sh.R, ctx->schedule == MOE_SCHED_PREFILL, ctx->expert_align, ctx->M, ctx->c_rank, ctx->o,
      ctx->n_exp, ctx->n_recv);
  const moe_status_t rc = launch_ok(ctx);
  if (rc == MOE_OK) ctx->planned = true;
  return rc;
}

/* ---------------------------------------------------------------------------------------------
 * Window addresses of the expert-parallel group: export, handshake, cached table. */
namespace {

// Base and size of the device allocation that contains p.  The runtime API has no call for it, so the driver's
// is looked up at run time (the library links no driver library and loads on a machine without one).
bool allocation_range(const void* p, uintptr_t* base, size_t* size) {
  typedef int (*range_fn)(unsigned long long*, size_t*, unsigned long long);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult found;
  if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &found) != cudaSuccess || fn == nullptr ||
      found != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return false;
  }
  unsigned long long b = 0;
  size_t n = 0;
  if (reinterpret_cast<range_fn>(fn)(&b, &n, (unsigned long long)reinterpret_cast<uintptr_t>(p)) != 0) return false;
  *base = (uintptr_t)b;
  *size = n;
  return true;
}

void release_mappings(moe_ctx* ctx) {
  for (int d = 0; d < ctx->shape.R; ++d)
    if (ctx->peer_mapping[d] != nullptr) {
      cudaIpcCloseMemHandle(ctx->peer_mapping[d]);
      cudaGetLastError();
      ctx->peer_mapping[d] = nullptr;
    }
  ctx->peers_installed = false;
}

size_t state_bytes_for(int32_t R) { return align_up(sizeof(uint32_t) * MOE_SYNC_SLOTS * (size_t)R); }

// Parts of a window allocation, byte offsets from its first row (see MOE_WINDOW_* in the header).
struct WindowParts {
  size_t state, box, codes, scales, total;
};
WindowParts window_parts(const moe_shape_t& sh, int64_t capacity_rows, int32_t flags) {
  WindowParts p;
  const size_t rows = (size_t)capacity_rows * sh.H * 2;
  size_t at = flags != 0 ? align_up(rows) : rows;
  p.state = at;
  if (flags & MOE_WINDOW_STATE) at += state_bytes_for(sh.R);
  p.box = at;
  if (flags & MOE_WINDOW_COUNTS) at += align_up(counts_box_bytes(sh.E, sh.R));
  p.codes = at;
  if (flags & (MOE_WINDOW_QUANT | MOE_WINDOW_QUANT_GROUP)) at += align_up((size_t)capacity_rows * sh.H);
  p.scales = at;
  if (flags & MOE_WINDOW_QUANT) at += align_up((size_t)capacity_rows * sizeof(float));
  if (flags & MOE_WINDOW_QUANT_GROUP) at += align_up((size_t)capacity_rows * (sh.H / QUANT_GROUP) * sizeof(float));
  p.total = at;
  return p;
}

// Known bits only, and at most one form of quantised parts.
bool window_flags_ok(int32_t flags) {
  if ((flags & ~(MOE_WINDOW_STATE | MOE_WINDOW_QUANT | MOE_WINDOW_QUANT_GROUP | MOE_WINDOW_COUNTS)) != 0) return false;
  if ((flags & MOE_WINDOW_COUNTS) != 0 && (flags & MOE_WINDOW_STATE) == 0) return false;   // the mailbox follows the flags
  return (flags & MOE_WINDOW_QUANT) == 0 || (flags & MOE_WINDOW_QUANT_GROUP) == 0;
}
// ... and a shape the group-wise parts exist for.
bool window_flags_fit(int32_t flags, const moe_shape_t& sh) {
  return window_flags_ok(flags) && ((flags & MOE_WINDOW_QUANT_GROUP) == 0 || sh.H % QUANT_GROUP == 0);
}

// Copies the addresses of every rank's rows, state region, code window and scale tensor to the device tables on
// `stream` and marks them installed.
moe_status_t install_table(moe_ctx* ctx, int32_t my_rank, int64_t capacity_rows, int32_t flags, cudaStream_t st) {
  const int R = ctx->shape.R;
  void* all[5 * MOE_MAX_R];
  const WindowParts parts = window_parts(ctx->shape, capacity_rows, flags);
  for (int d = 0; d < R; ++d) {
    char* base = static_cast<char*>(ctx->peer_ptr[d]);
    all[d] = base;
    all[R + d] = (flags & MOE_WINDOW_STATE) ? base + parts.state : nullptr;
    const bool quant = (flags & (MOE_WINDOW_QUANT | MOE_WINDOW_QUANT_GROUP)) != 0;
    all[2 * R + d] = quant ? base + parts.codes : nullptr;
    all[3 * R + d] = quant ? base + parts.scales : nullptr;
    all[4 * R + d] = (flags & MOE_WINDOW_COUNTS) ? base + parts.box : nullptr;
  }
  // pageable source: the runtime has staged the bytes by the time the call returns
  if (cudaMemcpyAsync(ctx->peer_table, all, sizeof(void*) * 5 * R, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  ctx->peer_capacity = capacity_rows;
  ctx->my_rank = my_rank;
  ctx->peers_have_state = (flags & MOE_WINDOW_STATE) != 0;
  ctx->peers_have_quant = (flags & MOE_WINDOW_QUANT) != 0;
  ctx->peers_have_quant_group = (flags & MOE_WINDOW_QUANT_GROUP) != 0;
  ctx->peers_have_counts = (flags & MOE_WINDOW_COUNTS) != 0;
  ctx->peers_installed = true;
  return MOE_OK;
}

moe_status_t table_fresh(const moe_ctx* ctx, const int32_t* generations) {
  if (!ctx->peers_installed) return MOE_ERR_STALE_PEERS;
  if (generations != nullptr)
    for (int d = 0; d < ctx->shape.R; ++d)
      if (generations[d] != ctx->peer_gen[d]) return MOE_ERR_STALE_PEERS;
  return MOE_OK;
}

}  // namespace

moe_status_t moe_window_export(const void* window, int64_t bytes, int32_t generation, int32_t flags,
                               moe_window_handle_t* out) {
  if (window == nullptr || out == nullptr || bytes <= 0 || !aligned16(window) || !window_flags_ok(flags))
    return MOE_ERR_INVALID_ARG;
  static_assert(sizeof(cudaIpcMemHandle_t) == sizeof(out->ipc), "handle size");
  uintptr_t base = 0;
  size_t size = 0;
  if (!allocation_range(window, &base, &size)) return MOE_ERR_CUDA;
  const uintptr_t at = reinterpret_cast<uintptr_t>(window);
  if (at < base || at + (uint64_t)bytes > base + size) return MOE_ERR_INVALID_ARG;   // the window spans allocations
  cudaIpcMemHandle_t h;
  if (cudaIpcGetMemHandle(&h, reinterpret_cast<void*>(base)) != cudaSuccess) {
    cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  std::memcpy(out->ipc, &h, sizeof(h));
  out->offset = (int64_t)(at - base);
  out->bytes = bytes;
  out->generation = generation;
  out->flags = flags;
  out->reserved = 0;
  if (cudaGetDevice(&out->device) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

moe_status_t moe_peers_open(moe_ctx_t* ctx, const moe_window_handle_t* handles, int32_t my_rank, void* my_window,
                            int64_t capacity_rows, void* stream) {
  if (ctx == nullptr || handles == nullptr || my_window == nullptr || my_rank < 0 || my_rank >= ctx->shape.R ||
      capacity_rows < 0 || !aligned16(my_window))
    return MOE_ERR_INVALID_ARG;
  // every rank exports the same parts, and enough bytes for them at this capacity
  const int32_t flags = handles[my_rank].flags;
  if (!window_flags_fit(flags, ctx->shape)) return MOE_ERR_INVALID_ARG;
  const int64_t need = (int64_t)window_parts(ctx->shape, capacity_rows, flags).total;
  for (int d = 0; d < ctx->shape.R; ++d)
    if (handles[d].flags != flags || handles[d].bytes < need || (handles[d].offset & 15) != 0) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return MOE_ERR_CUDA;   // nothing in flight reads the old table
  release_mappings(ctx);
  for (int d = 0; d < ctx->shape.R; ++d) {
    ctx->peer_gen[d] = handles[d].generation;
    if (d == my_rank) {
      ctx->peer_ptr[d] = my_window;
      continue;
    }
    cudaIpcMemHandle_t h;
    std::memcpy(&h, handles[d].ipc, sizeof(h));
    void* base = nullptr;
    if (cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess || base == nullptr) {
      cudaGetLastError();
      release_mappings(ctx);
      return MOE_ERR_CUDA;
    }
    ctx->peer_mapping[d] = base;
    ctx->peer_ptr[d] = static_cast<char*>(base) + handles[d].offset;
  }
  return install_table(ctx, my_rank, capacity_rows, flags, st);
}

moe_status_t moe_peers_set(moe_ctx_t* ctx, const void* const* window_bases, const int32_t* generations, int32_t my_rank,
                           int64_t capacity_rows, int32_t flags, void* stream) {
  if (ctx == nullptr || window_bases == nullptr || capacity_rows < 0 || my_rank < 0 || my_rank >= ctx->shape.R ||
      !window_flags_fit(flags, ctx->shape))
    return MOE_ERR_INVALID_ARG;
  for (int d = 0; d < ctx->shape.R; ++d)
    if (window_bases[d] == nullptr || !aligned16(window_bases[d])) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return MOE_ERR_CUDA;
  release_mappings(ctx);
  for (int d = 0; d < ctx->shape.R; ++d) {
    ctx->peer_ptr[d] = const_cast<void*>(window_bases[d]);
    ctx->peer_gen[d] = generations != nullptr ? generations[d] : 0;
  }
  return install_table(ctx, my_rank, capacity_rows, flags, st);
}

size_t moe_state_bytes(int32_t R) { return (R < 1 || R > MOE_MAX_R) ? 0 : state_bytes_for(R); }

size_t moe_window_bytes(const moe_shape_t* shape, int64_t capacity_rows, int32_t flags) {
  if (!shape_valid(shape) || capacity_rows < 0 || !window_flags_fit(flags, *shape)) return 0;
  return window_parts(*shape, capacity_rows, flags).total;
}

moe_status_t moe_signal_peers(moe_ctx_t* ctx, int32_t slot, uint32_t epoch, void* stream) {
  if (ctx == nullptr || slot < 0 || slot >= MOE_SYNC_SLOTS) return MOE_ERR_INVALID_ARG;
  if (!ctx->peers_installed || !ctx->peers_have_state) return MOE_ERR_STALE_PEERS;
  const int R = ctx->shape.R;
  signal_peers_kernel<<<1, R < 32 ? 32 : (R + 31) / 32 * 32, 0, static_cast<cudaStream_t>(stream)>>>(
      ctx->state_table, R, ctx->my_rank, slot, epoch);
  return launch_ok(ctx);
}

moe_status_t moe_wait_peers(moe_ctx_t* ctx, int32_t slot, uint32_t epoch, void* stream) {
  if (ctx == nullptr || slot < 0 || slot >= MOE_SYNC_SLOTS) return MOE_ERR_INVALID_ARG;
  if (!ctx->peers_installed || !ctx->peers_have_state) return MOE_ERR_STALE_PEERS;
  const int R = ctx->shape.R;
  const unsigned char* mine = static_cast<const unsigned char*>(ctx->peer_ptr[ctx->my_rank]) +
                              window_parts(ctx->shape, ctx->peer_capacity, MOE_WINDOW_STATE).state;
  wait_peers_kernel<<<1, R < 32 ? 32 : (R + 31) / 32 * 32, 0, static_cast<cudaStream_t>(stream)>>>(
      mine, R, slot, epoch, ctx->starve_wait_ms > 0 ? ctx->starve_wait_ms : WAIT_LIMIT_MS_DEFAULT, &ctx->ctl->status);
  return launch_ok(ctx);
}

moe_status_t moe_push_counts(moe_ctx_t* ctx, uint32_t epoch, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->layout_done) return MOE_ERR_NOT_PLANNED;
  if (!ctx->peers_installed || !ctx->peers_have_counts) return MOE_ERR_STALE_PEERS;
  const moe_shape_t& sh = ctx->shape;
  push_counts_kernel<<<(sh.R + PUSH_RANKS_PER_CTA - 1) / PUSH_RANKS_PER_CTA, 1024, 0, static_cast<cudaStream_t>(stream)>>>(
      ctx->box_table, ctx->M + (size_t)ctx->my_rank * sh.E, sh.E, sh.R, ctx->my_rank, epoch);
  return launch_ok(ctx);
}

moe_status_t moe_notify_peers(moe_ctx_t* ctx, uint32_t epoch, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->layout_done) return MOE_ERR_NOT_PLANNED;
  if (!ctx->peers_installed || !ctx->peers_have_counts) return MOE_ERR_STALE_PEERS;
  const moe_shape_t& sh = ctx->shape;
  unsigned char* mine = static_cast<unsigned char*>(ctx->peer_ptr[ctx->my_rank]) +
                        window_parts(sh, ctx->peer_capacity, MOE_WINDOW_STATE | MOE_WINDOW_COUNTS).box;
  notify_box_kernel<<<sh.R, 256, cluster_notify_smem_ints(sh.E, sh.R) * (int)sizeof(int32_t),
                      static_cast<cudaStream_t>(stream)>>>(
      mine, sh.E, sh.R, epoch, ctx->starve_wait_ms > 0 ? ctx->starve_wait_ms : WAIT_LIMIT_MS_DEFAULT,
      ctx->schedule == MOE_SCHED_PREFILL, ctx->expert_align, ctx->M, ctx->c_rank, ctx->o, ctx->n_exp, ctx->n_recv,
      &ctx->ctl->status);
  const moe_status_t rc = launch_ok(ctx);
  if (rc == MOE_OK) {
    ctx->planned = true;
    ctx->notified_by_box = true;
  }
  return rc;
}

moe_status_t moe_peers_check(const moe_ctx_t* ctx, const int32_t* generations) {
  if (ctx == nullptr || generations == nullptr) return MOE_ERR_INVALID_ARG;
  return table_fresh(ctx, generations);
}

moe_status_t moe_peers_close(moe_ctx_t* ctx, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MOE_ERR_CUDA;
  release_mappings(ctx);
  return MOE_OK;
}

moe_status_t moe_dispatch_cached(moe_ctx_t* ctx, const void* x, const int32_t* generations, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  const moe_status_t fresh = table_fresh(ctx, generations);
  if (fresh != MOE_OK) return fresh;
  return dispatch_impl(ctx, x, nullptr, reinterpret_cast<const void* const*>(ctx->peer_table), ctx->peer_capacity, stream);
}

moe_status_t moe_dispatch_quant_cached(moe_ctx_t* ctx, const void* x, const int32_t* generations, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  const moe_status_t fresh = table_fresh(ctx, generations);
  if (fresh != MOE_OK) return fresh;
  if (!ctx->peers_have_quant) return MOE_ERR_STALE_PEERS;   // the installed windows reserve no room for codes and scales
  return dispatch_quant_impl(ctx, x, nullptr, nullptr, ctx->peer_capacity, stream, false,
                             reinterpret_cast<const void* const*>(ctx->code_table), ctx->scale_table);
}

moe_status_t moe_dispatch_quant_group_cached(moe_ctx_t* ctx, const void* x, const int32_t* generations,
                                             int32_t group_size, void* stream) {
  if (ctx == nullptr || group_size != QUANT_GROUP) return MOE_ERR_INVALID_ARG;
  const moe_status_t fresh = table_fresh(ctx, generations);
  if (fresh != MOE_OK) return fresh;
  if (!ctx->peers_have_quant_group) return MOE_ERR_STALE_PEERS;   // no room for codes and group scales in the installed windows
  return dispatch_quant_impl(ctx, x, nullptr, nullptr, ctx->peer_capacity, stream, false,
                             reinterpret_cast<const void* const*>(ctx->code_table), ctx->scale_table, group_size);
}

moe_status_t moe_combine_cached(moe_ctx_t* ctx, const int32_t* generations, const float* topk_w, void* y, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  const moe_status_t fresh = table_fresh(ctx, generations);
  if (fresh != MOE_OK) return fresh;
  return combine_impl(ctx, nullptr, reinterpret_cast<const void* const*>(ctx->peer_table), ctx->peer_capacity, topk_w, y,
                      stream);
}

moe_status_t moe_slots(moe_ctx_t* c, int64_t capacity_rows, int32_t* slots, void* stream) {
  moe_ctx* ctx = c;
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  if (!ctx->planned) return MOE_ERR_NOT_PLANNED;
  if (capacity_rows < 0 || (int64_t)ctx->shape.R * capacity_rows >= (int64_t)1 << 31) return MOE_ERR_INVALID_ARG;
  if (ctx->T > 0 && slots == nullptr) return MOE_ERR_INVALID_ARG;
  RowArgs a = row_args(ctx, capacity_rows, false);
  a.topk_idx = ctx->topk_idx;
  const int64_t B = (int64_t)ctx->T * ctx->shape.K;
  int grid = (int)((B + 255) / 256);
  if (grid < 1) grid = 1;
  if (grid > ctx->num_sms * 8) grid = ctx->num_sms * 8;
  slots_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(slots, a, ctx->map);
  return launch_ok(ctx);
}

moe_status_t moe_expert_ranges(moe_ctx_t* ctx, int64_t capacity_rows, int64_t* row_start, int32_t* row_count,
                               void* stream) {
  if (ctx == nullptr || row_start == nullptr || row_count == nullptr || capacity_rows < 0) return MOE_ERR_INVALID_ARG;
  if (!ctx->planned) return MOE_ERR_NOT_PLANNED;
  const int E = ctx->shape.E;
  expert_ranges_kernel<<<(E + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      ctx->o, ctx->n_exp, E, ctx->shape.R, capacity_rows, row_start, row_count);
  return launch_ok(ctx);
}

moe_status_t moe_expert_tiles(moe_ctx_t* ctx, int64_t capacity_rows, int32_t tile_rows, int64_t max_tiles,
                              int32_t* tile_expert, int64_t* tile_row, int32_t* tile_valid, int32_t* n_tiles,
                              void* stream) {
  if (ctx == nullptr || capacity_rows < 0 || tile_rows < 1 || max_tiles < 0 || n_tiles == nullptr) return MOE_ERR_INVALID_ARG;
  if (max_tiles > 0 && (tile_expert == nullptr || tile_row == nullptr || tile_valid == nullptr)) return MOE_ERR_INVALID_ARG;
  if (!ctx->planned) return MOE_ERR_NOT_PLANNED;
  const int E = ctx->shape.E;
  expert_tiles_kernel<<<1, 1024, (2 * E + 1 + 33) * (int)sizeof(int32_t), static_cast<cudaStream_t>(stream)>>>(
      ctx->o, ctx->n_exp, E, ctx->shape.R, capacity_rows, tile_rows, max_tiles, tile_expert, tile_row, tile_valid, n_tiles);
  return launch_ok(ctx);
}

moe_status_t moe_forward_host(moe_ctx_t* ctx, moe_schedule_t schedule, int32_t T, const int32_t* rank_tok_start,
                              const void* x_host, const int32_t* topk_idx_host, const float* topk_w_host,
                              void* x_dev, int32_t* topk_idx_dev, float* topk_w_dev, void* windows_dev,
                              int64_t capacity_rows, void* y_dev, void* y_host, void* stream) {
  if (ctx == nullptr || T < 0 || T > ctx->shape.T_max) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (x_host == nullptr || topk_idx_host == nullptr || topk_w_host == nullptr || x_dev == nullptr ||
                topk_idx_dev == nullptr || topk_w_dev == nullptr || windows_dev == nullptr || y_dev == nullptr ||
                y_host == nullptr))
    return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t row_bytes = (size_t)ctx->shape.H * 2, B = (size_t)T * ctx->shape.K;
  if (T > 0) {
    if (cudaMemcpyAsync(topk_idx_dev, topk_idx_host, B * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(topk_w_dev, topk_w_host, B * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return MOE_ERR_CUDA;
  }
  moe_status_t rc = moe_plan(ctx, schedule, topk_idx_dev, T, rank_tok_start, stream);
  if (rc != MOE_OK || T == 0) return rc;

  // Token chunks flow through a three-stream pipeline: an upload stream copies chunk c of x to the
  // device, the caller's stream dispatches and combines it (identity experts: a token's output needs
  // only its own rows), and a download stream copies its outputs back, so both copy directions and the
  // kernels overlap.  Nothing here allocates device memory; streams and events are created on first use.
  if (ctx->out_stream == nullptr) {
    if (cudaStreamCreateWithFlags(&ctx->out_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&ctx->in_stream, cudaStreamNonBlocking) != cudaSuccess)
      return MOE_ERR_CUDA;
    for (int i = 0; i < 2 * FWD_CHUNKS + 2; ++i)
      if (cudaEventCreateWithFlags(&ctx->fwd_events[i], cudaEventDisableTiming) != cudaSuccess) return MOE_ERR_CUDA;
  }
  cudaEvent_t* up = ctx->fwd_events;                      // [c]: chunk c uploaded
  cudaEvent_t* done = ctx->fwd_events + FWD_CHUNKS;       // [c]: chunk c combined
  cudaEvent_t start = ctx->fwd_events[2 * FWD_CHUNKS], finish = ctx->fwd_events[2 * FWD_CHUNKS + 1];
  const int chunks = T >= 4 * FWD_CHUNKS ? FWD_CHUNKS : 1;
  char* xd = static_cast<char*>(x_dev);
  const char* xh = static_cast<const char*>(x_host);
  char* yd = static_cast<char*>(y_dev);
  char* yh = static_cast<char*>(y_host);
  // Uploads may overwrite x_dev only after everything enqueued before this call has used it.
  if (cudaEventRecord(start, st) != cudaSuccess || cudaStreamWaitEvent(ctx->in_stream, start, 0) != cudaSuccess)
    return MOE_ERR_CUDA;
  for (int c = 0; c < chunks; ++c) {
    const int32_t t0 = (int32_t)((int64_t)T * c / chunks), t1 = (int32_t)((int64_t)T * (c + 1) / chunks);
    if (cudaMemcpyAsync(xd + t0 * row_bytes, xh + t0 * row_bytes, (size_t)(t1 - t0) * row_bytes, cudaMemcpyHostToDevice,
                        ctx->in_stream) != cudaSuccess ||
        cudaEventRecord(up[c], ctx->in_stream) != cudaSuccess || cudaStreamWaitEvent(st, up[c], 0) != cudaSuccess)
      return MOE_ERR_CUDA;
    rc = moe_dispatch_range(ctx, x_dev, windows_dev, capacity_rows, t0, t1, stream);
    if (rc != MOE_OK) return rc;
    rc = moe_combine_range(ctx, windows_dev, capacity_rows, topk_w_dev, y_dev, t0, t1, stream);
    if (rc != MOE_OK) return rc;
    if (cudaEventRecord(done[c], st) != cudaSuccess || cudaStreamWaitEvent(ctx->out_stream, done[c], 0) != cudaSuccess ||
        cudaMemcpyAsync(yh + t0 * row_bytes, yd + t0 * row_bytes, (size_t)(t1 - t0) * row_bytes, cudaMemcpyDeviceToHost,
                        ctx->out_stream) != cudaSuccess)
      return MOE_ERR_CUDA;
  }
  // The caller's stream finishes only after the last download, so synchronising it (moe_status) is enough.
  if (cudaEventRecord(finish, ctx->out_stream) != cudaSuccess || cudaStreamWaitEvent(st, finish, 0) != cudaSuccess)
    return MOE_ERR_CUDA;
  return MOE_OK;
}

moe_status_t moe_set_option(moe_ctx_t* ctx, moe_option_t option, int64_t value) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  switch (option) {
    case MOE_OPT_DISPATCH_PATH:
      if (value != MOE_DISPATCH_AUTO && value != MOE_DISPATCH_REGISTERS && value != MOE_DISPATCH_BULK)
        return MOE_ERR_INVALID_ARG;
      ctx->dispatch_path = (int32_t)value;
      return MOE_OK;
    case MOE_OPT_TEST_STARVE_WAIT_MS:
      if (value < 0 || value > 10000) return MOE_ERR_INVALID_ARG;
      ctx->starve_wait_ms = (int32_t)value;
      return MOE_OK;
    case MOE_OPT_GRANULE:
      if (value < 0 || value > (1 << 20)) return MOE_ERR_INVALID_ARG;
      ctx->granule_override = (int32_t)value;
      return MOE_OK;
    case MOE_OPT_EXPERT_ALIGN:
      if (value < 1 || value > 4096) return MOE_ERR_INVALID_ARG;
      if ((int64_t)ctx->shape.T_max * ctx->shape.K + (int64_t)ctx->shape.E * (value - 1) >= ((int64_t)1 << 31))
        return MOE_ERR_INVALID_ARG;   // padded row counts must stay in int32
      ctx->expert_align = (int32_t)value;
      ctx->planned = false;           // offsets of an earlier plan no longer describe the layout asked for
      ctx->slots_for_C = -1;
      ctx->layout_done = false;
      return MOE_OK;
    case MOE_OPT_CLUSTER_PLAN:
      if (value != 0 && value != 1) return MOE_ERR_INVALID_ARG;
      ctx->cluster_plan = (int32_t)value;
      return MOE_OK;
    case MOE_OPT_OVERLAP:
      if (value != 0 && value != 1) return MOE_ERR_INVALID_ARG;
      ctx->overlap = (int32_t)value;
      return MOE_OK;
    case MOE_OPT_SLOT_REUSE:
      if (value != 0 && value != 1) return MOE_ERR_INVALID_ARG;
      ctx->slot_reuse = (int32_t)value;
      return MOE_OK;
  }
  return MOE_ERR_INVALID_ARG;
}

moe_status_t moe_status(moe_ctx_t* ctx, void* stream) {
  if (ctx == nullptr) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t word = 0;
  if (cudaMemcpyAsync(&word, &ctx->ctl->status, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (word != 0) {
    if (cudaMemsetAsync(&ctx->ctl->status, 0, sizeof(word), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
      return MOE_ERR_CUDA;
    // A plan that saw a routing index outside [0, E) left that branch out of its counts: it describes no
    // valid layout, so it does not survive the report (a later dispatch returns MOE_ERR_NOT_PLANNED
    // instead of silently skipping the branch).
    ctx->slots_for_C = -1;   // a dispatch that stopped early has not recorded every row
    if (word == MOE_ERR_BAD_INDEX || (word == MOE_ERR_TIMEOUT && ctx->notified_by_box)) {
      ctx->planned = false;
      ctx->layout_done = false;
    }
  }
  return (word >= 0 && word <= MOE_ERR_STALE_PEERS) ? static_cast<moe_status_t>(word) : MOE_ERR_CUDA;
}

const char* moe_status_string(moe_status_t status) {
  switch (status) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_BAD_INDEX: return "routing index outside [0, E)";
    case MOE_ERR_CAPACITY: return "expert window capacity too small";
    case MOE_ERR_NOT_PLANNED: return "no plan: call moe_plan first";
    case MOE_ERR_TIMEOUT: return "bounded device wait expired";
    case MOE_ERR_CUDA: return "CUDA error";
    case MOE_ERR_STALE_PEERS: return "window address table missing or out of date";
  }
  return "unknown status";
}

int64_t moe_launch_count(const moe_ctx_t* ctx) { return ctx == nullptr ? 0 : ctx->launches; }

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// moe_slots_noalloc: routing indexes -> window slots with no caller workspace.
//
// Some callers of this library have no device memory to hand over for control state and may not
// obtain any: a plug-in running inside an engine that reserved the whole HBM for its own pool at
// start-up, or a latency-critical decode loop where a device allocation (which can stall the
// device) is forbidden after initialisation.  For them the planning scratch lives in the
// file-scope device array below, which every GPU that loads this library holds until the process
// exits.  The entry point runs the same planning kernels as moe_plan(DECODE) + moe_slots, pointed
// at that array.
namespace {

constexpr int32_t NOALLOC_MAX_BRANCHES = 65536;  // T * K
constexpr int32_t NOALLOC_MAX_E = 512;
constexpr int32_t NOALLOC_MAX_R = 64;
constexpr int32_t NOALLOC_MAX_TILES = NOALLOC_MAX_BRANCHES / (ROUNDS_DECODE * PLAN_THREADS) + NOALLOC_MAX_R;

struct NoallocScratch {
  Control ctl;
  int32_t M[NOALLOC_MAX_R * NOALLOC_MAX_E];
  int32_t c_rank[NOALLOC_MAX_R * NOALLOC_MAX_R];
  int32_t o[NOALLOC_MAX_E * NOALLOC_MAX_R];
  int32_t n_exp[NOALLOC_MAX_E];
  int32_t tile_rank[NOALLOC_MAX_BRANCHES];
  int32_t tile_hist[(size_t)NOALLOC_MAX_TILES * NOALLOC_MAX_E];
};

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoallocScratch)];  // about 1.2 MB

// The three launches below use the kernels' default (not opted-in) dynamic shared memory, so the largest
// request an admitted shape can make must fit 48 KB: the Notify scratch with the count matrix staged
// (R*E <= NOTIFY_STAGE_MAX entries plus one padding column per expert), and the per-warp counters of a tile.
static_assert((2 * NOALLOC_MAX_E + 1 + 33 + NOTIFY_STAGE_MAX + NOALLOC_MAX_E) * sizeof(int32_t) <= 48 * 1024,
              "Notify scratch of the no-alloc entry point exceeds the default shared-memory limit");
static_assert(PLAN_WARPS * NOALLOC_MAX_E * sizeof(int32_t) <= 48 * 1024,
              "tile counters of the no-alloc entry point exceed the default shared-memory limit");

constexpr int NOALLOC_MAX_DEVICES = 64;
// Device address of the array, per device; nullptr = not looked up yet.  Atomics: host threads that make
// the first call on a device at the same time all store the same address.
std::atomic<NoallocScratch*> g_noalloc_ptr[NOALLOC_MAX_DEVICES];

// In host code g_noalloc_scratch is only a handle for the runtime, not a device address, so the
// address each device uses is looked up once, with that device current.
NoallocScratch* noalloc_scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return nullptr;
  NoallocScratch* sc = g_noalloc_ptr[dev].load(std::memory_order_acquire);
  if (sc == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return nullptr;
    }
    sc = static_cast<NoallocScratch*>(p);
    g_noalloc_ptr[dev].store(sc, std::memory_order_release);
  }
  return sc;
}

}  // namespace

extern "C" moe_status_t moe_slots_noalloc(const int32_t* topk_idx, int32_t T, int32_t K, int32_t E, int32_t R,
                                          const int32_t* rank_tok_start, int64_t capacity_rows, int32_t* slots,
                                          int32_t* n_recv, int32_t* status, void* stream) {
  if (T < 0 || K < 1 || K > MOE_MAX_K || E < 1 || R < 1 || E % R != 0 || capacity_rows < 0) return MOE_ERR_INVALID_ARG;
  if (E > NOALLOC_MAX_E || R > NOALLOC_MAX_R || (int64_t)T * K > NOALLOC_MAX_BRANCHES) {
    std::fprintf(stderr,
                 "moe_slots_noalloc: T*K=%lld, E=%d, R=%d exceed the built-in scratch (T*K <= %d, E <= %d, R <= %d); "
                 "use moe_plan + moe_slots with a caller workspace instead\n",
                 (long long)T * K, E, R, NOALLOC_MAX_BRANCHES, NOALLOC_MAX_E, NOALLOC_MAX_R);
    return MOE_ERR_INVALID_ARG;
  }
  if ((int64_t)R * capacity_rows >= (int64_t)1 << 31) return MOE_ERR_INVALID_ARG;
  if (n_recv == nullptr || status == nullptr || (T > 0 && (topk_idx == nullptr || slots == nullptr)))
    return MOE_ERR_INVALID_ARG;
  if (rank_tok_start == nullptr && T % R != 0) return MOE_ERR_INVALID_ARG;
  if (rank_tok_start != nullptr) {
    if (rank_tok_start[0] != 0 || rank_tok_start[R] != T) return MOE_ERR_INVALID_ARG;
    for (int r = 0; r < R; ++r)
      if (rank_tok_start[r + 1] < rank_tok_start[r]) return MOE_ERR_INVALID_ARG;
  }
  NoallocScratch* sc = noalloc_scratch_for_current_device();
  if (sc == nullptr) return MOE_ERR_CUDA;

  const int tile_branches = ROUNDS_DECODE * PLAN_THREADS;
  RankMap map;
  std::memset(&map, 0, sizeof(map));
  map.R = R;
  map.uniform_tokens = (rank_tok_start == nullptr && T > 0) ? T / R : 0;
  while ((1 << map.tile_shift) < tile_branches) ++map.tile_shift;
  int32_t tiles = 0;
  for (int r = 0; r <= R; ++r) {
    const int32_t tok = rank_tok_start != nullptr ? rank_tok_start[r] : (int32_t)((int64_t)T / R * r);
    map.tok_start[r] = tok;
    map.tile_start[r] = tiles;
    if (r < R) {
      const int32_t next = rank_tok_start != nullptr ? rank_tok_start[r + 1] : (int32_t)((int64_t)T / R * (r + 1));
      tiles += (int32_t)(((int64_t)(next - tok) * K + tile_branches - 1) / tile_branches);
    }
  }

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left; only the control words and the caller's
  // status word must start at zero, everything else is fully rewritten before it is read.
  if (cudaMemsetAsync(&sc->ctl, 0, sizeof(Control), st) != cudaSuccess ||
      cudaMemsetAsync(status, 0, sizeof(int32_t), st) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (tiles > 0)
    plan_tile_kernel<ROUNDS_DECODE><<<tiles, PLAN_THREADS, PLAN_WARPS * E * (int)sizeof(int32_t), st>>>(
        topk_idx, map, K, E, sc->tile_rank, sc->tile_hist, status);
  plan_scan_kernel<<<R, PLAN_THREADS, notify_smem_ints(E, R) * (int)sizeof(int32_t), st>>>(
      sc->tile_hist, map, E, 0, 1, sc->M, sc->c_rank, sc->o, sc->n_exp, n_recv, &sc->ctl, PLAN_TICKET, 0);
  RowArgs a = {};   // every field the kernel is handed has a defined value
  a.topk_idx = topk_idx;
  a.small_off = sc->tile_rank;
  a.small_out = nullptr;
  a.slot_out = nullptr;
  a.slot_in = nullptr;
  a.tile_base = sc->tile_hist;
  a.large_off = sc->o;
  a.n_recv = n_recv;
  a.status = status;
  a.C = capacity_rows;
  a.T = T;
  a.K = K;
  a.E = E;
  a.R = R;
  a.E_r = E / R;
  a.H16 = 0;
  a.work = nullptr;
  a.work_done = nullptr;
  a.granule = 1;
  a.items_per_row = 0;
  a.n_items = 0;
  a.n_head = 0;
  a.head_rows = 0;
  a.tail_granule = 1;
  a.tail_items_per_row = 1;
  a.win_base = nullptr;
  a.scale_base = nullptr;
  a.prefetch_meta = 0;
  a.static_first = 0;
  a.t_begin = 0;
  a.t_count = T;
  a.wait_limit_ms = WAIT_LIMIT_MS_DEFAULT;
  a.test_starve = 0;
  int grid = (int)(((int64_t)T * K + 255) / 256);
  if (grid < 1) grid = 1;
  slots_kernel<<<grid, 256, 0, st>>>(slots, a, map);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
