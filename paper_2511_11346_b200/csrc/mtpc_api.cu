// Host side of the C ABI declared in include/mtpc.h: argument checks, workspace carving, TMA descriptor
// encoding and kernel launches. Every step of the path runs in the kernels of this library; there is no CPU
// or library fallback.
#include <cuda.h>
#include <cuda_runtime.h>
#include <initializer_list>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "../../include/mtpc.h"
#include "mtpc_backward.cuh"
#include "mtpc_circuit.cuh"
#include "mtpc_decode.cuh"
#include "mtpc_gemm.cuh"
#include "mtpc_lowrank.cuh"
#include "mtpc_lowrank_gemm.cuh"

namespace {

using namespace mtpc;

constexpr size_t kAlign = 256;
constexpr int kMaxPhases = 5;
constexpr size_t kSlotSmemLimit = 160 * 1024;   // latent-draw tables of the draft slot kernel kept in shared memory up to this
constexpr int kMaxDraftVocab = 512;     // many-position draft: the v logits of a unit live in 512 TMEM columns
constexpr int kHostChunkPositions = 2048;   // host-buffer calls upload and process this many positions at a time
constexpr int kWorkCounterWord = 16;   // word of the 256-byte status area used as the circuit kernels' work counter
constexpr int kSmemLimit = 232448;   // 227 KB of dynamic shared memory per CTA on sm_100
// Hidden states of one rasterisation block of the projection kernel: small enough to stay L2-resident next to the
// weight tiles streaming past (data read by all SMs ends up in both halves of the 126 MB L2).
constexpr size_t kHiddenBlockBytes = 36u << 20;
// Many-position draft, sampling pass grouped by unit: hidden states staged per (window, slot) pair, at most this much
// at a time (longer calls are processed in chunks of positions).
constexpr size_t kGroupStageBytes = 1u << 30;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

// How one launch of the projection kernel tiles the N axis and uses shared / tensor memory.
struct Tiling {
  int tile_cols;        // accumulator width of an emission tile
  int group_units;      // emission units per work group
  int group_tiles;      // tiles of a full group
  int num_groups;       // groups covering all n*r units
  int slot_stride, num_slots, stages, stage_bytes, smem;
  int pair_stages, pair_stage_bytes, pair_smem;   // the same ring when two CTAs share every MMA (half a weight tile per CTA)
};

struct Layout {
  // derived sizes
  int S, sum_rows, sum_cols, sum_tiles;
  Tiling lp;            // log-likelihood mode: 256-column tiles over the flattened (i,k,b) axis
  Tiling sm;            // sampling mode: one unit per group, equal tiles of <= 256 columns
  size_t max_windows;
  // workspace offsets (bytes)
  size_t off_status, off_wemit, off_wsum, off_hidden, off_logA, off_G, off_logw, off_sel, off_logits, off_unit_lse;
  size_t off_prefix, off_partial, off_sum_bias;   // training loss: prefix log-marginals [max_positions, n], per-sequence terms
  int decode_max_p;     // positions the few-position draft path can take (0: path not available)
  bool can_draft;       // v <= 512: the sampling kernels hold a whole input unit on chip
  bool can_draft_many;  // the sampling epilogue of the projection kernel can tile a unit (draft of more than 128 positions)
  bool sample_two_pass; // ... but only by streaming the unit's tiles through tensor memory twice (v > 512): draws sorted by unit
  size_t off_h_hidden, off_h_targets, off_h_uniforms, off_h_bytes, off_h_out;
  // grouped sampling pass of the many-position draft (0 entries: not available)
  size_t group_entries;   // (window, slot) pairs that can be staged at once
  size_t off_grp_ints, off_grp_tiles, off_grp_perm, off_grp_stage;
  // acceptance stage after a many-position draft: first rejected slot and staging row per window, the recomputed logits
  // [accept_rows, r v] and unit log-sum-exps [accept_rows, r] of that slot
  size_t accept_rows;     // windows that can be handled at once (0: not available)
  size_t off_acc_rej, off_acc_row, off_acc_logits, off_acc_lse;
  size_t total;
};

int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

// Shared-memory ring and TMEM slots for tiles of `tile_cols` emission columns and `sum_cols` sum columns.
bool fit_tiling(Tiling* t, int sum_cols) {
  const int widest = t->tile_cols > sum_cols ? t->tile_cols : sum_cols;
  t->slot_stride = (widest + 31) / 32 * 32;
  t->num_slots = kTmemCols / t->slot_stride;
  if (t->num_slots > kMaxSlots) t->num_slots = kMaxSlots;
  t->stage_bytes = (kABytes + widest * kBlockK * 2 + 1023) / 1024 * 1024;   // A tile + one B tile
  const int ctl = 1024 + static_cast<int>(sizeof(GemmControl));
  int stages = (kSmemLimit - ctl) / t->stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  t->stages = stages;
  t->smem = stages * t->stage_bytes + ctl;
  t->pair_stage_bytes = (kABytes + widest / 2 * kBlockK * 2 + 1023) / 1024 * 1024;   // A tile + half a B tile
  t->pair_stages = (kSmemLimit - ctl) / t->pair_stage_bytes;
  if (t->pair_stages > kMaxStages) t->pair_stages = kMaxStages;
  t->pair_smem = t->pair_stages * t->pair_stage_bytes + ctl;
  return stages >= 2 && t->num_slots >= 2;
}

int plan(const mtpc_config& c, Layout* L) {
  if (c.family < MTPC_CP || c.family > MTPC_BTREE) return MTPC_ERR_SHAPE;
  if (c.io_dtype != MTPC_F32 && c.io_dtype != MTPC_BF16) return MTPC_ERR_SHAPE;
  if (c.n < 1 || c.r < 1 || c.v < 1 || c.d < 1 || c.max_positions < 1 || c.max_windows_per_pos < 1)
    return MTPC_ERR_SHAPE;
  if ((c.flags & ~MTPC_FLAG_HMM_CONTEXTUAL) != 0) return MTPC_ERR_UNSUPPORTED;
  const bool ctx = (c.flags & MTPC_FLAG_HMM_CONTEXTUAL) != 0;
  if (ctx && c.family != MTPC_HMM) return MTPC_ERR_UNSUPPORTED;
  if (c.n > 64 || c.max_windows_per_pos > 64) return MTPC_ERR_UNSUPPORTED;
  if (!is_pow2(c.r) || c.r > 128) return MTPC_ERR_UNSUPPORTED;
  if (c.family != MTPC_CP && c.r > 32) return MTPC_ERR_UNSUPPORTED;
  if (c.family == MTPC_BTREE && (c.n < 2 || !is_pow2(c.n))) return MTPC_ERR_UNSUPPORTED;
  if (c.d % kBlockK != 0) return MTPC_ERR_UNSUPPORTED;
  if (c.v % 16 != 0) return MTPC_ERR_UNSUPPORTED;
  if (c.v_valid != 0 && (c.v_valid > c.v || c.v_valid <= c.v - 16)) return MTPC_ERR_SHAPE;
  if (static_cast<int64_t>(c.n) * c.r * c.v > (1ll << 30)) return MTPC_ERR_SHAPE;

  L->S = (c.family == MTPC_BTREE) ? 1 + (c.n - 2) * c.r : (ctx ? 1 + (c.n - 1) * c.r : 1);
  L->sum_rows = L->S * c.r;
  // sum tile: a multiple of both r and 16, at most 256 columns
  const int unit = c.r > 16 ? c.r : 16;
  int sum_cols = (L->sum_rows + unit - 1) / unit * unit;
  if (sum_cols > 256) sum_cols = 256 / unit * unit;
  L->sum_cols = sum_cols;
  L->sum_tiles = (L->sum_rows + sum_cols - 1) / sum_cols;
  const int emit_units = c.n * c.r;
  // sampling: emission unit -> equal tiles of <= 256 columns, each a multiple of 16, all in TMEM at once
  // (a unit of more than 512 symbols does not fit tensor memory: such heads draft through the few-position path only)
  L->can_draft = true;
  L->sample_two_pass = c.v > kMaxDraftVocab;
  if (!L->sample_two_pass) {
    int chunks = (c.v + 255) / 256;
    while (c.v % chunks != 0 || (c.v / chunks) % 16 != 0) ++chunks;
    L->sm.tile_cols = c.v / chunks;
    L->sm.group_units = 1;
    L->sm.group_tiles = chunks;
    L->sm.num_groups = emit_units;
    // (no such split, e.g. v = 272 = 17 x 16: only the few-position draft path, which needs none, is available)
    L->can_draft_many = fit_tiling(&L->sm, sum_cols) && L->sm.num_slots >= chunks;
  } else {
    // 256-column tiles, the last one ragged (its tail columns are masked), streamed through two accumulator slots
    L->sm.tile_cols = 256;
    L->sm.group_units = 1;
    L->sm.group_tiles = (c.v + 255) / 256;
    L->sm.num_groups = emit_units;
    L->can_draft_many = fit_tiling(&L->sm, sum_cols);
  }
  if (!L->can_draft_many) memset(&L->sm, 0, sizeof(L->sm));
  // log-likelihood: 256-column tiles; a group is the shortest run of whole units that is a whole number of tiles
  const int lcm = c.v / gcd_int(c.v, 256) * 256;
  L->lp.tile_cols = 256;
  L->lp.group_units = lcm / c.v;
  L->lp.group_tiles = lcm / 256;
  if (L->lp.group_units > emit_units) {   // fewer units than one full group: a single, partial group
    L->lp.group_units = emit_units;
    L->lp.group_tiles = (emit_units * c.v + 255) / 256;
  }
  L->lp.num_groups = (emit_units + L->lp.group_units - 1) / L->lp.group_units;
  if (!fit_tiling(&L->lp, sum_cols)) return MTPC_ERR_UNSUPPORTED;

  L->max_windows = static_cast<size_t>(c.max_positions) * c.max_windows_per_pos;
  const size_t elt = c.io_dtype == MTPC_F32 ? 4 : 2;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  L->off_status = take(256);
  const bool f32 = c.io_dtype == MTPC_F32;
  L->off_wemit = take(f32 ? static_cast<size_t>(c.n) * c.r * c.v * c.d * 2 : 0);
  L->off_wsum = take(f32 ? static_cast<size_t>(L->sum_rows) * c.d * 2 : 0);
  L->off_hidden = take(f32 ? static_cast<size_t>(c.max_positions) * c.d * 2 : 0);
  L->off_logA = take(c.family == MTPC_HMM && !ctx ? static_cast<size_t>(c.n - 1) * c.r * c.r * 4 : 0);
  L->off_sum_bias = take(ctx ? static_cast<size_t>(L->sum_rows) * 4 : 0);
  L->off_G = take(L->max_windows * c.n * c.r * 4);
  L->off_logw = take(static_cast<size_t>(c.max_positions) * L->sum_rows * 4);
  L->off_sel = take(L->max_windows * c.n * 4);
  // (latents of more than 32 values are handled for the mixture only; HMM and BTree are limited to r <= 32 anyway)
  L->decode_max_p = L->can_draft ? (c.max_positions < kDecodeMaxP ? c.max_positions : kDecodeMaxP) : 0;
  L->off_logits = take(static_cast<size_t>(L->decode_max_p) * emit_units * c.v * 4);
  L->off_unit_lse = take(static_cast<size_t>(L->decode_max_p) * emit_units * 4);
  L->off_prefix = take(static_cast<size_t>(c.max_positions) * c.n * 4);
  L->off_partial = take(static_cast<size_t>(c.max_positions) * c.n * 4);
  L->off_h_hidden = take(static_cast<size_t>(c.max_positions) * c.d * elt);
  L->off_h_targets = take(static_cast<size_t>(c.max_positions) * c.n * 4);
  L->off_h_uniforms = take(L->max_windows * 2 * c.n * 4);
  L->off_h_bytes = take(L->max_windows * c.n * 4);
  L->off_h_out = take(L->max_windows * 4);
  // grouped sampling: only heads that can be asked for a many-position draft carry the staging area
  L->group_entries = 0;
  if (L->can_draft_many && c.max_positions > L->decode_max_p && emit_units <= kGroupMaxUnits) {
    const size_t cap = kGroupStageBytes / (static_cast<size_t>(c.d) * 2);
    const size_t all = L->max_windows * c.n;
    L->group_entries = all < cap ? all : cap;
    if (L->group_entries < static_cast<size_t>(c.max_windows_per_pos) * c.n) L->group_entries = 0;   // not even one position
  }
  const size_t ge = L->group_entries;
  L->off_grp_ints = take(ge ? (3 * static_cast<size_t>(emit_units) + 64) * 4 : 0);     // counts | cursors | offsets | tile count
  L->off_grp_tiles = take(ge ? (emit_units + ge / 128 + 1) * sizeof(GroupTile) : 0);
  L->off_grp_perm = take(ge * 4);
  L->off_grp_stage = take(ge * c.d * 2);
  L->accept_rows = 0;
  if (ge > 0) {
    const size_t cap = kGroupStageBytes / (static_cast<size_t>(c.r) * c.v * 4);
    L->accept_rows = L->max_windows < cap ? L->max_windows : cap;
    if (L->accept_rows > ge) L->accept_rows = ge;                               // they share the staging rows
    if (L->accept_rows < static_cast<size_t>(c.max_windows_per_pos)) L->accept_rows = 0;
  }
  const size_t ar = L->accept_rows;
  L->off_acc_rej = take(ar ? L->max_windows * 4 : 0);
  L->off_acc_row = take(ar ? L->max_windows * 4 : 0);
  L->off_acc_logits = take(ar * c.r * c.v * 4);
  L->off_acc_lse = take(ar * c.r * 4);
  L->total = off;
  return MTPC_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 matrix [rows, cols] row-major (row pitch `pitch` elements, 0 = cols) -> tiles of box_rows x 64 elements,
// 128-byte swizzle, zero fill outside.
int make_tmap(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint64_t pitch = 0) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return MTPC_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return MTPC_ERR_WORKSPACE;
  if (pitch == 0) pitch = cols;
  if ((pitch * 2) % 16 != 0) return MTPC_ERR_WORKSPACE;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {pitch * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(kBlockK), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MTPC_OK : MTPC_ERR_CUDA;
}

// bf16 matrix [rows, cols] row-major read as an MN-major operand (its columns are the operand's M or N index, its rows
// the K index): boxes of 64 columns x 64 rows, 128-byte swizzle, zero fill outside.
int make_tmap_mn(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return MTPC_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0 || (pitch * 2) % 16 != 0) return MTPC_ERR_WORKSPACE;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {pitch * 2};
  cuuint32_t box[2] = {64, static_cast<cuuint32_t>(kBlockK)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MTPC_OK : MTPC_ERR_CUDA;
}

}  // namespace

struct mtpc_head {
  mtpc_config cfg;
  Layout L;
  uint8_t* ws;
  const void* W_emit_bf16;
  const void* W_sum_bf16;
  CUtensorMap tm_emit_lp, tm_emit_sm, tm_sum;   // W_emit with the box of either tiling; W_sum
  CUtensorMap tm_emit_lp2, tm_emit_sm2, tm_sum2; // the same with boxes of half the rows: what one CTA of a pair stages
  int projection_variant;                       // 0: chosen per launch; 1: every CTA alone; 2: CTA pairs (cta_group::2)
  int draft_grouping;                           // many-position draft: 0 chosen per call; 1 never sort the draws by unit; 2 always
  // factored low-rank head (App. G; mtpc_create_head_lowrank): rank k > 0, no composed W_emit
  int lr_k;
  const void* lr_W_base;                        // [n, v, d] bf16
  const void* lr_A;                             // [n, r, v, k] bf16
  const void* lr_B;                             // [n, r, k, d] bf16
  size_t lr_off_arep;                           // workspace: A as [n, v, r, k]
  size_t lr_off_dec;                            // workspace: few-position draft products base [P, n v] | z [P, n r k]
  size_t lr_off_base;                           // workspace: long drafts: W_base h [T, n v] fp32 (0: not reserved)
  CUtensorMap tm_lrB_dec;                       // B [n r k, d] for the few-position draft path
  size_t lr_off_zhl, lr_off_partial;            // workspace: z = B h as bf16 halves [T, n r, 2, k]; per-panel partial log-sum-exps
  LowRankGemmParams lr_params;                  // everything of the factored projection launch that does not depend on the call
  int max_pairs;                                // clusters of two projection CTAs that can be resident at once
  CUtensorMap tm_emit_dec, tm_sum_dec;          // the same matrices in the few-position draft path's tiles
  int decode_tile_rows, decode_sum_tile_rows;
  int num_sms;
  cudaStream_t copy_stream; // host-buffer calls: uploads run here, ahead of the kernels (created on first use)
  cudaEvent_t* copy_events; // [copy_event_count]: "chunk c is on the device"; [0] doubles as "the call may start"
  int copy_event_count;
  int draft_P;              // positions whose draft state (logits, or after a many-position draft G and log omega) is in the workspace (0: none)
  int draft_wpp;            // windows per position of that draft
  const void* draft_hidden; // many-position draft: the bf16 hidden states it read (the acceptance stage stages rows of them)
  int ring;                 // calls whose per-kernel events are retained (0 = timing off)
  cudaEvent_t* ev;          // [ring][kMaxPhases][2]
  int* ring_phases;         // [ring] phases recorded by the call in that slot
  uint64_t calls;           // timed calls so far
  uint64_t launches;
  uint64_t wait_limit_ns;   // limit of the pipeline waits inside the tcgen05 kernels (kWaitLimitNs; a test may shorten it)
};

namespace {

template <typename T>
T* at(mtpc_head* h, size_t off) { return reinterpret_cast<T*>(h->ws + off); }

int valid_symbols(const mtpc_config& c) { return c.v_valid > 0 ? c.v_valid : c.v; }
bool is_ctx(const mtpc_head* h) { return (h->cfg.flags & MTPC_FLAG_HMM_CONTEXTUAL) != 0; }
// HMM transition log-probabilities as the kernels read them: position p's tables start at base + p * stride.
// Static transitions: one set in the workspace, stride 0. Contextual (App. H): the sum units after the first one
// in every position's row of log omega.
const float* hmm_tables(mtpc_head* h) {
  return is_ctx(h) ? at<float>(h, h->L.off_logw) + h->cfg.r : at<float>(h, h->L.off_logA);
}
int hmm_table_stride(const mtpc_head* h) { return is_ctx(h) ? h->L.sum_rows : 0; }
const float* sum_bias(mtpc_head* h) { return is_ctx(h) ? at<float>(h, h->L.off_sum_bias) : nullptr; }

struct PhaseTimer {
  mtpc_head* h;
  cudaStream_t st;
  int idx, slot;
  PhaseTimer(mtpc_head* head, cudaStream_t s) : h(head), st(s), idx(0), slot(0) {
    if (h->ring > 0) {
      slot = static_cast<int>(h->calls % h->ring);
      h->ring_phases[slot] = 0;
      h->calls++;
    }
  }
  cudaEvent_t* pair() { return h->ev + (static_cast<size_t>(slot) * kMaxPhases + idx) * 2; }
  void begin() { if (h->ring > 0 && idx < kMaxPhases) cudaEventRecord(pair()[0], st); }
  void end() {
    if (h->ring > 0 && idx < kMaxPhases) {
      cudaEventRecord(pair()[1], st);
      h->ring_phases[slot] = idx + 1;
    }
    ++idx;
  }
};

int check_launch() { return cudaGetLastError() == cudaSuccess ? MTPC_OK : MTPC_ERR_CUDA; }

// Launch `kernel`, optionally allowed to start before the kernel ahead of it in the stream has finished (programmatic
// dependent launch): such a kernel calls grid_dependency_wait() before it touches the earlier kernel's results.
template <typename... Params, typename... Args>
void launch_kernel(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool dependent,
                   Args&&... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

// Launch the projection kernel for `rows` positions over the emission groups (with_emit) and / or the sum tiles.
// Units per work item of the log-likelihood mode. An item covers its units with 256-column tiles; unless the
// units end on a tile boundary the last tile is partly wasted (its tail belongs to the next item, which recomputes it).
// Items are dealt round-robin to `ctas` persistent CTAs, so a launch takes about rounds x tiles-per-item tile times:
// pick the count that minimises that (v = 320: 4 units = 5 tiles, nothing wasted; v = 272: 8 units = 9 tiles, 6 % wasted
// but twice as many items as the waste-free 16 units = 17 tiles).
int choose_group_units(int v, int emit_units, int m_tiles, int ctas) {
  int best = 1;
  long long best_cost = -1;
  const int limit = emit_units < 64 ? emit_units : 64;
  for (int u = 1; u <= limit; ++u) {
    const long long tiles = (static_cast<long long>(u) * v + 255) / 256;
    const long long groups = (emit_units + u - 1) / u;
    const long long rounds = (groups * m_tiles + ctas - 1) / ctas;
    const long long cost = rounds * tiles;
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = u; }
  }
  return best;
}

struct GroupArgs {           // grouped sampling pass: the staged hidden states and their tiles (mtpc_group.cuh)
  const void* stage = nullptr;
  int entries = 0;                           // rows of the staging buffer in use
  const GroupTile* tiles = nullptr;
  const int* num_tiles = nullptr;
  const int* perm = nullptr;
  const int* unit_sel = nullptr;             // this chunk's rows of the selected units
  int max_tiles = 0;
  bool by_slot = false;                      // rows sorted by slot; the kernel writes the slot's logits (acceptance stage)
};

struct GradArgs {            // what the projection kernel keeps for the backward pass (training calls only)
  float* lse_out = nullptr;                  // the units' log-sum-exps [T, n, r]
  float* logit_out = nullptr;                // the emission logits [T, n r v] fp32
  size_t logit_pitch = 0;
};

int launch_gemm(mtpc_head* h, int mode, const void* hidden_bf16, int rows, int wpp, bool with_emit, bool with_sum,
                const int* targets, const float* uniforms, int* out_bytes, cudaStream_t st,
                const GradArgs* ga = nullptr, bool targets_are_drafts = false, const GroupArgs* grp = nullptr) {
  if (rows <= 0 || (!with_emit && !with_sum)) return MTPC_OK;
  const mtpc_config& c = h->cfg;
  const Layout& L = h->L;
  const Tiling& tl = mode == kModeSample ? L.sm : L.lp;
  if (grp != nullptr && (grp->by_slot ? mode != kModeLogprob : mode != kModeSample)) return MTPC_ERR_SHAPE;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  if (ga) {
    p.lse_out = ga->lse_out;
    p.logit_out = ga->logit_out;
    p.logit_pitch = ga->logit_pitch;
  }
  int rc = grp ? make_tmap(&p.tm_a, grp->stage, static_cast<uint64_t>(grp->entries), static_cast<uint64_t>(c.d), kBlockM)
               : make_tmap(&p.tm_a, hidden_bf16, static_cast<uint64_t>(rows), static_cast<uint64_t>(c.d), kBlockM);
  if (rc != MTPC_OK) return rc;
  p.tm_emit = mode == kModeSample ? h->tm_emit_sm : h->tm_emit_lp;
  p.tm_sum = h->tm_sum;
  p.T = rows;
  p.m_tiles = (rows + kBlockM - 1) / kBlockM;
  // Two CTAs per MMA when there are at least two m-tiles to pair up (and the device can hold a cluster at all)
  const bool pair = grp == nullptr &&
                    (h->projection_variant == 2 || (h->projection_variant == 0 && p.m_tiles >= 2 && h->max_pairs > 0));
  const int ctas = pair ? 2 : 1;
  const int workers = pair ? h->max_pairs : h->num_sms;               // CTAs, or CTA pairs, resident at once
  p.m_units = (p.m_tiles + ctas - 1) / ctas;
  p.kblocks = c.d / kBlockK;
  {
    const size_t unit_bytes = static_cast<size_t>(kBlockM) * ctas * c.d * 2;
    const int cap_units = kHiddenBlockBytes / unit_bytes > 0 ? static_cast<int>(kHiddenBlockBytes / unit_bytes) : 1;
    const int nblocks = (p.m_units + cap_units - 1) / cap_units;
    p.m_block = (p.m_units + nblocks - 1) / nblocks;
  }
  p.n = c.n; p.r = c.r; p.v = c.v;
  p.vv = valid_symbols(c);
  p.emit_units = c.n * c.r;
  p.num_groups = with_emit ? tl.num_groups : 0;
  p.group_units = tl.group_units;
  if (mode != kModeSample && with_emit) {
    p.group_units = choose_group_units(c.v, p.emit_units, p.m_units, workers);
    p.num_groups = (p.emit_units + p.group_units - 1) / p.group_units;
  }
  p.tile_cols = tl.tile_cols;
  p.num_sum_tiles = with_sum ? L.sum_tiles : 0;
  p.sum_cols = L.sum_cols;
  p.sum_rows = L.sum_rows;
  p.slot_stride = tl.slot_stride;
  p.num_slots = tl.num_slots;
  p.stages = pair ? tl.pair_stages : tl.stages;
  p.stage_bytes = pair ? tl.pair_stage_bytes : tl.stage_bytes;
  if (pair) {
    p.tm_emit = mode == kModeSample ? h->tm_emit_sm2 : h->tm_emit_lp2;
    p.tm_sum = h->tm_sum2;
  }
  p.wpp = wpp;
  p.targets = targets;
  p.missing_is_nan = targets_are_drafts ? 1 : 0;
  p.G = at<float>(h, L.off_G);
  p.logw = at<float>(h, L.off_logw);
  p.sum_bias = sum_bias(h);
  p.unit_sel = at<int>(h, L.off_sel);
  if (grp) {
    p.group_tiles = grp->tiles;
    p.group_num_tiles = grp->num_tiles;
    p.group_perm = grp->perm;
    p.group_two_pass = (L.sample_two_pass && !grp->by_slot) ? 1 : 0;
    p.unit_sel = grp->unit_sel;
  }
  p.uniforms = uniforms;
  p.out_bytes = out_bytes;
  p.status = at<unsigned>(h, L.off_status);
  p.wait_limit_ns = h->wait_limit_ns;
  const long long items = grp ? grp->max_tiles : static_cast<long long>(p.m_units) * (p.num_groups + p.num_sum_tiles);
  const int grid = ctas * static_cast<int>(items < workers ? items : workers);
  const size_t smem = pair ? tl.pair_smem : tl.smem;
  if (grp && grp->by_slot) {
    mtpc_gemm_kernel<kModeLogitsGrouped, 1><<<grid, kGemmThreads, smem, st>>>(p);
  } else if (grp) {
    mtpc_gemm_kernel<kModeSampleGrouped, 1><<<grid, kGemmThreads, smem, st>>>(p);
  } else if (!pair) {
    if (mode == kModeLogprob)
      mtpc_gemm_kernel<kModeLogprob, 1><<<grid, kGemmThreads, smem, st>>>(p);
    else
      mtpc_gemm_kernel<kModeSample, 1><<<grid, kGemmThreads, smem, st>>>(p);
  } else {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (mode == kModeLogprob) cudaLaunchKernelEx(&cfg, mtpc_gemm_kernel<kModeLogprob, 2>, p);
    else cudaLaunchKernelEx(&cfg, mtpc_gemm_kernel<kModeSample, 2>, p);
  }
  h->launches++;
  return check_launch();
}

// Shared memory of one CTA of the binary-tree circuit kernel (see circuit_btree_kernel).
size_t hmm_stream_smem_bytes(int r) { return static_cast<size_t>(kCircuitWarps) * (kHmmDepth * r * r + 32) * sizeof(float); }
size_t btree_smem_bytes(int n, int r, bool with_prefix) {
  return static_cast<size_t>(kCircuitWarps) * btree_warp_floats(n, r, with_prefix) * sizeof(float);
}

// Circuit evaluation of W windows: out[w] = joint log-prob (may be NULL when prefix is given); prefix (may be NULL)
// [W, n] = log-marginals of the prefixes x_0..x_i.
// dependent: the launch directly follows draft_slot_kernel, which has zeroed the work counter, and may overlap its tail.
int launch_circuit(mtpc_head* h, int W, int wpp, float* out, float* prefix, cudaStream_t st, bool dependent = false,
                   bool raw_mixture = false) {
  if (W <= 0) return MTPC_OK;
  const mtpc_config& c = h->cfg;
  const Layout& L = h->L;
  const float* G = at<float>(h, L.off_G);
  const float* logw = at<float>(h, L.off_logw);
  const int blocks = (W + kCircuitWarps - 1) / kCircuitWarps;
  const int threads = kCircuitWarps * 32;
  // kernels that stream per-position tables hand out windows through a counter next to the status word
  unsigned* counter = at<unsigned>(h, L.off_status) + kWorkCounterWord;
  const int resident = blocks < 8 * h->num_sms ? blocks : 8 * h->num_sms;   // more CTAs than an SM can hold do no harm
  if (!dependent && (c.family == MTPC_BTREE || c.family == MTPC_HMM)) {
    if (cudaMemsetAsync(counter, 0, sizeof(unsigned), st) != cudaSuccess) return MTPC_ERR_CUDA;
  }
  if (c.family == MTPC_CP) {
    launch_kernel(circuit_cp_kernel, blocks, threads, 0, st, dependent, G, logw, out, prefix, W, wpp, c.n, c.r, L.sum_rows,
                  raw_mixture ? 1 : 0);
  } else if (c.family == MTPC_HMM) {
    launch_kernel(circuit_hmm_stream_kernel, resident, threads, hmm_stream_smem_bytes(c.r), st, dependent, G, logw,
                  hmm_tables(h), hmm_table_stride(h), out, prefix, counter, W, wpp, c.n, c.r, L.sum_rows);
  } else if (prefix != nullptr) {
    launch_kernel(circuit_btree_kernel<true>, resident, threads, btree_smem_bytes(c.n, c.r, true), st, dependent, G, logw,
                  out, prefix, counter, W, wpp, c.n, c.r, L.sum_rows);
  } else {
    launch_kernel(circuit_btree_kernel<false>, resident, threads, btree_smem_bytes(c.n, c.r, false), st, dependent, G,
                  logw, out, static_cast<float*>(nullptr), counter, W, wpp, c.n, c.r, L.sum_rows);
  }
  h->launches++;
  return check_launch();
}

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the function, not to a head or a call: whoever sets it last
// wins. So every kernel that may ask for more than 48 KB gets the device's full limit, once and for all, and heads of
// different shapes (or a head and the static entry point) cannot lower it under each other.
template <typename K>
bool allow_full_smem(K kernel) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) == cudaSuccess;
}
bool set_circuit_attributes() {
  bool ok = allow_full_smem(circuit_hmm_stream_kernel);
  ok &= allow_full_smem(circuit_btree_kernel<false>);
  ok &= allow_full_smem(circuit_btree_kernel<true>);
  return ok;
}

// How many clusters of two projection CTAs the device holds at once (0: none, the single-CTA kernel is used).
int resident_pairs(int smem_bytes) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(2);
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, mtpc_gemm_kernel<kModeLogprob, 2>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return clusters;
}

// Rows per emission tile of the few-position draft path: the height in [64, 128] (multiple of 8) that leaves the
// least idle time when the tiles are dealt evenly to `ctas` persistent CTAs; ties go to the taller tile.
int decode_tile_rows(long long rows, int ctas) {
  int best = 128;
  double best_eff = 0.0;
  for (int tr = 128; tr >= 64; tr -= 8) {
    const long long tiles = (rows + tr - 1) / tr;
    const long long per_cta = (tiles + ctas - 1) / ctas;
    const double eff = static_cast<double>(rows) / (static_cast<double>(per_cta) * ctas * tr);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = tr; }
  }
  return best;
}

// Few-position draft path: one pass over all weight rows with the positions on the N axis.
int launch_decode_gemm(mtpc_head* h, const void* hidden_bf16, int P, cudaStream_t st) {
  const mtpc_config& c = h->cfg;
  const Layout& L = h->L;
  DecodeParams p;
  memset(&p, 0, sizeof(p));
  p.P = P;
  p.Ppad = (P + 15) / 16 * 16;
  int rc = make_tmap(&p.tm_h, hidden_bf16, static_cast<uint64_t>(P), static_cast<uint64_t>(c.d), p.Ppad);
  if (rc != MTPC_OK) return rc;
  p.tm_emit = h->tm_emit_dec;
  p.tm_sum = h->tm_sum_dec;
  p.kblocks = c.d / kBlockK;
  p.emit_rows = c.n * c.r * c.v;
  p.logits = at<float>(h, L.off_logits);
  if (h->lr_k > 0) {
    // a factored low-rank head streams W_base and B instead of the composed tensor: base = W_base h and z = B h, from
    // which lowrank_expand_kernel forms the logits
    p.tm_emit2 = h->tm_lrB_dec;
    p.emit_rows = c.n * c.v;
    p.emit2_rows = c.n * c.r * h->lr_k;
    p.logits = reinterpret_cast<float*>(h->ws + h->lr_off_dec);
    p.logits2 = p.logits + static_cast<size_t>(L.decode_max_p) * p.emit_rows;
  }
  p.sum_rows = L.sum_rows;
  p.r = c.r;
  p.tile_rows = h->decode_tile_rows;
  p.sum_tile_rows = h->decode_sum_tile_rows;
  p.tile_bytes = p.tile_rows * kBlockK * 2;
  p.emit_tiles = (p.emit_rows + p.tile_rows - 1) / p.tile_rows;
  p.emit2_tiles = (p.emit2_rows + p.tile_rows - 1) / p.tile_rows;
  p.sum_tiles = (p.sum_rows + p.sum_tile_rows - 1) / p.sum_tile_rows;
  p.tile_stride = (p.Ppad + 31) / 32 * 32;
  p.pass_tiles = kTmemCols / (2 * p.tile_stride);                     // two slots of pass_tiles accumulators
  if (p.pass_tiles > kDecodeMaxTiles) p.pass_tiles = kDecodeMaxTiles;
  // stage = weight tiles + hidden tile, padded so that a 128-row operand read from the last tile's base stays inside
  int stage = p.pass_tiles * p.tile_bytes + p.Ppad * kBlockK * 2;
  const int reach = (p.pass_tiles - 1) * p.tile_bytes + kABytes;
  if (stage < reach) stage = reach;
  p.stage_bytes = (stage + 1023) / 1024 * 1024;
  const int ctl = 1024 + static_cast<int>(sizeof(GemmControl));
  p.stages = (kSmemLimit - ctl) / p.stage_bytes;
  if (p.stages > kMaxStages) p.stages = kMaxStages;
  p.logw = at<float>(h, L.off_logw);
  p.sum_bias = sum_bias(h);
  p.status = at<unsigned>(h, L.off_status);
  p.wait_limit_ns = h->wait_limit_ns;
  const int tiles = p.emit_tiles + p.emit2_tiles + p.sum_tiles;
  const int grid = tiles < h->num_sms ? tiles : h->num_sms;
  mtpc_decode_gemm_kernel<<<grid, kGemmThreads, p.stages * p.stage_bytes + ctl, st>>>(p);
  h->launches++;
  if (h->lr_k > 0) {
    launch_kernel(lowrank_expand_kernel, dim3(c.n * c.r, (c.v + kExpandThreads - 1) / kExpandThreads), kExpandThreads,
                  static_cast<size_t>(P) * h->lr_k * sizeof(float), st, h->ring == 0, p.logits, p.logits2,
                  static_cast<const __nv_bfloat16*>(h->lr_A), at<float>(h, L.off_logits), P, c.n, c.r, c.v, h->lr_k);
    h->launches++;
  }
  return check_launch();
}

// hidden (io_dtype, device) -> bf16 device pointer the GEMM reads
int stage_hidden(mtpc_head* h, const void* hidden, int rows, const void** out_bf16, cudaStream_t st) {
  if (h->cfg.io_dtype == MTPC_BF16) { *out_bf16 = hidden; return MTPC_OK; }
  __nv_bfloat16* dst = at<__nv_bfloat16>(h, h->L.off_hidden);
  const size_t count = static_cast<size_t>(rows) * h->cfg.d;
  if (count) {
    const int blocks = static_cast<int>((count + 255) / 256 < 4096 ? (count + 255) / 256 : 4096);
    f32_to_bf16_kernel<<<blocks, 256, 0, st>>>(static_cast<const float*>(hidden), dst, count);
    h->launches++;
    if (check_launch() != MTPC_OK) return MTPC_ERR_CUDA;
  }
  *out_bf16 = dst;
  return MTPC_OK;
}

// One operand of a plain GEMM: a bf16 matrix in device memory, either [rows = M or N, K] with K contiguous (K-major) or
// [rows = K, M or N] with the M / N index contiguous (MN-major); pitch in elements.
struct GemmOperand {
  const void* ptr;
  size_t pitch;
  bool mn_major;
};

// Optional extras of a plain GEMM launch: bf16 output instead of fp32, and several products of one shape in a launch
// (see PlainGemmParams); a_* / b_* extents: the whole matrices the batched operands are windows of (M or N, then K).
struct PlainGemmExtra {
  void* C_bf16 = nullptr;
  int batches = 1, a_m_step = 0, a_k_step = 0, b_n_step = 0, b_k_step = 0;
  size_t c_step = 0;
  long long a_extent_m = 0, a_extent_k = 0, b_extent_n = 0, b_extent_k = 0;
};
int launch_plain_gemm(mtpc_head* h, GemmOperand A, GemmOperand B0, int K0, GemmOperand B1, int K1, int a_k1, float* C,
                      size_t ldc, int M, int N, cudaStream_t st, void* C_hilo = nullptr, int split_k = 0,
                      const PlainGemmExtra* extra = nullptr);
// parts: 1 = sum-unit tiles (log omega), 2 = z = B h and the repacked A, 4 = the factored kernel (and its merge)
int launch_lowrank_projection(mtpc_head* h, const void* hidden_bf16, int T, const int* targets, cudaStream_t st,
                              const GradArgs* ga = nullptr, int parts = 7, bool targets_are_drafts = false);

// out [T] (joint) and / or prefix [T, n] (prefix log-marginals); either may be NULL, not both.
int window_logprob_impl(mtpc_head* h, const void* hidden, const int32_t* targets, int32_t T, float* out, float* prefix,
                        cudaStream_t st) {
  const void* hb = nullptr;
  h->draft_P = 0;   // log omega of the last draft is overwritten below
  int rc = stage_hidden(h, hidden, T, &hb, st);
  if (rc != MTPC_OK) return rc;
  PhaseTimer pt(h, st);
  pt.begin();
  if (h->lr_k > 0) rc = launch_lowrank_projection(h, hb, T, targets, st);
  else rc = launch_gemm(h, kModeLogprob, hb, T, 1, true, true, targets, nullptr, nullptr, st);
  pt.end();
  if (rc != MTPC_OK) return rc;
  pt.begin();
  rc = launch_circuit(h, T, 1, out, prefix, st);
  pt.end();
  return rc;
}

// out_logprob [W] (joint) and / or out_prefix [W, n] (prefix log-marginals of the draft); either may be NULL, not both.
int draft_sample_impl(mtpc_head* h, const void* hidden, int32_t P, int32_t wpp, const float* uniforms,
                      int32_t* out_bytes, float* out_logprob, float* out_prefix, cudaStream_t st) {
  const mtpc_config& c = h->cfg;
  const Layout& L = h->L;
  const int W = P * wpp;
  if (!L.can_draft) return MTPC_ERR_UNSUPPORTED;
  if (h->lr_k > 0 && P > L.decode_max_p && wpp == 1 && c.v <= kMaxDraftVocab && h->lr_off_base != 0) {
    // A long draft on a factored head, one window per position: log omega, the latent draws, then every (window, slot)
    // forms the logits of its one selected unit from W_base h and B h (lowrank_draw_kernel) and draws its byte; the
    // evidence of the drafted bytes under every unit is the factored projection with them as targets. No logits are
    // kept: no acceptance stage after such a draft.
    const int k = h->lr_k;
    h->draft_P = 0;
    PhaseTimer pt(h, st);
    pt.begin();
    int rc = launch_lowrank_projection(h, hidden, P, nullptr, st, nullptr, /*parts=*/1 | 2);
    pt.end();
    if (rc != MTPC_OK) return rc;
    pt.begin();
    latent_sample_kernel<<<(W + 127) / 128, 128, 0, st>>>(c.family, at<float>(h, L.off_logw), hmm_tables(h), uniforms,
                                                          at<int>(h, L.off_sel), out_bytes, at<unsigned>(h, L.off_status), W,
                                                          wpp, c.n, c.r, L.sum_rows, hmm_table_stride(h));
    h->launches++;
    pt.end();
    if ((rc = check_launch()) != MTPC_OK) return rc;
    pt.begin();
    float* base = reinterpret_cast<float*>(h->ws + h->lr_off_base);
    rc = launch_plain_gemm(h, GemmOperand{hidden, static_cast<size_t>(c.d), false},
                           GemmOperand{h->lr_W_base, static_cast<size_t>(c.d), false}, c.d,
                           GemmOperand{h->lr_W_base, static_cast<size_t>(c.d), false}, 0, 0, base,
                           static_cast<size_t>(c.n) * c.v, P, c.n * c.v, st);
    if (rc != MTPC_OK) return rc;
    {
      const int pairs = W * c.n;
      int blocks = (pairs + kDrawWarps - 1) / kDrawWarps;
      if (blocks > 32 * h->num_sms) blocks = 32 * h->num_sms;
      lowrank_draw_kernel<<<blocks, 32 * kDrawWarps, static_cast<size_t>(kDrawWarps) * c.v * sizeof(float), st>>>(
          base, reinterpret_cast<const __nv_bfloat16*>(h->ws + h->lr_off_zhl), static_cast<const __nv_bfloat16*>(h->lr_A),
          at<int>(h, L.off_sel), uniforms, out_bytes, at<unsigned>(h, L.off_status), W, wpp, c.n, c.r, c.v, valid_symbols(c), k);
      h->launches++;
    }
    pt.end();
    if ((rc = check_launch()) != MTPC_OK) return rc;
    pt.begin();
    rc = launch_lowrank_projection(h, hidden, P, out_bytes, st, nullptr, /*parts=*/4, /*targets_are_drafts=*/true);
    pt.end();
    if (rc != MTPC_OK) return rc;
    pt.begin();
    rc = launch_circuit(h, W, wpp, out_logprob, out_prefix, st);
    pt.end();
    if (rc == MTPC_OK) {               // G, log omega, W_base h and B h stay in place for an acceptance call
      h->draft_P = P;
      h->draft_wpp = wpp;
      h->draft_hidden = nullptr;
    }
    return rc;
  }
  if (h->lr_k > 0 && P > L.decode_max_p) {
    // Otherwise (several windows per position, or units wider than 512 symbols) the few-position path runs chunk after
    // chunk of positions: W_base, B and A are small enough to stay in L2. Only the last chunk's logits remain: no
    // acceptance stage after such a draft either.
    for (int p0 = 0; p0 < P; p0 += L.decode_max_p) {
      const int pc = P - p0 < L.decode_max_p ? P - p0 : L.decode_max_p;
      const size_t w0 = static_cast<size_t>(p0) * wpp;
      const int rc = draft_sample_impl(h, static_cast<const uint8_t*>(hidden) + static_cast<size_t>(p0) * c.d * 2, pc, wpp,
                                       uniforms + w0 * 2 * c.n, out_bytes + w0 * c.n, out_logprob ? out_logprob + w0 : nullptr,
                                       out_prefix ? out_prefix + w0 * c.n : nullptr, st);
      if (rc != MTPC_OK) return rc;
    }
    h->draft_P = 0;
    return MTPC_OK;
  }
  const void* hb = nullptr;
  int rc = stage_hidden(h, hidden, P, &hb, st);
  if (rc != MTPC_OK) return rc;
  PhaseTimer pt(h, st);
  h->draft_P = 0;
  if (P <= L.decode_max_p) {
    // Few positions: every weight row is read once. 1. all logits (emission -> scratch, sum units -> log omega)
    // 2. per (position, slot): latent draws, byte draws, evidence of the drafted bytes  3. circuit evaluation
    pt.begin();
    rc = launch_decode_gemm(h, hb, P, st);
    pt.end();
    if (rc != MTPC_OK) return rc;
    pt.begin();
    {
      int chain = 0;                                       // longest chain of latent-draw tables of any slot
      if (c.family == MTPC_HMM) chain = c.n - 1;
      if (c.family == MTPC_BTREE) { for (int m = c.n; m > 2; m >>= 1) ++chain; }
      const size_t base = static_cast<size_t>((2 * c.r + 3) & ~3) * sizeof(float);
      const size_t with_tables = base + static_cast<size_t>(chain) * c.r * c.r * sizeof(float);
      const int in_smem = chain > 0 && with_tables <= kSlotSmemLimit;
      // builds of the narrow kernel that unroll 4, 8, 10 or 16 batches of 32 symbols: the smallest that covers v
      auto* slot_kernel = c.v > kMaxDraftVocab ? draft_slot_kernel<true, 16>
                          : c.v <= 128 ? draft_slot_kernel<false, 4>
                          : c.v <= 256 ? draft_slot_kernel<false, 8>
                          : c.v <= 320 ? draft_slot_kernel<false, 10> : draft_slot_kernel<false, 16>;
      launch_kernel(slot_kernel, dim3(c.n, P), kSlotThreads,
                    in_smem ? with_tables : base, st, h->ring == 0, c.family,
                    at<float>(h, L.off_logits), at<float>(h, L.off_logw), hmm_tables(h), uniforms, out_bytes,
                    at<float>(h, L.off_G), at<float>(h, L.off_unit_lse), at<unsigned>(h, L.off_status),
                    at<unsigned>(h, L.off_status) + kWorkCounterWord, wpp, c.n, c.r, c.v, valid_symbols(c), L.sum_rows,
                    hmm_table_stride(h), in_smem);
    }
    h->launches++;
    h->draft_P = P;
    h->draft_wpp = wpp;
    pt.end();
    if ((rc = check_launch()) != MTPC_OK) return rc;
    pt.begin();
    rc = launch_circuit(h, W, wpp, out_logprob, out_prefix, st, /*dependent=*/h->ring == 0, /*raw_mixture=*/c.r > 32);
    pt.end();
    return rc;
  }
  if (!L.can_draft_many) return MTPC_ERR_UNSUPPORTED;
  // 1. sum-unit weights (Sec. 3.3) -> 2. latent draws at the sum units (Algorithm 1)
  pt.begin();
  rc = launch_gemm(h, kModeLogprob, hb, P, 1, false, true, nullptr, nullptr, nullptr, st);
  pt.end();
  if (rc != MTPC_OK) return rc;
  pt.begin();
  latent_sample_kernel<<<(W + 127) / 128, 128, 0, st>>>(c.family, at<float>(h, L.off_logw), hmm_tables(h), uniforms,
                                                        at<int>(h, L.off_sel), out_bytes,
                                                        at<unsigned>(h, L.off_status), W, wpp, c.n, c.r, L.sum_rows,
                                                        hmm_table_stride(h));
  h->launches++;
  pt.end();
  if ((rc = check_launch()) != MTPC_OK) return rc;
  // 3. byte draws at the selected input units. With few windows per position against many units per slot the draws
  // are first sorted by unit, so that every window is multiplied by the one unit it samples from.
  if (L.sample_two_pass && L.group_entries == 0) return MTPC_ERR_UNSUPPORTED;
  const bool grouped = L.sample_two_pass ||
                       (L.group_entries > 0 && h->draft_grouping != 1 && (h->draft_grouping == 2 || wpp * 4 <= c.r));
  if (grouped) {
    const int units = c.n * c.r;
    int* ints = at<int>(h, L.off_grp_ints);
    int* counts = ints, *cursors = ints + units, *offsets = ints + 2 * units, *num_tiles = ints + 3 * units;
    GroupTile* tiles = at<GroupTile>(h, L.off_grp_tiles);
    int* perm = at<int>(h, L.off_grp_perm);
    __nv_bfloat16* stage = at<__nv_bfloat16>(h, L.off_grp_stage);
    const int chunk_pos = static_cast<int>(L.group_entries / (static_cast<size_t>(wpp) * c.n));   // >= 1 by construction
    for (int p0 = 0; p0 < P; p0 += chunk_pos) {
      const int pc = P - p0 < chunk_pos ? P - p0 : chunk_pos;
      const int entries = pc * wpp * c.n;
      const size_t w0 = static_cast<size_t>(p0) * wpp;
      const int* sel = at<int>(h, L.off_sel) + w0 * c.n;
      pt.begin();
      if (cudaMemsetAsync(ints, 0, static_cast<size_t>(2 * units) * 4, st) != cudaSuccess) return MTPC_ERR_CUDA;
      const int cblocks = (entries + kGroupThreads - 1) / kGroupThreads;
      group_count_kernel<<<cblocks < 4 * h->num_sms ? cblocks : 4 * h->num_sms, kGroupThreads, units * sizeof(int), st>>>(
          sel, counts, entries, c.n, c.r);
      group_scan_kernel<<<1, kGroupScanThreads, 0, st>>>(counts, offsets, tiles, num_tiles, units);
      const int gblocks = (entries + kGroupThreads / 32 - 1) / (kGroupThreads / 32);
      group_gather_kernel<<<gblocks < 16 * h->num_sms ? gblocks : 16 * h->num_sms, kGroupThreads, 0, st>>>(
          sel, static_cast<const __nv_bfloat16*>(hb) + static_cast<size_t>(p0) * c.d, offsets, cursors, perm, stage, entries,
          c.n, c.r, wpp, c.d, static_cast<int*>(nullptr));
      h->launches += 3;
      if ((rc = check_launch()) != MTPC_OK) return rc;
      GroupArgs ga;
      ga.stage = stage;
      ga.entries = entries;
      ga.tiles = tiles;
      ga.num_tiles = num_tiles;
      ga.perm = perm;
      ga.unit_sel = sel;
      ga.max_tiles = units + entries / 128 + 1;
      rc = launch_gemm(h, kModeSample, hb, pc, wpp, true, false, nullptr, uniforms + w0 * 2 * c.n, out_bytes + w0 * c.n, st,
                       nullptr, false, &ga);
      pt.end();
      if (rc != MTPC_OK) return rc;
    }
  } else {
    pt.begin();
    rc = launch_gemm(h, kModeSample, hb, P, wpp, true, false, nullptr, uniforms, out_bytes, st);
    pt.end();
    if (rc != MTPC_OK) return rc;
  }
  // 4. evidence of the drafted bytes under every unit -> 5. joint log-prob with the latents summed out
  pt.begin();
  rc = launch_gemm(h, kModeLogprob, hb, P, wpp, true, false, out_bytes, nullptr, nullptr, st, nullptr,
                   /*targets_are_drafts=*/true);
  pt.end();
  if (rc != MTPC_OK) return rc;
  pt.begin();
  rc = launch_circuit(h, W, wpp, out_logprob, out_prefix, st);
  pt.end();
  if (rc == MTPC_OK) {                 // G, log omega and the hidden states stay in place for an acceptance call
    h->draft_P = P;
    h->draft_wpp = wpp;
    h->draft_hidden = hb;
  }
  return rc;
}

// ---------------------------------------------------------------- backward pass (host side)
size_t round64(size_t x) { return (x + 63) / 64 * 64; }

// Carving of the backward workspace for T positions (all buffers 256-byte aligned).
// The sum-unit logit gradients sit to the right of the emission logit gradients in one matrix [T, Kd], Kd = Nc + Spad.
struct BackwardLayout {
  size_t Nc, Spad, Kd;
  size_t off_lse, off_post, off_logits, off_dlogit, off_dsum_f32, off_coeff, total;
};
void plan_backward(const mtpc_config& c, const Layout& L, int T, BackwardLayout* B) {
  B->Nc = static_cast<size_t>(c.n) * c.r * c.v;
  B->Spad = round64(L.sum_rows);
  B->Kd = B->Nc + B->Spad;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  B->off_lse = take(static_cast<size_t>(T) * c.n * c.r * 4);
  B->off_post = take(static_cast<size_t>(T) * c.n * c.r * 4);
  B->off_logits = take(static_cast<size_t>(T) * B->Nc * 4);              // [T, Nc] fp32: the emission logits of the forward pass
  B->off_dlogit = take(static_cast<size_t>(T) * B->Kd * 2);          // [T, Nc | Spad] bf16
  B->off_dsum_f32 = take(static_cast<size_t>(T) * L.sum_rows * 4);   // Eq. 6: sum-unit logit gradients accumulated over the passes
  B->off_coeff = take(static_cast<size_t>(T) * c.n * 4);             // Eq. 6: weights of the prefix marginals
  B->total = off;
}

// C[M, N] fp32 (pitch ldc) = A B^T over K = K0 + K1: segment 0 multiplies A's K range [0, K0) with B0, segment 1 (K1 > 0)
// A's K range [a_k1, a_k1 + K1) with B1.
// C_hilo != NULL (then C is NULL): the result leaves as two bf16 halves per entry, see PlainGemmParams.
int launch_plain_gemm(mtpc_head* h, GemmOperand A, GemmOperand B0, int K0, GemmOperand B1, int K1, int a_k1, float* C,
                      size_t ldc, int M, int N, cudaStream_t st, void* C_hilo, int split_k, const PlainGemmExtra* extra) {
  if (M <= 0 || N <= 0 || K0 <= 0) return MTPC_OK;
  if (K1 > 0 && (A.mn_major || B1.mn_major != B0.mn_major)) return MTPC_ERR_SHAPE;
  const PlainGemmExtra none;
  const PlainGemmExtra& x = extra ? *extra : none;
  if (x.batches < 1 || (x.batches > 1 && K1 > 0)) return MTPC_ERR_SHAPE;
  PlainGemmParams p;
  memset(&p, 0, sizeof(p));
  const int Ka = K1 > 0 ? a_k1 + K1 : K0;                      // extent of A along K
  const uint64_t a_m = x.a_extent_m ? x.a_extent_m : M, a_k = x.a_extent_k ? x.a_extent_k : Ka;
  const uint64_t b_n = x.b_extent_n ? x.b_extent_n : N, b_k = x.b_extent_k ? x.b_extent_k : K0;
  int rc = A.mn_major ? make_tmap_mn(&p.tm_a, A.ptr, a_k, a_m, A.pitch) : make_tmap(&p.tm_a, A.ptr, a_m, a_k, kBlockM, A.pitch);
  if (rc == MTPC_OK)
    rc = B0.mn_major ? make_tmap_mn(&p.tm_b[0], B0.ptr, b_k, b_n, B0.pitch) : make_tmap(&p.tm_b[0], B0.ptr, b_n, b_k, kPlainTileN, B0.pitch);
  if (rc == MTPC_OK && K1 > 0)
    rc = B1.mn_major ? make_tmap_mn(&p.tm_b[1], B1.ptr, K1, N, B1.pitch) : make_tmap(&p.tm_b[1], B1.ptr, N, K1, kPlainTileN, B1.pitch);
  if (rc != MTPC_OK) return rc;
  p.M = M; p.N = N;
  p.a_k0[0] = 0;
  p.a_k0[1] = a_k1;
  p.seg_kblocks[0] = (K0 + kBlockK - 1) / kBlockK;
  p.seg_kblocks[1] = K1 > 0 ? (K1 + kBlockK - 1) / kBlockK : 0;
  p.m_tiles = (M + kBlockM - 1) / kBlockM;
  // batched products with a rank for N: 64-column accumulator tiles
  const int tile_n = (x.batches > 1 && N <= 64 && B0.mn_major) ? 64 : kPlainTileN;
  p.n_tiles = (N + tile_n - 1) / tile_n;
  p.stage_bytes = kABytes + tile_n * kBlockK * 2;
  const int ctl = 1024 + static_cast<int>(sizeof(GemmControl));
  p.stages = (kSmemLimit - ctl) / p.stage_bytes;
  if (p.stages > kMaxStages) p.stages = kMaxStages;
  p.wide_stores = (reinterpret_cast<uintptr_t>(C) % 32 == 0 && ldc % 8 == 0 && x.c_step % 8 == 0) ? 1 : 0;
  p.C = C;
  p.ldc = ldc;
  p.C_hilo = static_cast<__nv_bfloat16*>(C_hilo);
  p.split_k = split_k;
  p.C_bf16 = static_cast<__nv_bfloat16*>(x.C_bf16);
  if ((C != nullptr) + (C_hilo != nullptr) + (x.C_bf16 != nullptr) != 1) return MTPC_ERR_NULL;
  if (C_hilo != nullptr && (split_k < 16 || split_k % 16 != 0 || N % split_k != 0)) return MTPC_ERR_SHAPE;
  if (x.C_bf16 != nullptr && (reinterpret_cast<uintptr_t>(x.C_bf16) % 32 != 0 || ldc % 16 != 0 || x.c_step % 16 != 0))
    return MTPC_ERR_WORKSPACE;
  p.batches = x.batches;
  p.a_m_step = x.a_m_step; p.a_k_step = x.a_k_step; p.b_n_step = x.b_n_step; p.b_k_step = x.b_k_step;
  p.c_step = x.c_step;
  p.status = at<unsigned>(h, h->L.off_status);
  p.wait_limit_ns = h->wait_limit_ns;
  const long long items = static_cast<long long>(p.m_tiles) * p.n_tiles * p.batches;
  const int grid = static_cast<int>(items < h->num_sms ? items : h->num_sms);
  const size_t smem = p.stages * p.stage_bytes + ctl;
  if (tile_n == 64 && A.mn_major) plain_gemm_kernel<true, true, 64><<<grid, kGemmThreads, smem, st>>>(p);
  else if (tile_n == 64) plain_gemm_kernel<false, true, 64><<<grid, kGemmThreads, smem, st>>>(p);
  else if (A.mn_major && B0.mn_major) plain_gemm_kernel<true, true><<<grid, kGemmThreads, smem, st>>>(p);
  else if (!A.mn_major && B0.mn_major) plain_gemm_kernel<false, true><<<grid, kGemmThreads, smem, st>>>(p);
  else if (!A.mn_major && !B0.mn_major) plain_gemm_kernel<false, false><<<grid, kGemmThreads, smem, st>>>(p);
  else return MTPC_ERR_SHAPE;
  h->launches++;
  return check_launch();
}

#ifndef MTPC_LR_GROUPS
#define MTPC_LR_GROUPS 2
#endif
constexpr int kLrGroups = MTPC_LR_GROUPS;   // epilogue groups of the factored projection kernel (<= kLrMaxGroups)
// Tiling of the factored projection (mtpc_lowrank_gemm.cuh) for a head shape; false: the shape does not fit.
bool plan_lowrank(const mtpc_config& c, int k, LowRankGemmParams* p) {
  if (k < 16 || k > kLrMaxRank || k % 16 != 0 || c.v % 16 != 0) return false;
  // the fewest panels whose two base buffers leave room for the correction slots (two per epilogue group, chunks of at
  // least 16 columns; as many groups, up to kLrGroups and the number of components, as leave chunks of at least 32)
  int panels = 0, pc = 0, stride = 0, spare = 0;
  for (int np = 1; np <= kLrMaxPanels; ++np) {
    pc = ((c.v + np - 1) / np + 15) / 16 * 16;          // the last panel may be narrower
    stride = (pc + 31) / 32 * 32;
    spare = kTmemCols - 2 * stride;
    if (pc <= 256 && spare >= 32) { panels = (c.v + pc - 1) / pc; break; }
  }
  if (panels == 0) return false;
  int groups = kLrGroups < c.r ? kLrGroups : c.r;
  while (groups > 1 && spare / (2 * groups) < 32) --groups;
  int chunk = spare / (2 * groups) / 16 * 16;
  if (chunk > 96) chunk = 96;
  if (chunk > pc) chunk = pc;
  p->groups = groups;
  p->n = c.n; p->r = c.r; p->v = c.v; p->k = k;
  p->vv = c.v_valid > 0 ? c.v_valid : c.v;
  p->kblocks = c.d / kBlockK;
  p->panels = panels;
  p->panel_cols = pc;
  p->acc_stride = stride;
  p->chunk_cols = chunk;
  p->nchunk = (pc + chunk - 1) / chunk;
  p->corr_col0 = 2 * stride;
  p->base_stage_bytes = kABytes + pc * kBlockK * 2;                                  // a multiple of 1024 (pc % 16 == 0)
  p->corr_stage_bytes = 2 * kBlockM * 128 + p->nchunk * chunk * 128;                 // two z boxes and the A' boxes of 64 / k components
  const int ctl = 1024 + static_cast<int>(sizeof(LowRankControl));
  // at least two correction entries (one in use, the next on its way); the base ring takes the rest, at least two K blocks
  for (int cs = kLrCorrStages; cs >= 2; --cs) {
    const int left = kSmemLimit - ctl - cs * p->corr_stage_bytes;
    int bs = left / p->base_stage_bytes;
    if (bs > kMaxStages) bs = kMaxStages;
    if (bs >= 3 || (bs == 2 && cs == 2)) {
      p->corr_stages = cs;
      p->base_stages = bs;
      return true;
    }
  }
  return false;
}

// Factored projection of a low-rank head: log omega by the dense kernel's sum tiles, z = B h by a plain GEMM that writes
// it as two bf16 halves, A repacked, then the factored kernel (and the merge of its panels) writes G.
int launch_lowrank_projection(mtpc_head* h, const void* hidden_bf16, int T, const int* targets, cudaStream_t st,
                              const GradArgs* ga, int parts, bool targets_are_drafts) {
  const mtpc_config& c = h->cfg;
  const Layout& L = h->L;
  const int units = c.n * c.r, k = h->lr_k;
  int rc = MTPC_OK;
  if (parts & 1) rc = launch_gemm(h, kModeLogprob, hidden_bf16, T, 1, false, true, targets, nullptr, nullptr, st);
  if (rc != MTPC_OK) return rc;
  __nv_bfloat16* zhl = reinterpret_cast<__nv_bfloat16*>(h->ws + h->lr_off_zhl);
  if (parts & 2) {
    const GemmOperand hid{hidden_bf16, static_cast<size_t>(c.d), false};
    const GemmOperand bmat{h->lr_B, static_cast<size_t>(c.d), false};          // [n r k, d], K = d contiguous
    // z = B h, leaving the GEMM's epilogue already split into its two bf16 halves [T, n r, 2, k]
    rc = launch_plain_gemm(h, hid, bmat, c.d, bmat, 0, 0, nullptr, 0, T, units * k, st, zhl, k);
    if (rc != MTPC_OK) return rc;
    // A as [n, v, r, k]: the adaptor columns of adjacent components side by side (remade every call: A may have changed)
    const size_t pieces = static_cast<size_t>(units) * c.v * (k / 8);
    lowrank_repack_kernel<<<static_cast<unsigned>((pieces + 255) / 256), 256, 0, st>>>(
        static_cast<const uint4*>(h->lr_A), reinterpret_cast<uint4*>(h->ws + h->lr_off_arep), c.n, c.r, c.v, k / 8);
    h->launches += 1;
  }
  if (!(parts & 4)) return check_launch();
  LowRankGemmParams p = h->lr_params;
  rc = make_tmap(&p.tm_h, hidden_bf16, static_cast<uint64_t>(T), static_cast<uint64_t>(c.d), kBlockM);
  if (rc == MTPC_OK) rc = make_tmap(&p.tm_z, zhl, static_cast<uint64_t>(T), static_cast<uint64_t>(units) * 2 * k, kBlockM);
  if (rc != MTPC_OK) return rc;
  p.T = T;
  p.m_tiles = (T + kBlockM - 1) / kBlockM;
  p.targets = targets;
  p.G = at<float>(h, L.off_G);
  p.status = at<unsigned>(h, L.off_status);
  p.wait_limit_ns = h->wait_limit_ns;
  p.missing_is_nan = targets_are_drafts ? 1 : 0;
  if (ga != nullptr) {                 // a training call keeps every logit and every unit's log-sum-exp
    p.logit_out = ga->logit_out;
    p.logit_pitch = ga->logit_pitch;
    p.lse_out = ga->lse_out;
  }
  const size_t entries = static_cast<size_t>(T) * units;
  p.partial = reinterpret_cast<float2*>(h->ws + h->lr_off_partial);
  p.target_logit = reinterpret_cast<float*>(h->ws + h->lr_off_partial +
                                            static_cast<size_t>(p.panels) * c.max_positions * units * sizeof(float2));
  const long long items = static_cast<long long>(p.m_tiles) * c.n * p.panels;
  const int grid = static_cast<int>(items < h->num_sms ? items : h->num_sms);
  const int ctl = 1024 + static_cast<int>(sizeof(LowRankControl));
  mtpc_lowrank_gemm_kernel<<<grid, kLrRoleThreads + 128 * p.groups,
                             p.base_stages * p.base_stage_bytes + p.corr_stages * p.corr_stage_bytes + ctl, st>>>(p);
  h->launches += 1;
  if (p.panels > 1) {     // several panels per unit: their partial log-sum-exps are combined into G
    lowrank_merge_kernel<<<static_cast<unsigned>((entries + 255) / 256), 256, 0, st>>>(
        p.partial, p.target_logit, targets, p.G, p.lse_out, p.status, entries, c.r, p.vv, p.panels, p.missing_is_nan);
    h->launches += 1;
  }
  return check_launch();
}

// Warps per CTA of the circuit backward kernels: as many of 8, 4, 2, 1 as keep the CTA's shared memory within the limit
// (long windows need n x r floats of messages per warp). 0: not even one warp fits.
size_t circuit_backward_smem(const mtpc_head* h, int warps) {
  const mtpc_config& c = h->cfg;
  if (c.family == MTPC_HMM) return hmm_backward_smem_floats(c.n, c.r, !is_ctx(h), warps) * sizeof(float);
  if (c.family == MTPC_BTREE) return static_cast<size_t>(warps) * btree_backward_warp_floats(c.n, c.r) * sizeof(float);
  return 0;
}
int circuit_backward_warps(const mtpc_head* h) {
  for (int w = kCircuitWarps; w >= 1; w >>= 1)
    if (circuit_backward_smem(h, w) <= static_cast<size_t>(kSmemLimit)) return w;
  return 0;
}

// `loss_coeff` (HMM, tree): the weights [W, n] of the prefix log-marginals in Eq. 6; the whole gradient in one launch.
int launch_circuit_backward(mtpc_head* h, CircuitBackwardArgs a, float* dT, cudaStream_t st,
                            const float* loss_coeff = nullptr) {
  const mtpc_config& c = h->cfg;
  const Layout& L = h->L;
  a.G = at<float>(h, L.off_G);
  a.logw = at<float>(h, L.off_logw);
  a.n = c.n;
  a.r = c.r;
  a.sum_rows = L.sum_rows;
  unsigned* counter = at<unsigned>(h, L.off_status) + kWorkCounterWord;
  const int warps = c.family == MTPC_CP ? kCircuitWarps : circuit_backward_warps(h);
  if (warps == 0) return MTPC_ERR_UNSUPPORTED;
  const int blocks = (a.W + warps - 1) / warps;
  const int threads = warps * 32;
  const int resident = blocks < 8 * h->num_sms ? blocks : 8 * h->num_sms;
  const size_t smem = circuit_backward_smem(h, warps);
  if (c.family != MTPC_CP && cudaMemsetAsync(counter, 0, sizeof(unsigned), st) != cudaSuccess) return MTPC_ERR_CUDA;
  if (c.family == MTPC_CP) {
    circuit_cp_backward_kernel<<<blocks, threads, 0, st>>>(a);
  } else if (c.family == MTPC_HMM && loss_coeff != nullptr) {
    circuit_hmm_loss_backward_kernel<<<resident, threads, smem, st>>>(a, loss_coeff, hmm_tables(h), hmm_table_stride(h), dT,
                                                                     counter);
  } else if (c.family == MTPC_HMM) {
    circuit_hmm_backward_kernel<<<resident, threads, smem, st>>>(a, hmm_tables(h), hmm_table_stride(h), dT, counter);
  } else {
    circuit_btree_backward_kernel<<<resident, threads, smem, st>>>(a, loss_coeff, counter);
  }
  h->launches++;
  return check_launch();
}

// Shared-memory attributes of the circuit backward kernels (per function: always the full limit, see allow_full_smem).
int set_backward_attributes(const mtpc_head* head) {
  if (head->cfg.family == MTPC_CP) return MTPC_OK;
  if (circuit_backward_warps(head) == 0) return MTPC_ERR_UNSUPPORTED;
  bool ok = allow_full_smem(circuit_hmm_backward_kernel);
  ok &= allow_full_smem(circuit_hmm_loss_backward_kernel);
  ok &= allow_full_smem(circuit_btree_backward_kernel);
  return ok ? MTPC_OK : MTPC_ERR_CUDA;
}

// Phases 3 and 4 of a backward call: the logit gradients (post, lse and the kept logits -> bf16 rows) and the plain GEMMs.
// The sum-unit logit gradients are already in place to the right of dlogit. Every GEMM operand is read where it lies:
// the weights and the hidden states in the caller's buffers, the gradient matrix along its rows or down its columns.
int backward_tail(mtpc_head* head, const BackwardLayout& B, uint8_t* bw, const void* hb, const int32_t* targets, int T,
                  float* d_hidden, float* dW_emit, float* dW_sum, PhaseTimer& pt, cudaStream_t st) {
  const mtpc_config& c = head->cfg;
  const Layout& L = head->L;
  __nv_bfloat16* dlogit = reinterpret_cast<__nv_bfloat16*>(bw + B.off_dlogit);
  __nv_bfloat16* dsum = dlogit + B.Nc;
  const int Nc = static_cast<int>(B.Nc);
  pt.begin();
  LogitGradArgs la;
  la.logits = reinterpret_cast<const float*>(bw + B.off_logits);
  la.lse = reinterpret_cast<const float*>(bw + B.off_lse);
  la.post = reinterpret_cast<const float*>(bw + B.off_post);
  la.targets = targets;
  la.dlogit = dlogit;
  la.pitch = B.Kd;
  la.T = T; la.Nc = Nc; la.n = c.n; la.r = c.r; la.v = c.v;
  {
    const int col_blocks = (Nc / 8 + 255) / 256;
    int row_blocks = (16 * head->num_sms + col_blocks - 1) / col_blocks;   // enough CTAs to fill the device, each walks rows
    if (row_blocks > T) row_blocks = T;
    if (row_blocks > 65535) row_blocks = 65535;
    logit_gradient_kernel<<<dim3(col_blocks, row_blocks), 256, 0, st>>>(la);
  }
  head->launches++;
  int rc = check_launch();
  pt.end();
  if (rc != MTPC_OK) return rc;
  pt.begin();
  const GemmOperand g_rows{dlogit, B.Kd, false};            // [T, Nc | S r] along its rows: K = the logit index
  const GemmOperand g_cols{dlogit, B.Kd, true};             // the same matrix down its columns: K = the position
  const GemmOperand s_cols{dsum, B.Kd, true};
  const GemmOperand w_emit{head->W_emit_bf16, static_cast<size_t>(c.d), true};   // [Nc, d]: N = d contiguous
  const GemmOperand w_sum{head->W_sum_bf16, static_cast<size_t>(c.d), true};
  const GemmOperand hid{hb, static_cast<size_t>(c.d), true};                     // [T, d]: N = d contiguous, K = the position
  // d hidden [T, d] = dlogit [T, Nc] W_emit [Nc, d] + dsum [T, S r] W_sum [S r, d]
  rc = launch_plain_gemm(head, g_rows, w_emit, Nc, w_sum, L.sum_rows, Nc, d_hidden, c.d, T, c.d, st);
  // dW_emit [Nc, d] = dlogit^T [Nc, T] hidden [T, d];  dW_sum [S r, d] = dsum^T [S r, T] hidden [T, d]
  if (rc == MTPC_OK) rc = launch_plain_gemm(head, g_cols, hid, T, hid, 0, 0, dW_emit, c.d, Nc, c.d, st);
  if (rc == MTPC_OK) rc = launch_plain_gemm(head, s_cols, hid, T, hid, 0, 0, dW_sum, c.d, L.sum_rows, c.d, st);
  pt.end();
  return rc;
}

// Backward workspace of a factored head: the dense layout (log-sum-exps, posteriors, kept logits, logit gradients), then
//   sy    [T, n v | n r k | S r padded] bf16: the logit gradients summed over a slot's components, multiplied by the
//         adaptors A, and those of the sum units: the A operand of d hidden and of the three weight-gradient GEMMs;
//   wcat  [n v + n r k, d] bf16: W_base and B one after the other (one K segment of d hidden);
//   apad  [n r, v rounded up to 64, k] bf16: A with zero rows between the units.
struct LowRankBackwardLayout {
  BackwardLayout B;
  size_t Ksy, pitch, v64;
  size_t off_sy, off_wcat, off_apad, total;
};
void plan_lowrank_backward(const mtpc_config& c, const Layout& L, int k, int T, LowRankBackwardLayout* R) {
  plan_backward(c, L, T, &R->B);
  const size_t units = static_cast<size_t>(c.n) * c.r;
  R->Ksy = static_cast<size_t>(c.n) * c.v + units * k;
  R->pitch = R->Ksy + R->B.Spad;
  R->v64 = round64(c.v);
  size_t off = R->B.total;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  R->off_sy = take(static_cast<size_t>(T) * R->pitch * 2);
  R->off_wcat = take(R->Ksy * c.d * 2);
  R->off_apad = take(units * R->v64 * k * 2);
  R->total = off;
}

// Phases 3 and 4 of a training call on a factored head: logit gradients g [T, n r v] (bf16), their sum over a slot's
// components, the zero-padded A, W_base and B in a row; then the GEMMs. The sum units' logit gradients are already in the
// right-hand columns of sy.
int lowrank_backward_tail(mtpc_head* head, const LowRankBackwardLayout& R, uint8_t* bw, const void* hb, const int32_t* targets,
                          int T, float* d_hidden, float* dW_base, float* dA, float* dB, float* dW_sum, PhaseTimer& pt,
                          cudaStream_t st) {
  const mtpc_config& c = head->cfg;
  const Layout& L = head->L;
  const BackwardLayout& B = R.B;
  const int k = head->lr_k, units = c.n * c.r;
  __nv_bfloat16* sy = reinterpret_cast<__nv_bfloat16*>(bw + R.off_sy);
  int rc = MTPC_OK;
  pt.begin();
  __nv_bfloat16* dlogit = reinterpret_cast<__nv_bfloat16*>(bw + B.off_dlogit);
  const int Nc = static_cast<int>(B.Nc);
  LogitGradArgs la;
  la.logits = reinterpret_cast<const float*>(bw + B.off_logits);
  la.lse = reinterpret_cast<const float*>(bw + B.off_lse);
  la.post = reinterpret_cast<const float*>(bw + B.off_post);
  la.targets = targets;
  la.dlogit = dlogit;
  la.pitch = B.Kd;
  la.T = T; la.Nc = Nc; la.n = c.n; la.r = c.r; la.v = c.v;
  {
    const int col_blocks = (Nc / 8 + 255) / 256;
    int row_blocks = (16 * head->num_sms + col_blocks - 1) / col_blocks;
    if (row_blocks > T) row_blocks = T;
    if (row_blocks > 65535) row_blocks = 65535;
    logit_gradient_kernel<<<dim3(col_blocks, row_blocks), 256, 0, st>>>(la);
  }
  {
    const size_t pieces = static_cast<size_t>(T) * (c.n * c.v / 8);
    lowrank_component_sum_kernel<<<static_cast<unsigned>((pieces + 255) / 256), 256, 0, st>>>(dlogit, B.Kd, sy, R.pitch, T,
                                                                                               c.n, c.r, c.v);
    const size_t pad_pieces = static_cast<size_t>(units) * R.v64 * (k / 8);
    lowrank_pad_kernel<<<static_cast<unsigned>((pad_pieces + 255) / 256), 256, 0, st>>>(
        static_cast<const uint4*>(head->lr_A), reinterpret_cast<uint4*>(bw + R.off_apad), units, c.v, static_cast<int>(R.v64), k / 8);
  }
  head->launches += 3;
  uint8_t* wcat = bw + R.off_wcat;
  const size_t base_bytes = static_cast<size_t>(c.n) * c.v * c.d * 2;
  bool fail = cudaMemcpyAsync(wcat, head->lr_W_base, base_bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess;
  fail |= cudaMemcpyAsync(wcat + base_bytes, head->lr_B, static_cast<size_t>(units) * k * c.d * 2, cudaMemcpyDeviceToDevice, st) != cudaSuccess;
  if (fail || (rc = check_launch()) != MTPC_OK) return MTPC_ERR_CUDA;
  pt.end();
  // 4. the GEMMs
  pt.begin();
  const GemmOperand none{nullptr, 0, false};
  const GemmOperand hid{hb, static_cast<size_t>(c.d), true};
  {   // y_ij = g_ij A_ij [T, k], one product per unit, into the middle columns of sy
    PlainGemmExtra x;
    x.C_bf16 = sy + static_cast<size_t>(c.n) * c.v;
    x.batches = units;
    x.a_k_step = c.v;
    x.b_k_step = static_cast<int>(R.v64);
    x.c_step = k;
    x.a_extent_m = T; x.a_extent_k = Nc;
    x.b_extent_n = k; x.b_extent_k = static_cast<long long>(units) * R.v64;
    rc = launch_plain_gemm(head, GemmOperand{dlogit, B.Kd, false}, GemmOperand{bw + R.off_apad, static_cast<size_t>(k), true},
                           static_cast<int>(R.v64), none, 0, 0, nullptr, R.pitch, T, k, st, nullptr, 0, &x);
  }
  // d hidden [T, d] = [s | y] [W_base ; B] + dsum W_sum
  if (rc == MTPC_OK)
    rc = launch_plain_gemm(head, GemmOperand{sy, R.pitch, false}, GemmOperand{wcat, static_cast<size_t>(c.d), true},
                           static_cast<int>(R.Ksy), GemmOperand{head->W_sum_bf16, static_cast<size_t>(c.d), true}, L.sum_rows,
                           static_cast<int>(R.Ksy), d_hidden, c.d, T, c.d, st);
  // dW_base = s^T h, dB = y^T h, dW_sum = dsum^T h: sy down its columns
  if (rc == MTPC_OK)
    rc = launch_plain_gemm(head, GemmOperand{sy, R.pitch, true}, hid, T, hid, 0, 0, dW_base, c.d, c.n * c.v, c.d, st);
  if (rc == MTPC_OK)
    rc = launch_plain_gemm(head, GemmOperand{sy + static_cast<size_t>(c.n) * c.v, R.pitch, true}, hid, T, hid, 0, 0, dB, c.d,
                           units * k, c.d, st);
  if (rc == MTPC_OK)
    rc = launch_plain_gemm(head, GemmOperand{sy + R.Ksy, R.pitch, true}, hid, T, hid, 0, 0, dW_sum, c.d, L.sum_rows, c.d, st);
  if (rc == MTPC_OK) {   // dA_ij [v, k] = g_ij^T z_ij, one product per unit, on the bf16 high half of z the forward pass left
    PlainGemmExtra x;
    x.batches = units;
    x.a_m_step = c.v;
    x.b_n_step = 2 * k;
    x.c_step = static_cast<size_t>(c.v) * k;
    x.a_extent_m = Nc; x.a_extent_k = T;
    x.b_extent_n = static_cast<long long>(units) * 2 * k; x.b_extent_k = T;
    rc = launch_plain_gemm(head, GemmOperand{dlogit, B.Kd, true},
                           GemmOperand{head->ws + head->lr_off_zhl, static_cast<size_t>(units) * 2 * k, true}, T, none, 0, 0, dA,
                           k, c.v, k, st, nullptr, 0, &x);
  }
  pt.end();
  return rc;
}

int check_call(mtpc_head* h, int32_t rows) {
  if (!h) return MTPC_ERR_NULL;
  if (rows < 0 || rows > h->cfg.max_positions) return MTPC_ERR_SHAPE;
  return MTPC_OK;
}

}  // namespace

// The vector paths of the low-rank kernels need d a multiple of 4 and 16-byte aligned pointers.
static bool lowrank_vector_ok(int d, std::initializer_list<const void*> ptrs) {
  if (d % 4) return false;
  for (const void* p : ptrs)
    if (reinterpret_cast<uintptr_t>(p) % 16) return false;
  return true;
}

// Everything the head derives from the parameters: bf16 copies of fp32 weights, the tensor maps on the weight
// matrices, the log-softmaxed static HMM transitions or the contextual transition bias. Used at creation and again
// whenever the caller's parameters have changed (mtpc_update_parameters).
static int bind_parameters(mtpc_head* h, const void* W_emit, const void* W_sum, const float* T_static, cudaStream_t st) {
  const mtpc_config* cfg = &h->cfg;
  const Layout& L = h->L;
  const bool ctx = (cfg->flags & MTPC_FLAG_HMM_CONTEXTUAL) != 0;
  const size_t emit_count = static_cast<size_t>(cfg->n) * cfg->r * cfg->v * cfg->d;
  const size_t sum_count = static_cast<size_t>(L.sum_rows) * cfg->d;
  if (cfg->io_dtype == MTPC_F32) {
    f32_to_bf16_kernel<<<2048, 256, 0, st>>>(static_cast<const float*>(W_emit), at<__nv_bfloat16>(h, L.off_wemit),
                                             emit_count);
    f32_to_bf16_kernel<<<256, 256, 0, st>>>(static_cast<const float*>(W_sum), at<__nv_bfloat16>(h, L.off_wsum),
                                            sum_count);
    h->launches += 2;
    h->W_emit_bf16 = h->ws + L.off_wemit;
    h->W_sum_bf16 = h->ws + L.off_wsum;
  } else {
    h->W_emit_bf16 = W_emit;
    h->W_sum_bf16 = W_sum;
  }
  if (ctx) {
    // bias of the contextual transition logits, laid out like the sum-unit rows: zeros for the initial unit
    bool bad = cudaMemsetAsync(h->ws + L.off_sum_bias, 0, static_cast<size_t>(L.sum_rows) * 4, st) != cudaSuccess;
    if (T_static && cfg->n > 1)
      bad |= cudaMemcpyAsync(h->ws + L.off_sum_bias + static_cast<size_t>(cfg->r) * 4, T_static,
                             static_cast<size_t>(cfg->n - 1) * cfg->r * cfg->r * 4, cudaMemcpyDeviceToDevice,
                             st) != cudaSuccess;
    if (bad) return MTPC_ERR_CUDA;
  } else if (cfg->family == MTPC_HMM && cfg->n > 1) {
    const int rows = (cfg->n - 1) * cfg->r;
    log_softmax_rows_kernel<<<(rows + 127) / 128, 128, 0, st>>>(T_static, at<float>(h, L.off_logA), rows, cfg->r);
    h->launches++;
  }
  if (check_launch() != MTPC_OK) return MTPC_ERR_CUDA;
  const uint64_t emit_rows = static_cast<uint64_t>(cfg->n) * cfg->r * cfg->v;
  const bool dense = h->lr_k == 0;      // a factored low-rank head has no composed W_emit: only the sum-unit maps
  int rc = MTPC_OK;
  if (dense) rc = make_tmap(&h->tm_emit_lp, h->W_emit_bf16, emit_rows, cfg->d, L.lp.tile_cols);
  if (rc == MTPC_OK && dense && L.can_draft_many) rc = make_tmap(&h->tm_emit_sm, h->W_emit_bf16, emit_rows, cfg->d, L.sm.tile_cols);
  if (rc == MTPC_OK) rc = make_tmap(&h->tm_sum, h->W_sum_bf16, L.sum_rows, cfg->d, L.sum_cols);
  if (rc == MTPC_OK && dense) rc = make_tmap(&h->tm_emit_lp2, h->W_emit_bf16, emit_rows, cfg->d, L.lp.tile_cols / 2);
  if (rc == MTPC_OK && dense && L.can_draft_many) rc = make_tmap(&h->tm_emit_sm2, h->W_emit_bf16, emit_rows, cfg->d, L.sm.tile_cols / 2);
  if (rc == MTPC_OK) rc = make_tmap(&h->tm_sum2, h->W_sum_bf16, L.sum_rows, cfg->d, L.sum_cols / 2);
  const uint64_t base_rows = static_cast<uint64_t>(cfg->n) * cfg->v, adapt_rows = static_cast<uint64_t>(cfg->n) * cfg->r * h->lr_k;
  h->decode_tile_rows = decode_tile_rows(static_cast<long long>(dense ? emit_rows : base_rows + adapt_rows), h->num_sms);
  if (rc == MTPC_OK && dense) rc = make_tmap(&h->tm_emit_dec, h->W_emit_bf16, emit_rows, cfg->d, h->decode_tile_rows);
  if (rc == MTPC_OK && !dense) rc = make_tmap(&h->tm_emit_dec, h->lr_W_base, base_rows, cfg->d, h->decode_tile_rows);
  if (rc == MTPC_OK && !dense) rc = make_tmap(&h->tm_lrB_dec, h->lr_B, adapt_rows, cfg->d, h->decode_tile_rows);
  h->decode_sum_tile_rows = h->decode_tile_rows / 32 * 32;   // whole groups of r <= 32 rows per warp; fits the tile pitch
  if (rc == MTPC_OK) rc = make_tmap(&h->tm_sum_dec, h->W_sum_bf16, L.sum_rows, cfg->d, h->decode_sum_tile_rows);
  h->draft_P = 0;                                              // logits left by an earlier draft belong to the old parameters
  return rc;
}

extern "C" {

int mtpc_workspace_bytes(const mtpc_config* cfg, size_t* out_bytes) {
  if (!cfg || !out_bytes) return MTPC_ERR_NULL;
  Layout L;
  int rc = plan(*cfg, &L);
  if (rc != MTPC_OK) return rc;
  *out_bytes = L.total;
  return MTPC_OK;
}

// lowrank: NULL for a dense head; else the rank and the three parameter tensors of App. G (W_emit is NULL then).
struct LowRankSpec {
  int k;
  const void* W_base;
  const void* A;
  const void* B;
};

// Workspace of a factored head beyond the dense layout: z = B h as two bf16 halves [T, n r, 2, k] (written by the GEMM
// that computes it), where a unit is cut into panels the panels' (maximum, sum) pairs and the targets' logits, and the
// copy of A the factored kernel reads.
static int lowrank_extra_bytes(const mtpc_config& c, int k, int panels, size_t base_total, size_t* off_zhl,
                               size_t* off_partial, size_t* off_arep, size_t* off_dec, size_t* off_base, size_t* total) {
  const size_t units = static_cast<size_t>(c.n) * c.r;
  size_t off = align_up(base_total);
  *off_zhl = off;
  off += align_up(static_cast<size_t>(c.max_positions) * units * 2 * k * 2);
  *off_partial = off;
  if (panels > 1) off += align_up(static_cast<size_t>(c.max_positions) * units * (panels * sizeof(float2) + sizeof(float)));
  *off_arep = off;                      // the copy of A laid out [n, v, r, k]
  off += align_up(units * c.v * k * 2);
  *off_dec = off;                       // few-position draft: base = W_base h [P, n v] and z = B h [P, n r k], fp32
  off += align_up(static_cast<size_t>(c.max_positions < kDecodeMaxP ? c.max_positions : kDecodeMaxP) *
                  (static_cast<size_t>(c.n) * c.v + units * k) * 4);
  *off_base = 0;                        // long drafts (more positions than that path takes): W_base h [T, n v] fp32
  if (c.max_positions > kDecodeMaxP && c.v <= kMaxDraftVocab) {
    *off_base = off;
    off += align_up(static_cast<size_t>(c.max_positions) * c.n * c.v * 4);
  }
  *total = off;
  return MTPC_OK;
}

static int create_head_impl(const mtpc_config* cfg, const void* W_emit, const LowRankSpec* lowrank, const void* W_sum,
                            const float* T_static, void* workspace, size_t workspace_bytes, void* stream, mtpc_head** out) {
  if (!cfg || !W_sum || !workspace || !out) return MTPC_ERR_NULL;
  if (!lowrank && !W_emit) return MTPC_ERR_NULL;
  if (lowrank && (!lowrank->W_base || !lowrank->A || !lowrank->B)) return MTPC_ERR_NULL;
  *out = nullptr;
  Layout L;
  int rc = plan(*cfg, &L);
  if (rc != MTPC_OK) return rc;
  LowRankGemmParams lrp;
  memset(&lrp, 0, sizeof(lrp));
  size_t lr_zhl = 0, lr_partial = 0, lr_arep = 0, lr_dec = 0, lr_base = 0;
  if (lowrank) {
    if (cfg->io_dtype != MTPC_BF16) return MTPC_ERR_UNSUPPORTED;
    if (!plan_lowrank(*cfg, lowrank->k, &lrp)) return MTPC_ERR_UNSUPPORTED;
    lowrank_extra_bytes(*cfg, lowrank->k, lrp.panels, L.total, &lr_zhl, &lr_partial, &lr_arep, &lr_dec, &lr_base, &L.total);
  }
  const bool ctx = (cfg->flags & MTPC_FLAG_HMM_CONTEXTUAL) != 0;
  if (cfg->family == MTPC_HMM && cfg->n > 1 && !ctx && !T_static) return MTPC_ERR_NULL;
  if (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0) return MTPC_ERR_WORKSPACE;
  int dev = 0, cc_major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MTPC_ERR_CUDA;
  if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || cc_major != 10)
    return MTPC_ERR_CUDA;   // tcgen05 / TMEM code: sm_100 only
  mtpc_head* h = new (std::nothrow) mtpc_head;
  if (!h) return MTPC_ERR_CUDA;
  memset(h, 0, sizeof(*h));
  h->cfg = *cfg;
  h->L = L;
  h->ws = static_cast<uint8_t*>(workspace);
  h->wait_limit_ns = kWaitLimitNs;
  if (lowrank) {
    h->lr_k = lowrank->k;
    h->lr_W_base = lowrank->W_base;
    h->lr_A = lowrank->A;
    h->lr_B = lowrank->B;
    h->lr_off_zhl = lr_zhl;
    h->lr_off_partial = lr_partial;
    h->lr_off_arep = lr_arep;
    h->lr_off_dec = lr_dec;
    h->lr_off_base = lr_base;
    h->lr_params = lrp;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool fail = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess;
  // the attribute is per function, not per head: always ask for the full 227 KB so that heads do not undo each other
  fail |= cudaFuncSetAttribute(mtpc_gemm_kernel<kModeLogprob, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kSmemLimit) != cudaSuccess;
  fail |= cudaFuncSetAttribute(mtpc_gemm_kernel<kModeSample, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kSmemLimit) != cudaSuccess;
  fail |= !allow_full_smem(mtpc_gemm_kernel<kModeSampleGrouped, 1>);
  fail |= !allow_full_smem(mtpc_gemm_kernel<kModeLogitsGrouped, 1>);
  fail |= !allow_full_smem(mtpc_gemm_kernel<kModeLogprob, 2>);
  fail |= !allow_full_smem(mtpc_gemm_kernel<kModeSample, 2>);
  h->max_pairs = fail ? 0 : resident_pairs(L.lp.pair_smem);
  fail |= !allow_full_smem(plain_gemm_kernel<false, false>);
  fail |= !allow_full_smem(plain_gemm_kernel<false, true>);
  fail |= !allow_full_smem(plain_gemm_kernel<true, true>);
  fail |= !allow_full_smem(plain_gemm_kernel<true, true, 64>);
  fail |= !allow_full_smem(plain_gemm_kernel<false, true, 64>);
  fail |= cudaFuncSetAttribute(mtpc_decode_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) !=
          cudaSuccess;
  const int slot_smem = static_cast<int>(kSlotSmemLimit);
  fail |= cudaFuncSetAttribute(draft_slot_kernel<false, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, slot_smem) != cudaSuccess;
  fail |= cudaFuncSetAttribute(draft_slot_kernel<false, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, slot_smem) != cudaSuccess;
  fail |= cudaFuncSetAttribute(draft_slot_kernel<false, 10>, cudaFuncAttributeMaxDynamicSharedMemorySize, slot_smem) != cudaSuccess;
  fail |= cudaFuncSetAttribute(draft_slot_kernel<false, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, slot_smem) != cudaSuccess;
  fail |= cudaFuncSetAttribute(draft_slot_kernel<true, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, slot_smem) != cudaSuccess;
  fail |= !set_circuit_attributes();
  fail |= !allow_full_smem(spec_accept_kernel);
  fail |= cudaMemsetAsync(h->ws + L.off_status, 0, 256, st) != cudaSuccess;
  if (fail) { delete h; return MTPC_ERR_CUDA; }

  rc = bind_parameters(h, W_emit, W_sum, T_static, st);
  if (rc == MTPC_OK && lowrank) {
    fail = !allow_full_smem(mtpc_lowrank_gemm_kernel);
    rc = fail ? MTPC_ERR_CUDA
              : make_tmap(&h->lr_params.tm_w, lowrank->W_base, static_cast<uint64_t>(cfg->n) * cfg->v, cfg->d,
                          h->lr_params.panel_cols);
    if (rc == MTPC_OK)
      rc = make_tmap(&h->lr_params.tm_a, h->ws + h->lr_off_arep, static_cast<uint64_t>(cfg->n) * cfg->v,
                     static_cast<uint64_t>(cfg->r) * lowrank->k, h->lr_params.chunk_cols);
  }
  if (rc != MTPC_OK) { delete h; return rc; }
  *out = h;
  return MTPC_OK;
}

int mtpc_create_head(const mtpc_config* cfg, const void* W_emit, const void* W_sum, const float* T_static,
                     void* workspace, size_t workspace_bytes, void* stream, mtpc_head** out) {
  if (!W_emit) return MTPC_ERR_NULL;
  return create_head_impl(cfg, W_emit, nullptr, W_sum, T_static, workspace, workspace_bytes, stream, out);
}

int mtpc_lowrank_workspace_bytes(const mtpc_config* cfg, int32_t k, size_t* out_bytes) {
  if (!cfg || !out_bytes) return MTPC_ERR_NULL;
  Layout L;
  int rc = plan(*cfg, &L);
  if (rc != MTPC_OK) return rc;
  LowRankGemmParams lrp;
  if (cfg->io_dtype != MTPC_BF16 || !plan_lowrank(*cfg, k, &lrp)) return MTPC_ERR_UNSUPPORTED;
  size_t a = 0, b = 0, c3 = 0, c4 = 0, c5 = 0;
  return lowrank_extra_bytes(*cfg, k, lrp.panels, L.total, &a, &b, &c3, &c4, &c5, out_bytes);
}

int mtpc_create_head_lowrank(const mtpc_config* cfg, int32_t k, const void* W_base, const void* A, const void* B,
                             const void* W_sum, const float* T_static, void* workspace, size_t workspace_bytes,
                             void* stream, mtpc_head** out) {
  const LowRankSpec spec{k, W_base, A, B};
  return create_head_impl(cfg, nullptr, &spec, W_sum, T_static, workspace, workspace_bytes, stream, out);
}


int mtpc_update_parameters(mtpc_head* head, const void* W_emit, const void* W_sum, const float* T_static, void* stream) {
  if (!head || !W_sum || (!W_emit && head->lr_k == 0)) return MTPC_ERR_NULL;   // a factored head has no W_emit to rebind
  const mtpc_config& c = head->cfg;
  if (c.family == MTPC_HMM && c.n > 1 && !(c.flags & MTPC_FLAG_HMM_CONTEXTUAL) && !T_static) return MTPC_ERR_NULL;
  return bind_parameters(head, W_emit, W_sum, T_static, static_cast<cudaStream_t>(stream));
}

int mtpc_window_logprob(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T, float* out_logprob,
                        void* stream) {
  int rc = check_call(head, T);
  if (rc != MTPC_OK) return rc;
  if (T == 0) return MTPC_OK;
  if (!hidden || !targets || !out_logprob) return MTPC_ERR_NULL;
  return window_logprob_impl(head, hidden, targets, T, out_logprob, nullptr, static_cast<cudaStream_t>(stream));
}

int mtpc_window_prefix_logprob(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                               float* out_prefix_logprob, void* stream) {
  int rc = check_call(head, T);
  if (rc != MTPC_OK) return rc;
  if (T == 0) return MTPC_OK;
  if (!hidden || !targets || !out_prefix_logprob) return MTPC_ERR_NULL;
  return window_logprob_impl(head, hidden, targets, T, nullptr, out_prefix_logprob, static_cast<cudaStream_t>(stream));
}

int mtpc_draft_sample(mtpc_head* head, const void* hidden, int32_t P, int32_t wpp, const float* uniforms,
                      int32_t* out_bytes, float* out_logprob, void* stream) {
  int rc = check_call(head, P);
  if (rc != MTPC_OK) return rc;
  if (wpp < 1 || wpp > head->cfg.max_windows_per_pos) return MTPC_ERR_SHAPE;
  if (P == 0) return MTPC_OK;
  if (!hidden || !uniforms || !out_bytes || !out_logprob) return MTPC_ERR_NULL;
  return draft_sample_impl(head, hidden, P, wpp, uniforms, out_bytes, out_logprob, nullptr,
                           static_cast<cudaStream_t>(stream));
}

int mtpc_draft_sample_prefix(mtpc_head* head, const void* hidden, int32_t P, int32_t wpp, const float* uniforms,
                             int32_t* out_bytes, float* out_prefix_logprob, void* stream) {
  int rc = check_call(head, P);
  if (rc != MTPC_OK) return rc;
  if (wpp < 1 || wpp > head->cfg.max_windows_per_pos) return MTPC_ERR_SHAPE;
  if (P == 0) return MTPC_OK;
  if (!hidden || !uniforms || !out_bytes || !out_prefix_logprob) return MTPC_ERR_NULL;
  return draft_sample_impl(head, hidden, P, wpp, uniforms, out_bytes, nullptr, out_prefix_logprob,
                           static_cast<cudaStream_t>(stream));
}

int mtpc_speculative_accept(mtpc_head* head, int32_t P, int32_t wpp, const int32_t* draft_bytes,
                            const float* prefix_logprob, const float* target_probs, const float* accept_uniforms,
                            int32_t* out_accepted, int32_t* out_next_byte, void* stream) {
  int rc = check_call(head, P);
  if (rc != MTPC_OK) return rc;
  if (wpp < 1 || wpp > head->cfg.max_windows_per_pos) return MTPC_ERR_SHAPE;
  if (P == 0) return MTPC_OK;
  if (!draft_bytes || !prefix_logprob || !target_probs || !accept_uniforms || !out_accepted || !out_next_byte)
    return MTPC_ERR_NULL;
  if (head->draft_P != P || head->draft_wpp != wpp) return MTPC_ERR_STATE;
  const mtpc_config& c = head->cfg;
  const Layout& L = head->L;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int W = P * wpp;
  const size_t smem = accept_warp_floats(c.family, c.n, c.r, c.v) * sizeof(float);
  if (smem > static_cast<size_t>(kSmemLimit)) return MTPC_ERR_UNSUPPORTED;      // a residual row of more than ~56k symbols
  PhaseTimer pt(head, st);
  if (P <= L.decode_max_p) {
    // after a few-position draft: every logit of the drafted positions is still in the workspace
    pt.begin();
    spec_accept_kernel<<<W, kAcceptThreads, smem, st>>>(
        c.family, at<float>(head, L.off_logits), at<float>(head, L.off_unit_lse), at<float>(head, L.off_logw),
        hmm_tables(head), draft_bytes, prefix_logprob, target_probs, accept_uniforms, out_accepted,
        out_next_byte, at<unsigned>(head, L.off_status), W, wpp, c.n, c.r, c.v, valid_symbols(c), L.sum_rows,
        hmm_table_stride(head), static_cast<const float*>(nullptr), static_cast<const int*>(nullptr));
    head->launches++;
    pt.end();
    return check_launch();
  }
  // After a many-position draft no logits were kept. The evidence of the drafted bytes (G) and log omega are still in
  // the workspace; what is missing is, for every window rejected at byte s, the r v logits of slot s. So: run the tests,
  // sort the rejected windows by s, stage their hidden states, recompute those logits with one sorted projection pass,
  // then run the acceptance kernel on them. In chunks of positions whose windows fit the scratch.
  const bool factored = head->lr_k > 0;     // (a long draft on a factored head left W_base h and B h instead of needing the hidden states)
  if (L.accept_rows == 0 || (!factored && !head->draft_hidden)) return MTPC_ERR_UNSUPPORTED;
  if (factored && head->lr_off_base == 0) return MTPC_ERR_UNSUPPORTED;
  int* ints = at<int>(head, L.off_grp_ints);
  int* counts = ints, *cursors = ints + c.n, *offsets = ints + 2 * c.n, *num_tiles = ints + 3 * c.n;
  GroupTile* tiles = at<GroupTile>(head, L.off_grp_tiles);
  int* perm = at<int>(head, L.off_grp_perm);
  __nv_bfloat16* stage = at<__nv_bfloat16>(head, L.off_grp_stage);
  int* rej = at<int>(head, L.off_acc_rej);
  int* row_of = at<int>(head, L.off_acc_row);
  float* lg = at<float>(head, L.off_acc_logits);
  float* lse = at<float>(head, L.off_acc_lse);
  const int chunk_pos = static_cast<int>(L.accept_rows / wpp);                  // >= 1 by construction
  const float* tables = hmm_tables(head);
  const int tstride = hmm_table_stride(head);
  for (int p0 = 0; p0 < P; p0 += chunk_pos) {
    const int pc = P - p0 < chunk_pos ? P - p0 : chunk_pos;
    const int wc = pc * wpp;
    const size_t w0 = static_cast<size_t>(p0) * wpp;
    const int32_t* xb = draft_bytes + w0 * c.n;
    const float* pre = prefix_logprob + w0 * c.n;
    const float* tp = target_probs + w0 * (c.n + 1) * c.v;
    const float* ua = accept_uniforms + w0 * (c.n + 1);
    pt.begin();
    accept_test_kernel<<<(wc + 7) / 8, 256, 0, st>>>(xb, pre, tp, ua, rej, wc, c.n, c.v, valid_symbols(c));
    if (factored) {
      // the slot's logits from W_base h and B h, window by window: no sort, no staging, no projection pass
      const int pairs = wc * c.r;
      int blocks = (pairs + kDrawWarps - 1) / kDrawWarps;
      if (blocks > 32 * head->num_sms) blocks = 32 * head->num_sms;
      lowrank_slot_logits_kernel<<<blocks, 32 * kDrawWarps, 0, st>>>(
          reinterpret_cast<const float*>(head->ws + head->lr_off_base), reinterpret_cast<const __nv_bfloat16*>(head->ws + head->lr_off_zhl),
          static_cast<const __nv_bfloat16*>(head->lr_A), rej, lg, lse, row_of, wc, static_cast<int>(w0), wpp, c.n, c.r, c.v,
          valid_symbols(c), head->lr_k);
      head->launches += 2;
      pt.end();
      int rcf = check_launch();
      if (rcf != MTPC_OK) return rcf;
      pt.begin();
      spec_accept_kernel<<<wc, kAcceptThreads, smem, st>>>(
          c.family, lg, lse, at<float>(head, L.off_logw) + static_cast<size_t>(p0) * L.sum_rows,
          tables + static_cast<size_t>(p0) * tstride, xb, pre, tp, ua, out_accepted + w0, out_next_byte + w0,
          at<unsigned>(head, L.off_status), wc, wpp, c.n, c.r, c.v, valid_symbols(c), L.sum_rows, tstride,
          at<float>(head, L.off_G) + w0 * c.n * c.r, row_of);
      head->launches++;
      pt.end();
      if ((rcf = check_launch()) != MTPC_OK) return rcf;
      continue;
    }
    if (cudaMemsetAsync(ints, 0, static_cast<size_t>(2 * c.n) * 4, st) != cudaSuccess) return MTPC_ERR_CUDA;
    const int cblocks = (wc + kGroupThreads - 1) / kGroupThreads;
    group_count_kernel<<<cblocks < 4 * head->num_sms ? cblocks : 4 * head->num_sms, kGroupThreads, c.n * sizeof(int), st>>>(
        rej, counts, wc, 1, c.n);
    group_scan_kernel<<<1, kGroupScanThreads, 0, st>>>(counts, offsets, tiles, num_tiles, c.n);
    const int gblocks = (wc + kGroupThreads / 32 - 1) / (kGroupThreads / 32);
    group_gather_kernel<<<gblocks < 16 * head->num_sms ? gblocks : 16 * head->num_sms, kGroupThreads, 0, st>>>(
        rej, static_cast<const __nv_bfloat16*>(head->draft_hidden) + static_cast<size_t>(p0) * c.d, offsets, cursors, perm,
        stage, wc, 1, c.n, wpp, c.d, row_of);
    head->launches += 4;
    int rc2 = check_launch();
    if (rc2 != MTPC_OK) return rc2;
    GroupArgs ga;
    ga.stage = stage;
    ga.entries = wc;
    ga.tiles = tiles;
    ga.num_tiles = num_tiles;
    ga.perm = perm;
    ga.unit_sel = rej;
    ga.max_tiles = c.n + wc / 128 + 1;
    ga.by_slot = true;
    GradArgs out;
    out.lse_out = lse;
    out.logit_out = lg;
    out.logit_pitch = static_cast<size_t>(c.r) * c.v;
    rc2 = launch_gemm(head, kModeLogprob, head->draft_hidden, pc, wpp, true, false, nullptr, nullptr, nullptr, st, &out, false,
                      &ga);
    pt.end();
    if (rc2 != MTPC_OK) return rc2;
    pt.begin();
    spec_accept_kernel<<<wc, kAcceptThreads, smem, st>>>(
        c.family, lg, lse, at<float>(head, L.off_logw) + static_cast<size_t>(p0) * L.sum_rows,
        tables + static_cast<size_t>(p0) * tstride, xb, pre, tp, ua, out_accepted + w0, out_next_byte + w0,
        at<unsigned>(head, L.off_status), wc, wpp, c.n, c.r, c.v, valid_symbols(c), L.sum_rows, tstride,
        at<float>(head, L.off_G) + w0 * c.n * c.r, row_of);
    head->launches++;
    pt.end();
    if ((rc2 = check_launch()) != MTPC_OK) return rc2;
  }
  return MTPC_OK;
}

int mtpc_window_loss(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                     int32_t sequence_length, float gamma, float* out_slot_loss, float* out_loss, void* stream) {
  if (!head) return MTPC_ERR_NULL;
  if (num_sequences < 1 || sequence_length < 1) return MTPC_ERR_SHAPE;
  const int64_t T64 = static_cast<int64_t>(num_sequences) * sequence_length;
  if (T64 > head->cfg.max_positions) return MTPC_ERR_SHAPE;
  if (!hidden || !targets || !out_slot_loss || !out_loss) return MTPC_ERR_NULL;
  const int T = static_cast<int>(T64);
  const Layout& L = head->L;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* prefix = at<float>(head, L.off_prefix);
  float* partial = at<float>(head, L.off_partial);
  int rc = window_logprob_impl(head, hidden, targets, T, nullptr, prefix, st);   // phases 0 and 1
  if (rc != MTPC_OK) return rc;
  loss_partial_kernel<<<num_sequences, kLossThreads, 0, st>>>(prefix, targets, partial, sequence_length, head->cfg.n);
  loss_final_kernel<<<1, kLossThreads, 0, st>>>(partial, out_slot_loss, out_loss, num_sequences, head->cfg.n, gamma);
  head->launches += 2;
  return check_launch();
}

int mtpc_backward_workspace_bytes(const mtpc_config* cfg, int32_t T, size_t* out_bytes) {
  if (!cfg || !out_bytes) return MTPC_ERR_NULL;
  if (T < 1) return MTPC_ERR_SHAPE;
  Layout L;
  int rc = plan(*cfg, &L);
  if (rc != MTPC_OK) return rc;
  BackwardLayout B;
  plan_backward(*cfg, L, T, &B);
  *out_bytes = B.total;
  return MTPC_OK;
}

int mtpc_window_logprob_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                                 const float* weight, void* bwd_workspace, size_t bwd_workspace_bytes,
                                 float* out_logprob, float* d_hidden, float* dW_emit, float* dW_sum, float* dT_static,
                                 void* stream) {
  int rc = check_call(head, T);
  if (rc != MTPC_OK) return rc;
  if (T == 0) return MTPC_OK;
  if (!hidden || !targets || !weight || !bwd_workspace || !d_hidden || !dW_emit || !dW_sum) return MTPC_ERR_NULL;
  if (head->lr_k > 0) return MTPC_ERR_UNSUPPORTED;
  const mtpc_config& c = head->cfg;
  const bool static_hmm = c.family == MTPC_HMM && !is_ctx(head) && c.n > 1;
  if (static_hmm && !dT_static) return MTPC_ERR_NULL;
  BackwardLayout B;
  plan_backward(c, head->L, T, &B);
  if (bwd_workspace_bytes < B.total || (reinterpret_cast<uintptr_t>(bwd_workspace) % kAlign) != 0)
    return MTPC_ERR_WORKSPACE;
  if ((rc = set_backward_attributes(head)) != MTPC_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* bw = static_cast<uint8_t*>(bwd_workspace);
  const void* hb = nullptr;
  head->draft_P = 0;
  rc = stage_hidden(head, hidden, T, &hb, st);
  if (rc != MTPC_OK) return rc;
  PhaseTimer pt(head, st);
  // 1. forward projection, keeping the units' log-sum-exps
  pt.begin();
  GradArgs fwd;
  fwd.lse_out = reinterpret_cast<float*>(bw + B.off_lse);
  fwd.logit_out = reinterpret_cast<float*>(bw + B.off_logits);
  fwd.logit_pitch = B.Nc;
  rc = launch_gemm(head, kModeLogprob, hb, T, 1, true, true, targets, nullptr, nullptr, st, &fwd);
  pt.end();
  if (rc != MTPC_OK) return rc;
  // 2. circuit backward: posteriors of the input units and of the sum units
  pt.begin();
  if (static_hmm && cudaMemsetAsync(dT_static, 0, static_cast<size_t>(c.n - 1) * c.r * c.r * 4, st) != cudaSuccess)
    return MTPC_ERR_CUDA;
  CircuitBackwardArgs a;
  memset(&a, 0, sizeof(a));
  a.targets = targets;
  a.weight = weight;
  a.weight_stride = 1;
  a.out = out_logprob;
  a.post = reinterpret_cast<float*>(bw + B.off_post);
  a.dsum = reinterpret_cast<__nv_bfloat16*>(bw + B.off_dlogit) + B.Nc;      // columns [Nc, Nc + S r) of the dlogit rows
  a.dsum_pitch = static_cast<int>(B.Kd);
  a.len = c.n;
  a.W = T;
  rc = launch_circuit_backward(head, a, dT_static, st);
  pt.end();
  if (rc != MTPC_OK) return rc;
  // 3., 4. logit gradients from the kept logits, then the plain GEMMs
  return backward_tail(head, B, bw, hb, targets, T, d_hidden, dW_emit, dW_sum, pt, st);
}

int mtpc_lowrank_backward_workspace_bytes(const mtpc_config* cfg, int32_t k, int32_t T, size_t* out_bytes) {
  if (!cfg || !out_bytes) return MTPC_ERR_NULL;
  if (T < 1) return MTPC_ERR_SHAPE;
  Layout L;
  int rc = plan(*cfg, &L);
  if (rc != MTPC_OK) return rc;
  LowRankGemmParams lrp;
  if (cfg->io_dtype != MTPC_BF16 || !plan_lowrank(*cfg, k, &lrp)) return MTPC_ERR_UNSUPPORTED;
  LowRankBackwardLayout R;
  plan_lowrank_backward(*cfg, L, k, T, &R);
  *out_bytes = R.total;
  return MTPC_OK;
}

int mtpc_lowrank_window_logprob_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                                         const float* weight, void* bwd_workspace, size_t bwd_workspace_bytes,
                                         float* out_logprob, float* d_hidden, float* dW_base, float* dA, float* dB,
                                         float* dW_sum, float* dT_static, void* stream) {
  int rc = check_call(head, T);
  if (rc != MTPC_OK) return rc;
  if (T == 0) return MTPC_OK;
  if (!hidden || !targets || !weight || !bwd_workspace || !d_hidden || !dW_base || !dA || !dB || !dW_sum) return MTPC_ERR_NULL;
  if (head->lr_k == 0) return MTPC_ERR_STATE;                  // a head on a composed tensor: mtpc_window_logprob_backward
  const mtpc_config& c = head->cfg;
  const Layout& L = head->L;
  const int k = head->lr_k;
  const bool static_hmm = c.family == MTPC_HMM && !is_ctx(head) && c.n > 1;
  if (static_hmm && !dT_static) return MTPC_ERR_NULL;
  LowRankBackwardLayout R;
  plan_lowrank_backward(c, L, k, T, &R);
  const BackwardLayout& B = R.B;
  if (bwd_workspace_bytes < R.total || (reinterpret_cast<uintptr_t>(bwd_workspace) % kAlign) != 0) return MTPC_ERR_WORKSPACE;
  if ((rc = set_backward_attributes(head)) != MTPC_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* bw = static_cast<uint8_t*>(bwd_workspace);
  const void* hb = hidden;                                     // (factored heads are bf16)
  head->draft_P = 0;
  PhaseTimer pt(head, st);
  // 1. factored forward projection, keeping every logit and every unit's log-sum-exp
  pt.begin();
  GradArgs fwd;
  fwd.lse_out = reinterpret_cast<float*>(bw + B.off_lse);
  fwd.logit_out = reinterpret_cast<float*>(bw + B.off_logits);
  fwd.logit_pitch = B.Nc;
  rc = launch_lowrank_projection(head, hb, T, targets, st, &fwd);
  pt.end();
  if (rc != MTPC_OK) return rc;
  // 2. circuit backward: posteriors of the input units; the sum units' logit gradients go to the right of sy
  pt.begin();
  if (static_hmm && cudaMemsetAsync(dT_static, 0, static_cast<size_t>(c.n - 1) * c.r * c.r * 4, st) != cudaSuccess)
    return MTPC_ERR_CUDA;
  __nv_bfloat16* sy = reinterpret_cast<__nv_bfloat16*>(bw + R.off_sy);
  CircuitBackwardArgs a;
  memset(&a, 0, sizeof(a));
  a.targets = targets;
  a.weight = weight;
  a.weight_stride = 1;
  a.out = out_logprob;
  a.post = reinterpret_cast<float*>(bw + B.off_post);
  a.dsum = sy + R.Ksy;
  a.dsum_pitch = static_cast<int>(R.pitch);
  a.len = c.n;
  a.W = T;
  rc = launch_circuit_backward(head, a, dT_static, st);
  pt.end();
  if (rc != MTPC_OK) return rc;
  // 3., 4. logit gradients and what is derived from them, then the GEMMs
  return lowrank_backward_tail(head, R, bw, hb, targets, T, d_hidden, dW_base, dA, dB, dW_sum, pt, st);
}

}  // extern "C"

// Eq. 6 loss and its gradients, on a head built on a composed tensor (dW_emit) or on a factored one (dW_base, dA, dB): the
// two differ in the projection that keeps the logits and in the GEMMs at the end.
static int window_loss_backward_impl(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                                     int32_t sequence_length, float gamma, void* bwd_workspace, size_t bwd_workspace_bytes,
                                     float* out_slot_loss, float* out_loss, float* d_hidden, float* dW_emit, float* dW_base,
                                     float* dA, float* dB, float* dW_sum, float* dT_static, void* stream) {
  if (!head) return MTPC_ERR_NULL;
  if (num_sequences < 1 || sequence_length < 1) return MTPC_ERR_SHAPE;
  const int64_t T64 = static_cast<int64_t>(num_sequences) * sequence_length;
  if (T64 > head->cfg.max_positions) return MTPC_ERR_SHAPE;
  if (!hidden || !targets || !bwd_workspace || !out_slot_loss || !out_loss || !d_hidden || !dW_sum) return MTPC_ERR_NULL;
  const bool factored = head->lr_k > 0;
  if (factored ? (!dW_base || !dA || !dB) : !dW_emit) return MTPC_ERR_NULL;
  const int T = static_cast<int>(T64);
  const mtpc_config& c = head->cfg;
  const Layout& L = head->L;
  const bool static_hmm = c.family == MTPC_HMM && !is_ctx(head) && c.n > 1;
  if (static_hmm && !dT_static) return MTPC_ERR_NULL;
  LowRankBackwardLayout R;
  memset(&R, 0, sizeof(R));
  if (factored) plan_lowrank_backward(c, L, head->lr_k, T, &R);
  else plan_backward(c, L, T, &R.B);
  const BackwardLayout& B = R.B;
  if (bwd_workspace_bytes < (factored ? R.total : B.total) || (reinterpret_cast<uintptr_t>(bwd_workspace) % kAlign) != 0)
    return MTPC_ERR_WORKSPACE;
  int rc = set_backward_attributes(head);
  if (rc != MTPC_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* bw = static_cast<uint8_t*>(bwd_workspace);
  float* post = reinterpret_cast<float*>(bw + B.off_post);
  float* dsum_f32 = reinterpret_cast<float*>(bw + B.off_dsum_f32);
  float* coeff = reinterpret_cast<float*>(bw + B.off_coeff);
  float* prefix = at<float>(head, L.off_prefix);
  float* partial = at<float>(head, L.off_partial);
  const void* hb = nullptr;
  head->draft_P = 0;
  rc = stage_hidden(head, hidden, T, &hb, st);
  if (rc != MTPC_OK) return rc;
  PhaseTimer pt(head, st);
  // 1. forward projection (keeping the log-sum-exps), prefix marginals, the loss of Eq. 6 and the weight of every prefix
  pt.begin();
  GradArgs fwd;
  fwd.lse_out = reinterpret_cast<float*>(bw + B.off_lse);
  fwd.logit_out = reinterpret_cast<float*>(bw + B.off_logits);
  fwd.logit_pitch = B.Nc;
  rc = factored ? launch_lowrank_projection(head, hb, T, targets, st, &fwd)
                : launch_gemm(head, kModeLogprob, hb, T, 1, true, true, targets, nullptr, nullptr, st, &fwd);
  if (rc == MTPC_OK) rc = launch_circuit(head, T, 1, nullptr, prefix, st);
  if (rc != MTPC_OK) return rc;
  // the sum units' logit gradients (bf16): to the right of dlogit, or of [s | y] on a factored head
  __nv_bfloat16* dsum_bf16 = factored ? reinterpret_cast<__nv_bfloat16*>(bw + R.off_sy) + R.Ksy
                                      : reinterpret_cast<__nv_bfloat16*>(bw + B.off_dlogit) + B.Nc;
  const size_t dsum_bf16_pitch = factored ? R.pitch : B.Kd;
  loss_partial_kernel<<<num_sequences, kLossThreads, 0, st>>>(prefix, targets, partial, sequence_length, c.n);
  loss_final_kernel<<<1, kLossThreads, 0, st>>>(partial, out_slot_loss, out_loss, num_sequences, c.n, gamma);
  loss_coeff_kernel<<<num_sequences, kLossThreads, 0, st>>>(targets, coeff, sequence_length, c.n, num_sequences, gamma);
  head->launches += 3;
  pt.end();
  if ((rc = check_launch()) != MTPC_OK) return rc;
  // 2. circuit backward. HMM: every prefix marginal is a forward message, so one reverse sweep gives the whole gradient.
  // Mixture and tree: one pass per prefix length, accumulating.
  pt.begin();
  if (static_hmm && cudaMemsetAsync(dT_static, 0, static_cast<size_t>(c.n - 1) * c.r * c.r * 4, st) != cudaSuccess)
    return MTPC_ERR_CUDA;
  if (c.family == MTPC_HMM) {
    CircuitBackwardArgs a;
    memset(&a, 0, sizeof(a));
    a.targets = targets;
    a.post = post;
    a.dsum = dsum_bf16;
    a.dsum_pitch = static_cast<int>(dsum_bf16_pitch);
    a.len = c.n;
    a.W = T;
    if ((rc = launch_circuit_backward(head, a, dT_static, st, coeff)) != MTPC_OK) return rc;
  } else {
    bool bad = cudaMemsetAsync(post, 0, static_cast<size_t>(T) * c.n * c.r * 4, st) != cudaSuccess;
    bad |= cudaMemsetAsync(dsum_f32, 0, static_cast<size_t>(T) * L.sum_rows * 4, st) != cudaSuccess;
    if (bad) return MTPC_ERR_CUDA;
    CircuitBackwardArgs a;
    memset(&a, 0, sizeof(a));
    a.targets = targets;
    a.post = post;
    a.dsum_f32 = dsum_f32;
    a.dsum_pitch = L.sum_rows;
    a.accumulate = 1;
    a.W = T;
    if (c.family == MTPC_BTREE) {                 // every prefix length of a window by the same warp, back to back
      a.len = c.n;
      if ((rc = launch_circuit_backward(head, a, dT_static, st, coeff)) != MTPC_OK) return rc;
    } else {
      for (int j = 0; j < c.n; ++j) {               // mixture: one cheap pass per prefix length
        a.weight = coeff + j;
        a.weight_stride = c.n;
        a.len = j + 1;
        if ((rc = launch_circuit_backward(head, a, dT_static, st)) != MTPC_OK) return rc;
      }
    }
    const size_t total = static_cast<size_t>(T) * L.sum_rows;
    const int blocks = static_cast<int>((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
    f32_rows_to_bf16_kernel<<<blocks, 256, 0, st>>>(dsum_f32, dsum_bf16, T, L.sum_rows, L.sum_rows, dsum_bf16_pitch);
    head->launches++;
  }
  pt.end();
  if ((rc = check_launch()) != MTPC_OK) return rc;
  if (factored) return lowrank_backward_tail(head, R, bw, hb, targets, T, d_hidden, dW_base, dA, dB, dW_sum, pt, st);
  return backward_tail(head, B, bw, hb, targets, T, d_hidden, dW_emit, dW_sum, pt, st);
}

extern "C" {

int mtpc_window_loss_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                              int32_t sequence_length, float gamma, void* bwd_workspace, size_t bwd_workspace_bytes,
                              float* out_slot_loss, float* out_loss, float* d_hidden, float* dW_emit, float* dW_sum,
                              float* dT_static, void* stream) {
  if (head && head->lr_k > 0) return MTPC_ERR_UNSUPPORTED;     // a factored head: mtpc_lowrank_window_loss_backward
  return window_loss_backward_impl(head, hidden, targets, num_sequences, sequence_length, gamma, bwd_workspace,
                                   bwd_workspace_bytes, out_slot_loss, out_loss, d_hidden, dW_emit, nullptr, nullptr, nullptr,
                                   dW_sum, dT_static, stream);
}

int mtpc_lowrank_window_loss_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                                      int32_t sequence_length, float gamma, void* bwd_workspace, size_t bwd_workspace_bytes,
                                      float* out_slot_loss, float* out_loss, float* d_hidden, float* dW_base, float* dA,
                                      float* dB, float* dW_sum, float* dT_static, void* stream) {
  if (head && head->lr_k == 0) return MTPC_ERR_STATE;          // a head on a composed tensor: mtpc_window_loss_backward
  return window_loss_backward_impl(head, hidden, targets, num_sequences, sequence_length, gamma, bwd_workspace,
                                   bwd_workspace_bytes, out_slot_loss, out_loss, d_hidden, nullptr, dW_base, dA, dB, dW_sum,
                                   dT_static, stream);
}

// Streams and events of the chunked host-buffer path; no device memory is allocated.
static int ensure_copy_pipeline(mtpc_head* head, int chunks) {
  if (!head->copy_stream && cudaStreamCreateWithFlags(&head->copy_stream, cudaStreamNonBlocking) != cudaSuccess)
    return MTPC_ERR_CUDA;
  if (head->copy_event_count < chunks + 1) {
    cudaEvent_t* ev = static_cast<cudaEvent_t*>(calloc(chunks + 1, sizeof(cudaEvent_t)));
    if (!ev) return MTPC_ERR_CUDA;
    for (int i = 0; i < chunks + 1; ++i) {
      if (i < head->copy_event_count) ev[i] = head->copy_events[i];
      else if (cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) != cudaSuccess) { free(ev); return MTPC_ERR_CUDA; }
    }
    free(head->copy_events);
    head->copy_events = ev;
    head->copy_event_count = chunks + 1;
  }
  return MTPC_OK;
}

int mtpc_lowrank_compose(int32_t n, int32_t r, int32_t v, int32_t d, int32_t k, const void* W_base, const void* A,
                         const void* B, void* W_emit_out, void* stream) {
  if (!W_base || !A || !B || !W_emit_out) return MTPC_ERR_NULL;
  if (n < 1 || r < 1 || v < 1 || d < 1 || k < 1 || static_cast<int64_t>(n) * r > 65535 ||
      (v + kComposeCtaRows - 1) / kComposeCtaRows > 65535)
    return MTPC_ERR_SHAPE;
  if (k > kLowRankMaxK) return MTPC_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const auto* w = static_cast<const __nv_bfloat16*>(W_base);
  const auto* a = static_cast<const __nv_bfloat16*>(A);
  const auto* b = static_cast<const __nv_bfloat16*>(B);
  auto* u = static_cast<__nv_bfloat16*>(W_emit_out);
  const int rows = (v + kComposeCtaRows - 1) / kComposeCtaRows;
  if (lowrank_vector_ok(d, {W_base, B, W_emit_out})) {
    const size_t smem = compose_smem_bytes(k, 4);
    if (cudaFuncSetAttribute(lowrank_compose_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
        cudaSuccess)
      return MTPC_ERR_CUDA;
    lowrank_compose_kernel<4><<<dim3((d + 4 * kLowRankThreads - 1) / (4 * kLowRankThreads), rows, n * r), kLowRankThreads, smem,
                                st>>>(w, a, b, u, r, v, d, k);
  } else {
    const size_t smem = compose_smem_bytes(k, 1);
    lowrank_compose_kernel<1><<<dim3((d + kLowRankThreads - 1) / kLowRankThreads, rows, n * r), kLowRankThreads, smem, st>>>(
        w, a, b, u, r, v, d, k);
  }
  return check_launch();
}

int mtpc_lowrank_backward(int32_t n, int32_t r, int32_t v, int32_t d, int32_t k, const void* A, const void* B,
                          const float* dW_emit, float* dW_base, float* dA, float* dB, void* stream) {
  if (!A || !B || !dW_emit || !dW_base || !dA || !dB) return MTPC_ERR_NULL;
  if (n < 1 || r < 1 || v < 1 || d < 1 || k < 1 || v > 65535 || static_cast<int64_t>(n) * r > 65535) return MTPC_ERR_SHAPE;
  if (k > kLowRankMaxK) return MTPC_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const auto* a = static_cast<const __nv_bfloat16*>(A);
  const auto* b = static_cast<const __nv_bfloat16*>(B);
  const int units = n * r, kchunks = (k + kRankChunk - 1) / kRankChunk;
  auto blocks = [&](int cv) { return (d + cv * kLowRankThreads - 1) / (cv * kLowRankThreads); };
  if (lowrank_vector_ok(d, {B, dW_emit, dW_base, dB})) {
    lowrank_dw_kernel<4><<<dim3(blocks(4), v, n), kLowRankThreads, 0, st>>>(dW_emit, dW_base, r, v, d);
    lowrank_da_kernel<4><<<dim3((v + 31) / 32, units), kLowRankThreads, 0, st>>>(dW_emit, b, dA, v, d, k);
    lowrank_db_kernel<4><<<dim3(blocks(4), kchunks, units), kLowRankThreads, 0, st>>>(dW_emit, a, dB, v, d, k);
  } else {
    lowrank_dw_kernel<1><<<dim3(blocks(1), v, n), kLowRankThreads, 0, st>>>(dW_emit, dW_base, r, v, d);
    lowrank_da_kernel<1><<<dim3((v + 31) / 32, units), kLowRankThreads, 0, st>>>(dW_emit, b, dA, v, d, k);
    lowrank_db_kernel<1><<<dim3(blocks(1), kchunks, units), kLowRankThreads, 0, st>>>(dW_emit, a, dB, v, d, k);
  }
  return check_launch();
}

int mtpc_window_logprob_host(mtpc_head* head, const void* hidden_host, const int32_t* targets_host, int32_t T,
                             float* out_logprob_host, void* stream) {
  int rc = check_call(head, T);
  if (rc != MTPC_OK) return rc;
  if (T == 0) return MTPC_OK;
  if (!hidden_host || !targets_host || !out_logprob_host) return MTPC_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Layout& L = head->L;
  const mtpc_config& c = head->cfg;
  const size_t elt = c.io_dtype == MTPC_F32 ? 4 : 2;
  uint8_t* dh = head->ws + L.off_h_hidden;
  int32_t* dt = at<int32_t>(head, L.off_h_targets);
  float* dout = at<float>(head, L.off_h_out);
  // The positions are uploaded in chunks on a second stream while the kernels of the chunks before run on `stream`:
  // only the first chunk's upload is not hidden behind compute.
  const int chunks = (T + kHostChunkPositions - 1) / kHostChunkPositions;
  if ((rc = ensure_copy_pipeline(head, chunks)) != MTPC_OK) return rc;
  cudaStream_t cs = head->copy_stream;
  bool fail = cudaEventRecord(head->copy_events[chunks], st) != cudaSuccess;     // uploads wait for earlier work on `stream`
  fail |= cudaStreamWaitEvent(cs, head->copy_events[chunks], 0) != cudaSuccess;
  for (int k = 0; k < chunks && !fail; ++k) {
    const size_t t0 = static_cast<size_t>(k) * kHostChunkPositions;
    const size_t tc = (T - t0) < static_cast<size_t>(kHostChunkPositions) ? (T - t0) : kHostChunkPositions;
    fail |= cudaMemcpyAsync(dh + t0 * c.d * elt, static_cast<const uint8_t*>(hidden_host) + t0 * c.d * elt, tc * c.d * elt,
                            cudaMemcpyHostToDevice, cs) != cudaSuccess;
    fail |= cudaMemcpyAsync(dt + t0 * c.n, targets_host + t0 * c.n, tc * c.n * 4, cudaMemcpyHostToDevice, cs) != cudaSuccess;
    fail |= cudaEventRecord(head->copy_events[k], cs) != cudaSuccess;
  }
  if (fail) return MTPC_ERR_CUDA;
  for (int k = 0; k < chunks; ++k) {
    const size_t t0 = static_cast<size_t>(k) * kHostChunkPositions;
    const int tc = static_cast<int>((T - t0) < static_cast<size_t>(kHostChunkPositions) ? (T - t0) : kHostChunkPositions);
    if (cudaStreamWaitEvent(st, head->copy_events[k], 0) != cudaSuccess) return MTPC_ERR_CUDA;
    rc = window_logprob_impl(head, dh + t0 * c.d * elt, dt + t0 * c.n, tc, dout + t0, nullptr, st);
    if (rc != MTPC_OK) { cudaStreamSynchronize(cs); return rc; }
  }
  fail = cudaMemcpyAsync(out_logprob_host, dout, static_cast<size_t>(T) * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess;
  fail |= cudaStreamSynchronize(st) != cudaSuccess;
  return fail ? MTPC_ERR_CUDA : MTPC_OK;
}

int mtpc_draft_sample_host(mtpc_head* head, const void* hidden_host, int32_t P, int32_t wpp,
                           const float* uniforms_host, int32_t* out_bytes_host, float* out_logprob_host,
                           void* stream) {
  int rc = check_call(head, P);
  if (rc != MTPC_OK) return rc;
  if (wpp < 1 || wpp > head->cfg.max_windows_per_pos) return MTPC_ERR_SHAPE;
  if (P == 0) return MTPC_OK;
  if (!hidden_host || !uniforms_host || !out_bytes_host || !out_logprob_host) return MTPC_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Layout& L = head->L;
  const mtpc_config& c = head->cfg;
  const size_t elt = c.io_dtype == MTPC_F32 ? 4 : 2;
  const size_t W = static_cast<size_t>(P) * wpp;
  void* dh = head->ws + L.off_h_hidden;
  float* du = at<float>(head, L.off_h_uniforms);
  int32_t* db = at<int32_t>(head, L.off_h_bytes);
  float* dout = at<float>(head, L.off_h_out);
  bool fail = cudaMemcpyAsync(dh, hidden_host, static_cast<size_t>(P) * c.d * elt, cudaMemcpyHostToDevice, st) !=
              cudaSuccess;
  fail |= cudaMemcpyAsync(du, uniforms_host, W * 2 * c.n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess;
  if (fail) return MTPC_ERR_CUDA;
  rc = draft_sample_impl(head, dh, P, wpp, du, db, dout, nullptr, st);
  if (rc != MTPC_OK) return rc;
  fail = cudaMemcpyAsync(out_bytes_host, db, W * c.n * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess;
  fail |= cudaMemcpyAsync(out_logprob_host, dout, W * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess;
  fail |= cudaStreamSynchronize(st) != cudaSuccess;
  return fail ? MTPC_ERR_CUDA : MTPC_OK;
}

int mtpc_get_status(mtpc_head* head, void* stream, uint32_t* out_flags) {
  if (!head || !out_flags) return MTPC_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t flags = 0;
  void* dev = head->ws + head->L.off_status;
  if (cudaMemcpyAsync(&flags, dev, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MTPC_ERR_CUDA;
  if (cudaMemsetAsync(dev, 0, 4, st) != cudaSuccess) return MTPC_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MTPC_ERR_CUDA;
  *out_flags = flags;
  return (flags & MTPC_STATUS_TIMEOUT) ? MTPC_ERR_TIMEOUT : MTPC_OK;
}

static void free_timing(mtpc_head* head) {
  if (head->ev) {
    for (size_t i = 0; i < static_cast<size_t>(head->ring) * kMaxPhases * 2; ++i) cudaEventDestroy(head->ev[i]);
    free(head->ev);
    free(head->ring_phases);
  }
  head->ev = nullptr;
  head->ring_phases = nullptr;
  head->ring = 0;
  head->calls = 0;
}

int mtpc_set_timing(mtpc_head* head, int32_t ring) {
  if (!head) return MTPC_ERR_NULL;
  if (ring < 0 || ring > 4096) return MTPC_ERR_SHAPE;
  free_timing(head);
  if (ring == 0) return MTPC_OK;
  const size_t count = static_cast<size_t>(ring) * kMaxPhases * 2;
  head->ev = static_cast<cudaEvent_t*>(calloc(count, sizeof(cudaEvent_t)));
  head->ring_phases = static_cast<int*>(calloc(ring, sizeof(int)));
  if (!head->ev || !head->ring_phases) { free(head->ev); free(head->ring_phases); head->ev = nullptr; return MTPC_ERR_CUDA; }
  head->ring = ring;
  for (size_t i = 0; i < count; ++i)
    if (cudaEventCreate(&head->ev[i]) != cudaSuccess) { head->ring = 0; return MTPC_ERR_CUDA; }
  return MTPC_OK;
}

int mtpc_get_timing(mtpc_head* head, int32_t calls_back, float* out_ms, int32_t capacity, int32_t* out_count) {
  if (!head || !out_ms || !out_count) return MTPC_ERR_NULL;
  *out_count = 0;
  if (head->ring == 0) return MTPC_OK;
  if (calls_back < 0 || calls_back >= head->ring || static_cast<uint64_t>(calls_back) >= head->calls)
    return MTPC_ERR_SHAPE;
  const int slot = static_cast<int>((head->calls - 1 - calls_back) % head->ring);
  const int nph = head->ring_phases[slot];
  for (int i = 0; i < nph && i < capacity; ++i) {
    cudaEvent_t* pair = head->ev + (static_cast<size_t>(slot) * kMaxPhases + i) * 2;
    if (cudaEventSynchronize(pair[1]) != cudaSuccess) return MTPC_ERR_CUDA;
    if (cudaEventElapsedTime(&out_ms[i], pair[0], pair[1]) != cudaSuccess) return MTPC_ERR_CUDA;
    *out_count = i + 1;
  }
  return MTPC_OK;
}

int mtpc_debug_set_wait_limit_ns(mtpc_head* head, uint64_t limit_ns) {
  if (!head) return MTPC_ERR_NULL;
  head->wait_limit_ns = limit_ns == 0 ? kWaitLimitNs : limit_ns;
  return MTPC_OK;
}

int mtpc_debug_set_projection_variant(mtpc_head* head, int32_t variant) {
  if (!head) return MTPC_ERR_NULL;
  if (variant < 0 || variant > 2) return MTPC_ERR_SHAPE;
  if (variant == 2 && head->max_pairs <= 0) return MTPC_ERR_UNSUPPORTED;
  head->projection_variant = variant;
  return MTPC_OK;
}

int mtpc_debug_set_draft_grouping(mtpc_head* head, int32_t mode) {
  if (!head) return MTPC_ERR_NULL;
  if (mode < 0 || mode > 2) return MTPC_ERR_SHAPE;
  if (mode == 2 && head->L.group_entries == 0) return MTPC_ERR_UNSUPPORTED;
  head->draft_grouping = mode;
  return MTPC_OK;
}

int mtpc_launch_count(mtpc_head* head, uint64_t* out_count) {
  if (!head || !out_count) return MTPC_ERR_NULL;
  *out_count = head->launches;
  return MTPC_OK;
}

int mtpc_destroy(mtpc_head* head) {
  if (!head) return MTPC_ERR_NULL;
  free_timing(head);
  for (int i = 0; i < head->copy_event_count; ++i) cudaEventDestroy(head->copy_events[i]);
  free(head->copy_events);
  if (head->copy_stream) cudaStreamDestroy(head->copy_stream);
  delete head;
  return MTPC_OK;
}

const char* mtpc_status_string(int code) {
  switch (code) {
    case MTPC_OK: return "ok";
    case MTPC_ERR_NULL: return "a required pointer is NULL";
    case MTPC_ERR_SHAPE: return "a size argument is out of range";
    case MTPC_ERR_UNSUPPORTED: return "configuration not supported by this version";
    case MTPC_ERR_WORKSPACE: return "workspace too small or misaligned";
    case MTPC_ERR_CUDA: return "a CUDA call failed (no sm_100 device, launch error, or driver entry point missing)";
    case MTPC_ERR_TIMEOUT: return "a device-side bounded wait expired";
    case MTPC_ERR_STATE:
      return "the head holds no draft state for this call (mtpc_speculative_accept must follow a draft of the same positions)";
    case MTPC_ERR_STATIC_SCRATCH:
      return "the call needs more scratch than the library's built-in static array holds (mtpc_window_logprob_static)";
    default: return "unknown status code";
  }
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------------------
// mtpc_window_logprob_static: the window log-likelihood for callers that have no device allocator at hand.
// All scratch (status word, log-softmaxed HMM transitions, G, log omega) is carved out of one file-scope device
// array, so the call needs neither a head nor a caller-made workspace and allocates nothing.
// ------------------------------------------------------------------------------------------------------------
namespace {

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[MTPC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices];   // device address of the array on each device, 0 = not looked up yet

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the address the
// kernels need comes from cudaGetSymbolAddress, asked once per device with that device current.
int static_scratch_address(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MTPC_ERR_CUDA;
  void* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return MTPC_ERR_CUDA;
    __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);   // every thread gets the same answer
  }
  *out = static_cast<unsigned char*>(p);
  return MTPC_OK;
}

}  // namespace

extern "C" int mtpc_window_logprob_static(const mtpc_config* cfg, const void* W_emit, const void* W_sum,
                                          const float* T_static, const void* hidden, const int32_t* targets,
                                          int32_t T, float* out_logprob, uint32_t* out_status, void* stream) {
  if (!cfg) return MTPC_ERR_NULL;
  if (cfg->io_dtype != MTPC_BF16) return MTPC_ERR_UNSUPPORTED;   // fp32 inputs would need rounded copies of the weights
  if (cfg->flags != 0) return MTPC_ERR_UNSUPPORTED;
  if (T < 0) return MTPC_ERR_SHAPE;
  mtpc_config c = *cfg;
  c.max_positions = T > 0 ? T : 1;
  c.max_windows_per_pos = 1;
  Layout L;
  int rc = plan(c, &L);
  if (rc != MTPC_OK) return rc;
  // Carve only what this call needs: [status | logA (HMM) | G | log omega].
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  L.off_status = take(256);
  L.off_logA = take(c.family == MTPC_HMM ? static_cast<size_t>(c.n - 1) * c.r * c.r * 4 : 0);
  L.off_G = take(static_cast<size_t>(c.max_positions) * c.n * c.r * 4);
  L.off_logw = take(static_cast<size_t>(c.max_positions) * L.sum_rows * 4);
  L.off_sel = L.off_wemit = L.off_wsum = L.off_hidden = L.off_logits = L.off_unit_lse = 0;   // unused by this call
  L.off_prefix = L.off_partial = L.off_sum_bias = 0;
  L.off_h_hidden = L.off_h_targets = L.off_h_uniforms = L.off_h_bytes = L.off_h_out = 0;
  L.total = off;
  if (L.total > static_cast<size_t>(MTPC_STATIC_SCRATCH_BYTES)) return MTPC_ERR_STATIC_SCRATCH;
  if (T == 0) return MTPC_OK;
  if (!W_emit || !W_sum || !hidden || !targets || !out_logprob) return MTPC_ERR_NULL;
  if (c.family == MTPC_HMM && c.n > 1 && !T_static) return MTPC_ERR_NULL;

  int dev = 0, cc_major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MTPC_ERR_CUDA;
  if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || cc_major != 10)
    return MTPC_ERR_CUDA;
  unsigned char* scratch = nullptr;
  if ((rc = static_scratch_address(&scratch)) != MTPC_OK) return rc;

  mtpc_head h;                       // host-side bookkeeping only, lives for the duration of this call
  memset(&h, 0, sizeof(h));
  h.cfg = c;
  h.L = L;
  h.ws = scratch;
  h.W_emit_bf16 = W_emit;
  h.W_sum_bf16 = W_sum;
  h.wait_limit_ns = kWaitLimitNs;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool fail = cudaDeviceGetAttribute(&h.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess;
  fail |= cudaFuncSetAttribute(mtpc_gemm_kernel<kModeLogprob, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kSmemLimit) != cudaSuccess;
  fail |= !set_circuit_attributes();
  // The array keeps whatever the previous call left in it. Only the status word has to start at zero; G, log omega
  // and logA are fully rewritten for the rows this call reads.
  fail |= cudaMemsetAsync(scratch + L.off_status, 0, 256, st) != cudaSuccess;
  if (fail) return MTPC_ERR_CUDA;
  if (c.family == MTPC_HMM && c.n > 1) {
    const int rows = (c.n - 1) * c.r;
    log_softmax_rows_kernel<<<(rows + 127) / 128, 128, 0, st>>>(T_static, at<float>(&h, L.off_logA), rows, c.r);
    if (check_launch() != MTPC_OK) return MTPC_ERR_CUDA;
  }
  rc = make_tmap(&h.tm_emit_lp, W_emit, static_cast<uint64_t>(c.n) * c.r * c.v, c.d, L.lp.tile_cols);
  if (rc == MTPC_OK) rc = make_tmap(&h.tm_sum, W_sum, L.sum_rows, c.d, L.sum_cols);
  if (rc != MTPC_OK) return rc;
  rc = window_logprob_impl(&h, hidden, targets, T, out_logprob, nullptr, st);
  if (rc != MTPC_OK) return rc;
  if (out_status &&
      cudaMemcpyAsync(out_status, scratch + L.off_status, 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return MTPC_ERR_CUDA;
  return MTPC_OK;
}
