// Projection kernel of the MtPC head (Sec. 3.3): logits = h W^T on the tcgen05 tensor cores, with the softmax
// over the vocabulary, the evidence gather (log phi at the target byte) or the inverse-CDF byte draw
// (Algorithm 1, input units), and the log-softmax of the sum-unit logits all done in the epilogue straight
// out of tensor memory. The [positions, n, r, v] logit tensor never exists in HBM, except when a training call asks the
// epilogue to keep it for the backward pass (logit_out).
//
// One persistent CTA per SM, 6 warps:
//   warp 0      TMA producer: per 64-wide K block, one 128-row tile of h and the v rows of one emission unit
//               (or one tile of sum-unit rows) into a ring of shared-memory stages (128-byte swizzle).
//   warp 1      allocates the 512 TMEM columns, issues tcgen05.mma (M=128, N=chunk, K=16) from one thread.
//   warps 2..5  epilogue; warp w reads TMEM lanes 32*(w%4)..+31, one thread per position (row), so every
//               row-wise reduction over the vocabulary is a plain in-thread loop.
// The N axis of the GEMM is the flattened (slot i, unit k, byte b) row index of W_emit. A work item is 128
// positions x one "group": `group_units` consecutive emission units = a run of rows that starts at a unit
// boundary, covered by accumulator tiles of `tile_cols` columns. The log-likelihood mode uses 256-column tiles
// whatever v is (v=320: 4 units = 1280 rows = 5 tiles; v=256: 1 unit = 1 tile): a tile may then hold the end
// of one unit and the start of the next, and the epilogue carries its running max / sum across tiles and
// closes a unit whenever its v-th column has been consumed. The sampling mode needs a whole unit on chip at
// once and uses one unit per group (v=320 -> 2 tiles of 160). Sum-unit rows form work items of their own
// (one tile of `sum_cols` columns). Accumulators live in a ring of TMEM slots, so the epilogue of one tile
// overlaps the MMAs of the next. Every barrier wait is bounded: when one runs out the CTA raises
// MTPC_STATUS_TIMEOUT in the status word, drains its copies, frees its TMEM and returns.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>

#include "mtpc_group.cuh"
#include "mtpc_ptx.cuh"

namespace mtpc {

constexpr int kBlockM = 128;         // positions per tile (= TMEM lanes)
constexpr int kBlockK = 64;          // bf16 elements per 128-byte swizzled row
#ifndef MTPC_MAX_STAGES
#define MTPC_MAX_STAGES 8
#endif
constexpr int kMaxStages = MTPC_MAX_STAGES;
constexpr int kMaxSlots = 16;
constexpr int kTmemCols = 512;
constexpr int kGemmThreads = 192;
constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;   // 1 s per barrier wait (the default, and always the limit of the drain waits)
constexpr uint64_t kAbortSettleNs = 200ull * 1000ull;            // 0.2 ms: far longer than any copy or MMA in flight takes
constexpr int kABytes = kBlockM * kBlockK * 2;                   // 16 KB
constexpr uint32_t kStatusBadTarget = 1u, kStatusBadUniform = 2u, kStatusTimeout = 4u;

// kModeSampleGrouped: the byte draws again, on rows that were sorted by the unit they sample from (mtpc_group.cuh):
// a work item is one GroupTile instead of (m-tile, unit).
// kModeLogitsGrouped: rows sorted by SLOT (the acceptance stage after a many-position draft): a work item is a GroupTile
// whose `unit` is a slot; the logits of the slot's r units and their log-sum-exps are written out per staged row.
enum { kModeLogprob = 0, kModeSample = 1, kModeSampleGrouped = 2, kModeLogitsGrouped = 3 };

struct GemmParams {
  CUtensorMap tm_a;      // hidden  [T, d]        box 64 x 128
  CUtensorMap tm_emit;   // W_emit  [n*r*v, d]    box 64 x tile_cols
  CUtensorMap tm_sum;    // W_sum   [S*r, d]      box 64 x sum_cols
  int T, m_tiles, kblocks;
  int m_units;                       // M work units: m-tiles, or pairs of m-tiles when two CTAs share every MMA
  int m_block;                       // M work units per rasterisation block (see tile_coord)
  int n, r, v;
  int vv;                            // symbols that exist (<= v, > v - 16): the columns [vv, v) of every unit are padding
  int emit_units;                    // n * r
  int num_groups;                    // emission groups in this launch (0: sum tiles only)
  int group_units;                   // emission units per full group (the last group may hold fewer)
  int tile_cols;                     // accumulator width of an emission tile
  int num_sum_tiles;                 // sum tiles in this launch (0: emission groups only)
  int sum_cols, sum_rows;            // sum tile width; S * r
  int slot_stride, num_slots;
  int stages, stage_bytes;
  int wpp;                           // windows (target rows) per position
  const int* targets;                // [T*wpp, n]
  int missing_is_nan;                // a negative target is a refused draw (G = NaN), not a byte to sum out (G = 0)
  float* G;                          // [T*wpp, n, r]   log phi at the target
  float* logw;                       // [T, S*r]        log-softmaxed sum-unit weights
  const float* sum_bias;             // [S*r] or NULL   added to the sum-unit logits before their softmax
  float* lse_out;                    // [T, n, r] or NULL: log-sum-exp of every input unit, kept for the backward pass
  float* logit_out;                  // [T, n*r*v] fp32 with row pitch logit_pitch, or NULL: the emission logits themselves,
  size_t logit_pitch;                // kept for the backward pass (padding columns as -inf); wpp == 1 only
  const int* unit_sel;               // [T*wpp, n]      selected input unit per token (sample mode)
  const float* uniforms;             // [T*wpp, 2n]
  int* out_bytes;                    // [T*wpp, n]
  const GroupTile* group_tiles;      // grouped sampling: the work items, ...
  const int* group_num_tiles;        // ... how many there are (device memory: written by the kernel that made them), ...
  const int* group_perm;             // ... and which (window, slot) pair every row of the staged hidden states (tm_a) holds
  int group_two_pass;                // grouped sampling of a unit too wide for tensor memory: its tiles are computed twice
  unsigned* status;
  uint64_t wait_limit_ns;            // limit of every pipeline wait (kWaitLimitNs unless a test shortened it)
};

struct GemmControl {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tfull[kMaxSlots];
  uint64_t tempty[kMaxSlots];
  uint64_t drain;
  uint64_t wait_limit_ns;
  uint32_t tmem_base;
  volatile int abort;
};

__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fast_lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, GemmControl* ctl, unsigned* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  uint32_t it = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++it & 63u) == 0) {
      if (ctl->abort) return false;
      if (global_timer_ns() - t0 > ctl->wait_limit_ns) {
        ctl->abort = 1;
        atomicOr(status, kStatusTimeout);
        return false;
      }
    }
  }
}
// Lane 0 waits, the whole warp learns the outcome (keeps the warp converged for the .sync.aligned TMEM loads).
__device__ __forceinline__ bool bounded_wait_warp(uint32_t bar, uint32_t parity, GemmControl* ctl, unsigned* status,
                                                  int lane) {
  int ok = 1;
  if (lane == 0) ok = bounded_wait(bar, parity, ctl, status) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

struct TileCoord {
  int mt, is_sum, ntiles, cols, brow0, unit0, nunits;
  int arow, count;   // first row of the A operand and the rows that count (set by the caller for ungrouped items)
  int wrap;          // tiles per sweep over the item's weight rows: tile t reads the rows of tile t % wrap
};
// A grouped item: `count` staged rows from `row0` on, against the tiles of the one unit they sample from (by_slot: of the
// r units of the one slot whose logits they need).
__device__ __forceinline__ TileCoord group_coord(const GemmParams& p, int item, bool by_slot) {
  const GroupTile g = p.group_tiles[item];
  TileCoord c;
  c.mt = 0;
  c.is_sum = 0;
  c.unit0 = by_slot ? g.unit * p.r : g.unit;
  c.nunits = by_slot ? p.r : 1;
  c.cols = p.tile_cols;
  c.brow0 = c.unit0 * p.v;
  c.wrap = (c.nunits * p.v + p.tile_cols - 1) / p.tile_cols;
  c.ntiles = p.group_two_pass ? 2 * c.wrap : c.wrap;
  c.arow = g.row0;
  c.count = g.count;
  return c;
}
// Work items (c.mt counts M work units: m-tiles, or pairs of m-tiles in the CTA-pair kernel). Emission items come
// first, in blocks of m_block units: inside a block the unit runs fastest and
// the group next, so the CTAs that run at the same time share a few groups' weights through L2 while the block's
// hidden states (m_block x 128 rows) stay L2-resident for every group; a block is finished before the next one
// starts, so the weights are streamed from HBM once per block and the hidden states once. Sum items follow,
// m-tile fastest.
__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int item) {
  TileCoord c;
  const int emit_items = p.num_groups * p.m_units;
  int g;
  if (item < emit_items) {
    const int per_block = p.m_block * p.num_groups;
    const int blk = item / per_block;
    const int rem = item - blk * per_block;
    const int m0 = blk * p.m_block;
    const int mcount = min(p.m_block, p.m_units - m0);   // only the last block can be short
    g = rem / mcount;
    c.mt = m0 + (rem - g * mcount);
  } else {
    const int rem = item - emit_items;
    g = p.num_groups + rem / p.m_units;
    c.mt = rem % p.m_units;
  }
  c.is_sum = g >= p.num_groups;
  if (c.is_sum) {
    c.ntiles = 1;
    c.cols = p.sum_cols;
    c.brow0 = (g - p.num_groups) * p.sum_cols;
    c.unit0 = g - p.num_groups;   // index of the sum tile
    c.nunits = 0;
  } else {
    c.unit0 = g * p.group_units;
    c.nunits = min(p.group_units, p.emit_units - c.unit0);
    c.cols = p.tile_cols;
    c.brow0 = c.unit0 * p.v;
    c.ntiles = (c.nunits * p.v + p.tile_cols - 1) / p.tile_cols;
  }
  return c;
}

// Padding columns of a unit (vocabulary not a multiple of 16) count as logit = -inf: never the maximum, no mass.
__device__ __forceinline__ void mask_padding(float (&x)[16], int col_in_unit, int vv) {
  if (col_in_unit + 16 > vv) {
#pragma unroll
    for (int q = 0; q < 16; ++q)
      if (col_in_unit + q >= vv) x[q] = -CUDART_INF_F;
  }
}

// log-softmax over groups of R adjacent columns inside one 16-column batch (R in {1,2,4,8,16}).
template <int R>
__device__ __forceinline__ void sum_groups_in_batch(const float (&x)[16], float* dst, int col0, int sum_rows) {
#pragma unroll
  for (int g = 0; g < 16 / R; ++g) {
    float m = x[g * R];
#pragma unroll
    for (int q = 1; q < R; ++q) m = fmaxf(m, x[g * R + q]);
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < R; ++q) s += fast_ex2((x[g * R + q] - m) * kLog2e);
    const float lse = m + fast_lg2(s) * kLn2;
    if (col0 + g * R < sum_rows) {
#pragma unroll
      for (int q = 0; q < R; ++q) dst[col0 + g * R + q] = x[g * R + q] - lse;
    }
  }
}

// CTAS = 1: every CTA works alone (cta_group::1). CTAS = 2: the kernel is launched in clusters of two CTAs that share
// every MMA (cta_group::2, M = 256): the pair covers 256 positions, each CTA stages its own 128 rows of h and HALF of the
// weight tile (the leader, cluster rank 0, the first half of the tile's columns), so a CTA moves a third less data from
// L2 to shared memory per MMA; the leader's warp 1 issues the MMAs for both, each CTA's epilogue warps read their own
// 128 accumulator rows. Barriers: full[s] lives in the leader and counts the bytes of both CTAs' copies; empty[s] and
// tfull[slot] exist in both CTAs and are signalled together by the leader's commits; tempty[slot] lives in the leader
// and collects the arrivals of both CTAs' epilogue warps.
template <int MODE, int CTAS>
__global__ void __launch_bounds__(kGemmThreads, 1) mtpc_gemm_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (tiles_addr - raw_addr);
  GemmControl* ctl = reinterpret_cast<GemmControl*>(tiles + static_cast<size_t>(p.stages) * p.stage_bytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  constexpr bool kGrouped = MODE == kModeSampleGrouped || MODE == kModeLogitsGrouped;
  static_assert(!kGrouped || CTAS == 1, "grouped tiles are ragged: no pairing");
  const int num_items = kGrouped ? *p.group_num_tiles : (p.num_groups + p.num_sum_tiles) * p.m_units;
  const uint32_t cta_rank = CTAS == 2 ? cluster_cta_rank() : 0u;      // 0 = the pair's leader
  auto coord = [&](int item) {
    if (kGrouped) return group_coord(p, item, MODE == kModeLogitsGrouped);
    TileCoord c = tile_coord(p, item);
    c.arow = (c.mt * CTAS + static_cast<int>(cta_rank)) * kBlockM;
    c.count = min(kBlockM, p.T - c.arow);                             // <= 0: a pair's second CTA past the last position
    c.wrap = c.ntiles;
    return c;
  };
  const int first_item = CTAS == 2 ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int item_step = CTAS == 2 ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int s = 0; s < p.num_slots; ++s) {
      mbar_init(smem_u32(&ctl->tfull[s]), 1);
      mbar_init(smem_u32(&ctl->tempty[s]), 4 * CTAS);
    }
    mbar_init(smem_u32(&ctl->drain), 1);
    ctl->abort = 0;
    ctl->wait_limit_ns = p.wait_limit_ns;
    fence_mbar_init();
    tma_prefetch_desc(&p.tm_a);
    tma_prefetch_desc(&p.tm_emit);
    tma_prefetch_desc(&p.tm_sum);
  }
  if (warp == 1) {
    if (CTAS == 2) {
      tmem_alloc_pair(smem_u32(&ctl->tmem_base), kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();   // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued_mask = 0, phase_mask = 0;
      bool ok = true;
      for (int item = first_item; item < num_items && ok; item += item_step) {
        const TileCoord tc = coord(item);
        const CUtensorMap* tmb = tc.is_sum ? &p.tm_sum : &p.tm_emit;
        const int brows = tc.cols / CTAS;                                 // weight rows this CTA stages per tile
        const uint32_t bytes = CTAS * (kABytes + brows * (kBlockK * 2));   // of both CTAs' copies when paired
        const int arow = tc.arow;
        for (int t = 0; t < tc.ntiles && ok; ++t) {
          for (int kb = 0; kb < p.kblocks; ++kb) {
            if (!bounded_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
            const uint32_t a_dst = tiles_addr + stage * p.stage_bytes;
            const int brow = tc.brow0 + (t % tc.wrap) * tc.cols + static_cast<int>(cta_rank) * brows;
            if (CTAS == 2) {
              const uint32_t full = cluster_map_shared(smem_u32(&ctl->full[stage]), 0);   // the leader's barrier
              if (cta_rank == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[stage]), bytes);
              tma_load_2d_pair(a_dst, &p.tm_a, full, kb * kBlockK, arow);
              tma_load_2d_pair(a_dst + kABytes, tmb, full, kb * kBlockK, brow);
            } else {
              const uint32_t full = smem_u32(&ctl->full[stage]);
              mbar_arrive_expect_tx(full, bytes);
              tma_load_2d(a_dst, &p.tm_a, full, kb * kBlockK, arow);
              tma_load_2d(a_dst + kABytes, tmb, full, kb * kBlockK, brow);
            }
            issued_mask |= 1u << stage;
            phase_mask = (phase_mask & ~(1u << stage)) | (phase << stage);
            if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; }
          }
        }
      }
      // The CTA must not go away with copies in flight. After a full run they have all landed already (the MMA warp
      // consumed them); after an abort, by this warp or by another one, give them a bounded chance to land.
      if (CTAS == 1 || cta_rank == 0) {
        for (int s = 0; s < p.stages; ++s)
          if (issued_mask & (1u << s)) {
            const uint32_t bar = smem_u32(&ctl->full[s]);
            const uint32_t par = (phase_mask >> s) & 1u;
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(bar, par) && global_timer_ns() - t0 < kWaitLimitNs) {}
          }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && cta_rank == 0) {
      uint32_t stage = 0, phase = 0, use = 0;
      bool ok = true;
      for (int item = first_item; item < num_items && ok; item += item_step) {
        const TileCoord tc = coord(item);
        const uint32_t idesc = umma_idesc_bf16(kBlockM * CTAS, tc.cols);
        for (int t = 0; t < tc.ntiles && ok; ++t, ++use) {
          const uint32_t slot = use % p.num_slots;
          if (!bounded_wait(smem_u32(&ctl->tempty[slot]), ((use / p.num_slots) & 1u) ^ 1u, ctl, p.status)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + slot * p.slot_stride;
          for (int kb = 0; kb < p.kblocks; ++kb) {
            if (!bounded_wait(smem_u32(&ctl->full[stage]), phase, ctl, p.status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = tiles_addr + stage * p.stage_bytes;
            const uint64_t a_desc = umma_smem_desc_sw128(a_addr);
            const uint64_t b_desc = umma_smem_desc_sw128(a_addr + kABytes);
#pragma unroll
            for (int kk = 0; kk < kBlockK / 16; ++kk) {   // +32 bytes per K=16 step inside the swizzled row
              if (CTAS == 2) umma_bf16_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
              else umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
            }
            if (CTAS == 2) umma_commit_pair(smem_u32(&ctl->empty[stage]));   // frees the stage in both CTAs
            else umma_commit(smem_u32(&ctl->empty[stage]));
            if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (CTAS == 2) umma_commit_pair(smem_u32(&ctl->tfull[slot]));      // the accumulators of both CTAs are ready
          else umma_commit(smem_u32(&ctl->tfull[slot]));
        }
      }
      if (!ok) {   // wait (bounded) for the MMAs already issued before TMEM is freed
        if (CTAS == 2) umma_commit_pair(smem_u32(&ctl->drain));
        else umma_commit(smem_u32(&ctl->drain));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    uint32_t use = 0;
    bool ok = true;
    // a drained accumulator slot is handed back to the MMA issuer: the leader's, also from the peer's epilogue warps
    auto release_slot = [&](uint32_t slot) {
      if (CTAS == 2) mbar_arrive_cluster(cluster_map_shared(smem_u32(&ctl->tempty[slot]), 0));
      else mbar_arrive(smem_u32(&ctl->tempty[slot]));
    };
    for (int item = first_item; item < num_items && ok; item += item_step) {
      const TileCoord tc = coord(item);
      const int row = tc.arow + quarter * 32 + lane;
      const bool valid = quarter * 32 + lane < tc.count;
      const int nbatch = tc.cols / 16;

      if (tc.is_sum) {
        // ---- sum-unit logits -> log omega (Sec. 3.3): log-softmax over groups of r adjacent columns
        const uint32_t slot = use % p.num_slots;
        if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (use / p.num_slots) & 1u, ctl, p.status, lane)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t tcol = lane_base + slot * p.slot_stride;
        const int col_base = tc.unit0 * p.sum_cols;
        float* dst = p.logw + static_cast<size_t>(valid ? row : 0) * p.sum_rows;
        if (p.r <= 16) {
          for (int b = 0; b < nbatch; ++b) {
            float x[16];
            tmem_ld16(tcol + b * 16, x);
            if (valid) {
              const int col0 = col_base + b * 16;
              if (p.sum_bias != nullptr) {
#pragma unroll
                for (int q = 0; q < 16; ++q)
                  if (col0 + q < p.sum_rows) x[q] += p.sum_bias[col0 + q];
              }
              switch (p.r) {
                case 1: sum_groups_in_batch<1>(x, dst, col0, p.sum_rows); break;
                case 2: sum_groups_in_batch<2>(x, dst, col0, p.sum_rows); break;
                case 4: sum_groups_in_batch<4>(x, dst, col0, p.sum_rows); break;
                case 8: sum_groups_in_batch<8>(x, dst, col0, p.sum_rows); break;
                default: sum_groups_in_batch<16>(x, dst, col0, p.sum_rows); break;
              }
            }
          }
        } else {
          const int bpg = p.r / 16;   // batches per group
          for (int g = 0; g < tc.cols / p.r; ++g) {
            float m = -CUDART_INF_F, s = 0.f;
            const int gcol = col_base + g * p.r;
            const bool biased = p.sum_bias != nullptr && gcol < p.sum_rows;
            for (int b = 0; b < bpg; ++b) {
              float x[16];
              tmem_ld16(tcol + (g * bpg + b) * 16, x);
              if (biased) {
#pragma unroll
                for (int q = 0; q < 16; ++q) x[q] += p.sum_bias[gcol + b * 16 + q];
              }
              float bm = x[0];
#pragma unroll
              for (int q = 1; q < 16; ++q) bm = fmaxf(bm, x[q]);
              const float mn = fmaxf(m, bm);
              s *= fast_ex2((m - mn) * kLog2e);
#pragma unroll
              for (int q = 0; q < 16; ++q) s += fast_ex2((x[q] - mn) * kLog2e);
              m = mn;
            }
            const float lse = m + fast_lg2(s) * kLn2;
            for (int b = 0; b < bpg; ++b) {
              float x[16];
              tmem_ld16(tcol + (g * bpg + b) * 16, x);
              if (biased) {
#pragma unroll
                for (int q = 0; q < 16; ++q) x[q] += p.sum_bias[gcol + b * 16 + q];
              }
              if (valid && gcol < p.sum_rows) {
#pragma unroll
                for (int q = 0; q < 16; ++q) x[q] -= lse;
                // r is a multiple of 16 here, so the rows of log omega (S r floats) and this offset are 64-byte aligned
                st_global_v8(dst + gcol + b * 16, x);
                st_global_v8(dst + gcol + b * 16 + 8, x + 8);
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) release_slot(slot);
        use += 1;
        continue;
      }

      if (MODE == kModeLogitsGrouped) {
        // ---- the slot's logits and unit log-sum-exps per staged row (logit_out [rows, r v], lse_out [rows, r]): what the
        // acceptance stage needs to form the circuit's conditional of the first rejected byte
        int col = 0, k = 0;                                       // column inside the slot's r v columns; unit index
        float m = -CUDART_INF_F, s = 0.f;
        for (int t = 0; t < tc.ntiles && ok; ++t, ++use) {
          const uint32_t slot = use % p.num_slots;
          if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (use / p.num_slots) & 1u, ctl, p.status, lane)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t tcol = lane_base + slot * p.slot_stride;
          for (int b = 0; b < nbatch && k < p.r; ++b) {
            float x[16];
            tmem_ld16(tcol + b * 16, x);
            mask_padding(x, col - k * p.v, p.vv);
            if (valid) {
              float* l = p.logit_out + static_cast<size_t>(row) * p.logit_pitch + col;
              st_global_v8(l, x);
              st_global_v8(l + 8, x + 8);
            }
            float bm = x[0];
#pragma unroll
            for (int q = 1; q < 16; ++q) bm = fmaxf(bm, x[q]);
            const float mn = fmaxf(m, bm);
            const float mn2 = mn * kLog2e;
            s *= fast_ex2((m - mn) * kLog2e);
#pragma unroll
            for (int q = 0; q < 16; ++q) s += fast_ex2(fmaf(x[q], kLog2e, -mn2));
            m = mn;
            col += 16;
            if (col == (k + 1) * p.v) {
              if (valid) p.lse_out[static_cast<size_t>(row) * p.r + k] = m + fast_lg2(s) * kLn2;
              ++k;
              m = -CUDART_INF_F; s = 0.f;
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) release_slot(slot);
        }
        if (!ok) break;
      } else if (MODE == kModeLogprob) {
        // ---- log phi at the target byte: online log-sum-exp over the v columns of each unit + gather. The
        // running (m, s) and the gathered logit live across tile boundaries; a unit is closed when its v-th
        // column has been consumed.
        const size_t wrow0 = static_cast<size_t>(valid ? row : 0) * p.wpp;
        const int units_end = tc.unit0 + tc.nunits;
        int unit = tc.unit0, col_in_unit = 0;
        int slot_i = unit / p.r, k = unit - slot_i * p.r;
        float m = -CUDART_INF_F, s = 0.f, tval = 0.f;
        int tgt = (p.wpp == 1 && valid) ? p.targets[wrow0 * p.n + slot_i] : -1;
        for (int t = 0; t < tc.ntiles && ok; ++t, ++use) {
          const uint32_t slot = use % p.num_slots;
          if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (use / p.num_slots) & 1u, ctl, p.status, lane)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t tcol = lane_base + slot * p.slot_stride;
          // one batch of 16 accumulator columns of this row; false once the item's last unit has been closed
          auto consume = [&](const uint32_t (&raw)[16], int b) -> bool {
            float x[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = __uint_as_float(raw[q]);
            mask_padding(x, col_in_unit, p.vv);
            if (p.logit_out != nullptr && valid) {                       // row of W_emit = column of the logit matrix
              float* l = p.logit_out + static_cast<size_t>(row) * p.logit_pitch + tc.brow0 + t * tc.cols + b * 16;
              st_global_v8(l, x);                                        // 64-byte aligned: v and the tile widths are multiples of 16
              st_global_v8(l + 8, x + 8);
            }
            float bm = x[0];
#pragma unroll
            for (int q = 1; q < 16; ++q) bm = fmaxf(bm, x[q]);
            const float mn = fmaxf(m, bm);
            const float mn2 = mn * kLog2e;
            s *= fast_ex2((m - mn) * kLog2e);
#pragma unroll
            for (int q = 0; q < 16; ++q) s += fast_ex2(fmaf(x[q], kLog2e, -mn2));
            m = mn;
            if (p.wpp == 1) {
              const int rel = tgt - col_in_unit;
              if (static_cast<unsigned>(rel) < 16u) {
#pragma unroll
                for (int q = 0; q < 16; ++q)
                  if (rel == q) tval = x[q];
              }
            } else if (valid) {
              for (int j = 0; j < p.wpp; ++j) {
                const int rel = p.targets[(wrow0 + j) * p.n + slot_i] - col_in_unit;
                if (static_cast<unsigned>(rel) < 16u) {
                  float val = 0.f;
#pragma unroll
                  for (int q = 0; q < 16; ++q)
                    if (rel == q) val = x[q];
                  p.G[((wrow0 + j) * p.n + slot_i) * p.r + k] = val;   // raw logit; normalised below
                }
              }
            }
            col_in_unit += 16;
            if (col_in_unit == p.v) {
              // ---- unit (slot_i, k) complete
              const float lse = m + fast_lg2(s) * kLn2;
              if (valid && p.lse_out != nullptr)
                p.lse_out[(static_cast<size_t>(row) * p.n + slot_i) * p.r + k] = lse;
              if (valid) {
                for (int j = 0; j < p.wpp; ++j) {
                  const int tj = (p.wpp == 1) ? tgt : p.targets[(wrow0 + j) * p.n + slot_i];
                  float* g = p.G + ((wrow0 + j) * p.n + slot_i) * p.r + k;
                  if (tj < 0) {
                    *g = p.missing_is_nan ? CUDART_NAN_F : 0.f;   // marginalised byte: the input unit sums to 1
                  } else if (tj >= p.vv) {
                    *g = CUDART_NAN_F;
                    atomicOr(p.status, kStatusBadTarget);
                  } else {
                    *g = ((p.wpp == 1) ? tval : *g) - lse;
                  }
                }
              }
              ++unit;
              col_in_unit = 0;
              m = -CUDART_INF_F; s = 0.f; tval = 0.f;
              if (unit < units_end) {
                slot_i = unit / p.r;
                k = unit - slot_i * p.r;
                tgt = (p.wpp == 1 && valid) ? p.targets[wrow0 * p.n + slot_i] : -1;
              }
            }
            return unit < units_end;
          };
          // The load of the next batch is in flight while this one goes through the exponentials (two register buffers).
          uint32_t ra[16], rb[16];
          tmem_ld16_issue(tcol, ra);
          tmem_ld_wait16(ra);
          for (int b = 0;;) {
            const bool more_b = b + 1 < nbatch;
            if (more_b) tmem_ld16_issue(tcol + (b + 1) * 16, rb);
            const bool go_a = consume(ra, b);
            if (more_b) tmem_ld_wait16(rb);
            if (!go_a || !more_b) break;
            ++b;
            const bool more_a = b + 1 < nbatch;
            if (more_a) tmem_ld16_issue(tcol + (b + 1) * 16, ra);
            const bool go_b = consume(rb, b);
            if (more_a) tmem_ld_wait16(ra);
            if (!go_b || !more_a) break;
            ++b;
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) release_slot(slot);
        }
        if (!ok) break;
      } else {
        // ---- byte draws (Algorithm 1, input units): inverse CDF of softmax(logits) for every window of this
        // row whose selected unit for this slot is k. One unit per group: all its tiles stay in TMEM until the end.
        const int slot_i = tc.unit0 / p.r;
        const int k = tc.unit0 - slot_i * p.r;
        unsigned long long pending = 0ull;
        size_t wrow0 = 0;
        int nwin = p.wpp;
        if (MODE == kModeSampleGrouped) {
          // the row holds one (window, slot) pair, and the slot is this tile's
          if (valid) { wrow0 = static_cast<size_t>(p.group_perm[row] / p.n); pending = 1ull; }
          nwin = 1;
        } else {
          wrow0 = static_cast<size_t>(valid ? row : 0) * p.wpp;
          if (valid)
            for (int j = 0; j < nwin; ++j)
              if (p.unit_sel[(wrow0 + j) * p.n + slot_i] == k) pending |= 1ull << j;
        }
        if (MODE == kModeSampleGrouped && p.group_two_pass) {
          // ---- a unit wider than tensor memory: its tiles stream through the accumulator ring twice. Sweep 1: running
          // maximum and sum of exponentials (the sum in fp64, 16 terms at a time, so that tens of thousands of terms
          // keep the precision the draw needs). Sweep 2: the scan u * total < running sum over the recomputed tiles.
          const float uval = valid ? p.uniforms[wrow0 * (2 * p.n) + p.n + slot_i] : 0.f;
          float m = -CUDART_INF_F;
          double total = 0.0, cum = 0.0, thr = 0.0;
          int found = p.vv - 1;   // rounding may leave no index: the last one
          bool hit = false;
          for (int t = 0; t < tc.ntiles && ok; ++t, ++use) {
            const uint32_t slot = use % p.num_slots;
            if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (use / p.num_slots) & 1u, ctl, p.status, lane)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t tcol = lane_base + slot * p.slot_stride;
            const bool second = t >= tc.wrap;
            if (t == tc.wrap) thr = static_cast<double>(uval) * total;
            const int col_tile = (t % tc.wrap) * tc.cols;
            for (int b = 0; b < nbatch && col_tile + b * 16 < p.vv; ++b) {
              float x[16];
              tmem_ld16(tcol + b * 16, x);
              const int col0 = col_tile + b * 16;
              mask_padding(x, col0, p.vv);
              if (!second) {
                float bm = x[0];
#pragma unroll
                for (int q = 1; q < 16; ++q) bm = fmaxf(bm, x[q]);
                if (bm > m) {                                   // rescale what was summed so far to the new maximum
                  total *= static_cast<double>(fast_ex2((m - bm) * kLog2e));
                  m = bm;
                }
                const float m2 = m * kLog2e;
                float part = 0.f;
#pragma unroll
                for (int q = 0; q < 16; ++q) part += fast_ex2(fmaf(x[q], kLog2e, -m2));
                total += static_cast<double>(part);
              } else if (!hit) {
                const float m2 = m * kLog2e;
                const float rest = static_cast<float>(thr - cum);   // what the threshold still needs inside this batch
                float part = 0.f;
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                  part += fast_ex2(fmaf(x[q], kLog2e, -m2));
                  if (!hit && rest < part) { hit = true; found = col0 + q; }
                }
                cum += static_cast<double>(part);
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) release_slot(slot);
          }
          if (!ok) break;
          if (valid) {
            if (!(uval >= 0.f && uval < 1.f)) {
              found = -1;
              atomicOr(p.status, kStatusBadUniform);
            }
            p.out_bytes[wrow0 * p.n + slot_i] = found;
          }
          continue;
        }
        for (int c = 0; c < tc.ntiles && ok; ++c) {
          const uint32_t u = use + c;
          if (!bounded_wait_warp(smem_u32(&ctl->tfull[u % p.num_slots]), (u / p.num_slots) & 1u, ctl, p.status,
                                 lane))
            ok = false;
        }
        if (!ok) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, pending != 0ull)) {
          float m = -CUDART_INF_F;
          for (int c = 0; c < tc.ntiles; ++c) {
            const uint32_t tcol = lane_base + ((use + c) % p.num_slots) * p.slot_stride;
            for (int b = 0; b < nbatch; ++b) {
              float x[16];
              tmem_ld16(tcol + b * 16, x);
              mask_padding(x, c * tc.cols + b * 16, p.vv);
#pragma unroll
              for (int q = 0; q < 16; ++q) m = fmaxf(m, x[q]);
            }
          }
          const float m2 = m * kLog2e;
          float total = 0.f;   // same terms in the same order as the running sum of the scan below
          for (int c = 0; c < tc.ntiles; ++c) {
            const uint32_t tcol = lane_base + ((use + c) % p.num_slots) * p.slot_stride;
            for (int b = 0; b < nbatch; ++b) {
              float x[16];
              tmem_ld16(tcol + b * 16, x);
              mask_padding(x, c * tc.cols + b * 16, p.vv);
#pragma unroll
              for (int q = 0; q < 16; ++q) total += fast_ex2(fmaf(x[q], kLog2e, -m2));
            }
          }
          while (__any_sync(0xffffffffu, pending != 0ull)) {
            const int j = pending ? __ffsll(static_cast<long long>(pending)) - 1 : -1;
            float uval = 0.f;
            if (j >= 0) uval = p.uniforms[(wrow0 + j) * (2 * p.n) + p.n + slot_i];
            const float thr = uval * total;
            float cum = 0.f;
            int found = p.vv - 1;   // rounding may leave no index: the last one
            bool hit = false;
            for (int c = 0; c < tc.ntiles; ++c) {
              const uint32_t tcol = lane_base + ((use + c) % p.num_slots) * p.slot_stride;
              for (int b = 0; b < nbatch; ++b) {
                float x[16];
                tmem_ld16(tcol + b * 16, x);
                const int col0 = c * tc.cols + b * 16;
                mask_padding(x, col0, p.vv);
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                  cum += fast_ex2(fmaf(x[q], kLog2e, -m2));
                  if (!hit && thr < cum) { hit = true; found = col0 + q; }
                }
              }
            }
            if (j >= 0) {
              if (!(uval >= 0.f && uval < 1.f)) {
                found = -1;
                atomicOr(p.status, kStatusBadUniform);
              }
              p.out_bytes[(wrow0 + j) * p.n + slot_i] = found;
              pending &= pending - 1ull;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0)
          for (int c = 0; c < tc.ntiles; ++c) release_slot((use + c) % p.num_slots);
        use += tc.ntiles;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) {
    // A CTA of a pair may leave only when its partner no longer needs it (MMAs read both CTAs' shared memory and write
    // both CTAs' tensor memory; copies and arrivals cross over). After a run in which some wait gave up, first let
    // whatever is still in flight land: the peer's copies are counted on the leader's barriers and cannot be awaited here.
    if (ctl->abort && threadIdx.x == 0) {
      const uint64_t t0 = global_timer_ns();
      while (global_timer_ns() - t0 < kAbortSettleNs) {}
    }
    __syncthreads();      // every warp converged again before the cluster-wide barrier
    cluster_sync_all();
  }
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace mtpc
