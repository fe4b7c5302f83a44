// Draft path for few positions (decode-time speculative drafting, Algorithm 1): the cost is one pass over the
// emission weights, so the work is organised around streaming them from HBM exactly once.
//
//   mtpc_decode_gemm_kernel   logits[p, row] = W[row] . h_p for every weight row (emission and sum-unit rows) and
//                             every position p < P <= 128, with the roles of the operands swapped with respect
//                             to the training-shaped kernel: 128 weight rows sit on the M axis (TMEM lanes), the
//                             positions on the N axis (TMEM columns). Emission logits go to a small scratch
//                             [P, n*r*v] fp32 (P is tiny here, so this is a few MB against hundreds of MB of
//                             weights); sum-unit logits are log-softmaxed over their groups of r rows (= lanes,
//                             by warp shuffles) and written as log omega [P, S*r]. A mixture of more than 32
//                             components (CP, r = 64 or 128) spans several warps: its logits are written as they
//                             are, and the kernels that follow normalise them where they need to.
//                             Weight rows are cut into tiles of `tile_rows` <= 128 rows, chosen by the host so that
//                             the tiles divide evenly over the persistent CTAs; each CTA takes a contiguous run
//                             of tiles and walks K once per pass of up to three tiles, which share one copy of
//                             the hidden-state block, so the bytes in flight per SM stay high and the hidden
//                             states cross L2 once per pass instead of once per tile.
//   draft_slot_kernel         one CTA per (position, window slot i): log-sum-exp of the r input units of the
//                             slot, then per window (one warp each): latent draws down to the unit that owns
//                             slot i, the byte by inverse CDF of that unit's categorical, and the evidence
//                             G[w, i, k] = log phi_k(byte) for all k, which the circuit kernels then reduce.
#pragma once
#include "mtpc_circuit.cuh"
#include "mtpc_gemm.cuh"

namespace mtpc {

constexpr int kDecodeMaxP = 128;                   // positions per call on this path
#ifndef MTPC_DECODE_MAX_TILES
#define MTPC_DECODE_MAX_TILES 3
#endif
constexpr int kDecodeMaxTiles = MTPC_DECODE_MAX_TILES;   // weight tiles that share one copy of the hidden states
constexpr int kSlotThreads = 512;

struct DecodeParams {
  CUtensorMap tm_h;      // hidden [P, d]       box 64 x Ppad
  CUtensorMap tm_emit;   // W_emit [n*r*v, d]   box 64 x tile_rows
  CUtensorMap tm_sum;    // W_sum  [S*r, d]     box 64 x sum_tile_rows
  CUtensorMap tm_emit2;  // a second matrix of emission-like rows [emit2_rows, d], box 64 x tile_rows (a factored
                         // low-rank head: tm_emit = W_base, tm_emit2 = B); unused when emit2_tiles == 0
  int P, Ppad, kblocks;
  int emit_rows, sum_rows, r;
  int emit2_rows, emit2_tiles;
  int tile_rows;                 // rows of an emission tile (a multiple of 8, <= 128)
  int sum_tile_rows;             // rows of a sum tile (a multiple of 32, <= tile_rows rounded up to 32)
  int tile_bytes;                // shared-memory pitch of a weight tile
  int emit_tiles, sum_tiles;
  int pass_tiles;                // tiles per pass (<= kDecodeMaxTiles)
  int tile_stride;               // TMEM columns per tile
  int stages, stage_bytes;
  float* logits;         // [P, emit_rows]
  float* logits2;        // [P, emit2_rows]
  float* logw;           // [P, sum_rows]
  const float* sum_bias; // [sum_rows] or NULL: added to the sum-unit logits before their softmax
  unsigned* status;
  uint64_t wait_limit_ns;   // limit of every pipeline wait
};

// Tile `t` of the launch: emission tiles first, then those of the second matrix, then sum tiles.
struct DecodeTile {
  int is_sum, second, index, rows;   // which matrix, tile index within it, rows per tile
};
__device__ __forceinline__ DecodeTile decode_tile(const DecodeParams& p, int t) {
  DecodeTile d;
  d.is_sum = t >= p.emit_tiles + p.emit2_tiles;
  d.second = !d.is_sum && t >= p.emit_tiles;
  d.index = d.is_sum ? t - p.emit_tiles - p.emit2_tiles : (d.second ? t - p.emit_tiles : t);
  d.rows = d.is_sum ? p.sum_tile_rows : p.tile_rows;
  return d;
}

// A CTA walks its run of tiles in passes of up to pass_tiles tiles (of either matrix). Shared-memory stage:
// pass_tiles weight tiles at a pitch of tile_bytes (the MMA reads 128 rows from each tile's base: what lies beyond
// the tile's own rows is other data, and the TMEM lanes it produces are never read), then the hidden tile
// (Ppad rows x 128 bytes) followed by slack so that the last tile's 128-row read stays inside the stage.
// Tensor memory: two slots of pass_tiles * tile_stride columns.
__global__ void __launch_bounds__(kGemmThreads, 1) mtpc_decode_gemm_kernel(const __grid_constant__ DecodeParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (tiles_addr - raw_addr);
  GemmControl* ctl = reinterpret_cast<GemmControl*>(tiles + static_cast<size_t>(p.stages) * p.stage_bytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_tiles = p.emit_tiles + p.emit2_tiles + p.sum_tiles;
  const int tile_begin = static_cast<int>(static_cast<long long>(blockIdx.x) * total_tiles / gridDim.x);
  const int tile_end = static_cast<int>(static_cast<long long>(blockIdx.x + 1) * total_tiles / gridDim.x);
  const uint32_t hidden_off = p.pass_tiles * p.tile_bytes;
  const uint32_t slot_cols = p.pass_tiles * p.tile_stride;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&ctl->tfull[s]), 1);
      mbar_init(smem_u32(&ctl->tempty[s]), 4);
    }
    mbar_init(smem_u32(&ctl->drain), 1);
    ctl->abort = 0;
    ctl->wait_limit_ns = p.wait_limit_ns;
    fence_mbar_init();
    tma_prefetch_desc(&p.tm_h);
    tma_prefetch_desc(&p.tm_emit);
    tma_prefetch_desc(&p.tm_sum);
    if (p.emit2_tiles > 0) tma_prefetch_desc(&p.tm_emit2);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  grid_launch_dependents();   // the per-slot kernel may be scheduled as SMs free up; it waits for this grid's results

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued_mask = 0, phase_mask = 0;
      bool ok = true;
      for (int cur = tile_begin; cur < tile_end && ok;) {
        const int ntiles = min(p.pass_tiles, tile_end - cur);
        uint32_t bytes = p.Ppad * (kBlockK * 2);                   // out-of-range rows are zero-filled and counted
        for (int q = 0; q < ntiles; ++q) bytes += decode_tile(p, cur + q).rows * (kBlockK * 2);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctl->full[stage]);
          const uint32_t dst = tiles_addr + stage * p.stage_bytes;
          mbar_arrive_expect_tx(full, bytes);
          for (int q = 0; q < ntiles; ++q) {
            const DecodeTile t = decode_tile(p, cur + q);
            tma_load_2d(dst + q * p.tile_bytes, t.is_sum ? &p.tm_sum : (t.second ? &p.tm_emit2 : &p.tm_emit), full,
                        kb * kBlockK, t.index * t.rows);
          }
          tma_load_2d(dst + hidden_off, &p.tm_h, full, kb * kBlockK, 0);
          issued_mask |= 1u << stage;
          phase_mask = (phase_mask & ~(1u << stage)) | (phase << stage);
          if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; }
        }
        cur += ntiles;
      }
      // no copy may still be in flight when the CTA goes away (they have all landed unless some warp gave up)
      for (int s = 0; s < p.stages; ++s)
        if (issued_mask & (1u << s)) {
          const uint32_t bar = smem_u32(&ctl->full[s]);
          const uint32_t par = (phase_mask >> s) & 1u;
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(bar, par) && global_timer_ns() - t0 < kWaitLimitNs) {}
        }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: D[row, p] = W[row, :] . h[p, :]
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, use = 0;
      bool ok = true;
      const uint32_t idesc = umma_idesc_bf16(kBlockM, p.Ppad);
      for (int cur = tile_begin; cur < tile_end && ok; ++use) {
        const int ntiles = min(p.pass_tiles, tile_end - cur);
        cur += ntiles;
        const uint32_t slot = use & 1u;
        if (!bounded_wait(smem_u32(&ctl->tempty[slot]), ((use >> 1) & 1u) ^ 1u, ctl, p.status)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + slot * slot_cols;
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->full[stage]), phase, ctl, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t w_addr = tiles_addr + stage * p.stage_bytes;
          const uint64_t b_desc = umma_smem_desc_sw128(w_addr + hidden_off);
          for (int q = 0; q < ntiles; ++q) {
            const uint64_t a_desc = umma_smem_desc_sw128(w_addr + q * p.tile_bytes);
#pragma unroll
            for (int kk = 0; kk < kBlockK / 16; ++kk)
              umma_bf16(d_tmem + q * p.tile_stride, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&ctl->empty[stage]));
          if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&ctl->tfull[slot]));
      }
      if (!ok) {
        umma_commit(smem_u32(&ctl->drain));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue: warp q owns lanes 32q .. 32q+31
    const int quarter = warp & 3;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    uint32_t use = 0;
    bool ok = true;
    for (int cur = tile_begin; cur < tile_end && ok; ++use) {
      const int ntiles = min(p.pass_tiles, tile_end - cur);
      const uint32_t slot = use & 1u;
      if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (use >> 1) & 1u, ctl, p.status, lane)) {
        ok = false;
        break;
      }
      tc_fence_after();
      for (int q = 0; q < ntiles; ++q) {
        const DecodeTile t = decode_tile(p, cur + q);
        if (quarter * 32 >= t.rows) continue;                      // warp-uniform: none of this warp's lanes is a row
        const int nrows = t.is_sum ? p.sum_rows : (t.second ? p.emit2_rows : p.emit_rows);
        float* dst = t.is_sum ? p.logw : (t.second ? p.logits2 : p.logits);
        const uint32_t tcol = lane_base + slot * slot_cols + q * p.tile_stride;
        const int local = quarter * 32 + lane;
        const int row = t.index * t.rows + local;
        const bool mine = local < t.rows && row < nrows;
        const float bias = (t.is_sum && p.sum_bias != nullptr && mine) ? p.sum_bias[row] : 0.f;
        for (int b = 0; b < (p.P + 15) / 16; ++b) {
          float x[16];
          tmem_ld16(tcol + b * 16, x);
          if (t.is_sum && p.r <= 32) {
#pragma unroll
            for (int c = 0; c < 16; ++c) x[c] += bias;
            // log-softmax over the r rows of a sum unit = r adjacent lanes (r a power of two <= 32); the 16
            // positions of the batch are reduced side by side so that the shuffles overlap
            float m[16], e[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) m[c] = x[c];
            for (int off = 1; off < p.r; off <<= 1) {
#pragma unroll
              for (int c = 0; c < 16; ++c) m[c] = fmaxf(m[c], __shfl_xor_sync(0xffffffffu, m[c], off));
            }
#pragma unroll
            for (int c = 0; c < 16; ++c) e[c] = fast_ex2((x[c] - m[c]) * kLog2e);
            for (int off = 1; off < p.r; off <<= 1) {
#pragma unroll
              for (int c = 0; c < 16; ++c) e[c] += __shfl_xor_sync(0xffffffffu, e[c], off);
            }
#pragma unroll
            for (int c = 0; c < 16; ++c) x[c] = x[c] - m[c] - fast_lg2(e[c]) * kLn2;
          }
          if (mine) {
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              const int pos = b * 16 + c;
              if (pos < p.P) dst[static_cast<size_t>(pos) * nrows + row] = x[c];   // 32 lanes -> 128 contiguous bytes
            }
          }
        }
      }
      cur += ntiles;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tempty[slot]));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------- per-(position, slot) sampling
// Inclusive warp scan (sum).
__device__ __forceinline__ float warp_scan_incl(float x, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const float y = __shfl_up_sync(kFull, x, off);
    if (lane >= off) x += y;
  }
  return x;
}
// Categorical draw over r <= 32 log-probabilities held one per lane (lanes >= r hold anything): the smallest
// j with u < p_0 + ... + p_j, else r - 1. All lanes return the same index.
__device__ __forceinline__ int warp_inv_cdf_logp(float logp, int r, float u, int lane) {
  const float pr = lane < r ? expf(logp) : 0.f;
  const float cum = warp_scan_incl(pr, lane);
  const unsigned hit = __ballot_sync(kFull, lane < r && u < cum);
  return hit ? __ffs(hit) - 1 : r - 1;
}

// The same draw over the softmax of r <= 128 unnormalised logits x[0..r): lane l owns the consecutive indices
// [l * per, (l + 1) * per), per = ceil(r / 32) <= 4; u * total < running sum, index order, no division.
__device__ __forceinline__ int warp_inv_cdf_logits_wide(const float* __restrict__ x, int r, float u, int lane) {
  const int per = (r + 31) / 32;
  const int k0 = lane * per;
  float xv[4];
  float m = -CUDART_INF_F;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    xv[q] = (q < per && k0 + q < r) ? x[k0 + q] : -CUDART_INF_F;
    m = fmaxf(m, xv[q]);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, off));
  float part = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    xv[q] = __expf(xv[q] - m);       // padding: exp(-inf) = 0
    part += xv[q];
  }
  const float incl = warp_scan_incl(part, lane);
  const float total = __shfl_sync(kFull, incl, 31);
  const float thr = u * total;
  const unsigned hit = __ballot_sync(kFull, thr < incl);
  if (!hit) return r - 1;
  const int src = __ffs(hit) - 1;
  const float before = __shfl_up_sync(kFull, incl, 1);
  int found = -1;
  if (lane == src) {
    float cum = lane == 0 ? 0.f : before;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (found < 0 && q < per && k0 + q < r) {
        cum += xv[q];
        if (thr < cum) found = k0 + q;
      }
    if (found < 0) found = min(k0 + per, r) - 1;
  }
  return __shfl_sync(kFull, found, src);
}

// Tables the latent draws of slot i walk through (Algorithm 1 at the sum units), in the order they are used.
// CP: none. HMM: the transitions into steps 1..i. BTree: the nodes on the path from the root (exclusive) down to
// the deepest internal node above token i.
__device__ __forceinline__ int slot_chain_length(int family, int n, int i) {
  if (family == 1) return i;
  if (family == 2) return 31 - __clz(n / 2 + (i >> 1));   // depth of the owner node n/2 - 1 + i/2 in heap order
  return 0;
}
// Global address of table `step` (0-based) of the chain. lw: this position's log omega; hmm: this position's
// (or the static) transition tables [n-1, r, r].
__device__ __forceinline__ const float* slot_chain_table(int family, const float* lw, const float* hmm, int n, int r,
                                                         int i, int step) {
  if (family == 1) return hmm + static_cast<size_t>(step) * r * r;
  const int code = n / 2 + (i >> 1);                       // owner + 1
  const int depth = 31 - __clz(code);
  const int node = (code >> (depth - 1 - step)) - 1;       // path node at level step + 1
  return lw + r + static_cast<size_t>(node - 1) * r * r;
}

constexpr int kSlotMaxPerLane = 16;   // symbols a lane holds at a time: 512 per warp pass
// Sum of exp(x[b] - m) over the symbols [c0, c0 + 512) that exist (b < vv); lane l takes l, l + 32, ... of the chunk.
__device__ __forceinline__ float warp_chunk_sum(const float* __restrict__ x, int c0, int vv, float m, int lane) {
  float xv[kSlotMaxPerLane];
#pragma unroll
  for (int q = 0; q < kSlotMaxPerLane; ++q) {
    const int b = c0 + lane + 32 * q;
    xv[q] = b < vv ? x[b] : -CUDART_INF_F;
  }
  float s = 0.f;
#pragma unroll
  for (int q = 0; q < kSlotMaxPerLane; ++q) s += __expf(xv[q] - m);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(kFull, s, off);
  return s;
}
// Inverse CDF inside one chunk of 32 * per symbols starting at c0, on the weights exp(x[b] - m): lane l owns the
// consecutive symbols [c0 + l*per, c0 + (l+1)*per). The threshold is u * (the chunk's total) when `relative`, else
// `thr` itself. Returns the smallest symbol whose running sum exceeds the threshold; the last existing symbol of
// the chunk if rounding leaves none. All lanes return the same value.
template <int NQ>   // per <= NQ <= kSlotMaxPerLane: the steps that are unrolled
__device__ __forceinline__ int warp_inv_cdf_chunk(const float* __restrict__ x, int c0, int per, int vv, float m, float thr,
                                                  bool relative, int lane) {
  const int b0 = c0 + lane * per;
  float ev[NQ];
#pragma unroll
  for (int q = 0; q < NQ; ++q) ev[q] = (q < per && b0 + q < vv) ? x[b0 + q] : -CUDART_INF_F;
  float part = 0.f;
#pragma unroll
  for (int q = 0; q < NQ; ++q) {
    ev[q] = __expf(ev[q] - m);
    part += ev[q];
  }
  const float incl = warp_scan_incl(part, lane);
  if (relative) thr *= __shfl_sync(kFull, incl, 31);
  const unsigned hit = __ballot_sync(kFull, thr < incl);
  int byte = min(c0 + 32 * per, vv) - 1;
  if (hit) {
    const int src = __ffs(hit) - 1;
    int found = -1;
    const float before = __shfl_up_sync(kFull, incl, 1);
    if (lane == src) {
      float cum = lane == 0 ? 0.f : before;
#pragma unroll
      for (int q = 0; q < NQ; ++q)
        if (found < 0 && q < per && b0 + q < vv) {
          cum += ev[q];
          if (thr < cum) found = b0 + q;
        }
      if (found < 0) found = min(b0 + per, vv) - 1;   // the lane's total passed the threshold: its last byte
    }
    byte = __shfl_sync(kFull, found, src);
  }
  return byte;
}

// logA: HMM transition log-probabilities [n-1, r, r]; position p reads them at logA + p * logA_stride (stride 0:
// one static set for all positions; stride sum_rows with logA = log omega + r: contextual tables, App. H).
// grid = (n, P), 16 warps. Shared memory: 2 * r floats (max and log-sum-exp of each unit of the slot), then, when
// tables_in_smem, the chain's tables (slot_chain_length * r * r floats), fetched by cp.async while the log-sum-exps
// are computed, so that the data-dependent row reads of the latent draws do not each cost a trip to L2.
// The log-sum-exps also go to unit_lse_out [P, n, r], so that later calls can turn the retained logits into log phi.
// WIDE: vocabularies of more than 512 symbols (a separate build: the narrow one keeps a unit's logits in 16 registers per lane).
template <bool WIDE, int NQ>   // NQ: batches of 32 symbols of a unit that are unrolled (v <= 32 NQ; WIDE: 16)
__global__ void __launch_bounds__(kSlotThreads, 2) draft_slot_kernel(
    int family, const float* __restrict__ logits, const float* __restrict__ logw, const float* __restrict__ logA,
    const float* __restrict__ uniforms, int* __restrict__ out_bytes, float* __restrict__ G,
    float* __restrict__ unit_lse_out, unsigned* status, unsigned* work_counter, int wpp, int n, int r, int v, int vv,
    int sum_rows, int logA_stride, int tables_in_smem) {
  extern __shared__ __align__(16) float sm[];
  grid_launch_dependents();
  grid_dependency_wait();     // the logits and log omega come from the kernel before this one
  if (work_counter != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0)
    *work_counter = 0;        // the circuit kernel that follows hands out its windows through this counter
  float* unit_max = sm;
  float* unit_lse = sm + r;
  float* tabs = sm + ((2 * r + 3) & ~3);
  const int i = blockIdx.x;
  const int pos = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nwarps = kSlotThreads / 32;
  const int rr = r * r;
  const float* row = logits + (static_cast<size_t>(pos) * n + i) * r * v;   // [r, v] logits of this slot
  const float* lw = logw + static_cast<size_t>(pos) * sum_rows;
  const float* hmm = logA + static_cast<size_t>(pos) * logA_stride;
  const int chain = slot_chain_length(family, n, i);

  if (tables_in_smem) {
    for (int step = 0; step < chain; ++step) {
      const float* src = slot_chain_table(family, lw, hmm, n, r, i, step);
      float* dst = tabs + step * rr;
      const bool vec = (rr & 3) == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) == 0;
      if (vec) {
        for (int e = threadIdx.x * 4; e < rr; e += kSlotThreads * 4) cp_async_16(dst + e, src + e);
      } else {
        for (int e = threadIdx.x; e < rr; e += kSlotThreads) cp_async_4(dst + e, src + e);
      }
    }
    cp_async_commit();
  }

  // ---- log-sum-exp of every input unit of the slot: a lane's logits are fetched in batches of independent loads
  // (one batch covers 512 symbols; wider vocabularies take several, merged online)
  constexpr int kChunk = kSlotMaxPerLane * 32;
  for (int k = warp; k < r; k += nwarps) {
    const float* x = row + static_cast<size_t>(k) * v;
    float m = -CUDART_INF_F, s = 0.f;
    for (int c0 = 0; c0 < (WIDE ? v : 1); c0 += kChunk) {
      float xv[NQ];
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const int b = c0 + lane + 32 * q;
        xv[q] = b < vv ? x[b] : -CUDART_INF_F;   // [vv, v): padding symbols
      }
      float cm = xv[0];
#pragma unroll
      for (int q = 1; q < NQ; ++q) cm = fmaxf(cm, xv[q]);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) cm = fmaxf(cm, __shfl_xor_sync(kFull, cm, off));
      const float mn = fmaxf(m, cm);           // finite from the first chunk on (symbol 0 always exists)
      float cs = 0.f;
#pragma unroll
      for (int q = 0; q < NQ; ++q) cs += __expf(xv[q] - mn);   // padding: exp(-inf) = 0
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) cs += __shfl_xor_sync(kFull, cs, off);
      s = s * __expf(m - mn) + cs;             // first chunk: 0 * exp(-inf) = 0
      m = mn;
    }
    if (lane == 0) {
      unit_max[k] = m;
      unit_lse[k] = m + __logf(s);
      unit_lse_out[(static_cast<size_t>(pos) * n + i) * r + k] = unit_lse[k];   // kept for the acceptance stage
    }
  }
  if (tables_in_smem) cp_async_wait<0>();
  __syncthreads();

  const int per = (v + 31) / 32;   // consecutive bytes per lane in the CDF scan (<= kSlotMaxPerLane)
  const int nlat = (family == 0) ? 1 : (family == 1 ? n : n - 1);
  for (int j = warp; j < wpp; j += nwarps) {
    const size_t w = static_cast<size_t>(pos) * wpp + j;
    const float* u = uniforms + w * 2 * n;
    const float ub = u[n + i];
    // ---- latent draws down to the unit that owns slot i; every uniform the window's latent draws use is checked
    bool bad = false;
    for (int c = lane; c < nlat; c += 32) bad |= !(u[c] >= 0.f && u[c] < 1.f);
    bad = __any_sync(kFull, bad) || !(ub >= 0.f && ub < 1.f);
    int byte = -1;
    if (bad) {
      if (lane == 0) atomicOr(status, 2u);
    } else {
      int z = r > 32 ? warp_inv_cdf_logits_wide(lw, r, u[0], lane)     // CP only; the mixture logits are unnormalised
                     : warp_inv_cdf_logp(lane < r ? lw[lane] : 0.f, r, u[0], lane);
      if (family == 1) {
        for (int st = 0; st < chain; ++st) {
          const float* tab = tables_in_smem ? tabs + st * rr : hmm + static_cast<size_t>(st) * rr;
          z = warp_inv_cdf_logp(lane < r ? tab[z * r + lane] : 0.f, r, u[st + 1], lane);
        }
      } else if (family == 2) {
        const int code = n / 2 + (i >> 1);
        for (int st = 0; st < chain; ++st) {
          const int node = (code >> (chain - 1 - st)) - 1;
          const float* tab = tables_in_smem ? tabs + st * rr : lw + r + static_cast<size_t>(node - 1) * rr;
          z = warp_inv_cdf_logp(lane < r ? tab[z * r + lane] : 0.f, r, u[node], lane);
        }
      }
      const float* x = row + static_cast<size_t>(z) * v;
      const float m = unit_max[z];
      if (!WIDE) {
        // ---- inverse CDF over the v bytes of unit z: lane l owns bytes [l*per, (l+1)*per)
        byte = warp_inv_cdf_chunk<NQ>(x, 0, per, vv, m, ub, true, lane);
      } else {
        // ---- wide vocabulary: 512 symbols at a time. First the total (chunk sums in fp32, added up in fp64), then
        // the chunk the threshold u * total falls into, then the draw inside that chunk.
        double total = 0.0;
        for (int c0 = 0; c0 < v; c0 += kChunk) total += static_cast<double>(warp_chunk_sum(x, c0, vv, m, lane));
        const double thr = static_cast<double>(ub) * total;
        double before = 0.0;
        byte = vv - 1;                           // rounding may leave no index: the last one
        for (int c0 = 0; c0 < v; c0 += kChunk) {
          const float cs = warp_chunk_sum(x, c0, vv, m, lane);
          if (thr < before + static_cast<double>(cs)) {
            byte = warp_inv_cdf_chunk<kSlotMaxPerLane>(x, c0, kSlotMaxPerLane, vv, m, static_cast<float>(thr - before), false, lane);
            break;
          }
          before += static_cast<double>(cs);
        }
      }
    }
    if (lane == 0) out_bytes[w * n + i] = byte;
    // evidence of the drafted byte under every input unit of the slot; a draw that was refused (byte -1) has none:
    // NaN, so that the window's log-prob comes out as NaN rather than as the joint of its other bytes
    for (int k = lane; k < r; k += 32)
      G[(w * n + i) * r + k] = byte < 0 ? CUDART_NAN_F : row[static_cast<size_t>(k) * v + byte] - unit_lse[k];
  }
}

// ---------------------------------------------------------------- acceptance stage (Algorithm 3)
constexpr int kAcceptThreads = 256;

// Shared memory of one CTA (= one window) of spec_accept_kernel, in floats: the residual weights of the v bytes, the weight and the
// log-sum-exp of every input unit of the slot (2 r), and for the binary tree the product and sum-layer vectors of every
// node, one staged table and one vector.
__host__ __device__ inline size_t accept_warp_floats(int family, int n, int r, int v) {
  return 4 + static_cast<size_t>(v) + 2 * static_cast<size_t>(r) +                // 4: the accepted length, for all warps
         (family == 2 ? 2 * static_cast<size_t>(n - 1) * r + static_cast<size_t>(r) * (r + 1) + r : 0);
}

// One CTA per drafted window w (position p = w / wpp): warp 0 runs the tests and the short latent recursions, all
// warps share the residual row (v bytes x r units of exponentials, the bulk of the work), warp 0 draws. Inputs: the draft's bytes and prefix log-marginals, the
// target model's conditionals along the draft, one uniform per test plus one for the last byte; the logits and
// per-unit log-sum-exps the draft call left in the workspace.
//   1. s = 0; while s < n: the draft's conditional of byte s is q_s = exp(prefix[s] - prefix[s-1]) (prefix[-1] = 0);
//      stop if alpha_s > p(x_s) / q_s, tested as alpha_s * q_s > p(x_s); else s += 1.
//   2. s == n: the extra byte is drawn from the target row n.
//      s <  n: it is drawn from max(0, p(.) - q(. | x_0..x_{s-1})) / Z. The circuit's conditional of slot s is a
//      mixture of the slot's r input units, q(b | ..) = sum_k c_k phi_{s,k}(b), with c the posterior of the latent that
//      owns slot s given the accepted bytes: CP: omega_k prod_{i<s} phi_{i,k}(x_i); HMM: the one-step prediction
//      from alpha_{s-1}; BTree: the upward pass with the bytes >= s summed out, then the downward pass along the
//      path from the root to the node that owns token s.
//   Both draws are inverse-CDF on unnormalised weights (u * total < running sum, index order, no division).
__global__ void __launch_bounds__(kAcceptThreads) spec_accept_kernel(
    int family, const float* __restrict__ logits, const float* __restrict__ unit_lse, const float* __restrict__ logw,
    const float* __restrict__ logA, const int* __restrict__ bytes, const float* __restrict__ prefix,
    const float* __restrict__ target, const float* __restrict__ uniforms, int* __restrict__ out_accepted,
    int* __restrict__ out_next, unsigned* status, int W, int wpp, int n, int r, int v, int vv, int sum_rows,
    int logA_stride, const float* __restrict__ evidence, const int* __restrict__ row_of) {
  // evidence != NULL (after a many-position draft): log phi of the drafted bytes comes from evidence [W, n, r] (the G the
  // draft left), and `logits` [rows, r v] / `unit_lse` [rows, r] hold only the slot of each rejected window's first
  // rejected byte, at row row_of[w].
  extern __shared__ float sm[];
  int& accepted_len = *reinterpret_cast<int*>(sm);       // s, or -1: the window's inputs were refused
  const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int w = blockIdx.x;
  if (w >= W) return;
  float* mres = sm + 4;
  const int pos = w / wpp;
  const int* x = bytes + static_cast<size_t>(w) * n;
  const float* pre = prefix + static_cast<size_t>(w) * n;
  const float* u = uniforms + static_cast<size_t>(w) * (n + 1);
  const float* tp = target + static_cast<size_t>(w) * (n + 1) * v;
  const float* lw = logw + static_cast<size_t>(pos) * sum_rows;
  const bool has = lane < r;

  float* cw = mres + v;                                  // [r] weight of every input unit of slot s
  float* cl = cw + r;                                    // [r] its log-sum-exp
  if (wib == 0) {
  // ---- 1. acceptance tests
  bool bad_u = false, bad_x = false;
  for (int c = lane; c <= n; c += 32) bad_u |= !(u[c] >= 0.f && u[c] < 1.f);
  for (int c = lane; c < n; c += 32) bad_x |= static_cast<unsigned>(x[c]) >= static_cast<unsigned>(vv);
  bad_u = __any_sync(kFull, bad_u);
  bad_x = __any_sync(kFull, bad_x);
  if (bad_u || bad_x) {
    if (lane == 0) {
      atomicOr(status, bad_u ? 2u : 1u);
      out_accepted[w] = -1;
      out_next[w] = -1;
      accepted_len = -1;
    }
  } else {
  // lane i runs the test of byte i (all loads in flight at once); the first rejecting lane ends the accepted run
  int s = n;
  for (int base = 0; base < n && s == n; base += 32) {
    const int i = base + lane;
    bool rej = false;
    if (i < n) {
      const float q = __expf(pre[i] - (i > 0 ? pre[i - 1] : 0.f));
      rej = u[i] * q > tp[static_cast<size_t>(i) * v + x[i]];
    }
    const unsigned m = __ballot_sync(kFull, rej);
    if (m) s = base + __ffs(m) - 1;
  }
  if (lane == 0) {
    out_accepted[w] = s;
    accepted_len = s;
  }
  if (s < n) {
    // ---- 2. c[k]: log-weight of input unit k of slot s given the accepted bytes (lane = k)
    auto g_at = [&](int i, int k) -> float {   // log phi_{i,k}(x_i)
      if (evidence != nullptr) return evidence[(static_cast<size_t>(w) * n + i) * r + k];
      const size_t unit = (static_cast<size_t>(pos) * n + i) * r + k;
      return logits[unit * v + x[i]] - unit_lse[unit];
    };
    auto g_of = [&](int i) -> float { return g_at(i, lane); };
    // log-sum-exp of unit k of slot s
    auto lse_of = [&](int k) -> float {
      return evidence != nullptr ? unit_lse[static_cast<size_t>(row_of[w]) * r + k]
                                 : unit_lse[(static_cast<size_t>(pos) * n + s) * r + k];
    };
    float c = 0.f;
    if (family == 0) {
      // mixture of up to 128 components: lane handles k = lane, lane + 32, ...; the weights need no normalisation of
      // log omega (they are normalised below), so unnormalised mixture logits (r > 32) are as good
      float cq[4];
      float m = -CUDART_INF_F, sacc = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int k = lane + 32 * q;
        cq[q] = -CUDART_INF_F;
        if (k < r) {
          float a = lw[k];
#pragma unroll 4
          for (int i = 0; i < s; ++i) a += g_at(i, k);      // independent gathers: several in flight
          cq[q] = a;
          lse_merge(m, sacc, a, 1.f);
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float m2 = __shfl_xor_sync(kFull, m, off);
        const float s2 = __shfl_xor_sync(kFull, sacc, off);
        lse_merge(m, sacc, m2, s2);
      }
      const float lse_all = m + __logf(sacc);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int k = lane + 32 * q;
        if (k < r) {
          cw[k] = __expf(cq[q] - lse_all);
          cl[k] = lse_of(k);
        }
      }
    } else if (family == 1) {
      float alpha = has ? lw[lane] : -CUDART_INF_F;
      for (int i = 0; i < s; ++i) {
        // alpha_i = g_i + (i == 0 ? log pi : LSE_a(alpha_{i-1}[a] + logA[i-1][a][.])); then one more prediction step
        if (has) alpha += g_of(i);
        float m = alpha;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, off));
        const float e = has ? __expf(alpha - m) : 0.f;
        const float* A = logA + static_cast<size_t>(pos) * logA_stride + static_cast<size_t>(i) * r * r;
        float acc = 0.f;
        for (int a0 = 0; a0 < r; a0 += 16) {           // sixteen rows of the table in flight at a time
          float tv[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) tv[q] = (has && a0 + q < r) ? __ldg(A + (a0 + q) * r + lane) : -CUDART_INF_F;
#pragma unroll
          for (int q = 0; q < 16; ++q)
            if (a0 + q < r) acc = fmaf(__shfl_sync(kFull, e, a0 + q), __expf(tv[q]), acc);
        }
        alpha = has ? m + __logf(acc) : -CUDART_INF_F;
      }
      c = alpha;
    } else {
      float* prod = cl + r;
      float* S = prod + (n - 1) * r;
      float* table = S + (n - 1) * r;
      float* cur = table + r * (r + 1);
      const int first_leaf_node = n / 2 - 1;
      for (int j = n - 2; j >= first_leaf_node; --j) {
        const int t0 = 2 * (j - first_leaf_node);
        if (has) prod[j * r + lane] = (t0 < s ? g_of(t0) : 0.f) + (t0 + 1 < s ? g_of(t0 + 1) : 0.f);
      }
      __syncwarp();
      for (int j = first_leaf_node - 1; j >= 0; --j) {
        float acc = 0.f;
        for (int side = 0; side < 2; ++side) {
          const int ch = 2 * j + 1 + side;
          const float sc = btree_sum_layer<16>(lw + r + static_cast<size_t>(ch - 1) * r * r, prod + ch * r, table, lane, r);
          if (has) S[ch * r + lane] = sc;
          acc += sc;
        }
        if (has) prod[j * r + lane] = acc;
        __syncwarp();
      }
      // downward: up[z] = log-weight of the rest of the circuit seen from the current path node with latent z
      const int owner = first_leaf_node + (s >> 1);
      const int code = owner + 1;
      const int depth = 31 - __clz(code);
      int node = 0;
      float up = has ? lw[lane] : -CUDART_INF_F;
      for (int lvl = depth - 1; lvl >= 0; --lvl) {
        const int child = 2 * node + 1 + ((code >> lvl) & 1);
        const int sib = (child & 1) ? child + 1 : child - 1;
        if (has) cur[lane] = up + S[sib * r + lane];
        __syncwarp();
        // the child's table [parent value z][own value b], staged into the padded shared tile first
        btree_stage_table<16>(lw + r + static_cast<size_t>(child - 1) * r * r, table, lane, r);
        __syncwarp();
        float m = -CUDART_INF_F;
        for (int z = 0; z < r; ++z) m = fmaxf(m, has ? cur[z] + table[z * (r + 1) + lane] : -CUDART_INF_F);
        float acc = 0.f;
        for (int z = 0; z < r; ++z) acc += has ? __expf(cur[z] + table[z * (r + 1) + lane] - m) : 0.f;
        up = has ? m + __logf(acc) : -CUDART_INF_F;
        __syncwarp();
        node = child;
      }
      const int other_leaf = s ^ 1;
      c = up + ((has && other_leaf < s) ? g_of(other_leaf) : 0.f);
    }
    if (family != 0) {                                   // HMM, BTree: one weight per lane (r <= 32)
      const float c_lse = warp_lse(c, has);              // every lane takes part in the shuffles
      if (has) {
        cw[lane] = __expf(c - c_lse);
        cl[lane] = lse_of(lane);
      }
    }
  }
  }
  }   // warp 0
  __syncthreads();
  const int s = accepted_len;
  if (s < 0) return;
  const float* trow = tp + static_cast<size_t>(s) * v;
  // ---- residual weights of the v bytes, all warps
  if (s == n) {
    for (int b = threadIdx.x; b < v; b += kAcceptThreads) mres[b] = b < vv ? trow[b] : 0.f;
  } else {
    const float* lrow = evidence != nullptr ? logits + static_cast<size_t>(row_of[w]) * r * v
                                            : logits + (static_cast<size_t>(pos) * n + s) * r * v;   // [r, v] logits of slot s
    for (int b = threadIdx.x; b < v; b += kAcceptThreads) {
      float q = 0.f;
      if (b < vv) {
        // the r logits of byte b come from r different rows: eight loads in flight at a time, two accumulation chains
        float q1 = 0.f;
        int k = 0;
        for (; k + 8 <= r; k += 8) {
          float xv[8];
#pragma unroll
          for (int t = 0; t < 8; ++t) xv[t] = lrow[static_cast<size_t>(k + t) * v + b];
#pragma unroll
          for (int t = 0; t < 8; t += 2) {
            q = fmaf(cw[k + t], __expf(xv[t] - cl[k + t]), q);
            q1 = fmaf(cw[k + t + 1], __expf(xv[t + 1] - cl[k + t + 1]), q1);
          }
        }
        for (; k < r; ++k) q = fmaf(cw[k], __expf(lrow[static_cast<size_t>(k) * v + b] - cl[k]), q);
        q += q1;
      }
      mres[b] = b < vv ? fmaxf(0.f, trow[b] - q) : 0.f;   // padding symbols carry no mass
    }
  }
  __syncthreads();
  if (wib != 0) return;

  // ---- 3. inverse CDF over the weights in mres (warp 0): lane l owns bytes [l*per, (l+1)*per)
  const int per = (v + 31) / 32;
  const int b0 = lane * per;
  float part = 0.f;
  for (int q = 0; q < per; ++q)
    if (b0 + q < v) part += mres[b0 + q];
  const float incl = warp_scan_incl(part, lane);
  const float total = __shfl_sync(kFull, incl, 31);
  const float thr = u[n] * total;
  const unsigned hit = __ballot_sync(kFull, thr < incl);
  int byte = vv - 1;   // rounding may leave no index: the last one
  if (hit) {
    const int src = __ffs(hit) - 1;
    int found = -1;
    const float before = __shfl_up_sync(kFull, incl, 1);
    if (lane == src) {
      float cum = lane == 0 ? 0.f : before;
      for (int q = 0; q < per && found < 0; ++q)
        if (b0 + q < vv) {
          cum += mres[b0 + q];
          if (thr < cum) found = b0 + q;
        }
      if (found < 0) found = min(b0 + per, vv) - 1;
    }
    byte = __shfl_sync(kFull, found, src);
  }
  if (lane == 0) out_next[w] = byte;
}

// The tests of Algorithm 3 alone, one warp per window: first_rejected[w] = s if the draft is rejected at byte s < n, else -1
// (everything accepted, or inputs that the acceptance kernel will refuse). Decides which slot's logits the acceptance
// stage after a many-position draft has to recompute for the window.
__global__ void accept_test_kernel(const int* __restrict__ bytes, const float* __restrict__ prefix,
                                   const float* __restrict__ target, const float* __restrict__ uniforms,
                                   int* __restrict__ first_rejected, int W, int n, int v, int vv) {
  const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= W) return;
  const int* x = bytes + static_cast<size_t>(w) * n;
  const float* pre = prefix + static_cast<size_t>(w) * n;
  const float* u = uniforms + static_cast<size_t>(w) * (n + 1);
  const float* tp = target + static_cast<size_t>(w) * (n + 1) * v;
  bool bad = false;
  for (int c = lane; c <= n; c += 32) bad |= !(u[c] >= 0.f && u[c] < 1.f);
  for (int c = lane; c < n; c += 32) bad |= static_cast<unsigned>(x[c]) >= static_cast<unsigned>(vv);
  bad = __any_sync(kFull, bad);
  int s = n;
  if (!bad) {
    for (int base = 0; base < n && s == n; base += 32) {
      const int i = base + lane;
      bool rej = false;
      if (i < n) {
        const float q = __expf(pre[i] - (i > 0 ? pre[i - 1] : 0.f));
        rej = u[i] * q > tp[static_cast<size_t>(i) * v + x[i]];
      }
      const unsigned m = __ballot_sync(kFull, rej);
      if (m) s = base + __ffs(m) - 1;
    }
  }
  if (lane == 0) first_rejected[w] = (bad || s == n) ? -1 : s;
}

}  // namespace mtpc
