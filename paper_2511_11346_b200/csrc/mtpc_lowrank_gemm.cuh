// Projection kernel of a head whose unembeddings are shared across the components of a slot and adapted by low-rank
// terms (App. G): U_ij = W_i + A_ij B_ij, so logit[t, i, j, :] = W_i h_t + A_ij (B_ij h_t). The composed [n, r, v, d]
// tensor is never formed. Per (128 positions, slot i):
//   base    = h W_i^T            one weight-sized-over-r contraction (K = d), v accumulator columns kept in tensor memory;
//   corr_j  = z_j A_ij^T         for each of the r components one K = k contraction on z_j = B_ij h (computed by a plain
//                                GEMM beforehand whose epilogue splits it into two bf16 halves, z = hi + lo, so that rounding z to the
//                                tensor cores' operand type costs 2^-17 instead of 2^-9), in chunks of `chunk_cols` columns
//                                through a few accumulator slots (enough of them in flight to cover the round trip
//                                slot released -> MMAs issued -> commit seen, which is longer than a chunk's epilogue);
//   epilogue: x = base + corr_j, then exactly the log-likelihood epilogue of the dense kernel (online log-sum-exp over the
//             unit's v columns, target gather, G = logit[target] - LSE).
// FLOPs per position: 2 d (n v + n r k) + 4 n r v k instead of 2 d n r v.
// Roles: warp 0 TMA producer, warp 1 MMA issuer, then `groups` epilogue groups of four warps (one thread per position):
// group g takes the components j = g, g + groups, ... of a slot and owns two correction slots. The epilogue (one
// exponential per logit, n r v of them per position) is what bounds this kernel once the contraction has shrunk, and a
// lone warp per scheduler cannot keep the special-function pipe busy: several groups can.
// One shared-memory ring carries both kinds of entries: a 64-wide K block of (h, W_i), or the operands of one component's
// correction (z_hi, z_lo: k/16 boxes of 128 rows x 16 each; A_ij: k/16 x nchunk boxes of chunk_cols rows x 16), all as
// 32-byte rows with the 32-byte swizzle, so every correction MMA (K = 16) starts at the base of its own box.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>

#include "mtpc_gemm.cuh"

namespace mtpc {

constexpr int kLrMaxRank = 32;          // k <= 32 (a multiple of 16)
constexpr int kLrMaxGroups = 3;         // epilogue groups: 64 + 128 * groups threads per CTA
constexpr int kLrBaseSlot = kMaxSlots - 1;   // barrier index of the base accumulator (0 .. corr_slots - 1: the correction slots)

struct LowRankGemmParams {
  CUtensorMap tm_h;      // hidden [T, d]              box 64 x 128, 128-byte swizzle
  CUtensorMap tm_w;      // W_base [n*v, d]            box 64 x base_box_rows, 128-byte swizzle
  CUtensorMap tm_z;      // z      [T, n*r*2*k]        box 16 x 128, 32-byte swizzle (unit u: hi at (2u)k, lo at (2u+1)k)
  CUtensorMap tm_a;      // A      [n*r*v, k]          box 16 x chunk_cols, 32-byte swizzle
  int T, m_tiles, kblocks;
  int n, r, v, vv, k;
  int base_boxes, base_box_rows;     // W_i is fetched as base_boxes boxes of base_box_rows rows (v > 256: two halves)
  int chunk_cols, nchunk;            // correction chunks: nchunk = ceil(v / chunk_cols)
  int corr_col0;                     // first tensor-memory column of correction slot 0 (slot s follows at + s * chunk_cols)
  int groups;                        // epilogue groups (1 .. kLrMaxGroups), each with two correction slots of chunk_cols columns
  int stages, stage_bytes;
  const int* targets;                // [T, n]
  float* G;                          // [T, n, r]
  unsigned* status;
  uint64_t wait_limit_ns;
};

// K-major operand tile whose rows are `row_bytes` (32, 64 or 128) wide and swizzled with that span: 8-row groups are
// 8 * row_bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc_kmajor(uint32_t smem_addr, uint32_t row_bytes) {
  const uint64_t layout = row_bytes == 128 ? 2 : (row_bytes == 64 ? 4 : 6);
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>((8 * row_bytes) >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= layout << 61;
  return d;
}

__global__ void __launch_bounds__(64 + 128 * kLrMaxGroups, 1) mtpc_lowrank_gemm_kernel(const __grid_constant__ LowRankGemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (tiles_addr - raw_addr);
  GemmControl* ctl = reinterpret_cast<GemmControl*>(tiles + static_cast<size_t>(p.stages) * p.stage_bytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_items = p.m_tiles * p.n;                 // slot fastest: the CTAs running together share the hidden tiles
  const int kq = p.k / 16;                                // K = 16 steps of one correction
  const uint32_t zbox = kBlockM * 32;                     // bytes of one z box (128 rows x 32 bytes)
  const uint32_t abox = static_cast<uint32_t>(p.chunk_cols) * 32;
  const uint32_t a_off = 2 * kq * zbox;                   // correction entry: [z_hi boxes | z_lo boxes | A boxes (q, c)]
  const uint32_t base_b_off = kABytes;                    // base entry: [h tile | W_i boxes]

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int s = 0; s < 2 * p.groups; ++s) {
      mbar_init(smem_u32(&ctl->tfull[s]), 1);
      mbar_init(smem_u32(&ctl->tempty[s]), 4);
    }
    mbar_init(smem_u32(&ctl->tfull[kLrBaseSlot]), 1);
    mbar_init(smem_u32(&ctl->tempty[kLrBaseSlot]), 4 * p.groups);
    mbar_init(smem_u32(&ctl->drain), 1);
    ctl->abort = 0;
    ctl->wait_limit_ns = p.wait_limit_ns;
    fence_mbar_init();
    tma_prefetch_desc(&p.tm_h);
    tma_prefetch_desc(&p.tm_w);
    tma_prefetch_desc(&p.tm_z);
    tma_prefetch_desc(&p.tm_a);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued_mask = 0, phase_mask = 0;
      bool ok = true;
      const uint32_t base_bytes = kABytes + static_cast<uint32_t>(p.base_boxes * p.base_box_rows) * (kBlockK * 2);
      const uint32_t corr_bytes = 2 * kq * zbox + static_cast<uint32_t>(kq * p.nchunk) * abox;
      auto advance = [&]() {
        issued_mask |= 1u << stage;
        phase_mask = (phase_mask & ~(1u << stage)) | (phase << stage);
        if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; }
      };
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
        const int mt = item / p.n, slot_i = item - mt * p.n;
        for (int kb = 0; kb < p.kblocks && ok; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctl->full[stage]);
          const uint32_t dst = tiles_addr + stage * p.stage_bytes;
          mbar_arrive_expect_tx(full, base_bytes);
          tma_load_2d(dst, &p.tm_h, full, kb * kBlockK, mt * kBlockM);
          for (int q = 0; q < p.base_boxes; ++q)
            tma_load_2d(dst + base_b_off + q * p.base_box_rows * (kBlockK * 2), &p.tm_w, full, kb * kBlockK,
                        slot_i * p.v + q * p.base_box_rows);
          advance();
        }
        for (int j = 0; j < p.r && ok; ++j) {
          if (!bounded_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctl->full[stage]);
          const uint32_t dst = tiles_addr + stage * p.stage_bytes;
          const int unit = slot_i * p.r + j;
          mbar_arrive_expect_tx(full, corr_bytes);
          for (int part = 0; part < 2; ++part)
            for (int q = 0; q < kq; ++q)
              tma_load_2d(dst + (part * kq + q) * zbox, &p.tm_z, full, (2 * unit + part) * p.k + 16 * q, mt * kBlockM);
          for (int q = 0; q < kq; ++q)
            for (int c = 0; c < p.nchunk; ++c)
              tma_load_2d(dst + a_off + (q * p.nchunk + c) * abox, &p.tm_a, full, 16 * q, unit * p.v + c * p.chunk_cols);
          advance();
        }
      }
      // no copy may still be in flight when the CTA goes away
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
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, it = 0;
      uint32_t cuse[kLrMaxGroups] = {0, 0, 0};                      // chunks issued so far for each epilogue group
      bool ok = true;
      const int base_n = p.base_box_rows;                           // columns per base MMA (v, or v / 2)
      const uint32_t idesc_base = umma_idesc_bf16(kBlockM, base_n);
      auto next_stage = [&]() { if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; } };
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++it) {
        // ---- base: all K blocks into columns [0, v)
        if (!bounded_wait(smem_u32(&ctl->tempty[kLrBaseSlot]), (it & 1u) ^ 1u, ctl, p.status)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->full[stage]), phase, ctl, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t addr = tiles_addr + stage * p.stage_bytes;
          const uint64_t a_desc = umma_smem_desc_sw128(addr);
          for (int q = 0; q < p.base_boxes; ++q) {
            const uint64_t b_desc = umma_smem_desc_sw128(addr + base_b_off + q * base_n * (kBlockK * 2));
#pragma unroll
            for (int kk = 0; kk < kBlockK / 16; ++kk)
              umma_bf16(tmem_base + q * base_n, a_desc + 2 * kk, b_desc + 2 * kk, idesc_base, (kb | kk) != 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&ctl->empty[stage]));
          next_stage();
        }
        if (!ok) break;
        umma_commit(smem_u32(&ctl->tfull[kLrBaseSlot]));
        // ---- corrections, `groups` components at a time (component j0 + g belongs to epilogue group g): their chunks
        // are issued in turn, chunk c of component j0 + g into slot 2 g + (that group's chunk count & 1)
        for (int j0 = 0; j0 < p.r && ok; j0 += p.groups) {
          const int ng = min(p.groups, p.r - j0);
          uint32_t addr[kLrMaxGroups], estage[kLrMaxGroups];
          for (int g = 0; g < ng && ok; ++g) {
            if (!bounded_wait(smem_u32(&ctl->full[stage]), phase, ctl, p.status)) { ok = false; break; }
            addr[g] = tiles_addr + stage * p.stage_bytes;
            estage[g] = stage;
            next_stage();
          }
          if (!ok) break;
          tc_fence_after();
          for (int c = 0; c < p.nchunk && ok; ++c) {
            const int width = min(p.chunk_cols, p.v - c * p.chunk_cols);
            const uint32_t idesc = umma_idesc_bf16(kBlockM, width);
            for (int g = 0; g < ng; ++g) {
              const uint32_t slot = 2 * g + (cuse[g] & 1u);
              if (!bounded_wait(smem_u32(&ctl->tempty[slot]), ((cuse[g] >> 1) & 1u) ^ 1u, ctl, p.status)) { ok = false; break; }
              tc_fence_after();
              const uint32_t d_tmem = tmem_base + p.corr_col0 + slot * p.chunk_cols;
              uint32_t acc = 0;
              for (int part = 0; part < 2; ++part)
                for (int q = 0; q < kq; ++q) {
                  umma_bf16(d_tmem, umma_smem_desc_kmajor(addr[g] + (part * kq + q) * zbox, 32),
                            umma_smem_desc_kmajor(addr[g] + a_off + (q * p.nchunk + c) * abox, 32), idesc, acc);
                  acc = 1;
                }
              umma_commit(smem_u32(&ctl->tfull[slot]));
              ++cuse[g];
            }
          }
          if (!ok) break;
          for (int g = 0; g < ng; ++g) umma_commit(smem_u32(&ctl->empty[estage[g]]));
        }
      }
      if (!ok) {   // wait (bounded) for the MMAs already issued before tensor memory is freed
        umma_commit(smem_u32(&ctl->drain));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;
    const int group = (warp - 2) >> 2;                        // this warp's epilogue group: components group, group + groups, ...
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    uint32_t it = 0, cuse = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++it) {
      const int mt = item / p.n, slot_i = item - mt * p.n;
      const int row = mt * kBlockM + quarter * 32 + lane;
      const bool valid = row < p.T;
      const int tgt = valid ? p.targets[static_cast<size_t>(row) * p.n + slot_i] : -1;
      if (!bounded_wait_warp(smem_u32(&ctl->tfull[kLrBaseSlot]), it & 1u, ctl, p.status, lane)) { ok = false; break; }
      tc_fence_after();
      for (int j = group; j < p.r && ok; j += p.groups) {
        float m = -CUDART_INF_F, s = 0.f, tval = 0.f;
        for (int c = 0; c < p.nchunk; ++c, ++cuse) {
          const uint32_t slot = 2 * group + (cuse & 1u);
          if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (cuse >> 1) & 1u, ctl, p.status, lane)) { ok = false; break; }
          tc_fence_after();
          const int col_chunk = c * p.chunk_cols;
          const int width = min(p.chunk_cols, p.v - col_chunk);
          const uint32_t ccol = lane_base + p.corr_col0 + slot * p.chunk_cols;
          // one batch of 16 columns: correction + base, then the dense kernel's online log-sum-exp and target gather
          auto consume = [&](const uint32_t (&rc)[16], const uint32_t (&rb)[16], int b) {
            float x[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = __uint_as_float(rc[q]) + __uint_as_float(rb[q]);
            const int col0 = col_chunk + b * 16;
            mask_padding(x, col0, p.vv);
            // short dependent chains: reduce as trees
            float t8[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) t8[q] = fmaxf(x[q], x[q + 8]);
            const float bm = fmaxf(fmaxf(fmaxf(t8[0], t8[1]), fmaxf(t8[2], t8[3])), fmaxf(fmaxf(t8[4], t8[5]), fmaxf(t8[6], t8[7])));
            const float mn = fmaxf(m, bm);
            const float mn2 = mn * kLog2e;
            const float rescale = fast_ex2((m - mn) * kLog2e);
            float e[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) e[q] = fast_ex2(fmaf(x[q], kLog2e, -mn2));
#pragma unroll
            for (int q = 0; q < 8; ++q) e[q] += e[q + 8];
            s = fmaf(s, rescale, ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7])));
            m = mn;
            const int rel = tgt - col0;
            if (static_cast<unsigned>(rel) < 16u) {
#pragma unroll
              for (int q = 0; q < 16; ++q)
                if (rel == q) tval = x[q];
            }
          };
          // both loads of the next batch are in flight while this one goes through the exponentials
          const int nb = width / 16;
          uint32_t c0[16], b0[16], c1[16], b1[16];
          tmem_ld16_issue(ccol, c0);
          tmem_ld16_issue(lane_base + col_chunk, b0);
          tmem_ld_wait16(c0);
          tmem_ld_wait16(b0);
          for (int b = 0; b < nb; b += 2) {
            if (b + 1 < nb) {
              tmem_ld16_issue(ccol + (b + 1) * 16, c1);
              tmem_ld16_issue(lane_base + col_chunk + (b + 1) * 16, b1);
            }
            consume(c0, b0, b);
            if (b + 1 >= nb) break;
            tmem_ld_wait16(c1);
            tmem_ld_wait16(b1);
            if (b + 2 < nb) {
              tmem_ld16_issue(ccol + (b + 2) * 16, c0);
              tmem_ld16_issue(lane_base + col_chunk + (b + 2) * 16, b0);
            }
            consume(c1, b1, b + 1);
            if (b + 2 < nb) {
              tmem_ld_wait16(c0);
              tmem_ld_wait16(b0);
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&ctl->tempty[slot]));
        }
        if (!ok) break;
        if (valid) {
          float* g = p.G + (static_cast<size_t>(row) * p.n + slot_i) * p.r + j;
          if (tgt < 0) {
            *g = 0.f;                                  // marginalised byte: the input unit sums to 1
          } else if (tgt >= p.vv) {
            *g = CUDART_NAN_F;
            atomicOr(p.status, kStatusBadTarget);
          } else {
            *g = tval - (m + fast_lg2(s) * kLn2);
          }
        }
      }
      if (!ok) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tempty[kLrBaseSlot]));   // the next item's base may overwrite the columns
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace mtpc
