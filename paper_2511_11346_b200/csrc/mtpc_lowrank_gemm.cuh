// Projection kernel of a head whose unembeddings are shared across the components of a slot and adapted by low-rank
// terms (App. G): U_ij = W_i + A_ij B_ij, so logit[t, i, j, :] = W_i h_t + A_ij (B_ij h_t). The composed [n, r, v, d]
// tensor is never formed. A unit's v columns are cut into `panels` panels of panel_cols columns (the last one may be
// narrower); a work item is (128 positions, slot i, panel):
//   base    = h W_i^T            the panel's columns of the one weight-sized-over-r contraction (K = d), accumulated into one
//                                of TWO tensor-memory buffers, so that the next item's base runs while this item's
//                                corrections and epilogue are under way;
//   corr_j  = z_j A_ij^T         for each of the r components one K = 2k contraction on z_j = B_ij h (computed by a plain
//                                GEMM beforehand whose epilogue splits it into two bf16 halves, z = hi + lo, so that rounding z to
//                                the tensor cores' operand type costs 2^-17 instead of 2^-9), in chunks of chunk_cols columns
//                                through two accumulator slots per epilogue group;
//   epilogue: x = base + corr_j, then the log-likelihood epilogue of the dense kernel on the panel (online log-sum-exp,
//             target gather). One panel: G = logit[target] - LSE directly. Several: every panel leaves (max, sum of
//             exponentials) per (position, slot, component), the panel that holds the target leaves its logit, and
//             lowrank_merge_kernel combines them - so the items are independent and deal out evenly.
// FLOPs per position: 2 d (n v + n r k) + 4 n r v k instead of 2 d n r v.
// Roles: warp 0 TMA producer of the base operands, warp 1 MMA issuer of the base, warp 2 TMA producer of the correction
// operands, warps 3 .. 2 + groups one MMA issuer of corrections per epilogue group (issuing one of these small MMAs holds
// its thread for a few hundred cycles although the tensor pipe is nearly idle: the issuers must not queue behind each
// other), then from warp 8 on `groups` epilogue groups of four warps (one thread per position): group g takes the
// components j = g, g + groups, ... The two pipelines share nothing but the tensor cores: each has its
// own shared-memory ring and its own barriers. Base ring: a 64-wide K block of h and of the panel's rows of W_i. Correction
// ring: one entry holds the operands of 64 / k components, all as 128-byte rows with the 128-byte swizzle (few large boxes
// instead of many 32-byte-row ones): z as boxes of 128 positions x 64 values = [hi | lo] of 32 / k adjacent
// components, and A as boxes of chunk_cols vocabulary rows x 64 values = the k adaptor columns of 64 / k adjacent components,
// read from a copy of A laid out [n, v, r, k] (lowrank_repack_kernel, made on every call: A is small and may have changed).
// A correction MMA (K = 16) addresses its operands inside those rows, 32 bytes apart, like the K steps of the base.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>

#include "mtpc_circuit.cuh"
#include "mtpc_decode.cuh"
#include "mtpc_gemm.cuh"

namespace mtpc {

constexpr int kLrMaxRank = 32;          // k <= 32 (a multiple of 16)
constexpr int kLrMaxGroups = 2;         // epilogue groups: 256 + 128 * groups threads per CTA (512: 128 registers each)
constexpr int kLrMaxPanels = 8;
constexpr int kLrCorrStages = 4;        // entries of the correction operand ring (at most)
constexpr int kLrRoleThreads = 256;     // the single-thread roles, one warp each: warps 0 .. 2 + groups (the rest idle)

struct LowRankGemmParams {
  CUtensorMap tm_h;      // hidden [T, d]              box 64 x 128, 128-byte swizzle
  CUtensorMap tm_w;      // W_base [n*v, d]            box 64 x panel_cols, 128-byte swizzle
  CUtensorMap tm_z;      // z      [T, n*r*2*k]        box 64 x 128, 128-byte swizzle (unit u: hi at (2u)k, lo at (2u+1)k)
  CUtensorMap tm_a;      // A'     [n*v, r*k]          box 64 x chunk_cols, 128-byte swizzle (row (i, b): A[i, 0..r-1, b, :])
  int T, m_tiles, kblocks;
  int n, r, v, vv, k;
  int panels, panel_cols;            // panel q covers the columns [q panel_cols, min(v, (q + 1) panel_cols)) of a unit
  int acc_stride;                    // tensor-memory columns between the two base buffers (panel_cols rounded up to 32)
  int chunk_cols, nchunk;            // correction chunks of a full panel: nchunk = ceil(panel_cols / chunk_cols)
  int corr_col0;                     // first tensor-memory column of correction slot 0 (slot s follows at + s * chunk_cols)
  int groups;                        // epilogue groups (1 .. kLrMaxGroups), each with two correction slots of chunk_cols columns
  int base_stages, base_stage_bytes, corr_stages, corr_stage_bytes;
  const int* targets;                // [T, n]
  float* G;                          // [T, n, r]
  float2* partial;                   // panels > 1: [panels, T n r] (running maximum, sum of exponentials) of each panel
  float* target_logit;               // panels > 1: [T n r] logit of the target, written by the panel that holds it
  float* logit_out;                  // training: every logit [T, n r v] fp32 at a pitch of logit_pitch (NULL: not kept) ...
  size_t logit_pitch;
  float* lse_out;                    // ... and every unit's log-sum-exp [T, n r] (with several panels: by the merge kernel)
  int missing_is_nan;                // the targets are drafted bytes: -1 is a refused draw (G = NaN), not a marginalised byte (G = 0)
  unsigned* status;
  uint64_t wait_limit_ns;
};

struct LowRankControl {
  GemmControl g;                     // full / empty: base ring; tfull / tempty: correction slots; abort, limits, tmem_base
  uint64_t cfull[kLrCorrStages];     // correction operand ring
  uint64_t cempty[kLrCorrStages];
  uint64_t afull[2];                 // base accumulators
  uint64_t aempty[2];
  uint64_t drain2[kLrMaxGroups];
};

// Wait (bounded) until the copies a producer still has in flight have landed: no copy may be in flight when the CTA goes.
__device__ __forceinline__ void lowrank_drain_ring(uint64_t* full, int stages, uint32_t issued_mask, uint32_t phase_mask) {
  for (int s = 0; s < stages; ++s)
    if (issued_mask & (1u << s)) {
      const uint32_t bar = smem_u32(&full[s]);
      const uint32_t par = (phase_mask >> s) & 1u;
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(bar, par) && global_timer_ns() - t0 < kWaitLimitNs) {}
    }
}

struct LowRankItem {
  int mt, slot, panel;
  int width;     // columns of this panel (the last panel of a unit may be narrower), a multiple of 16
  int nchunk;    // correction chunks that cover them
};
// panel fastest, then slot: the CTAs that run together share the hidden tile (and the slot's W_i) through L2
__device__ __forceinline__ LowRankItem lowrank_item(const LowRankGemmParams& p, int item) {
  LowRankItem c;
  c.panel = item % p.panels;
  const int rest = item / p.panels;
  c.slot = rest % p.n;
  c.mt = rest / p.n;
  c.width = min(p.panel_cols, p.v - c.panel * p.panel_cols);
  c.nchunk = (c.width + p.chunk_cols - 1) / p.chunk_cols;
  return c;
}

__global__ void __launch_bounds__(kLrRoleThreads + 128 * kLrMaxGroups, 1)
mtpc_lowrank_gemm_kernel(const __grid_constant__ LowRankGemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base_ring = (raw_addr + 1023u) & ~1023u;
  const uint32_t corr_ring = base_ring + static_cast<uint32_t>(p.base_stages * p.base_stage_bytes);
  uint8_t* tiles = smem_raw + (base_ring - raw_addr);
  LowRankControl* lc = reinterpret_cast<LowRankControl*>(tiles + static_cast<size_t>(p.base_stages) * p.base_stage_bytes +
                                                         static_cast<size_t>(p.corr_stages) * p.corr_stage_bytes);
  GemmControl* ctl = &lc->g;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_items = p.m_tiles * p.n * p.panels;
  const int kq = p.k / 16;                                // K = 16 steps of one half of a correction
  const int ca = 64 / p.k;                                // components per correction entry (= per box of A')
  const int cz = 32 / p.k;                                // components per box of z; an entry has ca / cz = 2 of them
  const int nent = (p.r + ca - 1) / ca;                   // correction entries per item
  const uint32_t zbox = kBlockM * 128;                    // bytes of one z box (128 rows x 128 bytes)
  const uint32_t abox = static_cast<uint32_t>(p.chunk_cols) * 128;
  const uint32_t a_off = 2 * zbox;                        // correction entry: [z box 0 | z box 1 | A' boxes c = 0 .. nchunk - 1]

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.base_stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int s = 0; s < p.corr_stages; ++s) {
      mbar_init(smem_u32(&lc->cfull[s]), 1);
      mbar_init(smem_u32(&lc->cempty[s]), p.groups);        // every correction issuer hands an entry back
    }
    for (int s = 0; s < 2 * p.groups; ++s) {
      mbar_init(smem_u32(&ctl->tfull[s]), 1);
      mbar_init(smem_u32(&ctl->tempty[s]), 4);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&lc->afull[s]), 1);
      mbar_init(smem_u32(&lc->aempty[s]), 4 * p.groups);
    }
    mbar_init(smem_u32(&ctl->drain), 1);
    for (int g = 0; g < p.groups; ++g) mbar_init(smem_u32(&lc->drain2[g]), 1);
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
    // ------------------------------------------------------------------ TMA producer, base operands
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued_mask = 0, phase_mask = 0;
      bool ok = true;
      const uint32_t bytes = kABytes + static_cast<uint32_t>(p.panel_cols) * (kBlockK * 2);
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
        const LowRankItem w = lowrank_item(p, item);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctl->full[stage]);
          const uint32_t dst = base_ring + stage * p.base_stage_bytes;
          mbar_arrive_expect_tx(full, bytes);
          tma_load_2d(dst, &p.tm_h, full, kb * kBlockK, w.mt * kBlockM);
          // the box is panel_cols rows high also for a narrower last panel: the rows past it (the next slot's, or
          // zeros past the end of W_base) are not multiplied
          tma_load_2d(dst + kABytes, &p.tm_w, full, kb * kBlockK, w.slot * p.v + w.panel * p.panel_cols);
          issued_mask |= 1u << stage;
          phase_mask = (phase_mask & ~(1u << stage)) | (phase << stage);
          if (++stage == static_cast<uint32_t>(p.base_stages)) { stage = 0; phase ^= 1u; }
        }
      }
      lowrank_drain_ring(ctl->full, p.base_stages, issued_mask, phase_mask);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer, base: item `it` into buffer it & 1
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, it = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++it) {
        const uint32_t idesc = umma_idesc_bf16(kBlockM, lowrank_item(p, item).width);
        const uint32_t buf = it & 1u;
        if (!bounded_wait(smem_u32(&lc->aempty[buf]), ((it >> 1) & 1u) ^ 1u, ctl, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * p.acc_stride;
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->full[stage]), phase, ctl, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t addr = base_ring + stage * p.base_stage_bytes;
          const uint64_t a_desc = umma_smem_desc_sw128(addr);
          const uint64_t b_desc = umma_smem_desc_sw128(addr + kABytes);
#pragma unroll
          for (int kk = 0; kk < kBlockK / 16; ++kk)
            umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          umma_commit(smem_u32(&ctl->empty[stage]));
          if (++stage == static_cast<uint32_t>(p.base_stages)) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&lc->afull[buf]));
      }
      if (!ok || ctl->abort) {   // wait (bounded) for the MMAs already issued before tensor memory is freed
        umma_commit(smem_u32(&ctl->drain));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&ctl->drain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ------------------------------------------------------------------ TMA producer, correction operands
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued_mask = 0, phase_mask = 0;
      bool ok = true;
      const uint32_t bytes = 2 * zbox + static_cast<uint32_t>(p.nchunk) * abox;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
        const LowRankItem w = lowrank_item(p, item);
        for (int e = 0; e < nent; ++e) {
          if (!bounded_wait(smem_u32(&lc->cempty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
          const uint32_t full = smem_u32(&lc->cfull[stage]);
          const uint32_t dst = corr_ring + stage * p.corr_stage_bytes;
          const int unit0 = w.slot * p.r + e * ca;           // first component of the entry
          mbar_arrive_expect_tx(full, bytes);
          // boxes may cover components past the slot's last (the next slot's, or zeros past the end) and, for A',
          // rows past the panel: none of that is multiplied
          for (int bx = 0; bx < 2; ++bx)
            tma_load_2d(dst + bx * zbox, &p.tm_z, full, (unit0 + bx * cz) * 2 * p.k, w.mt * kBlockM);
          for (int c = 0; c < p.nchunk; ++c)
            tma_load_2d(dst + a_off + c * abox, &p.tm_a, full, e * ca * p.k,
                        w.slot * p.v + w.panel * p.panel_cols + c * p.chunk_cols);
          issued_mask |= 1u << stage;
          phase_mask = (phase_mask & ~(1u << stage)) | (phase << stage);
          if (++stage == static_cast<uint32_t>(p.corr_stages)) { stage = 0; phase ^= 1u; }
        }
      }
      lowrank_drain_ring(lc->cfull, p.corr_stages, issued_mask, phase_mask);
    }
    __syncwarp();
  } else if (warp >= 3 && warp < 3 + p.groups) {
    // ------------------------------------------------------------------ MMA issuer of the corrections of one epilogue
    // group: its components in turn, chunk c of the group's u-th chunk overall into slot 2 g + (u & 1)
    if (lane == 0) {
      const int g = warp - 3;
      uint32_t stage = 0, phase = 0, cuse = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
        const LowRankItem w = lowrank_item(p, item);
        for (int e = 0; e < nent && ok; ++e) {
          if (!bounded_wait(smem_u32(&lc->cfull[stage]), phase, ctl, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t entry = corr_ring + stage * p.corr_stage_bytes;
          for (int l = 0; l < ca && ok; ++l) {
            const int j = e * ca + l;
            if (j >= p.r) break;
            if (j % p.groups != g) continue;
            // descriptors step in 16-byte units: the component's [hi | lo] inside its z box, its k columns inside the A' box
            const uint64_t z_desc = umma_smem_desc_sw128(entry + (l / cz) * zbox) + ((l % cz) * 2 * p.k) / 8;
            for (int c = 0; c < w.nchunk; ++c, ++cuse) {
              const int width = min(p.chunk_cols, w.width - c * p.chunk_cols);
              const uint32_t idesc = umma_idesc_bf16(kBlockM, width);
              const uint64_t a_desc = umma_smem_desc_sw128(entry + a_off + c * abox) + (l * p.k) / 8;
              const uint32_t slot = 2 * g + (cuse & 1u);
              if (!bounded_wait(smem_u32(&ctl->tempty[slot]), ((cuse >> 1) & 1u) ^ 1u, ctl, p.status)) { ok = false; break; }
              tc_fence_after();
              const uint32_t d_tmem = tmem_base + p.corr_col0 + slot * p.chunk_cols;
              uint32_t acc = 0;
              for (int part = 0; part < 2; ++part)
                for (int q = 0; q < kq; ++q) {
                  umma_bf16(d_tmem, z_desc + (part * p.k + 16 * q) / 8, a_desc + (16 * q) / 8, idesc, acc);
                  acc = 1;
                }
              umma_commit(smem_u32(&ctl->tfull[slot]));
            }
          }
          if (!ok) break;
          umma_commit(smem_u32(&lc->cempty[stage]));           // (also for an entry none of whose components are this group's)
          if (++stage == static_cast<uint32_t>(p.corr_stages)) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok || ctl->abort) {
        umma_commit(smem_u32(&lc->drain2[g]));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&lc->drain2[g]), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
    __syncwarp();
  } else if (warp >= kLrRoleThreads / 32) {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;
    const int group = (warp - kLrRoleThreads / 32) >> 2;      // this warp's epilogue group: components group, group + groups, ...
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    const size_t entries = static_cast<size_t>(p.T) * p.n * p.r;
    uint32_t it = 0, cuse = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++it) {
      const LowRankItem w = lowrank_item(p, item);
      const int row = w.mt * kBlockM + quarter * 32 + lane;
      const bool valid = row < p.T;
      const int tgt = valid ? p.targets[static_cast<size_t>(row) * p.n + w.slot] : -1;
      const int panel_col0 = w.panel * p.panel_cols;
      const uint32_t buf = it & 1u;
      if (!bounded_wait_warp(smem_u32(&lc->afull[buf]), (it >> 1) & 1u, ctl, p.status, lane)) { ok = false; break; }
      tc_fence_after();
      const uint32_t bcol = lane_base + buf * p.acc_stride;
      for (int j = group; j < p.r && ok; j += p.groups) {
        float m = -CUDART_INF_F, s = 0.f, tval = 0.f;
        for (int c = 0; c < w.nchunk; ++c, ++cuse) {
          const uint32_t slot = 2 * group + (cuse & 1u);
          if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (cuse >> 1) & 1u, ctl, p.status, lane)) { ok = false; break; }
          tc_fence_after();
          const int col_chunk = c * p.chunk_cols;             // first column of the chunk inside the panel
          const int width = min(p.chunk_cols, w.width - col_chunk);
          const uint32_t ccol = lane_base + p.corr_col0 + slot * p.chunk_cols;
          // one batch of 16 columns: correction + base, then the dense kernel's online log-sum-exp and target gather
          auto consume = [&](const uint32_t (&rc)[16], const uint32_t (&rb)[16], int b) {
            float x[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = __uint_as_float(rc[q]) + __uint_as_float(rb[q]);
            const int col0 = panel_col0 + col_chunk + b * 16; // column inside the unit
            mask_padding(x, col0, p.vv);
            if (p.logit_out != nullptr && valid) {            // row of the logit matrix: (slot, component, symbol)
              float* l = p.logit_out + static_cast<size_t>(row) * p.logit_pitch + (static_cast<size_t>(w.slot) * p.r + j) * p.v + col0;
              st_global_v8(l, x);
              st_global_v8(l + 8, x + 8);
            }
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
          tmem_ld16_issue(bcol + col_chunk, b0);
          tmem_ld_wait16(c0);
          tmem_ld_wait16(b0);
          for (int b = 0; b < nb; b += 2) {
            if (b + 1 < nb) {
              tmem_ld16_issue(ccol + (b + 1) * 16, c1);
              tmem_ld16_issue(bcol + col_chunk + (b + 1) * 16, b1);
            }
            consume(c0, b0, b);
            if (b + 1 >= nb) break;
            tmem_ld_wait16(c1);
            tmem_ld_wait16(b1);
            if (b + 2 < nb) {
              tmem_ld16_issue(ccol + (b + 2) * 16, c0);
              tmem_ld16_issue(bcol + col_chunk + (b + 2) * 16, b0);
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
          const size_t e = (static_cast<size_t>(row) * p.n + w.slot) * p.r + j;
          if (p.panels == 1) {
            if (p.lse_out != nullptr) p.lse_out[e] = m + fast_lg2(s) * kLn2;
            if (tgt < 0) {
              p.G[e] = p.missing_is_nan ? CUDART_NAN_F : 0.f;   // marginalised byte: the input unit sums to 1
            } else if (tgt >= p.vv) {
              p.G[e] = CUDART_NAN_F;
              atomicOr(p.status, kStatusBadTarget);
            } else {
              p.G[e] = tval - (m + fast_lg2(s) * kLn2);
            }
          } else {
            // (padding is less than 16 columns and a panel at least 16 wide: every panel has existing symbols)
            p.partial[static_cast<size_t>(w.panel) * entries + e] = make_float2(m, s);
            if (static_cast<unsigned>(tgt - panel_col0) < static_cast<unsigned>(w.width)) p.target_logit[e] = tval;
          }
        }
      }
      if (!ok) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&lc->aempty[buf]));   // the base of the item after next may overwrite the buffer
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// G[t, i, j] = logit[target] - LSE over the unit, from the per-panel (maximum, sum of exponentials) the factored projection
// left: one thread per (position, slot, component). Targets < 0 (marginalised): 0; targets >= vv: NaN and the status bit.
__global__ void lowrank_merge_kernel(const float2* __restrict__ partial, const float* __restrict__ target_logit,
                                     const int* __restrict__ targets, float* __restrict__ G, float* __restrict__ lse_out,
                                     unsigned* status, size_t entries, int r, int vv, int panels, int missing_is_nan) {
  const size_t e = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= entries) return;
  float m = -CUDART_INF_F, s = 0.f;
  for (int q = 0; q < panels; ++q) {
    const float2 ms = partial[static_cast<size_t>(q) * entries + e];
    lse_merge(m, s, ms.x, ms.y);
  }
  const float lse = m + __logf(s);
  if (lse_out != nullptr) lse_out[e] = lse;
  const int tgt = targets[e / r];
  if (tgt < 0) { G[e] = missing_is_nan ? CUDART_NAN_F : 0.f; return; }
  if (tgt >= vv) {
    G[e] = CUDART_NAN_F;
    atomicOr(status, kStatusBadTarget);
    return;
  }
  G[e] = target_logit[e] - lse;
}

// A [n, r, v, k] -> A' [n, v, r, k] (bf16, k a multiple of 8): one 16-byte piece per thread.
__global__ void lowrank_repack_kernel(const uint4* __restrict__ A, uint4* __restrict__ out, int n, int r, int v, int kv) {
  const size_t total = static_cast<size_t>(n) * r * v * kv;      // kv = k / 8 pieces per row
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int q = static_cast<int>(idx % kv);
  size_t rest = idx / kv;
  const int j = static_cast<int>(rest % r);
  rest /= r;
  const int b = static_cast<int>(rest % v);
  const int i = static_cast<int>(rest / v);
  out[idx] = A[((static_cast<size_t>(i) * r + j) * v + b) * kv + q];
}

// Few-position draft on a factored head: logits[p, i, j, b] = base[p, i, b] + sum_q A[i, j, b, q] z[p, i, j, q], from the
// two small products the weight pass left (base = W_base h [P, n v], z = B h [P, n r k], fp32). One CTA per (unit,
// 256 symbols): a thread keeps its symbol's adaptor row in registers and walks the positions, whose z rows sit in shared
// memory. Launched as a programmatic dependent of the weight pass.
constexpr int kExpandThreads = 256;
__global__ void __launch_bounds__(kExpandThreads) lowrank_expand_kernel(const float* __restrict__ base,
                                                                        const float* __restrict__ z,
                                                                        const __nv_bfloat16* __restrict__ A,
                                                                        float* __restrict__ logits, int P, int n, int r,
                                                                        int v, int k) {
  extern __shared__ float zs[];                                 // [P, k]
  grid_launch_dependents();
  grid_dependency_wait();
  const int unit = blockIdx.x, i = unit / r;
  const int b = blockIdx.y * kExpandThreads + threadIdx.x;
  const size_t units = static_cast<size_t>(n) * r;
  for (int e = threadIdx.x; e < P * k; e += kExpandThreads) zs[e] = z[(static_cast<size_t>(e / k) * units + unit) * k + e % k];
  __syncthreads();
  if (b >= v) return;
  float a[kLrMaxRank];
  const uint4* arow = reinterpret_cast<const uint4*>(A + (static_cast<size_t>(unit) * v + b) * k);   // k bf16 = k / 8 pieces
#pragma unroll
  for (int q = 0; q < kLrMaxRank / 8; ++q) {
    if (q * 8 < k) {
      const uint4 piece = arow[q];
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&piece);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float2 f = __bfloat1622float2(h2[t]);
        a[q * 8 + 2 * t] = f.x;
        a[q * 8 + 2 * t + 1] = f.y;
      }
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) a[q * 8 + t] = 0.f;
    }
  }
  for (int pos = 0; pos < P; ++pos) {
    float acc = base[(static_cast<size_t>(pos) * n + i) * v + b];
    const float* zp = zs + pos * k;
#pragma unroll
    for (int q = 0; q < kLrMaxRank; ++q)
      if (q < k) acc = fmaf(a[q], zp[q], acc);
    logits[(static_cast<size_t>(pos) * units + unit) * v + b] = acc;
  }
}

// Backward pass of a factored head (App. G): with g = d loss / d logit [T, n r v] (bf16), the gradients are
//   dW_base[i] = (sum_j g_ij)^T h,   dA_ij = g_ij^T (B_ij h),   dB_ij = (g_ij A_ij)^T h,
//   d hidden   = (sum_j g_ij) W_base[i] + (g_ij A_ij) B_ij  summed over the slots and components.
// lowrank_component_sum_kernel: S[t, i, b] = sum_j g[t, i, j, b], written as bf16 into a matrix of pitch out_pitch (where
// it is the A operand of the GEMMs that follow). Eight symbols per thread, 16-byte loads and stores.
__global__ void __launch_bounds__(256) lowrank_component_sum_kernel(const __nv_bfloat16* __restrict__ g, size_t g_pitch,
                                                                    __nv_bfloat16* __restrict__ out, size_t out_pitch, int T,
                                                                    int n, int r, int v) {
  const int per_row = n * v / 8;                                 // 16-byte pieces of one row of S
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(T) * per_row) return;
  const int t = static_cast<int>(idx / per_row), c = static_cast<int>(idx % per_row) * 8;
  const int i = c / v, b = c - i * v;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  const __nv_bfloat16* src = g + static_cast<size_t>(t) * g_pitch + static_cast<size_t>(i) * r * v + b;
  for (int j = 0; j < r; ++j) {
    const uint4 piece = *reinterpret_cast<const uint4*>(src + static_cast<size_t>(j) * v);
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&piece);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 f = __bfloat1622float2(h2[q]);
      acc[2 * q] += f.x;
      acc[2 * q + 1] += f.y;
    }
  }
  __align__(16) __nv_bfloat16 o[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) o[q] = __float2bfloat16_rn(acc[q]);
  *reinterpret_cast<uint4*>(out + static_cast<size_t>(t) * out_pitch + c) = *reinterpret_cast<const uint4*>(o);
}

// A [n r, v, k] -> [n r, v64, k] with v64 = v rounded up to 64 and zero rows past v: the batched GEMM g_ij A_ij walks K in
// blocks of 64 symbols, and what it reads of g past a unit's own columns must meet zeros.
__global__ void lowrank_pad_kernel(const uint4* __restrict__ A, uint4* __restrict__ out, int units, int v, int v64, int kv) {
  const size_t total = static_cast<size_t>(units) * v64 * kv;    // kv = k / 8 pieces per row
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int q = static_cast<int>(idx % kv);
  const size_t rest = idx / kv;
  const int b = static_cast<int>(rest % v64);
  const size_t u = rest / v64;
  out[idx] = b < v ? A[(u * v + b) * kv + q] : make_uint4(0u, 0u, 0u, 0u);
}

// Byte draws of a long draft on a factored head (Algorithm 1, input-unit step): one warp per (window, slot) forms the v
// logits of the one unit the window's latent draw selected, base[t, i, :] + A[i, z] (B[i, z] h_t), in shared memory and draws
// the byte by inverse CDF on exp(logit - max) - v k multiply-adds per draw, no tensor cores and no pass over the other
// units. base = W_base h [P, n v] fp32 and z = B h (two bf16 halves [P, n r, 2, k]) come from two plain GEMMs.
// v <= 512. A refused latent draw (unit_sel < 0) or byte uniform leaves the byte at -1 (preset by the latent kernel).
constexpr int kDrawWarps = 8;
__global__ void __launch_bounds__(32 * kDrawWarps) lowrank_draw_kernel(
    const float* __restrict__ base, const __nv_bfloat16* __restrict__ zhl, const __nv_bfloat16* __restrict__ A,
    const int* __restrict__ unit_sel, const float* __restrict__ uniforms, int* __restrict__ out_bytes, unsigned* status, int W,
    int wpp, int n, int r, int v, int vv, int k) {
  extern __shared__ float draw_sm[];                              // kDrawWarps x v logits
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* x = draw_sm + warp * v;
  const size_t units = static_cast<size_t>(n) * r;
  const int pairs = W * n;
  const int per = (v + 31) / 32;
  for (int e = blockIdx.x * kDrawWarps + warp; e < pairs; e += gridDim.x * kDrawWarps) {
    const int w = e / n, i = e - w * n;
    const int z = unit_sel[e];
    if (z < 0) continue;                                          // warp-uniform
    const float ub = uniforms[static_cast<size_t>(w) * 2 * n + n + i];
    if (!(ub >= 0.f && ub < 1.f)) {
      if (lane == 0) atomicOr(status, 2u);
      continue;
    }
    const size_t t = static_cast<size_t>(w / wpp);
    const size_t unit = static_cast<size_t>(i) * r + z;
    const __nv_bfloat16* zrow = zhl + (t * units + unit) * 2 * k;
    const float zmine = lane < k ? __bfloat162float(zrow[lane]) + __bfloat162float(zrow[k + lane]) : 0.f;
    float zq[kLrMaxRank];
#pragma unroll
    for (int q = 0; q < kLrMaxRank; ++q) zq[q] = __shfl_sync(0xffffffffu, zmine, q);
    const float* brow = base + (t * n + i) * v;
    float m = -CUDART_INF_F;
    for (int b = lane; b < v; b += 32) {
      float acc = brow[b];
      const uint4* arow = reinterpret_cast<const uint4*>(A + (unit * v + b) * k);
#pragma unroll
      for (int q8 = 0; q8 < kLrMaxRank / 8; ++q8) {
        if (q8 * 8 < k) {
          const uint4 piece = arow[q8];
          const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&piece);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float2 f = __bfloat1622float2(h2[u]);
            acc = fmaf(f.x, zq[q8 * 8 + 2 * u], acc);
            acc = fmaf(f.y, zq[q8 * 8 + 2 * u + 1], acc);
          }
        }
      }
      if (b >= vv) acc = -CUDART_INF_F;                           // [vv, v): padding symbols
      x[b] = acc;
      m = fmaxf(m, acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    __syncwarp();
    const int byte = warp_inv_cdf_chunk<kSlotMaxPerLane>(x, 0, per, vv, m, ub, true, lane);
    if (lane == 0) out_bytes[e] = byte;
    __syncwarp();                                                 // x is reused by the warp's next pair
  }
}

// Acceptance stage after a long draft on a factored head (Algorithm 3): for every window whose draft was rejected at byte s
// (first_rejected[w] = s >= 0) the r v logits of slot s and the r log-sum-exps, which no call kept:
// logits[w, j, :] = base[t, s, :] + A[s, j] (B[s, j] h_t). One warp per (window, component); rows of the outputs are the
// windows themselves (row_of[w] = w). Padding symbols get -inf, as in the projection kernels.
__global__ void __launch_bounds__(32 * kDrawWarps) lowrank_slot_logits_kernel(
    const float* __restrict__ base, const __nv_bfloat16* __restrict__ zhl, const __nv_bfloat16* __restrict__ A,
    const int* __restrict__ first_rejected, float* __restrict__ logits, float* __restrict__ unit_lse, int* __restrict__ row_of,
    int W, int w_first, int wpp, int n, int r, int v, int vv, int k) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t units = static_cast<size_t>(n) * r;
  const int pairs = W * r;
  for (int e = blockIdx.x * kDrawWarps + warp; e < pairs; e += gridDim.x * kDrawWarps) {
    const int w = e / r, j = e - w * r;
    if (j == 0 && lane == 0) row_of[w] = w;
    const int s = first_rejected[w];
    if (s < 0) continue;                                          // warp-uniform: everything accepted, no residual draw
    const size_t t = static_cast<size_t>((w_first + w) / wpp);
    const size_t unit = static_cast<size_t>(s) * r + j;
    const __nv_bfloat16* zrow = zhl + (t * units + unit) * 2 * k;
    const float zmine = lane < k ? __bfloat162float(zrow[lane]) + __bfloat162float(zrow[k + lane]) : 0.f;
    float zq[kLrMaxRank];
#pragma unroll
    for (int q = 0; q < kLrMaxRank; ++q) zq[q] = __shfl_sync(0xffffffffu, zmine, q);
    const float* brow = base + (t * n + s) * v;
    float* out = logits + (static_cast<size_t>(w) * r + j) * v;
    float m = -CUDART_INF_F, sum = 0.f;
    for (int b = lane; b < v; b += 32) {
      float acc = brow[b];
      const uint4* arow = reinterpret_cast<const uint4*>(A + (unit * v + b) * k);
#pragma unroll
      for (int q8 = 0; q8 < kLrMaxRank / 8; ++q8) {
        if (q8 * 8 < k) {
          const uint4 piece = arow[q8];
          const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&piece);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float2 f = __bfloat1622float2(h2[u]);
            acc = fmaf(f.x, zq[q8 * 8 + 2 * u], acc);
            acc = fmaf(f.y, zq[q8 * 8 + 2 * u + 1], acc);
          }
        }
      }
      if (b >= vv) acc = -CUDART_INF_F;
      out[b] = acc;
      lse_merge(m, sum, acc, 1.f);                                // running (maximum, sum of exponentials) of this lane's symbols
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
      const float s2 = __shfl_xor_sync(0xffffffffu, sum, off);
      lse_merge(m, sum, m2, s2);
    }
    if (lane == 0) unit_lse[static_cast<size_t>(w) * r + j] = m + __logf(sum);
  }
}

}  // namespace mtpc