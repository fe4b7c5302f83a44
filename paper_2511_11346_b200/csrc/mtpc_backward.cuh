// Backward pass of the window log-likelihood (training, Sec. 4.1 / Eq. 6): gradient of
//     L = sum_t weight[t] * log q(x_t | h_t)
// with respect to the hidden states, the emission weights, the sum-unit weights and the static transition logits.
//
// Stages (host side in mtpc_api.cu):
//   1. forward projection kernel, also keeping the emission logits ([T, n r v] fp32, streamed out of the epilogue) and
//      the log-sum-exp of every input unit (lse [T, n, r]);
//   2. circuit backward (this file): one warp per window runs the upward and the downward pass of the circuit and
//      writes post[w, i, k] = weight * d log q / d G[w, i, k] (the posterior of "token i is emitted by unit k") and
//      dsum[w, :] = weight * d log q / d (sum-unit logits), i.e. posterior minus prior of every sum unit, in bf16;
//   3. logit_gradient_kernel (this file): dlogit = post * (onehot(target) - exp(logit - lse)), one streaming pass over
//      the kept logits, written once as bf16 rows;
//   4. plain bf16 GEMMs (plain_gemm_kernel, this file) on those, every operand read where it lies (the tensor cores
//      take either orientation): d hidden = dlogit W + dsum R, dW = dlogit^T h, dR = dsum^T h.
// Only the training calls materialise the logits (fp32, and their bf16 gradient, as the operands of the two weight-sized
// GEMMs); recomputing them on chip instead was measured: a fourth weight-sized contraction against 0.6 ms of streaming.
#pragma once
#include <cuda_bf16.h>

#include "mtpc_circuit.cuh"
#include "mtpc_gemm.cuh"

namespace mtpc {

// Arguments the three circuit backward kernels share beyond the forward ones:
//   weight, weight_stride   window w is weighted by weight[w * weight_stride]
//   len                     only the first `len` slots carry evidence, the later bytes are summed out: the kernels then
//                           differentiate the prefix marginal log q(x_0..x_{len-1}) (len = n: the joint)
//   accumulate              0: post and dsum are overwritten (dsum as bf16). 1: results are ADDED to post and to the fp32
//                           buffer dsum_f32 (several passes with different len and weights, Eq. 6); only slots < len are
//                           touched, the buffers must have been zeroed before the first pass.
//   dsum_pitch              row pitch, in elements, of whichever of dsum / dsum_f32 is written
struct CircuitBackwardArgs {
  const float* G;
  const float* logw;
  const int* targets;
  const float* weight;
  int weight_stride;
  float* out;                 // [W] log q of the (prefix) window, or NULL
  float* post;                // [W, n, r]
  __nv_bfloat16* dsum;        // [W, dsum_pitch] (accumulate == 0)
  float* dsum_f32;            // [W, dsum_pitch] (accumulate == 1)
  int dsum_pitch;
  int len, accumulate;
  int W, n, r, sum_rows;
};
// Accumulating passes add by reduction instructions (no value returned, so no wait for the round trip): every address
// is only ever touched by one lane, in program order, so the sums keep their order and stay reproducible.
__device__ __forceinline__ void put_post(const CircuitBackwardArgs& a, size_t idx, float v) {
  if (a.accumulate) atomicAdd(a.post + idx, v);
  else a.post[idx] = v;
}
__device__ __forceinline__ void put_dsum(const CircuitBackwardArgs& a, size_t idx, float v) {
  if (a.accumulate) atomicAdd(a.dsum_f32 + idx, v);
  else a.dsum[idx] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------- circuit backward: mixture (Eq. CP)
// log q = LSE_k a_k, a_k = log omega_k + sum_i G[i, k]:  d log q / d a_k = rho_k = softmax(a)_k for every slot and for
// the mixture weight; through the softmax of the mixture logits: rho_k - omega_k.
__global__ void circuit_cp_backward_kernel(const CircuitBackwardArgs a_) {
  const int w = blockIdx.x * kCircuitWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= a_.W) return;
  const int n = a_.n, r = a_.r, len = a_.len;
  const float* g = a_.G + static_cast<size_t>(w) * n * r;
  const float* lw = a_.logw + static_cast<size_t>(w) * a_.sum_rows;
  const float wt = a_.weight[static_cast<size_t>(w) * a_.weight_stride];
  float a[4];
  float m = -CUDART_INF_F, s = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int k = lane + 32 * q;
    a[q] = -CUDART_INF_F;
    if (k < r) {
      a[q] = lw[k];
      for (int i = 0; i < len; ++i) a[q] += g[i * r + k];
      lse_merge(m, s, a[q], 1.f);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(kFull, m, off);
    const float s2 = __shfl_xor_sync(kFull, s, off);
    lse_merge(m, s, m2, s2);
  }
  const float logq = m + __logf(s);
  if (lane == 0 && a_.out != nullptr) a_.out[w] = logq;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int k = lane + 32 * q;
    if (k < r) {
      const float rho = __expf(a[q] - logq);
      for (int i = 0; i < len; ++i)
        put_post(a_, (static_cast<size_t>(w) * n + i) * r + k, a_.targets[static_cast<size_t>(w) * n + i] >= 0 ? wt * rho : 0.f);
      for (int i = len; i < n && !a_.accumulate; ++i) a_.post[(static_cast<size_t>(w) * n + i) * r + k] = 0.f;
      put_dsum(a_, static_cast<size_t>(w) * a_.dsum_pitch + k, wt * (rho - __expf(lw[k])));
    }
  }
}

// ---------------------------------------------------------------- gradient of one row of a transition table
// Lane = row (the conditioning value). For every column b: out[b] = wt * (exp(base + row[b] + pc[b]) - exp(row[b]) * gam),
// i.e. pairwise posterior minus conditional probability times the posterior of the conditioning value (the gradient
// with respect to the row's logits). `row` and `pc` are in shared memory; the results go either to a bf16 row in global
// memory (contextual tables: one set per position), or by atomic adds to an fp32 row in shared memory (static tables,
// summed over the windows), or added to an fp32 row in global memory (several passes accumulating, Eq. 6). R a multiple of 4: float4 reads rotated by the lane (conflict-free), 8-byte stores.
template <int R>
__device__ __forceinline__ void row_grad_vec(const float* row, const float* pc, float base, float gam, float wt, int lane,
                                             __nv_bfloat16* dst, float* acc_row, float* f32_row) {
  constexpr int Q = R / 4;
  const float4* row4 = reinterpret_cast<const float4*>(row);
  const float4* pc4 = reinterpret_cast<const float4*>(pc);
#pragma unroll
  for (int q = 0; q < Q; ++q) {
    const int j = (q + lane) & (Q - 1);
    const float4 a = row4[j];
    const float4 p = pc4[j];
    const float ox = wt * (__expf(base + a.x + p.x) - __expf(a.x) * gam);
    const float oy = wt * (__expf(base + a.y + p.y) - __expf(a.y) * gam);
    const float oz = wt * (__expf(base + a.z + p.z) - __expf(a.z) * gam);
    const float ow = wt * (__expf(base + a.w + p.w) - __expf(a.w) * gam);
    if (acc_row != nullptr) {
      atomicAdd(acc_row + 4 * j, ox);
      atomicAdd(acc_row + 4 * j + 1, oy);
      atomicAdd(acc_row + 4 * j + 2, oz);
      atomicAdd(acc_row + 4 * j + 3, ow);
    } else if (f32_row != nullptr) {
      // this lane owns the row, so the additions to one address keep their order; issued as a reduction (no value comes
      // back), the warp does not wait for the round trip to L2 that a read-add-write would cost
      atomicAdd(reinterpret_cast<float4*>(f32_row + 4 * j), make_float4(ox, oy, oz, ow));
    } else {
      __nv_bfloat162 lo = __floats2bfloat162_rn(ox, oy);
      __nv_bfloat162 hi = __floats2bfloat162_rn(oz, ow);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(dst + 4 * j) = pk;
    }
  }
}
__device__ __forceinline__ void row_grad(const float* row, const float* pc, float base, float gam, float wt, int lane, int r,
                                         __nv_bfloat16* dst, float* acc_row, float* f32_row) {
  switch (r) {
    case 32: row_grad_vec<32>(row, pc, base, gam, wt, lane, dst, acc_row, f32_row); return;
    case 16: row_grad_vec<16>(row, pc, base, gam, wt, lane, dst, acc_row, f32_row); return;
    case 8: row_grad_vec<8>(row, pc, base, gam, wt, lane, dst, acc_row, f32_row); return;
    case 4: row_grad_vec<4>(row, pc, base, gam, wt, lane, dst, acc_row, f32_row); return;
    default: break;
  }
  for (int q = 0; q < r; ++q) {                       // start at column `lane` (r a power of two): conflict-free
    const int b = (q + lane) & (r - 1);
    const float la = row[b];
    const float o = wt * (__expf(base + la + pc[b]) - __expf(la) * gam);
    if (acc_row != nullptr) atomicAdd(acc_row + b, o);
    else if (f32_row != nullptr) atomicAdd(f32_row + b, o);
    else dst[b] = __float2bfloat16_rn(o);
  }
}

// ---------------------------------------------------------------- circuit backward: HMM (Eq. HMM), forward-backward
// Forward messages alpha_i (kept for all steps in shared memory), backward messages
// beta_{i-1}[a] = LSE_b(logA_i[a][b] + G[i][b] + beta_i[b]). Posterior of the state: gamma_i = exp(alpha_i + beta_i - log q)
// = d log q / d G[i, .]; pairwise posterior xi_i[a][b] = exp(alpha_{i-1}[a] + logA_i[a][b] + G[i][b] + beta_i[b] - log q)
// = d log q / d logA_i[a][b]; through the row softmax of the transition logits: xi_i[a][b] - A_i[a][b] gamma_{i-1}[a].
// Tables as in circuit_hmm_stream_kernel (static: stride 0; contextual: one set per position inside log omega).
// Contextual: the transition-logit gradients go to dsum (bf16, one row per position). Static: they are summed over
// the windows into dT [n-1, r, r] (fp32): per CTA in shared memory first, then one atomicAdd per entry and CTA.
// Shared memory: per warp n*r (alpha) + 2*r*r (tables) + 64 floats; static: + (n-1)*r*r floats per CTA.  r <= 32.
__host__ __device__ inline size_t hmm_backward_warp_floats(int n, int r) {
  return static_cast<size_t>(n) * r + 2 * r * r + 64;             // alphas, two tables, two vectors of 32
}
__host__ __device__ inline size_t hmm_backward_smem_floats(int n, int r, bool is_static, int warps) {
  return static_cast<size_t>(warps) * hmm_backward_warp_floats(n, r) + (is_static ? static_cast<size_t>(n - 1) * r * r : 0);
}

__global__ void circuit_hmm_backward_kernel(const CircuitBackwardArgs a_, const float* __restrict__ tables,
                                            int table_stride, float* __restrict__ dT, unsigned* work_counter) {
  extern __shared__ __align__(16) float sm[];
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  const int n = a_.n, r = a_.r, len = a_.len;
  const int rr = r * r;
  const bool is_static = table_stride == 0;
  float* acc = sm;                                                       // static only: [n-1, r, r]
  float* mine = sm + (is_static ? (n - 1) * rr : 0) + static_cast<size_t>(wib) * hmm_backward_warp_floats(n, r);
  float* alphas = mine;                                                  // [n, r]
  float* tabs = alphas + n * r;
  float* cvec = tabs + 2 * rr;
  const bool has = lane < r;
  if (is_static) {
    for (int e = threadIdx.x; e < (n - 1) * rr; e += blockDim.x) acc[e] = 0.f;
    __syncthreads();
  }
  // The steps after `len` carry no evidence and the transitions are normalised: the recursion stops at step len - 1.
  for (int w = next_window(work_counter, lane); w < a_.W; w = next_window(work_counter, lane)) {
    const float* g = a_.G + static_cast<size_t>(w) * n * r;
    const float* lw = a_.logw + static_cast<size_t>(w) * a_.sum_rows;
    const float* tb = tables + static_cast<size_t>(w) * table_stride;
    const float wt = a_.weight[static_cast<size_t>(w) * a_.weight_stride];
    const size_t prow = static_cast<size_t>(w) * n * r;
    const size_t drow = static_cast<size_t>(w) * a_.dsum_pitch;
    // ---- forward, keeping every alpha_i
    if (len > 1) warp_table_load_async(tabs, tb, rr, lane);
    float alpha = has ? lw[lane] + g[lane] : -CUDART_INF_F;
    if (has) alphas[lane] = alpha;
    for (int i = 1; i < len; ++i) {
      if (i + 1 < len) {
        warp_table_load_async(tabs + (i & 1) * rr, tb + static_cast<size_t>(i) * rr, rr, lane);
        cp_async_wait<1>();
      } else {
        cp_async_wait<0>();
      }
      __syncwarp();
      const float* A = tabs + ((i - 1) & 1) * rr;
      float m = alpha;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, off));
      cvec[lane] = has ? __expf(alpha - m) : 0.f;
      __syncwarp();
      if (has) {
        const float s = hmm_matvec(cvec, A, lane, r);
        alpha = (m == -CUDART_INF_F) ? -CUDART_INF_F : g[i * r + lane] + m + __logf(s);
        alphas[i * r + lane] = alpha;
      }
      __syncwarp();
    }
    const float logq = warp_lse(alpha, has);
    if (lane == 0 && a_.out != nullptr) a_.out[w] = logq;
    // ---- backward: tables in reverse order; the table of step len - 1 is still in its buffer
    float beta = 0.f;                                                    // beta_{len-1}
    for (int i = len - 1; i >= 1; --i) {
      if (i < len - 1) {
        cp_async_wait<0>();
        __syncwarp();
      }
      if (i - 1 >= 1) warp_table_load_async(tabs + (i & 1) * rr, tb + static_cast<size_t>(i - 2) * rr, rr, lane);
      const float* A = tabs + ((i - 1) & 1) * rr;
      const bool valid = a_.targets[static_cast<size_t>(w) * n + i] >= 0;
      if (has) {
        const float gamma = __expf(alphas[i * r + lane] + beta - logq);
        put_post(a_, prow + static_cast<size_t>(i) * r + lane, valid ? wt * gamma : 0.f);
        cvec[lane] = g[i * r + lane] + beta;
      }
      __syncwarp();
      const float beta_prev = sum_layer_staged(A, cvec, lane, r);        // lane a: LSE_b(logA[a][b] + c[b])
      if (has) {
        const float al = alphas[(i - 1) * r + lane];
        const float gam_prev = __expf(al + beta_prev - logq);
        const size_t off = static_cast<size_t>(r) + static_cast<size_t>(i - 1) * rr + lane * r;
        row_grad(A + lane * r, cvec, al - logq, gam_prev, wt, lane, r,
                 (is_static || a_.accumulate) ? nullptr : a_.dsum + drow + off,
                 is_static ? acc + static_cast<size_t>(i - 1) * rr + lane * r : nullptr,
                 (!is_static && a_.accumulate) ? a_.dsum_f32 + drow + off : nullptr);
      }
      beta = beta_prev;
      __syncwarp();                                                      // cvec and the table buffer are free again
    }
    if (has) {
      const float gamma0 = __expf(alphas[lane] + beta - logq);
      put_post(a_, prow + lane, a_.targets[static_cast<size_t>(w) * n] >= 0 ? wt * gamma0 : 0.f);
      put_dsum(a_, drow + lane, wt * (gamma0 - __expf(lw[lane])));
      if (!a_.accumulate) {                                              // slots and tables past the prefix: no gradient
        for (int i = len; i < n; ++i) a_.post[prow + static_cast<size_t>(i) * r + lane] = 0.f;
        if (!is_static)
          for (int e = (len - 1) * rr + lane; e < (n - 1) * rr; e += r) a_.dsum[drow + r + e] = __float2bfloat16_rn(0.f);
      }
    }
    __syncwarp();
  }
  if (is_static) {
    __syncthreads();
    for (int e = threadIdx.x; e < (n - 1) * rr; e += blockDim.x) {
      const float v = acc[e];
      if (v != 0.f) atomicAdd(dT + e, v);
    }
  }
}

// ---------------------------------------------------------------- Eq. 6 through the HMM in one pass
// The training loss is linear in the prefix log-marginals, L = sum_j coeff[w, j] log p_j, and for the HMM
// p_j = sum_z exp(alpha_j[z]) is the forward message of step j summed over the state (later steps integrate to one). One
// forward recursion therefore gives every prefix, and one reverse sweep gives the whole gradient: with
// abar_i[z] = dL / d alpha_i[z] (plain numbers of either sign, bounded by sum_j |coeff_j|),
//   abar_{n-1} = coeff_{n-1} softmax(alpha_{n-1}),
//   prop_{i-1}[a] = sum_b exp(alpha_{i-1}[a] + logA_i[a][b] + G[i][b] - alpha_i[b]) abar_i[b]     (a conditional probability
//   abar_{i-1}[a] = coeff_{i-1} softmax(alpha_{i-1})[a] + prop_{i-1}[a]                             times abar_i[b])
// and dL/dG[i] = abar_i, dL/d logA_i[a][b] = the summand of prop_{i-1}[a]; through the row softmax of the transition
// logits: summand - A_i[a][b] prop_{i-1}[a]; initial unit: abar_0 - omega sum_z abar_0[z]. Same streaming of the tables
// and the same outputs as circuit_hmm_backward_kernel with accumulate == 0 (post fp32, dsum bf16, static dT by atomics).
template <int R>
__device__ __forceinline__ void row_grad_mult_vec(const float* row, const float* pc, const float* mult, float base, float gam,
                                                  int lane, __nv_bfloat16* dst, float* acc_row) {
  constexpr int Q = R / 4;
  const float4* row4 = reinterpret_cast<const float4*>(row);
  const float4* pc4 = reinterpret_cast<const float4*>(pc);
  const float4* mu4 = reinterpret_cast<const float4*>(mult);
#pragma unroll
  for (int q = 0; q < Q; ++q) {
    const int j = (q + lane) & (Q - 1);
    const float4 a = row4[j];
    const float4 p = pc4[j];
    const float4 mu = mu4[j];
    const float ox = __expf(base + a.x + p.x) * mu.x - __expf(a.x) * gam;
    const float oy = __expf(base + a.y + p.y) * mu.y - __expf(a.y) * gam;
    const float oz = __expf(base + a.z + p.z) * mu.z - __expf(a.z) * gam;
    const float ow = __expf(base + a.w + p.w) * mu.w - __expf(a.w) * gam;
    if (acc_row != nullptr) {
      atomicAdd(acc_row + 4 * j, ox);
      atomicAdd(acc_row + 4 * j + 1, oy);
      atomicAdd(acc_row + 4 * j + 2, oz);
      atomicAdd(acc_row + 4 * j + 3, ow);
    } else {
      __nv_bfloat162 lo = __floats2bfloat162_rn(ox, oy);
      __nv_bfloat162 hi = __floats2bfloat162_rn(oz, ow);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(dst + 4 * j) = pk;
    }
  }
}
// Lane = row a of the table: out[b] = exp(base + row[b] + pc[b]) mult[b] - exp(row[b]) gam, to a bf16 row in global memory
// or by atomic adds to an fp32 row in shared memory.
__device__ __forceinline__ void row_grad_mult(const float* row, const float* pc, const float* mult, float base, float gam,
                                              int lane, int r, __nv_bfloat16* dst, float* acc_row) {
  switch (r) {
    case 32: row_grad_mult_vec<32>(row, pc, mult, base, gam, lane, dst, acc_row); return;
    case 16: row_grad_mult_vec<16>(row, pc, mult, base, gam, lane, dst, acc_row); return;
    case 8: row_grad_mult_vec<8>(row, pc, mult, base, gam, lane, dst, acc_row); return;
    case 4: row_grad_mult_vec<4>(row, pc, mult, base, gam, lane, dst, acc_row); return;
    default: break;
  }
  for (int q = 0; q < r; ++q) {
    int b = q + lane;                                   // start at column `lane`: fewer bank conflicts
    if (b >= r) b -= r;
    const float la = row[b];
    const float o = __expf(base + la + pc[b]) * mult[b] - __expf(la) * gam;
    if (acc_row != nullptr) atomicAdd(acc_row + b, o);
    else dst[b] = __float2bfloat16_rn(o);
  }
}

__global__ void circuit_hmm_loss_backward_kernel(const CircuitBackwardArgs a_, const float* __restrict__ coeff,
                                                 const float* __restrict__ tables, int table_stride, float* __restrict__ dT,
                                                 unsigned* work_counter) {
  extern __shared__ __align__(16) float sm[];
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  const int n = a_.n, r = a_.r;
  const int rr = r * r;
  const bool is_static = table_stride == 0;
  float* acc = sm;                                                       // static only: [n-1, r, r]
  float* mine = sm + (is_static ? (n - 1) * rr : 0) + static_cast<size_t>(wib) * hmm_backward_warp_floats(n, r);
  float* alphas = mine;                                                  // [n, r]
  float* tabs = alphas + n * r;
  float* cvec = tabs + 2 * rr;                                           // G[i] - alpha_i (log domain)
  float* dvec = cvec + 32;                                               // abar_i (plain)
  const bool has = lane < r;
  if (is_static) {
    for (int e = threadIdx.x; e < (n - 1) * rr; e += blockDim.x) acc[e] = 0.f;
    __syncthreads();
  }
  for (int w = next_window(work_counter, lane); w < a_.W; w = next_window(work_counter, lane)) {
    const float* g = a_.G + static_cast<size_t>(w) * n * r;
    const float* lw = a_.logw + static_cast<size_t>(w) * a_.sum_rows;
    const float* tb = tables + static_cast<size_t>(w) * table_stride;
    const float* cw = coeff + static_cast<size_t>(w) * n;
    const int* tg = a_.targets + static_cast<size_t>(w) * n;
    const size_t prow = static_cast<size_t>(w) * n * r;
    const size_t drow = static_cast<size_t>(w) * a_.dsum_pitch;
    // ---- forward, keeping every alpha_i
    if (n > 1) warp_table_load_async(tabs, tb, rr, lane);
    float alpha = has ? lw[lane] + g[lane] : -CUDART_INF_F;
    if (has) alphas[lane] = alpha;
    for (int i = 1; i < n; ++i) {
      if (i + 1 < n) {
        warp_table_load_async(tabs + (i & 1) * rr, tb + static_cast<size_t>(i) * rr, rr, lane);
        cp_async_wait<1>();
      } else {
        cp_async_wait<0>();
      }
      __syncwarp();
      const float* A = tabs + ((i - 1) & 1) * rr;
      float m = alpha;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, off));
      cvec[lane] = has ? __expf(alpha - m) : 0.f;
      __syncwarp();
      if (has) {
        const float s = hmm_matvec(cvec, A, lane, r);
        alpha = (m == -CUDART_INF_F) ? -CUDART_INF_F : g[i * r + lane] + m + __logf(s);
        alphas[i * r + lane] = alpha;
      }
      __syncwarp();
    }
    float lp = warp_lse(alpha, has);                                     // log p_{n-1}: the joint
    if (lane == 0 && a_.out != nullptr) a_.out[w] = lp;
    // ---- reverse sweep: tables in reverse order; the table of step n - 1 is still in its buffer
    float abar = has ? cw[n - 1] * __expf(alpha - lp) : 0.f;
    for (int i = n - 1; i >= 1; --i) {
      if (i < n - 1) {
        cp_async_wait<0>();
        __syncwarp();
      }
      if (i - 1 >= 1) warp_table_load_async(tabs + (i & 1) * rr, tb + static_cast<size_t>(i - 2) * rr, rr, lane);
      const float* A = tabs + ((i - 1) & 1) * rr;
      const float al_i = has ? alphas[i * r + lane] : -CUDART_INF_F;
      if (has) {
        a_.post[prow + static_cast<size_t>(i) * r + lane] = tg[i] >= 0 ? abar : 0.f;
        cvec[lane] = al_i == -CUDART_INF_F ? -CUDART_INF_F : g[i * r + lane] - al_i;
        dvec[lane] = abar;
      } else {
        cvec[lane] = -CUDART_INF_F;
        dvec[lane] = 0.f;
      }
      __syncwarp();
      const float al = has ? alphas[(i - 1) * r + lane] : -CUDART_INF_F;
      const float lp_prev = warp_lse(al, has);                           // log p_{i-1}
      float prop = 0.f;
      if (has) {
        const float* row = A + lane * r;
        for (int q = 0; q < r; ++q) {
          int b = q + lane;
          if (b >= r) b -= r;
          prop += __expf(al + row[b] + cvec[b]) * dvec[b];
        }
        const size_t off = static_cast<size_t>(r) + static_cast<size_t>(i - 1) * rr + lane * r;
        row_grad_mult(row, cvec, dvec, al, prop, lane, r, is_static ? nullptr : a_.dsum + drow + off,
                      is_static ? acc + static_cast<size_t>(i - 1) * rr + lane * r : nullptr);
      }
      abar = has ? cw[i - 1] * __expf(al - lp_prev) + prop : 0.f;
      __syncwarp();                                                      // cvec, dvec and the table buffer are free again
    }
    float total = abar;                                                  // sum_z abar_0[z]
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) total += __shfl_xor_sync(kFull, total, off);
    if (has) {
      a_.post[prow + lane] = tg[0] >= 0 ? abar : 0.f;
      a_.dsum[drow + lane] = __float2bfloat16_rn(abar - __expf(lw[lane]) * total);
    }
    __syncwarp();
  }
  if (is_static) {
    __syncthreads();
    for (int e = threadIdx.x; e < (n - 1) * rr; e += blockDim.x) {
      const float v = acc[e];
      if (v != 0.f) atomicAdd(dT + e, v);
    }
  }
}

// ---------------------------------------------------------------- circuit backward: binary tree (Eq. BTree)
// Upward pass as in circuit_btree_kernel (prod[j][z], S[c][z]); downward pass with U[j][z] = log-weight of everything
// outside node j's subtree given z_j = z: U[0] = log omega_root, U[c][b] = LSE_z(U[j][z] + S[sibling][z] + logOmega_c[z][b]).
// Posterior of a latent: gamma_j = exp(U[j] + prod[j] - log q); a token's evidence gradient is its owner's gamma.
// Pairwise posterior xi_c[z][b] = exp(U[j][z] + S[sib][z] + logOmega_c[z][b] + prod[c][b] - log q); through the row
// softmax: xi_c[z][b] - Omega_c[z][b] gamma_j[z]. The tables are streamed twice (up: deepest parents first; down: in
// address order). Shared memory per warp: 3*(n-1)*r + 2*r*r + 32 floats.  r <= 32.
__host__ __device__ inline size_t btree_backward_warp_floats(int n, int r) {
  return 3 * static_cast<size_t>(n - 1) * r + 2 * static_cast<size_t>(r) * r + 32;
}

// With `loss_coeff` [W, n] (Eq. 6: L = sum_l coeff[w, l-1] log p_l over the prefix lengths l) the warp runs the pass of
// every prefix length on its window back to back, accumulating (accumulate == 1): the window's tables and gradient rows
// are then re-used out of L2 instead of being streamed from HBM once per prefix length.
__global__ void circuit_btree_backward_kernel(const CircuitBackwardArgs a_, const float* __restrict__ loss_coeff,
                                              unsigned* work_counter) {
  extern __shared__ __align__(16) float sm[];
  const int wib = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n = a_.n, r = a_.r;
  int len = a_.len;                                                      // prefix length of the current pass
  float* prod = sm + static_cast<size_t>(wib) * btree_backward_warp_floats(n, r);
  float* S = prod + (n - 1) * r;
  float* U = S + (n - 1) * r;
  float* tabs = U + (n - 1) * r;
  float* cur = tabs + 2 * r * r;
  const bool has = lane < r;
  const int first_leaf_node = n / 2 - 1;
  const int rr = r * r;
  const int ntab = n - 2;
  auto child_of = [&](int t) { return 2 * (first_leaf_node - 1 - (t >> 1)) + 1 + (t & 1); };
  // A node whose tokens all lie at or after `len` sees no evidence: its subtree evaluates to one, its table has no
  // gradient, and it is skipped (first token of heap node c: index within its level times the level's width).
  auto has_evidence = [&](int c) {
    const int depth = 31 - __clz(c + 1);
    return ((c + 1 - (1 << depth)) * (n >> depth)) < len;
  };
  for (int w = next_window(work_counter, lane); w < a_.W; w = next_window(work_counter, lane)) {
    const float* g = a_.G + static_cast<size_t>(w) * n * r;
    const float* lw = a_.logw + static_cast<size_t>(w) * a_.sum_rows;
    const size_t drow = static_cast<size_t>(w) * a_.dsum_pitch;
    for (len = loss_coeff ? 1 : a_.len; len <= (loss_coeff ? n : a_.len); ++len) {
    const float wt = loss_coeff ? loss_coeff[static_cast<size_t>(w) * n + len - 1]
                                : a_.weight[static_cast<size_t>(w) * a_.weight_stride];
    if (loss_coeff != nullptr && wt == 0.f) continue;                    // the same for every lane of the warp
    // ---- upward (tokens >= len are summed out: their input units output one)
    for (int j = n - 2; j >= first_leaf_node; --j) {
      const int t0 = 2 * (j - first_leaf_node);
      if (has) prod[j * r + lane] = (t0 < len ? g[t0 * r + lane] : 0.f) + (t0 + 1 < len ? g[(t0 + 1) * r + lane] : 0.f);
    }
    auto next_up = [&](int t) {                                          // next table of the upward pass that is needed
      while (t < ntab && !has_evidence(child_of(t))) ++t;
      return t;
    };
    int buf = 0;
    int tn = next_up(0);
    if (tn < ntab) warp_table_load_async(tabs, lw + r + static_cast<size_t>(child_of(tn) - 1) * rr, rr, lane);
    __syncwarp();
    float acc = 0.f;
    for (int t = 0; t < ntab; ++t) {
      const int c = child_of(t);
      float sc = 0.f;                                                    // a subtree without evidence: log 1
      if (t == tn) {
        tn = next_up(t + 1);
        if (tn < ntab) {
          warp_table_load_async(tabs + (buf ^ 1) * rr, lw + r + static_cast<size_t>(child_of(tn) - 1) * rr, rr, lane);
          cp_async_wait<1>();
        } else {
          cp_async_wait<0>();
        }
        __syncwarp();
        sc = sum_layer_staged(tabs + buf * rr, prod + c * r, lane, r);
        buf ^= 1;
      }
      if (has) S[c * r + lane] = sc;
      acc += sc;
      if (t & 1) {
        if (has) prod[((c - 2) >> 1) * r + lane] = acc;
        acc = 0.f;
      }
      __syncwarp();
    }
    const float logq = warp_lse(has ? lw[lane] + prod[lane] : 0.f, has);
    if (lane == 0 && a_.out != nullptr) a_.out[w] = logq;
    // ---- downward, children c = 1 .. n-2 in address order
    if (has) {
      U[lane] = lw[lane];
      put_dsum(a_, drow + lane, wt * (__expf(lw[lane] + prod[lane] - logq) - __expf(lw[lane])));
    }
    auto next_down = [&](int c) {
      while (c <= ntab && !has_evidence(c)) ++c;
      return c;
    };
    buf = 0;
    int cn = next_down(1);
    if (cn <= ntab) warp_table_load_async(tabs, lw + r + static_cast<size_t>(cn - 1) * rr, rr, lane);
    __syncwarp();
    for (int c = cn; c <= ntab; c = cn) {
      const int j = (c - 1) >> 1;
      const int sib = (c & 1) ? c + 1 : c - 1;
      cn = next_down(c + 1);
      if (cn <= ntab) {
        warp_table_load_async(tabs + (buf ^ 1) * rr, lw + r + static_cast<size_t>(cn - 1) * rr, rr, lane);
        cp_async_wait<1>();
      } else {
        cp_async_wait<0>();
      }
      if (has) cur[lane] = U[j * r + lane] + S[sib * r + lane];          // in[z]
      __syncwarp();
      const float* tab = tabs + buf * rr;
      buf ^= 1;
      if (has) {
        // message to the child: lane b, over the parent's values z (column of the table)
        float m = -CUDART_INF_F;
        for (int z = 0; z < r; ++z) m = fmaxf(m, cur[z] + tab[z * r + lane]);
        float s = 0.f;
        for (int z = 0; z < r; ++z) s += __expf(cur[z] + tab[z * r + lane] - m);
        U[c * r + lane] = (m == -CUDART_INF_F) ? -CUDART_INF_F : m + __logf(s);
        // gradient of the child's table: lane z (row), over the child's values b
        const float in_z = cur[lane];
        const float gam_parent = __expf(U[j * r + lane] + prod[j * r + lane] - logq);
        const size_t off = static_cast<size_t>(r) + static_cast<size_t>(c - 1) * rr + lane * r;
        row_grad(tab + lane * r, prod + c * r, in_z - logq, gam_parent, wt, lane, r,
                 a_.accumulate ? nullptr : a_.dsum + drow + off, nullptr, a_.accumulate ? a_.dsum_f32 + drow + off : nullptr);
      }
      __syncwarp();
    }
    // ---- evidence gradients: token i under its owner's posterior
    for (int i = 0; i < n; ++i) {
      const int o = first_leaf_node + (i >> 1);
      const bool valid = a_.targets[static_cast<size_t>(w) * n + i] >= 0;
      if (has) {
        const size_t idx = (static_cast<size_t>(w) * n + i) * r + lane;
        if (i < len) put_post(a_, idx, valid ? wt * __expf(U[o * r + lane] + prod[o * r + lane] - logq) : 0.f);
        else if (!a_.accumulate) a_.post[idx] = 0.f;
      }
    }
    __syncwarp();
    }                                                                    // prefix lengths
  }
}

// fp32 [rows, cols] (pitch src_pitch) -> bf16 (pitch dst_pitch): the accumulated sum-unit logit gradients become the
// tensor cores' operand.
__global__ void f32_rows_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int cols,
                                        size_t src_pitch, size_t dst_pitch) {
  const size_t total = static_cast<size_t>(rows) * cols;
  for (size_t e = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; e < total;
       e += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t rw = e / cols, c = e - rw * cols;
    dst[rw * dst_pitch + c] = __float2bfloat16_rn(src[rw * src_pitch + c]);
  }
}

// ---------------------------------------------------------------- gradient with respect to the emission logits
// dlogit[t, c] = post[t, u] * (onehot(target[t, i] == c - u v) - exp(logit[t, c] - lse[t, u])),  u = c / v = i r + k,
// from the logits and log-sum-exps the forward pass kept (padding columns hold -inf: no mass, zero gradient; a
// marginalised byte has no gradient). Written once, as bf16 rows [T, pitch]: both weight-sized GEMMs read this one
// matrix, d hidden along its rows (K-major) and dW down its columns (MN-major). One streaming pass: a thread converts
// 8 adjacent logits (two 16-byte loads, one 16-byte store); v is a multiple of 16, so they belong to one unit.
struct LogitGradArgs {
  const float* logits;       // [T, Nc], pitch Nc
  const float* lse;          // [T, n r]
  const float* post;         // [T, n r]
  const int* targets;        // [T, n]
  __nv_bfloat16* dlogit;     // [T, pitch]
  size_t pitch;
  int T, Nc, n, r, v;
};

__global__ void __launch_bounds__(256) logit_gradient_kernel(const LogitGradArgs a) {
  const int c = (blockIdx.x * 256 + threadIdx.x) * 8;
  if (c >= a.Nc) return;
  const int units = a.n * a.r;
  const int u = c / a.v;
  const int i = u / a.r;
  const int col_in_unit = c - u * a.v;
  for (int t = blockIdx.y; t < a.T; t += gridDim.y) {
    const int tgt = a.targets[static_cast<size_t>(t) * a.n + i];
    const size_t tu = static_cast<size_t>(t) * units + u;
    const float pst = tgt >= 0 ? a.post[tu] : 0.f;
    const float lse2 = a.lse[tu] * kLog2e;
    const float4* src = reinterpret_cast<const float4*>(a.logits + static_cast<size_t>(t) * a.Nc + c);
    const float4 x0 = __ldcs(src), x1 = __ldcs(src + 1);
    const float xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
    const int rel = tgt - col_in_unit;
    __align__(16) __nv_bfloat16 o[8];
#pragma unroll
    for (int q = 0; q < 8; ++q)
      o[q] = __float2bfloat16_rn(pst * ((rel == q ? 1.f : 0.f) - fast_ex2(fmaf(xs[q], kLog2e, -lse2))));
    *reinterpret_cast<uint4*>(a.dlogit + static_cast<size_t>(t) * a.pitch + c) = *reinterpret_cast<const uint4*>(o);
  }
}

// ---------------------------------------------------------------- plain bf16 GEMM on the tcgen05 tensor cores
// C[M, N] (fp32, row-major, pitch ldc) = A[M, K] B[N, K]^T with bf16 operands read where they lie, in either
// orientation: K-major (K contiguous in memory: 64-element K boxes of 128 or 256 rows) or MN-major (the M / N index
// contiguous: 64 x 64 boxes, two for the 128 rows of A, four for the 256 columns of B). Out-of-range rows and
// columns read as zero. The K axis may consist of two segments with a B matrix each (d hidden sums over the emission
// rows and the sum-unit rows, which are separate matrices); A then continues at column a_k0[1]. Same pipeline as the
// projection kernel: one persistent CTA per SM, warp 0 TMA producer, warp 1 MMA issuer (M=128, N=256 tiles, two TMEM
// slots), warps 2..5 epilogue (one thread per row, 16 fp32 columns per step).
struct PlainGemmParams {
  CUtensorMap tm_a;      // K-major: A [M, K], box 64 (k) x 128; MN-major: A^T [K, M], box 64 (m) x 64 (k)
  CUtensorMap tm_b[2];   // per K segment. K-major: B [N, K], box 64 (k) x 256; MN-major: B^T [K, N], box 64 (n) x 64 (k)
  int a_k0[2];           // K coordinate of A at which each segment starts (multiples of 8)
  int seg_kblocks[2];    // 64-wide K blocks per segment (segment 1: 0 if unused)
  int M, N;
  int m_tiles, n_tiles;
  int stages, stage_bytes;
  int wide_stores;       // C and ldc allow 32-byte stores
  float* C;
  size_t ldc;
  // Instead of C (C == NULL): the result split into two bf16 halves, x = hi + lo, written as [M, N / split_k, 2, split_k]
  // (group g of split_k columns: hi at column (2 g) split_k, lo at (2 g + 1) split_k; split_k a multiple of 16).
  __nv_bfloat16* C_hilo;
  int split_k;
  // Instead of C (C == NULL, C_hilo == NULL): the result rounded to bf16, [M, N] at a pitch of ldc elements.
  __nv_bfloat16* C_bf16;
  // Several independent products of the same shape in one launch (batches > 1; one K segment): product q reads A at
  // its M / K coordinates plus q * a_m_step / q * a_k_step, B at its N / K coordinates plus q * b_n_step / q * b_k_step,
  // and writes at C (or C_bf16) + q * c_step elements. Rows of A and columns of B past M and N are then another product's
  // data, not zeros: they reach accumulator rows and columns that are not written. Along K the operands must agree on
  // zeros past the product's own extent (the caller pads one of them).
  int batches, a_m_step, a_k_step, b_n_step, b_k_step;
  size_t c_step;
  unsigned* status;
  uint64_t wait_limit_ns;   // limit of every pipeline wait
};
constexpr int kPlainTileN = 256;
constexpr uint32_t kMnBoxBytes = 64 * kBlockK * 2;   // one 64 x 64 bf16 box: 8 KB

// TN: columns of an accumulator tile: 256, or 64 for the batched products whose N is a rank (MN-major B only: the boxes
// of the tensor map are 64 wide) - what is fetched, multiplied and read back for columns that do not exist is a quarter.
template <bool A_MN, bool B_MN, int TN = 256>
__global__ void __launch_bounds__(kGemmThreads, 1) plain_gemm_kernel(const __grid_constant__ PlainGemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (tiles_addr - raw_addr);
  GemmControl* ctl = reinterpret_cast<GemmControl*>(tiles + static_cast<size_t>(p.stages) * p.stage_bytes);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // n-tile fastest: the CTAs running together cover a few m-tiles x all n-tiles, so the (larger) A operand is
  // streamed from HBM once and the B operand once per wave of m-tiles
  const int per_batch = p.m_tiles * p.n_tiles;
  const int num_items = per_batch * p.batches;
  const int kblocks = p.seg_kblocks[0] + p.seg_kblocks[1];
  constexpr uint32_t kSlots = 2;
  constexpr uint32_t kBBytes = TN * kBlockK * 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (uint32_t s = 0; s < kSlots; ++s) {
      mbar_init(smem_u32(&ctl->tfull[s]), 1);
      mbar_init(smem_u32(&ctl->tempty[s]), 4);
    }
    mbar_init(smem_u32(&ctl->drain), 1);
    ctl->abort = 0;
    ctl->wait_limit_ns = p.wait_limit_ns;
    fence_mbar_init();
    tma_prefetch_desc(&p.tm_a);
    tma_prefetch_desc(&p.tm_b[0]);
    if (p.seg_kblocks[1] > 0) tma_prefetch_desc(&p.tm_b[1]);
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
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued_mask = 0, phase_mask = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
        const int bt = item / per_batch, rest = item - bt * per_batch;
        const int nt = rest % p.n_tiles, mt = rest / p.n_tiles;
        const int am = mt * kBlockM + bt * p.a_m_step, ak = bt * p.a_k_step;    // this product's corner of A ...
        const int bn = nt * TN + bt * p.b_n_step, bk = bt * p.b_k_step;   // ... and of B
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, p.status)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctl->full[stage]);
          const uint32_t a_dst = tiles_addr + stage * p.stage_bytes;
          const int seg = kb >= p.seg_kblocks[0] ? 1 : 0;
          const int kloc = (kb - (seg ? p.seg_kblocks[0] : 0)) * kBlockK;      // K offset inside the segment
          mbar_arrive_expect_tx(full, kABytes + kBBytes);
          if (A_MN) {
#pragma unroll
            for (int q = 0; q < kBlockM / 64; ++q)
              tma_load_2d(a_dst + q * kMnBoxBytes, &p.tm_a, full, am + q * 64, p.a_k0[seg] + kloc + ak);
          } else {
            tma_load_2d(a_dst, &p.tm_a, full, p.a_k0[seg] + kloc + ak, am);
          }
          if (B_MN) {
#pragma unroll
            for (int q = 0; q < TN / 64; ++q)
              tma_load_2d(a_dst + kABytes + q * kMnBoxBytes, &p.tm_b[seg], full, bn + q * 64, kloc + bk);
          } else {
            tma_load_2d(a_dst + kABytes, &p.tm_b[seg], full, kloc + bk, bn);
          }
          issued_mask |= 1u << stage;
          phase_mask = (phase_mask & ~(1u << stage)) | (phase << stage);
          if (++stage == static_cast<uint32_t>(p.stages)) { stage = 0; phase ^= 1u; }
        }
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
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, use = 0;
      bool ok = true;
      const uint32_t idesc = umma_idesc_bf16(kBlockM, TN, A_MN, B_MN);
      // descriptor advance per K=16 step, in 16-byte units: 32 bytes along a swizzled K-major row, two 8-row groups
      // (2048 bytes) down an MN-major box
      constexpr uint32_t kStepA = A_MN ? 128u : 2u, kStepB = B_MN ? 128u : 2u;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++use) {
        const uint32_t slot = use % kSlots;
        if (!bounded_wait(smem_u32(&ctl->tempty[slot]), ((use / kSlots) & 1u) ^ 1u, ctl, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + slot * TN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!bounded_wait(smem_u32(&ctl->full[stage]), phase, ctl, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = tiles_addr + stage * p.stage_bytes;
          const uint64_t a_desc = A_MN ? umma_smem_desc_mn_sw128(a_addr, kMnBoxBytes) : umma_smem_desc_sw128(a_addr);
          const uint64_t b_desc = B_MN ? umma_smem_desc_mn_sw128(a_addr + kABytes, kMnBoxBytes)
                                       : umma_smem_desc_sw128(a_addr + kABytes);
#pragma unroll
          for (int kk = 0; kk < kBlockK / 16; ++kk)
            umma_bf16(d_tmem, a_desc + kStepA * kk, b_desc + kStepB * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
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
    const int quarter = warp & 3;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    uint32_t use = 0;
    for (int item = blockIdx.x; item < num_items; item += gridDim.x, ++use) {
      const int bt = item / per_batch, rest = item - bt * per_batch;
      const int nt = rest % p.n_tiles, mt = rest / p.n_tiles;
      const uint32_t slot = use % kSlots;
      if (!bounded_wait_warp(smem_u32(&ctl->tfull[slot]), (use / kSlots) & 1u, ctl, p.status, lane)) break;
      tc_fence_after();
      const int row = mt * kBlockM + quarter * 32 + lane;
      const uint32_t tcol = lane_base + slot * TN;
      const size_t coff = static_cast<size_t>(row < p.M ? row : 0) * p.ldc + static_cast<size_t>(bt) * p.c_step;
      float* crow = p.C + coff;
      for (int b = 0; b < TN / 16; ++b) {
        const int col0 = nt * TN + b * 16;
        if (col0 >= p.N) break;                          // (warp-uniform) the rest of the tile lies past the last column
        float x[16];
        tmem_ld16(tcol + b * 16, x);
        if (row < p.M && p.C == nullptr && p.C_hilo == nullptr) {
          __align__(16) __nv_bfloat16 o[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) o[q] = __float2bfloat16_rn(x[q]);
          uint4* dst = reinterpret_cast<uint4*>(p.C_bf16 + coff + col0);      // ldc, c_step and C_bf16 keep 16 columns 32-byte aligned
          dst[0] = reinterpret_cast<const uint4*>(o)[0];
          dst[1] = reinterpret_cast<const uint4*>(o)[1];
        } else if (row < p.M && col0 < p.N && p.C == nullptr) {
          // 16 columns of one group: 32 bytes of high halves and 32 bytes of low halves
          const int grp = col0 / p.split_k, q0 = col0 - grp * p.split_k;
          __align__(16) __nv_bfloat16 hi[16], lo[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            hi[q] = __float2bfloat16_rn(x[q]);
            lo[q] = __float2bfloat16_rn(x[q] - __bfloat162float(hi[q]));
          }
          __nv_bfloat16* dst = p.C_hilo + static_cast<size_t>(row) * (2 * p.N) + static_cast<size_t>(2 * grp) * p.split_k + q0;
          reinterpret_cast<uint4*>(dst)[0] = reinterpret_cast<const uint4*>(hi)[0];
          reinterpret_cast<uint4*>(dst)[1] = reinterpret_cast<const uint4*>(hi)[1];
          reinterpret_cast<uint4*>(dst + p.split_k)[0] = reinterpret_cast<const uint4*>(lo)[0];
          reinterpret_cast<uint4*>(dst + p.split_k)[1] = reinterpret_cast<const uint4*>(lo)[1];
        } else if (row < p.M && col0 < p.N) {          // N is a multiple of 16
          if (p.wide_stores) {                         // 32-byte aligned rows: one full sector per store
            st_global_v8(crow + col0, x);
            st_global_v8(crow + col0 + 8, x + 8);
          } else {
            float4* c4 = reinterpret_cast<float4*>(crow + col0);
#pragma unroll
            for (int q = 0; q < 4; ++q) c4[q] = make_float4(x[4 * q], x[4 * q + 1], x[4 * q + 2], x[4 * q + 3]);
          }
        }
      }
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

}  // namespace mtpc
