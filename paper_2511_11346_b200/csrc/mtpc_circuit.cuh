// Circuit evaluation in log space (Eq. CP, Eq. HMM, Eq. BTree), latent ancestral sampling (Algorithm 1, sum
// units) and the small preparation kernels. One warp evaluates one window; lane = latent value.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>
#include <stdint.h>

#include "mtpc_ptx.cuh"

namespace mtpc {

constexpr int kCircuitWarps = 8;
constexpr unsigned kFull = 0xffffffffu;

// (m, s) represents log-sum-exp = m + log s. Merging tolerates empty operands (m = -inf, s = 0).
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn == -CUDART_INF_F) { m = mn; s = 0.f; return; }
  s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
  m = mn;
}
__device__ __forceinline__ float warp_lse(float val, bool has) {
  float m = has ? val : -CUDART_INF_F;
  float s = has ? 1.f : 0.f;
  if (has && val != val) { m = 0.f; s = val; }   // NaN must survive the max
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(kFull, m, off);
    const float s2 = __shfl_xor_sync(kFull, s, off);
    lse_merge(m, s, m2, s2);
  }
  return m + __logf(s);
}

// Eq. (CP): out[w] = LSE_k( log omega[p, k] + sum_i G[w, i, k] ),  p = w / wpp.
// With `prefix` (may be NULL) the kernel also writes prefix[w, i] = log q(x_0..x_i), the joint with the later bytes
// summed out (Algorithm 3's marginals): for a mixture that is the same log-sum-exp over the first i+1 slots only.
__global__ void circuit_cp_kernel(const float* __restrict__ G, const float* __restrict__ logw,
                                  float* __restrict__ out, float* __restrict__ prefix, int W, int wpp, int n, int r,
                                  int sum_rows, int raw_mixture) {
  grid_dependency_wait();   // G and log omega come from the kernel before this one
  const int w = blockIdx.x * kCircuitWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= W) return;
  const float* g = G + static_cast<size_t>(w) * n * r;
  const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
  // raw_mixture: logw holds the mixture LOGITS (the few-position draft path with more than 32 components leaves the
  // softmax to its consumers): log omega_k = logit_k - LSE(logits), so LSE(logits) is subtracted from every result.
  float norm = 0.f;
  if (raw_mixture) {
    float m = -CUDART_INF_F, s = 0.f;
    for (int k = lane; k < r; k += 32) lse_merge(m, s, lw[k], 1.f);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float m2 = __shfl_xor_sync(kFull, m, off);
      const float s2 = __shfl_xor_sync(kFull, s, off);
      lse_merge(m, s, m2, s2);
    }
    norm = m + __logf(s);
  }
  if (prefix != nullptr) {
    // running sums of up to 4 units per lane (r <= 128); one warp log-sum-exp per slot
    float a[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) a[q] = (lane + 32 * q < r) ? lw[lane + 32 * q] : 0.f;
    float last = 0.f;
    for (int i = 0; i < n; ++i) {
      float m = -CUDART_INF_F, s = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int k = lane + 32 * q;
        if (k < r) {
          a[q] += g[i * r + k];
          if (a[q] != a[q]) { m = 0.f; s = a[q]; } else lse_merge(m, s, a[q], 1.f);
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float m2 = __shfl_xor_sync(kFull, m, off);
        const float s2 = __shfl_xor_sync(kFull, s, off);
        lse_merge(m, s, m2, s2);
      }
      last = m + __logf(s) - norm;
      if (lane == 0) prefix[static_cast<size_t>(w) * n + i] = last;
    }
    if (lane == 0 && out != nullptr) out[w] = last;
    return;
  }
  float m = -CUDART_INF_F, s = 0.f;
  for (int k = lane; k < r; k += 32) {
    float a = lw[k];
    for (int i = 0; i < n; ++i) a += g[i * r + k];
    if (a != a) { m = 0.f; s = a; continue; }
    lse_merge(m, s, a, 1.f);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(kFull, m, off);
    const float s2 = __shfl_xor_sync(kFull, s, off);
    lse_merge(m, s, m2, s2);
  }
  if (lane == 0) out[w] = m + __logf(s) - norm;
}

// Eq. (BTree), bottom-up over the heap-ordered latent tree. Node j >= 1 has the table
// logOmega_j[a][b] = logw[p, r + (j-1) r^2 + a r + b] (parent's value a, own value b); the deepest internal node
// n/2-1+m multiplies the input units of tokens 2m and 2m+1. prod[j][z] is the product unit under z_j = z.

// One sum layer seen from the parent: returns, for lane = parent value z, LSE_b(logOmega_c[z][b] + pc[b]).
// tab: the child's r x r table in global memory; pc: r floats in shared memory (written before the call; the
// function synchronises the warp); table: r * (r+1) floats of per-warp shared scratch.
// An r x r table from global memory into a padded shared tile (row pitch r + 1), by one warp. ROWS > 1: that many rows'
// loads are in flight before the first store - for a kernel where one warp walks many tables on its own (a load-store pair
// per row costs one memory round trip per row); a kernel with many such warps per SM hides that latency and is better
// off with the plain loop's few registers.
template <int ROWS>
__device__ __forceinline__ void btree_stage_table(const float* __restrict__ tab, float* table, int lane, int r) {
  const bool has = lane < r;
  if (ROWS == 1) {
    for (int a = 0; a < r; ++a)
      if (has) table[a * (r + 1) + lane] = tab[a * r + lane];
    return;
  }
  for (int a0 = 0; a0 < r; a0 += ROWS) {
    float t[ROWS];
#pragma unroll
    for (int q = 0; q < ROWS; ++q) t[q] = (has && a0 + q < r) ? tab[(a0 + q) * r + lane] : 0.f;
#pragma unroll
    for (int q = 0; q < ROWS; ++q)
      if (has && a0 + q < r) table[(a0 + q) * (r + 1) + lane] = t[q];
  }
}

template <int ROWS = 1>
__device__ __forceinline__ float btree_sum_layer(const float* __restrict__ tab, const float* pc, float* table,
                                                 int lane, int r) {
  const bool has = lane < r;
  btree_stage_table<ROWS>(tab, table, lane, r);    // coalesced rows -> padded shared tile
  __syncwarp();
  float res = 0.f;
  if (has) {
    const float* row = table + lane * (r + 1);     // row z = lane, over the child's values b
    float m = -CUDART_INF_F;
    for (int b = 0; b < r; ++b) m = fmaxf(m, row[b] + pc[b]);
    float s = 0.f;
    for (int b = 0; b < r; ++b) s += __expf(row[b] + pc[b] - m);
    res = (m == -CUDART_INF_F) ? -CUDART_INF_F : m + __logf(s);
    if (s != s) res = s;                           // NaN evidence must survive the max
  }
  __syncwarp();
  return res;
}

// Dynamic work distribution for the kernels whose cost per window is large: every warp takes the next window index
// from a counter the host zeroes before the launch, so that all SMs stay busy until the last window.
__device__ __forceinline__ int next_window(unsigned* counter, int lane) {
  unsigned w = 0;
  if (lane == 0) w = atomicAdd(counter, 1u);
  return static_cast<int>(__shfl_sync(kFull, w, 0));
}

// ---- asynchronous staging of an r x r table (global -> shared) by one warp, for kernels that stream one set of
// tables per position from HBM: the copy of the next table is in flight while the current one is reduced.
__device__ __forceinline__ void cp_async_16(float* dst, const float* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst))),
               "l"(src)
               : "memory");
}
__device__ __forceinline__ void cp_async_4(float* dst, const float* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst))),
               "l"(src)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// Copies `count` floats; 16 bytes per request when both addresses allow it (count, src and dst multiples of 4 floats).
__device__ __forceinline__ void warp_table_load_async(float* dst, const float* __restrict__ src, int count, int lane) {
  const bool vec = (count & 3) == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) == 0;
  if (vec) {
    for (int e = lane * 4; e < count; e += 128) cp_async_16(dst + e, src + e);
  } else {
    for (int e = lane; e < count; e += 32) cp_async_4(dst + e, src + e);
  }
  cp_async_commit();
}
// The same sum layer as btree_sum_layer on a table already in shared memory, unpadded [z][b]; lane z walks its row
// starting at column z, so that the 32 lanes hit 32 different banks. R a multiple of 4 (both arrays 16-byte aligned):
// the row and the child's vector are read as float4, rotated by the lane so that a quarter-warp's requests fall in
// different bank groups, and reduced in registers (max, then sum of exponentials).
template <int R>
__device__ __forceinline__ float sum_layer_staged_vec(const float* tab, const float* pc, int lane) {
  if (lane >= R) return 0.f;
  constexpr int Q = R / 4;
  const float4* row4 = reinterpret_cast<const float4*>(tab + lane * R);
  const float4* pc4 = reinterpret_cast<const float4*>(pc);
  float v[R];
#pragma unroll
  for (int q = 0; q < Q; ++q) {
    const int j = (q + lane) & (Q - 1);
    const float4 a = row4[j];
    const float4 b = pc4[j];
    v[4 * q] = a.x + b.x;
    v[4 * q + 1] = a.y + b.y;
    v[4 * q + 2] = a.z + b.z;
    v[4 * q + 3] = a.w + b.w;
  }
  float m = v[0];
#pragma unroll
  for (int q = 1; q < R; ++q) m = fmaxf(m, v[q]);
  float s = 0.f;
#pragma unroll
  for (int q = 0; q < R; ++q) s += __expf(v[q] - m);
  float res = (m == -CUDART_INF_F) ? -CUDART_INF_F : m + __logf(s);
  if (s != s) res = s;                             // NaN evidence must survive the max
  return res;
}
__device__ __forceinline__ float sum_layer_staged(const float* tab, const float* pc, int lane, int r) {
  switch (r) {
    case 32: return sum_layer_staged_vec<32>(tab, pc, lane);
    case 16: return sum_layer_staged_vec<16>(tab, pc, lane);
    case 8: return sum_layer_staged_vec<8>(tab, pc, lane);
    case 4: return sum_layer_staged_vec<4>(tab, pc, lane);
    default: break;
  }
  if (lane >= r) return 0.f;
  const float* row = tab + lane * r;
  float m = -CUDART_INF_F;
  for (int b = 0; b < r; ++b) m = fmaxf(m, row[b] + pc[b]);
  float s = 0.f;
  for (int b = 0; b < r; ++b) s += __expf(row[b] + pc[b] - m);
  float res = (m == -CUDART_INF_F) ? -CUDART_INF_F : m + __logf(s);
  if (s != s) res = s;
  return res;
}

// Shared memory per warp: (n-1) * r floats of prod + 2 * r * r floats (two staged tables); with PREFIX another
// (n-1) * r floats (the sum-layer outputs S[c][z], kept for the prefix passes) + r floats.  r <= 32.
// The n-2 tables of a position (57 KB at n = 16, r = 32) are read exactly once, in the order the bottom-up pass
// needs them, through a two-deep cp.async pipeline: this kernel is bound by that stream from HBM.
// PREFIX: also writes prefix[w, i] = log q(x_0..x_i). Summing the later bytes out sets their input units to one,
// so every subtree right of token i evaluates to one, every subtree left of it keeps its value, and only the
// nodes on the path from token i's owner to the root have to be re-evaluated.
__host__ __device__ inline int btree_warp_floats(int n, int r, bool with_prefix) {
  return (n - 1) * r + 2 * r * r + (with_prefix ? (n - 1) * r + r : 0);
}

template <bool PREFIX>
__global__ void circuit_btree_kernel(const float* __restrict__ G, const float* __restrict__ logw,
                                     float* __restrict__ out, float* __restrict__ prefix, unsigned* work_counter,
                                     int W, int wpp, int n, int r, int sum_rows) {
  extern __shared__ __align__(16) float sm[];
  grid_dependency_wait();   // G, log omega and the zeroed work counter come from the kernels before this one
  const int wib = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  float* prod = sm + static_cast<size_t>(wib) * btree_warp_floats(n, r, PREFIX);
  float* tabs = prod + (n - 1) * r;                // two tables; the prefix passes reuse the space as one padded table
  float* table = tabs;
  float* S = tabs + 2 * r * r;                     // PREFIX only
  float* cur = S + (n - 1) * r;                    // PREFIX only
  const bool has = lane < r;
  const int first_leaf_node = n / 2 - 1;
  const int rr = r * r;
  const int ntab = n - 2;                          // table t belongs to child c(t) of node j(t), deepest parents first
  auto child_of = [&](int t) { return 2 * (first_leaf_node - 1 - (t >> 1)) + 1 + (t & 1); };
  for (int w = next_window(work_counter, lane); w < W; w = next_window(work_counter, lane)) {
  const float* g = G + static_cast<size_t>(w) * n * r;
  const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
  if (ntab > 0) warp_table_load_async(tabs, lw + r + static_cast<size_t>(child_of(0) - 1) * rr, rr, lane);
  for (int j = n - 2; j >= first_leaf_node; --j) {
    const int m = j - first_leaf_node;
    if (has) prod[j * r + lane] = g[(2 * m) * r + lane] + g[(2 * m + 1) * r + lane];
  }
  __syncwarp();
  float acc = 0.f;
  for (int t = 0; t < ntab; ++t) {
    const int c = child_of(t);
    if (t + 1 < ntab) {
      warp_table_load_async(tabs + ((t + 1) & 1) * rr, lw + r + static_cast<size_t>(child_of(t + 1) - 1) * rr, rr, lane);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncwarp();                                  // table t is in shared memory for every lane
    const float sc = sum_layer_staged(tabs + (t & 1) * rr, prod + c * r, lane, r);
    if (PREFIX && has) S[c * r + lane] = sc;
    acc += sc;
    if (t & 1) {                                   // both children of node j done
      if (has) prod[((c - 2) >> 1) * r + lane] = acc;
      acc = 0.f;
    }
    __syncwarp();                                  // the buffer may be overwritten, prod[j] may be read
  }
  const float res = warp_lse(has ? lw[lane] + prod[lane] : 0.f, has);
  if (lane == 0 && out != nullptr) out[w] = res;
  if (PREFIX) {
    if (lane == 0) prefix[static_cast<size_t>(w) * n + n - 1] = res;
    for (int i = 0; i < n - 1; ++i) {
      int c = first_leaf_node + (i >> 1);
      bool full = (i & 1) != 0;                    // both tokens of the owner are inside the prefix
      float val = has ? (full ? prod[c * r + lane] : g[i * r + lane]) : 0.f;
      while (c > 0) {
        const bool is_right = (c & 1) == 0;
        float sc;
        if (full) {
          sc = has ? S[c * r + lane] : 0.f;
        } else {
          if (has) cur[lane] = val;
          __syncwarp();
          sc = btree_sum_layer(lw + r + static_cast<size_t>(c - 1) * r * r, cur, table, lane, r);
        }
        val = sc + ((is_right && has) ? S[(c - 1) * r + lane] : 0.f);   // left sibling: inside; right sibling: one
        full = full && is_right;
        c = (c - 1) >> 1;
      }
      const float pre = warp_lse(has ? lw[lane] + val : 0.f, has);
      if (lane == 0) prefix[static_cast<size_t>(w) * n + i] = pre;
    }
  }
  __syncwarp();                                    // the next window reuses the warp's shared memory
  }
}

// sum_a e[a] * exp(A[a][lane]) for lane < r: e (r floats) and the table A [r, r] are in shared memory. Every lane reads
// four e's per request (a broadcast) and keeps four independent accumulation chains.
__device__ __forceinline__ float hmm_matvec(const float* evec, const float* A, int lane, int r) {
  float s = 0.f;
  if ((r & 3) == 0) {
    const float4* e4 = reinterpret_cast<const float4*>(evec);
    float s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 4
    for (int a = 0; a < r; a += 4) {
      const float4 ev = e4[a >> 2];
      s = fmaf(ev.x, __expf(A[a * r + lane]), s);
      s1 = fmaf(ev.y, __expf(A[(a + 1) * r + lane]), s1);
      s2 = fmaf(ev.z, __expf(A[(a + 2) * r + lane]), s2);
      s3 = fmaf(ev.w, __expf(A[(a + 3) * r + lane]), s3);
    }
    s = (s + s1) + (s2 + s3);
  } else {
    for (int a = 0; a < r; ++a) s = fmaf(evec[a], __expf(A[a * r + lane]), s);
  }
  return s;
}

// Eq. (HMM), forward recursion over the window: alpha_0[k] = log pi[k] + G[0,k];
// alpha_i[k] = G[i,k] + LSE_a(alpha_{i-1}[a] + logA_i[a][k]); out = LSE_k alpha_{n-1}[k].  r <= 32.
// The inner log-sum-exp is taken as one scaled matrix-vector product per step: with m = max_a alpha_{i-1}[a],
// alpha_i[k] = G[i,k] + m + log sum_a exp(alpha_{i-1}[a] - m) exp(logA_i[a][k]).
// The transition tables are streamed per window: position p = w / wpp reads logA_i[a][k] at
// tables[p * table_stride + (i-1) r^2 + a r + k]. Contextual transitions (App. H): tables = log omega + r and
// table_stride = sum_rows, 28 KB per position at n = 8, r = 32, read exactly once from HBM, which bounds the kernel.
// Static transitions: table_stride = 0, the one set of tables stays in L2. One warp per window, lane = state; table
// i+1 is copied into shared memory by cp.async while table i is reduced (kHmmDepth buffers per warp).
// Shared memory per warp: kHmmDepth * r * r + 32 floats. With `prefix` (may be NULL) also writes prefix[w, i] = LSE_k alpha_i[k].
constexpr int kHmmDepth = 2;   // table buffers per warp (deeper pipelines were measured and bought nothing)
__global__ void circuit_hmm_stream_kernel(const float* __restrict__ G, const float* __restrict__ logw,
                                          const float* __restrict__ tables, int table_stride,
                                          float* __restrict__ out, float* __restrict__ prefix, unsigned* work_counter,
                                          int W, int wpp, int n, int r, int sum_rows) {
  extern __shared__ __align__(16) float sm[];
  grid_dependency_wait();   // G, log omega and the zeroed work counter come from the kernels before this one
  const int lane = threadIdx.x & 31;
  const int rr = r * r;
  float* tabs = sm + static_cast<size_t>(threadIdx.x >> 5) * (kHmmDepth * rr + 32);
  float* evec = tabs + kHmmDepth * rr;
  const bool has = lane < r;
  for (int w = next_window(work_counter, lane); w < W; w = next_window(work_counter, lane)) {
    const float* g = G + static_cast<size_t>(w) * n * r;
    const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
    const float* tb = tables + static_cast<size_t>(w / wpp) * table_stride;   // logA_1 .. logA_{n-1} of this position
    // kHmmDepth - 1 tables are in flight ahead of the one being reduced; every step commits exactly one copy group (an
    // empty one once the tables run out), so "all but the newest kHmmDepth - 1 groups" always means "table i has landed"
#pragma unroll
    for (int s = 0; s < kHmmDepth - 1; ++s) {
      if (s < n - 1) warp_table_load_async(tabs + s * rr, tb + static_cast<size_t>(s) * rr, rr, lane);
      else cp_async_commit();
    }
    float alpha = has ? lw[lane] + g[lane] : -CUDART_INF_F;
    for (int i = 1; i < n; ++i) {
      const int nxt = i - 1 + kHmmDepth - 1;                 // index of the table to fetch now
      if (nxt < n - 1) warp_table_load_async(tabs + (nxt % kHmmDepth) * rr, tb + static_cast<size_t>(nxt) * rr, rr, lane);
      else cp_async_commit();
      cp_async_wait<kHmmDepth - 1>();
      __syncwarp();                                      // table i is in shared memory for every lane
      if (prefix != nullptr) {
        const float pre = warp_lse(alpha, has);
        if (lane == 0) prefix[static_cast<size_t>(w) * n + i - 1] = pre;
      }
      const float* A = tabs + ((i - 1) % kHmmDepth) * rr;
      const float gi = has ? g[i * r + lane] : 0.f;
      float m = alpha;
      const bool poisoned = __any_sync(kFull, alpha != alpha);   // NaN evidence (a target or a draw that was refused)
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, off));
      // e[a] = exp(alpha[a] - m) goes through shared memory: every lane then reads four of them per request
      // (a broadcast) instead of one shuffle each
      evec[lane] = has ? __expf(alpha - m) : 0.f;
      __syncwarp();
      if (has) {
        const float s = hmm_matvec(evec, A, lane, r);
        alpha = (m == -CUDART_INF_F) ? -CUDART_INF_F : gi + m + __logf(s);
        if (poisoned) alpha = CUDART_NAN_F;              // the max above skips NaN: it would be lost when every state is NaN
      }
      __syncwarp();                                      // the buffers may be overwritten
    }
    const float res = warp_lse(alpha, has);
    if (lane == 0) {
      if (out != nullptr) out[w] = res;
      if (prefix != nullptr) prefix[static_cast<size_t>(w) * n + n - 1] = res;
    }
  }
}

// ---------------------------------------------------------------- latent draws (Algorithm 1, sum units)
// Inverse CDF over r log-probabilities: the smallest j with u < p_0 + ... + p_j, else r - 1.
__device__ __forceinline__ int inv_cdf_logp(const float* __restrict__ logp, int r, float u) {
  float cum = 0.f;
  int found = r - 1;
  bool hit = false;
  for (int j = 0; j < r; ++j) {
    cum += expf(logp[j]);
    if (!hit && u < cum) { hit = true; found = j; }
  }
  return found;
}

// One thread per window. Writes unit_sel[w, i] = the input unit chosen for token i and presets out_bytes to -1.
__global__ void latent_sample_kernel(int family, const float* __restrict__ logw, const float* __restrict__ logA,
                                     const float* __restrict__ uniforms, int* __restrict__ unit_sel,
                                     int* __restrict__ out_bytes, unsigned* status, int W, int wpp, int n, int r,
                                     int sum_rows, int logA_stride) {
  const int w = blockIdx.x * blockDim.x + threadIdx.x;
  if (w >= W) return;
  const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
  const float* u = uniforms + static_cast<size_t>(w) * 2 * n;
  int* sel = unit_sel + static_cast<size_t>(w) * n;
  bool bad = false;
  for (int i = 0; i < n; ++i) out_bytes[static_cast<size_t>(w) * n + i] = -1;
  const int nlat = (family == 0) ? 1 : (family == 1 ? n : n - 1);
  for (int i = 0; i < nlat; ++i) bad |= !(u[i] >= 0.f && u[i] < 1.f);
  if (bad) {
    atomicOr(status, 2u);
    for (int i = 0; i < n; ++i) sel[i] = -1;
    return;
  }
  if (family == 0) {
    const int z = inv_cdf_logp(lw, r, u[0]);
    for (int i = 0; i < n; ++i) sel[i] = z;
  } else if (family == 1) {
    int z = inv_cdf_logp(lw, r, u[0]);
    sel[0] = z;
    for (int i = 1; i < n; ++i) {
      z = inv_cdf_logp(logA + static_cast<size_t>(w / wpp) * logA_stride + (static_cast<size_t>(i - 1) * r + z) * r, r, u[i]);
      sel[i] = z;
    }
  } else {
    int zs[63];
    zs[0] = inv_cdf_logp(lw, r, u[0]);
    for (int j = 1; j < n - 1; ++j)
      zs[j] = inv_cdf_logp(lw + r + (static_cast<size_t>(j - 1) * r + zs[(j - 1) >> 1]) * r, r, u[j]);
    for (int i = 0; i < n; ++i) sel[i] = zs[n / 2 - 1 + (i >> 1)];
  }
}

// ---------------------------------------------------------------- training loss (Eq. 6)
// Eq. (6): L_j = -(1/N) sum_i (1/V_ij) sum_t log p(x_{t+j} | x_{<t+j}), L = sum_j gamma^(j-1) L_j, over N sequences of
// L positions with overlapping windows. The conditional of slot j given the context and the window's earlier bytes
// is the difference of consecutive prefix log-marginals; V_ij counts the valid (non-negative) targets of slot j in
// sequence i. Two kernels, both with a fixed reduction order, so the result does not change from run to run.
constexpr int kLossThreads = 256;

// grid = N. partial[i, j] = (1/V_ij) sum_{t valid} (prefix[t, j] - prefix[t, j-1]), 0 if V_ij = 0.
__global__ void __launch_bounds__(kLossThreads) loss_partial_kernel(const float* __restrict__ prefix,
                                                                    const int* __restrict__ targets,
                                                                    float* __restrict__ partial, int L, int n) {
  __shared__ float ssum[kLossThreads / 32];
  __shared__ int scnt[kLossThreads / 32];
  const int i = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int j = 0; j < n; ++j) {
    float sum = 0.f;
    int cnt = 0;
    for (int t = threadIdx.x; t < L; t += kLossThreads) {
      const size_t row = (static_cast<size_t>(i) * L + t) * n;
      if (targets[row + j] >= 0) {
        sum += prefix[row + j] - (j > 0 ? prefix[row + j - 1] : 0.f);
        cnt += 1;
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      sum += __shfl_xor_sync(kFull, sum, off);
      cnt += __shfl_xor_sync(kFull, cnt, off);
    }
    if (lane == 0) { ssum[warp] = sum; scnt[warp] = cnt; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      int c = 0;
      for (int q = 0; q < kLossThreads / 32; ++q) { tot += ssum[q]; c += scnt[q]; }
      partial[static_cast<size_t>(i) * n + j] = c > 0 ? tot / static_cast<float>(c) : 0.f;
    }
    __syncthreads();
  }
}

// One CTA; warp q reduces the slots q, q + warps, ...: slot_loss[j] = -(1/N) sum_i partial[i, j]; then
// loss = sum_j gamma^j slot_loss[j] (j counted from 0).
__global__ void __launch_bounds__(kLossThreads) loss_final_kernel(const float* __restrict__ partial,
                                                                  float* __restrict__ slot_loss,
                                                                  float* __restrict__ loss, int N, int n, float gamma) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int j = warp; j < n; j += kLossThreads / 32) {
    float sum = 0.f;
    for (int i = lane; i < N; i += 32) sum += partial[static_cast<size_t>(i) * n + j];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(kFull, sum, off);
    if (lane == 0) slot_loss[j] = -sum / static_cast<float>(N);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f, wgt = 1.f;
    for (int j = 0; j < n; ++j) { tot += wgt * slot_loss[j]; wgt *= gamma; }
    *loss = tot;
  }
}

// Coefficients of the prefix log-marginals in Eq. (6). With c[t, j] = -gamma^j / (N V_ij) for a valid target (i the
// sequence of position t) and 0 otherwise, L = sum_t sum_j c[t, j] (P[t, j] - P[t, j-1]) = sum_t sum_j coeff[t, j] P[t, j]
// with coeff[t, j] = c[t, j] - c[t, j+1] (c[t, n] = 0): the weights of the n backward passes. grid = N, n <= 64.
__global__ void __launch_bounds__(kLossThreads) loss_coeff_kernel(const int* __restrict__ targets,
                                                                  float* __restrict__ coeff, int L, int n, int N,
                                                                  float gamma) {
  __shared__ int scnt[kLossThreads / 32];
  __shared__ float cj[64];
  const int i = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float wgt = 1.f;
  for (int j = 0; j < n; ++j) {
    int cnt = 0;
    for (int t = threadIdx.x; t < L; t += kLossThreads) cnt += targets[(static_cast<size_t>(i) * L + t) * n + j] >= 0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(kFull, cnt, off);
    if (lane == 0) scnt[warp] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
      int c = 0;
      for (int q = 0; q < kLossThreads / 32; ++q) c += scnt[q];
      cj[j] = c > 0 ? -wgt / (static_cast<float>(N) * static_cast<float>(c)) : 0.f;
    }
    wgt *= gamma;
    __syncthreads();
  }
  for (int t = threadIdx.x; t < L; t += kLossThreads) {
    const size_t row = (static_cast<size_t>(i) * L + t) * n;
    for (int j = 0; j < n; ++j) {
      const float here = targets[row + j] >= 0 ? cj[j] : 0.f;
      const float next = (j + 1 < n && targets[row + j + 1] >= 0) ? cj[j + 1] : 0.f;
      coeff[row + j] = here - next;
    }
  }
}

// ---------------------------------------------------------------- preparation
__global__ void f32_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t count) {
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (; i < count; i += stride) dst[i] = __float2bfloat16_rn(src[i]);
}

// Row-wise log-softmax of the static transition logits: one thread per row of r entries.
__global__ void log_softmax_rows_kernel(const float* __restrict__ src, float* __restrict__ dst, int rows, int r) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const float* x = src + static_cast<size_t>(row) * r;
  float m = x[0];
  for (int j = 1; j < r; ++j) m = fmaxf(m, x[j]);
  float s = 0.f;
  for (int j = 0; j < r; ++j) s += expf(x[j] - m);
  const float lse = m + logf(s);
  for (int j = 0; j < r; ++j) dst[static_cast<size_t>(row) * r + j] = x[j] - lse;
}

}  // namespace mtpc
