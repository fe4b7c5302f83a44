// Circuit evaluation in log space (Eq. CP, Eq. HMM, Eq. BTree), latent ancestral sampling (Algorithm 1, sum
// units) and the small preparation kernels. One warp evaluates one window; lane = latent value.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>
#include <stdint.h>

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
                                  int sum_rows) {
  const int w = blockIdx.x * kCircuitWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= W) return;
  const float* g = G + static_cast<size_t>(w) * n * r;
  const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
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
      last = m + __logf(s);
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
  if (lane == 0) out[w] = m + __logf(s);
}

// Eq. (HMM), forward recursion over the window: alpha_0[k] = log pi[k] + G[0,k];
// alpha_i[k] = G[i,k] + LSE_a(alpha_{i-1}[a] + logA[i-1][a][k]); out = LSE_k alpha_{n-1}[k].  r <= 32.
// The inner log-sum-exp is taken as one scaled matrix-vector product per step: with m = max_a alpha_{i-1}[a],
// alpha_i[k] = G[i,k] + m + log sum_a exp(alpha_{i-1}[a] - m) A[i-1][a][k], A = exp(logA) staged once per CTA in
// shared memory ((n-1) r^2 floats; read straight from global memory when that does not fit). One warp per
// window, lane = state; CTAs stride over the windows. With `prefix` (may be NULL) the kernel also writes
// prefix[w, i] = log q(x_0..x_i) = LSE_k alpha_i[k]. Contextual transitions (App. H): logA = log omega + r and
// logA_stride = sum_rows, so that position p reads its own tables (never staged: tables_in_smem = 0).
__global__ void circuit_hmm_kernel(const float* __restrict__ G, const float* __restrict__ logw,
                                   const float* __restrict__ logA, float* __restrict__ out,
                                   float* __restrict__ prefix, int W, int wpp, int n, int r, int sum_rows,
                                   int tables_in_smem, int logA_stride) {
  extern __shared__ float A_lin[];
  const int lane = threadIdx.x & 31;
  const int count = (n - 1) * r * r;
  if (tables_in_smem) {
    for (int e = threadIdx.x; e < count; e += blockDim.x) A_lin[e] = __expf(__ldg(logA + e));
    __syncthreads();
  }
  const bool has = lane < r;
  for (int w = blockIdx.x * kCircuitWarps + (threadIdx.x >> 5); w < W; w += gridDim.x * kCircuitWarps) {
    const float* g = G + static_cast<size_t>(w) * n * r;
    const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
    float alpha = has ? lw[lane] + g[lane] : -CUDART_INF_F;
    for (int i = 1; i < n; ++i) {
      if (prefix != nullptr) {   // log q(x_0..x_{i-1}) = LSE_k alpha_{i-1}[k]: the later steps sum to one
        const float pre = warp_lse(alpha, has);
        if (lane == 0) prefix[static_cast<size_t>(w) * n + i - 1] = pre;
      }
      const float gi = has ? g[i * r + lane] : 0.f;
      float m = alpha;                                   // fmaxf drops NaNs; they come back through e below
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, off));
      const float e = has ? __expf(alpha - m) : 0.f;     // NaN if alpha is NaN or if every state is impossible
      float s = 0.f;
      if (tables_in_smem) {
        const float* A = A_lin + static_cast<size_t>(i - 1) * r * r;
        for (int a = 0; a < r; ++a) s = fmaf(__shfl_sync(kFull, e, a), has ? A[a * r + lane] : 0.f, s);
      } else {
        const float* A = logA + static_cast<size_t>(w / wpp) * logA_stride + static_cast<size_t>(i - 1) * r * r;
        for (int a = 0; a < r; ++a) s = fmaf(__shfl_sync(kFull, e, a), has ? __expf(__ldg(A + a * r + lane)) : 0.f, s);
      }
      if (has) alpha = (m == -CUDART_INF_F) ? -CUDART_INF_F : gi + m + __logf(s);
    }
    const float res = warp_lse(alpha, has);
    if (lane == 0) {
      if (out != nullptr) out[w] = res;
      if (prefix != nullptr) prefix[static_cast<size_t>(w) * n + n - 1] = res;
    }
  }
}

// Eq. (BTree), bottom-up over the heap-ordered latent tree. Node j >= 1 has the table
// logOmega_j[a][b] = logw[p, r + (j-1) r^2 + a r + b] (parent's value a, own value b); the deepest internal node
// n/2-1+m multiplies the input units of tokens 2m and 2m+1. prod[j][z] is the product unit under z_j = z.

// One sum layer seen from the parent: returns, for lane = parent value z, LSE_b(logOmega_c[z][b] + pc[b]).
// tab: the child's r x r table in global memory; pc: r floats in shared memory (written before the call; the
// function synchronises the warp); table: r * (r+1) floats of per-warp shared scratch.
__device__ __forceinline__ float btree_sum_layer(const float* __restrict__ tab, const float* pc, float* table,
                                                 int lane, int r) {
  const bool has = lane < r;
  for (int a = 0; a < r; ++a)                      // coalesced rows -> padded shared tile
    if (has) table[a * (r + 1) + lane] = tab[a * r + lane];
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

// Shared memory per warp: (n-1) * r floats of prod + r * (r+1) floats of one staged table; with PREFIX another
// (n-1) * r floats (the sum-layer outputs S[c][z], kept for the prefix passes) + r floats.  r <= 32.
// PREFIX: also writes prefix[w, i] = log q(x_0..x_i). Summing the later bytes out sets their input units to one,
// so every subtree right of token i evaluates to one, every subtree left of it keeps its value, and only the
// nodes on the path from token i's owner to the root have to be re-evaluated.
template <bool PREFIX>
__global__ void circuit_btree_kernel(const float* __restrict__ G, const float* __restrict__ logw,
                                     float* __restrict__ out, float* __restrict__ prefix, int W, int wpp, int n, int r,
                                     int sum_rows) {
  extern __shared__ float sm[];
  const int wib = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int w = blockIdx.x * kCircuitWarps + wib;
  const int per_warp = (n - 1) * r + r * (r + 1) + (PREFIX ? (n - 1) * r + r : 0);
  float* prod = sm + static_cast<size_t>(wib) * per_warp;
  float* table = prod + (n - 1) * r;
  float* S = table + r * (r + 1);                  // PREFIX only
  float* cur = S + (n - 1) * r;                    // PREFIX only
  if (w >= W) return;
  const float* g = G + static_cast<size_t>(w) * n * r;
  const float* lw = logw + static_cast<size_t>(w / wpp) * sum_rows;
  const bool has = lane < r;
  const int first_leaf_node = n / 2 - 1;
  for (int j = n - 2; j >= first_leaf_node; --j) {
    const int m = j - first_leaf_node;
    if (has) prod[j * r + lane] = g[(2 * m) * r + lane] + g[(2 * m + 1) * r + lane];
  }
  __syncwarp();
  for (int j = first_leaf_node - 1; j >= 0; --j) {
    float acc = 0.f;
    for (int side = 0; side < 2; ++side) {
      const int c = 2 * j + 1 + side;
      const float sc = btree_sum_layer(lw + r + static_cast<size_t>(c - 1) * r * r, prod + c * r, table, lane, r);
      if (PREFIX && has) S[c * r + lane] = sc;
      acc += sc;
    }
    if (has) prod[j * r + lane] = acc;
    __syncwarp();
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
