// Low-rank-adapted unembeddings (App. G, "Unembedding parameter sharing"): the unembedding matrix of token i and
// component j is U[i, j] = W[i] + A[i, j] B[i, j], with W[i] [v, d] shared by the r components of slot i and a rank-k
// adaptor A[i, j] [v, k], B[i, j] [k, d]. The head itself keeps working on the composed tensor U [n, r, v, d] (bf16): these
// kernels build it from the shared parameters and carry the gradient of U back to them.
//
// All four are streaming kernels over the [n r, v, d] tensor (U or its gradient) with k multiply-adds per element on
// the CUDA cores: every thread owns a few adjacent columns (vector loads) and a block of rows or of ranks, so that
// the small operand (a tile of A or B) is read once per register tile, from shared memory. CV is the number of
// adjacent columns per thread: the vector width when d and the pointers allow it, else 1.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace mtpc {

constexpr int kLowRankThreads = 256;
constexpr int kLowRankMaxK = 64;
constexpr int kComposeRows = 8;      // rows of U in a thread's register tile in the composition
constexpr int kComposeCtaRows = 32;  // rows of U a CTA of the composition walks
constexpr int kRankChunk = 16;       // ranks per register tile in the gradient kernels
constexpr int kDaCols = 512;         // columns of B staged per step of lowrank_da_kernel
constexpr int kDbRows = 256;         // rows of A staged per step of lowrank_db_kernel

inline size_t compose_smem_bytes(int k, int cv) {
  return static_cast<size_t>(k) * (kLowRankThreads * cv * 2 + kComposeCtaRows * 4);
}

template <int CV>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, float (&out)[CV]) {
  if constexpr (CV == 4) {
    const uint2 raw = *reinterpret_cast<const uint2*>(p);
    const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
    const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
    out[0] = lo.x, out[1] = lo.y, out[2] = hi.x, out[3] = hi.y;
  } else {
#pragma unroll
    for (int t = 0; t < CV; ++t) out[t] = __bfloat162float(p[t]);
  }
}

template <int CV>
__device__ __forceinline__ void load_f32(const float* p, float (&out)[CV]) {
  if constexpr (CV == 4) {
    const float4 x = *reinterpret_cast<const float4*>(p);
    out[0] = x.x, out[1] = x.y, out[2] = x.z, out[3] = x.w;
  } else if constexpr (CV == 2) {
    const float2 x = *reinterpret_cast<const float2*>(p);
    out[0] = x.x, out[1] = x.y;
  } else {
#pragma unroll
    for (int t = 0; t < CV; ++t) out[t] = p[t];
  }
}

template <int CV>
__device__ __forceinline__ void store_f32(float* p, const float (&x)[CV]) {
  if constexpr (CV == 4) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  } else if constexpr (CV == 2) {
    *reinterpret_cast<float2*>(p) = make_float2(x[0], x[1]);
  } else {
#pragma unroll
    for (int t = 0; t < CV; ++t) p[t] = x[t];
  }
}

// U[i, j, b, c] = bf16( W[i, b, c] + sum_q A[i, j, b, q] B[i, j, q, c] ), fp32 accumulation in the order q = 0..k-1.
// grid = (ceil(d / (256 CV)), ceil(v / 32), n r). A thread owns CV columns: it fetches its k values of B per column
// once (all loads in flight together, parked in its own slots of shared memory), then walks 4 blocks of 8 rows, the
// next block's rows of W prefetched while the current one is computed. Dynamic shared memory:
// compose_smem_bytes(k, CV).
template <int CV>
__global__ void __launch_bounds__(kLowRankThreads) lowrank_compose_kernel(const __nv_bfloat16* __restrict__ W,
                                                                         const __nv_bfloat16* __restrict__ A,
                                                                         const __nv_bfloat16* __restrict__ B,
                                                                         __nv_bfloat16* __restrict__ U, int r, int v,
                                                                         int d, int k) {
  extern __shared__ __align__(16) unsigned char lowrank_smem[];
  __nv_bfloat16* b_s = reinterpret_cast<__nv_bfloat16*>(lowrank_smem);                       // [k][256 CV]
  float* a_s = reinterpret_cast<float*>(lowrank_smem + static_cast<size_t>(k) * kLowRankThreads * CV * 2);  // [k][32]
  const int unit = blockIdx.z, i = unit / r;
  const int row0 = blockIdx.y * kComposeCtaRows;
  const int c = (blockIdx.x * kLowRankThreads + threadIdx.x) * CV;
  const bool in = c < d;
  {
    const __nv_bfloat16* Bu = B + static_cast<size_t>(unit) * k * d + c;
    __nv_bfloat16* mine = b_s + threadIdx.x * CV;
#pragma unroll 8
    for (int q = 0; q < k; ++q, Bu += d, mine += kLowRankThreads * CV) {
      if constexpr (CV == 4) {
        *reinterpret_cast<uint2*>(mine) = in ? *reinterpret_cast<const uint2*>(Bu) : make_uint2(0u, 0u);
      } else {
#pragma unroll
        for (int t = 0; t < CV; ++t) mine[t] = in ? Bu[t] : __float2bfloat16_rn(0.f);
      }
    }
  }
  for (int e = threadIdx.x; e < k * kComposeCtaRows; e += kLowRankThreads) {
    const int q = e / kComposeCtaRows, rr = e % kComposeCtaRows;
    a_s[e] = row0 + rr < v ? __bfloat162float(A[(static_cast<size_t>(unit) * v + row0 + rr) * k + q]) : 0.f;
  }
  __syncthreads();
  if (!in) return;
  const __nv_bfloat16* Wi = W + static_cast<size_t>(i) * v * d + c;
  struct alignas(2 * CV) Raw { __nv_bfloat16 e[CV]; };               // CV bf16 values as they lie in memory
  auto load_w = [&](int b0, Raw (&w)[kComposeRows]) {
#pragma unroll
    for (int rr = 0; rr < kComposeRows; ++rr) {
      if (b0 + rr < v) {
        w[rr] = *reinterpret_cast<const Raw*>(Wi + static_cast<size_t>(b0 + rr) * d);
      } else {
#pragma unroll
        for (int t = 0; t < CV; ++t) w[rr].e[t] = __float2bfloat16_rn(0.f);
      }
    }
  };
  Raw wn[kComposeRows];
  load_w(row0, wn);
  for (int rb = 0; rb < kComposeCtaRows / kComposeRows; ++rb) {
    const int b0 = row0 + rb * kComposeRows;
    if (b0 >= v) break;
    // Accumulators as pairs of adjacent rows: one packed fp32 multiply-add (two independent round-to-nearest FMAs)
    // takes the pair of A values as they lie in shared memory and the B value twice.
    float2 acc[kComposeRows / 2][CV];
#pragma unroll
    for (int rr = 0; rr < kComposeRows; ++rr) {
      float w[CV];
      load_bf16<CV>(wn[rr].e, w);
#pragma unroll
      for (int t = 0; t < CV; ++t) (rr & 1 ? acc[rr / 2][t].y : acc[rr / 2][t].x) = w[t];
    }
    load_w(b0 + kComposeRows, wn);                                  // beyond the last row: zeros, never stored
    const __nv_bfloat16* mine = b_s + threadIdx.x * CV;
    const float* arow = a_s + rb * kComposeRows;
#pragma unroll 4
    for (int q = 0; q < k; ++q, mine += kLowRankThreads * CV, arow += kComposeCtaRows) {
      float bv[CV];
      load_bf16<CV>(mine, bv);
      float2 b2[CV];
#pragma unroll
      for (int t = 0; t < CV; ++t) b2[t] = make_float2(bv[t], bv[t]);
#pragma unroll
      for (int r4 = 0; r4 < kComposeRows; r4 += 4) {
        const float4 a = *reinterpret_cast<const float4*>(arow + r4);
        const float2 a01 = make_float2(a.x, a.y), a23 = make_float2(a.z, a.w);
#pragma unroll
        for (int t = 0; t < CV; ++t) {
          acc[r4 / 2][t] = __ffma2_rn(a01, b2[t], acc[r4 / 2][t]);
          acc[r4 / 2 + 1][t] = __ffma2_rn(a23, b2[t], acc[r4 / 2 + 1][t]);
        }
      }
    }
#pragma unroll
    for (int rr = 0; rr < kComposeRows; ++rr) {
      if (b0 + rr >= v) break;
      float o[CV];
#pragma unroll
      for (int t = 0; t < CV; ++t) o[t] = rr & 1 ? acc[rr / 2][t].y : acc[rr / 2][t].x;
      __nv_bfloat16* dst = U + (static_cast<size_t>(unit) * v + b0 + rr) * d + c;
      if constexpr (CV == 4) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(o[0], o[1]);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(o[2], o[3]);
        *reinterpret_cast<uint2*>(dst) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
      } else {
#pragma unroll
        for (int t = 0; t < CV; ++t) dst[t] = __float2bfloat16_rn(o[t]);
      }
    }
  }
}

// dW[i, b, c] = sum_j dU[i, j, b, c].  grid = (ceil(d / (256 CV)), v, n).
template <int CV>
__global__ void __launch_bounds__(kLowRankThreads) lowrank_dw_kernel(const float* __restrict__ dU, float* __restrict__ dW,
                                                                    int r, int v, int d) {
  const int i = blockIdx.z, b = blockIdx.y;
  const int c = (blockIdx.x * kLowRankThreads + threadIdx.x) * CV;
  if (c >= d) return;
  float acc[CV];
#pragma unroll
  for (int t = 0; t < CV; ++t) acc[t] = 0.f;
#pragma unroll 4
  for (int j = 0; j < r; ++j) {
    float x[CV];
    load_f32<CV>(dU + ((static_cast<size_t>(i) * r + j) * v + b) * d + c, x);
#pragma unroll
    for (int t = 0; t < CV; ++t) acc[t] += x[t];
  }
  store_f32<CV>(dW + (static_cast<size_t>(i) * v + b) * d + c, acc);
}

// dA[i, j, b, q] = sum_c dU[i, j, b, c] B[i, j, q, c].  grid = (ceil(v / 32), n r); a warp owns 4 rows and every column,
// a lane CV adjacent columns of each 32 CV-wide stripe; 16 ranks at a time, their rows of B staged 512 columns at a
// time in shared memory (as fp32). The lanes' partial sums meet in a butterfly at the end of each block of ranks.
template <int CV>
__global__ void __launch_bounds__(kLowRankThreads, 2) lowrank_da_kernel(const float* __restrict__ dU,
                                                                       const __nv_bfloat16* __restrict__ B,
                                                                       float* __restrict__ dA, int v, int d, int k) {
  __shared__ __align__(16) float b_s[kRankChunk][kDaCols];          // fp32: converted once per stripe, not once per use
  constexpr int kIters = kDaCols / (32 * CV);                     // column groups of a lane per stripe
  const int unit = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b0 = blockIdx.x * 32 + warp * 4;
  const float* rows = dU + (static_cast<size_t>(unit) * v + b0) * d;
  auto load_x = [&](int col, float (&x)[4][CV]) {                  // zeros beyond the last row or column
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      if (b0 + rr < v && col < d) {
        load_f32<CV>(rows + static_cast<size_t>(rr) * d + col, x[rr]);
      } else {
#pragma unroll
        for (int t = 0; t < CV; ++t) x[rr][t] = 0.f;
      }
    }
  };
  for (int q0 = 0; q0 < k; q0 += kRankChunk) {
    float acc[4][kRankChunk];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
      for (int q = 0; q < kRankChunk; ++q) acc[rr][q] = 0.f;
    float x[4][CV];
    load_x(lane * CV, x);
    for (int c0 = 0; c0 < d; c0 += kDaCols) {
      __syncthreads();                                            // the previous stripe has been consumed
      for (int e = threadIdx.x * CV; e < kRankChunk * kDaCols; e += kLowRankThreads * CV) {
        const int q = e / kDaCols, cc = e % kDaCols;
        const bool in = q0 + q < k && c0 + cc < d;               // d is a multiple of CV: the CV columns are in or out together
        float bv[CV];
        if (in) {
          load_bf16<CV>(B + (static_cast<size_t>(unit) * k + q0 + q) * d + c0 + cc, bv);
        } else {
#pragma unroll
          for (int t = 0; t < CV; ++t) bv[t] = 0.f;
        }
        store_f32<CV>(&b_s[q][cc], bv);
      }
      __syncthreads();
#pragma unroll
      for (int it = 0; it < kIters; ++it) {
        const int cc = (it * 32 + lane) * CV;
        float xn[4][CV];                                          // the lane's next columns (of this stripe or the next one)
        load_x(c0 + cc + 32 * CV, xn);
#pragma unroll
        for (int q = 0; q < kRankChunk; ++q) {
          float bv[CV];
          load_f32<CV>(&b_s[q][cc], bv);
#pragma unroll
          for (int rr = 0; rr < 4; ++rr)
#pragma unroll
            for (int t = 0; t < CV; ++t) acc[rr][q] = fmaf(x[rr][t], bv[t], acc[rr][q]);
        }
#pragma unroll
        for (int rr = 0; rr < 4; ++rr)
#pragma unroll
          for (int t = 0; t < CV; ++t) x[rr][t] = xn[rr][t];
      }
    }
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
      for (int q = 0; q < kRankChunk; ++q) {
        float s = acc[rr][q];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0 && b0 + rr < v && q0 + q < k) dA[(static_cast<size_t>(unit) * v + b0 + rr) * k + q0 + q] = s;
      }
  }
}

// dB[i, j, q, c] = sum_b A[i, j, b, q] dU[i, j, b, c].  grid = (ceil(d / (256 CV)), ceil(k / 16), n r): a thread owns
// CV columns x 16 ranks and walks the v rows in order; 256 rows of A at a time sit in shared memory (fp32).
template <int CV>
__global__ void __launch_bounds__(kLowRankThreads, 2) lowrank_db_kernel(const float* __restrict__ dU,
                                                                    const __nv_bfloat16* __restrict__ A,
                                                                    float* __restrict__ dB, int v, int d, int k) {
  __shared__ __align__(16) float a_s[kDbRows][kRankChunk];
  const int unit = blockIdx.z, q0 = blockIdx.y * kRankChunk;
  const int c = (blockIdx.x * kLowRankThreads + threadIdx.x) * CV;
  float acc[kRankChunk][CV];
#pragma unroll
  for (int q = 0; q < kRankChunk; ++q)
#pragma unroll
    for (int t = 0; t < CV; ++t) acc[q][t] = 0.f;
  for (int b0 = 0; b0 < v; b0 += kDbRows) {
    __syncthreads();                                              // the previous block of rows has been consumed
    for (int e = threadIdx.x; e < kDbRows * kRankChunk; e += kLowRankThreads) {
      const int bb = e / kRankChunk, q = e % kRankChunk;
      a_s[bb][q] = b0 + bb < v && q0 + q < k ? __bfloat162float(A[(static_cast<size_t>(unit) * v + b0 + bb) * k + q0 + q]) : 0.f;
    }
    __syncthreads();
    if (c < d) {
      const int rows = min(kDbRows, v - b0);
      const float* g = dU + (static_cast<size_t>(unit) * v + b0) * d + c;
#pragma unroll 4
      for (int bb = 0; bb < rows; ++bb) {
        float x[CV];
        load_f32<CV>(g + static_cast<size_t>(bb) * d, x);
#pragma unroll
        for (int q4 = 0; q4 < kRankChunk; q4 += 4) {
          const float4 a = *reinterpret_cast<const float4*>(&a_s[bb][q4]);
          const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int t = 0; t < CV; ++t) acc[q4 + u][t] = fmaf(av[u], x[t], acc[q4 + u][t]);
        }
      }
    }
  }
  if (c >= d) return;
#pragma unroll
  for (int q = 0; q < kRankChunk; ++q)
    if (q0 + q < k) store_f32<CV>(dB + (static_cast<size_t>(unit) * k + q0 + q) * d + c, acc[q]);
}

}  // namespace mtpc
