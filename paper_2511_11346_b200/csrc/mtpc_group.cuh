// Grouping of the byte draws of a many-position draft by the input unit they sample from (Algorithm 1, input-unit
// step). After the latent draws every (window, slot) pair knows its unit (i, z). A counting sort over the n*r units
// packs the hidden states of the pairs that share a unit into consecutive rows of a staging buffer, so that the
// sampling pass of the projection kernel multiplies each pair by the one unit it samples from: windows * n * v * d
// multiply-adds instead of positions * n * r * v * d.
//   group_count_kernel   histogram of the pairs over the units
//   group_scan_kernel    exclusive scan -> first staging row of every unit, and the list of 128-row tiles
//   group_gather_kernel  every pair takes the next free row of its unit and copies its hidden state there
// The order of the pairs inside a unit depends on the order of the atomic increments; nothing downstream depends on it
// (every row is sampled on its own, with its own uniform).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace mtpc {

constexpr int kGroupThreads = 256;
constexpr int kGroupScanThreads = 1024;
constexpr int kGroupMaxUnits = 8192;    // n <= 64 slots x r <= 128 units

// One tile of the grouped sampling pass: `count` <= 128 staging rows starting at `row0`, all sampling from emission
// unit `unit` (= slot * r + component).
struct GroupTile {
  int unit, row0, count, pad;
};

// counts[unit] += 1 for every (window, slot) pair with a selected unit (pairs of windows whose latent draw was refused
// have none). Shared-memory histogram per CTA, flushed once.
__global__ void __launch_bounds__(kGroupThreads) group_count_kernel(const int* __restrict__ unit_sel,
                                                                    int* __restrict__ counts, int entries, int n, int r) {
  extern __shared__ int hist[];
  const int units = n * r;
  for (int k = threadIdx.x; k < units; k += kGroupThreads) hist[k] = 0;
  __syncthreads();
  for (int e = blockIdx.x * kGroupThreads + threadIdx.x; e < entries; e += gridDim.x * kGroupThreads) {
    const int z = unit_sel[e];
    if (z >= 0) atomicAdd(&hist[(e % n) * r + z], 1);
  }
  __syncthreads();
  for (int k = threadIdx.x; k < units; k += kGroupThreads)
    if (hist[k]) atomicAdd(&counts[k], hist[k]);
}

// One CTA. offsets[u] = number of pairs in the units before u; tiles = every unit cut into runs of <= 128 rows, in
// unit order; *num_tiles = how many. Thread t owns the units [t * per, (t + 1) * per).
__global__ void __launch_bounds__(kGroupScanThreads) group_scan_kernel(const int* __restrict__ counts,
                                                                       int* __restrict__ offsets,
                                                                       GroupTile* __restrict__ tiles,
                                                                       int* __restrict__ num_tiles, int units) {
  __shared__ int warp_rows[kGroupScanThreads / 32], warp_tiles[kGroupScanThreads / 32];
  const int per = (units + kGroupScanThreads - 1) / kGroupScanThreads;
  const int u0 = threadIdx.x * per;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int rows = 0, ntl = 0;
  for (int q = 0; q < per; ++q) {
    const int c = (u0 + q < units) ? counts[u0 + q] : 0;
    rows += c;
    ntl += (c + 127) >> 7;
  }
  // inclusive scan of (rows, tiles) over the CTA: within the warp by shuffles, across warps through shared memory
  int rs = rows, ts = ntl;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, rs, off);
    const int b = __shfl_up_sync(0xffffffffu, ts, off);
    if (lane >= off) { rs += a; ts += b; }
  }
  if (lane == 31) { warp_rows[warp] = rs; warp_tiles[warp] = ts; }
  __syncthreads();
  if (warp == 0) {
    int a = warp_rows[lane], b = warp_tiles[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, a, off);
      const int y = __shfl_up_sync(0xffffffffu, b, off);
      if (lane >= off) { a += x; b += y; }
    }
    warp_rows[lane] = a;
    warp_tiles[lane] = b;
    if (lane == 31) *num_tiles = b;
  }
  __syncthreads();
  int row = rs - rows + (warp ? warp_rows[warp - 1] : 0);     // exclusive prefix of this thread's first unit
  int tile = ts - ntl + (warp ? warp_tiles[warp - 1] : 0);
  for (int q = 0; q < per; ++q) {
    const int u = u0 + q;
    if (u >= units) break;
    const int c = counts[u];
    offsets[u] = row;
    for (int done = 0; done < c; done += 128) {
      GroupTile t;
      t.unit = u;
      t.row0 = row + done;
      t.count = c - done < 128 ? c - done : 128;
      t.pad = 0;
      tiles[tile++] = t;
    }
    row += c;
  }
}

// One warp per (window, slot) pair: lane 0 takes the next free staging row of the pair's unit, the warp copies the
// window's hidden state (d bf16, d a multiple of 8, rows 16-byte aligned) there and records which pair the row holds
// (and, where row_of is given, which row a pair got).
__global__ void __launch_bounds__(kGroupThreads) group_gather_kernel(const int* __restrict__ unit_sel,
                                                                     const __nv_bfloat16* __restrict__ hidden,
                                                                     const int* __restrict__ offsets,
                                                                     int* __restrict__ cursors, int* __restrict__ perm,
                                                                     __nv_bfloat16* __restrict__ stage, int entries, int n,
                                                                     int r, int wpp, int d, int* __restrict__ row_of) {
  const int lane = threadIdx.x & 31;
  const int warps = gridDim.x * (kGroupThreads / 32);
  const int vecs = d / 8;                                      // 16-byte pieces per row
  for (int e = blockIdx.x * (kGroupThreads / 32) + (threadIdx.x >> 5); e < entries; e += warps) {
    const int z = unit_sel[e];
    if (z < 0) continue;                                       // warp-uniform: the whole warp reads the same entry
    int row = 0;
    if (lane == 0) {
      const int u = (e % n) * r + z;
      row = offsets[u] + atomicAdd(&cursors[u], 1);
      perm[row] = e;
      if (row_of != nullptr) row_of[e] = row;                  // the inverse map, for callers that look a pair's row up
    }
    row = __shfl_sync(0xffffffffu, row, 0);
    const uint4* src = reinterpret_cast<const uint4*>(hidden + static_cast<size_t>((e / n) / wpp) * d);
    uint4* dst = reinterpret_cast<uint4*>(stage + static_cast<size_t>(row) * d);
    for (int q = lane; q < vecs; q += 32) dst[q] = src[q];
  }
}

}  // namespace mtpc
