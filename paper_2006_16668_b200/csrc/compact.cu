// Compaction of the filled slots of every expert (Algorithm 2's dispatch restricted to the slots
// that hold a token).  The capacity stage leaves slot_token [E, G, C] with -1 in empty slots - 13 to
// 30 % of them at the paper's shapes - and the grouped GEMMs of the expert FFN would multiply those
// zero rows too.  Here the filled slots of expert e, in (group, position) order, become rows
// 0 .. kept[e]-1 of its block, the row-tile list of the GEMMs follows kept[e], and the combine
// finds a slot's row through slot_crow.  Rows stay in slot order, so results per row are the bits
// the uncompacted form gives.
#include "kernels.cuh"

namespace gshard {

namespace {

constexpr int kCompactThreads = 256;

// One CTA per expert: ordered stream compaction of its G*C slots with ballot / popcount scans.
__global__ void __launch_bounds__(kCompactThreads) compact_kernel(const int32_t* __restrict__ slot_token, int rows,
                                                                  int S, int C, int32_t* __restrict__ crow_token,
                                                                  int32_t* __restrict__ slot_crow,
                                                                  int32_t* __restrict__ kept) {
  __shared__ int warp_count[kCompactThreads / 32];
  __shared__ int running;
  const int e = blockIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const long long base = (long long)e * rows;
  if (threadIdx.x == 0) running = 0;
  __syncthreads();
  for (int r0 = 0; r0 < rows; r0 += kCompactThreads) {
    const int r = r0 + threadIdx.x;
    const int tok = r < rows ? slot_token[base + r] : -1;
    const bool filled = tok >= 0 && tok < S;
    const unsigned ballot = __ballot_sync(0xffffffffu, filled);
    if (lane == 0) warp_count[w] = __popc(ballot);
    __syncthreads();
    int before = running;
    for (int i = 0; i < w; ++i) before += warp_count[i];
    const int j = before + __popc(ballot & ((1u << lane) - 1u));
    if (r < rows) slot_crow[base + r] = filled ? j : -1;
    if (filled) crow_token[base + j] = (r / C) * S + tok;            // global token index g*S + s
    __syncthreads();
    if (threadIdx.x == 0) {
      int add = 0;
      for (int i = 0; i < kCompactThreads / 32; ++i) add += warp_count[i];
      running += add;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) kept[e] = running;
}

// Three exclusive prefixes over the experts (one CTA, in order), each with E + 1 entries, stored one
// after the other in tile_base: [0] of t = ceil(kept / 128), the 128-row tiles of the single-CTA GEMM;
// [1] of t / 2, the 256-row tiles a launch on CTA pairs covers; [2] of t mod 2, the one 128-row tile
// that remains behind them.  Behind the prefixes, for each of the three lists, the expert that owns
// every row tile (max_tiles entries per list).
__global__ void __launch_bounds__(1024) tile_prefix_kernel(const int32_t* __restrict__ kept, int E, int max_tiles,
                                                           int32_t* __restrict__ tile_base) {
  __shared__ int warp_sum[3][32];
  __shared__ int running[3];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (threadIdx.x < 3) running[threadIdx.x] = 0;
  __syncthreads();
  for (int e0 = 0; e0 < E; e0 += 1024) {
    const int e = e0 + threadIdx.x;
    const int tiles = e < E ? (kept[e] + 127) / 128 : 0;
    const int v[3] = {tiles, tiles / 2, tiles % 2};
    int incl[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      incl[k] = v[k];
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl[k], off);
        if (lane >= off) incl[k] += u;
      }
      if (lane == 31) warp_sum[k][w] = incl[k];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      int before = running[k];
      for (int i = 0; i < w; ++i) before += warp_sum[k][i];
      if (e < E) tile_base[(size_t)k * (E + 1) + e] = before + incl[k] - v[k];
    }
    __syncthreads();
    if (threadIdx.x < 3) {
      int add = 0;
      for (int i = 0; i < 32; ++i) add += warp_sum[threadIdx.x][i];
      running[threadIdx.x] += add;
    }
    __syncthreads();
  }
  if (threadIdx.x < 3) tile_base[(size_t)threadIdx.x * (E + 1) + E] = running[threadIdx.x];
  // tile_problem lists behind the prefixes, max_tiles entries each: the expert that owns every row tile
  __syncthreads();
  int32_t* tile_problem = tile_base + 3 * (size_t)(E + 1);
  for (int e = threadIdx.x; e < E; e += 1024)
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      const int32_t* base = tile_base + (size_t)k * (E + 1);
      for (int j = base[e]; j < base[e + 1]; ++j) tile_problem[(size_t)k * max_tiles + j] = e;
    }
}

}  // namespace

void launch_compact(const Dims& d, const int32_t* slot_token, int32_t* crow_token, int32_t* slot_crow, int32_t* kept,
                    int32_t* tile_base, cudaStream_t st) {
  compact_kernel<<<d.E, kCompactThreads, 0, st>>>(slot_token, d.rows, d.S, d.C, crow_token, slot_crow, kept);
  tile_prefix_kernel<<<1, 1024, 0, st>>>(kept, d.E, compact_max_tiles(d), tile_base);
  count_launch(2);
}

}  // namespace gshard
