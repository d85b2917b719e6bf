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

// tile_base[e] = sum over e' < e of ceil(kept[e'] / 128), tile_base[E] = total (one CTA, in order).
__global__ void __launch_bounds__(1024) tile_prefix_kernel(const int32_t* __restrict__ kept, int E,
                                                           int32_t* __restrict__ tile_base) {
  __shared__ int warp_sum[32];
  __shared__ int running;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (threadIdx.x == 0) running = 0;
  __syncthreads();
  for (int e0 = 0; e0 < E; e0 += 1024) {
    const int e = e0 + threadIdx.x;
    const int tiles = e < E ? (kept[e] + 127) / 128 : 0;
    int incl = tiles;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += v;
    }
    if (lane == 31) warp_sum[w] = incl;
    __syncthreads();
    int before = running;
    for (int i = 0; i < w; ++i) before += warp_sum[i];
    if (e < E) tile_base[e] = before + incl - tiles;
    __syncthreads();
    if (threadIdx.x == 0) {
      int add = 0;
      for (int i = 0; i < 32; ++i) add += warp_sum[i];
      running += add;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) tile_base[E] = running;
}

}  // namespace

void launch_compact(const Dims& d, const int32_t* slot_token, int32_t* crow_token, int32_t* slot_crow, int32_t* kept,
                    int32_t* tile_base, cudaStream_t st) {
  compact_kernel<<<d.E, kCompactThreads, 0, st>>>(slot_token, d.rows, d.S, d.C, crow_token, slot_crow, kept);
  tile_prefix_kernel<<<1, 1024, 0, st>>>(kept, d.E, tile_base);
  count_launch(2);
}

}  // namespace gshard
