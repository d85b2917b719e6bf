// Pieces shared by the single-launch expert-FFN kernels (groups of single CTAs, groups of CTA pairs):
// cross-CTA counter waits, and the epilogue's conversion / staging / row stores.
#pragma once
#include "kernels.cuh"
#include "sm100_ptx.cuh"

namespace gshard {
namespace ffn_shared {

constexpr int kStgRowBytes = 128;
constexpr int kStgWarpBytes = 32 * kStgRowBytes;

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// `poll_ns`: pause between polls.  The hand-over waits on the critical path poll fast; the row-gather
// warp, which waits for a whole unit to finish, polls slowly so that it does not load the counters'
// L2 lines.
__device__ __forceinline__ bool wait_counter(const int* ctr, int target, volatile int* abort_flag,
                                             uint32_t poll_ns = 32, uint64_t limit_ns = 2000000000ull) {
  if (ld_acquire(ctr) >= target) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t it = 0;
  const uint32_t check_mask = poll_ns >= 1000 ? 0u : 63u;
  while (true) {
    if (ld_acquire(ctr) >= target) return true;
    __nanosleep(poll_ns);
    if ((++it & check_mask) == 0) {
      if (*abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) return false;
    }
  }
}

// 32 fp32 accumulator values of this thread's row -> bf16 (optionally ReLU) -> staging row pieces.
__device__ __forceinline__ void stage_chunk(const uint32_t* r, bool relu, unsigned char* srow, int lane, int piece0) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float a = __uint_as_float(r[8 * i + 2 * j]), b = __uint_as_float(r[8 * i + 2 * j + 1]);
      if (relu) { a = fmaxf(a, 0.f); b = fmaxf(b, 0.f); }
      const __nv_bfloat162 pr = __floats2bfloat162_rn(a, b);
      w[j] = *reinterpret_cast<const uint32_t*>(&pr);
    }
    *reinterpret_cast<uint4*>(srow + (((piece0 + i) ^ (lane & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// Staged 32 rows x 64 bf16 columns -> global rows of `ld` elements starting at dst (row 0, col 0 of
// the staged block); rows >= row_limit and columns >= col_limit are skipped.
__device__ __forceinline__ void flush_block(const unsigned char* stg, __nv_bfloat16* dst, long long ld, int row_limit,
                                            int col_limit, int lane) {
  __syncwarp();
  const int piece = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = 4 * i + (lane >> 3);
    if (r < row_limit && piece * 8 < col_limit) {
      const uint4 val = *reinterpret_cast<const uint4*>(stg + r * kStgRowBytes + ((piece ^ (r & 7)) * 16));
      *reinterpret_cast<uint4*>(dst + (long long)r * ld + piece * 8) = val;
    }
  }
  __syncwarp();
}

}  // namespace ffn_shared
}  // namespace gshard
