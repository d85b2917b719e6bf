// Expert FFN in ONE persistent launch: h = relu(buf . wi) and out = h . wo (eq. (2)) for all
// experts, with the hidden activations h kept in a small ring that stays resident in L2 instead
// of making a round trip through HBM.
//
// Same CTA structure as the grouped GEMM (TMA producer warp, tcgen05 issuer warp, four epilogue
// warps, two TMEM accumulators).  The tile list interleaves the two GEMMs expert by expert:
//   ... G1(e) tiles, G2(e - lag) tiles, G1(e+1) tiles, G2(e+1 - lag) tiles ...
// and is dealt round-robin to the CTAs, each walking its part in order.  A G2 tile may start
// loading h rows only when every G1 tile of that (expert, row tile) has stored them:
//   ready[e, mt]  counts finished G1 epilogue warps  (release by the writer, acquire by the
//                 TMA producer, then a proxy fence before the async-proxy load)
//   done[e, mt]   counts finished G2 epilogue warps; a G1 tile of expert e + ring waits for it
//                 before it overwrites the ring slot.
// A dependency always points to a tile that is earlier in the global order and every CTA walks
// that order, with all CTAs co-resident (grid <= SM count, one CTA per SM), so the earliest
// unfinished tile can always proceed.  Every wait is bounded in wall time and reports
// GSHARD_ERR_TIMEOUT through the status word instead of hanging.
#include <cuda.h>

#include "kernels.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace gshard {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kThreads = 192;
constexpr int kABytes = BM * BK * 2;
constexpr int kBBytes = BN * BK * 2;
constexpr int kBoxBytes = 64 * 64 * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kStages = 4;
constexpr int kTmemCols = 2 * BN;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;

struct FusedParams {
  __nv_bfloat16* h;      // ring [ring][rows][H]
  __nv_bfloat16* out;    // [E][rows][M]
  int rows, M, H, E;
  int m_tiles, n1_tiles, n2_tiles, T1, T2, lag, ring, k1_blocks, k2_blocks;
  long long total_tiles;
  int* ready;            // [E * m_tiles]
  int* done;             // [E * m_tiles]
  int* status;
};

struct Tile {
  int phase;   // 1: h = relu(buf . wi), 2: out = h . wo
  int e, mt, nt;
};

__device__ __forceinline__ Tile decode_tile(const FusedParams& p, long long idx) {
  Tile t;
  int local;
  const long long head = (long long)p.lag * p.T1;
  const int P = p.T1 + p.T2;
  if (idx < head) {
    t.phase = 1; t.e = (int)(idx / p.T1); local = (int)(idx % p.T1);
  } else {
    const long long i2 = idx - head;
    const long long mid = (long long)(p.E - p.lag) * P;
    if (i2 < mid) {
      const int j = p.lag + (int)(i2 / P);
      const int r = (int)(i2 % P);
      if (r < p.T1) { t.phase = 1; t.e = j; local = r; }
      else { t.phase = 2; t.e = j - p.lag; local = r - p.T1; }
    } else {
      const long long i3 = i2 - mid;
      t.phase = 2; t.e = p.E - p.lag + (int)(i3 / p.T2); local = (int)(i3 % p.T2);
    }
  }
  t.mt = local % p.m_tiles;
  t.nt = local / p.m_tiles;
  return t;
}

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Spins until *ctr >= target; false on abort or after limit_ns.
__device__ __forceinline__ bool wait_counter(const int* ctr, int target, volatile int* abort_flag,
                                             uint64_t limit_ns = 2000000000ull) {
  if (ld_acquire(ctr) >= target) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t it = 0;
  while (true) {
    if (ld_acquire(ctr) >= target) return true;
    __nanosleep(64);
    if ((++it & 63u) == 0) {
      if (*abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) return false;
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
ffn_fused_kernel(const __grid_constant__ CUtensorMap map_buf, const __grid_constant__ CUtensorMap map_wi,
                 const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_wo,
                 const FusedParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;
  uint64_t* acc_full = bars + 2 * kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, 4); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_buf); ptx::prefetch_tensormap(&map_wi);
    ptx::prefetch_tensormap(&map_h); ptx::prefetch_tensormap(&map_wo);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = true;
  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      const uint64_t pol_w = ptx::policy_evict_first();    // weights: read exactly once
      const uint64_t pol_a = ptx::policy_evict_last();     // buf / h: re-read by the other column tiles
      int stage = 0; uint32_t phase = 0;
      for (long long idx = blockIdx.x; idx < p.total_tiles && ok; idx += gridDim.x) {
        const Tile t = decode_tile(p, idx);
        const CUtensorMap* ma = t.phase == 1 ? &map_buf : &map_h;
        const CUtensorMap* mb = t.phase == 1 ? &map_wi : &map_wo;
        const int kblocks = t.phase == 1 ? p.k1_blocks : p.k2_blocks;
        const int a_batch = t.phase == 1 ? t.e : (t.e % p.ring);
        if (t.phase == 2) {
          // h rows of this (expert, row tile) must be complete and visible to the async proxy
          if (!wait_counter(p.ready + (size_t)t.e * p.m_tiles + t.mt, p.n1_tiles * 4, abort_flag)) { ok = false; break; }
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sa = smem + stage * kStageBytes;
          unsigned char* sb = sa + kABytes;
          ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)kStageBytes);
          ptx::tma_load_3d(sa, ma, full + stage, kb * BK, t.mt * BM, a_batch, pol_a);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            ptx::tma_load_3d(sb + j * kBoxBytes, mb, full + stage, t.nt * BN + j * 64, kb * BK, t.e, pol_w);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, BN, false, true);   // A K-major, B MN-major
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (long long idx = blockIdx.x; idx < p.total_tiles && ok; idx += gridDim.x) {
        const Tile t = decode_tile(p, idx);
        const int kblocks = t.phase == 1 ? p.k1_blocks : p.k2_blocks;
        if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * kStageBytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = ptx::make_smem_desc(sa + k * 32, 16, 1024);
            const uint64_t db = ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024);
            ptx::umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(empty + stage);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(acc_full + acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------------------
    const int q = warp & 3;
    int acc = 0; uint32_t acc_phase = 0;
    for (long long idx = blockIdx.x; idx < p.total_tiles && ok; idx += gridDim.x) {
      const Tile t = decode_tile(p, idx);
      if (!ptx::mbar_wait(acc_full + acc, acc_phase, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const int row = t.mt * BM + q * 32 + lane;
      const bool row_ok = row < p.rows;
      const int cols = t.phase == 1 ? p.H : p.M;
      __nv_bfloat16* base;
      if (t.phase == 1) {
        // the ring slot may still be read by the G2 tiles of the expert that used it before
        if (t.e >= p.ring &&
            !wait_counter(p.done + (size_t)(t.e - p.ring) * p.m_tiles + t.mt, p.n2_tiles * 4, abort_flag)) {
          ok = false; break;
        }
        base = p.h + ((size_t)(t.e % p.ring) * p.rows + row) * p.H;
      } else {
        base = p.out + ((size_t)t.e * p.rows + row) * p.M;
      }
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        const int col0 = t.nt * BN + c * 32;
        if (col0 >= cols) break;
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + (uint32_t)(acc * BN + c * 32) + ((uint32_t)(q * 32) << 16), r);
        ptx::tmem_ld_wait();
        if (!row_ok) continue;
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          v[i] = __uint_as_float(r[i]);
          if (t.phase == 1) v[i] = fmaxf(v[i], 0.f);
        }
        __nv_bfloat16* dst = base + col0;
        if (col0 + 32 <= cols) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const __nv_bfloat162 pr = __floats2bfloat162_rn(v[8 * i + 2 * j], v[8 * i + 2 * j + 1]);
              w[j] = *reinterpret_cast<const uint32_t*>(&pr);
            }
            reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        } else {
          for (int i = 0; i < 32; ++i) if (col0 + i < cols) dst[i] = __float2bfloat16_rn(v[i]);
        }
      }
      // accumulator free for the issuer; then publish this warp's part of the tile
      ptx::tc_fence_before_sync();
      if (t.phase == 1) {
        __threadfence();                                     // h stores visible GPU-wide ...
        asm volatile("fence.proxy.async;" ::: "memory");     // ... and to the async proxy (TMA)
      }
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(acc_empty + acc);
        int* ctr = (t.phase == 1 ? p.ready : p.done) + (size_t)t.e * p.m_tiles + t.mt;
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(ctr) : "memory");
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ------------------------------ teardown ---------------------------------------------------
  if (!ok) {
    *abort_flag = 1;
    set_device_status(p.status, GSHARD_ERR_TIMEOUT);
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) { __nanosleep(1000); }
  }
  __syncwarp();
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

// Ring length (experts) for a shape: long enough that producers run `lag` experts ahead of the
// consumers and a slot is not reused before its readers are long gone.
void ffn_fused_schedule(int rows, int H, int E, int* lag, int* ring) {
  const int m_tiles = ceil_div(rows, BM);
  const int T1 = m_tiles * ceil_div(H, BN);
  int l = ceil_div(2 * 148, T1);                 // G1 runs >= two waves of CTAs ahead of G2
  if (l < 1) l = 1;
  if (l > E) l = E;
  int r = 2 * l + 2;
  if (r > E) r = E;
  *lag = l; *ring = r;
}

// h_ring: [ring][rows][H] bf16 (ring == E stores every expert's activations, e.g. for backward).
// flags: 2 * E * m_tiles ints of scratch.
int launch_ffn_fused(const Dims& d, const void* buf, const void* wi, const void* wo, void* h_ring, int ring,
                     void* out, int* flags, int* status, cudaStream_t st) {
  FusedParams p;
  p.h = static_cast<__nv_bfloat16*>(h_ring);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.rows = d.rows; p.M = d.M; p.H = d.H; p.E = d.E;
  p.m_tiles = ceil_div(d.rows, BM);
  p.n1_tiles = ceil_div(d.H, BN);
  p.n2_tiles = ceil_div(d.M, BN);
  p.T1 = p.m_tiles * p.n1_tiles;
  p.T2 = p.m_tiles * p.n2_tiles;
  int lag, ring_default;
  ffn_fused_schedule(d.rows, d.H, d.E, &lag, &ring_default);
  p.lag = lag;
  p.ring = ring;
  if (ring < lag + 1 && ring < d.E) return GSHARD_ERR_INTERNAL;
  p.k1_blocks = ceil_div(d.M, BK);
  p.k2_blocks = ceil_div(d.H, BK);
  p.total_tiles = (long long)d.E * (p.T1 + p.T2);
  p.ready = flags;
  p.done = flags + (size_t)d.E * p.m_tiles;
  p.status = status;
  if (cudaMemsetAsync(flags, 0, sizeof(int) * 2 * (size_t)d.E * p.m_tiles, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  CUtensorMap m_buf, m_wi, m_h, m_wo;
  const long long rows = d.rows;
  bool okm = make_map(&m_buf, buf, d.M, rows, d.E, d.M, rows * d.M, BK, BM);
  okm = okm && make_map(&m_wi, wi, d.H, d.M, d.E, d.H, (long long)d.M * d.H, 64, BK);
  okm = okm && make_map(&m_h, h_ring, d.H, rows, ring, d.H, rows * d.H, BK, BM);
  okm = okm && make_map(&m_wo, wo, d.M, d.H, d.E, d.M, (long long)d.H * d.M, 64, BK);
  if (!okm) return GSHARD_ERR_CUDA;
  int sms = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = (int)(p.total_tiles < sms ? p.total_tiles : sms);
  if (cudaFuncSetAttribute(ffn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  ffn_fused_kernel<<<grid, kThreads, kSmemBytes, st>>>(m_buf, m_wi, m_h, m_wo, p);
  count_launch();
  return cudaPeekAtLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

}  // namespace gshard
