// Expert FFN out[e] = relu(buf[e] . wi[e]) . wo[e] (eq. (2)) for experts with MORE than 128 rows, as
// ONE persistent launch of CTA pairs (tcgen05.mma.cta_group::2, 256 x 256 tiles) that runs both
// grouped GEMMs in waves of experts, so that GEMM-2 reads the hidden activations h while they are
// still in L2 instead of after a 2 x |h| round trip through HBM (h is still written once: the
// caller may keep it for the backward pass, and its dirty lines are written back anyway).
//
// Work-item list (static, pair p takes items p, p + pairs, ...): step e holds the GEMM-1 items of
// expert e (256-row tile x a run of 256-wide hidden column tiles, contraction M) followed by the GEMM-2
// items of expert e - L (256-row tile x 256 output columns, contraction H); a GEMM-1 item has H/M
// column tiles, so that every item contracts the same amount and the pairs stay in step.  The lag L gives the GEMM-1 tiles of an expert
// time to finish on the other pairs before its GEMM-2 tiles come up, and is chosen so that the h of
// L experts fits L2 with room to spare.
// Dependency: a GEMM-2 tile needs every GEMM-1 tile of its (expert, row tile).  Each epilogue warp
// of a GEMM-1 tile, after its rows of h are written, fences them (GPU scope and async proxy) and
// counts itself in done[expert][row tile] (release); the producers of a GEMM-2 tile acquire the
// full count before their first TMA load of h.  A tile only ever waits for tiles EARLIER in the
// list, and every pair walks its tiles in list order, so the waits cannot deadlock; they are
// bounded in wall time all the same and report GSHARD_ERR_TIMEOUT.
// Pair protocol as in umma2_gemm.cu.  No load is multicast.
#include <cuda.h>

#include "kernels.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "umma_epilogue.cuh"

namespace gshard {

namespace {

using namespace umma_epi;

constexpr int BM = 128, BK = 64, BN = 256, BNH = BN / 2;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kABytes = BM * BK * 2;          // 16 KB
constexpr int kBBytes = BNH * BK * 2;         // 16 KB: this CTA's half of the B tile
constexpr int kBoxBytes = 64 * 64 * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kStages = 6;
constexpr int kTmemCols = 2 * BN;
constexpr int kBarOff = kStages * kStageBytes;
constexpr int kStgOff = kBarOff + 256;
constexpr int kSmemBytes = kStgOff + kEpiWarps * kStgWarpBytes + 1024;

// What the shared epilogue needs to know about one of the two outputs.
struct OutDesc {
  void* C;
  const void* mask;
  int rows, cols;
  long long c_ld, c_bs;
  int out_f32, relu;
  int keep_in_l2;               // the rows are read back by a later tile of the same launch
};
__device__ __forceinline__ bool epi_keep_in_l2(const OutDesc& o) { return o.keep_in_l2 != 0; }

struct ChainParams {
  OutDesc o1, o2;               // h (ReLU) and out
  int E, m_pairs, n1, n2;       // 256-row tiles per expert; 256-column tiles of h and of out
  int k1, k2;                   // 64-deep k-blocks of GEMM-1 (M) and GEMM-2 (H)
  int wave;                     // lag L in experts between GEMM-1 and GEMM-2 of an expert
  int sub1, n1g;                // GEMM-1 column tiles per work item, items per (expert, row tile)
  long long total_items;
  int* done;                    // [E][m_pairs] finished GEMM-1 epilogue warps
  int* status;
};

struct ChainTile { int phase, e, mt, nt; };

// Work-item list: step e = 0 .. E + L - 1 holds the GEMM-1 items of expert e (while e < E) followed by
// the GEMM-2 items of expert e - L (once e >= L), L = p.wave.  A GEMM-1 item is a run of sub1 column
// tiles of one row tile (nt = first of them), a GEMM-2 item one tile, so that all items take about
// the same time and the static round-robin over pairs stays in step.
__device__ __forceinline__ ChainTile decode(const ChainParams& p, long long tile) {
  const long long g1 = (long long)p.m_pairs * p.n1g, g2 = (long long)p.m_pairs * p.n2;
  const int L = p.wave;
  const long long head = g1 * L;                       // steps 0 .. L-1: GEMM-1 only
  const long long mid = (g1 + g2) * (p.E - L);         // steps L .. E-1: both
  ChainTile t;
  long long r;
  if (tile < head) {
    t.phase = 0; t.e = (int)(tile / g1); r = tile % g1;
  } else if (tile < head + mid) {
    const long long u = tile - head;
    const int step = L + (int)(u / (g1 + g2));
    r = u % (g1 + g2);
    if (r < g1) { t.phase = 0; t.e = step; }
    else { t.phase = 1; t.e = step - L; r -= g1; }
  } else {
    const long long u = tile - head - mid;
    t.phase = 1; t.e = p.E - L + (int)(u / g2); r = u % g2;
  }
  t.mt = (int)(r % p.m_pairs);
  t.nt = (int)(r / p.m_pairs) * (t.phase ? 1 : p.sub1);
  return t;
}

// Column tiles of a work item.
__device__ __forceinline__ int item_tiles(const ChainParams& p, const ChainTile& t) {
  return t.phase ? 1 : min(p.sub1, p.n1 - t.nt);
}

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ bool wait_counter(const int* ctr, int target, volatile int* abort_flag) {
  if (ld_acquire(ctr) >= target) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t it = 0;
  while (true) {
    if (ld_acquire(ctr) >= target) return true;
    __nanosleep(64);
    if ((++it & 63u) == 0 && (*abort_flag || ptx::globaltimer_ns() - t0 > 2000000000ull)) return false;
  }
}

__global__ void __launch_bounds__(kThreads, 1)
ffn_chained_kernel(const __grid_constant__ CUtensorMap map_buf, const __grid_constant__ CUtensorMap map_wi,
                   const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_wo,
                   const ChainParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kBarOff);
  uint64_t* full = bars;                      // [kStages]  used in the leader
  uint64_t* empty = bars + kStages;           // [kStages]  in each CTA
  uint64_t* acc_full = bars + 2 * kStages;    // [2]        in each CTA
  uint64_t* acc_empty = acc_full + 2;         // [2]        used in the leader (both epilogues arrive)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();     // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, 2 * kEpiWarps); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_buf); ptx::prefetch_tensormap(&map_wi);
    ptx::prefetch_tensormap(&map_h); ptx::prefetch_tensormap(&map_wo);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync_all();                          // barriers of both CTAs initialised before any remote use
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const int g1_target = p.n1 * 2 * kEpiWarps;       // epilogue warps of all GEMM-1 tiles of one (expert, row tile)

  bool ok = true;
  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      const uint64_t pol_w = ptx::policy_evict_first();    // weights: read once
      const uint64_t pol_a = ptx::policy_evict_last();     // buf and h: re-read from L2
      int stage = 0; uint32_t phase = 0;
      for (long long item = pair; item < p.total_items && ok; item += n_pairs) {
        const ChainTile t = decode(p, item);
        const int row0 = t.mt * 2 * BM + (int)rank * BM;      // this CTA's 128 rows of the 256-row tile
        const int kbs = t.phase ? p.k2 : p.k1;
        const CUtensorMap* ma = t.phase ? &map_h : &map_buf;
        const CUtensorMap* mb = t.phase ? &map_wo : &map_wi;
        if (t.phase) {
          // every GEMM-1 tile of this (expert, row tile) has written its part of h
          if (!wait_counter(p.done + (long long)t.e * p.m_pairs + t.mt, g1_target, abort_flag)) { ok = false; break; }
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        for (int sub = 0; sub < item_tiles(p, t) && ok; ++sub) {
          const int col0 = (t.nt + sub) * BN + (int)rank * BNH;   // this CTA's half of the B columns
          for (int kb = 0; kb < kbs; ++kb) {
            if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + stage * kStageBytes;
            unsigned char* sb = sa + kABytes;
            const uint32_t bar = ptx::map_to_cta(ptx::smem_u32(full + stage), 0);
            if (rank == 0) ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(2 * kStageBytes));
            ptx::tma_load_3d_pair(sa, ma, bar, kb * BK, row0, t.e, pol_a);
#pragma unroll
            for (int j = 0; j < BNH / 64; ++j)
              ptx::tma_load_3d_pair(sb + j * kBoxBytes, mb, bar, col0 + j * 64, kb * BK, t.e, pol_w);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) -------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(2 * BM, BN, false, true);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (long long item = pair; item < p.total_items && ok; item += n_pairs) {
        const ChainTile t = decode(p, item);
        const int kbs = t.phase ? p.k2 : p.k1;
        for (int sub = 0; sub < item_tiles(p, t) && ok; ++sub) {
        if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < kbs; ++kb) {
          if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * kStageBytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            ptx::umma_bf16_pair(d_tmem, ptx::make_smem_desc(sa + k * 32, 16, 1024),
                                ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024), idesc, (kb | k) != 0 ? 1u : 0u);
          ptx::umma_commit_pair(empty + stage);             // stage free in both CTAs
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit_pair(acc_full + acc);              // accumulator complete in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs, own 128 rows) ----------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    unsigned char* stg = smem + kStgOff + ew * kStgWarpBytes;
    int acc = 0; uint32_t acc_phase = 0;
    for (long long item = pair; item < p.total_items && ok; item += n_pairs) {
      const ChainTile t = decode(p, item);
      const int tile_row0 = t.mt * 2 * BM + (int)rank * BM;
      for (int sub = 0; sub < item_tiles(p, t) && ok; ++sub) {
      const TileCoord tc{t.mt, t.nt + sub, t.e};
      if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      if (t.phase == 0) {
        epilogue_tile<BN, false>(p.o1, tc, tile_row0, tmem_base + (uint32_t)(acc * BN), q, half, stg, lane, nullptr);
      } else {
        epilogue_tile<BN, false>(p.o2, tc, tile_row0, tmem_base + (uint32_t)(acc * BN), q, half, stg, lane, nullptr);
      }
      ptx::tc_fence_before_sync();
      if (t.phase == 0) {
        __threadfence();                                     // this warp's rows of h visible GPU-wide ...
        asm volatile("fence.proxy.async;" ::: "memory");     // ... and to the async proxy (TMA)
      }
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive_remote_relaxed(ptx::map_to_cta(ptx::smem_u32(acc_empty + acc), 0));   // the leader's barrier
        if (t.phase == 0)
          asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.done + (long long)t.e * p.m_pairs + t.mt)
                       : "memory");
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
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
  ptx::cluster_sync_all();             // no CTA frees TMEM or exits while its peer may still use it
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace

// bf16, more than one 128-row tile per expert, whole 64-deep k-blocks.
bool ffn_chained_supported(const Dims& d) {
  return d.bf16 && !d.simt && d.rows > 128 && d.M % 64 == 0 && d.H % 64 == 0;
}

size_t ffn_chained_scratch_bytes(const Dims& d) {
  return (size_t)d.E * ceil_div(d.rows, 2 * BM) * sizeof(int);
}

int launch_ffn_chained(const Dims& d, const void* buf, const void* wi, const void* wo, void* h, void* out,
                       void* scratch, int* status, cudaStream_t st) {
  ChainParams p;
  const long long rows = d.rows;
  p.o1 = OutDesc{h, nullptr, d.rows, d.H, d.H, rows * d.H, 0, 1, 1};
  p.o2 = OutDesc{out, nullptr, d.rows, d.M, d.M, rows * d.M, 0, 0, 0};
  p.E = d.E;
  p.m_pairs = ceil_div(d.rows, 2 * BM);
  p.n1 = ceil_div(d.H, BN);
  p.n2 = ceil_div(d.M, BN);
  p.k1 = ceil_div(d.M, BK);
  p.k2 = ceil_div(d.H, BK);
  // the h of L experts (rows x H bf16 each) should take at most about half of L2
  const long long h_bytes = rows * d.H * 2;
  long long wave = (64ll << 20) / (h_bytes > 0 ? h_bytes : 1);
  if (wave < 1) wave = 1;
  if (wave > d.E) wave = d.E;
  p.wave = (int)wave;
  p.sub1 = p.k2 / p.k1 > 1 ? p.k2 / p.k1 : 1;        // a GEMM-1 item contracts as much as a GEMM-2 tile
  if (p.sub1 > p.n1) p.sub1 = p.n1;
  p.n1g = ceil_div(p.n1, p.sub1);
  p.total_items = (long long)d.E * p.m_pairs * (p.n1g + p.n2);
  p.done = static_cast<int*>(scratch);
  p.status = status;
  if (cudaMemsetAsync(p.done, 0, ffn_chained_scratch_bytes(d), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  CUtensorMap m_buf, m_wi, m_h, m_wo;
  bool okm = make_map(&m_buf, buf, d.M, rows, d.E, d.M, rows * d.M, BK, BM);
  okm = okm && make_map(&m_wi, wi, d.H, d.M, d.E, d.H, (long long)d.M * d.H, 64, BK);
  okm = okm && make_map(&m_h, h, d.H, rows, d.E, d.H, rows * d.H, BK, BM);
  okm = okm && make_map(&m_wo, wo, d.M, d.H, d.E, d.M, (long long)d.H * d.M, 64, BK);
  if (!okm) return GSHARD_ERR_CUDA;
  const int sms = device_sms();
  long long pairs = sms / 2;
  if (pairs > p.total_items) pairs = p.total_items;
  if (cudaFuncSetAttribute(ffn_chained_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  // GEMM-2 items wait for GEMM-1 items of other pairs: cooperative launch, so that the runtime
  // guarantees the whole grid is resident at once (a refusal launches nothing; the caller then
  // runs the two grouped-GEMM launches).
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (cudaLaunchKernelEx(&cfg, ffn_chained_kernel, m_buf, m_wi, m_h, m_wo, p) != cudaSuccess) {
    cudaGetLastError();
    return GSHARD_ERR_UNSUPPORTED_SHAPE;
  }
  count_launch();
  return GSHARD_OK;
}

}  // namespace gshard
