// Grouped bf16 GEMM on the 5th-generation tensor cores: C[b] = act(A[b] . B[b]) for a batch of
// independent problems (the experts), fp32 accumulation in tensor memory.
//
// One persistent CTA per SM walks a static list of 128 x BN output tiles.  Warp roles:
//   warp 0      TMA producer: cp.async.bulk.tensor loads of A and B k-blocks (64 deep) into a
//               ring of 128-byte-swizzled shared-memory stages, completion on mbarriers
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128, N=BN, K=16) from shared-memory
//               descriptors into one of two TMEM accumulators; tcgen05.commit frees the stage
//   warps 2..9  epilogue: two warps per TMEM lane quarter, each taking half of the tile's columns.
//               tcgen05.ld the finished accumulator (thread = row, two 32-column loads in flight),
//               apply ReLU / mask, convert, stage in swizzled shared memory and write 128-byte row
//               segments; overlaps the next tile's MMAs through the second accumulator
// Operands may be K-major or MN-major in global memory (the expert weights wi [M,H] and wo [H,M]
// are contiguous along the non-contracted dimension); the layout goes into the tensor map, the
// shared-memory descriptor and the instruction descriptor - nothing is transposed in memory.
// Tile order: the tiles that share the larger operand run back to back (row tiles fastest when B
// is larger, column tiles fastest when A is), then batch, so that operand leaves HBM once and the
// other is re-read from L2.
#include <cuda.h>

#include "kernels.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "umma_epilogue.cuh"

namespace gshard {

namespace {

using namespace umma_epi;

constexpr int BM = 128, BK = 64;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kABytes = BM * BK * 2;        // 16 KB
constexpr int kBoxBytes = 64 * 64 * 2;      // one 64x64 box of an MN-major operand

template <int BN> struct Cfg {
  static constexpr int b_bytes = BN * BK * 2;
  static constexpr int stage_bytes = kABytes + b_bytes;
  static constexpr int stages = (BN == 256) ? 4 : 6;
  static constexpr int tmem_cols = 2 * BN;   // two accumulators
  static constexpr int bar_off = stages * stage_bytes;
  static constexpr int stg_off = bar_off + 1024;     // 1024-byte aligned: the staging rows leave by swizzled TMA stores
  static constexpr int smem_bytes = stg_off + kEpiWarps * kStgWarpBytes + 1024 /*alignment slack*/;
};

struct Params {
  void* C;
  const uint32_t* mask_bits;   // optional [batch][rows][cols/32]: output zeroed where the bit is clear
  uint32_t* mask_bits_out;     // optional, same layout: bit = accumulator value positive
  int rows, cols, K, batch;
  long long c_ld, c_bs;
  int m_tiles, n_tiles, total_tiles, k_blocks;
  int out_f32, relu;
  int a_stream, b_stream;
  int n_fastest;   // tile order: column tiles fastest (A is the larger operand) instead of row tiles
  int* status;
  // Ragged batches (compacted expert rows): problem b owns the row tiles [tile_base[b], tile_base[b+1])
  // of a device-side prefix array with batch + 1 entries; nullptr = every problem has m_tiles row tiles.
  const int* tile_base;
  const int* tile_problem;     // with tile_base: the problem that owns each row tile
  // with tile_base: problem b's tiles start behind the 2 * (pair_base[b+1] - pair_base[b]) row tiles that
  // a launch on CTA pairs covers; nullptr = they start at row 0
  const int* pair_base;
  int tma_store;   // epilogue rows leave by bulk tensor stores through map_c
};

// Tile index -> (row tile, column tile, problem).
__device__ __forceinline__ int total_tiles_of(const Params& p) {
  return p.tile_base ? __ldg(p.tile_base + p.batch) * p.n_tiles : p.total_tiles;
}
__device__ __forceinline__ TileCoord decode(const Params& p, int tile) {
  if (p.tile_base) {
    TileCoord t = decode_ragged(p, tile);
    if (p.pair_base) t.mt += 2 * (__ldg(p.pair_base + t.b + 1) - __ldg(p.pair_base + t.b));
    return t;
  }
  TileCoord t;
  t.mt = p.n_fastest ? (tile / p.n_tiles) % p.m_tiles : tile % p.m_tiles;
  t.nt = p.n_fastest ? tile % p.n_tiles : (tile / p.m_tiles) % p.n_tiles;
  t.b = tile / (p.m_tiles * p.n_tiles);
  return t;
}

// TF32: A and B hold fp32 values that the tensor core reads as TF32 (K-major operands only: with a
// 32-bit MN-major operand the instruction returns zeros).  A shared-memory row is still 128 bytes,
// i.e. 32 elements: a k-block is 32 deep and an MMA contracts 8; stage sizes in bytes are those of
// the bf16 form.
template <bool A_K, bool B_K, int BN, bool MASK, bool TF32 = false>
__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c, const Params p) {
  using C_ = Cfg<BN>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C_::bar_off);
  uint64_t* full = bars;                       // [stages]
  uint64_t* empty = bars + C_::stages;         // [stages]
  uint64_t* acc_full = bars + 2 * C_::stages;  // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int BKE = TF32 ? 32 : 64;                  // elements per k-block (128 bytes)
  constexpr int kBoxMN = TF32 ? 32 : 64;               // MN extent of one box of an MN-major operand
  constexpr int kBoxB = kBoxMN * BKE * (TF32 ? 4 : 2); // its bytes
  constexpr int kStepMN = TF32 ? 1024 : 2048;          // bytes of the K rows one MMA contracts (8 or 16 x 128)

  if (threadIdx.x == 0) {
    for (int s = 0; s < C_::stages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, kEpiWarps); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, C_::tmem_cols);
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
      const uint64_t pol_a = p.a_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      const uint64_t pol_b = p.b_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      int stage = 0; uint32_t phase = 0;
      const int total_tiles = total_tiles_of(p);
      TileCoord t = (int)blockIdx.x < total_tiles ? decode(p, blockIdx.x) : TileCoord{};
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const TileCoord cur = t;
        if (tile + (int)gridDim.x < total_tiles) t = decode(p, tile + gridDim.x);   // the next tile's coordinates load meanwhile
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sa = smem + stage * C_::stage_bytes;
          unsigned char* sb = sa + kABytes;
          ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)C_::stage_bytes);
          if (A_K) {
            ptx::tma_load_3d(sa, &map_a, full + stage, kb * BKE, cur.mt * BM, cur.b, pol_a);
          } else {
#pragma unroll
            for (int j = 0; j < BM / kBoxMN; ++j)
              ptx::tma_load_3d(sa + j * kBoxB, &map_a, full + stage, cur.mt * BM + j * kBoxMN, kb * BKE, cur.b, pol_a);
          }
          if (B_K) {
            ptx::tma_load_3d(sb, &map_b, full + stage, kb * BKE, cur.nt * BN, cur.b, pol_b);
          } else {
#pragma unroll
            for (int j = 0; j < BN / kBoxMN; ++j)
              ptx::tma_load_3d(sb + j * kBoxB, &map_b, full + stage, cur.nt * BN + j * kBoxMN, kb * BKE, cur.b, pol_b);
          }
          if (++stage == C_::stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = TF32 ? ptx::make_idesc_tf32(BM, BN, !A_K, !B_K) : ptx::make_idesc_bf16(BM, BN, !A_K, !B_K);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      const int total_tiles = total_tiles_of(p);
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * C_::stage_bytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int k = 0; k < 4; ++k) {              // 4 MMAs per k-block: 4 x 16 bf16 or 4 x 8 tf32
            const uint64_t da = A_K ? ptx::make_smem_desc(sa + k * 32, 16, 1024)
                                    : ptx::make_smem_desc(sa + k * kStepMN, kBoxB, 1024);
            const uint64_t db = B_K ? ptx::make_smem_desc(sb + k * 32, 16, 1024)
                                    : ptx::make_smem_desc(sb + k * kStepMN, kBoxB, 1024);
            if (TF32) ptx::umma_tf32(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
            else ptx::umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(empty + stage);           // stage reusable once these MMAs have read it
          if (++stage == C_::stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(acc_full + acc);            // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------------------
    const int ew = warp - 2;
    const int q = warp & 3;                          // TMEM lane quarter this warp may access
    const int half = ew >> 2;                        // which half of the tile's columns
    unsigned char* stg = smem + C_::stg_off + ew * kStgWarpBytes;
    int acc = 0; uint32_t acc_phase = 0;
    const int total_tiles = total_tiles_of(p);
    TileCoord tn = (int)blockIdx.x < total_tiles ? decode(p, blockIdx.x) : TileCoord{};
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const TileCoord t = tn;
      if (tile + (int)gridDim.x < total_tiles) tn = decode(p, tile + gridDim.x);
      if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      epilogue_tile<BN, MASK>(p, p.tma_store ? &map_c : nullptr, t, t.mt * BM, tmem_base + (uint32_t)(acc * BN), q, half,
                              stg, lane);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_relaxed(acc_empty + acc);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    epilogue_finish(p.tma_store ? &map_c : nullptr, lane);
  }

  // ------------------------------ teardown ---------------------------------------------------
  if (!ok) {
    *abort_flag = 1;
    set_device_status(p.status, GSHARD_ERR_TIMEOUT);
    // give copies and MMAs already in flight a bounded time to land before the CTA's shared and
    // tensor memory are released
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) { __nanosleep(1000); }
  }
  __syncwarp();
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, C_::tmem_cols);
  }
}


// ---- short-contraction variant: B tile resident in shared memory -------------------------------
//
// For C[b] = A[b]^T-like products with both operands MN-major and a contraction of at most 256 (the
// expert weight gradients dwo = h^T.dout and dwi = buf^T.dh, contraction = rows per expert) a
// 128 x 256 tile needs only 16 MMAs but 192 KB of operands, so the general kernel is bound by the
// L2 -> shared-memory feed.  Here a CTA takes a whole column block of one problem (fixed batch and
// 256-column tile) and walks its row tiles: the 256-column slice of B (up to 256 x 256, 128 KB) is
// loaded once and stays, only the 64 KB A tile changes, which cuts the operand feed to a third.
// Each of B's four k-blocks has its own full/empty barrier pair, so that the next column block's B
// arrives k-block by k-block behind the last row tile's MMAs.
namespace resb {
constexpr int BN = 256;
constexpr int kMaxKBlocks = 4;
constexpr int kBBlockBytes = BN * BK * 2;                        // 32 KB per k-block
constexpr int kAStages = 4;
constexpr int a_off = kMaxKBlocks * kBBlockBytes;                // 128 KB
constexpr int bar_off = a_off + kAStages * kABytes;              // + 64 KB
constexpr int stg_off = bar_off + 1024;
constexpr int smem_bytes = stg_off + kEpiWarps * kStgWarpBytes + 1024;
constexpr int tmem_cols = 2 * BN;
}  // namespace resb

__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_resident_b_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                            const __grid_constant__ CUtensorMap map_c, const Params p) {
  using namespace resb;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + bar_off);
  uint64_t* full = bars;                         // [kAStages]   A k-block landed
  uint64_t* empty = full + kAStages;             // [kAStages]   A k-block consumed
  uint64_t* b_full = empty + kAStages;           // [kMaxKBlocks] B k-block landed
  uint64_t* b_empty = b_full + kMaxKBlocks;      // [kMaxKBlocks] B k-block no longer needed by this column block
  uint64_t* acc_full = b_empty + kMaxKBlocks;    // [2]
  uint64_t* acc_empty = acc_full + 2;            // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_groups = p.n_tiles * p.batch;      // column blocks

  if (threadIdx.x == 0) {
    for (int s = 0; s < kAStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int s = 0; s < kMaxKBlocks; ++s) { ptx::mbar_init(b_full + s, 1); ptx::mbar_init(b_empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, kEpiWarps); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, tmem_cols);
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
      const uint64_t pol_a = p.a_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      const uint64_t pol_b = p.b_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      int stage = 0; uint32_t phase = 0, b_phase = 0;
      for (int grp = blockIdx.x; grp < n_groups && ok; grp += gridDim.x, b_phase ^= 1u) {
        const int nt = grp % p.n_tiles, b = grp / p.n_tiles;
        for (int mt = 0; mt < p.m_tiles && ok; ++mt) {
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (mt == 0) {
              if (!ptx::mbar_wait(b_empty + kb, b_phase ^ 1u, abort_flag)) { ok = false; break; }
              unsigned char* sb = smem + kb * kBBlockBytes;
              ptx::mbar_arrive_expect_tx(b_full + kb, (uint32_t)kBBlockBytes);
#pragma unroll
              for (int j = 0; j < BN / 64; ++j)
                ptx::tma_load_3d(sb + j * kBoxBytes, &map_b, b_full + kb, nt * BN + j * 64, kb * BK, b, pol_b);
            }
            if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + a_off + stage * kABytes;
            ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)kABytes);
#pragma unroll
            for (int j = 0; j < BM / 64; ++j)
              ptx::tma_load_3d(sa + j * kBoxBytes, &map_a, full + stage, mt * BM + j * 64, kb * BK, b, pol_a);
            if (++stage == kAStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, BN, true, true);
      int stage = 0; uint32_t phase = 0, b_phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int grp = blockIdx.x; grp < n_groups && ok; grp += gridDim.x, b_phase ^= 1u) {
        for (int mt = 0; mt < p.m_tiles && ok; ++mt) {
          if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (mt == 0 && !ptx::mbar_wait(b_full + kb, b_phase, abort_flag)) { ok = false; break; }
            if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t sa = ptx::smem_u32(smem + a_off + stage * kABytes);
            const uint32_t sb = ptx::smem_u32(smem + kb * kBBlockBytes);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k) {
              const uint64_t da = ptx::make_smem_desc(sa + k * 2048, kBoxBytes, 1024);
              const uint64_t db = ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024);
              ptx::umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            ptx::umma_commit(empty + stage);
            if (mt == p.m_tiles - 1) ptx::umma_commit(b_empty + kb);   // last use of this B k-block
            if (++stage == kAStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          ptx::umma_commit(acc_full + acc);
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    unsigned char* stg = smem + stg_off + ew * kStgWarpBytes;
    int acc = 0; uint32_t acc_phase = 0;
    for (int grp = blockIdx.x; grp < n_groups && ok; grp += gridDim.x) {
      TileCoord t;
      t.nt = grp % p.n_tiles; t.b = grp / p.n_tiles;
      for (t.mt = 0; t.mt < p.m_tiles; ++t.mt) {
        if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        epilogue_tile<BN, false>(p, p.tma_store ? &map_c : nullptr, t, t.mt * BM, tmem_base + (uint32_t)(acc * BN), q,
                                 half, stg, lane);
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_relaxed(acc_empty + acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    epilogue_finish(p.tma_store ? &map_c : nullptr, lane);
  }

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
    ptx::tmem_dealloc(tmem_base, tmem_cols);
  }
}

// ---- host side ------------------------------------------------------------------------------

template <bool A_K, bool B_K, int BN, bool MASK, bool TF32 = false>
int launch_t(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const Params& p, int grid,
             cudaStream_t st) {
  auto kern = umma_gemm_kernel<A_K, B_K, BN, MASK, TF32>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::smem_bytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  kern<<<grid, kThreads, Cfg<BN>::smem_bytes, st>>>(ma, mb, mc, p);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

}  // namespace

int launch_umma_gemm(const UmmaGemm& g, int* status, cudaStream_t st) {
  if (g.rows <= 0 || g.cols <= 0 || g.K <= 0 || g.batch <= 0) return GSHARD_OK;
  if ((g.mask_bits || g.mask_bits_out) && g.cols % 32) return GSHARD_ERR_INTERNAL;   // one word per 32 columns
  const int BN = g.cols > 128 ? 256 : 128;
  // fp32 operands read as TF32: the tensor core takes 32-bit operands K-major only (an MN-major
  // one yields zeros), so both operands must be contiguous along the contraction
  if (g.tf32 && (!g.a_kmajor || !g.b_kmajor || g.mask_bits || !g.out_f32)) return GSHARD_ERR_INTERNAL;
  const int esz = g.tf32 ? 4 : 2;
  const int bke = 128 / esz;                     // elements per 128-byte k-block row
  CUtensorMap ma, mb;
  bool okm;
  if (g.a_kmajor) okm = make_map(&ma, g.A, g.K, g.rows, g.batch, g.a_ld, g.a_bs, bke, BM, esz);
  else            okm = make_map(&ma, g.A, g.rows, g.K, g.batch, g.a_ld, g.a_bs, bke, bke, esz);
  if (g.b_kmajor) okm = okm && make_map(&mb, g.B, g.K, g.cols, g.batch, g.b_ld, g.b_bs, bke, BN, esz);
  else            okm = okm && make_map(&mb, g.B, g.cols, g.K, g.batch, g.b_ld, g.b_bs, bke, bke, esz);
  if (!okm) return GSHARD_ERR_CUDA;
  CUtensorMap mc;
  const bool tma_store = store_map_for(g, &mc);
  Params p;
  p.tma_store = tma_store ? 1 : 0;
  p.C = g.C; p.mask_bits = g.mask_bits; p.mask_bits_out = g.mask_bits_out; p.rows = g.rows; p.cols = g.cols; p.K = g.K; p.batch = g.batch;
  p.c_ld = g.c_ld; p.c_bs = g.c_bs;
  p.m_tiles = ceil_div(g.rows, BM); p.n_tiles = ceil_div(g.cols, BN);
  p.total_tiles = p.m_tiles * p.n_tiles * g.batch;
  p.k_blocks = ceil_div(g.K, bke);
  p.out_f32 = g.out_f32; p.relu = g.relu; p.a_stream = g.a_stream; p.b_stream = g.b_stream;
  // stream the larger operand once: walk the tiles that share it back to back
  p.n_fastest = (g.rows > g.cols) ? 1 : 0;
  p.status = status;
  p.tile_base = g.tile_base;
  p.pair_base = g.tile_base ? g.pair_base : nullptr;
  p.tile_problem = g.tile_problem;
  if (g.tile_base && !g.tile_problem) return GSHARD_ERR_INTERNAL;
  if (g.tile_base && g.tf32) return GSHARD_ERR_INTERNAL;
  if (g.tile_base) p.n_fastest = 0;            // ragged lists are walked with the row tiles fastest
  int sms = device_sms();
  if (g.max_ctas > 0 && sms > g.max_ctas) sms = g.max_ctas;
  if (!g.tf32 && !g.tile_base && !g.a_kmajor && !g.b_kmajor && !g.mask_bits && BN == 256 && p.k_blocks <= resb::kMaxKBlocks && p.m_tiles >= 4) {
    // short contraction, several row tiles per column block: keep the B tile resident
    const int n_groups = p.n_tiles * g.batch;
    if (cudaFuncSetAttribute(umma_gemm_resident_b_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             resb::smem_bytes) != cudaSuccess)
      return GSHARD_ERR_CUDA;
    umma_gemm_resident_b_kernel<<<n_groups < sms ? n_groups : sms, kThreads, resb::smem_bytes, st>>>(ma, mb, mc, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
  }
  const int grid = (p.total_tiles < sms && !g.tile_base) ? p.total_tiles : sms;   // ragged: count known on the device only
  if (g.tf32)
    return BN == 256 ? launch_t<true, true, 256, false, true>(ma, mb, mc, p, grid, st)
                     : launch_t<true, true, 128, false, true>(ma, mb, mc, p, grid, st);
#define GSHARD_DISPATCH(AK, BKM)                                                                    \
  (p.mask_bits ? (BN == 256 ? launch_t<AK, BKM, 256, true>(ma, mb, mc, p, grid, st)                          \
                       : launch_t<AK, BKM, 128, true>(ma, mb, mc, p, grid, st))                         \
          : (BN == 256 ? launch_t<AK, BKM, 256, false>(ma, mb, mc, p, grid, st)                         \
                       : launch_t<AK, BKM, 128, false>(ma, mb, mc, p, grid, st)))
  if (g.a_kmajor && g.b_kmajor) return GSHARD_DISPATCH(true, true);
  if (g.a_kmajor && !g.b_kmajor) return GSHARD_DISPATCH(true, false);
  if (!g.a_kmajor && g.b_kmajor) return GSHARD_DISPATCH(false, true);
  return GSHARD_DISPATCH(false, false);
#undef GSHARD_DISPATCH
}

}  // namespace gshard
