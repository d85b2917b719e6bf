// Grouped bf16 GEMM with the two-SM tensor-core instruction (tcgen05.mma.cta_group::2): a pair of
// CTAs (a cluster of two) computes a 256 x 256 output tile, each CTA holding 128 rows of A, HALF
// of the B tile (128 of its 256 columns) and the accumulator of its own 128 rows in its TMEM.
// Per 64-deep k-block a CTA loads 32 KB instead of the 48 KB a lone 128 x 256 tile needs, which
// takes the operand feed (about 91 B/clk per SM for the one-SM kernel) below what an SM can draw
// from L2 - the limit of the one-SM kernel on shapes with many rows per expert.
//
// Roles per CTA as in the one-SM kernel (warp 0 TMA producer, warp 1 MMA, warps 2..9 epilogue),
// with the pair protocol:
//   * both producers issue cta_group::2 TMA loads into their own shared memory that complete on
//     the LEADER's (cluster rank 0) full barrier; the leader's producer arms it with the bytes of
//     both CTAs.  No load is multicast.
//   * only the leader's MMA thread issues tcgen05.mma.cta_group::2; tcgen05.commit multicasts the
//     "stage free" and "accumulator complete" arrivals to the same barrier in both CTAs.
//   * the peer's epilogue warps release the accumulator on the leader's barrier (remote arrive).
//   * TMEM is allocated and freed with the cta_group::2 forms by warp 1 of both CTAs; cluster
//     barriers order barrier initialisation before, and teardown after, all cross-CTA traffic.
// Every mbarrier wait is bounded in wall time and reports GSHARD_ERR_TIMEOUT; a CTA that gave up
// still reaches the final cluster barrier, so its peer is not left waiting.
//
// Two kernels: umma2_gemm_kernel, the general one (tile list regular or ragged - compacted expert
// rows -, ReLU / mask epilogues), and umma2_gemm_resident_b_kernel for the weight gradients, whose
// contraction is an expert's rows (at most 256): a pair keeps a 256-column slice of B resident and walks
// the row tiles of that column block.
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
constexpr int kStgOff = kBarOff + 1024;        // 1024-byte aligned: the staging rows leave by swizzled TMA stores
constexpr int kSmemBytes = kStgOff + kEpiWarps * kStgWarpBytes + 1024;

struct Params2 {
  void* C;
  const uint32_t* mask_bits;   // optional [batch][rows][cols/32]: output zeroed where the bit is clear
  uint32_t* mask_bits_out;     // optional, same layout: bit = accumulator value positive
  int rows, cols, K, batch;
  long long c_ld, c_bs;
  int m_tiles, n_tiles, total_tiles, k_blocks;   // tiles of 256 x 256
  int out_f32, relu;
  int a_stream, b_stream;
  int n_fastest;
  int* status;
  int tma_store;   // epilogue rows leave by bulk tensor stores through map_c
  // Ragged batches (compacted expert rows): problem b owns the 256-row tiles [tile_base[b], tile_base[b+1])
  // of a device-side prefix array with batch + 1 entries; nullptr = every problem has m_tiles row tiles.
  const int* tile_base;
  const int* tile_problem;     // with tile_base: the problem that owns each row tile
};

// Tile index -> (row tile, column tile, problem).
__device__ __forceinline__ int total_tiles_of(const Params2& p) {
  return p.tile_base ? __ldg(p.tile_base + p.batch) * p.n_tiles : p.total_tiles;
}
__device__ __forceinline__ TileCoord decode(const Params2& p, int tile) {
  if (p.tile_base) return decode_ragged(p, tile);
  TileCoord t;
  t.mt = p.n_fastest ? (tile / p.n_tiles) % p.m_tiles : tile % p.m_tiles;
  t.nt = p.n_fastest ? tile % p.n_tiles : (tile / p.m_tiles) % p.n_tiles;
  t.b = tile / (p.m_tiles * p.n_tiles);
  return t;
}

template <bool A_K, bool B_K, bool MASK>
__global__ void __launch_bounds__(kThreads, 1)
umma2_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_c, const Params2 p) {
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
  const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, 2 * kEpiWarps); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync_all();                               // barriers of both CTAs initialised before any remote use
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = true;
  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      const uint64_t pol_a = p.a_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      const uint64_t pol_b = p.b_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      int stage = 0; uint32_t phase = 0;
      const int total_tiles = total_tiles_of(p);
      TileCoord tn = pair < total_tiles ? decode(p, pair) : TileCoord{};
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        const TileCoord t = tn;
        if (tile + n_pairs < total_tiles) tn = decode(p, tile + n_pairs);   // the next tile's coordinates load meanwhile
        const int row0 = t.mt * 2 * BM + (int)rank * BM;      // this CTA's 128 rows of the 256-row tile
        const int col0 = t.nt * BN + (int)rank * BNH;         // this CTA's half of the B columns
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sa = smem + stage * kStageBytes;
          unsigned char* sb = sa + kABytes;
          const uint32_t bar = ptx::map_to_cta(ptx::smem_u32(full + stage), 0);
          if (rank == 0) ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(2 * kStageBytes));
          if (A_K) {
            ptx::tma_load_3d_pair(sa, &map_a, bar, kb * BK, row0, t.b, pol_a);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j)
              ptx::tma_load_3d_pair(sa + j * kBoxBytes, &map_a, bar, row0 + j * 64, kb * BK, t.b, pol_a);
          }
          if (B_K) {
            ptx::tma_load_3d_pair(sb, &map_b, bar, kb * BK, col0, t.b, pol_b);
          } else {
#pragma unroll
            for (int j = 0; j < BNH / 64; ++j)
              ptx::tma_load_3d_pair(sb + j * kBoxBytes, &map_b, bar, col0 + j * 64, kb * BK, t.b, pol_b);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) -------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(2 * BM, BN, !A_K, !B_K);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      const int total_tiles = total_tiles_of(p);
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * kStageBytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = A_K ? ptx::make_smem_desc(sa + k * 32, 16, 1024)
                                    : ptx::make_smem_desc(sa + k * 2048, kBoxBytes, 1024);
            const uint64_t db = B_K ? ptx::make_smem_desc(sb + k * 32, 16, 1024)
                                    : ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024);
            ptx::umma_bf16_pair(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit_pair(empty + stage);             // stage free in both CTAs
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit_pair(acc_full + acc);              // accumulator complete in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs, own 128 rows) ----------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    unsigned char* stg = smem + kStgOff + ew * kStgWarpBytes;
    int acc = 0; uint32_t acc_phase = 0;
    const int total_tiles = total_tiles_of(p);
    TileCoord tn = pair < total_tiles ? decode(p, pair) : TileCoord{};
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
      const TileCoord t = tn;
      if (tile + n_pairs < total_tiles) tn = decode(p, tile + n_pairs);
      const int tile_row0 = t.mt * 2 * BM + (int)rank * BM;     // this CTA's 128 rows of the 256-row tile
      if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      epilogue_tile<BN, MASK>(p, p.tma_store ? &map_c : nullptr, t, tile_row0, tmem_base + (uint32_t)(acc * BN), q, half,
                              stg, lane);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_remote_relaxed(ptx::map_to_cta(ptx::smem_u32(acc_empty + acc), 0));   // the leader's barrier
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    epilogue_finish(p.tma_store ? &map_c : nullptr, lane);
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
  ptx::cluster_sync_all();                  // no CTA frees TMEM or exits while its peer may still use it
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ---- short-contraction variant on pairs: B tile resident, deep A ring -----------------------------
//
// The expert weight gradients dwo = h^T . dout and dwi = buf^T . dh contract over the rows of an expert
// (at most 256), both operands MN-major, and write an output the size of the weights.  A 256 x 256
// tile is then only 16 MMAs of work per CTA for 64 KB of A, so what bounds the kernel is how many A
// bytes it can keep in flight: with the 64 KB A ring of the single-CTA resident-B kernel a tile took
// about one memory latency (2.7 us against 1.1 us of tensor time).  On a pair each CTA holds only its
// half of the resident B slice (64 KB for 256 columns x 256 deep), which leaves room for an A ring of
// eight 16 KB k-blocks: two row tiles in flight.  A pair takes a whole column block of one problem
// (fixed batch index and 256-column tile) and walks its 256-row tiles; B's k-blocks have their own
// full/empty barriers so that the next column block's B arrives behind the last row tile's MMAs.
// Two shapes of the same 192 KB: DBL = false, one B slice and an A ring of eight k-blocks (two row tiles in
// flight), for problems with many row tiles per column block; DBL = true, TWO B slices and an A ring of
// four k-blocks: the next column block's B slice is loaded while the current one is being used, for
// problems with few row tiles per column block, where waiting for B at every switch would dominate.
namespace resb2 {
constexpr int kMaxKBlocks = 4;
template <bool DBL> struct Lay {
  static constexpr int kBBufs = DBL ? 2 : 1;
  static constexpr int kAStages = DBL ? 4 : 8;
  static constexpr int a_off = kBBufs * kMaxKBlocks * kBBytes;         // 64 KB per B slice half
  static constexpr int bar_off = a_off + kAStages * kABytes;
  static constexpr int stg_off = bar_off + 1024;                       // 1024-byte aligned for the swizzled bulk stores
  static constexpr int smem_bytes = stg_off + kEpiWarps * kStgWarpBytes + 1024;
  static_assert(smem_bytes <= 232448, "shared memory budget");
};
}  // namespace resb2

template <bool DBL>
__global__ void __launch_bounds__(kThreads, 1)
umma2_gemm_resident_b_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                             const __grid_constant__ CUtensorMap map_c, const Params2 p) {
  using namespace resb2;
  using L = Lay<DBL>;
  constexpr int kAStages = L::kAStages, a_off = L::a_off, bar_off = L::bar_off, stg_off = L::stg_off;
  constexpr int kBBars = L::kBBufs * kMaxKBlocks;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + bar_off);
  uint64_t* full = bars;                         // [kAStages]    A k-block landed (leader's barrier counts both CTAs)
  uint64_t* empty = full + kAStages;             // [kAStages]    A k-block consumed (in each CTA)
  uint64_t* b_full = empty + kAStages;           // [kBBars] B k-block of a slice landed (leader)
  uint64_t* b_empty = b_full + kBBars;           // [kBBars] B k-block no longer needed (in each CTA)
  uint64_t* acc_full = b_empty + kBBars;         // [2]           in each CTA
  uint64_t* acc_empty = acc_full + 2;            // [2]           leader (both epilogues arrive)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_groups = p.n_tiles * p.batch;      // column blocks

  if (threadIdx.x == 0) {
    for (int s = 0; s < kAStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int s = 0; s < kBBars; ++s) { ptx::mbar_init(b_full + s, 1); ptx::mbar_init(b_empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, 2 * kEpiWarps); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync_all();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = true;
  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      const uint64_t pol_a = p.a_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      const uint64_t pol_b = p.b_stream ? ptx::policy_evict_first() : ptx::policy_evict_last();
      int stage = 0; uint32_t phase = 0;
      // B slice of column block grp_x, the it_x-th of this pair: buffer it_x mod kBBufs, whose barriers
      // change phase every kBBufs column blocks
      auto load_b = [&](int grp_x, int it_x) {
        const int buf = it_x % L::kBBufs;
        const uint32_t ph = (uint32_t)(it_x / L::kBBufs) & 1u;
        const int nt = grp_x % p.n_tiles, b = grp_x / p.n_tiles;
        const int col0 = nt * BN + (int)rank * BNH;            // this CTA's half of the B columns
        for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
          const int bi = buf * kMaxKBlocks + kb;
          if (!ptx::mbar_wait(b_empty + bi, ph ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sb = smem + bi * kBBytes;
          const uint32_t bbar = ptx::map_to_cta(ptx::smem_u32(b_full + bi), 0);
          if (rank == 0) ptx::mbar_arrive_expect_tx(b_full + bi, (uint32_t)(2 * kBBytes));
#pragma unroll
          for (int j = 0; j < BNH / 64; ++j)
            ptx::tma_load_3d_pair(sb + j * kBoxBytes, &map_b, bbar, col0 + j * 64, kb * BK, b, pol_b);
        }
      };
      int it = 0;
      if (DBL && pair < n_groups) load_b(pair, 0);
      for (int grp = pair; grp < n_groups && ok; grp += n_pairs, ++it) {
        const int b = grp / p.n_tiles;
        if (!DBL) load_b(grp, it);                             // k-block by k-block behind the previous block's last MMAs
        for (int mt = 0; mt < p.m_tiles && ok; ++mt) {
          const int row0 = mt * 2 * BM + (int)rank * BM;       // this CTA's 128 rows of the 256-row tile
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + a_off + stage * kABytes;
            const uint32_t bar = ptx::map_to_cta(ptx::smem_u32(full + stage), 0);
            if (rank == 0) ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(2 * kABytes));
#pragma unroll
            for (int j = 0; j < BM / 64; ++j)
              ptx::tma_load_3d_pair(sa + j * kBoxBytes, &map_a, bar, row0 + j * 64, kb * BK, b, pol_a);
            if (++stage == kAStages) { stage = 0; phase ^= 1u; }
          }
          // the next column block's B slice goes into the other buffer once this block's first tile is on its way
          if (DBL && mt == 0 && ok && grp + n_pairs < n_groups) load_b(grp + n_pairs, it + 1);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) -------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(2 * BM, BN, true, true);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      int it = 0;
      for (int grp = pair; grp < n_groups && ok; grp += n_pairs, ++it) {
        const int bbase = (it % L::kBBufs) * kMaxKBlocks;
        const uint32_t b_phase = (uint32_t)(it / L::kBBufs) & 1u;
        for (int mt = 0; mt < p.m_tiles && ok; ++mt) {
          if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (mt == 0 && !ptx::mbar_wait(b_full + bbase + kb, b_phase, abort_flag)) { ok = false; break; }
            if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t sa = ptx::smem_u32(smem + a_off + stage * kABytes);
            const uint32_t sb = ptx::smem_u32(smem + (bbase + kb) * kBBytes);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              ptx::umma_bf16_pair(d_tmem, ptx::make_smem_desc(sa + k * 2048, kBoxBytes, 1024),
                                  ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024), idesc, (kb | k) != 0 ? 1u : 0u);
            ptx::umma_commit_pair(empty + stage);
            if (mt == p.m_tiles - 1) ptx::umma_commit_pair(b_empty + bbase + kb);   // last use of this B k-block
            if (++stage == kAStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          ptx::umma_commit_pair(acc_full + acc);
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs, own 128 rows) ----------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    unsigned char* stg = smem + stg_off + ew * kStgWarpBytes;
    int acc = 0; uint32_t acc_phase = 0;
    for (int grp = pair; grp < n_groups && ok; grp += n_pairs) {
      TileCoord t;
      t.nt = grp % p.n_tiles; t.b = grp / p.n_tiles;
      for (t.mt = 0; t.mt < p.m_tiles; ++t.mt) {
        const int tile_row0 = t.mt * 2 * BM + (int)rank * BM;
        if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        epilogue_tile<BN, false>(p, p.tma_store ? &map_c : nullptr, t, tile_row0, tmem_base + (uint32_t)(acc * BN), q, half,
                                 stg, lane);
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_remote_relaxed(ptx::map_to_cta(ptx::smem_u32(acc_empty + acc), 0));
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
  ptx::cluster_sync_all();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <bool DBL>
int launch2_resident_b(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const Params2& p, int pairs,
                       cudaStream_t st) {
  constexpr int smem_bytes = resb2::Lay<DBL>::smem_bytes;
  if (cudaFuncSetAttribute(umma2_gemm_resident_b_kernel<DBL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           smem_bytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, umma2_gemm_resident_b_kernel<DBL>, ma, mb, mc, p) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  count_launch();
  return GSHARD_OK;
}

template <bool A_K, bool B_K, bool MASK>
int launch2_t(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const Params2& p, int pairs,
              cudaStream_t st) {
  auto kern = umma2_gemm_kernel<A_K, B_K, MASK>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, ma, mb, mc, p) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  count_launch();
  return GSHARD_OK;
}

}  // namespace

// C[b] = act(A[b] . B[b]) with 256 x 256 tiles on CTA pairs; same operand conventions as
// launch_umma_gemm.  Worth it when a problem has more than one 128-row tile.
int launch_umma2_gemm(const UmmaGemm& g, int* status, cudaStream_t st) {
  if (g.rows <= 0 || g.cols <= 0 || g.K <= 0 || g.batch <= 0) return GSHARD_OK;
  if ((g.mask_bits || g.mask_bits_out) && g.cols % 32) return GSHARD_ERR_INTERNAL;   // one word per 32 columns
  CUtensorMap ma, mb;
  bool okm;
  if (g.a_kmajor) okm = make_map(&ma, g.A, g.K, g.rows, g.batch, g.a_ld, g.a_bs, BK, BM);
  else            okm = make_map(&ma, g.A, g.rows, g.K, g.batch, g.a_ld, g.a_bs, 64, BK);
  if (g.b_kmajor) okm = okm && make_map(&mb, g.B, g.K, g.cols, g.batch, g.b_ld, g.b_bs, BK, BNH);
  else            okm = okm && make_map(&mb, g.B, g.cols, g.K, g.batch, g.b_ld, g.b_bs, 64, BK);
  if (!okm) return GSHARD_ERR_CUDA;
  CUtensorMap mc;
  const bool tma_store = store_map_for(g, &mc);
  Params2 p;
  p.tma_store = tma_store ? 1 : 0;
  p.C = g.C; p.mask_bits = g.mask_bits; p.mask_bits_out = g.mask_bits_out; p.rows = g.rows; p.cols = g.cols; p.K = g.K; p.batch = g.batch;
  p.c_ld = g.c_ld; p.c_bs = g.c_bs;
  p.m_tiles = ceil_div(g.rows, 2 * BM); p.n_tiles = ceil_div(g.cols, BN);
  p.total_tiles = p.m_tiles * p.n_tiles * g.batch;
  p.k_blocks = ceil_div(g.K, BK);
  p.out_f32 = g.out_f32; p.relu = g.relu; p.a_stream = g.a_stream; p.b_stream = g.b_stream;
  p.n_fastest = (g.rows > g.cols) ? 1 : 0;
  p.status = status;
  p.tile_base = g.ragged_on_pairs ? g.tile_base : nullptr;
  p.tile_problem = g.tile_problem;
  if (p.tile_base && !p.tile_problem) return GSHARD_ERR_INTERNAL;
  if (p.tile_base) p.n_fastest = 0;            // ragged lists are walked with the row tiles fastest
  const int sms = device_sms();
  int pairs = sms / 2;
  if (g.max_ctas > 0 && pairs > g.max_ctas / 2) pairs = g.max_ctas / 2 > 0 ? g.max_ctas / 2 : 1;
  if (!g.a_kmajor && !g.b_kmajor && !g.mask_bits && !g.mask_bits_out && !p.tile_base && !g.out_f32 &&
      p.k_blocks <= resb2::kMaxKBlocks && p.m_tiles >= 2) {
    // short contraction, several row tiles per column block: B slice resident, deep A ring
    const int n_groups = p.n_tiles * g.batch;
    const int np = pairs < n_groups ? pairs : n_groups;
    // few row tiles per column block: the B slice changes often, keep the next one loading meanwhile
    return p.m_tiles < 16 ? launch2_resident_b<true>(ma, mb, mc, p, np, st) : launch2_resident_b<false>(ma, mb, mc, p, np, st);
  }
  if (pairs > p.total_tiles && !p.tile_base) pairs = p.total_tiles;   // ragged: count known on the device only
#define GSHARD_DISPATCH2(AK, BKM) \
  (p.mask_bits ? launch2_t<AK, BKM, true>(ma, mb, mc, p, pairs, st) : launch2_t<AK, BKM, false>(ma, mb, mc, p, pairs, st))
  if (g.a_kmajor && g.b_kmajor) return GSHARD_DISPATCH2(true, true);
  if (g.a_kmajor && !g.b_kmajor) return GSHARD_DISPATCH2(true, false);
  if (!g.a_kmajor && g.b_kmajor) return GSHARD_DISPATCH2(false, true);
  return GSHARD_DISPATCH2(false, false);
#undef GSHARD_DISPATCH2
}

}  // namespace gshard
