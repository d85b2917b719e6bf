// Epilogue of the grouped tcgen05 GEMMs (one-SM and CTA-pair kernels): accumulator rows out of tensor
// memory, ReLU / mask, conversion, staging in swizzled shared memory, 128-byte row stores.  `P` is
// the kernel's parameter struct (C, mask, rows, cols, c_ld, c_bs, out_f32, relu).
#pragma once
#include "kernels.cuh"
#include "sm100_ptx.cuh"

namespace gshard {
namespace umma_epi {

constexpr int kTileRows = 128;
constexpr int kStgRowBytes = 128;           // staging: 32 rows x 128 bytes per warp
constexpr int kStgWarpBytes = 32 * kStgRowBytes;

struct TileCoord { int mt, nt, b; };

// Ragged batches (compacted expert rows).  Problem b owns the row tiles [tile_base[b], tile_base[b+1]) of
// a device-side prefix array with batch + 1 entries, and tile_problem[r] names the problem that owns
// row tile r, so a tile index is decoded with three loads and no search; the callers decode the NEXT
// tile before they work on the current one, which hides those loads.  Within a problem the row tiles
// run fastest: they share the B tile.
template <typename P>
__device__ __forceinline__ TileCoord decode_ragged(const P& p, int tile) {
  TileCoord t;
  t.b = __ldg(p.tile_problem + tile / p.n_tiles);
  const int first = __ldg(p.tile_base + t.b);
  const int m_b = __ldg(p.tile_base + t.b + 1) - first;
  const int i = tile - first * p.n_tiles;
  t.mt = i % m_b; t.nt = i / m_b;
  return t;
}

// Writes a warp's staged 32 rows x 128 bytes to C: lane l handles 16-byte piece (l & 7) of rows
// 4*i + (l >> 3); pieces beyond the matrix edge are skipped (cols is a multiple of the piece width).
// Whether the output rows should be kept in L2 (they are re-read soon by the same launch).  A kernel
// whose parameter struct wants that overloads this for its struct.
template <typename P>
__device__ __forceinline__ bool epi_keep_in_l2(const P&) { return false; }

template <typename P>
__device__ __forceinline__ void flush_rows(const unsigned char* stg, const P& p, int b, int row0, int col0,
                                           int lane) {
  __syncwarp();
  const bool keep = epi_keep_in_l2(p);
  const uint64_t pol = keep ? ptx::policy_evict_last() : 0ull;
  const int esz = p.out_f32 ? 4 : 2;
  const int piece = lane & 7;
  const int col = col0 + piece * (16 / esz);
  unsigned char* cbase = reinterpret_cast<unsigned char*>(p.C) + ((long long)b * p.c_bs + col) * esz;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = 4 * i + (lane >> 3);
    const int row = row0 + r;
    if (row < p.rows && col < p.cols) {
      const uint4 val = *reinterpret_cast<const uint4*>(stg + r * kStgRowBytes + ((piece ^ (r & 7)) * 16));
      uint4* dst = reinterpret_cast<uint4*>(cbase + (long long)row * p.c_ld * esz);
      if (keep)
        asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(dst), "r"(val.x), "r"(val.y),
                     "r"(val.z), "r"(val.w), "l"(pol)
                     : "memory");
      else
        *dst = val;
    }
  }
  __syncwarp();
}

// The same block through the TMA unit: the warp's 32 staged rows x 128 bytes (already in the 128-byte
// swizzle a tensor map expects, the staging block being 1024-byte aligned) leave as one bulk tensor
// store; rows and columns beyond the matrix are clipped by the tensor map.  Compared with flush_rows
// this takes the re-read of the staging rows and the global stores off the load/store pipe.  The
// staging block may be rewritten only after store_wait().
__device__ __forceinline__ void flush_rows_tma(const unsigned char* stg, const CUtensorMap* map_c, int b, int row0,
                                               int col0, int lane) {
  ptx::fence_proxy_async();          // this lane's staged bytes visible to the async proxy
  __syncwarp();
  if (lane == 0) {
    ptx::tma_store_3d(map_c, stg, col0, row0, b);
    ptx::tma_store_commit();
  }
}
__device__ __forceinline__ void store_wait(int lane) {
  if (lane == 0) ptx::tma_store_wait_read();
  __syncwarp();
}

// ReLU / mask on one 32-column chunk of this thread's row, then into the staging row (XOR-swizzled
// 16-byte pieces: conflict-free for the row-wise writes here and the piece-wise reads of the flush).
// mword: with MASK, bit i set = keep column i of the chunk.
template <bool MASK, typename P>
__device__ __forceinline__ void process_chunk(const uint32_t* r, const P& p, unsigned char* srow, int lane,
                                              int piece0, uint32_t mword) {
  float v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    v[i] = __uint_as_float(r[i]);
    if (p.relu) v[i] = fmaxf(v[i], 0.f);
    if (MASK && !((mword >> i) & 1u)) v[i] = 0.f;
  }
  if (p.out_f32) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      *reinterpret_cast<float4*>(srow + (((piece0 + i) ^ (lane & 7)) * 16)) =
          make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const __nv_bfloat162 pr = __floats2bfloat162_rn(v[8 * i + 2 * j], v[8 * i + 2 * j + 1]);
        w[j] = *reinterpret_cast<const uint32_t*>(&pr);
      }
      *reinterpret_cast<uint4*>(srow + (((piece0 + i) ^ (lane & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// First column of round c of this warp's half of the tile.
template <int BN>
__device__ __forceinline__ int round_col0(const TileCoord& t, int half, int c) {
  return t.nt * BN + half * (BN / 2) + c * 64;
}

// Bit i of the result: accumulator value i of the chunk is positive (the ReLU passes it).
__device__ __forceinline__ uint32_t positive_bits(const uint32_t* r) {
  uint32_t w = 0;
#pragma unroll
  for (int i = 0; i < 32; ++i) w |= (__uint_as_float(r[i]) > 0.f ? 1u : 0u) << i;
  return w;
}

// One epilogue warp's share of a finished 128 x BN accumulator whose first row is tile_row0: lane
// quarter q, column half `half`.  map_c: tensor map of C for bulk stores, or nullptr for plain 16-byte
// stores.  With MASK (bf16 output only) the output is zeroed where the bit of p.mask_bits
// ([batch][rows][cols/32] words, bit = column mod 32) is clear; the two words of a thread's row and
// round are fetched while the accumulator load is in flight.  With p.mask_bits_out the same layout is
// WRITTEN: bit = accumulator value positive (the ReLU mask the backward pass needs).
template <int BN, bool MASK, typename P>
__device__ __forceinline__ void epilogue_tile(const P& p, const CUtensorMap* map_c, const TileCoord& t, int tile_row0,
                                              uint32_t tmem_acc, int q, int half, unsigned char* stg, int lane) {
  constexpr int kHalfCols = BN / 2;
  unsigned char* srow = stg + lane * kStgRowBytes;
  const int row0 = tile_row0 + q * 32;
  const int row = row0 + lane;
  const long long word_row = ((long long)t.b * p.rows + row) * (p.cols >> 5);
  const uint32_t t_acc = tmem_acc + (uint32_t)(half * kHalfCols) + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
  for (int c = 0; c < kHalfCols / 64; ++c) {     // 64 columns per round: two TMEM loads in flight
    const int col0 = round_col0<BN>(t, half, c);
    if (col0 >= p.cols) break;                   // uniform over the warp
    uint32_t r0[32], r1[32];
    ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64), r0);
    ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64 + 32), r1);
    uint32_t m0 = 0, m1 = 0;
    if (MASK && row < p.rows) {
      m0 = __ldg(p.mask_bits + word_row + (col0 >> 5));
      if (col0 + 32 < p.cols) m1 = __ldg(p.mask_bits + word_row + (col0 >> 5) + 1);
    }
    if (map_c) store_wait(lane);                 // the previous bulk store has read the staging block
    ptx::tmem_ld_wait();
    if (p.mask_bits_out && row < p.rows) {
      p.mask_bits_out[word_row + (col0 >> 5)] = positive_bits(r0);
      if (col0 + 32 < p.cols) p.mask_bits_out[word_row + (col0 >> 5) + 1] = positive_bits(r1);
    }
    if (p.out_f32) {                             // 32 fp32 columns = one 128-byte staging row
      process_chunk<MASK>(r0, p, srow, lane, 0, m0);
      if (map_c) { flush_rows_tma(stg, map_c, t.b, row0, col0, lane); store_wait(lane); }
      else flush_rows(stg, p, t.b, row0, col0, lane);
      process_chunk<MASK>(r1, p, srow, lane, 0, m1);
      if (map_c) flush_rows_tma(stg, map_c, t.b, row0, col0 + 32, lane);
      else flush_rows(stg, p, t.b, row0, col0 + 32, lane);
    } else {                                     // 64 bf16 columns = one 128-byte staging row
      process_chunk<MASK>(r0, p, srow, lane, 0, m0);
      process_chunk<MASK>(r1, p, srow, lane, 4, m1);
      if (map_c) flush_rows_tma(stg, map_c, t.b, row0, col0, lane);
      else flush_rows(stg, p, t.b, row0, col0, lane);
    }
  }
}

// After a warp's last tile: its bulk stores have left shared memory and reached global memory.
__device__ __forceinline__ void epilogue_finish(const CUtensorMap* map_c, int lane) {
  if (map_c && lane == 0) ptx::tma_store_wait_all();
  __syncwarp();
}

}  // namespace umma_epi
}  // namespace gshard
