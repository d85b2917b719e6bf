// Expert FFN in ONE persistent launch without a round trip of the hidden activations through HBM:
// out[e] = relu(buf[e] . wi[e]) . wo[e]   (eq. (2)).
//
// CTAs work in groups of four on one (expert, 128-row tile) unit at a time.  The hidden dimension
// is cut into chunks of 256 columns; in round T rank r of the group computes chunk 4T + r of
// h = relu(buf . wi) (GEMM-1, N = 256, K = M) into a TMEM accumulator, its epilogue warps store the
// bf16 chunk into a small per-group scratch ring (four rounds deep, 1 MB per group, so it lives in
// L2 and is overwritten before it is written back), and every rank then multiplies all four chunks
// of the round into its own quarter of the output columns (GEMM-2, N = M/4, K = 256 per chunk),
// accumulated in a second TMEM accumulator over the whole hidden dimension.  Each rank streams a
// quarter of wi and a quarter of wo: every weight byte leaves HBM once and h never does.  Every
// shared-memory stage carries 32 KB of weights, as in the stand-alone grouped GEMM, so the same
// number of HBM bytes is in flight per SM.
//
// Per CTA: warp 0 TMA producer, warp 1 tcgen05 issuer, warps 2..5 epilogue.  One shared-memory
// ring feeds both GEMMs; the issue order is G1(T), G2(T-1), G1(T+1), G2(T), ... so the hand-over of
// round T (epilogue -> scratch -> flag -> TMA load) hides behind GEMM-1 of round T+1.
//   chunk hand-over  prod[group][rank] counts finished epilogue warps (release); the producers of
//                    all four ranks acquire it, then fence the async proxy before the TMA load.
//   ring reuse       safe without further flags.  Rank r overwrites the slot of round T when its
//                    epilogue of round T+4 runs, i.e. after its G1(T+4) completed; tcgen05 MMAs
//                    complete in issue order, so its G2(T+2) completed, which needed the round
//                    T+2 chunks of every rank r'; r' stored that chunk after its own G1(T+2)
//                    completed, and r' issued G2(T) before G1(T+2): r' is done reading round T.
//   row gather       optional (Algorithm 2's dispatch fused into this launch): a seventh warp of
//                    every rank copies a quarter of the NEXT units' token rows from x, through
//                    the slot index list, into a per-group, two-unit-deep A-slot in the scratch
//                    (zeros for empty slots) and counts the unit in gath[group][rank] (release);
//                    the gather warp then acquires all four counters and arrives on a local
//                    mbarrier that the CTA's producer waits on before a unit's first A load.  The
//                    slot of unit i is overwritten for unit i + 2 only after prod[] shows that all
//                    four ranks finished every GEMM-1 of unit i.  The [E, G*C, M] dispatch buffer
//                    is then neither written nor read.
// All CTAs are co-resident (grid <= SM count, one CTA per SM, cooperative launch) and every wait is
// bounded in wall time, reporting GSHARD_ERR_TIMEOUT through the status word instead of hanging.
#include <cuda.h>

#include "kernels.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "ffn_shared.cuh"

namespace gshard {

namespace {

using namespace ffn_shared;

constexpr int BM = 128, BK = 64;
constexpr int KC = 256;                       // hidden columns per chunk
constexpr int kGroup = 4;                     // CTAs per unit
constexpr int kRing = 4;                      // scratch ring depth in rounds
constexpr int kEpiWarps = 4;
constexpr int kThreads = 64 + 32 * kEpiWarps + 32;   // + the row-gather warp
constexpr int kGatherWarp = 2 + kEpiWarps;
constexpr int kASlots = 2;                    // gathered units in flight per group
constexpr int kABytes = BM * BK * 2;          // 16 KB
constexpr int kBoxBytes = 64 * 64 * 2;        // 8 KB
constexpr int kStageBytes = kABytes + 4 * kBoxBytes;   // 48 KB: A + up to 256 B-columns
constexpr int kStages = 4;
constexpr int kBarOff = kStages * kStageBytes;
constexpr int kStgOff = kBarOff + 256;
constexpr int kSmemBytes = kStgOff + kEpiWarps * kStgWarpBytes + 1024;
constexpr uint32_t kOutCol = 0, kG1Col = 256; // TMEM columns: out accumulator, GEMM-1 accumulator

struct GroupParams {
  __nv_bfloat16* scratch;   // [groups][kRing][kGroup][128][KC]
  __nv_bfloat16* out;       // [E][rows][M]
  int rows, M, H, E;
  int m_tiles, rounds, k1_blocks, NW;   // NW = M / 4 output columns per rank
  int units, groups;
  int* prod;                // [groups][kGroup] finished epilogue warps per rank
  int* status;
  // row-gather mode (x != nullptr): A rows of unit (e, mt) come from x[G*S, M] through
  // slot_token[E][G*C] into a_slots[groups][kASlots][128][M]
  const uint4* x;
  const int32_t* slot_token;
  uint4* a_slots;
  int* gath;                // [groups][kGroup] units gathered by each rank
  int S, C;
};

__global__ void __launch_bounds__(kThreads, 1)
ffn_group4_kernel(const __grid_constant__ CUtensorMap map_buf, const __grid_constant__ CUtensorMap map_wi,
                  const __grid_constant__ CUtensorMap map_hs, const __grid_constant__ CUtensorMap map_wo,
                  const GroupParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kBarOff);
  uint64_t* full = bars;                    // [kStages]
  uint64_t* empty = bars + kStages;         // [kStages]
  uint64_t* g1_full = bars + 2 * kStages;   // [1]
  uint64_t* g1_empty = g1_full + 1;         // [1]
  uint64_t* out_full = g1_empty + 1;        // [1]
  uint64_t* out_empty = out_full + 1;       // [1]
  uint64_t* a_ready = out_empty + 1;        // [kASlots] gathered rows of a unit complete on all ranks
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(a_ready + kASlots);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = blockIdx.x / kGroup, rank = blockIdx.x % kGroup;
  // units of this group: group, group + groups, ...
  const int my_units = group < p.units ? (p.units - group + p.groups - 1) / p.groups : 0;
  const int total_T = my_units * p.rounds;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    ptx::mbar_init(g1_full, 1);
    ptx::mbar_init(g1_empty, kEpiWarps);
    ptx::mbar_init(out_full, 1);
    ptx::mbar_init(out_empty, kEpiWarps);
    for (int a = 0; a < kASlots; ++a) ptx::mbar_init(a_ready + a, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_buf); ptx::prefetch_tensormap(&map_wi);
    ptx::prefetch_tensormap(&map_hs); ptx::prefetch_tensormap(&map_wo);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const int wo_boxes = (p.NW + 63) / 64;

  bool ok = true;
  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      const uint64_t pol_w = ptx::policy_evict_first();    // weights: read exactly once
      const uint64_t pol_a = ptx::policy_evict_last();     // buf and the h chunks: re-read from L2
      int stage = 0; uint32_t phase = 0;
      for (int T = 0; T <= total_T && ok; ++T) {
        if (T < total_T) {                                 // GEMM-1 of round T: chunk 4t + rank
          const int u = group + (T / p.rounds) * p.groups, t = T % p.rounds;
          const int e = u / p.m_tiles, mt = u % p.m_tiles;
          const int hcol = (t * kGroup + rank) * KC;
          const int ui = T / p.rounds;
          if (p.x && t == 0) {                             // this unit's gathered rows are complete
            if (!ptx::mbar_wait(a_ready + (ui % kASlots), (uint32_t)(ui / kASlots) & 1u, abort_flag)) { ok = false; break; }
            asm volatile("fence.proxy.async;" ::: "memory");
          }
          const int a_row = p.x ? 0 : mt * BM;
          const int a_idx = p.x ? group * kASlots + (ui % kASlots) : e;
          for (int kb = 0; kb < p.k1_blocks; ++kb) {
            if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + stage * kStageBytes;
            unsigned char* sb = sa + kABytes;
            ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(kABytes + (KC / 64) * kBoxBytes));
            ptx::tma_load_3d(sa, &map_buf, full + stage, kb * BK, a_row, a_idx, pol_a);
#pragma unroll
            for (int j = 0; j < KC / 64; ++j)
              ptx::tma_load_3d(sb + j * kBoxBytes, &map_wi, full + stage, hcol + j * 64, kb * BK, e, pol_w);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
        }
        if (T >= 1) {                                      // GEMM-2 of round T-1: all four chunks
          const int Tp = T - 1;
          const int u = group + (Tp / p.rounds) * p.groups, t = Tp % p.rounds;
          const int e = u / p.m_tiles;
          for (int rr = 0; rr < kGroup && ok; ++rr) {
            // chunk of rank rr: complete and visible to the async proxy before the TMA load
            if (!wait_counter(p.prod + group * kGroup + rr, (Tp + 1) * kEpiWarps, abort_flag)) { ok = false; break; }
            asm volatile("fence.proxy.async;" ::: "memory");
            const int slot = (group * kRing + (Tp % kRing)) * kGroup + rr;
            const int hrow = (t * kGroup + rr) * KC;       // rows of wo = hidden index
            for (int kk = 0; kk < KC / BK; ++kk) {
              if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
              unsigned char* sa = smem + stage * kStageBytes;
              unsigned char* sb = sa + kABytes;
              ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(kABytes + wo_boxes * kBoxBytes));
              ptx::tma_load_3d(sa, &map_hs, full + stage, kk * BK, 0, slot, pol_a);
              for (int j = 0; j < wo_boxes; ++j)
                ptx::tma_load_3d(sb + j * kBoxBytes, &map_wo, full + stage, rank * p.NW + j * 64, hrow + kk * BK, e, pol_w);
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (lane == 0) {
      const uint32_t idesc1 = ptx::make_idesc_bf16(BM, KC, false, true);
      const uint32_t idesc2 = ptx::make_idesc_bf16(BM, p.NW, false, true);
      int stage = 0; uint32_t phase = 0;
      for (int T = 0; T <= total_T && ok; ++T) {
        if (T < total_T) {
          if (!ptx::mbar_wait(g1_empty, ((uint32_t)T & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + kG1Col;
          for (int kb = 0; kb < p.k1_blocks; ++kb) {
            if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t sa = ptx::smem_u32(smem + stage * kStageBytes);
            const uint32_t sb = sa + kABytes;
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              ptx::umma_bf16(d_tmem, ptx::make_smem_desc(sa + k * 32, 16, 1024),
                             ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024), idesc1, (kb | k) != 0 ? 1u : 0u);
            ptx::umma_commit(empty + stage);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          ptx::umma_commit(g1_full);
        }
        if (T >= 1) {
          const int Tp = T - 1;
          const int ui = Tp / p.rounds, t = Tp % p.rounds;
          if (t == 0) {     // first GEMM-2 of a unit: the previous unit's output must have been read out
            if (!ptx::mbar_wait(out_empty, ((uint32_t)ui & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after_sync();
          }
          const uint32_t d_tmem = tmem_base + kOutCol;
          for (int rr = 0; rr < kGroup && ok; ++rr) {
            for (int kk = 0; kk < KC / BK; ++kk) {
              if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
              ptx::tc_fence_after_sync();
              const uint32_t sa = ptx::smem_u32(smem + stage * kStageBytes);
              const uint32_t sb = sa + kABytes;
#pragma unroll
              for (int k = 0; k < BK / 16; ++k)
                ptx::umma_bf16(d_tmem, ptx::make_smem_desc(sa + k * 32, 16, 1024),
                               ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024), idesc2,
                               (t | rr | kk | k) != 0 ? 1u : 0u);
              ptx::umma_commit(empty + stage);
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
          }
          if (!ok) break;
          if (t == p.rounds - 1) ptx::umma_commit(out_full);
        }
      }
    }
  } else if (warp == kGatherWarp) {
    // ------------------------------ row gather --------------------------------------------
    if (p.x) {
      const int row_vec = p.M / 8;                           // 16-byte pieces per row
      const uint64_t pol_keep = ptx::policy_evict_last();    // the slots are re-read 32 times from L2
      constexpr int kRowsPerRank = BM / kGroup;
      for (int ui = 0; ui < my_units && ok; ++ui) {
        const int u = group + ui * p.groups;
        const int e = u / p.m_tiles, mt = u % p.m_tiles;
        if (ui >= kASlots) {
          // the slot's previous unit: every rank has finished all of its GEMM-1 rounds
          const int target = (ui - kASlots + 1) * p.rounds * kEpiWarps;
          int w = 1;
          if (lane < kGroup) w = wait_counter(p.prod + group * kGroup + lane, target, abort_flag, 2000) ? 1 : 0;
          if (__any_sync(0xffffffffu, w == 0)) { ok = false; break; }
        }
        uint4* dst = p.a_slots + ((size_t)(group * kASlots + (ui % kASlots)) * BM + rank * kRowsPerRank) * row_vec;
#pragma unroll 1
        for (int r0 = 0; r0 < kRowsPerRank; r0 += 4) {
          const uint4* src[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int row = mt * BM + rank * kRowsPerRank + r0 + i;
            src[i] = nullptr;
            if (row < p.rows) {
              const int s_tok = __ldg(p.slot_token + (long long)e * p.rows + row);
              if (s_tok >= 0) src[i] = p.x + ((long long)(row / p.C) * p.S + s_tok) * row_vec;
            }
          }
          for (int v0 = 0; v0 < row_vec; v0 += 32 * 4) {
            uint4 val[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int v = v0 + j * 32 + lane;
                val[i][j] = (src[i] && v < row_vec) ? __ldg(src[i] + v) : make_uint4(0u, 0u, 0u, 0u);
              }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int v = v0 + j * 32 + lane;
                if (v < row_vec)
                  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(
                                   dst + (size_t)(r0 + i) * row_vec + v),
                               "r"(val[i][j].x), "r"(val[i][j].y), "r"(val[i][j].z), "r"(val[i][j].w), "l"(pol_keep)
                               : "memory");
              }
          }
        }
        __threadfence();                                     // rows visible GPU-wide ...
        asm volatile("fence.proxy.async;" ::: "memory");     // ... and to the async proxy (TMA)
        __syncwarp();
        if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.gath + group * kGroup + rank) : "memory");
        // all four quarters of the unit are in place: tell this CTA's producer through shared
        // memory, so that its only wait at the start of a unit is a local one
        int w = 1;
        if (lane < kGroup) w = wait_counter(p.gath + group * kGroup + lane, ui + 1, abort_flag, 500) ? 1 : 0;
        if (__any_sync(0xffffffffu, w == 0)) { ok = false; break; }
        asm volatile("fence.proxy.async;" ::: "memory");
        if (lane == 0) ptx::mbar_arrive(a_ready + (ui % kASlots));
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------------------
    const int ew = warp - 2;
    const int q = warp & 3;                                  // TMEM lane quarter
    unsigned char* stg = smem + kStgOff + ew * kStgWarpBytes;
    unsigned char* srow = stg + lane * kStgRowBytes;
    const uint32_t lane_sel = (uint32_t)(q * 32) << 16;
    for (int T = 0; T <= total_T && ok; ++T) {
      if (T < total_T) {
        // h chunk of round T: TMEM -> relu -> bf16 -> scratch slot of this rank
        if (!ptx::mbar_wait_warp(g1_full, (uint32_t)T & 1u, abort_flag, lane)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const int slot = (group * kRing + (T % kRing)) * kGroup + rank;
        __nv_bfloat16* dst = p.scratch + ((size_t)slot * BM + q * 32) * KC;
        const uint32_t t_acc = tmem_base + kG1Col + lane_sel;
#pragma unroll 1
        for (int c = 0; c < KC / 64; ++c) {
          uint32_t r0[32], r1[32];
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64), r0);
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64 + 32), r1);
          ptx::tmem_ld_wait();
          stage_chunk(r0, true, srow, lane, 0);
          stage_chunk(r1, true, srow, lane, 4);
          flush_block(stg, dst + c * 64, KC, 32, 64, lane);
        }
        ptx::tc_fence_before_sync();
        __threadfence();                                     // chunk visible GPU-wide ...
        asm volatile("fence.proxy.async;" ::: "memory");     // ... and to the async proxy (TMA)
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(g1_empty);
          asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.prod + group * kGroup + rank) : "memory");
        }
      }
      if (T >= 1 && (T - 1) % p.rounds == p.rounds - 1) {
        // a unit is complete: its output quarter TMEM -> bf16 -> out
        const int ui = (T - 1) / p.rounds;
        const int u = group + ui * p.groups;
        const int e = u / p.m_tiles, mt = u % p.m_tiles;
        if (!ptx::mbar_wait_warp(out_full, (uint32_t)ui & 1u, abort_flag, lane)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const int row0 = mt * BM + q * 32;
        __nv_bfloat16* dst = p.out + ((size_t)e * p.rows + row0) * p.M + rank * p.NW;
        const uint32_t t_acc = tmem_base + kOutCol + lane_sel;
#pragma unroll 1
        for (int c = 0; c * 64 < p.NW; ++c) {
          uint32_t r0[32], r1[32];
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64), r0);
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64 + 32), r1);
          ptx::tmem_ld_wait();
          stage_chunk(r0, false, srow, lane, 0);
          stage_chunk(r1, false, srow, lane, 4);
          flush_block(stg, dst + c * 64, p.M, p.rows - row0, p.NW - c * 64, lane);
        }
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(out_empty);
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
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

// Shapes the four-CTA kernel handles: the output columns split evenly over four ranks with at most
// 256 per rank, the hidden dimension in whole rounds of four 256-column chunks.
bool ffn_fused_supported(const Dims& d) {
  return d.bf16 && d.M % 64 == 0 && d.M <= 1024 && d.H % (kGroup * KC) == 0 && (d.M / 4) % 16 == 0 &&
         device_sms() >= kGroup;
}

// Scratch bytes: the per-group chunk ring plus the hand-over counters.
size_t ffn_fused_scratch_bytes(const Dims& d) {
  const size_t groups = 256 / kGroup;            // enough for any SM count up to 256
  return groups * kRing * kGroup * BM * KC * 2 + 256 + groups * 2 * kGroup * sizeof(int) + 256 +
         groups * kASlots * BM * (size_t)d.M * 2;
}

int launch_ffn_fused(const Dims& d, const void* buf, const void* wi, const void* wo, void* scratch, void* out,
                     int* status, cudaStream_t st, const void* x_gather, const int32_t* slot_token) {
  GroupParams p;
  const int sms = device_sms();
  p.groups = sms / kGroup;
  if (p.groups > 256 / kGroup) p.groups = 256 / kGroup;
  p.rows = d.rows; p.M = d.M; p.H = d.H; p.E = d.E;
  p.m_tiles = ceil_div(d.rows, BM);
  p.rounds = d.H / (kGroup * KC);
  p.k1_blocks = ceil_div(d.M, BK);
  p.NW = d.M / kGroup;
  p.units = d.E * p.m_tiles;
  if (p.groups > p.units) p.groups = p.units;
  const size_t ring_bytes = (size_t)(256 / kGroup) * kRing * kGroup * BM * KC * 2;
  p.scratch = static_cast<__nv_bfloat16*>(scratch);
  p.prod = reinterpret_cast<int*>(static_cast<unsigned char*>(scratch) + ring_bytes + 256);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.gath = p.prod + (256 / kGroup) * kGroup;
  p.a_slots = reinterpret_cast<uint4*>(static_cast<unsigned char*>(scratch) + ring_bytes + 256 +
                                       (size_t)(256 / kGroup) * 2 * kGroup * sizeof(int) + 256);
  p.x = static_cast<const uint4*>(x_gather);
  p.slot_token = slot_token; p.S = d.S; p.C = d.C;
  p.status = status;
  if (cudaMemsetAsync(p.prod, 0, sizeof(int) * (256 / kGroup) * 2 * kGroup, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  CUtensorMap m_buf, m_wi, m_hs, m_wo;
  const long long rows = d.rows;
  bool okm = x_gather ? make_map(&m_buf, p.a_slots, d.M, BM, (long long)p.groups * kASlots, d.M, (long long)BM * d.M, BK, BM)
                      : make_map(&m_buf, buf, d.M, rows, d.E, d.M, rows * d.M, BK, BM);
  okm = okm && make_map(&m_wi, wi, d.H, d.M, d.E, d.H, (long long)d.M * d.H, 64, BK);
  okm = okm && make_map(&m_hs, scratch, KC, BM, (long long)p.groups * kRing * kGroup, KC, (long long)BM * KC, BK, BM);
  okm = okm && make_map(&m_wo, wo, d.M, d.H, d.E, d.M, (long long)d.H * d.M, 64, BK);
  if (!okm) return GSHARD_ERR_CUDA;
  if (cudaFuncSetAttribute(ffn_group4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  // The four CTAs of a group wait on one another's counters, so every CTA of the grid must be
  // resident at once.  A cooperative launch makes the runtime guarantee that: it starts the grid
  // only when all of it fits beside whatever else the process is running, and refuses a grid that
  // can never fit.  A refusal launches nothing and is reported as "unsupported" so that the caller
  // falls back to the two grouped-GEMM launches.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.groups * kGroup), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, ffn_group4_kernel, m_buf, m_wi, m_hs, m_wo, p) != cudaSuccess) {
    cudaGetLastError();
    return GSHARD_ERR_UNSUPPORTED_SHAPE;
  }
  count_launch();
  return GSHARD_OK;
}

}  // namespace gshard
