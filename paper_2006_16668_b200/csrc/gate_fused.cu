// Gating for the bf16 dtype in one tensor-core kernel (Algorithm 1: "g <- softmax(wg . x)" and
// "top_2"): logits = x . wg on tcgen05 with fp32 accumulation, and in the epilogue - while the
// accumulator is read out of tensor memory - the running row maximum, the running sum of
// exponentials (online softmax) and the two largest logits with their expert indices (softmax is
// monotone, so top-2 of the gates is top-2 of the logits; scanning experts in ascending order with
// strict comparisons makes the lowest index win ties).
//
// A persistent CTA owns a tile of 128 tokens and walks all expert-column tiles of that row tile,
// so x is streamed from HBM once (the 128 x M panel is re-read from L2 per column tile) and the
// per-token state lives in the registers of the epilogue thread that owns the token's TMEM lane.
// The fp32 logits are also stored: the mean gates m_e need the final row normaliser and are
// summed by a second, bandwidth-bound pass (gate.cu).
#include <cuda.h>

#include "kernels.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace gshard {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kABytes = BM * BK * 2;
constexpr int kBBytes = BN * BK * 2;
constexpr int kBoxBytes = 64 * 64 * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kStages = 4;
constexpr int kTmemCols = 2 * BN;
constexpr int kBarOff = kStages * kStageBytes;
constexpr int kStgOff = kBarOff + 256;
constexpr int kStgRowBytes = 128;
constexpr int kStgWarpBytes = 32 * kStgRowBytes;
constexpr int kSmemBytes = kStgOff + kEpiWarps * kStgWarpBytes + 1024;

struct GateParams {
  long long N;          // tokens
  int E, M;
  int row_tiles, n_tiles, k_blocks;
  float* logits;        // [N,E] fp32
  int32_t* expert_idx;  // [N,2]
  float* gate12;        // [N,2] raw softmax values of the two picks
  float* rowmax;        // [N]
  float* rowinv;        // [N] 1 / sum exp(logit - rowmax)
  int* status;
};

// (v1,i1),(v2,i2) <- top-2 of the union with (b1,k1),(b2,k2); larger value first, lower expert
// index on equal values.
__device__ __forceinline__ void top2_merge(float& v1, int& i1, float& v2, int& i2, float b1, int k1, float b2, int k2) {
  const bool first = b1 > v1 || (b1 == v1 && k1 < i1);          // the other set's best beats v1
  // candidates for second place: the loser of that comparison and the winner's own second
  const float l_v = first ? v1 : b1;
  const int l_i = first ? i1 : k1;
  const float w_v = first ? b2 : v2;
  const int w_i = first ? k2 : i2;
  v1 = first ? b1 : v1;
  i1 = first ? k1 : i1;
  const bool second = l_v > w_v || (l_v == w_v && l_i < w_i);
  v2 = second ? l_v : w_v;
  i2 = second ? l_i : w_i;
}

// 2^x with the hardware approximation (relative error about 2^-22, far inside the tolerance of the
// softmax sums; one instruction instead of the range-checked library sequence).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ int tile_cols(const GateParams& p, int nt) {   // multiple of 16, <= BN
  const int left = p.E - nt * BN;
  const int c = left < BN ? left : BN;
  return (c + 15) & ~15;
}

__global__ void __launch_bounds__(kThreads, 1)
gate_fused_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                  const GateParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;
  uint64_t* acc_full = bars + 2 * kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* x_full = acc_empty + 2;            // upper-half results of a row tile written
  uint64_t* x_empty = x_full + 1;              // ... and read
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(x_empty + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, kEpiWarps); }
    ptx::mbar_init(x_full, kEpiWarps / 2);
    ptx::mbar_init(x_empty, kEpiWarps / 2);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_x);
    ptx::prefetch_tensormap(&map_wg);
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
    if (lane == 0) {
      const uint64_t pol_x = ptx::policy_evict_last();     // a row panel is re-read for every column tile
      const uint64_t pol_w = ptx::policy_evict_last();     // wg is shared by every CTA
      int stage = 0; uint32_t phase = 0;
      for (int rt = blockIdx.x; rt < p.row_tiles && ok; rt += gridDim.x) {
        for (int nt = 0; nt < p.n_tiles && ok; ++nt) {
          const int boxes = (tile_cols(p, nt) + 63) / 64;
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + stage * kStageBytes;
            unsigned char* sb = sa + kABytes;
            ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(kABytes + boxes * kBoxBytes));
            ptx::tma_load_3d(sa, &map_x, full + stage, kb * BK, rt * BM, 0, pol_x);
            for (int j = 0; j < boxes; ++j)
              ptx::tma_load_3d(sb + j * kBoxBytes, &map_wg, full + stage, nt * BN + j * 64, kb * BK, 0, pol_w);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int rt = blockIdx.x; rt < p.row_tiles && ok; rt += gridDim.x) {
        for (int nt = 0; nt < p.n_tiles && ok; ++nt) {
          const uint32_t idesc = ptx::make_idesc_bf16(BM, tile_cols(p, nt), false, true);
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
    }
  } else {
    // epilogue: two warps per TMEM lane quarter; a thread owns one token (lane) and one half of
    // each column tile, and carries its state across the column tiles of the row tile.  The
    // running top-2 and the exp-sum are kept as four independent chains (columns i mod 4) so that
    // the per-element updates overlap instead of forming one long dependency chain; each chain
    // scans its columns in ascending order with strict comparisons, and chains (and then the two
    // halves, through shared memory) are merged with an explicit lowest-index tie rule.
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    constexpr int kHalfCols = BN / 2;
    unsigned char* stg = smem + kStgOff + ew * kStgWarpBytes;       // 32 rows x 128 B staging
    unsigned char* srow = stg + lane * kStgRowBytes;
    // exchange slot of this token: the staging row of the half-1 warp of the same lane quarter
    float* xchg = reinterpret_cast<float*>(smem + kStgOff + ((4 + (ew & 3)) * kStgWarpBytes) + lane * kStgRowBytes);
    int acc = 0; uint32_t acc_phase = 0, x_phase = 0;
    const float ninf = __int_as_float(0xff800000);
    constexpr float kLog2e = 1.4426950408889634f;
    for (int rt = blockIdx.x; rt < p.row_tiles && ok; rt += gridDim.x) {
      // the exchange slots alias the upper-half warps' staging rows: those warps may not stage
      // logits of this row tile before the previous tile's results have been read
      if (half == 1 && !ptx::mbar_wait_warp(x_empty, x_phase ^ 1u, abort_flag, lane)) { ok = false; break; }
      const long long row0 = (long long)rt * BM + q * 32;
      const long long row = row0 + lane;
      const bool row_ok = row < p.N;
      float m = ninf;                        // running maximum of this thread's columns
      float s4[4] = {0.f, 0.f, 0.f, 0.f};    // partial sums of exp(logit - m)
      float a1[4], a2[4];                    // per chain: two largest logits ...
      int j1[4], j2[4];                      // ... and their expert indices
#pragma unroll
      for (int k = 0; k < 4; ++k) { a1[k] = ninf; a2[k] = ninf; j1[k] = 0x7fffffff; j2[k] = 0x7fffffff; }
      for (int nt = 0; nt < p.n_tiles; ++nt) {
        if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t t_acc = tmem_base + (uint32_t)(acc * BN + half * kHalfCols) + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
        for (int c = 0; c < kHalfCols / 64; ++c) {      // 64 columns per round: two TMEM loads in flight
          const int cbase = nt * BN + half * kHalfCols + c * 64;
          if (cbase >= p.E) break;                       // uniform over the warp
          uint32_t r[2][32];
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64), r[0]);
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(c * 64 + 32), r[1]);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const int col0 = cbase + hh * 32;
            const int nv = min(32, p.E - col0);
            if (nv <= 0) break;                          // uniform over the warp
            float v[32];
            float cm[4] = {ninf, ninf, ninf, ninf};
            if (nv == 32) {                              // uniform over the warp
#pragma unroll
              for (int i = 0; i < 32; ++i) { v[i] = __uint_as_float(r[hh][i]); cm[i & 3] = fmaxf(cm[i & 3], v[i]); }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                v[i] = i < nv ? __uint_as_float(r[hh][i]) : ninf;
                cm[i & 3] = fmaxf(cm[i & 3], v[i]);
              }
            }
            const float cmax = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
            if (cmax > m) {
              const float sc = __expf(m - cmax);        // exp(-inf) = 0 on the first chunk
#pragma unroll
              for (int k = 0; k < 4; ++k) s4[k] *= sc;
              m = cmax;
            }
            const float ml = m * kLog2e;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int k = i & 3;
              s4[k] += ex2_approx(fmaf(v[i], kLog2e, -ml));  // exp(v - m); 0 for the padded columns
              const bool gt1 = v[i] > a1[k];
              const bool gt2 = v[i] > a2[k];
              a2[k] = gt1 ? a1[k] : (gt2 ? v[i] : a2[k]);
              j2[k] = gt1 ? j1[k] : (gt2 ? col0 + i : j2[k]);
              a1[k] = gt1 ? v[i] : a1[k];
              j1[k] = gt1 ? col0 + i : j1[k];
            }
            // logits: stage the 32 fp32 of this row (one 128-byte staging row, XOR-swizzled pieces),
            // then write 128-byte row segments: 8 lanes per row, 4 rows per instruction
#pragma unroll
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<float4*>(srow + ((i ^ (lane & 7)) * 16)) =
                  make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            __syncwarp();
            {
              const int piece = lane & 7;
              const int col = col0 + piece * 4;
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int rr = 4 * i + (lane >> 3);
                if (row0 + rr < p.N && col < p.E) {
                  const float4 val = *reinterpret_cast<const float4*>(stg + rr * kStgRowBytes + ((piece ^ (rr & 7)) * 16));
                  __stcs(reinterpret_cast<float4*>(p.logits + (row0 + rr) * p.E + col), val);
                }
              }
            }
            __syncwarp();
          }
        }
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_relaxed(acc_empty + acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) break;
      // merge this thread's four chains: larger value first, lower index on equal values
      float v1 = a1[0], v2 = a2[0];
      int i1 = j1[0], i2 = j2[0];
#pragma unroll
      for (int k = 1; k < 4; ++k) top2_merge(v1, i1, v2, i2, a1[k], j1[k], a2[k], j2[k]);
      float ssum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      // hand the upper half's result to the thread that owns the lower half of the same token
      // (bounded mbarrier hand-shake instead of a CTA barrier, so that a warp that gave up on a
      // wait cannot leave the others stuck)
      if (half == 1) {
        xchg[0] = m; xchg[1] = ssum; xchg[2] = v1; xchg[3] = v2;
        reinterpret_cast<int*>(xchg)[4] = i1; reinterpret_cast<int*>(xchg)[5] = i2;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(x_full);
      } else {
        if (!ptx::mbar_wait_warp(x_full, x_phase, abort_flag, lane)) { ok = false; break; }
      }
      if (half == 0 && row_ok) {
        const float m1 = xchg[0], s1 = xchg[1];
        top2_merge(v1, i1, v2, i2, xchg[2], reinterpret_cast<const int*>(xchg)[4], xchg[3],
                   reinterpret_cast<const int*>(xchg)[5]);
        const float mm = fmaxf(m, m1);
        ssum = ssum * expf(m - mm) + s1 * expf(m1 - mm);   // exp(-inf) = 0 when a half had no columns
        const float inv = 1.0f / ssum;
        p.expert_idx[2 * row] = i1;
        p.expert_idx[2 * row + 1] = i2;
        p.gate12[2 * row] = inv;                          // exp(v1 - mm) = 1
        p.gate12[2 * row + 1] = expf(v2 - mm) * inv;
        p.rowmax[row] = mm;
        p.rowinv[row] = inv;
      }
      if (half == 0) {
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(x_empty);          // exchange slots free again
      }
      x_phase ^= 1u;
    }
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
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

int launch_gate_fused(const Dims& d, const void* x, const void* wg, float* logits, int32_t* expert_idx,
                      float* gate12, float* rowmax, float* rowinv, int* status, cudaStream_t st) {
  GateParams p;
  p.N = d.N; p.E = d.E; p.M = d.M;
  p.row_tiles = (int)((d.N + BM - 1) / BM);
  p.n_tiles = ceil_div(d.E, BN);
  p.k_blocks = ceil_div(d.M, BK);
  p.logits = logits; p.expert_idx = expert_idx; p.gate12 = gate12; p.rowmax = rowmax; p.rowinv = rowinv;
  p.status = status;
  CUtensorMap mx, mw;
  bool okm = make_map(&mx, x, d.M, d.N, 1, d.M, 0, BK, BM);
  okm = okm && make_map(&mw, wg, d.E, d.M, 1, d.E, 0, 64, BK);
  if (!okm) return GSHARD_ERR_CUDA;
  const int sms = device_sms();
  const int grid = p.row_tiles < sms ? p.row_tiles : sms;
  if (cudaFuncSetAttribute(gate_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  gate_fused_kernel<<<grid, kThreads, kSmemBytes, st>>>(mx, mw, p);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

}  // namespace gshard
