// Gating for the bf16 dtype on CTA pairs (tcgen05.mma.cta_group::2): the same computation as
// gate_fused.cu - logits = x . wg with fp32 accumulation and, while the accumulator is read out of
// tensor memory, the online softmax statistics and the top-2 pick of Algorithm 1, plus the stored
// fp32 logits for the mean-gate pass (here in the granule-transposed layout [E/4][N][4]) - but a pair of CTAs (a cluster of two) works on 256 tokens:
// each CTA loads its own 128 token rows of x and only HALF of the 256-expert slice of wg per
// k-block (32 KB per stage instead of 48 KB), and the leader's MMA thread multiplies both halves
// into the accumulators of both CTAs.  The one-SM kernel is bound by the operand feed from L2
// (768 KB per 128 x 256 tile); the pair needs 512 KB per CTA for the same tile.  Each CTA's
// epilogue works on its own 128 rows exactly as in the one-SM kernel.
// Pair protocol (as in umma2_gemm.cu): both producers' loads complete on the leader's full
// barrier, tcgen05.commit arrives on the stage / accumulator barriers of both CTAs, the peer's
// epilogue releases the accumulator on the leader's barrier, cluster barriers bracket all
// cross-CTA traffic.  No load is multicast.  Every wait is bounded.
#include <cuda.h>

#include "kernels.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace gshard {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kEpiWarps = 16;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kABytes = BM * BK * 2;
constexpr int BNH = BN / 2;
constexpr int kBBytes = BNH * BK * 2;          // this CTA's half of the wg tile
constexpr int kBoxBytes = 64 * 64 * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kStages = 6;
constexpr int kTmemCols = 2 * BN;
constexpr int kBarOff = kStages * kStageBytes;
constexpr int kStgOff = kBarOff + 256;
constexpr int kXchgOff = kStgOff;                                // 24 B [4 quarters][3 parts][32 rows]
constexpr int kSmemBytes = kXchgOff + 4 * 3 * 32 * 24 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget");

struct GateParams {
  long long N;          // tokens
  int E, M;
  int row_tiles, n_tiles, k_blocks;   // row tiles of 128 tokens; a pair takes two
  float* logits;        // fp32, granules of four experts: float4 [E/4][N]
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
gate_fused2_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                  const GateParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;
  uint64_t* acc_full = bars + 2 * kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* x_full = acc_empty + 2;            // [4] results of column parts 1..3 of a row quarter written
  uint64_t* x_empty = x_full + 4;              // [4] ... and read
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(x_empty + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int pair_tiles = (p.row_tiles + 1) / 2;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, 2 * kEpiWarps); }
    for (int qq = 0; qq < 4; ++qq) { ptx::mbar_init(x_full + qq, 3); ptx::mbar_init(x_empty + qq, 1); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_x);
    ptx::prefetch_tensormap(&map_wg);
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
    if (lane == 0) {
      const uint64_t pol_x = ptx::policy_evict_last();     // a row panel is re-read for every column tile
      const uint64_t pol_w = ptx::policy_evict_last();     // wg is shared by every CTA
      int stage = 0; uint32_t phase = 0;
      for (int pt = pair; pt < pair_tiles && ok; pt += n_pairs) {
        const int rt = 2 * pt + (int)rank;               // this CTA's 128 tokens of the pair's 256
        for (int nt = 0; nt < p.n_tiles && ok; ++nt) {
          const int half_cols = tile_cols(p, nt) / 2;      // this CTA's half of the tile's expert columns
          const int boxes = half_cols / 64;
          for (int kb = 0; kb < p.k_blocks; ++kb) {
            if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + stage * kStageBytes;
            unsigned char* sb = sa + kABytes;
            const uint32_t bar = ptx::map_to_cta(ptx::smem_u32(full + stage), 0);
            if (rank == 0) ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(2 * (kABytes + boxes * kBoxBytes)));
            ptx::tma_load_3d_pair(sa, &map_x, bar, kb * BK, rt * BM, 0, pol_x);
            for (int j = 0; j < boxes; ++j)
              ptx::tma_load_3d_pair(sb + j * kBoxBytes, &map_wg, bar, nt * BN + (int)rank * half_cols + j * 64, kb * BK, 0, pol_w);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {                      // the leader issues the MMAs of the pair
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int pt = pair; pt < pair_tiles && ok; pt += n_pairs) {
        for (int nt = 0; nt < p.n_tiles && ok; ++nt) {
          const uint32_t idesc = ptx::make_idesc_bf16(2 * BM, tile_cols(p, nt), false, true);
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
    }
  } else {
    // epilogue: four warps per TMEM lane quarter (sixteen in all, four per scheduler, so that they
    // hide each other's instruction latencies); a thread owns one token (lane) and a quarter (64)
    // of each column tile's experts, and carries its softmax state across the column tiles of the
    // row tile.  Within a column tile the top-2 and the exp-sum run as four independent chains
    // (columns i mod 4) with compile-time expert indices; the tile's result is merged into the
    // thread's running top-2 (explicit lowest-index tie rule), and at the end of the row tile the
    // four column parts of a token meet in shared memory.
    const int ew = warp - 2;
    const int q = warp & 3;
    const int part = ew >> 2;
    float* xslot = reinterpret_cast<float*>(smem + kXchgOff) + ((q * 3 + (part > 0 ? part - 1 : 0)) * 32 + lane) * 6;
    int acc = 0; uint32_t acc_phase = 0, x_phase = 0;
    const float ninf = __int_as_float(0xff800000);
    constexpr float kLog2e = 1.4426950408889634f;
    for (int pt = pair; pt < pair_tiles && ok; pt += n_pairs) {
      const int rt = 2 * pt + (int)rank;
      const long long row0 = (long long)rt * BM + q * 32;
      const long long row = row0 + lane;
      const bool row_ok = row < p.N;
      float m = ninf;                        // running maximum of this thread's columns
      float s4[4] = {0.f, 0.f, 0.f, 0.f};    // partial sums of exp(logit - m)
      float g1 = ninf, g2 = ninf;            // running two largest logits ...
      int gi1 = 0x7fffffff, gi2 = 0x7fffffff;   // ... and their expert indices
      for (int nt = 0; nt < p.n_tiles; ++nt) {
        if (!ptx::mbar_wait_warp(acc_full + acc, acc_phase, abort_flag, lane)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t t_acc = tmem_base + (uint32_t)(acc * BN + part * 64) + ((uint32_t)(q * 32) << 16);
        const int wcol0 = nt * BN + part * 64;           // first expert of this warp's columns in this tile
        float a1[4], a2[4];
        int j1[4], j2[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) { a1[k] = ninf; a2[k] = ninf; j1[k] = 0x3fffffff; j2[k] = 0x3fffffff; }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int col0 = wcol0 + hh * 32;
          const int nv = p.E - col0;                     // valid columns of this chunk (uniform over the warp)
          if (nv > 0) {
            uint32_t r[32];
            ptx::tmem_ld_32x32(t_acc + (uint32_t)(hh * 32), r);
            ptx::tmem_ld_wait();
            float v[32];
            float cm[4] = {ninf, ninf, ninf, ninf};
            if (nv >= 32) {
#pragma unroll
              for (int i = 0; i < 32; ++i) { v[i] = __uint_as_float(r[i]); cm[i & 3] = fmaxf(cm[i & 3], v[i]); }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) { v[i] = i < nv ? __uint_as_float(r[i]) : ninf; cm[i & 3] = fmaxf(cm[i & 3], v[i]); }
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
              j2[k] = gt1 ? j1[k] : (gt2 ? hh * 32 + i : j2[k]);
              a1[k] = gt1 ? v[i] : a1[k];
              j1[k] = gt1 ? hh * 32 + i : j1[k];
            }
            // logits, in 16-byte granules of four experts laid out [E/4][N]: the 32 lanes (32
            // consecutive tokens) of one store instruction write 512 contiguous bytes, so the rows
            // need no staging in shared memory (whose bandwidth the MMA operand reads and the TMA
            // writes already use up); the column-sum pass reads the same layout
            if (row_ok) {
              float4* dst = reinterpret_cast<float4*>(p.logits) + (long long)(col0 >> 2) * p.N + row;
#pragma unroll
              for (int i = 0; i < 8; ++i)
                if (col0 + 4 * i < p.E)
                  __stcs(dst + (long long)i * p.N, make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
            }
          }
        }
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_remote_relaxed(ptx::map_to_cta(ptx::smem_u32(acc_empty + acc), 0));   // the leader's barrier
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        // this column tile's four chains, then into the running top-2 (ascending expert order)
        float v1 = a1[0], v2 = a2[0];
        int i1 = j1[0], i2 = j2[0];
#pragma unroll
        for (int k = 1; k < 4; ++k) top2_merge(v1, i1, v2, i2, a1[k], j1[k], a2[k], j2[k]);
        top2_merge(g1, gi1, g2, gi2, v1, i1 + wcol0, v2, i2 + wcol0);
      }
      if (!ok) break;
      float ssum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      // the four column parts of a token meet in shared memory (bounded mbarrier hand-shakes
      // instead of a CTA barrier, so that a warp that gave up on a wait cannot leave the others stuck)
      if (part != 0) {
        if (!ptx::mbar_wait_warp(x_empty + q, x_phase ^ 1u, abort_flag, lane)) { ok = false; break; }
        xslot[0] = m; xslot[1] = ssum; xslot[2] = g1; xslot[3] = g2;
        reinterpret_cast<int*>(xslot)[4] = gi1; reinterpret_cast<int*>(xslot)[5] = gi2;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(x_full + q);
      } else {
        if (!ptx::mbar_wait_warp(x_full + q, x_phase, abort_flag, lane)) { ok = false; break; }
        const float* xs = reinterpret_cast<const float*>(smem + kXchgOff) + (q * 3 * 32 + lane) * 6;
#pragma unroll
        for (int o = 0; o < 3; ++o) {
          const float* ps = xs + o * 32 * 6;
          const float m1 = ps[0], s1 = ps[1];
          top2_merge(g1, gi1, g2, gi2, ps[2], reinterpret_cast<const int*>(ps)[4], ps[3], reinterpret_cast<const int*>(ps)[5]);
          const float mm = fmaxf(m, m1);
          ssum = ssum * expf(m - mm) + s1 * expf(m1 - mm);   // exp(-inf) = 0 when a part had no columns
          m = mm;
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(x_empty + q);        // exchange slots free again
        if (row_ok) {
          const float inv = 1.0f / ssum;
          p.expert_idx[2 * row] = gi1;
          p.expert_idx[2 * row + 1] = gi2;
          p.gate12[2 * row] = expf(g1 - m) * inv;            // g1 == m: exp(0) = 1
          p.gate12[2 * row + 1] = expf(g2 - m) * inv;
          p.rowmax[row] = m;
          p.rowinv[row] = inv;
        }
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
  ptx::cluster_sync_all();                  // no CTA frees TMEM or exits while its peer may still use it
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace

// Shapes the pair kernel takes: every 256-expert column tile splits into two halves of whole
// 64-column boxes.
bool gate_fused2_supported(const Dims& d) {
  return d.bf16 && !d.simt && d.E % 128 == 0 && d.M % 64 == 0;
}

int launch_gate_fused2(const Dims& d, const void* x, const void* wg, float* logits, int32_t* expert_idx,
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
  const int pair_tiles = (p.row_tiles + 1) / 2;
  const int pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
  if (cudaFuncSetAttribute(gate_fused2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
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
  if (cudaLaunchKernelEx(&cfg, gate_fused2_kernel, mx, mw, p) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  count_launch();
  return GSHARD_OK;
}

}  // namespace gshard
