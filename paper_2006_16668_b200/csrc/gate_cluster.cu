// Gating for the bf16 dtype with the mean gates fused in (Algorithm 1: "g <- softmax(wg . x)",
// "m_E <- mean of g", "top_2"): no logits leave the chip.
//
// A thread-block cluster of CL = ceil(E / 256) CTAs owns a tile of 128 tokens; CTA r computes the
// logits of experts [256 r, 256 r + 256) on tcgen05 (x k-blocks and its wg slice by TMA, fp32
// accumulator in tensor memory, two accumulators so that the next tile's MMAs run under this
// tile's epilogue).  The softmax normaliser of a token spans all CTAs, so the epilogue reads the
// accumulator twice:
//   pass 1  per thread (= token row, a quarter of the CTA's columns): running maximum, sum of
//           exponentials, two largest logits with their expert indices (lowest index wins ties);
//           the four column parts of a row are merged through shared memory, then the CTA's partial
//           (max, sum) is stored into the shared memory of EVERY CTA of the cluster and its top-2
//           into the CTA that finalises that row quarter (distributed shared memory), followed by a
//           remote mbarrier arrive (release.cluster)
//   pass 2  after all CL partials of the tile have arrived (acquire.cluster): global row maximum
//           and normaliser; the finalising warp merges the top-2 partials in ascending expert order
//           and writes e1, e2, g1, g2, row max, 1/Z; every warp re-reads its accumulator columns,
//           forms exp(l - max)/Z and adds them over its 32 rows with a shuffle transpose-reduce
//           (fixed tree), writing one row of column sums per 32-token block.
// gate_mean_kernel then adds a group's blocks in order: m[g,e] = (1/S) sum.  The partial-stat
// buffers are double-buffered by tile parity; a CTA cannot run two tiles ahead of a peer because
// each tile needs every peer's arrival, which a peer issues only after all of its epilogue warps
// finished the tile before.  Every wait is bounded; all CTAs meet at a cluster barrier before any
// of them exits (no CTA may receive a remote store after it has gone).
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
constexpr int kBoxBytes = 64 * 64 * 2;
constexpr int kStageBytes = kABytes + (BN / 64) * kBoxBytes;   // 48 KB
constexpr int kStages = 4;
constexpr int kTmemCols = 2 * BN;
constexpr int kMaxCl = 8;
constexpr int kBarOff = kStages * kStageBytes;
constexpr int kMzOff = kBarOff + 256;                          // float2 [2][kMaxCl][BM]
constexpr int kT2Off = kMzOff + 2 * kMaxCl * BM * 8;           // uint4  [2][8 slots][32]
constexpr int kPairOff = kT2Off + 2 * 8 * 32 * 16;             // 24 B   [4 quarters][3 parts][32]
constexpr int kSmemBytes = kPairOff + 4 * 3 * 32 * 24 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget");

struct ClusterGateParams {
  long long N;          // tokens
  int E, M;
  int row_tiles, k_blocks, cl, nclusters;
  int32_t* expert_idx;  // [N,2]
  float* gate12;        // [N,2] raw softmax values of the two picks
  float* rowmax;        // [N]
  float* rowinv;        // [N] 1 / sum exp(logit - rowmax)
  float* partial32;     // [ceil(N/32)][E] column sums of the softmax over 32-token blocks
  int* status;
};

__device__ __forceinline__ void st_remote_f2(uint32_t cluster_addr, float a, float b) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(cluster_addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void st_remote_u4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d)
               : "memory");
}
__device__ __forceinline__ bool try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t"
      ".reg .pred P;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 P, [%1], %2, %3;\n\t"
      "selp.b32 %0, 1, 0, P;\n\t"
      "}"
      : "=r"(ok)
      : "r"(ptx::smem_u32(bar)), "r"(parity), "r"(2000u)
      : "memory");
  return ok != 0;
}
// Whole-warp bounded wait with cluster-scope acquire (the data was stored by other CTAs).
__device__ __forceinline__ bool wait_warp_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int lane) {
  int done = 1;
  if (lane == 0) {
    done = 0;
    const uint64_t t0 = ptx::globaltimer_ns();
    uint32_t it = 0;
    while (true) {
      if (try_wait_cluster(bar, parity)) { done = 1; break; }
      if ((++it & 63u) == 0 && (*abort_flag || ptx::globaltimer_ns() - t0 > 2000000000ull)) break;
    }
  }
  done = __shfl_sync(0xffffffffu, done, 0);
  // every lane reads remote-written data: each takes its own acquire (returns at once, the phase
  // has completed) instead of one cluster-scope fence for the warp
  if (done && lane != 0) (void)try_wait_cluster(bar, parity);
  return done != 0;
}

// (v1,i1),(v2,i2) <- top-2 of the union with (b1,k1),(b2,k2); larger value first, lower expert
// index on equal values.
__device__ __forceinline__ void top2_merge(float& v1, int& i1, float& v2, int& i2, float b1, int k1, float b2, int k2) {
  const bool first = b1 > v1 || (b1 == v1 && k1 < i1);
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

__device__ __forceinline__ int cta_cols(const ClusterGateParams& p, int rank) {   // multiple of 16, <= BN
  const int left = p.E - rank * BN;
  const int c = left < BN ? left : BN;
  return c <= 0 ? 0 : (c + 15) & ~15;
}

// 2^x with the hardware approximation (relative error about 2^-22, far inside the tolerance of the
// softmax sums; one instruction instead of the range-checked library sequence).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// v[j] of lane l -> lane j returns sum over lanes of v[j] (fixed reduction tree).
__device__ __forceinline__ float transpose_reduce32(float* v, int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool up = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < off; ++i) {
      const float send = up ? v[i] : v[i + off];
      const float keep = up ? v[i + off] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return v[0];
}

__global__ void __launch_bounds__(kThreads, 1)
gate_cluster_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_wg,
                    const ClusterGateParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kBarOff);
  uint64_t* full = bars;                       // [kStages]
  uint64_t* empty = full + kStages;            // [kStages]
  uint64_t* acc_full = empty + kStages;        // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint64_t* pair_full = acc_empty + 2;         // [4] upper-half result of a row quarter written
  uint64_t* pair_empty = pair_full + 4;        // [4] ... and read
  uint64_t* stats_full = pair_empty + 4;       // [2] all CL partials of a tile have arrived
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(stats_full + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float2* mz = reinterpret_cast<float2*>(smem + kMzOff);
  uint4* t2 = reinterpret_cast<uint4*>(smem + kT2Off);
  float* pairbuf = reinterpret_cast<float*>(smem + kPairOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)ptx::cluster_ctarank();
  const int cid = blockIdx.x / p.cl;
  const int cols = cta_cols(p, rank);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(full + s, 1); ptx::mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(acc_full + a, 1); ptx::mbar_init(acc_empty + a, kEpiWarps); }
    for (int q = 0; q < 4; ++q) { ptx::mbar_init(pair_full + q, 3); ptx::mbar_init(pair_empty + q, 1); }
    for (int a = 0; a < 2; ++a) ptx::mbar_init(stats_full + a, (uint32_t)(p.cl * 4));
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
  ptx::cluster_sync_all();                          // every CTA's barriers exist before any remote arrive
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = true;
  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      const uint64_t pol = ptx::policy_evict_last();       // x tile: read by every CTA of the cluster; wg: by every cluster
      const int boxes = (cols + 63) / 64;
      int stage = 0; uint32_t phase = 0;
      for (int rt = cid; rt < p.row_tiles && ok; rt += p.nclusters) {
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait(empty + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sa = smem + stage * kStageBytes;
          unsigned char* sb = sa + kABytes;
          ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)(kABytes + boxes * kBoxBytes));
          ptx::tma_load_3d(sa, &map_x, full + stage, kb * BK, rt * BM, 0, pol);
          for (int j = 0; j < boxes; ++j)
            ptx::tma_load_3d(sb + j * kBoxBytes, &map_wg, full + stage, rank * BN + j * 64, kb * BK, 0, pol);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_bf16(BM, cols, false, true);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int rt = cid; rt < p.row_tiles && ok; rt += p.nclusters) {
        if (!ptx::mbar_wait(acc_empty + acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!ptx::mbar_wait(full + stage, phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * kStageBytes);
          const uint32_t sb = sa + kABytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            ptx::umma_bf16(d_tmem, ptx::make_smem_desc(sa + k * 32, 16, 1024),
                           ptx::make_smem_desc(sb + k * 2048, kBoxBytes, 1024), idesc, (kb | k) != 0 ? 1u : 0u);
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
    // Sixteen warps: four per TMEM lane quarter (= row quarter of the tile), each taking a quarter
    // (64) of the CTA's columns, so that four warps per scheduler hide each other's latencies.
    const int ew = warp - 2;
    const int q = warp & 3;                          // TMEM lane quarter this warp may access
    const int part = ew >> 2;                        // which 64 of the CTA's 256 columns
    const int qpc = (4 + p.cl - 1) / p.cl;           // row quarters finalised per CTA
    const int fin = q % p.cl;                        // CTA that finalises this row quarter
    float* pslot = pairbuf + ((q * 3 + (part > 0 ? part - 1 : 0)) * 32 + lane) * 6;
    const float ninf = __int_as_float(0xff800000);
    constexpr float kLog2e = 1.4426950408889634f;
    const int wcol0 = rank * BN + part * 64;         // first expert of this warp's columns
    // CTA partial of the tile whose pass 1 ran last (held by the part-0 warps until published)
    float c_m = ninf, c_s = 0.f, c_v1 = ninf, c_v2 = ninf;
    int c_i1 = 0, c_i2 = 0;

    // ---- pass 1 of the tile with running number `it1` in accumulator `acc1` --------------------
    // maximum, sum of exponentials and top-2 over this thread's 64 columns (four independent
    // chains, columns i mod 4; expert indices relative to wcol0 so that they are compile-time
    // constants in the unrolled scan)
    auto pass1 = [&](uint32_t it1, int acc1, uint32_t phase1) -> bool {
      const uint32_t t_acc = tmem_base + (uint32_t)(acc1 * BN + part * 64) + ((uint32_t)(q * 32) << 16);
      if (!ptx::mbar_wait_warp(acc_full + acc1, phase1, abort_flag, lane)) return false;
      ptx::tc_fence_after_sync();
      float m = ninf;
      float s4[4] = {0.f, 0.f, 0.f, 0.f};
      float a1[4], a2[4];
      int j1[4], j2[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) { a1[k] = ninf; a2[k] = ninf; j1[k] = 0x3fffffff; j2[k] = 0x3fffffff; }
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int nv = p.E - (wcol0 + hh * 32);      // valid columns of this chunk (uniform over the warp)
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
            const float sc = __expf(m - cmax);       // exp(-inf) = 0 on the first chunk
#pragma unroll
            for (int k = 0; k < 4; ++k) s4[k] *= sc;
            m = cmax;
          }
          const float ml = m * kLog2e;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int k = i & 3;
            s4[k] += ex2_approx(fmaf(v[i], kLog2e, -ml));
            const bool gt1 = v[i] > a1[k];
            const bool gt2 = v[i] > a2[k];
            a2[k] = gt1 ? a1[k] : (gt2 ? v[i] : a2[k]);
            j2[k] = gt1 ? j1[k] : (gt2 ? hh * 32 + i : j2[k]);
            a1[k] = gt1 ? v[i] : a1[k];
            j1[k] = gt1 ? hh * 32 + i : j1[k];
          }
        }
      }
      float v1 = a1[0], v2 = a2[0];
      int i1 = j1[0], i2 = j2[0];
#pragma unroll
      for (int k = 1; k < 4; ++k) top2_merge(v1, i1, v2, i2, a1[k], j1[k], a2[k], j2[k]);
      i1 += wcol0; i2 += wcol0;
      float ssum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
      const uint32_t pr_phase = it1 & 1u;
      if (part != 0) {                               // hand-over slot; the arrive follows in handoff()
        if (!ptx::mbar_wait_warp(pair_empty + q, pr_phase ^ 1u, abort_flag, lane)) return false;
        pslot[0] = m; pslot[1] = ssum; pslot[2] = v1; pslot[3] = v2;
        reinterpret_cast<int*>(pslot)[4] = i1; reinterpret_cast<int*>(pslot)[5] = i2;
      } else {
        c_m = m; c_s = ssum; c_v1 = v1; c_v2 = v2; c_i1 = i1; c_i2 = i2;
      }
      return true;
    };

    // ---- the four column parts of a row meet in shared memory: parts 1..3 release their slots,
    // part 0 merges them into the CTA's partial of the row -------------------------------------
    auto handoff = [&](uint32_t it1) -> bool {
      const uint32_t pr_phase = it1 & 1u;
      if (part != 0) {
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(pair_full + q);
        return true;
      }
      if (!ptx::mbar_wait_warp(pair_full + q, pr_phase, abort_flag, lane)) return false;
#pragma unroll
      for (int o = 0; o < 3; ++o) {                  // ascending column parts: ties keep the lowest index
        const float* ps = pairbuf + ((q * 3 + o) * 32 + lane) * 6;
        const float m1 = ps[0], s1 = ps[1];
        top2_merge(c_v1, c_i1, c_v2, c_i2, ps[2], reinterpret_cast<const int*>(ps)[4], ps[3],
                   reinterpret_cast<const int*>(ps)[5]);
        const float mm = fmaxf(c_m, m1);
        c_s = c_s * __expf(c_m - mm) + s1 * __expf(m1 - mm);   // exp(-inf) = 0 when a part had no columns
        c_m = mm;
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(pair_empty + q);
      return true;
    };

    // ---- part-0 warps: this CTA's partial of a row goes to every CTA ((max, sum)) and to the CTA
    // that finalises the row quarter (top-2), then one remote arrive per CTA --------------------
    auto publish = [&](uint32_t it1) {
      const uint32_t par = it1 & 1u;
      const uint32_t mz_addr = ptx::smem_u32(mz + ((par * kMaxCl + rank) * BM + q * 32 + lane));
      for (int r = 0; r < p.cl; ++r) st_remote_f2(ptx::map_to_cta(mz_addr, (uint32_t)r), c_m, c_s);
      const int slot = rank * qpc + q / p.cl;
      st_remote_u4(ptx::map_to_cta(ptx::smem_u32(t2 + ((par * 8 + slot) * 32 + lane)), (uint32_t)fin), __float_as_uint(c_v1),
                   __float_as_uint(c_v2), (uint32_t)c_i1, (uint32_t)c_i2);
      __syncwarp();
      if (lane < p.cl) ptx::mbar_arrive_remote_release(ptx::map_to_cta(ptx::smem_u32(stats_full + par), (uint32_t)lane));
    };

    // Tile loop.  Pass 1 and pass 2 of a tile run back to back (the second accumulator lets the
    // next tile's MMAs run meanwhile); an order that runs pass 1 of tile t+1 before pass 2 of tile t
    // hides the exchange latency but holds both accumulators and measured slower.  A peer overwrites
    // the parity buffer of tile t with tile t+2 only after it has received our partials of tile t+1,
    // which the part-0 warps send after all four warps of their row quarter finished tile t.
    int acc1 = 0; uint32_t phase1 = 0;               // accumulator of the current tile
    int acc2 = 0;
    const int n_my = cid < p.row_tiles ? (p.row_tiles - cid + p.nclusters - 1) / p.nclusters : 0;
    for (int t = 0; t < n_my && ok; ++t) {
      const uint32_t it = (uint32_t)t;
      const int rt = cid + t * p.nclusters;
      if (!(pass1(it, acc1, phase1) && handoff(it))) { ok = false; break; }
      if (part == 0) publish(it);
      if (++acc1 == 2) { acc1 = 0; phase1 ^= 1u; }
      const uint32_t par = it & 1u, st_phase = (it >> 1) & 1u;
      const long long row0 = (long long)rt * BM + q * 32;
      const long long row = row0 + lane;
      const bool row_ok = row < p.N;

      // ---- all partials of tile t: global maximum and normaliser of this thread's row ----------
      if (!wait_warp_cluster(stats_full + par, st_phase, abort_flag, lane)) { ok = false; break; }
      float mx = ninf;
      for (int r = 0; r < p.cl; ++r) mx = fmaxf(mx, mz[(par * kMaxCl + r) * BM + q * 32 + lane].x);
      float z = 0.f;
      for (int r = 0; r < p.cl; ++r) {
        const float2 pz = mz[(par * kMaxCl + r) * BM + q * 32 + lane];
        z += pz.y * __expf(pz.x - mx);
      }
      const float inv = 1.0f / z;
      if (part == 0 && rank == fin) {
        // merge the CL top-2 partials in ascending expert order (ties: lowest index)
        const uint4 f0 = t2[(par * 8 + (q / p.cl)) * 32 + lane];
        float w1 = __uint_as_float(f0.x), w2 = __uint_as_float(f0.y);
        int k1 = (int)f0.z, k2 = (int)f0.w;
        for (int r = 1; r < p.cl; ++r) {
          const uint4 fr = t2[(par * 8 + r * qpc + q / p.cl) * 32 + lane];
          top2_merge(w1, k1, w2, k2, __uint_as_float(fr.x), (int)fr.z, __uint_as_float(fr.y), (int)fr.w);
        }
        if (row_ok) {
          p.expert_idx[2 * row] = k1;
          p.expert_idx[2 * row + 1] = k2;
          p.gate12[2 * row] = expf(w1 - mx) * inv;          // w1 == mx: exp(0) = 1
          p.gate12[2 * row + 1] = expf(w2 - mx) * inv;
          p.rowmax[row] = mx;
          p.rowinv[row] = inv;
        }
      }

      // ---- pass 2: softmax values of this thread's row, summed over the warp's 32 rows --------
      const uint32_t t_acc = tmem_base + (uint32_t)(acc2 * BN + part * 64) + ((uint32_t)(q * 32) << 16);
      const float mxl = mx * kLog2e;
      const float scale = row_ok ? inv : 0.f;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int col0 = wcol0 + hh * 32;
        if (col0 < p.E) {                             // uniform over the warp
          uint32_t r[32];
          ptx::tmem_ld_32x32(t_acc + (uint32_t)(hh * 32), r);
          ptx::tmem_ld_wait();
          float pv[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) pv[i] = ex2_approx(fmaf(__uint_as_float(r[i]), kLog2e, -mxl)) * scale;
          const float cs = transpose_reduce32(pv, lane);
          if (row0 < p.N && col0 + lane < p.E) p.partial32[(row0 >> 5) * p.E + col0 + lane] = cs;
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_relaxed(acc_empty + acc2);
      acc2 ^= 1;
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
  ptx::cluster_sync_all();                  // no CTA leaves while a peer may still store into its shared memory
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

// Shapes the cluster kernel takes: at most eight 256-expert column tiles (one CTA each) and token
// groups made of whole 32-token blocks (a block's column sums belong to one group).
bool gate_cluster_supported(const Dims& d) {
  return d.bf16 && !d.simt && d.E <= kMaxCl * BN && d.E % 16 == 0 && d.S % 32 == 0 && d.M % 64 == 0;
}

// Launches the kernel; returns GSHARD_ERR_UNSUPPORTED_SHAPE without launching when no cluster of the
// needed size can be resident (the caller then takes the two-pass form).
int launch_gate_cluster(const Dims& d, const void* x, const void* wg, int32_t* expert_idx, float* gate12,
                        float* rowmax, float* rowinv, float* partial32, int* status, cudaStream_t st) {
  ClusterGateParams p;
  p.N = d.N; p.E = d.E; p.M = d.M;
  p.row_tiles = (int)((d.N + BM - 1) / BM);
  p.k_blocks = ceil_div(d.M, BK);
  p.cl = ceil_div(d.E, BN);
  p.expert_idx = expert_idx; p.gate12 = gate12; p.rowmax = rowmax; p.rowinv = rowinv; p.partial32 = partial32;
  p.status = status;
  CUtensorMap mx, mw;
  bool okm = make_map(&mx, x, d.M, d.N, 1, d.M, 0, BK, BM);
  okm = okm && make_map(&mw, wg, d.E, d.M, 1, d.E, 0, 64, BK);
  if (!okm) return GSHARD_ERR_CUDA;
  if (cudaFuncSetAttribute(gate_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // every cluster of the grid must be resident at once (persistent tiles, peers wait on each other)
  const int sms = device_sms();
  cfg.gridDim = dim3((unsigned)(sms / p.cl * p.cl), 1, 1);
  int max_clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&max_clusters, gate_cluster_kernel, &cfg) != cudaSuccess || max_clusters < 1) {
    cudaGetLastError();
    return GSHARD_ERR_UNSUPPORTED_SHAPE;
  }
  p.nclusters = max_clusters < p.row_tiles ? max_clusters : p.row_tiles;
  cfg.gridDim = dim3((unsigned)(p.nclusters * p.cl), 1, 1);
  if (cudaLaunchKernelEx(&cfg, gate_cluster_kernel, mx, mw, p) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  count_launch();
  return GSHARD_OK;
}

}  // namespace gshard
