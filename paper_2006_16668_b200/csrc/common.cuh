// Shared declarations of the CUDA library: shape helpers, status word, element conversion.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include "../../include/gshard_moe.h"

namespace gshard {

constexpr int kGateTile = 128;        // tokens per column-sum partial of the mean gates
constexpr size_t kAlign = 256;        // alignment of every workspace region

__host__ __device__ inline size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }
__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Device status word: first error wins; 0 = OK.
__device__ inline void set_device_status(int* status, int code) { atomicCAS(status, 0, code); }

template <typename T> __device__ inline float to_f32(T v);
template <> __device__ inline float to_f32<float>(float v) { return v; }
template <> __device__ inline float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ inline T from_f32(float v);
template <> __device__ inline float from_f32<float>(float v) { return v; }
template <> __device__ inline __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16 bytes of a row as fp32 values: 4 floats, or 8 bfloat16 widened / rounded to nearest even.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int n = 4;
  __device__ static void load(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static uint4 store(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int n = 8;
  __device__ static void load(const uint4& v, float* f) {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static uint4 store(const float* f) {
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<const unsigned*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// Multiprocessors of the current device (grids of the persistent and grid-stride kernels).
inline int device_sms() {
  int sms = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
    cudaGetLastError();
    return 1;
  }
  return sms;
}

// Grid of the one-warp-per-row kernels (256 threads = 8 rows per block, grid-stride beyond 32
// blocks per multiprocessor).
inline int grid_for_rows(long long rows) {
  const long long blocks = (rows + 7) / 8;
  const long long cap = (long long)device_sms() * 32;
  return (int)(blocks < cap ? (blocks > 0 ? blocks : 1) : cap);
}

// NVTX range around a stage's launches (header-only NVTX 3: a no-op unless a profiler injects itself).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

struct LaunchCounter {
  int n = 0;
};
LaunchCounter& launch_counter();   // thread-local
inline void count_launch(int k = 1) { launch_counter().n += k; }

// Sizes derived from a shape.
struct Dims {
  int G, S, M, H, E, C;
  long long N;          // tokens
  long long R;          // slots = E*G*C
  int rows;             // rows per expert = G*C
  int tiles_per_group;  // ceil(S / kGateTile)
  size_t esize;         // bytes of one x / weight element
  bool bf16;
  bool simt;            // contractions on CUDA cores
  bool variant_a;
  bool fused_ffn;       // force the single-launch FFN (h handed over through L2)
  bool unfused_ffn;     // force the two grouped-GEMM launches (h through HBM)
  bool two_sm_mma;      // grouped GEMMs on CTA pairs (tcgen05 cta_group::2) where rows > 128
  bool add_residual;    // y = x + layer(x); dx gains dy
  bool one_sm_mma;      // never use CTA pairs for the grouped GEMMs
  bool gate_one_sm;     // stored-logits gating kernel on single CTAs instead of CTA pairs
  bool gate_cluster;    // gating on clusters with the mean-gate partial sums fused in (no stored logits)
  bool gather_dispatch; // single-launch FFN gathers its rows from x instead of reading a dispatch buffer
  bool tf32_experts;    // fp32 dtype: expert FFN contractions on the tensor cores in TF32
  bool compact_slots;   // grouped-GEMM expert FFN over compacted rows (empty slots skipped)
  bool bulk_dispatch;   // dispatch rows move through the TMA unit (cp.async.bulk) instead of 16-byte loads and stores
  bool plain_stores;    // GEMM epilogues write with 16-byte stores instead of bulk tensor (TMA) stores
  bool debug_checks;    // forward: verify the routing tensors on the device and record a violation in the status word
  bool bwd_paired;      // backward: read-heavy and write-heavy expert GEMMs side by side on half of the SMs each
};

inline Dims make_dims(const gshard_moe_shape& s) {
  Dims d;
  d.G = s.G; d.S = s.S; d.M = s.M; d.H = s.H; d.E = s.E; d.C = s.C;
  d.N = (long long)s.G * s.S;
  d.R = (long long)s.E * s.G * s.C;
  d.rows = s.G * s.C;
  d.tiles_per_group = ceil_div(s.S, kGateTile);
  d.bf16 = s.dtype == GSHARD_BF16;
  d.esize = d.bf16 ? 2 : 4;
  d.simt = !d.bf16 || (s.flags & GSHARD_FLAG_SIMT_CONTRACTIONS);
  d.variant_a = (s.flags & GSHARD_FLAG_SECOND_SKIP_FREES_SLOT) != 0;
  d.fused_ffn = (s.flags & GSHARD_FLAG_FUSED_FFN) != 0;
  d.unfused_ffn = (s.flags & GSHARD_FLAG_UNFUSED_FFN) != 0;
  d.two_sm_mma = (s.flags & GSHARD_FLAG_TWO_SM_MMA) != 0;
  d.gather_dispatch = (s.flags & GSHARD_FLAG_GATHER_DISPATCH) != 0;
  d.gate_cluster = (s.flags & GSHARD_FLAG_GATE_CLUSTER) != 0;
  d.gate_one_sm = (s.flags & GSHARD_FLAG_GATE_ONE_SM) != 0;
  d.one_sm_mma = (s.flags & GSHARD_FLAG_ONE_SM_MMA) != 0;
  d.add_residual = (s.flags & GSHARD_FLAG_ADD_RESIDUAL) != 0;
  d.bwd_paired = (s.flags & GSHARD_FLAG_BWD_PAIRED_GEMMS) != 0;
  d.plain_stores = (s.flags & GSHARD_FLAG_PLAIN_STORES) != 0;
  d.bulk_dispatch = (s.flags & GSHARD_FLAG_BULK_DISPATCH) != 0;
  d.debug_checks = (s.flags & GSHARD_FLAG_DEBUG_CHECKS) != 0;
  d.tf32_experts = !d.bf16 && (s.flags & GSHARD_FLAG_TF32_EXPERTS) != 0;
  // Compacted slots: on request, and by default wherever the expert FFN runs as two grouped GEMMs (more
  // than one 128-row tile per expert), so that the usual 13-30 % of empty slots free row tiles: the
  // kept rows run in 256-row tiles on CTA pairs and the 128-row tile that may remain on a single CTA.
  // Measured: MoE(128E) shape 3.44 against 3.79 ms per step for a burst, 3.88 against 4.11 ms sustained
  // under the power cap; MoE(512E) shape (256 slots per expert, mostly still one pair tile) 3.92 against
  // 4.00 ms and 4.26 against 4.36 ms.  A flag that names another GEMM form switches the default off.
  const bool other_form = (s.flags & (GSHARD_FLAG_ONE_SM_MMA | GSHARD_FLAG_TWO_SM_MMA | GSHARD_FLAG_FUSED_FFN)) != 0;
  d.compact_slots = d.bf16 && !d.simt && !(s.flags & GSHARD_FLAG_SAVE_FOR_BACKWARD) &&
                    ((s.flags & GSHARD_FLAG_COMPACT_SLOTS) != 0 || (d.rows > 128 && !other_form));
  return d;
}

}  // namespace gshard
