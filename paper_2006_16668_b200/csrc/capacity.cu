// Capacity assignment (Algorithm 1, the two token loops and l_aux) without a sequential scan
// over tokens.  The paper's running counter c_e gives token s the position
//   first choice : #{s' < s : e1(s') = e1(s)}
//   second choice: c1[e2(s)] + #{s' < s : e2(s') = e2(s)}      (c1 = counts after loop 1)
// i.e. a stable rank among the tokens of the group that picked the same expert.  One CTA
// handles one group: every warp owns a contiguous chunk of tokens, ranks its tokens inside the
// chunk with warp match/popcount against a per-warp histogram in shared memory, then an
// exclusive scan over the warps' histograms (per expert, in warp order) gives each chunk's
// offset.  Compact index lists are written; the dense [G,S,E,C] masks never exist.
#include "kernels.cuh"
#include "plan.cuh"

namespace gshard {

constexpr int kCapThreads = 512;

struct CapacityArgs {
  int S, E, C, G, warps_used, variant_a;
  const int32_t* expert_idx;   // [G,S,2]
  const float* gate12;         // [G,S,2]
  const float* u;              // [G,S]
  const float* m;              // [G,E]
  int32_t* slot;               // [G,S,2]  (also scratch for in-chunk ranks)
  float* weight;               // [G,S,2]
  uint8_t* flags;              // [G,S]
  int32_t* first_count;        // [G,E]
  int32_t* total_count;        // [G,E]
  int32_t* slot_token;         // [E,G,C]
  float* l_aux_group;          // [G]
  int32_t* stats_group;        // [G,8]
};

// Deterministic block sum (fixed tree), result valid in thread 0.
template <typename T>
__device__ T block_sum(T v, T* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  T r = 0;
  if (threadIdx.x == 0)
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) r += scratch[i];
  return r;
}

// Ranks one choice (k = 0 first, 1 second) of every token of the chunk inside the chunk and
// leaves the chunk's per-expert counts in hist_w.  In-chunk ranks go to slot[.,k] as scratch.
__device__ __forceinline__ void rank_chunk(const CapacityArgs& a, int g, int k, int lo, int hi,
                                           unsigned short* hist_w, bool second_pass) {
  const int lane = threadIdx.x & 31;
  const unsigned lt = (1u << lane) - 1u;
  for (int base = lo; base < hi; base += 32) {
    const int s = base + lane;
    const bool valid = s < hi;
    const long long t = (long long)g * a.S + (valid ? s : lo);
    // expert ids index shared-memory histograms: ids outside [0,E) (possible only through the
    // stage entry point, which takes them from the caller) are clamped instead of trusted
    int key = valid ? min(max(a.expert_idx[2 * t + k], 0), a.E - 1) : -1 - lane;
    bool counts = valid;
    if (second_pass && a.variant_a && valid) counts = (a.flags[t] & 2u) != 0;
    if (!counts) key = -1 - lane;           // unique key: matches nobody
    const unsigned mask = __match_any_sync(0xffffffffu, key);
    const int rank = __popc(mask & lt);
    int before = 0;
    if (counts) before = hist_w[key];
    __syncwarp();
    if (counts && rank == 0) hist_w[key] = (unsigned short)(before + __popc(mask));
    __syncwarp();
    if (valid) a.slot[2 * t + k] = counts ? before + rank : 0;
  }
}

__global__ void __launch_bounds__(kCapThreads) capacity_kernel(CapacityArgs a) {
  extern __shared__ unsigned char smem_raw[];
  int32_t* cnt = reinterpret_cast<int32_t*>(smem_raw);                       // [E] running c_e
  unsigned short* hist = reinterpret_cast<unsigned short*>(cnt + a.E);       // [warps_used][E]
  __shared__ float red_f[kCapThreads / 32];
  __shared__ int red_i[kCapThreads / 32];

  const int g = blockIdx.x;
  const int tid = threadIdx.x, w = tid >> 5;
  const int W = a.warps_used;
  const int chunk = (a.S + W - 1) / W;
  const int lo = min(a.S, w * chunk), hi = (w < W) ? min(a.S, lo + chunk) : lo;

  // empty slots are -1; this group's part of slot_token is E rows of C entries
  for (int i = tid; i < a.E * a.C; i += blockDim.x) {
    const int e = i / a.C, c = i % a.C;
    a.slot_token[((long long)e * a.G + g) * a.C + c] = -1;
  }
  for (int i = tid; i < W * a.E; i += blockDim.x) hist[i] = 0;
  __syncthreads();

  // ---- first loop of Algorithm 1 ---------------------------------------------------------
  if (w < W) rank_chunk(a, g, 0, lo, hi, hist + (size_t)w * a.E, false);
  __syncthreads();
  float aux = 0.f;
  for (int e = tid; e < a.E; e += blockDim.x) {
    int run = 0;
    for (int ww = 0; ww < W; ++ww) {
      const int t = hist[(size_t)ww * a.E + e];
      hist[(size_t)ww * a.E + e] = (unsigned short)run;
      run += t;
    }
    cnt[e] = run;                                     // c_e after the first loop, unclipped
    a.first_count[(long long)g * a.E + e] = run;
    aux += ((float)run / (float)a.S) * a.m[(long long)g * a.E + e];
  }
  __syncthreads();
  const float aux_sum = block_sum<float>(aux, red_f);
  if (tid == 0) a.l_aux_group[g] = aux_sum / (float)a.E;

  int n_first_dropped = 0, n_rnd_skipped = 0, n_cap_dropped = 0, n_overflowed = 0, n_filled = 0;
  for (int s = lo + (tid & 31); s < hi; s += 32) {
    const long long t = (long long)g * a.S + s;
    const int e1 = min(max(a.expert_idx[2 * t], 0), a.E - 1);
    const float g1 = a.gate12[2 * t], g2 = a.gate12[2 * t + 1];
    const float den = g1 + g2;
    const float w1 = g1 / den, w2 = g2 / den;
    const int pos = (int)hist[(size_t)w * a.E + e1] + a.slot[2 * t];
    unsigned f = 0;
    if (pos < a.C) {
      f |= 1u;
      a.slot[2 * t] = pos;
      a.slot_token[((long long)e1 * a.G + g) * a.C + pos] = s;
      ++n_filled;
    } else {
      a.slot[2 * t] = -1;
      ++n_first_dropped;
    }
    if (2.0f * w2 > a.u[t]) f |= 2u;                   // random routing test, strict >
    a.weight[2 * t] = w1;
    a.weight[2 * t + 1] = w2;
    a.flags[t] = (uint8_t)f;
  }
  __syncthreads();

  // ---- second loop: counters continue from the first loop --------------------------------
  for (int i = tid; i < W * a.E; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  if (w < W) rank_chunk(a, g, 1, lo, hi, hist + (size_t)w * a.E, true);
  __syncthreads();
  for (int e = tid; e < a.E; e += blockDim.x) {
    int run = cnt[e];
    for (int ww = 0; ww < W; ++ww) {
      const int t = hist[(size_t)ww * a.E + e];
      hist[(size_t)ww * a.E + e] = (unsigned short)min(run, 65535);
      run += t;
    }
    a.total_count[(long long)g * a.E + e] = run;
  }
  __syncthreads();
  for (int s = lo + (tid & 31); s < hi; s += 32) {
    const long long t = (long long)g * a.S + s;
    const int e2 = min(max(a.expert_idx[2 * t + 1], 0), a.E - 1);
    unsigned f = a.flags[t];
    const bool pass = (f & 2u) != 0;
    const int pos = (int)hist[(size_t)w * a.E + e2] + a.slot[2 * t + 1];
    if (pass && pos < a.C) {
      f |= 4u;
      a.slot[2 * t + 1] = pos;
      a.slot_token[((long long)e2 * a.G + g) * a.C + pos] = s;
      ++n_filled;
    } else {
      a.slot[2 * t + 1] = -1;
      if (!pass) ++n_rnd_skipped; else ++n_cap_dropped;
    }
    if ((f & 5u) == 0) ++n_overflowed;
    a.flags[t] = (uint8_t)f;
  }
  const int vals[5] = {n_first_dropped, n_rnd_skipped, n_cap_dropped, n_overflowed, n_filled};
#pragma unroll
  for (int i = 0; i < 5; ++i) {
    const int r = block_sum<int>(vals[i], red_i);
    if (tid == 0) a.stats_group[g * 8 + i] = r;
  }
  if (tid < 3) a.stats_group[g * 8 + 5 + tid] = 0;
}

// Layer-level results: l_aux = mean over groups (fixed order), stats summed over groups.
// G_mean: the number of groups the mean is taken over (more than G when these G groups are one
// rank's share of a layer whose groups are spread over several GPUs; the shares are then added).
__global__ void capacity_finalize_kernel(const float* l_aux_group, const int32_t* stats_group, int G, int G_mean,
                                         float* l_aux, long long* stats) {
  if (threadIdx.x == 0 && l_aux) {
    float acc = 0.f;
    for (int g = 0; g < G; ++g) acc += l_aux_group[g];
    *l_aux = acc / (float)G_mean;
  }
  if (stats && threadIdx.x < 8) {
    long long acc = 0;
    for (int g = 0; g < G; ++g) acc += stats_group[g * 8 + threadIdx.x];
    stats[threadIdx.x] = acc;
  }
}

// Debug check (GSHARD_FLAG_DEBUG_CHECKS, gshard_moe_check_routing): what Algorithm 1 implies for the
// routing tensors.  Per token: two distinct experts in [0, E), positions in [-1, C), flag bits that
// agree with the positions, normalised weights that sum to one, and the slot a kept choice names
// holds this token.  Per slot: a token index in [-1, S), and the token it names lists this slot.
// A violation records GSHARD_ERR_INTERNAL in the status word; every access is bounds-checked first.
__global__ void __launch_bounds__(256) routing_check_kernel(const int32_t* __restrict__ expert_idx,
                                                            const int32_t* __restrict__ slot,
                                                            const float* __restrict__ weight,
                                                            const uint8_t* __restrict__ flags,
                                                            const int32_t* __restrict__ slot_token, long long N,
                                                            long long R, int G, int S, int E, int C, int* status) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  bool bad = false;
  if (i < N) {
    const int g = (int)(i / S), s = (int)(i % S);
    const int e[2] = {expert_idx[2 * i], expert_idx[2 * i + 1]};
    const int p[2] = {slot[2 * i], slot[2 * i + 1]};
    const float w1 = weight[2 * i], w2 = weight[2 * i + 1];
    const unsigned f = flags[i];
    bad |= e[0] < 0 || e[0] >= E || e[1] < 0 || e[1] >= E || e[0] == e[1];
    bad |= !(w1 >= 0.5f - 1e-6f) || !(w2 >= 0.f) || !(fabsf(w1 + w2 - 1.f) <= 1e-5f);
    bad |= ((f & 1u) != 0) != (p[0] >= 0) || ((f & 4u) != 0) != (p[1] >= 0) || ((f & 4u) && !(f & 2u)) || (f & ~7u);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      if (p[k] < -1 || p[k] >= C) { bad = true; continue; }
      if (p[k] >= 0 && e[k] >= 0 && e[k] < E) bad |= slot_token[((long long)e[k] * G + g) * C + p[k]] != s;
    }
  }
  if (i < R) {
    const int tok = slot_token[i];
    const int c = (int)(i % C), g = (int)((i / C) % G), e = (int)(i / ((long long)C * G));
    if (tok < -1 || tok >= S) {
      bad = true;
    } else if (tok >= 0) {
      const long long t = (long long)g * S + tok;
      const bool first = expert_idx[2 * t] == e && slot[2 * t] == c;
      const bool second = expert_idx[2 * t + 1] == e && slot[2 * t + 1] == c;
      bad |= !(first || second);
    }
  }
  if (bad) set_device_status(status, GSHARD_ERR_INTERNAL);
}

void launch_routing_check(const Dims& d, const int32_t* expert_idx, const int32_t* slot, const float* weight,
                          const uint8_t* flags, const int32_t* slot_token, int* status, cudaStream_t st) {
  const long long n = d.N > d.R ? d.N : d.R;
  routing_check_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(expert_idx, slot, weight, flags, slot_token, d.N, d.R,
                                                                    d.G, d.S, d.E, d.C, status);
  count_launch();
}

size_t capacity_smem_bytes(int E, int warps) { return (size_t)E * 4 + (size_t)warps * E * 2; }

int capacity_warps_for(int E) {
  int w = kCapThreads / 32;
  while (w > 1 && capacity_smem_bytes(E, w) > 200 * 1024) w >>= 1;
  return capacity_smem_bytes(E, w) <= 200 * 1024 ? w : 0;
}

int launch_capacity(const Dims& d, const int32_t* expert_idx, const float* gate12, const float* u,
                    const float* m, int32_t* slot, float* weight, uint8_t* flags, int32_t* first_count,
                    int32_t* total_count, int32_t* slot_token, float* l_aux_group, int32_t* stats_group,
                    float* l_aux, long long* stats, cudaStream_t st, int groups_in_mean) {
  NvtxRange range("gshard.capacity");
  CapacityArgs a;
  a.S = d.S; a.E = d.E; a.C = d.C; a.G = d.G;
  a.warps_used = capacity_warps_for(d.E);
  if (a.warps_used == 0) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  a.variant_a = d.variant_a ? 1 : 0;
  a.expert_idx = expert_idx; a.gate12 = gate12; a.u = u; a.m = m;
  a.slot = slot; a.weight = weight; a.flags = flags; a.first_count = first_count;
  a.total_count = total_count; a.slot_token = slot_token; a.l_aux_group = l_aux_group;
  a.stats_group = stats_group;
  const size_t smem = capacity_smem_bytes(d.E, a.warps_used);
  // set on every launch: the attribute is per device, and the call is cheap
  if (cudaFuncSetAttribute(capacity_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  capacity_kernel<<<d.G, kCapThreads, smem, st>>>(a);
  capacity_finalize_kernel<<<1, 32, 0, st>>>(l_aux_group, stats_group, d.G, groups_in_mean > 0 ? groups_in_mean : d.G,
                                             l_aux, stats);
  count_launch(2);
  return GSHARD_OK;
}

}  // namespace gshard

// ---------------------------------------------------------------------------------------------
// Capacity assignment for callers that cannot allocate device memory.
//
// The regular entry point takes its scratch (the per-group statistics block, and any routing
// output the caller left out) from a caller-supplied workspace.  Some callers have no way to
// provide one: an operator plugged into a host runtime that owns the allocator and forbids
// allocation inside its execute hook, or a serving loop whose memory pool is frozen after
// start-up.  For them the scratch below is part of the library image itself: every GPU that
// loads the library holds these 128 KB until the process exits.
namespace gshard {
constexpr int kStaticMaxGroups = 4096;                       // G limit of the static variant
static __device__ __align__(256) int32_t g_static_stats_group[kStaticMaxGroups * 8];

namespace {
// In host code the array's name above is only a host-side stand-in, not a device address; the
// address a kernel can use comes from cudaGetSymbolAddress with the target device current.  It is
// asked on every call: the lookup allocates nothing once the library's module is loaded on the
// device (the first call loads it), and a cached pointer would dangle after a device reset.
int static_scratch_for_current_device(int32_t** out) {
  int32_t* p = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_stats_group) != cudaSuccess || p == nullptr) {
    cudaGetLastError();
    return GSHARD_ERR_CUDA;
  }
  *out = p;
  return GSHARD_OK;
}
}  // namespace
}  // namespace gshard

extern "C" int gshard_moe_capacity_static(const gshard_moe_shape* shape, const int32_t* expert_idx,
                                          const float* gate12, const float* u, const float* m,
                                          const gshard_moe_routing* routing_out, float* l_aux,
                                          void* cuda_stream) {
  using namespace gshard;
  launch_counter().n = 0;
  const int rc = validate_shape(shape);
  if (rc != GSHARD_OK) return rc;
  if (shape->G > kStaticMaxGroups) return GSHARD_ERR_UNSUPPORTED_SHAPE;   // beyond the built-in scratch
  auto bad = [](const void* p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (bad(expert_idx) || bad(gate12) || bad(u) || bad(m) || routing_out == nullptr) return GSHARD_ERR_INVALID_ARG;
  const gshard_moe_routing& r = *routing_out;
  // no workspace to fall back on: every tensor the kernel writes must be the caller's
  if (!r.slot || !r.weight || !r.flags || !r.first_count || !r.total_count || !r.slot_token || !r.l_aux_group)
    return GSHARD_ERR_INVALID_ARG;
  int major = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GSHARD_ERR_CUDA;
  if (major != 10) return GSHARD_ERR_ARCH;
  int32_t* stats_group = nullptr;
  const int src = static_scratch_for_current_device(&stats_group);
  if (src != GSHARD_OK) return src;
  // The kernel overwrites all 8 statistics of each of its G groups before the finalize kernel
  // reads them, so nothing in the shared array has to be cleared between calls.
  return launch_capacity(make_dims(*shape), expert_idx, gate12, u, m, r.slot, r.weight, r.flags, r.first_count,
                         r.total_count, r.slot_token, r.l_aux_group, stats_group, l_aux,
                         reinterpret_cast<long long*>(r.stats), static_cast<cudaStream_t>(cuda_stream));
}
