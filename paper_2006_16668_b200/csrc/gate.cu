// Gating kernels on stored fp32 logits: row softmax statistics, the top-2 pick and the
// per-tile column sums of the gates (Algorithm 1: "g <- softmax(wg . x)", "top_2",
// "m_E <- (1/S) sum_s g_{s,E}").
#include "kernels.cuh"

namespace gshard {

struct Top2 {
  float v1, v2;
  int i1, i2;
};

// "a before b": larger value first, lower index on equal values.
__device__ __forceinline__ bool before(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}

__device__ __forceinline__ void top2_insert(Top2& t, float v, int i) {
  if (before(v, i, t.v1, t.i1)) { t.v2 = t.v1; t.i2 = t.i1; t.v1 = v; t.i1 = i; }
  else if (before(v, i, t.v2, t.i2)) { t.v2 = v; t.i2 = i; }
}

__device__ __forceinline__ Top2 top2_merge(const Top2& a, const Top2& b) {
  Top2 r;
  if (before(b.v1, b.i1, a.v1, a.i1)) {
    r.v1 = b.v1; r.i1 = b.i1;
    if (before(a.v1, a.i1, b.v2, b.i2)) { r.v2 = a.v1; r.i2 = a.i1; } else { r.v2 = b.v2; r.i2 = b.i2; }
  } else {
    r.v1 = a.v1; r.i1 = a.i1;
    if (before(b.v1, b.i1, a.v2, a.i2)) { r.v2 = b.v1; r.i2 = b.i1; } else { r.v2 = a.v2; r.i2 = a.i2; }
  }
  return r;
}

// One warp per token: row max, 1/sum(exp), the two largest logits and their indices.
// Softmax is monotone, so top-2 of the gates is top-2 of the logits.
__global__ void __launch_bounds__(256) gate_rows_kernel(const float* __restrict__ logits, long long N,
                                                        int E, int32_t* __restrict__ expert_idx,
                                                        float* __restrict__ gate12,
                                                        float* __restrict__ rowmax,
                                                        float* __restrict__ rowinv) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const float ninf = __int_as_float(0xff800000);
  for (long long t = warp; t < N; t += nwarps) {
    const float* row = logits + t * E;
    Top2 tp{ninf, ninf, 0x7fffffff, 0x7fffffff};
    for (int e = lane; e < E; e += 32) top2_insert(tp, row[e], e);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      Top2 o;
      o.v1 = __shfl_xor_sync(0xffffffffu, tp.v1, off);
      o.v2 = __shfl_xor_sync(0xffffffffu, tp.v2, off);
      o.i1 = __shfl_xor_sync(0xffffffffu, tp.i1, off);
      o.i2 = __shfl_xor_sync(0xffffffffu, tp.i2, off);
      tp = top2_merge(tp, o);
    }
    float sum = 0.f;
    for (int e = lane; e < E; e += 32) sum += expf(row[e] - tp.v1);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane == 0) {
      const float inv = 1.0f / sum;
      expert_idx[2 * t] = tp.i1;
      expert_idx[2 * t + 1] = tp.i2;
      gate12[2 * t] = inv;                        // exp(l1 - max) = 1
      gate12[2 * t + 1] = expf(tp.v2 - tp.v1) * inv;
      rowmax[t] = tp.v1;
      rowinv[t] = inv;
    }
  }
}

// Column sums of the gates over one tile of kGateTile tokens of one group; thread = expert.
// partial[(g*tiles_per_group + tile), e] = sum over the tile's tokens of softmax value.
__global__ void __launch_bounds__(128) gate_colsum_kernel(const float* __restrict__ logits,
                                                          const float* __restrict__ rowmax,
                                                          const float* __restrict__ rowinv, int S,
                                                          int E, int tiles_per_group,
                                                          float* __restrict__ partial) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  const int tile = blockIdx.y;
  const int g = tile / tiles_per_group;
  const int s0 = (tile % tiles_per_group) * kGateTile;
  const int s1 = min(S, s0 + kGateTile);
  __shared__ float smax[kGateTile], sinv[kGateTile];
  for (int i = threadIdx.x; i < s1 - s0; i += blockDim.x) {
    smax[i] = rowmax[(long long)g * S + s0 + i];
    sinv[i] = rowinv[(long long)g * S + s0 + i];
  }
  __syncthreads();
  if (e >= E) return;
  float acc = 0.f;
  const float* base = logits + ((long long)g * S + s0) * E + e;
  for (int i = 0; i < s1 - s0; ++i) acc += expf(base[(long long)i * E] - smax[i]) * sinv[i];
  partial[(long long)tile * E + e] = acc;
}

// m[g,e] = (1/S) * sum of the group's tile partials, added in tile order (reproducible).
__global__ void __launch_bounds__(128) gate_mean_kernel(const float* __restrict__ partial, int S, int E,
                                                        int tiles_per_group, float* __restrict__ m) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (e >= E) return;
  float acc = 0.f;
  for (int t = 0; t < tiles_per_group; ++t) acc += partial[((long long)g * tiles_per_group + t) * E + e];
  m[(long long)g * E + e] = acc / (float)S;
}

// Same column sums with four experts per thread (16-byte loads, four rows in flight): the
// bandwidth-bound form used whenever E is a multiple of 4.  Rows are added in ascending order.
__global__ void __launch_bounds__(128) gate_colsum4_kernel(const float4* __restrict__ logits,
                                                           const float* __restrict__ rowmax,
                                                           const float* __restrict__ rowinv, int S,
                                                           int E4, int tiles_per_group,
                                                           float4* __restrict__ partial) {
  const int e4 = blockIdx.x * blockDim.x + threadIdx.x;
  const int tile = blockIdx.y;
  const int g = tile / tiles_per_group;
  const int s0 = (tile % tiles_per_group) * kGateTile;
  const int n = min(S, s0 + kGateTile) - s0;
  __shared__ float smax[kGateTile], sinv[kGateTile];
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    smax[i] = rowmax[(long long)g * S + s0 + i];
    sinv[i] = rowinv[(long long)g * S + s0 + i];
  }
  __syncthreads();
  if (e4 >= E4) return;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  const float4* base = logits + ((long long)g * S + s0) * E4 + e4;
  int i = 0;
  for (; i + 4 <= n; i += 4) {
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = __ldcs(base + (long long)(i + j) * E4);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float mx = smax[i + j], iv = sinv[i + j];
      acc.x += expf(v[j].x - mx) * iv; acc.y += expf(v[j].y - mx) * iv;
      acc.z += expf(v[j].z - mx) * iv; acc.w += expf(v[j].w - mx) * iv;
    }
  }
  for (; i < n; ++i) {
    const float4 v = __ldcs(base + (long long)i * E4);
    const float mx = smax[i], iv = sinv[i];
    acc.x += expf(v.x - mx) * iv; acc.y += expf(v.y - mx) * iv;
    acc.z += expf(v.z - mx) * iv; acc.w += expf(v.w - mx) * iv;
  }
  partial[(long long)tile * E4 + e4] = acc;
}


// Column sums from logits stored in 16-byte granules of four experts, float4 [E/4][N] (the layout the
// CTA-pair gating kernel writes): a warp takes one granule column and a 128-token tile, its lanes
// read 32 consecutive tokens (512 contiguous bytes) per load, four granule columns in flight, and
// the 32 partial sums meet in a shuffle tree (fixed order).
__global__ void __launch_bounds__(128) gate_colsum_t_kernel(const float4* __restrict__ logits_t,
                                                            const float* __restrict__ rowmax,
                                                            const float* __restrict__ rowinv, long long N,
                                                            int S, int E4, int tiles_per_group,
                                                            float4* __restrict__ partial) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tile = blockIdx.y;
  const int g = tile / tiles_per_group;
  const int s0 = (tile % tiles_per_group) * kGateTile;
  const int n = min(S, s0 + kGateTile) - s0;
  const long long row0 = (long long)g * S + s0;
  constexpr float kLog2e = 1.4426950408889634f;
  float mxl[4], iv[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = r * 32 + lane;
    mxl[r] = i < n ? rowmax[row0 + i] * kLog2e : 0.f;
    iv[r] = i < n ? rowinv[row0 + i] : 0.f;          // rows past the group's end contribute nothing
  }
  // this block's granule columns: 64 per block, 16 per warp, four at a time
  const int c_first = blockIdx.x * 64 + warp * 16;
  for (int cb = 0; cb < 16; cb += 4) {
    float4 acc[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 v[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c4 = c_first + cb + j;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = r * 32 + lane;
        v[j][r] = (c4 < E4 && i < n) ? __ldcs(logits_t + (long long)c4 * N + row0 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        acc[j].x += exp2f(fmaf(v[j][r].x, kLog2e, -mxl[r])) * iv[r];
        acc[j].y += exp2f(fmaf(v[j][r].y, kLog2e, -mxl[r])) * iv[r];
        acc[j].z += exp2f(fmaf(v[j][r].z, kLog2e, -mxl[r])) * iv[r];
        acc[j].w += exp2f(fmaf(v[j][r].w, kLog2e, -mxl[r])) * iv[r];
      }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) {
        acc[j].x += __shfl_xor_sync(0xffffffffu, acc[j].x, off);
        acc[j].y += __shfl_xor_sync(0xffffffffu, acc[j].y, off);
        acc[j].z += __shfl_xor_sync(0xffffffffu, acc[j].z, off);
        acc[j].w += __shfl_xor_sync(0xffffffffu, acc[j].w, off);
      }
      const int c4 = c_first + cb + j;
      if (lane == 0 && c4 < E4) partial[(long long)tile * E4 + c4] = acc[j];
    }
  }
}

void launch_gate_rows(const Dims& d, const float* logits, int32_t* expert_idx, float* gate12,
                      float* rowmax, float* rowinv, cudaStream_t st) {
  const long long warps_needed = d.N;
  int blocks = (int)((warps_needed + 7) / 8);
  const long long cap = (long long)device_sms() * 16;
  if (blocks > cap) blocks = (int)cap;
  gate_rows_kernel<<<blocks, 256, 0, st>>>(logits, d.N, d.E, expert_idx, gate12, rowmax, rowinv);
  count_launch();
}

// m[g,e] from stored logits and row statistics (two launches).
void launch_gate_means(const Dims& d, const float* logits, const float* rowmax, const float* rowinv,
                       float* partial, float* m, cudaStream_t st) {
  if (d.E % 4 == 0) {
    dim3 grid(ceil_div(d.E / 4, 128), d.G * d.tiles_per_group);
    gate_colsum4_kernel<<<grid, 128, 0, st>>>(reinterpret_cast<const float4*>(logits), rowmax, rowinv, d.S, d.E / 4,
                                              d.tiles_per_group, reinterpret_cast<float4*>(partial));
  } else {
    dim3 grid(ceil_div(d.E, 128), d.G * d.tiles_per_group);
    gate_colsum_kernel<<<grid, 128, 0, st>>>(logits, rowmax, rowinv, d.S, d.E, d.tiles_per_group, partial);
  }
  gate_mean_kernel<<<dim3(ceil_div(d.E, 128), d.G), 128, 0, st>>>(partial, d.S, d.E, d.tiles_per_group, m);
  count_launch(2);
}

// m[g,e] from logits stored as float4 [E/4][N] and row statistics (two launches).
void launch_gate_means_t(const Dims& d, const float* logits_t, const float* rowmax, const float* rowinv,
                         float* partial, float* m, cudaStream_t st) {
  const int E4 = d.E / 4;
  dim3 grid(ceil_div(E4, 64), d.G * d.tiles_per_group);
  gate_colsum_t_kernel<<<grid, 128, 0, st>>>(reinterpret_cast<const float4*>(logits_t), rowmax, rowinv, d.N, d.S, E4,
                                             d.tiles_per_group, reinterpret_cast<float4*>(partial));
  gate_mean_kernel<<<dim3(ceil_div(d.E, 128), d.G), 128, 0, st>>>(partial, d.S, d.E, d.tiles_per_group, m);
  count_launch(2);
}

void launch_gate_mean_blocks(const Dims& d, const float* partial, int blocks_per_group, float* m, cudaStream_t st) {
  gate_mean_kernel<<<dim3(ceil_div(d.E, 128), d.G), 128, 0, st>>>(partial, d.S, d.E, blocks_per_group, m);
  count_launch();
}

}  // namespace gshard
