// Dispatch and combine as index-driven row copies (Algorithm 2's two one-hot einsums,
// "GSEC,GSM->EGCM" and "GSEC,GECM->GSM", restated as gathers; the paper itself shows the
// gather form with s_indices[E,G,C] in its section on mixing manual and automatic sharding).
// Both are HBM-bound: one warp moves one row with 16-byte accesses.
#include "kernels.cuh"

namespace gshard {

// buf[e, g*C + c, :] = x[g, slot_token[e,g,c], :]  or zeros for an empty slot.  The index list may
// come straight from a caller (stage entry point): a token index outside [0, S) is treated as an
// empty slot instead of being used as an address.
__global__ void __launch_bounds__(256) dispatch_kernel(const uint4* __restrict__ x,
                                                       const int32_t* __restrict__ slot_token,
                                                       uint4* __restrict__ buf, long long R, int G,
                                                       int S, int C, int row_vec) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = warp; r < R; r += nwarps) {
    const int tok = slot_token[r];                       // r = (e*G + g)*C + c
    const int g = (int)((r / C) % G);
    uint4* dst = buf + r * row_vec;
    if (tok >= 0 && tok < S) {
      const uint4* src = x + ((long long)g * S + tok) * row_vec;
      for (int i = lane; i < row_vec; i += 32) dst[i] = __ldg(src + i);
    } else {
      const uint4 z = make_uint4(0, 0, 0, 0);
      for (int i = lane; i < row_vec; i += 32) dst[i] = z;
    }
  }
}

// y[t,:] = w0*out[e0, g*C+slot0, :] + w1*out[e1, g*C+slot1, :] over the kept choices, fp32 FMA;
// with `residual` the token's input row is added (the residual connection around the layer).  A
// choice whose expert id is outside [0, E) or whose slot is outside [0, C) contributes nothing (the
// stage entry point takes these tensors from the caller; they are checked, not trusted).
template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(const uint4* __restrict__ out,
                                                      const int32_t* __restrict__ expert_idx,
                                                      const int32_t* __restrict__ slot,
                                                      const float* __restrict__ weight,
                                                      const uint4* __restrict__ residual,
                                                      uint4* __restrict__ y, long long N, int G, int S,
                                                      int C, int E, int row_vec,
                                                      const int32_t* __restrict__ slot_crow) {
  constexpr int n = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long t = warp; t < N; t += nwarps) {
    const int g = (int)(t / S);
    const int s0 = slot[2 * t], s1 = slot[2 * t + 1];
    const float w0 = weight[2 * t], w1 = weight[2 * t + 1];
    const int x0 = expert_idx[2 * t], x1 = expert_idx[2 * t + 1];
    const bool k0 = s0 >= 0 && s0 < C && x0 >= 0 && x0 < E, k1 = s1 >= 0 && s1 < C && x1 >= 0 && x1 < E;
    long long row0 = k0 ? ((long long)x0 * G + g) * C + s0 : 0, row1 = k1 ? ((long long)x1 * G + g) * C + s1 : 0;
    if (slot_crow) {                      // outputs stored by compacted row within the expert's block
      if (k0) row0 = (long long)x0 * G * C + slot_crow[row0];
      if (k1) row1 = (long long)x1 * G * C + slot_crow[row1];
    }
    const uint4* r0 = k0 ? out + row0 * row_vec : nullptr;
    const uint4* r1 = k1 ? out + row1 * row_vec : nullptr;
    uint4* dst = y + t * row_vec;
    // four 16-byte pieces per lane and row at a time, every load issued before the first use (the
    // rows are scattered in HBM)
    for (int i0 = lane; i0 < row_vec; i0 += 128) {
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      uint4 v0[4], v1[4], vr[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + 32 * k;
        const bool in = i < row_vec;
        v0[k] = (r0 && in) ? __ldg(r0 + i) : z;
        v1[k] = (r1 && in) ? __ldg(r1 + i) : z;
        vr[k] = (residual && in) ? __ldg(residual + t * row_vec + i) : z;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + 32 * k;
        if (i >= row_vec) break;
        float acc[n], f0[n], f1[n];
        Vec16<T>::load(vr[k], acc);
        Vec16<T>::load(v0[k], f0);
        Vec16<T>::load(v1[k], f1);
#pragma unroll
        for (int j = 0; j < n; ++j) acc[j] = fmaf(w1, f1[j], fmaf(w0, f0[j], acc[j]));
        dst[i] = Vec16<T>::store(acc);
      }
    }
  }
}

// Batched fp32 matrix transpose through a padded 32 x 32 shared-memory tile (coalesced both ways).
__global__ void __launch_bounds__(256) transpose_f32_kernel(const float* __restrict__ src, float* __restrict__ dst,
                                                            int rows, int cols) {
  __shared__ float tile[32][33];
  const long long base = (long long)blockIdx.z * rows * cols;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8 threads
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty + 8 * i, c = c0 + tx;
    if (r < rows && c < cols) tile[ty + 8 * i][tx] = src[base + (long long)r * cols + c];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = c0 + ty + 8 * i, r = r0 + tx;
    if (r < rows && c < cols) dst[base + (long long)c * rows + r] = tile[tx][ty + 8 * i];
  }
}

void launch_transpose_f32(const float* src, float* dst, int batch, int rows, int cols, cudaStream_t st) {
  const dim3 grid(ceil_div(cols, 32), ceil_div(rows, 32), batch);
  transpose_f32_kernel<<<grid, 256, 0, st>>>(src, dst, rows, cols);
  count_launch();
}

// Dispatch into compacted rows: row j of expert e is the token crow_token[e, j] (j < kept[e]).
__global__ void __launch_bounds__(256) dispatch_compact_kernel(const uint4* __restrict__ x,
                                                               const int32_t* __restrict__ crow_token,
                                                               const int32_t* __restrict__ kept,
                                                               uint4* __restrict__ buf, long long R, int rows,
                                                               long long N, int row_vec) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = warp; r < R; r += nwarps) {
    const int e = (int)(r / rows), j = (int)(r % rows);
    if (j >= kept[e]) continue;
    const long long t = crow_token[r];
    if (t < 0 || t >= N) continue;
    const uint4* src = x + t * row_vec;
    uint4* dst = buf + r * row_vec;
    for (int i = lane; i < row_vec; i += 32) dst[i] = __ldg(src + i);
  }
}

void launch_dispatch_compact(const Dims& d, const void* x, const int32_t* crow_token, const int32_t* kept, void* buf,
                             cudaStream_t st) {
  NvtxRange range("gshard.dispatch");
  const int row_vec = (int)((size_t)d.M * d.esize / 16);
  dispatch_compact_kernel<<<grid_for_rows(d.R), 256, 0, st>>>(reinterpret_cast<const uint4*>(x), crow_token, kept,
                                                              reinterpret_cast<uint4*>(buf), d.R, d.rows, d.N, row_vec);
  count_launch();
}

void launch_dispatch(const Dims& d, const void* x, const int32_t* slot_token, void* buf, cudaStream_t st) {
  NvtxRange range("gshard.dispatch");
  const int row_vec = (int)((size_t)d.M * d.esize / 16);
  dispatch_kernel<<<grid_for_rows(d.R), 256, 0, st>>>(reinterpret_cast<const uint4*>(x), slot_token,
                                                      reinterpret_cast<uint4*>(buf), d.R, d.G, d.S, d.C, row_vec);
  count_launch();
}

void launch_combine(const Dims& d, const void* out, const int32_t* expert_idx, const int32_t* slot,
                    const float* weight, void* y, cudaStream_t st, const void* residual, const int32_t* slot_crow) {
  NvtxRange range("gshard.combine");
  const int row_vec = (int)((size_t)d.M * d.esize / 16);
  if (d.bf16)
    combine_kernel<__nv_bfloat16><<<grid_for_rows(d.N), 256, 0, st>>>(
        reinterpret_cast<const uint4*>(out), expert_idx, slot, weight, reinterpret_cast<const uint4*>(residual),
        reinterpret_cast<uint4*>(y), d.N, d.G, d.S, d.C, d.E, row_vec, slot_crow);
  else
    combine_kernel<float><<<grid_for_rows(d.N), 256, 0, st>>>(
        reinterpret_cast<const uint4*>(out), expert_idx, slot, weight, reinterpret_cast<const uint4*>(residual),
        reinterpret_cast<uint4*>(y), d.N, d.G, d.S, d.C, d.E, row_vec, slot_crow);
  count_launch();
}

}  // namespace gshard
