// Dispatch and combine as index-driven row copies (Algorithm 2's two one-hot einsums,
// "GSEC,GSM->EGCM" and "GSEC,GECM->GSM", restated as gathers; the paper itself shows the
// gather form with s_indices[E,G,C] in its section on mixing manual and automatic sharding).
// Both are HBM-bound: one warp moves one row with 16-byte accesses.
#include "kernels.cuh"
#include "sm100_ptx.cuh"

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

// The same copy through the TMA unit (GSHARD_FLAG_BULK_DISPATCH).  Every warp owns a ring of kStages row
// buffers in shared memory; its lane 0 keeps kStages - 2 bulk loads (global -> shared, completion
// counted on an mbarrier per stage) and two bulk stores (shared -> global) in flight; an empty slot is
// a bulk store from a row of zeros.  No thread touches the data; the warp's other lanes only fetch the
// slot indices 32 rows ahead.  Row i of a warp's run uses stage i mod kStages; at
// step i the row i - (kStages - 2) is completed (wait for its bytes, issue its store), then at most two
// stores may still be reading shared memory - the one that last used stage i mod kStages was issued two
// steps earlier - and the load of row i is issued.
template <int kBulkWarps, int kBulkStages>
__global__ void __launch_bounds__(kBulkWarps * 32) dispatch_bulk_kernel(const unsigned char* __restrict__ x,
                                                                        const int32_t* __restrict__ slot_token,
                                                                        unsigned char* __restrict__ buf, long long R,
                                                                        int G, int S, int C, uint32_t row_bytes,
                                                                        int* status) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t bars[kBulkWarps][kBulkStages];
  __shared__ int no_abort;
  unsigned char* zero_row = smem;
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned char* ring = smem + (size_t)row_bytes * (1 + w * kBulkStages);
  for (uint32_t i = threadIdx.x * 16; i < row_bytes; i += blockDim.x * 16)
    *reinterpret_cast<uint4*>(zero_row + i) = make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) no_abort = 0;
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kBulkStages; ++s) ptx::mbar_init(&bars[w][s], 1);
    ptx::fence_mbar_init();
  }
  ptx::fence_proxy_async();                     // the zero row, written by threads, is read by bulk stores
  __syncthreads();

  volatile int* abort_flag = status ? status : &no_abort;
  // a warp owns a contiguous run of rows: coalesced index loads, one long run of destination bytes
  const long long nwarps = (long long)gridDim.x * kBulkWarps;
  const long long per_warp = (R + nwarps - 1) / nwarps;
  const long long row0 = ((long long)blockIdx.x * kBulkWarps + w) * per_warp;
  const long long n_rows = row0 < R ? (R - row0 < per_warp ? R - row0 : per_warp) : 0;
  constexpr int kLag = kBulkStages - 2;
  uint32_t parity = 0;                          // bit s: parity of the next completion on stage s
  uint32_t loaded = 0;                          // bit s: the row in stage s has a load in flight (not an empty slot)
  bool ok = true;
  // the whole warp fetches the indices of the next 32 rows; lane 0 alone drives the copies
  for (long long base = 0; base < n_rows + kLag; base += 32) {
    const long long mine = base + lane;
    const int tok_lane = mine < n_rows ? slot_token[row0 + mine] : -1;
#pragma unroll 1
    for (int k = 0; k < 32; ++k) {
      const long long i = base + k;
      if (i >= n_rows + kLag) break;            // uniform over the warp
      const int tok = __shfl_sync(0xffffffffu, tok_lane, k);
      if (lane != 0 || !ok) continue;
      const long long j = i - kLag;             // the row to complete
      if (j >= 0) {
        const int s = (int)(j % kBulkStages);
        unsigned char* dst = buf + (row0 + j) * (long long)row_bytes;
        if ((loaded >> s) & 1u) {
          ok = ptx::mbar_wait(&bars[w][s], (parity >> s) & 1u, abort_flag);
          parity ^= 1u << s;
          if (ok) ptx::bulk_store(dst, ring + (size_t)s * row_bytes, row_bytes);
        } else {
          ptx::bulk_store(dst, zero_row, row_bytes);
        }
        ptx::tma_store_commit();
      }
      if (i < n_rows && ok) {
        ptx::bulk_wait_read<2>();
        const int s = (int)(i % kBulkStages);
        if (tok >= 0 && tok < S) {
          const long long r = row0 + i;         // r = (e*G + g)*C + c
          const int g = (int)((r / C) % G);
          ptx::mbar_arrive_expect_tx(&bars[w][s], row_bytes);
          ptx::bulk_load(ring + (size_t)s * row_bytes, x + ((long long)g * S + tok) * (long long)row_bytes, row_bytes,
                         &bars[w][s]);
          loaded |= 1u << s;
        } else {
          loaded &= ~(1u << s);
        }
      }
    }
  }
  if (lane == 0) {
    if (!ok && status) set_device_status(status, GSHARD_ERR_TIMEOUT);
    ptx::tma_store_wait_all();                  // shared memory must outlive the stores that read it
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

void launch_dispatch(const Dims& d, const void* x, const int32_t* slot_token, void* buf, cudaStream_t st, int* status) {
  NvtxRange range("gshard.dispatch");
  const int row_vec = (int)((size_t)d.M * d.esize / 16);
  const size_t row_bytes = (size_t)d.M * d.esize;
  constexpr int kWarps = 16, kStages = 4;       // of the ring shapes tried (4-32 warps, 3-8 stages) the fastest
  const size_t bulk_smem = row_bytes * (1 + (size_t)kWarps * kStages);
  if (d.bulk_dispatch && bulk_smem <= 200 * 1024) {
    static thread_local int attr_device = -1;   // the attribute is per function and device
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_device != dev) {
      cudaFuncSetAttribute(dispatch_bulk_kernel<kWarps, kStages>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      attr_device = dev;
    }
    long long blocks = (d.R + kWarps - 1) / kWarps;
    const long long cap = device_sms();         // one CTA per multiprocessor: the rings fill its shared memory
    if (blocks > cap) blocks = cap;
    dispatch_bulk_kernel<kWarps, kStages><<<(int)blocks, kWarps * 32, bulk_smem, st>>>(
        static_cast<const unsigned char*>(x), slot_token, static_cast<unsigned char*>(buf), d.R, d.G, d.S, d.C,
        (uint32_t)row_bytes, status);
    count_launch();
    return;
  }
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
