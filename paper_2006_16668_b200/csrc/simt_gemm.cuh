// Batched GEMM on CUDA cores (fp32 FMA), generic strides.  It is the contraction of the
// GSHARD_F32 path (the paper trained in float32) and the debugging stand-in for the tcgen05
// path of the bf16 dtype (GSHARD_FLAG_SIMT_CONTRACTIONS).
#pragma once
#include "common.cuh"

namespace gshard {

struct SimtGemm {
  const void* A; const void* B; void* C;
  const void* mask;          // optional, laid out like C: output is zeroed where mask <= 0
  int rows, cols, K, batch;  // C[b] is rows x cols, contraction length K
  long long a_rs, a_cs, a_bs;  // A(b,i,k) = A[b*a_bs + i*a_rs + k*a_cs]
  long long b_rs, b_cs, b_bs;  // B(b,k,j) = B[b*b_bs + k*b_rs + j*b_cs]
  long long c_rs, c_bs;        // C(b,i,j) = C[b*c_bs + i*c_rs + j]
  int relu;                    // C = max(acc, 0)
  int accumulate;              // C += acc (read-modify-write)
};

template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256) simt_gemm_kernel(SimtGemm p) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int b = blockIdx.z;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  const TA* A = reinterpret_cast<const TA*>(p.A) + (long long)b * p.a_bs;
  const TB* B = reinterpret_cast<const TB*>(p.B) + (long long)b * p.b_bs;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  float acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;

  for (int k0 = 0; k0 < p.K; k0 += BK) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int idx = tid + r * 256;
      int i, k;
      if (p.a_cs == 1) { k = idx % BK; i = idx / BK; } else { i = idx % BM; k = idx / BM; }
      float v = 0.f;
      if (i0 + i < p.rows && k0 + k < p.K)
        v = to_f32<TA>(A[(long long)(i0 + i) * p.a_rs + (long long)(k0 + k) * p.a_cs]);
      As[k][i] = v;
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int idx = tid + r * 256;
      int j, k;
      if (p.b_cs == 1) { j = idx % BN; k = idx / BN; } else { k = idx % BK; j = idx / BK; }
      float v = 0.f;
      if (j0 + j < p.cols && k0 + k < p.K)
        v = to_f32<TB>(B[(long long)(k0 + k) * p.b_rs + (long long)(j0 + j) * p.b_cs]);
      Bs[k][j] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], bb[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) a[r] = As[k][ty * 4 + r];
#pragma unroll
      for (int c = 0; c < 4; ++c) bb[c] = Bs[k][tx * 4 + c];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], bb[c], acc[r][c]);
    }
    __syncthreads();
  }
  TC* C = reinterpret_cast<TC*>(p.C) + (long long)b * p.c_bs;
  const TC* Mk = p.mask ? reinterpret_cast<const TC*>(p.mask) + (long long)b * p.c_bs : nullptr;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = i0 + ty * 4 + r;
    if (i >= p.rows) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int j = j0 + tx * 4 + c;
      if (j >= p.cols) continue;
      float v = acc[r][c];
      if (p.relu) v = fmaxf(v, 0.f);
      const long long off = (long long)i * p.c_rs + j;
      if (Mk && !(to_f32<TC>(Mk[off]) > 0.f)) v = 0.f;
      if (p.accumulate) v += to_f32<TC>(C[off]);
      C[off] = from_f32<TC>(v);
    }
  }
}

template <typename TA, typename TB, typename TC>
inline void launch_simt_gemm(const SimtGemm& p, cudaStream_t st) {
  if (p.rows <= 0 || p.cols <= 0 || p.batch <= 0) return;
  dim3 grid(ceil_div(p.cols, 64), ceil_div(p.rows, 64), p.batch);
  simt_gemm_kernel<TA, TB, TC><<<grid, 256, 0, st>>>(p);
  count_launch();
}

}  // namespace gshard
