// Backward of L = <dy, y> + k * l_aux with the routing frozen.  The paper leaves the backward
// to automatic differentiation; these are the derivatives of eq. (1)-(3) and of Algorithm 1's
// combine weights and auxiliary loss, with the counts c_e constant (the paper states they are
// not differentiable).  Per token with raw gates a = g_{e1}, b = g_{e2}, D = a + b:
//   y = k1 (a/D) o1 + k2 (b/D) o2,  dw1 = k1 <dy,o1>,  dw2 = k2 <dy,o2>
//   dL/da = (b/D^2)(dw1 - dw2),  dL/db = (a/D^2)(dw2 - dw1)
//   dL/dg_{g,s,e} += k (1/G)(1/E)(c_{g,e}/S)(1/S)                      (dense, from l_aux)
//   dlogit = g * (dg - <g, dg>),  dwg = x^T dlogit,  dx += dlogit wg^T
//   expert path: dout[slot] = w dy,  dh = (dout wo^T) * 1[h > 0],  dwo = h^T dout,
//                dwi = buf^T dh,  dbuf = dh wi^T,  dx += dbuf[slot]
#include <mutex>

#include "gemm_dispatch.cuh"
#include "plan.cuh"

namespace gshard {

int gate_logits(const Dims& d, const void* x, const void* wg, float* logits, int* status, cudaStream_t st);

namespace {

// dw[t,k] = <dy[t,:], out[e_k, g*C+slot_k, :]> for kept choices, else 0.  One warp per token.
template <typename T>
__global__ void __launch_bounds__(256) combine_bwd_kernel(const uint4* __restrict__ dy, const uint4* __restrict__ out,
                                                          const int32_t* __restrict__ expert_idx,
                                                          const int32_t* __restrict__ slot, float* __restrict__ dw,
                                                          long long N, int G, int S, int C, int row_vec) {
  constexpr int n = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long t = warp; t < N; t += nwarps) {
    const int g = (int)(t / S);
    float acc[2] = {0.f, 0.f};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int sl = slot[2 * t + k];
      if (sl < 0) continue;
      const uint4* r = out + (((long long)expert_idx[2 * t + k] * G + g) * C + sl) * row_vec;
      const uint4* dyr = dy + t * row_vec;
      for (int i = lane; i < row_vec; i += 32) {
        float a[n], b[n];
        Vec16<T>::load(__ldg(r + i), a);
        Vec16<T>::load(__ldg(dyr + i), b);
#pragma unroll
        for (int j = 0; j < n; ++j) acc[k] = fmaf(a[j], b[j], acc[k]);
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
      acc[1] += __shfl_xor_sync(0xffffffffu, acc[1], off);
    }
    if (lane == 0) { dw[2 * t] = acc[0]; dw[2 * t + 1] = acc[1]; }
  }
}

// dout[e, g*C+c, :] = weight_k * dy[g, tok, :] for the token in the slot, zeros for an empty slot.
template <typename T>
__global__ void __launch_bounds__(256) dout_kernel(const uint4* __restrict__ dy, const int32_t* __restrict__ slot_token,
                                                   const int32_t* __restrict__ expert_idx,
                                                   const int32_t* __restrict__ slot, const float* __restrict__ weight,
                                                   uint4* __restrict__ dout, long long R, int G, int S, int C,
                                                   int row_vec) {
  constexpr int n = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = warp; r < R; r += nwarps) {
    const int tok = slot_token[r];
    const int c = (int)(r % C);
    const int g = (int)((r / C) % G);
    const int e = (int)(r / ((long long)C * G));
    uint4* dst = dout + r * row_vec;
    if (tok < 0) {
      for (int i = lane; i < row_vec; i += 32) dst[i] = make_uint4(0, 0, 0, 0);
      continue;
    }
    const long long t = (long long)g * S + tok;
    const int k = (expert_idx[2 * t] == e && slot[2 * t] == c) ? 0 : 1;
    const float w = weight[2 * t + k];
    const uint4* src = dy + t * row_vec;
    for (int i = lane; i < row_vec; i += 32) {
      float f[n];
      Vec16<T>::load(__ldg(src + i), f);
#pragma unroll
      for (int j = 0; j < n; ++j) f[j] *= w;
      dst[i] = Vec16<T>::store(f);
    }
  }
}

// Softmax backward per token (one warp): dlogit_e = p_e (dg_e - sum_e' p_e' dg_e').
template <typename T>
__global__ void __launch_bounds__(256) gate_bwd_kernel(const float* __restrict__ logits, const float* __restrict__ rowmax,
                                                       const float* __restrict__ rowinv,
                                                       const int32_t* __restrict__ expert_idx,
                                                       const float* __restrict__ gate12, const float* __restrict__ dw,
                                                       const int32_t* __restrict__ first_count, float aux_coef,
                                                       T* __restrict__ dlogits, long long N, int S, int E) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long t = warp; t < N; t += nwarps) {
    const int g = (int)(t / S);
    const float mx = rowmax[t], inv = rowinv[t];
    const int e1 = expert_idx[2 * t], e2 = expert_idx[2 * t + 1];
    const float a = gate12[2 * t], b = gate12[2 * t + 1], D = a + b;
    const float d1 = dw[2 * t], d2 = dw[2 * t + 1];
    const float dga = (b / (D * D)) * (d1 - d2), dgb = (a / (D * D)) * (d2 - d1);
    const float* row = logits + t * E;
    const int32_t* fc = first_count + (long long)g * E;
    float dot = 0.f;
    for (int e = lane; e < E; e += 32) {
      const float p = expf(row[e] - mx) * inv;
      float dg = aux_coef * (float)fc[e];
      if (e == e1) dg += dga;
      if (e == e2) dg += dgb;
      dot = fmaf(p, dg, dot);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    for (int e = lane; e < E; e += 32) {
      const float p = expf(row[e] - mx) * inv;
      float dg = aux_coef * (float)fc[e];
      if (e == e1) dg += dga;
      if (e == e2) dg += dgb;
      dlogits[t * E + e] = from_f32<T>(p * (dg - dot));
    }
  }
}

// dx[t,:] = dxg[t,:] (fp32, from the gating GEMM) + dbuf rows of the kept choices.
template <typename T>
__global__ void __launch_bounds__(256) dx_kernel(const float4* __restrict__ dxg, const uint4* __restrict__ dbuf,
                                                 const int32_t* __restrict__ expert_idx, const int32_t* __restrict__ slot,
                                                 const uint4* __restrict__ dy_res, uint4* __restrict__ dx, long long N,
                                                 int G, int S, int C, int row_vec) {
  constexpr int n = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long t = warp; t < N; t += nwarps) {
    const int g = (int)(t / S);
    const uint4* r[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int sl = slot[2 * t + k];
      r[k] = sl >= 0 ? dbuf + (((long long)expert_idx[2 * t + k] * G + g) * C + sl) * row_vec : nullptr;
    }
    for (int i = lane; i < row_vec; i += 32) {
      float acc[n];
      const float4* gsrc = dxg + (t * row_vec + i) * (n / 4);
#pragma unroll
      for (int j = 0; j < n / 4; ++j) {
        const float4 v = gsrc[j];
        acc[4 * j] = v.x; acc[4 * j + 1] = v.y; acc[4 * j + 2] = v.z; acc[4 * j + 3] = v.w;
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        if (!r[k]) continue;
        float f[n];
        Vec16<T>::load(__ldg(r[k] + i), f);
#pragma unroll
        for (int j = 0; j < n; ++j) acc[j] += f[j];
      }
      if (dy_res) {                                  // residual connection: dx also receives dy
        float f[n];
        Vec16<T>::load(__ldg(dy_res + t * row_vec + i), f);
#pragma unroll
        for (int j = 0; j < n; ++j) acc[j] += f[j];
      }
      dx[t * row_vec + i] = Vec16<T>::store(acc);
    }
  }
}

// out[i] = part[0][i] + part[1][i] + ... (fixed order), float4 elements.
__global__ void __launch_bounds__(256) sum_partials_kernel(const float4* __restrict__ part, float4* __restrict__ out,
                                                           long long n4, int splits) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 acc = part[i];
  for (int s = 1; s < splits; ++s) {
    const float4 v = part[(long long)s * n4 + i];
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  out[i] = acc;
}

// A second stream and two events per device for the pairs of expert GEMMs that run side by side
// (host-side objects, created on first use and kept for the life of the process).
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
SideStream* side_stream_for_current_device() {
  constexpr int kMaxDevices = 64;
  static SideStream pool[kMaxDevices];
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return nullptr; }
  std::lock_guard<std::mutex> lock(mu);
  SideStream& s = pool[dev];
  if (!s.stream) {
    cudaStream_t st = nullptr; cudaEvent_t a = nullptr, b = nullptr;
    if (cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    s.stream = st; s.fork = a; s.join = b;
  }
  return &s;
}

// Runs GEMMs `a` (on `st`) and `b` (on the side stream) at the same time, each on its share of the
// multiprocessors; `b` is ordered after everything enqueued on `st` so far and `st` continues only
// after both.  share_a: multiprocessors given to `a` (even).
int run_gemm_pair(const Dims& d, UmmaGemm a, UmmaGemm b, int share_a, int* status, cudaStream_t st) {
  SideStream* side = side_stream_for_current_device();
  const int sms = device_sms();
  if (!side || d.simt || share_a <= 0 || share_a >= sms) {
    int rc = run_gemm(d, a, status, st);
    return rc ? rc : run_gemm(d, b, status, st);
  }
  a.max_ctas = share_a; b.max_ctas = sms - share_a;
  if (cudaEventRecord(side->fork, st) != cudaSuccess || cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  int rc = run_gemm(d, a, status, st);
  if (rc) return rc;
  rc = run_gemm(d, b, status, side->stream);
  if (rc) return rc;
  if (cudaEventRecord(side->join, side->stream) != cudaSuccess || cudaStreamWaitEvent(st, side->join, 0) != cudaSuccess)
    return GSHARD_ERR_CUDA;
  return GSHARD_OK;
}

// Combine backward over the groups of `d`: dw (per token and choice) and dout (per slot) into the
// backward workspace laid out by plan_backward(d).
template <typename T>
int combine_bwd_t(const Dims& d, const unsigned char* ctx, const void* dy, unsigned char* ws, cudaStream_t st) {
  NvtxRange range("gshard.backward.combine");
  const BwdPlan bp = plan_backward(d);
  const CtxPlan cp = plan_context(d);
  const int32_t* expert_idx = reinterpret_cast<const int32_t*>(ctx + cp.expert_idx);
  const int32_t* slot = reinterpret_cast<const int32_t*>(ctx + cp.slot);
  const int row_vec = (int)((size_t)d.M * d.esize / 16);
  combine_bwd_kernel<T><<<grid_for_rows(d.N), 256, 0, st>>>(
      reinterpret_cast<const uint4*>(dy), reinterpret_cast<const uint4*>(ctx + cp.out), expert_idx, slot,
      reinterpret_cast<float*>(ws + bp.dw), d.N, d.G, d.S, d.C, row_vec);
  dout_kernel<T><<<grid_for_rows(d.R), 256, 0, st>>>(
      reinterpret_cast<const uint4*>(dy), reinterpret_cast<const int32_t*>(ctx + cp.slot_token), expert_idx, slot,
      reinterpret_cast<const float*>(ctx + cp.weight), reinterpret_cast<uint4*>(ws + bp.dout), d.R, d.G, d.S, d.C, row_vec);
  count_launch(2);
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

// Gating backward and dx over the groups of `d`.  groups_in_mean: the group count l_aux averages
// over (the global one when `d` is one rank's share of the groups).  dbuf: [E, G*C, M] of `d`.
template <typename T>
int gate_bwd_t(const Dims& d, const void* x, const void* wg, const unsigned char* ctx, const void* dy, float k_aux,
               int groups_in_mean, const void* dbuf, void* dx, float* dwg, unsigned char* ws, cudaStream_t st) {
  NvtxRange gate_range("gshard.backward.gate");
  const BwdPlan bp = plan_backward(d);
  const CtxPlan cp = plan_context(d);
  int* status = reinterpret_cast<int*>(ws + bp.status);
  const int32_t* expert_idx = reinterpret_cast<const int32_t*>(ctx + cp.expert_idx);
  const int32_t* slot = reinterpret_cast<const int32_t*>(ctx + cp.slot);
  const int32_t* first_count = reinterpret_cast<const int32_t*>(ctx + cp.first_count);
  const float* gate12 = reinterpret_cast<const float*>(ctx + cp.gate12);
  const float* rowmax = reinterpret_cast<const float*>(ctx + cp.rowmax);
  const float* rowinv = reinterpret_cast<const float*>(ctx + cp.rowinv);
  float* logits = reinterpret_cast<float*>(ws + bp.logits);
  T* dlogits = reinterpret_cast<T*>(ws + bp.dlogits);
  const float* dw = reinterpret_cast<const float*>(ws + bp.dw);
  float* dxg = reinterpret_cast<float*>(ws + bp.dxg);
  const int row_vec = (int)((size_t)d.M * d.esize / 16);
  // recompute the logits, softmax backward, two GEMMs
  int rc = gate_logits(d, x, wg, logits, status, st);
  if (rc) return rc;
  const float aux_coef = k_aux / ((float)groups_in_mean * (float)d.E * (float)d.S * (float)d.S);
  gate_bwd_kernel<T><<<grid_for_rows(d.N), 256, 0, st>>>(logits, rowmax, rowinv, expert_idx, gate12, dw, first_count,
                                                     aux_coef, dlogits, d.N, d.S, d.E);
  count_launch();
  // dwg = x^T . dlogits   [M x E] fp32
  UmmaGemm g{};
  g.A = x; g.B = dlogits; g.C = dwg; g.rows = d.M; g.cols = d.E; g.K = (int)d.N; g.batch = 1;
  g.a_kmajor = false; g.b_kmajor = false; g.a_ld = d.M; g.b_ld = d.E; g.c_ld = d.E; g.out_f32 = 1;
  // Few output tiles, very long contraction: split the token dimension over the batch index so that
  // every SM gets a share, then add the partial sums in a fixed order.  The partials live in the dxg
  // region, which is not written before the next GEMM.
  int splits = 1;
  if (!d.simt) {
    const long long tiles = (long long)ceil_div(d.M, 128) * ceil_div(d.E, d.E > 128 ? 256 : 128);
    for (int sp = (int)(device_sms() / tiles); sp > 1; --sp)
      if (d.N % ((long long)sp * 64) == 0 && (long long)sp * d.E <= d.N && ((long long)d.M * d.E) % 4 == 0) {
        splits = sp;
        break;
      }
  }
  if (splits > 1) {
    const long long kn = d.N / splits;
    g.C = dxg; g.K = (int)kn; g.batch = splits;
    g.a_bs = kn * d.M; g.b_bs = kn * d.E; g.c_bs = (long long)d.M * d.E;
  }
  rc = run_gemm(d, g, status, st);
  if (rc) return rc;
  if (splits > 1) {
    const long long n4 = (long long)d.M * d.E / 4;
    sum_partials_kernel<<<(int)((n4 + 255) / 256), 256, 0, st>>>(reinterpret_cast<const float4*>(dxg),
                                                                 reinterpret_cast<float4*>(dwg), n4, splits);
    count_launch();
  }
  // dxg = dlogits . wg^T   [N x M] fp32
  g = UmmaGemm{};
  g.A = dlogits; g.B = wg; g.C = dxg; g.rows = (int)d.N; g.cols = d.M; g.K = d.E; g.batch = 1;
  g.a_kmajor = true; g.b_kmajor = true; g.a_ld = d.E; g.b_ld = d.E; g.c_ld = d.M; g.out_f32 = 1;
  rc = run_gemm(d, g, status, st);
  if (rc) return rc;
  dx_kernel<T><<<grid_for_rows(d.N), 256, 0, st>>>(reinterpret_cast<const float4*>(dxg), reinterpret_cast<const uint4*>(dbuf),
                                               expert_idx, slot,
                                               d.add_residual ? reinterpret_cast<const uint4*>(dy) : nullptr,
                                               reinterpret_cast<uint4*>(dx), d.N, d.G, d.S, d.C, row_vec);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

}  // namespace

int backward_combine_stage(const Dims& d, const void* context, const void* dy, void* workspace, cudaStream_t st) {
  const unsigned char* ctx = static_cast<const unsigned char*>(context);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  return d.bf16 ? combine_bwd_t<__nv_bfloat16>(d, ctx, dy, ws, st) : combine_bwd_t<float>(d, ctx, dy, ws, st);
}

// Expert FFN backward over the problems of `d` (E experts with d.rows rows each).  dh and dbuf stream
// the weights (read-heavy), dwo and dwi write a gradient the size of the weights from short
// contractions (write-heavy).
int backward_expert_stage(const Dims& d, const void* dout, const void* h, const uint32_t* hbits, const void* buf,
                          const void* wi, const void* wo, void* dh, void* dbuf, void* dwi, void* dwo, int* status,
                          cudaStream_t st) {
  NvtxRange range("gshard.backward.expert_ffn");
  const long long rows = d.rows;
  UmmaGemm g_dh{}, g_dwo{}, g_dwi{}, g_dbuf{};
  // dh = (dout . wo^T) masked by h > 0
  g_dh.A = dout; g_dh.B = wo; g_dh.C = dh; g_dh.mask = h; g_dh.mask_bits = hbits; g_dh.rows = d.rows; g_dh.cols = d.H; g_dh.K = d.M; g_dh.batch = d.E;
  g_dh.a_kmajor = true; g_dh.b_kmajor = true;
  g_dh.a_ld = d.M; g_dh.a_bs = rows * d.M; g_dh.b_ld = d.M; g_dh.b_bs = (long long)d.H * d.M; g_dh.c_ld = d.H; g_dh.c_bs = rows * d.H;
  g_dh.b_stream = 1; g_dh.prefer_two_sm = 1;
  // dwo[e] = h[e]^T . dout[e]   [H x M]
  g_dwo.A = h; g_dwo.B = dout; g_dwo.C = dwo; g_dwo.rows = d.H; g_dwo.cols = d.M; g_dwo.K = d.rows; g_dwo.batch = d.E;
  g_dwo.a_kmajor = false; g_dwo.b_kmajor = false;
  g_dwo.a_ld = d.H; g_dwo.a_bs = rows * d.H; g_dwo.b_ld = d.M; g_dwo.b_bs = rows * d.M; g_dwo.c_ld = d.M; g_dwo.c_bs = (long long)d.H * d.M;
  // dwi[e] = buf[e]^T . dh[e]   [M x H]
  g_dwi.A = buf; g_dwi.B = dh; g_dwi.C = dwi; g_dwi.rows = d.M; g_dwi.cols = d.H; g_dwi.K = d.rows; g_dwi.batch = d.E;
  g_dwi.a_kmajor = false; g_dwi.b_kmajor = false;
  g_dwi.a_ld = d.M; g_dwi.a_bs = rows * d.M; g_dwi.b_ld = d.H; g_dwi.b_bs = rows * d.H; g_dwi.c_ld = d.H; g_dwi.c_bs = (long long)d.M * d.H;
  // dbuf = dh . wi^T   [rows x M]
  g_dbuf.A = dh; g_dbuf.B = wi; g_dbuf.C = dbuf; g_dbuf.rows = d.rows; g_dbuf.cols = d.M; g_dbuf.K = d.H; g_dbuf.batch = d.E;
  g_dbuf.a_kmajor = true; g_dbuf.b_kmajor = true;
  g_dbuf.a_ld = d.H; g_dbuf.a_bs = rows * d.H; g_dbuf.b_ld = d.H; g_dbuf.b_bs = (long long)d.M * d.H; g_dbuf.c_ld = d.M; g_dbuf.c_bs = rows * d.M;
  g_dbuf.b_stream = 1; g_dbuf.prefer_two_sm = 1;
  // On request each read-heavy GEMM shares the GPU with a write-heavy one (half of the multiprocessors
  // each, two streams).  Measured at the MoE(512E) training shape this is slower than running the four
  // one after another on all multiprocessors, so it is not the default.
  // dwo has 64 row tiles per column block at the paper's shapes: on CTA pairs each CTA keeps half of the
  // resident B slice and an A ring of two row tiles instead of one.  Isolated launches at the MoE(512E)
  // training shape: 2.15 against 2.43 ms.  dwi has only eight row tiles per column block; its pair form
  // (two B slices, so that the next one loads during the current block) measures 2.28 against 2.32 ms
  // and stays off.  Under the power cap the training step takes the same time either way (fewer
  // cycles at a lower clock).
  g_dwo.prefer_two_sm = d.H >= 16 * 128;
  const int share = d.bwd_paired ? (device_sms() / 2) & ~1 : 0;
  int rc = run_gemm_pair(d, g_dh, g_dwo, share, status, st);
  if (rc) return rc;
  return run_gemm_pair(d, g_dbuf, g_dwi, share, status, st);
}

int backward_gate_stage(const Dims& d, const void* x, const void* wg, const void* context, const void* dy, float k_aux,
                        int groups_in_mean, const void* dbuf, void* dx, float* dwg, void* workspace, cudaStream_t st) {
  const unsigned char* ctx = static_cast<const unsigned char*>(context);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  return d.bf16 ? gate_bwd_t<__nv_bfloat16>(d, x, wg, ctx, dy, k_aux, groups_in_mean, dbuf, dx, dwg, ws, st)
                : gate_bwd_t<float>(d, x, wg, ctx, dy, k_aux, groups_in_mean, dbuf, dx, dwg, ws, st);
}

int backward_device(const gshard_moe_shape* shape, const void* x, const void* wg, const void* wi, const void* wo,
                    const void* context, const void* dy, float k_aux, void* dx, float* dwg, void* dwi, void* dwo,
                    void* workspace, size_t workspace_bytes, cudaStream_t st) {
  NvtxRange range("gshard.backward");
  const Dims d = make_dims(*shape);
  const BwdPlan bp = plan_backward(d);
  const CtxPlan cp = plan_context(d);
  if (workspace_bytes < bp.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  const unsigned char* ctx = static_cast<const unsigned char*>(context);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int* status = reinterpret_cast<int*>(ws + bp.status);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  int rc = backward_combine_stage(d, ctx, dy, ws, st);
  if (rc) return rc;
  rc = backward_expert_stage(d, ws + bp.dout, ctx + cp.h, d.simt ? nullptr : reinterpret_cast<const uint32_t*>(ctx + cp.hbits),
                             ctx + cp.buf, wi, wo, ws + bp.dh, ws + bp.dbuf, dwi, dwo, status, st);
  if (rc) return rc;
  return backward_gate_stage(d, x, wg, ctx, dy, k_aux, d.G, ws + bp.dbuf, dx, dwg, ws, st);
}

}  // namespace gshard
