// One description of a batched contraction, run either on tcgen05 (bf16) or on CUDA cores.
#pragma once
#include "kernels.cuh"
#include "simt_gemm.cuh"

namespace gshard {

// A and B hold the configuration dtype; C holds float when g.out_f32, else the dtype.
inline int run_gemm(const Dims& d, const UmmaGemm& g_in, int* status, cudaStream_t st) {
  UmmaGemm g = g_in;
  if (d.plain_stores) g.plain_stores = 1;
  if (!d.simt) {
    // CTA pairs with the two-SM MMA read only half of the B tile from their own shared memory per
    // MMA and load a third fewer operand bytes per SM; the one-SM kernel's 128 x 256 tiles keep the
    // shared memory busy with 96 B/clk of operand reads plus 96 B/clk of TMA writes, which is what
    // holds its tensor pipe near 65 %.  Callers mark the GEMMs that measured faster on pairs (the two
    // forward expert GEMMs); the flags force either form everywhere.  A single row tile would leave
    // the second CTA of a pair without rows.
    if (g.tf32) return GSHARD_ERR_INTERNAL;   // bf16 operands cannot be read as TF32
    if (g.tile_base && g.ragged_on_pairs) return launch_umma2_gemm(g, status, st);   // a ragged list of 256-row tiles
    if (g.rows > 128 && !g.tile_base && !d.one_sm_mma && (d.two_sm_mma || g.prefer_two_sm)) {
      const int rc = launch_umma2_gemm(g, status, st);
      if (rc == GSHARD_OK) return rc;       // a refused cluster launch ran nothing: single CTAs take over
    }
    return launch_umma_gemm(g, status, st);
  }
  // fp32 dtype with the TF32 option: the GEMMs marked by their caller run on the tensor cores
  if (!d.bf16 && d.tf32_experts && g.tf32) return launch_umma_gemm(g, status, st);
  SimtGemm s{};
  s.A = g.A; s.B = g.B; s.C = g.C; s.mask = g.mask;
  s.rows = g.rows; s.cols = g.cols; s.K = g.K; s.batch = g.batch;
  s.a_rs = g.a_kmajor ? g.a_ld : 1; s.a_cs = g.a_kmajor ? 1 : g.a_ld; s.a_bs = g.a_bs;
  s.b_rs = g.b_kmajor ? 1 : g.b_ld; s.b_cs = g.b_kmajor ? g.b_ld : 1; s.b_bs = g.b_bs;
  s.c_rs = g.c_ld; s.c_bs = g.c_bs; s.relu = g.relu; s.accumulate = 0;
  if (d.bf16) {
    if (g.out_f32) launch_simt_gemm<__nv_bfloat16, __nv_bfloat16, float>(s, st);
    else launch_simt_gemm<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16>(s, st);
  } else {
    launch_simt_gemm<float, float, float>(s, st);
  }
  return GSHARD_OK;
}

}  // namespace gshard
