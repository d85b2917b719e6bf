// Host-side construction of TMA tensor maps (cuTensorMapEncodeTiled through the runtime's
// driver entry point lookup, so that the library does not link libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "kernels.cuh"

namespace gshard {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// 3-D bf16 tensor map {inner, outer, batch} with a {box_inner, box_outer, 1} box, 128-byte swizzle;
// out-of-range elements read as zero.  ld_elems / bs_elems: elements between consecutive outer
// rows / batches.
// esize 2: bfloat16 elements; esize 4: float elements (the box's inner extent stays 128 bytes).
inline bool make_map(CUtensorMap* map, const void* base, long long inner, long long outer, long long batch,
                     long long ld_elems, long long bs_elems, int box_inner, int box_outer, int esize = 2) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)ld_elems * esize, (cuuint64_t)(batch > 1 ? bs_elems : ld_elems * outer) * esize};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, esize == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
            const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of an output matrix batch C [batch][rows][cols] (row pitch c_ld, batch pitch c_bs elements)
// for the epilogue's 32-row x 128-byte stores.
inline bool make_store_map(CUtensorMap* map, void* base, long long cols, long long rows, long long batch,
                           long long c_ld, long long c_bs, int esize) {
  return make_map(map, base, cols, rows, batch, c_ld, c_bs, 128 / esize, 32, esize);
}

// The store map of a GEMM's output, when its layout allows bulk stores (16-byte aligned base and row
// pitch) and the caller did not ask for plain stores; false = use plain 16-byte stores.
inline bool store_map_for(const UmmaGemm& g, CUtensorMap* mc) {
  const int esize = g.out_f32 ? 4 : 2;
  if (g.plain_stores || (reinterpret_cast<uintptr_t>(g.C) & 15u) || (g.c_ld * esize) % 16 ||
      (g.batch > 1 && (g.c_bs * esize) % 16))
    return false;
  return make_store_map(mc, g.C, g.cols, g.rows, g.batch, g.c_ld, g.c_bs, esize);
}

}  // namespace gshard
