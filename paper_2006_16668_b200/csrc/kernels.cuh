// Launchers of the library's kernels (one .cu file each) as seen by the C-ABI layer.
#pragma once
#include "common.cuh"

namespace gshard {

// gate.cu: row statistics + top-2 on stored logits, tile column sums, mean gates.
void launch_gate_rows(const Dims& d, const float* logits, int32_t* expert_idx, float* gate12, float* rowmax,
                      float* rowinv, cudaStream_t st);
void launch_gate_means(const Dims& d, const float* logits, const float* rowmax, const float* rowinv,
                       float* partial, float* m, cudaStream_t st);

// gate_fused.cu: bf16 logits GEMM on tcgen05 with row statistics and top-2 in the epilogue.
// gate_cluster.cu: gating with the mean gates' partial sums fused in (clusters, distributed shared
// memory); partial32 holds one row of column sums per 32-token block.
bool gate_cluster_supported(const Dims& d);
int launch_gate_cluster(const Dims& d, const void* x, const void* wg, int32_t* expert_idx, float* gate12,
                        float* rowmax, float* rowinv, float* partial32, int* status, cudaStream_t st);
// gate.cu: m[g,e] = (1/S) * sum of the group's `blocks_per_group` partial rows, in order.
void launch_gate_mean_blocks(const Dims& d, const float* partial, int blocks_per_group, float* m, cudaStream_t st);
// gate.cu: the mean-gate pass over logits stored as float4 [E/4][N] (what gate_fused2 writes).
void launch_gate_means_t(const Dims& d, const float* logits_t, const float* rowmax, const float* rowinv,
                         float* partial, float* m, cudaStream_t st);
// gate_fused2.cu: the same gating kernel on CTA pairs (tcgen05 cta_group::2, half of the wg tile per CTA).
bool gate_fused2_supported(const Dims& d);
int launch_gate_fused2(const Dims& d, const void* x, const void* wg, float* logits, int32_t* expert_idx,
                       float* gate12, float* rowmax, float* rowinv, int* status, cudaStream_t st);
int launch_gate_fused(const Dims& d, const void* x, const void* wg, float* logits, int32_t* expert_idx,
                      float* gate12, float* rowmax, float* rowinv, int* status, cudaStream_t st);

// capacity.cu
int launch_capacity(const Dims& d, const int32_t* expert_idx, const float* gate12, const float* u, const float* m,
                    int32_t* slot, float* weight, uint8_t* flags, int32_t* first_count, int32_t* total_count,
                    int32_t* slot_token, float* l_aux_group, int32_t* stats_group, float* l_aux, long long* stats,
                    cudaStream_t st, int groups_in_mean = 0);
int capacity_warps_for(int E);
// Debug check of the routing tensors (every invariant Algorithm 1 implies for them); a violation
// records GSHARD_ERR_INTERNAL in *status, nothing traps.
void launch_routing_check(const Dims& d, const int32_t* expert_idx, const int32_t* slot, const float* weight,
                          const uint8_t* flags, const int32_t* slot_token, int* status, cudaStream_t st);

// dispatch_combine.cu
void launch_dispatch(const Dims& d, const void* x, const int32_t* slot_token, void* buf, cudaStream_t st,
                     int* status = nullptr);
// slot_crow (optional): the expert outputs are stored by compacted row; slot_crow[e, g*C+c] is the row.
void launch_combine(const Dims& d, const void* out, const int32_t* expert_idx, const int32_t* slot,
                    const float* weight, void* y, cudaStream_t st, const void* residual = nullptr,
                    const int32_t* slot_crow = nullptr);

// compact.cu: per expert, the filled slots in (group, position) order become rows 0 .. kept-1.
//   crow_token [E, G*C]  global token index (g*S + s) of compacted row j, j < kept[e]
//   slot_crow  [E, G*C]  compacted row of slot (g, c), or -1 for an empty slot
//   kept [E]; tile_base: three exclusive prefixes with E + 1 entries each (128-row tiles; 256-row
//   tiles for CTA pairs; the 128-row tile left behind those), then for each list the expert that owns
//   every row tile, compact_max_tiles(d) entries per list
inline int compact_max_tiles(const Dims& d) { return d.E * ((d.rows + 127) / 128); }
inline size_t compact_tile_ints(const Dims& d) { return 3 * ((size_t)d.E + 1) + 3 * (size_t)compact_max_tiles(d); }
void launch_compact(const Dims& d, const int32_t* slot_token, int32_t* crow_token, int32_t* slot_crow, int32_t* kept,
                    int32_t* tile_base, cudaStream_t st);
// buf[e, j, :] = x[crow_token[e, j], :] for j < kept[e]; other rows are left untouched
void launch_dispatch_compact(const Dims& d, const void* x, const int32_t* crow_token, const int32_t* kept, void* buf,
                             cudaStream_t st);

// dispatch_combine.cu: dst[b][c][r] = src[b][r][c] for a batch of fp32 matrices [rows, cols].
void launch_transpose_f32(const float* src, float* dst, int batch, int rows, int cols, cudaStream_t st);

// umma_gemm.cu: batched bf16 GEMM on tcgen05, C[b] = act(A[b] . B[b]).
struct UmmaGemm {
  const void* A; const void* B; void* C;
  const void* mask;          // CUDA-core path: optional tensor laid out like C, output zeroed where mask <= 0
  const uint32_t* mask_bits; // tensor-core path: the same as bits, [batch][rows][cols/32] words
  uint32_t* mask_bits_out;   // tensor-core path: write bit = (accumulator value > 0) in that layout
  int rows, cols, K, batch;
  bool a_kmajor;             // A stored [rows, K] (K contiguous); else stored [K, rows]
  bool b_kmajor;             // B stored [cols, K] (K contiguous); else stored [K, cols]
  long long a_ld, a_bs;      // elements between consecutive stored rows / between batches
  long long b_ld, b_bs;
  long long c_ld, c_bs;      // C is [rows, cols] row-major
  int out_f32;               // C is float instead of bf16
  int relu;
  int a_stream, b_stream;    // operand is read once: load with an evict-first L2 hint
  int prefer_two_sm;         // run on CTA pairs (cta_group::2) when a problem has more than 128 rows
  int tf32;                  // A and B hold float: contraction on the tensor cores in TF32 (both operands
                             // K-major, float output)
  const int* tile_base;      // ragged batch (device pointer, batch + 1 ints): problem b has
                             // tile_base[b+1] - tile_base[b] row tiles (128 rows on single CTAs, 256 rows on
                             // pairs)
  const int* tile_problem;   // with tile_base: the problem that owns each row tile (tile_base[batch] ints)
  const int* pair_base;      // single-CTA kernel with tile_base: problem b's row tiles start behind
                             // 2 * (pair_base[b+1] - pair_base[b]) tiles of 128 rows, which a launch on CTA
                             // pairs covers (same kind of prefix array)
  int ragged_on_pairs;       // tile_base counts 256-row tiles: run on CTA pairs
  int plain_stores;          // epilogue writes C with 16-byte stores instead of bulk tensor (TMA) stores
  int max_ctas;              // > 0: use at most this many CTAs (persistent grid), leaving the other
                             // multiprocessors to a kernel running beside this one on another stream
};
int launch_umma_gemm(const UmmaGemm& g, int* status, cudaStream_t st);
// umma2_gemm.cu: the same contraction with the two-SM MMA (CTA pairs, 256 x 256 tiles).
int launch_umma2_gemm(const UmmaGemm& g, int* status, cudaStream_t st);

// ffn_fused.cu: both expert GEMMs in one persistent launch; groups of four CTAs exchange 256-column
// chunks of the hidden activations through a small L2-resident scratch ring.
bool ffn_fused_supported(const Dims& d);
size_t ffn_fused_scratch_bytes(const Dims& d);
// With x_gather / slot_token the rows of GEMM-1's A operand are gathered from x[G*S, M] by index
// (TMA tile::gather4) and `buf` is not read.
int launch_ffn_fused(const Dims& d, const void* buf, const void* wi, const void* wo, void* scratch, void* out,
                     int* status, cudaStream_t st, const void* x_gather = nullptr,
                     const int32_t* slot_token = nullptr);

}  // namespace gshard
