// Byte offsets of every region of the caller's workspace / context buffers.  All regions are
// 256-byte aligned; the status word is the first word of the workspace.
#pragma once
#include <algorithm>
#include "common.cuh"
#include "kernels.cuh"

namespace gshard {

struct Carver {
  size_t off = 0;
  size_t take(size_t bytes) { const size_t o = off; off = align_up(off + bytes); return o; }
};

struct FwdPlan {
  size_t status, logits, rowmax, rowinv, partial, gate12, m, expert_idx, slot, weight, flags, first_count,
      total_count, slot_token, l_aux_group, stats_group, ffn_scratch, buf, h, out, wt, crow_token, slot_crow, kept,
      tile_base, total;
};

inline FwdPlan plan_forward(const Dims& d) {
  Carver c; FwdPlan p;
  const size_t N = (size_t)d.N, R = (size_t)d.R;
  p.status = c.take(256);
  p.logits = c.take(N * d.E * 4);
  p.rowmax = c.take(N * 4);
  p.rowinv = c.take(N * 4);
  // column-sum partials: one row per 128-token tile (two-pass gating) or per 32-token block
  // (cluster gating)
  p.partial = c.take(std::max((size_t)d.G * d.tiles_per_group, (size_t)((d.N + 31) / 32)) * d.E * 4);
  p.gate12 = c.take(N * 2 * 4);
  p.m = c.take((size_t)d.G * d.E * 4);
  p.expert_idx = c.take(N * 2 * 4);
  p.slot = c.take(N * 2 * 4);
  p.weight = c.take(N * 2 * 4);
  p.flags = c.take(N);
  p.first_count = c.take((size_t)d.G * d.E * 4);
  p.total_count = c.take((size_t)d.G * d.E * 4);
  p.slot_token = c.take(R * 4);
  p.l_aux_group = c.take((size_t)d.G * 4);
  p.stats_group = c.take((size_t)d.G * 8 * 4);
  p.ffn_scratch = c.take(ffn_fused_scratch_bytes(d));
  p.buf = c.take(R * d.M * d.esize);
  p.h = c.take(R * d.H * d.esize);
  p.out = c.take(R * d.M * d.esize);
  // TF32 expert contractions: transposed copies of both weight tensors (K-major B operands)
  p.wt = c.take(d.tf32_experts ? 2 * (size_t)d.E * d.M * d.H * 4 : 0);
  // compacted slots: row lists both ways, kept counts, row-tile prefix
  p.crow_token = c.take(d.compact_slots ? R * 4 : 0);
  p.slot_crow = c.take(d.compact_slots ? R * 4 : 0);
  p.kept = c.take(d.compact_slots ? (size_t)d.E * 4 : 0);
  p.tile_base = c.take(d.compact_slots ? compact_tile_ints(d) * 4 : 0);   // prefixes and tile owners (compact.cu)
  p.total = c.off;
  return p;
}

// Saved by the forward for the backward: routing, softmax row statistics, dispatched inputs, hidden
// activations (and their ReLU mask as bits) and expert outputs.
struct CtxPlan {
  size_t expert_idx, slot, weight, first_count, slot_token, gate12, rowmax, rowinv, h, out, hbits, buf, total;
};

inline CtxPlan plan_context(const Dims& d) {
  Carver c; CtxPlan p;
  const size_t N = (size_t)d.N, R = (size_t)d.R;
  p.expert_idx = c.take(N * 2 * 4);
  p.slot = c.take(N * 2 * 4);
  p.weight = c.take(N * 2 * 4);
  p.first_count = c.take((size_t)d.G * d.E * 4);
  p.slot_token = c.take(R * 4);
  p.gate12 = c.take(N * 2 * 4);
  p.rowmax = c.take(N * 4);
  p.rowinv = c.take(N * 4);
  p.h = c.take(R * d.H * d.esize);
  p.out = c.take(R * d.M * d.esize);
  p.hbits = c.take(d.simt ? 0 : R * (size_t)d.H / 8);   // ReLU mask as bits, written by the forward's GEMM-1
  p.buf = c.take(R * d.M * d.esize);                    // dispatched expert inputs (dwi contracts over them)
  p.total = c.off;
  return p;
}

struct StagePlan { size_t x, u, y, l_aux, total; };

inline StagePlan plan_staging(const Dims& d) {
  Carver c; StagePlan p;
  p.x = c.take((size_t)d.N * d.M * d.esize);
  p.u = c.take((size_t)d.N * 4);
  p.y = c.take((size_t)d.N * d.M * d.esize);
  p.l_aux = c.take(256);
  p.total = c.off;
  return p;
}

// Backward scratch: logits / dlogits [N,E], dout, dh, dbuf, per-token dw (the dispatched inputs come
// from the context).
struct BwdPlan {
  size_t status, logits, dlogits, dw, dout, dh, dbuf, dxg, total;
};

inline BwdPlan plan_backward(const Dims& d) {
  Carver c; BwdPlan p;
  const size_t N = (size_t)d.N, R = (size_t)d.R;
  p.status = c.take(256);
  p.logits = c.take(N * d.E * 4);
  p.dlogits = c.take(N * d.E * d.esize);
  p.dw = c.take(N * 2 * 4);
  p.dout = c.take(R * d.M * d.esize);
  p.dh = c.take(R * d.H * d.esize);
  p.dbuf = c.take(R * d.M * d.esize);
  p.dxg = c.take(N * d.M * 4);
  p.total = c.off;
  return p;
}

int validate_shape(const gshard_moe_shape* s);

// api.cu: the stages as launch sequences, shared by the whole-layer, stage and expert-parallel calls.
template <typename T> inline T* pick(T* user, unsigned char* ws, size_t off) {
  return user ? user : reinterpret_cast<T*>(ws + off);
}
int gate_stage(const Dims& d, const FwdPlan& pl, unsigned char* ws, const void* x, const void* wg,
               int32_t* expert_idx, float* gate12, float* m, float* rowmax, float* rowinv, cudaStream_t st);
bool ffn_runs_fused(const Dims& d, bool keep_h);
// With x / slot_token (only where ffn_runs_fused) the rows are gathered from x and buf is not read.
// wt: with d.tf32_experts, room for the transposed copies of wi and wo (2 * E * M * H floats).
int ffn_stage(const Dims& d, const void* buf, const void* wi, const void* wo, void* h, bool keep_h, void* out,
              void* fused_scratch, int* status, cudaStream_t st, const void* x, const int32_t* slot_token,
              void* wt = nullptr, const int* tile_base = nullptr, uint32_t* relu_bits_out = nullptr);
int check_device();

// The three parts of the backward pass (backward.cu); workspace laid out by plan_backward(d),
// context by plan_context(d).
int backward_combine_stage(const Dims& d, const void* context, const void* dy, void* workspace, cudaStream_t st);
int backward_expert_stage(const Dims& d, const void* dout, const void* h, const uint32_t* hbits, const void* buf,
                          const void* wi, const void* wo, void* dh, void* dbuf, void* dwi, void* dwo, int* status,
                          cudaStream_t st);
int backward_gate_stage(const Dims& d, const void* x, const void* wg, const void* context, const void* dy, float k_aux,
                        int groups_in_mean, const void* dbuf, void* dx, float* dwg, void* workspace, cudaStream_t st);

}  // namespace gshard
