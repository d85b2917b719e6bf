// Expert-parallel form of the layer (the paper's own partitioning, Algorithm 2 with the sharding
// annotations of the MoE layer): the groups G are split over the devices for gating, capacity
// assignment, dispatch and combine (wg replicated), the experts E are split over the devices for
// the expert FFN, and an AllToAll before and after the FFN changes between the two layouts
// ("GSEC,GSM->EGCM" is sharded on G on its inputs and on E on its output).
//
// Rank r of W holds groups [r*G/W, (r+1)*G/W) of x, u, y and experts [r*E/W, (r+1)*E/W) of wi, wo.
//   1. gating + capacity + dispatch over the local groups:   send [E, Gl*C, M] = [W][El, Gl*C, M]
//   2. AllToAll (equal splits): slab d goes to rank d        recv [W(src)][El, Gl*C, M]
//   3. regroup: rows of one local expert from all sources become contiguous, in global group
//      order                                                  in   [El, W*Gl*C = G*C, M]
//   4. expert FFN over the El local experts with G*C rows each (the same kernels as on one GPU)
//   5. inverse regroup, AllToAll back                         out  [E, Gl*C, M]
//   6. combine over the local groups; l_aux = sum over ranks of (sum of local group losses) / G
// The collectives are the caller's: two callbacks (all-to-all, all-reduce of floats) that enqueue
// on the given stream - NCCL behind torch.distributed in this repository's harness.  Every slab is
// received into this GPU's own workspace before any kernel or TMA load touches it; no tensor map
// ever covers another GPU's memory and no load is multicast.
#include <cstring>

#include "kernels.cuh"
#include "plan.cuh"

namespace gshard {

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Row of the FFN input [El, G*C, .] that holds row `row_local` (= gl*C + c) of local expert `el` in
// the slab received from rank `src`: the source's groups are global groups src*Gl + gl.
__host__ __device__ inline long long ep_ffn_row(int W, int El, int rows_local, int src, int el, int row_local) {
  return ((long long)el * W + src) * rows_local + row_local;
}
__host__ __device__ inline long long ep_slab_row(int El, int rows_local, int src, int el, int row_local) {
  return ((long long)src * El + el) * rows_local + row_local;
}

// dst/src as 16-byte vectors, row_vec per row.  inverse == 0: slab order -> FFN order.
__global__ void __launch_bounds__(256) ep_regroup_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int W,
                                                         int El, int rows_local, int row_vec, int inverse) {
  const long long chunk_vec = (long long)rows_local * row_vec;        // one (rank, expert) block is contiguous
  const long long total = (long long)W * El * chunk_vec;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long blk = i / chunk_vec, off = i % chunk_vec;
    const int s = (int)(blk / El), el = (int)(blk % El);              // blk indexes the slab order [W][El]
    const long long slab = ep_slab_row(El, rows_local, s, el, 0) * row_vec + off;
    const long long ffn = ep_ffn_row(W, El, rows_local, s, el, 0) * row_vec + off;
    if (inverse) dst[slab] = src[ffn]; else dst[ffn] = src[slab];
  }
}

void launch_ep_regroup(const void* src, void* dst, int W, int El, int rows_local, int row_vec, int inverse,
                       cudaStream_t st) {
  const long long total = (long long)W * El * rows_local * row_vec;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)device_sms() * 16;
  if (blocks > cap) blocks = cap;
  ep_regroup_kernel<<<(int)(blocks > 0 ? blocks : 1), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                                    W, El, rows_local, row_vec, inverse);
  count_launch();
}

int make_layout(const gshard_moe_shape* shape, int rank, int world, gshard_moe_ep_layout* out) {
  const int rc = validate_shape(shape);
  if (rc != GSHARD_OK) return rc;
  if (world < 1 || rank < 0 || rank >= world) return GSHARD_ERR_INVALID_ARG;
  if (shape->G % world || shape->E % world) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  gshard_moe_ep_layout l;
  l.rank = rank; l.world = world;
  l.groups_local = shape->G / world; l.experts_local = shape->E / world;
  l.group_begin = rank * l.groups_local; l.expert_begin = rank * l.experts_local;
  l.rows_local = l.groups_local * shape->C;
  const size_t esize = shape->dtype == GSHARD_BF16 ? 2 : 4;
  l.row_bytes = (size_t)shape->M * esize;
  l.bytes_per_peer = (size_t)l.experts_local * l.rows_local * l.row_bytes;
  l.local = *shape;  l.local.G = l.groups_local;                  // gating, capacity, dispatch, combine
  l.ffn = *shape;    l.ffn.E = l.experts_local;                   // expert FFN: all G groups' rows of El experts
  // the local problems must themselves be valid shapes (E stays global for the gating; El >= 1 for the FFN)
  const int rl = validate_shape(&l.local);
  if (rl != GSHARD_OK) return rl;
  *out = l;
  return GSHARD_OK;
}

}  // namespace

}  // namespace gshard

using namespace gshard;

extern "C" {

int gshard_moe_ep_plan(const gshard_moe_shape* shape, int rank, int world, gshard_moe_ep_layout* layout) {
  if (!layout) return GSHARD_ERR_INVALID_ARG;
  return make_layout(shape, rank, world, layout);
}

int gshard_moe_ep_regroup_host(const gshard_moe_ep_layout* l, const void* src, void* dst, size_t row_bytes,
                               int inverse) {
  if (!l || !src || !dst || row_bytes == 0 || l->world < 1 || l->experts_local < 1 || l->rows_local < 1)
    return GSHARD_ERR_INVALID_ARG;
  const unsigned char* s = static_cast<const unsigned char*>(src);
  unsigned char* d = static_cast<unsigned char*>(dst);
  for (int r = 0; r < l->world; ++r)
    for (int el = 0; el < l->experts_local; ++el)
      for (int row = 0; row < l->rows_local; ++row) {
        const size_t slab = (size_t)ep_slab_row(l->experts_local, l->rows_local, r, el, row) * row_bytes;
        const size_t ffn = (size_t)ep_ffn_row(l->world, l->experts_local, l->rows_local, r, el, row) * row_bytes;
        if (inverse) memcpy(d + slab, s + ffn, row_bytes); else memcpy(d + ffn, s + slab, row_bytes);
      }
  return GSHARD_OK;
}

size_t gshard_moe_ep_workspace_bytes(const gshard_moe_shape* shape, int world) {
  gshard_moe_ep_layout l;
  if (make_layout(shape, 0, world, &l) != GSHARD_OK) return 0;
  const Dims dl = make_dims(l.local);
  // the local forward plan (its buf / h / out regions have exactly the sizes the FFN over El experts
  // and G*C rows needs) plus two exchange buffers of one dispatch buffer each
  return plan_forward(dl).total + 2 * align_up((size_t)dl.R * dl.M * dl.esize);
}

size_t gshard_moe_ep_context_bytes(const gshard_moe_shape* shape, int world) {
  gshard_moe_ep_layout l;
  if (make_layout(shape, 0, world, &l) != GSHARD_OK) return 0;
  return plan_context(make_dims(l.local)).total;
}

size_t gshard_moe_ep_backward_workspace_bytes(const gshard_moe_shape* shape, int world) {
  gshard_moe_ep_layout l;
  if (make_layout(shape, 0, world, &l) != GSHARD_OK) return 0;
  const Dims dl = make_dims(l.local);
  return plan_backward(dl).total + 2 * align_up((size_t)dl.R * dl.M * dl.esize);
}

int gshard_moe_top2_forward_ep(const gshard_moe_shape* shape, int rank, int world, const void* x_local,
                               const void* wg, const void* wi_local, const void* wo_local, const float* u_local,
                               void* y_local, float* l_aux, const gshard_moe_routing* routing_out, void* context,
                               const gshard_ep_comm* comm, void* workspace, size_t workspace_bytes,
                               void* cuda_stream) {
  launch_counter().n = 0;
  gshard_moe_ep_layout l;
  const int rcl = make_layout(shape, rank, world, &l);
  if (rcl != GSHARD_OK) return rcl;
  const void* ptrs[] = {x_local, wg, wi_local, wo_local, u_local, y_local, workspace};
  for (const void* p : ptrs)
    if (p == nullptr || !aligned16(p)) return GSHARD_ERR_INVALID_ARG;
  if (l_aux == nullptr) return GSHARD_ERR_INVALID_ARG;
  if (world > 1 && (!comm || !comm->all_to_all || !comm->all_reduce_sum_f32)) return GSHARD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  const bool save = (shape->flags & GSHARD_FLAG_SAVE_FOR_BACKWARD) != 0;
  if (save && (!context || reinterpret_cast<uintptr_t>(context) % kAlign)) return GSHARD_ERR_INVALID_ARG;
  if (workspace_bytes < gshard_moe_ep_workspace_bytes(shape, world)) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  const int rcd = check_device();
  if (rcd != GSHARD_OK) return rcd;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Dims dl = make_dims(l.local);          // G = Gl, E global
  const Dims df = make_dims(l.ffn);            // G global, E = El: rows per expert = G*C
  const FwdPlan pl = plan_forward(dl);
  const CtxPlan cp = plan_context(dl);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  unsigned char* ctx = static_cast<unsigned char*>(context);
  const size_t slab_bytes = align_up((size_t)dl.R * dl.M * dl.esize);
  void* xa = ws + pl.total;                    // exchange buffers
  void* xb = ws + pl.total + slab_bytes;
  gshard_moe_routing r{};
  if (routing_out) r = *routing_out;
  int* status = reinterpret_cast<int*>(ws + pl.status);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  // with SAVE_FOR_BACKWARD the routing tensors and the activations the backward needs live in the
  // context: routing, softmax statistics and `out` in the LOCAL layout (this rank's groups), the
  // expert inputs, h and its ReLU mask in the FFN layout (this rank's experts, all groups)
  int32_t* expert_idx = save ? reinterpret_cast<int32_t*>(ctx + cp.expert_idx) : pick(r.expert_idx, ws, pl.expert_idx);
  int32_t* slot = save ? reinterpret_cast<int32_t*>(ctx + cp.slot) : pick(r.slot, ws, pl.slot);
  float* weight = save ? reinterpret_cast<float*>(ctx + cp.weight) : pick(r.weight, ws, pl.weight);
  int32_t* first_count = save ? reinterpret_cast<int32_t*>(ctx + cp.first_count) : pick(r.first_count, ws, pl.first_count);
  int32_t* slot_token = save ? reinterpret_cast<int32_t*>(ctx + cp.slot_token) : pick(r.slot_token, ws, pl.slot_token);
  float* gate12 = save ? reinterpret_cast<float*>(ctx + cp.gate12) : reinterpret_cast<float*>(ws + pl.gate12);
  float* rowmax = save ? reinterpret_cast<float*>(ctx + cp.rowmax) : reinterpret_cast<float*>(ws + pl.rowmax);
  float* rowinv = save ? reinterpret_cast<float*>(ctx + cp.rowinv) : reinterpret_cast<float*>(ws + pl.rowinv);
  float* m = pick(r.m, ws, pl.m);
  void* buf = ws + pl.buf;
  void* h = save ? static_cast<void*>(ctx + cp.h) : static_cast<void*>(ws + pl.h);
  void* out = save ? static_cast<void*>(ctx + cp.out) : static_cast<void*>(ws + pl.out);
  void* ffn_in_saved = save ? static_cast<void*>(ctx + cp.buf) : nullptr;

  int rc = gate_stage(dl, pl, ws, x_local, wg, expert_idx, gate12, m, rowmax, rowinv, st);
  if (rc != GSHARD_OK) return rc;
  // l_aux: this rank's group losses over the GLOBAL group count; the all-reduce below adds the shares
  rc = launch_capacity(dl, expert_idx, gate12, u_local, m, slot, weight, pick(r.flags, ws, pl.flags), first_count,
                       pick(r.total_count, ws, pl.total_count), slot_token, pick(r.l_aux_group, ws, pl.l_aux_group),
                       reinterpret_cast<int32_t*>(ws + pl.stats_group), l_aux, reinterpret_cast<long long*>(r.stats), st,
                       shape->G);
  if (rc != GSHARD_OK) return rc;
  // one rank: the dispatch buffer is the FFN input, so it goes straight to where the backward finds it
  if (world == 1 && save) buf = ffn_in_saved;
  launch_dispatch(dl, x_local, slot_token, buf, st, status);

  const int row_vec = (int)(l.row_bytes / 16);
  const void* ffn_in = buf;
  void* ffn_out = out;
  if (world > 1) {
    if (comm->all_to_all(comm->user, buf, xa, l.bytes_per_peer, cuda_stream) != 0) return GSHARD_ERR_CUDA;
    void* regrouped = save ? ffn_in_saved : xb;
    launch_ep_regroup(xa, regrouped, world, l.experts_local, l.rows_local, row_vec, 0, st);
    ffn_in = regrouped;
    ffn_out = xa;
  }
  rc = ffn_stage(df, ffn_in, wi_local, wo_local, h, save, ffn_out, ws + pl.ffn_scratch, status, st, nullptr, nullptr,
                 ws + pl.wt, nullptr, (save && !df.simt) ? reinterpret_cast<uint32_t*>(ctx + cp.hbits) : nullptr);
  if (rc != GSHARD_OK) return rc;
  if (world > 1) {
    launch_ep_regroup(xa, xb, world, l.experts_local, l.rows_local, row_vec, 1, st);
    if (comm->all_to_all(comm->user, xb, out, l.bytes_per_peer, cuda_stream) != 0) return GSHARD_ERR_CUDA;
    if (comm->all_reduce_sum_f32(comm->user, l_aux, 1, cuda_stream) != 0) return GSHARD_ERR_CUDA;
  }
  launch_combine(dl, out, expert_idx, slot, weight, y_local, st, dl.add_residual ? x_local : nullptr);
  if (save) {   // hand the caller the routing tensors it asked for
    struct { void* dst; const void* src; size_t n; } cps[] = {
        {r.expert_idx, expert_idx, (size_t)dl.N * 2 * 4}, {r.slot, slot, (size_t)dl.N * 2 * 4},
        {r.weight, weight, (size_t)dl.N * 2 * 4},         {r.first_count, first_count, (size_t)dl.G * dl.E * 4},
        {r.slot_token, slot_token, (size_t)dl.R * 4}};
    for (auto& c : cps)
      if (c.dst && cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int gshard_moe_top2_backward_ep(const gshard_moe_shape* shape, int rank, int world, const void* x_local, const void* wg,
                                const void* wi_local, const void* wo_local, const void* context, const void* dy_local,
                                float l_aux_weight, void* dx_local, float* dwg, void* dwi_local, void* dwo_local,
                                const gshard_ep_comm* comm, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  launch_counter().n = 0;
  gshard_moe_ep_layout l;
  const int rcl = make_layout(shape, rank, world, &l);
  if (rcl != GSHARD_OK) return rcl;
  if (!(shape->flags & GSHARD_FLAG_SAVE_FOR_BACKWARD)) return GSHARD_ERR_INVALID_ARG;
  const void* ptrs[] = {x_local, wg, wi_local, wo_local, context, dy_local, dx_local, dwg, dwi_local, dwo_local, workspace};
  for (const void* p : ptrs)
    if (p == nullptr || !aligned16(p)) return GSHARD_ERR_INVALID_ARG;
  if (world > 1 && (!comm || !comm->all_to_all || !comm->all_reduce_sum_f32)) return GSHARD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign || reinterpret_cast<uintptr_t>(context) % kAlign)
    return GSHARD_ERR_INVALID_ARG;
  if (workspace_bytes < gshard_moe_ep_backward_workspace_bytes(shape, world)) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  const int rcd = check_device();
  if (rcd != GSHARD_OK) return rcd;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Dims dl = make_dims(l.local);
  const Dims df = make_dims(l.ffn);
  const BwdPlan bp = plan_backward(dl);
  const CtxPlan cp = plan_context(dl);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  const unsigned char* ctx = static_cast<const unsigned char*>(context);
  const size_t slab_bytes = align_up((size_t)dl.R * dl.M * dl.esize);
  void* xa = ws + bp.total;
  void* xb = ws + bp.total + slab_bytes;
  int* status = reinterpret_cast<int*>(ws + bp.status);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  const int row_vec = (int)(l.row_bytes / 16);

  // 1. combine backward over the local groups: dw per choice, dout [E, Gl*C, M]
  int rc = backward_combine_stage(dl, ctx, dy_local, ws, st);
  if (rc != GSHARD_OK) return rc;
  // 2. the gradients of the expert outputs travel to the experts' owners, as the inputs did
  const void* dout_ffn = ws + bp.dout;
  void* dbuf_ffn = ws + bp.dbuf;
  if (world > 1) {
    if (comm->all_to_all(comm->user, ws + bp.dout, xa, l.bytes_per_peer, cuda_stream) != 0) return GSHARD_ERR_CUDA;
    launch_ep_regroup(xa, xb, world, l.experts_local, l.rows_local, row_vec, 0, st);
    dout_ffn = xb;
    dbuf_ffn = ws + bp.dout;                  // the local dout has been sent: its region takes dbuf in FFN order
  }
  // 3. expert FFN backward over the local experts and all groups' rows
  rc = backward_expert_stage(df, dout_ffn, ctx + cp.h, df.simt ? nullptr : reinterpret_cast<const uint32_t*>(ctx + cp.hbits),
                             ctx + cp.buf, wi_local, wo_local, ws + bp.dh, dbuf_ffn, dwi_local, dwo_local, status, st);
  if (rc != GSHARD_OK) return rc;
  // 4. the gradients of the expert inputs travel back to the groups' owners
  if (world > 1) {
    launch_ep_regroup(dbuf_ffn, xa, world, l.experts_local, l.rows_local, row_vec, 1, st);
    if (comm->all_to_all(comm->user, xa, ws + bp.dbuf, l.bytes_per_peer, cuda_stream) != 0) return GSHARD_ERR_CUDA;
  }
  // 5. gating backward and dx over the local groups; wg is replicated, so its gradient is the sum of
  //    the ranks' contributions
  rc = backward_gate_stage(dl, x_local, wg, ctx, dy_local, l_aux_weight, shape->G, ws + bp.dbuf, dx_local, dwg, ws, st);
  if (rc != GSHARD_OK) return rc;
  if (world > 1 && comm->all_reduce_sum_f32(comm->user, dwg, (size_t)dl.M * dl.E, cuda_stream) != 0) return GSHARD_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Expert-parallel forward with the exchange fused into the dispatch and combine kernels.
//
// Instead of dispatching into a local buffer and handing it to an AllToAll, the dispatch kernel
// writes every token row straight into the expert owner's input buffer over NVLink (peer stores),
// already in the layout the expert FFN reads ([El][G*C][M], rows in global group order), and the
// combine kernel gathers a token's (at most two) expert output rows straight out of the owners'
// output buffers (peer loads).  Each row crosses NVLink once, inside the kernel that produces or
// consumes it; the two AllToAll passes and the two regrouping copies of the collective form
// disappear.  The expert FFN itself only ever reads and writes this GPU's own memory (its TMA
// tensor maps never cover a peer's memory), and nothing is multicast.
// Ordering between ranks is the caller's, through one callback: rendezvous(phase) must make this
// rank's stream (a) publish "my work enqueued so far is done" and (b) wait for the same from every
// other rank - e.g. an interprocess event per rank, recorded and waited on; no kernel waits for
// another rank's kernel.
namespace gshard {
namespace {

constexpr int kMaxPeers = 64;
struct PeerPtrs { unsigned char* p[kMaxPeers]; };

// in_of(d) = peer d's exchange buffer; its first half is the FFN input [El][G*C][M], its second half
// the FFN output.  Row of (local expert el, global group g, position c): (el*G + g)*C + c.
template <typename V>
__global__ void __launch_bounds__(256) dispatch_p2p_kernel(const V* __restrict__ x, const int32_t* __restrict__ slot_token,
                                                           PeerPtrs peers, long long rows_all, int G, int Gl, int S, int C,
                                                           int El, int rank, int row_vec) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = warp; r < rows_all; r += nwarps) {       // r = (e*Gl + gl)*C + c over ALL experts, local groups
    const int tok = slot_token[r];
    const int c = (int)(r % C), gl = (int)((r / C) % Gl), e = (int)(r / ((long long)C * Gl));
    const int dest = e / El, el = e % El;
    V* dst = reinterpret_cast<V*>(peers.p[dest]) + (((long long)el * G + (rank * Gl + gl)) * C + c) * row_vec;
    if (tok >= 0 && tok < S) {
      const V* src = x + ((long long)gl * S + tok) * row_vec;
      for (int i = lane; i < row_vec; i += 32) dst[i] = __ldg(src + i);
    } else {
      for (int i = lane; i < row_vec; i += 32) dst[i] = make_uint4(0, 0, 0, 0);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) combine_p2p_kernel(PeerPtrs peers, size_t out_offset_bytes,
                                                          const int32_t* __restrict__ expert_idx,
                                                          const int32_t* __restrict__ slot, const float* __restrict__ weight,
                                                          const uint4* __restrict__ residual, uint4* __restrict__ y,
                                                          long long N, int G, int Gl, int S, int C, int E, int El, int rank,
                                                          int row_vec) {
  constexpr int n = Vec16<T>::n;
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long t = warp; t < N; t += nwarps) {
    const int gl = (int)(t / S);
    const uint4* rows[2] = {nullptr, nullptr};
    float w[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int e = expert_idx[2 * t + k], sl = slot[2 * t + k];
      w[k] = weight[2 * t + k];
      if (sl >= 0 && sl < C && e >= 0 && e < E)
        rows[k] = reinterpret_cast<const uint4*>(peers.p[e / El] + out_offset_bytes) +
                  (((long long)(e % El) * G + (rank * Gl + gl)) * C + sl) * row_vec;
    }
    // four 16-byte pieces per lane and row at a time, all loads issued before the first use: the rows
    // come over NVLink (plain loads - a peer's memory is not read through the read-only path)
    for (int i0 = lane; i0 < row_vec; i0 += 128) {
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      uint4 v0[4], v1[4], vr[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + 32 * k;
        const bool in = i < row_vec;
        v0[k] = (rows[0] && in) ? rows[0][i] : z;
        v1[k] = (rows[1] && in) ? rows[1][i] : z;
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
        for (int j = 0; j < n; ++j) acc[j] = fmaf(w[1], f1[j], fmaf(w[0], f0[j], acc[j]));
        y[t * row_vec + i] = Vec16<T>::store(acc);
      }
    }
  }
}

}  // namespace
}  // namespace gshard

extern "C" {

size_t gshard_moe_ep_p2p_buffer_bytes(const gshard_moe_shape* shape, int world) {
  gshard_moe_ep_layout l;
  if (make_layout(shape, 0, world, &l) != GSHARD_OK || world > kMaxPeers) return 0;
  const Dims dl = make_dims(l.local);
  return 2 * align_up((size_t)dl.R * dl.M * dl.esize);
}

int gshard_moe_top2_forward_ep_p2p(const gshard_moe_shape* shape, int rank, int world, const void* x_local,
                                   const void* wg, const void* wi_local, const void* wo_local, const float* u_local,
                                   void* y_local, float* l_aux, const gshard_moe_routing* routing_out,
                                   const gshard_ep_p2p* p2p, const gshard_ep_comm* comm, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream) {
  launch_counter().n = 0;
  gshard_moe_ep_layout l;
  const int rcl = make_layout(shape, rank, world, &l);
  if (rcl != GSHARD_OK) return rcl;
  if (world > kMaxPeers || (shape->flags & GSHARD_FLAG_SAVE_FOR_BACKWARD)) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  const void* ptrs[] = {x_local, wg, wi_local, wo_local, u_local, y_local, workspace};
  for (const void* p : ptrs)
    if (p == nullptr || !aligned16(p)) return GSHARD_ERR_INVALID_ARG;
  if (l_aux == nullptr || p2p == nullptr || p2p->peer_buffers == nullptr) return GSHARD_ERR_INVALID_ARG;
  if (world > 1 && p2p->rendezvous == nullptr) return GSHARD_ERR_INVALID_ARG;
  PeerPtrs peers{};
  for (int w = 0; w < world; ++w) {
    if (p2p->peer_buffers[w] == nullptr || reinterpret_cast<uintptr_t>(p2p->peer_buffers[w]) % kAlign) return GSHARD_ERR_INVALID_ARG;
    peers.p[w] = static_cast<unsigned char*>(p2p->peer_buffers[w]);
  }
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  const Dims dl = make_dims(l.local);
  const Dims df = make_dims(l.ffn);
  const FwdPlan pl = plan_forward(dl);
  if (workspace_bytes < pl.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  const int rcd = check_device();
  if (rcd != GSHARD_OK) return rcd;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  const size_t half = align_up((size_t)dl.R * dl.M * dl.esize);
  unsigned char* my_in = peers.p[rank];
  unsigned char* my_out = peers.p[rank] + half;
  gshard_moe_routing r{};
  if (routing_out) r = *routing_out;
  int* status = reinterpret_cast<int*>(ws + pl.status);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  int32_t* expert_idx = pick(r.expert_idx, ws, pl.expert_idx);
  int32_t* slot = pick(r.slot, ws, pl.slot);
  float* weight = pick(r.weight, ws, pl.weight);
  int32_t* slot_token = pick(r.slot_token, ws, pl.slot_token);
  float* gate12 = reinterpret_cast<float*>(ws + pl.gate12);
  float* m = pick(r.m, ws, pl.m);

  int rc = gate_stage(dl, pl, ws, x_local, wg, expert_idx, gate12, m, reinterpret_cast<float*>(ws + pl.rowmax),
                      reinterpret_cast<float*>(ws + pl.rowinv), st);
  if (rc != GSHARD_OK) return rc;
  rc = launch_capacity(dl, expert_idx, gate12, u_local, m, slot, weight, pick(r.flags, ws, pl.flags),
                       pick(r.first_count, ws, pl.first_count), pick(r.total_count, ws, pl.total_count), slot_token,
                       pick(r.l_aux_group, ws, pl.l_aux_group), reinterpret_cast<int32_t*>(ws + pl.stats_group), l_aux,
                       reinterpret_cast<long long*>(r.stats), st, shape->G);
  if (rc != GSHARD_OK) return rc;
#define GS_RENDEZVOUS(phase) \
  do { if (world > 1 && p2p->rendezvous(p2p->user, (phase), cuda_stream) != 0) return GSHARD_ERR_CUDA; } while (0)
  // phase 0: every rank is done with the previous use of the exchange buffers
  GS_RENDEZVOUS(0);
  const int row_vec = (int)(l.row_bytes / 16);
  {
    NvtxRange range("gshard.dispatch_p2p");
    dispatch_p2p_kernel<uint4><<<grid_for_rows(dl.R), 256, 0, st>>>(static_cast<const uint4*>(x_local), slot_token, peers,
                                                                    dl.R, shape->G, l.groups_local, dl.S, dl.C,
                                                                    l.experts_local, rank, row_vec);
    count_launch();
  }
  // phase 1: every rank's rows have arrived in the owners' input buffers
  GS_RENDEZVOUS(1);
  rc = ffn_stage(df, my_in, wi_local, wo_local, ws + pl.h, false, my_out, ws + pl.ffn_scratch, status, st, nullptr, nullptr,
                 ws + pl.wt);
  if (rc != GSHARD_OK) return rc;
  // phase 2: every rank's expert outputs are complete
  GS_RENDEZVOUS(2);
  {
    NvtxRange range("gshard.combine_p2p");
    const uint4* residual = dl.add_residual ? static_cast<const uint4*>(x_local) : nullptr;
    if (dl.bf16)
      combine_p2p_kernel<__nv_bfloat16><<<grid_for_rows(dl.N), 256, 0, st>>>(
          peers, half, expert_idx, slot, weight, residual, static_cast<uint4*>(y_local), dl.N, shape->G, l.groups_local, dl.S,
          dl.C, dl.E, l.experts_local, rank, row_vec);
    else
      combine_p2p_kernel<float><<<grid_for_rows(dl.N), 256, 0, st>>>(
          peers, half, expert_idx, slot, weight, residual, static_cast<uint4*>(y_local), dl.N, shape->G, l.groups_local, dl.S,
          dl.C, dl.E, l.experts_local, rank, row_vec);
    count_launch();
  }
#undef GS_RENDEZVOUS
  if (world > 1 && comm && comm->all_reduce_sum_f32 && comm->all_reduce_sum_f32(comm->user, l_aux, 1, cuda_stream) != 0)
    return GSHARD_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

}  // extern "C"
