// C-ABI layer: argument validation, workspace planning and the launch sequences of the forward
// pass and its stages.  Declarations and semantics: include/gshard_moe.h.
#include <cstring>

#include "kernels.cuh"
#include "gemm_dispatch.cuh"
#include "plan.cuh"

namespace gshard {

LaunchCounter& launch_counter() {
  static thread_local LaunchCounter c;
  return c;
}

struct FfnTiming { void* start = nullptr; void* stop = nullptr; };
static FfnTiming& ffn_timing() {
  static thread_local FfnTiming t;
  return t;
}

int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GSHARD_ERR_CUDA;
  return major == 10 ? GSHARD_OK : GSHARD_ERR_ARCH;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define GS_REQUIRE_PTR(p)                                          \
  do {                                                             \
    if ((p) == nullptr || !aligned16(p)) return GSHARD_ERR_INVALID_ARG; \
  } while (0)
#define GS_TRY(expr)                       \
  do {                                     \
    const int _rc = (expr);                \
    if (_rc != GSHARD_OK) return _rc;      \
  } while (0)

}  // namespace

// logits[N,E] = x[N,M] . wg[M,E], fp32 out.
int gate_logits(const Dims& d, const void* x, const void* wg, float* logits, int* status, cudaStream_t st) {
  UmmaGemm g{};
  g.A = x; g.B = wg; g.C = logits;
  g.rows = (int)d.N; g.cols = d.E; g.K = d.M; g.batch = 1;
  g.a_kmajor = true; g.b_kmajor = false;
  g.a_ld = d.M; g.b_ld = d.E; g.c_ld = d.E;
  g.out_f32 = 1; g.a_stream = 1;
  return run_gemm(d, g, status, st);
}

int gate_stage(const Dims& d, const FwdPlan& pl, unsigned char* ws, const void* x, const void* wg,
               int32_t* expert_idx, float* gate12, float* m, float* rowmax, float* rowinv, cudaStream_t st) {
  NvtxRange range("gshard.gate");
  float* logits = reinterpret_cast<float*>(ws + pl.logits);
  int* status = reinterpret_cast<int*>(ws + pl.status);
  if (d.simt) {
    GS_TRY(gate_logits(d, x, wg, logits, status, st));
    launch_gate_rows(d, logits, expert_idx, gate12, rowmax, rowinv, st);
  } else {
    // on request: mean gates fused into the gating kernel (no stored logits) where a cluster covers
    // all experts
    if (d.gate_cluster && gate_cluster_supported(d)) {
      float* partial32 = reinterpret_cast<float*>(ws + pl.partial);
      const int rc = launch_gate_cluster(d, x, wg, expert_idx, gate12, rowmax, rowinv, partial32, status, st);
      if (rc == GSHARD_OK) {
        launch_gate_mean_blocks(d, partial32, d.S / 32, m, st);
        return GSHARD_OK;
      }
      if (rc != GSHARD_ERR_UNSUPPORTED_SHAPE) return rc;
    }
    if (!d.gate_one_sm && gate_fused2_supported(d) &&
        launch_gate_fused2(d, x, wg, logits, expert_idx, gate12, rowmax, rowinv, status, st) == GSHARD_OK) {
      // the pair kernel stores the logits as float4 [E/4][N]; its own column-sum pass follows.  (If
      // the cluster launch is refused, nothing ran and the one-SM kernel below takes over.)
      launch_gate_means_t(d, logits, rowmax, rowinv, reinterpret_cast<float*>(ws + pl.partial), m, st);
      return GSHARD_OK;
    } else
      GS_TRY(launch_gate_fused(d, x, wg, logits, expert_idx, gate12, rowmax, rowinv, status, st));
  }
  launch_gate_means(d, logits, rowmax, rowinv, reinterpret_cast<float*>(ws + pl.partial), m, st);
  return GSHARD_OK;
}

// h = relu(buf . wi), out = h . wo for every expert (eq. (2)); weights are read once.
bool ffn_runs_fused(const Dims& d, bool keep_h) {
  const bool want_fused = d.fused_ffn || (!d.unfused_ffn && d.rows <= 128);
  return !d.simt && want_fused && !keep_h && ffn_fused_supported(d);
}

// With x / slot_token (only where ffn_runs_fused) the rows are gathered from x and buf is not read.
int ffn_stage(const Dims& d, const void* buf, const void* wi, const void* wo, void* h, bool keep_h, void* out,
              void* fused_scratch, int* status, cudaStream_t st, const void* x, const int32_t* slot_token,
              void* wt, const int* tile_base, uint32_t* relu_bits_out) {
  NvtxRange range("gshard.expert_ffn");
  const long long rows = d.rows;
  // One persistent launch in which the hidden activations never leave L2: the faster form when
  // the FFN is bound by streaming the expert weights (at most one 128-row tile per expert); with
  // more rows per expert the two grouped-GEMM launches keep the tensor pipe busier.  Not available
  // when the caller keeps h for the backward pass.
  // The single-launch form needs its whole grid resident at once and is launched cooperatively; when
  // the runtime refuses that (GSHARD_ERR_UNSUPPORTED_SHAPE, nothing launched) the two grouped-GEMM
  // launches below take over.
  if (!tile_base && ffn_runs_fused(d, keep_h)) {
    const int rc = launch_ffn_fused(d, buf, wi, wo, fused_scratch, out, status, st, x, slot_token);
    if (rc != GSHARD_ERR_UNSUPPORTED_SHAPE) return rc;
    if (x) launch_dispatch(d, x, slot_token, const_cast<void*>(buf), st, status);   // rows were to be gathered in the launch
  }
  UmmaGemm g{};
  g.A = buf; g.B = wi; g.C = h; g.rows = d.rows; g.cols = d.H; g.K = d.M; g.batch = d.E;
  g.a_kmajor = true; g.b_kmajor = false;
  g.a_ld = d.M; g.a_bs = rows * d.M; g.b_ld = d.H; g.b_bs = (long long)d.M * d.H; g.c_ld = d.H; g.c_bs = rows * d.H;
  g.relu = 1; g.b_stream = 1; g.prefer_two_sm = 1;
  if (!d.simt) g.mask_bits_out = relu_bits_out;   // the backward's ReLU mask, one bit per hidden activation
  UmmaGemm g2{};
  g2.A = h; g2.B = wo; g2.C = out; g2.rows = d.rows; g2.cols = d.M; g2.K = d.H; g2.batch = d.E;
  g2.a_kmajor = true; g2.b_kmajor = false;
  g2.a_ld = d.H; g2.a_bs = rows * d.H; g2.b_ld = d.M; g2.b_bs = (long long)d.H * d.M; g2.c_ld = d.M; g2.c_bs = rows * d.M;
  g2.b_stream = 1; g2.prefer_two_sm = 1;
  // Compacted rows: each expert's row-tile count comes from the device-side prefixes.  Either 128-row
  // tiles on single CTAs throughout, or (hybrid) the kept rows in 256-row tiles on CTA pairs and the one
  // 128-row tile that may remain behind them on a single CTA, in a second launch of each GEMM.
  const bool hybrid = tile_base && !d.one_sm_mma && d.rows > 128 && !(d.tf32_experts && wt);
  const int* pair_base = tile_base ? tile_base + (d.E + 1) : nullptr;
  const int* single_base = tile_base ? tile_base + 2 * (d.E + 1) : nullptr;
  const int* owners = tile_base ? tile_base + 3 * (d.E + 1) : nullptr;      // three lists of compact_max_tiles(d)
  const int max_tiles = compact_max_tiles(d);
  if (tile_base && !hybrid) {
    g.tile_base = tile_base; g.tile_problem = owners; g.prefer_two_sm = 0;
    g2.tile_base = tile_base; g2.tile_problem = owners; g2.prefer_two_sm = 0;
  }
  if (hybrid) {
    for (const UmmaGemm& whole : {g, g2}) {
      UmmaGemm on_pairs = whole, rest = whole;
      on_pairs.tile_base = pair_base; on_pairs.tile_problem = owners + max_tiles; on_pairs.ragged_on_pairs = 1;
      rest.tile_base = single_base; rest.tile_problem = owners + 2 * max_tiles; rest.pair_base = pair_base;
      rest.prefer_two_sm = 0;
      if (run_gemm(d, on_pairs, status, st) != GSHARD_OK) {   // a refused cluster launch ran nothing
        rest.tile_base = tile_base; rest.tile_problem = owners; rest.pair_base = nullptr;   // all tiles on single CTAs
      }
      GS_TRY(run_gemm(d, rest, status, st));
    }
    return GSHARD_OK;
  }
  if (d.tf32_experts && wt) {
    // The tensor core reads 32-bit operands K-major only, and the weights are contiguous along the
    // other dimension: transposed copies first (wi[e] [M,H] -> [H,M], wo[e] [H,M] -> [M,H]).
    float* wi_t = static_cast<float*>(wt);
    float* wo_t = wi_t + (size_t)d.E * d.M * d.H;
    launch_transpose_f32(static_cast<const float*>(wi), wi_t, d.E, d.M, d.H, st);
    launch_transpose_f32(static_cast<const float*>(wo), wo_t, d.E, d.H, d.M, st);
    g.B = wi_t; g.b_kmajor = true; g.b_ld = d.M; g.tf32 = 1; g.out_f32 = 1;
    g2.B = wo_t; g2.b_kmajor = true; g2.b_ld = d.H; g2.tf32 = 1; g2.out_f32 = 1;
  }
  GS_TRY(run_gemm(d, g, status, st));
  return run_gemm(d, g2, status, st);
}

int validate_shape(const gshard_moe_shape* s) {
  if (!s) return GSHARD_ERR_INVALID_ARG;
  if (s->G <= 0 || s->S <= 0 || s->M <= 0 || s->H <= 0 || s->E <= 0 || s->C <= 0) return GSHARD_ERR_INVALID_ARG;
  if (s->dtype != GSHARD_F32 && s->dtype != GSHARD_BF16) return GSHARD_ERR_INVALID_ARG;
  if (s->flags & ~GSHARD_FLAG_ALL) return GSHARD_ERR_INVALID_ARG;
  if ((s->flags & GSHARD_FLAG_FUSED_FFN) && (s->flags & GSHARD_FLAG_UNFUSED_FFN)) return GSHARD_ERR_INVALID_ARG;
  if (s->E < 2) return GSHARD_ERR_INVALID_ARG;
  if (s->M % 8 || s->H % 8) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  if (s->S > 32767 || s->E > 16384 || s->C > 32767) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  if ((long long)s->G * s->S > (1ll << 30) || (long long)s->E * s->G * s->C > (1ll << 30)) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  if (capacity_warps_for(s->E) == 0) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  // grid limits of the launches: the column-sum kernels index (group, 128-token tile) and the
  // group-level kernels the group through gridDim.y; the CUDA-core GEMM its 64-row tiles
  if ((long long)s->G * ((s->S + kGateTile - 1) / kGateTile) > 65535) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  if (((long long)s->G * s->S + 63) / 64 > 65535 && (s->dtype == GSHARD_F32 || (s->flags & GSHARD_FLAG_SIMT_CONTRACTIONS)))
    return GSHARD_ERR_UNSUPPORTED_SHAPE;
  // a tensor map's strides stay below 2^40 bytes
  if ((long long)s->G * s->S * std::max(s->M, s->E) >= (1ll << 37)) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  if ((long long)s->G * s->C * s->H >= (1ll << 37)) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  const bool umma = s->dtype == GSHARD_BF16 && !(s->flags & GSHARD_FLAG_SIMT_CONTRACTIONS);
  if (umma && (s->M % 64 || s->H % 64 || s->E % 16)) return GSHARD_ERR_UNSUPPORTED_SHAPE;
  return GSHARD_OK;
}

// The forward launch sequence on device buffers.
int forward_device(const gshard_moe_shape* shape, const void* x, const void* wg, const void* wi, const void* wo,
                   const float* u, void* y, float* l_aux, const gshard_moe_routing* ro, void* context,
                   void* workspace, size_t workspace_bytes, cudaStream_t st) {
  const Dims d = make_dims(*shape);
  const FwdPlan pl = plan_forward(d);
  if (workspace_bytes < pl.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  const bool save = (shape->flags & GSHARD_FLAG_SAVE_FOR_BACKWARD) != 0;
  if (save && (!context || reinterpret_cast<uintptr_t>(context) % kAlign)) return GSHARD_ERR_INVALID_ARG;
  unsigned char* ctx = static_cast<unsigned char*>(context);
  const CtxPlan cp = plan_context(d);
  gshard_moe_routing r{};
  if (ro) r = *ro;
  int* status = reinterpret_cast<int*>(ws + pl.status);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;

  // with SAVE_FOR_BACKWARD the small routing tensors and the big activations live in the context
  int32_t* expert_idx = save ? reinterpret_cast<int32_t*>(ctx + cp.expert_idx) : pick(r.expert_idx, ws, pl.expert_idx);
  int32_t* slot = save ? reinterpret_cast<int32_t*>(ctx + cp.slot) : pick(r.slot, ws, pl.slot);
  float* weight = save ? reinterpret_cast<float*>(ctx + cp.weight) : pick(r.weight, ws, pl.weight);
  int32_t* first_count = save ? reinterpret_cast<int32_t*>(ctx + cp.first_count) : pick(r.first_count, ws, pl.first_count);
  int32_t* slot_token = save ? reinterpret_cast<int32_t*>(ctx + cp.slot_token) : pick(r.slot_token, ws, pl.slot_token);
  float* gate12 = save ? reinterpret_cast<float*>(ctx + cp.gate12) : reinterpret_cast<float*>(ws + pl.gate12);
  float* rowmax = save ? reinterpret_cast<float*>(ctx + cp.rowmax) : reinterpret_cast<float*>(ws + pl.rowmax);
  float* rowinv = save ? reinterpret_cast<float*>(ctx + cp.rowinv) : reinterpret_cast<float*>(ws + pl.rowinv);
  void* h = save ? static_cast<void*>(ctx + cp.h) : static_cast<void*>(ws + pl.h);
  void* out = save ? static_cast<void*>(ctx + cp.out) : static_cast<void*>(ws + pl.out);
  uint8_t* flags = pick(r.flags, ws, pl.flags);
  int32_t* total_count = pick(r.total_count, ws, pl.total_count);
  float* m = pick(r.m, ws, pl.m);
  float* l_aux_group = pick(r.l_aux_group, ws, pl.l_aux_group);
  int32_t* stats_group = reinterpret_cast<int32_t*>(ws + pl.stats_group);
  void* buf = save ? static_cast<void*>(ctx + cp.buf) : static_cast<void*>(ws + pl.buf);

  GS_TRY(gate_stage(d, pl, ws, x, wg, expert_idx, gate12, m, rowmax, rowinv, st));
  GS_TRY(launch_capacity(d, expert_idx, gate12, u, m, slot, weight, flags, first_count, total_count, slot_token,
                         l_aux_group, stats_group, l_aux, reinterpret_cast<long long*>(r.stats), st));
  if (d.debug_checks) launch_routing_check(d, expert_idx, slot, weight, flags, slot_token, status, st);
  const bool gather = d.gather_dispatch && ffn_runs_fused(d, save);
  // compacted slots apply to the grouped-GEMM form of the FFN only
  const bool compact = d.compact_slots && !ffn_runs_fused(d, save);
  int32_t* crow_token = reinterpret_cast<int32_t*>(ws + pl.crow_token);
  int32_t* slot_crow = reinterpret_cast<int32_t*>(ws + pl.slot_crow);
  int32_t* kept = reinterpret_cast<int32_t*>(ws + pl.kept);
  int32_t* tile_base = reinterpret_cast<int32_t*>(ws + pl.tile_base);
  if (compact) {
    launch_compact(d, slot_token, crow_token, slot_crow, kept, tile_base, st);
    launch_dispatch_compact(d, x, crow_token, kept, buf, st);
  } else if (!gather) {
    launch_dispatch(d, x, slot_token, buf, st, status);
  }
  // optional event pair around the expert FFN, armed for one call by gshard_moe_time_expert_ffn
  FfnTiming& ft = ffn_timing();
  const bool timed = ft.start != nullptr && ft.stop != nullptr;
  if (timed && cudaEventRecord(static_cast<cudaEvent_t>(ft.start), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  GS_TRY(ffn_stage(d, buf, wi, wo, h, save, out, ws + pl.ffn_scratch, status, st, gather ? x : nullptr, slot_token,
                   ws + pl.wt, compact ? tile_base : nullptr,
                   (save && !d.simt) ? reinterpret_cast<uint32_t*>(ctx + cp.hbits) : nullptr));
  if (timed && cudaEventRecord(static_cast<cudaEvent_t>(ft.stop), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  ft.start = ft.stop = nullptr;
  launch_combine(d, out, expert_idx, slot, weight, y, st, d.add_residual ? x : nullptr, compact ? slot_crow : nullptr);

  if (save) {   // hand the caller the routing tensors it asked for
    struct { void* dst; const void* src; size_t n; } cps[] = {
        {r.expert_idx, expert_idx, (size_t)d.N * 2 * 4}, {r.slot, slot, (size_t)d.N * 2 * 4},
        {r.weight, weight, (size_t)d.N * 2 * 4},         {r.first_count, first_count, (size_t)d.G * d.E * 4},
        {r.slot_token, slot_token, (size_t)d.R * 4}};
    for (auto& c : cps)
      if (c.dst && cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int backward_device(const gshard_moe_shape* shape, const void* x, const void* wg, const void* wi, const void* wo,
                    const void* context, const void* dy, float k_aux, void* dx, float* dwg, void* dwi, void* dwo,
                    void* workspace, size_t workspace_bytes, cudaStream_t st);

}  // namespace gshard

using namespace gshard;

extern "C" {

int gshard_version(void) { return 210; }

const char* gshard_status_string(int s) {
  switch (s) {
    case GSHARD_OK: return "ok";
    case GSHARD_ERR_INVALID_ARG: return "invalid argument";
    case GSHARD_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case GSHARD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case GSHARD_ERR_CUDA: return "CUDA error";
    case GSHARD_ERR_ARCH: return "device is not sm_100";
    case GSHARD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case GSHARD_ERR_INTERNAL: return "internal error";
    default: return "unknown status";
  }
}

size_t gshard_moe_top2_workspace_bytes(const gshard_moe_shape* shape, int for_backward) {
  if (validate_shape(shape) != GSHARD_OK) return 0;
  const Dims d = make_dims(*shape);
  return for_backward ? plan_backward(d).total : plan_forward(d).total;
}

size_t gshard_moe_top2_context_bytes(const gshard_moe_shape* shape) {
  if (validate_shape(shape) != GSHARD_OK) return 0;
  return plan_context(make_dims(*shape)).total;
}

size_t gshard_moe_top2_host_staging_bytes(const gshard_moe_shape* shape) {
  if (validate_shape(shape) != GSHARD_OK) return 0;
  return plan_staging(make_dims(*shape)).total;
}

int gshard_moe_top2_forward(const gshard_moe_shape* shape, const void* x, const void* wg, const void* wi,
                            const void* wo, const float* u, void* y, float* l_aux,
                            const gshard_moe_routing* routing_out, void* context, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(x); GS_REQUIRE_PTR(wg); GS_REQUIRE_PTR(wi); GS_REQUIRE_PTR(wo); GS_REQUIRE_PTR(u);
  GS_REQUIRE_PTR(y); GS_REQUIRE_PTR(workspace);
  if (l_aux == nullptr) return GSHARD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  if (workspace_bytes < gshard_moe_top2_workspace_bytes(shape, 0)) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  return forward_device(shape, x, wg, wi, wo, u, y, l_aux, routing_out, context, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(cuda_stream));
}

int gshard_moe_top2_forward_host(const gshard_moe_shape* shape, const void* x_host, const void* wg, const void* wi,
                                 const void* wo, const float* u_host, void* y_host, float* l_aux_host,
                                 const gshard_moe_routing* routing_out, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  if (!x_host || !u_host || !y_host || !l_aux_host) return GSHARD_ERR_INVALID_ARG;
  GS_REQUIRE_PTR(wg); GS_REQUIRE_PTR(wi); GS_REQUIRE_PTR(wo); GS_REQUIRE_PTR(workspace);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  if (shape->flags & GSHARD_FLAG_SAVE_FOR_BACKWARD) return GSHARD_ERR_INVALID_ARG;
  const Dims d = make_dims(*shape);
  const size_t fwd = plan_forward(d).total;
  const StagePlan sp = plan_staging(d);
  if (workspace_bytes < fwd + sp.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* stg = static_cast<unsigned char*>(workspace) + fwd;
  void* xd = stg + sp.x; float* ud = reinterpret_cast<float*>(stg + sp.u);
  void* yd = stg + sp.y; float* ld = reinterpret_cast<float*>(stg + sp.l_aux);
  const size_t act_bytes = (size_t)d.N * d.M * d.esize;
  if (cudaMemcpyAsync(xd, x_host, act_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  if (cudaMemcpyAsync(ud, u_host, (size_t)d.N * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  GS_TRY(forward_device(shape, xd, wg, wi, wo, ud, yd, ld, routing_out, nullptr, workspace, fwd, st));
  if (cudaMemcpyAsync(y_host, yd, act_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  if (cudaMemcpyAsync(l_aux_host, ld, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GSHARD_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return GSHARD_ERR_CUDA;
  int status = 0;
  if (cudaMemcpy(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return GSHARD_ERR_CUDA;
  return status;
}

int gshard_moe_top2_forward_host_async(const gshard_moe_shape* shape, const void* x_host, const void* wg,
                                       const void* wi, const void* wo, const float* u_host, void* y_host,
                                       float* l_aux_host, const gshard_moe_routing* routing_out, void* workspace,
                                       size_t workspace_bytes, void* staging, size_t staging_bytes,
                                       void* copy_in_stream, void* compute_stream, void* copy_out_stream,
                                       void* ev_in, void* ev_done, void* ev_out) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  if (!x_host || !u_host || !y_host || !l_aux_host || !ev_in || !ev_done || !ev_out) return GSHARD_ERR_INVALID_ARG;
  GS_REQUIRE_PTR(wg); GS_REQUIRE_PTR(wi); GS_REQUIRE_PTR(wo); GS_REQUIRE_PTR(workspace); GS_REQUIRE_PTR(staging);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign || reinterpret_cast<uintptr_t>(staging) % kAlign)
    return GSHARD_ERR_INVALID_ARG;
  if (shape->flags & GSHARD_FLAG_SAVE_FOR_BACKWARD) return GSHARD_ERR_INVALID_ARG;
  const Dims d = make_dims(*shape);
  const size_t fwd = plan_forward(d).total;
  const StagePlan sp = plan_staging(d);
  if (workspace_bytes < fwd || staging_bytes < sp.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  cudaStream_t s_in = static_cast<cudaStream_t>(copy_in_stream);
  cudaStream_t s_cmp = static_cast<cudaStream_t>(compute_stream);
  cudaStream_t s_out = static_cast<cudaStream_t>(copy_out_stream);
  cudaEvent_t e_in = static_cast<cudaEvent_t>(ev_in), e_done = static_cast<cudaEvent_t>(ev_done),
              e_out = static_cast<cudaEvent_t>(ev_out);
  unsigned char* stg = static_cast<unsigned char*>(staging);
  void* xd = stg + sp.x; float* ud = reinterpret_cast<float*>(stg + sp.u);
  void* yd = stg + sp.y; float* ld = reinterpret_cast<float*>(stg + sp.l_aux);
  const size_t act_bytes = (size_t)d.N * d.M * d.esize;
#define GS_CUDA(call) do { if ((call) != cudaSuccess) return GSHARD_ERR_CUDA; } while (0)
  // inputs of this slot may be overwritten once the previous forward that used the slot has run
  GS_CUDA(cudaStreamWaitEvent(s_in, e_done, 0));
  GS_CUDA(cudaMemcpyAsync(xd, x_host, act_bytes, cudaMemcpyHostToDevice, s_in));
  GS_CUDA(cudaMemcpyAsync(ud, u_host, (size_t)d.N * 4, cudaMemcpyHostToDevice, s_in));
  GS_CUDA(cudaEventRecord(e_in, s_in));
  // the forward needs this slot's inputs, and its previous outputs must have left the device
  GS_CUDA(cudaStreamWaitEvent(s_cmp, e_in, 0));
  GS_CUDA(cudaStreamWaitEvent(s_cmp, e_out, 0));
  GS_TRY(forward_device(shape, xd, wg, wi, wo, ud, yd, ld, routing_out, nullptr, workspace, fwd, s_cmp));
  GS_CUDA(cudaEventRecord(e_done, s_cmp));
  GS_CUDA(cudaStreamWaitEvent(s_out, e_done, 0));
  GS_CUDA(cudaMemcpyAsync(y_host, yd, act_bytes, cudaMemcpyDeviceToHost, s_out));
  GS_CUDA(cudaMemcpyAsync(l_aux_host, ld, 4, cudaMemcpyDeviceToHost, s_out));
  GS_CUDA(cudaEventRecord(e_out, s_out));
#undef GS_CUDA
  return GSHARD_OK;
}

int gshard_moe_top2_backward(const gshard_moe_shape* shape, const void* x, const void* wg, const void* wi,
                             const void* wo, const void* context, const void* dy, float l_aux_weight, void* dx,
                             float* dwg, void* dwi, void* dwo, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(x); GS_REQUIRE_PTR(wg); GS_REQUIRE_PTR(wi); GS_REQUIRE_PTR(wo); GS_REQUIRE_PTR(context);
  GS_REQUIRE_PTR(dy); GS_REQUIRE_PTR(dx); GS_REQUIRE_PTR(dwg); GS_REQUIRE_PTR(dwi); GS_REQUIRE_PTR(dwo);
  GS_REQUIRE_PTR(workspace);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign || reinterpret_cast<uintptr_t>(context) % kAlign)
    return GSHARD_ERR_INVALID_ARG;
  if (workspace_bytes < gshard_moe_top2_workspace_bytes(shape, 1)) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  return backward_device(shape, x, wg, wi, wo, context, dy, l_aux_weight, dx, dwg, dwi, dwo, workspace,
                         workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int gshard_moe_gate(const gshard_moe_shape* shape, const void* x, const void* wg, int32_t* expert_idx,
                    float* gate12, float* m, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(x); GS_REQUIRE_PTR(wg); GS_REQUIRE_PTR(expert_idx); GS_REQUIRE_PTR(gate12); GS_REQUIRE_PTR(m);
  GS_REQUIRE_PTR(workspace);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  const Dims d = make_dims(*shape);
  const FwdPlan pl = plan_forward(d);
  if (workspace_bytes < pl.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  if (cudaMemsetAsync(ws + pl.status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  GS_TRY(gate_stage(d, pl, ws, x, wg, expert_idx, gate12, m, reinterpret_cast<float*>(ws + pl.rowmax),
                    reinterpret_cast<float*>(ws + pl.rowinv), st));
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int gshard_moe_capacity(const gshard_moe_shape* shape, const int32_t* expert_idx, const float* gate12,
                        const float* u, const float* m, const gshard_moe_routing* ro, float* l_aux,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(expert_idx); GS_REQUIRE_PTR(gate12); GS_REQUIRE_PTR(u); GS_REQUIRE_PTR(m);
  GS_REQUIRE_PTR(workspace);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  const Dims d = make_dims(*shape);
  const FwdPlan pl = plan_forward(d);
  if (workspace_bytes < pl.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  gshard_moe_routing r{};
  if (ro) r = *ro;
  return launch_capacity(d, expert_idx, gate12, u, m, pick(r.slot, ws, pl.slot), pick(r.weight, ws, pl.weight),
                         pick(r.flags, ws, pl.flags), pick(r.first_count, ws, pl.first_count),
                         pick(r.total_count, ws, pl.total_count), pick(r.slot_token, ws, pl.slot_token),
                         pick(r.l_aux_group, ws, pl.l_aux_group), reinterpret_cast<int32_t*>(ws + pl.stats_group),
                         l_aux, reinterpret_cast<long long*>(r.stats), static_cast<cudaStream_t>(cuda_stream));
}

int gshard_moe_dispatch(const gshard_moe_shape* shape, const void* x, const int32_t* slot_token, void* buf,
                        void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(x); GS_REQUIRE_PTR(slot_token); GS_REQUIRE_PTR(buf);
  GS_TRY(check_device());
  launch_dispatch(make_dims(*shape), x, slot_token, buf, static_cast<cudaStream_t>(cuda_stream));
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int gshard_moe_expert_ffn(const gshard_moe_shape* shape, const void* buf, const void* wi, const void* wo,
                          void* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(buf); GS_REQUIRE_PTR(wi); GS_REQUIRE_PTR(wo); GS_REQUIRE_PTR(out); GS_REQUIRE_PTR(workspace);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  const Dims d = make_dims(*shape);
  const FwdPlan pl = plan_forward(d);
  if (workspace_bytes < pl.total) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  if (cudaMemsetAsync(ws + pl.status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  GS_TRY(ffn_stage(d, buf, wi, wo, ws + pl.h, false, out, ws + pl.ffn_scratch,
                   reinterpret_cast<int*>(ws + pl.status), st, nullptr, nullptr, ws + pl.wt));
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int gshard_moe_combine(const gshard_moe_shape* shape, const void* out, const int32_t* expert_idx,
                       const int32_t* slot, const float* weight, void* y, void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  GS_REQUIRE_PTR(out); GS_REQUIRE_PTR(expert_idx); GS_REQUIRE_PTR(slot); GS_REQUIRE_PTR(weight); GS_REQUIRE_PTR(y);
  GS_TRY(check_device());
  launch_combine(make_dims(*shape), out, expert_idx, slot, weight, y, static_cast<cudaStream_t>(cuda_stream));
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

size_t gshard_dense_ffn_workspace_bytes(int64_t n_tokens, int32_t M, int32_t H, int32_t dtype) {
  if (n_tokens <= 0 || n_tokens > (1ll << 30) || M <= 0 || H <= 0 || M % 8 || H % 8) return 0;
  if (dtype != GSHARD_F32 && dtype != GSHARD_BF16) return 0;
  if (dtype == GSHARD_BF16 && (M % 64 || H % 64)) return 0;
  if (dtype == GSHARD_F32 && (n_tokens + 63) / 64 > 65535) return 0;
  // status word, hidden activations, and (fp32, for the TF32 option) the transposed weights
  return kAlign + align_up((size_t)n_tokens * H * (dtype == GSHARD_BF16 ? 2 : 4)) +
         (dtype == GSHARD_F32 ? align_up(2 * (size_t)M * H * 4) : 0);
}

int gshard_dense_ffn_forward(int64_t n_tokens, int32_t M, int32_t H, int32_t dtype, uint32_t flags, const void* x,
                             const void* wi, const void* wo, void* y, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
  launch_counter().n = 0;
  if (flags & ~(GSHARD_FLAG_TF32_EXPERTS | GSHARD_FLAG_ONE_SM_MMA | GSHARD_FLAG_SIMT_CONTRACTIONS))
    return GSHARD_ERR_INVALID_ARG;
  const size_t need = gshard_dense_ffn_workspace_bytes(n_tokens, M, H, dtype);
  if (need == 0) return (n_tokens <= 0 || M <= 0 || H <= 0) ? GSHARD_ERR_INVALID_ARG : GSHARD_ERR_UNSUPPORTED_SHAPE;
  GS_REQUIRE_PTR(x); GS_REQUIRE_PTR(wi); GS_REQUIRE_PTR(wo); GS_REQUIRE_PTR(y); GS_REQUIRE_PTR(workspace);
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  if (workspace_bytes < need) return GSHARD_ERR_WORKSPACE_TOO_SMALL;
  GS_TRY(check_device());
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int* status = reinterpret_cast<int*>(ws);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  // the expert FFN's two grouped GEMMs with a single problem of n_tokens rows
  gshard_moe_shape one{};
  one.G = 1; one.S = 1; one.C = 1; one.E = 2; one.M = M; one.H = H; one.dtype = dtype; one.flags = flags;
  Dims d = make_dims(one);
  d.rows = (int)n_tokens;
  void* h = ws + kAlign;
  UmmaGemm g{};
  g.A = x; g.B = wi; g.C = h; g.rows = d.rows; g.cols = H; g.K = M; g.batch = 1;
  g.a_kmajor = true; g.b_kmajor = false; g.a_ld = M; g.b_ld = H; g.c_ld = H;
  g.relu = 1; g.a_stream = 1; g.prefer_two_sm = 1;
  UmmaGemm g2{};
  g2.A = h; g2.B = wo; g2.C = y; g2.rows = d.rows; g2.cols = M; g2.K = H; g2.batch = 1;
  g2.a_kmajor = true; g2.b_kmajor = false; g2.a_ld = H; g2.b_ld = M; g2.c_ld = M;
  g2.a_stream = 1; g2.prefer_two_sm = 1;
  if (d.tf32_experts) {          // K-major (transposed) copies of the weights, as in the expert FFN
    float* wi_t = reinterpret_cast<float*>(ws + kAlign + align_up((size_t)n_tokens * H * 4));
    float* wo_t = wi_t + (size_t)M * H;
    launch_transpose_f32(static_cast<const float*>(wi), wi_t, 1, M, H, st);
    launch_transpose_f32(static_cast<const float*>(wo), wo_t, 1, H, M, st);
    g.B = wi_t; g.b_kmajor = true; g.b_ld = M; g.tf32 = 1; g.out_f32 = 1;
    g2.B = wo_t; g2.b_kmajor = true; g2.b_ld = H; g2.tf32 = 1; g2.out_f32 = 1;
  }
  GS_TRY(run_gemm(d, g, status, st));
  GS_TRY(run_gemm(d, g2, status, st));
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int gshard_moe_last_device_status(void* workspace, void* cuda_stream) {
  if (!workspace) return GSHARD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return GSHARD_ERR_CUDA;
  int status = 0;
  if (cudaMemcpy(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return GSHARD_ERR_CUDA;
  return status;
}

int gshard_moe_check_routing(const gshard_moe_shape* shape, const gshard_moe_routing* routing, void* workspace,
                             void* cuda_stream) {
  launch_counter().n = 0;
  GS_TRY(validate_shape(shape));
  if (!routing || !workspace || reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  GS_REQUIRE_PTR(routing->expert_idx); GS_REQUIRE_PTR(routing->slot); GS_REQUIRE_PTR(routing->weight);
  GS_REQUIRE_PTR(routing->flags); GS_REQUIRE_PTR(routing->slot_token);
  GS_TRY(check_device());
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int* status = static_cast<int*>(workspace);
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  launch_routing_check(make_dims(*shape), routing->expert_idx, routing->slot, routing->weight, routing->flags,
                       routing->slot_token, status, st);
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}

int gshard_moe_last_launch_count(void) { return launch_counter().n; }

int gshard_moe_time_expert_ffn(void* start_event, void* stop_event) {
  if ((start_event == nullptr) != (stop_event == nullptr)) return GSHARD_ERR_INVALID_ARG;
  ffn_timing().start = start_event;
  ffn_timing().stop = stop_event;
  return GSHARD_OK;
}

}  // extern "C"
