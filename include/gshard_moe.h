/*
 * gshard_moe.h - C ABI of the B200 (sm_100a) top-2 gated Mixture-of-Experts FFN layer.
 *
 * The layer is the one defined by the GShard paper (arxiv 2006.16668):
 *   eq. (1)-(3)   y_s = sum_e G_{s,e} * FFN_e(x_s),  FFN_e(x) = wo_e . ReLU(wi_e . x), no bias
 *   Algorithm 1   group-level top-2 gating: softmax gates, mean gates m_e, first-choice
 *                 loop, auxiliary loss l_aux = (1/E) sum_e (c_e/S) m_e, second-choice loop
 *                 with random routing (keep iff c < C and 2*g2 > rnd)
 *   Algorithm 2   tensor layouts: inputs [G,S,M], wg [M,E], wi [E,M,H], wo [E,H,M],
 *                 dispatched expert inputs [E,G,C,M], outputs [G,S,M]
 *
 * Conventions for every call
 *   - All tensor arguments are DEVICE pointers unless the name ends in _host; tensors are
 *     contiguous, row-major, 16-byte aligned, owned by the caller.  The library allocates no
 *     device memory: scratch comes from the caller's `workspace`.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default
 *     stream) and the call returns without synchronising, except the *_host calls and
 *     gshard_moe_last_device_status.
 *   - Return value: a gshard_status.  Errors that the host can detect (null or misaligned
 *     pointer, non-positive size, unsupported shape, short workspace, device that is not
 *     sm_100) launch nothing.  Anomalies seen on the device (a bounded wait that ran out)
 *     set a status word in the workspace, never trap, and are read back with
 *     gshard_moe_last_device_status.
 *   - dtype GSHARD_F32: x, wg, wi, wo, y (and dy, dx, dwi, dwo) are float; all arithmetic is
 *     fp32 on CUDA cores.  dtype GSHARD_BF16: they are bfloat16; contractions run on the
 *     tcgen05 tensor cores with fp32 accumulation; softmax, top-2, weights, l_aux are fp32.
 *     u, l_aux, weight, m, dwg are always float.
 *   - Outputs are bit-reproducible from run to run (no atomics in any reduction).
 *   - Every stage's launches sit inside an NVTX range (gshard.gate, .capacity, .dispatch,
 *     .expert_ffn, .combine, .backward.*), visible to a profiler that injects NVTX.
 */
#ifndef GSHARD_MOE_H_
#define GSHARD_MOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GSHARD_OK = 0,
  GSHARD_ERR_INVALID_ARG = 1,
  GSHARD_ERR_UNSUPPORTED_SHAPE = 2,
  GSHARD_ERR_WORKSPACE_TOO_SMALL = 3,
  GSHARD_ERR_CUDA = 4,
  GSHARD_ERR_ARCH = 5,
  GSHARD_ERR_TIMEOUT = 6,
  GSHARD_ERR_INTERNAL = 7
} gshard_status;

typedef enum { GSHARD_F32 = 0, GSHARD_BF16 = 1 } gshard_dtype;

/* flags of gshard_moe_shape.  Bits 1, 2, 1024 and 8192 change what is computed or kept (saved context,
 * reading of the second loop, residual, TF32); the others choose between kernel forms of the bf16
 * tensor-core path or add checks; the defaults are the forms that measured fastest on B200, results
 * agree within the stated tolerances whichever form runs. */
#define GSHARD_FLAG_SAVE_FOR_BACKWARD 1u      /* forward fills `context` for the backward call */
#define GSHARD_FLAG_SECOND_SKIP_FREES_SLOT 2u /* other reading of Algorithm 1's second loop: a token
                                                 that fails 2*g2 > rnd does not advance the counter
                                                 of its second expert */
#define GSHARD_FLAG_SIMT_CONTRACTIONS 4u      /* bf16 only: run every contraction on CUDA cores (fp32
                                                 FMA) instead of tcgen05; for debugging */
#define GSHARD_FLAG_FUSED_FFN 8u              /* force the single-launch expert FFN (hidden activations
                                                 handed over through L2, never written to HBM) where
                                                 the shape allows it; by default it is used when an
                                                 expert has at most 128 rows */
/* The single-launch form (FUSED_FFN and its GATHER_DISPATCH mode) is a persistent grid whose CTAs
 * wait on one another, one CTA per multiprocessor.  It is launched cooperatively: the runtime
 * starts it only when the whole grid can be resident, so work of other streams that holds
 * multiprocessors delays it instead of breaking it; if the runtime refuses the launch, the two
 * grouped-GEMM launches run instead. */
#define GSHARD_FLAG_UNFUSED_FFN 16u           /* force the two grouped-GEMM launches instead (hidden
                                                 activations make a round trip through HBM) */
#define GSHARD_FLAG_TWO_SM_MMA 32u            /* every grouped GEMM with more than 128 rows per problem
                                                 runs on CTA pairs (tcgen05 cta_group::2, 256 x 256
                                                 tiles); by default the forward expert GEMMs and two
                                                 of the backward ones (dh, dbuf) do */
#define GSHARD_FLAG_GATHER_DISPATCH 64u       /* forward with the single-launch expert FFN: a warp of
                                                 every CTA gathers the next experts' token rows from x
                                                 by the slot index list into an L2-resident buffer while
                                                 the GEMMs run, and the [E, G*C, M] dispatch buffer of
                                                 Algorithm 2 is not written; ignored where that FFN
                                                 form is not in use */
#define GSHARD_FLAG_GATE_CLUSTER 128u         /* gating with the mean gates' partial sums fused in: a
                                                 thread-block cluster holds all E logits of a token
                                                 tile in tensor memory and exchanges the softmax
                                                 statistics through distributed shared memory, so no
                                                 logits are stored (needs E <= 2048, S % 32 == 0;
                                                 elsewhere ignored).  Default: logits stored once,
                                                 column sums in a second pass */
#define GSHARD_FLAG_GATE_ONE_SM 256u          /* gating GEMM on single CTAs with row-major stored
                                                 logits.  By default, where E % 128 == 0, it runs on CTA
                                                 pairs (each CTA loads half of the wg tile) and stores
                                                 the logits in 16-byte granules laid out [E/4][N] */
#define GSHARD_FLAG_ONE_SM_MMA 512u           /* no grouped GEMM runs on CTA pairs (128 x 256 tiles on
                                                 single CTAs everywhere) */
#define GSHARD_FLAG_ADD_RESIDUAL 1024u        /* forward: y = x + layer(x), the residual connection
                                                 around the layer (section 2.2, expert capacity:
                                                 overflowed tokens pass through it) folded into the
                                                 combine; backward: dx also receives dy.  Not applied
                                                 by the stage call gshard_moe_combine */
#define GSHARD_FLAG_PLAIN_STORES 2048u        /* the grouped GEMMs write their output tiles with 16-byte
                                                 stores from the epilogue warps instead of bulk tensor
                                                 (TMA) stores out of the staging rows; same bits, for
                                                 comparisons */
#define GSHARD_FLAG_BWD_PAIRED_GEMMS 4096u    /* backward: the GEMM that computes dh runs beside the one
                                                 for dwo, and dbuf beside dwi, each on half of the
                                                 multiprocessors (second, library-owned stream), so
                                                 that HBM sees reads and writes mixed.  Measured
                                                 slower than the default (one after another on all
                                                 multiprocessors); kept for measurement */
#define GSHARD_FLAG_TF32_EXPERTS 8192u        /* dtype GSHARD_F32 only (ignored for bf16): the two expert
                                                 FFN contractions of the forward run on the tensor cores
                                                 with the fp32 operands read as TF32 (10-bit mantissa,
                                                 fp32 accumulation), the way the paper's float32
                                                 training would run on this hardware; gating, softmax,
                                                 top-2 and the combine stay exact fp32, so the routing
                                                 does not change.  y then agrees with the fp32 result to
                                                 about 1e-3 relative instead of 1e-6.  The tensor core
                                                 reads 32-bit operands only when they are contiguous
                                                 along the contraction, which wi [E,M,H] and wo [E,H,M]
                                                 are not: each call first writes transposed copies of
                                                 both into the workspace (its size grows by their
                                                 size) */
#define GSHARD_FLAG_COMPACT_SLOTS 16384u      /* forward, bf16, grouped-GEMM form of the expert FFN
                                                 (more than 128 rows per expert): the filled slots of
                                                 each expert are compacted to the front of its block,
                                                 the GEMMs run only the row tiles that hold kept rows
                                                 (13 to 30 % of the slots are empty at the paper's
                                                 shapes: 256-row tiles on CTA pairs, then at most one
                                                 128-row tile on a single CTA; with ONE_SM_MMA 128-row
                                                 tiles throughout), empty rows are neither zero-filled
                                                 nor multiplied, and the combine finds its rows through
                                                 the compaction index.  Kept rows get the same bits.
                                                 This is the default for that form of the FFN unless
                                                 ONE_SM_MMA, TWO_SM_MMA or FUSED_FFN names another;
                                                 the flag then adds it back.  Ignored with
                                                 SAVE_FOR_BACKWARD and where the single-launch FFN
                                                 runs */
#define GSHARD_FLAG_DEBUG_CHECKS 32768u       /* forward: after the capacity stage a kernel verifies the
                                                 routing tensors (expert ids, positions, flags, weights,
                                                 the inverse slot list; every access bounds-checked) and
                                                 records GSHARD_ERR_INTERNAL in the status word on a
                                                 violation - nothing traps */
#define GSHARD_FLAG_BULK_DISPATCH 65536u      /* dispatch: token rows move through the TMA unit (bulk
                                                 global->shared->global copies, empty slots as bulk
                                                 stores of a zero row) instead of 16-byte loads and
                                                 stores; same bytes.  Applies to the dispatch into the
                                                 full [E, G*C, M] buffer (gshard_moe_dispatch, the
                                                 single-launch FFN, SAVE_FOR_BACKWARD), not to the
                                                 dispatch into compacted rows */
#define GSHARD_FLAG_ALL 131071u

/* G groups of S tokens, model dim M, expert hidden dim H, E experts, per-group capacity C
 * (Algorithm 1 "Data"; the paper sets C = 2N/(G*E) = 2S/E).  Limits: M % 8 == 0, H % 8 == 0,
 * E >= 2, S <= 32767, C <= 32767, E <= 16384; dtype BF16 without SIMT flag also needs M % 64 == 0,
 * H % 64 == 0, E % 16 == 0. */
typedef struct {
  int32_t G, S, M, H, E, C;
  int32_t dtype;   /* gshard_dtype */
  uint32_t flags;
} gshard_moe_shape;

/* Compact routing result (the non-zeros of Algorithm 2's combine_weights [G,S,E,C] and
 * dispatch_mask).  Device pointers, caller-allocated; any may be NULL to skip that output. */
typedef struct {
  int32_t* expert_idx;   /* [G,S,2]  e1, e2 (Algorithm 1 top_2)                              */
  int32_t* slot;         /* [G,S,2]  buffer position c in [0,C) or -1 when not dispatched     */
  float* weight;         /* [G,S,2]  g1/(g1+g2), g2/(g1+g2) (normalised values, kept or not) */
  uint8_t* flags;        /* [G,S]    bit0 first kept, bit1 2*g2>rnd passed, bit2 second kept  */
  int32_t* first_count;  /* [G,E]    c_e after the first loop (unclipped; enters l_aux)       */
  int32_t* total_count;  /* [G,E]    c_e after the second loop                                */
  int32_t* slot_token;   /* [E,G,C]  token index s within the group, or -1 for an empty slot  */
  float* m;              /* [G,E]    mean gates m_e                                           */
  float* l_aux_group;    /* [G]      Algorithm 1's per-group l_aux                            */
  int64_t* stats;        /* [8] 0 first choices dropped, 1 second choices that failed the
                                random test, 2 second choices that passed but found no room,
                                3 tokens with both choices dropped, 4 slots filled, 5..7 zero */
} gshard_moe_routing;

int gshard_version(void);
const char* gshard_status_string(int status);

/* Scratch sizes in bytes for a shape.  for_backward != 0 gives the size the backward call
 * needs.  Returns 0 for an invalid or unsupported shape. */
size_t gshard_moe_top2_workspace_bytes(const gshard_moe_shape* shape, int for_backward);
/* Size of the saved-for-backward `context` buffer that the forward fills when
 * GSHARD_FLAG_SAVE_FOR_BACKWARD is set. */
size_t gshard_moe_top2_context_bytes(const gshard_moe_shape* shape);
/* Extra workspace the *_host call needs for its device copies of x, u, y, l_aux. */
size_t gshard_moe_top2_host_staging_bytes(const gshard_moe_shape* shape);

/* The whole layer forward (Algorithm 2 with Algorithm 1 as Top2Gating), eq. (1)-(3).
 *   x [G,S,M], wg [M,E], wi [E,M,H], wo [E,H,M]: dtype; u [G,S] float in [0,1): the `rnd`
 *   of Algorithm 1, one per token (all zeros: every second choice passes the test).
 *   y [G,S,M] dtype: layer output WITHOUT the residual connection; a token whose two
 *   choices were both dropped gets zeros.  l_aux: one float, the mean over groups of
 *   Algorithm 1's group loss.  routing_out: NULL or a struct of optional outputs.
 *   context: NULL, or gshard_moe_top2_context_bytes() bytes when SAVE_FOR_BACKWARD is set.
 *   workspace: at least gshard_moe_top2_workspace_bytes(shape, 0) bytes, 256-byte aligned;
 *   its contents are scratch.
 * The call only enqueues kernels and memsets on cuda_stream (no allocation, no synchronisation, no
 * work on other streams), so it may be recorded into a CUDA graph by stream capture and replayed
 * on new contents of the same buffers. */
int gshard_moe_top2_forward(const gshard_moe_shape* shape, const void* x, const void* wg,
                            const void* wi, const void* wo, const float* u, void* y,
                            float* l_aux, const gshard_moe_routing* routing_out, void* context,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Same layer, activations on the HOST: x_host, u_host are read and y_host, l_aux_host are
 * written in (preferably pinned) host memory; weights wg, wi, wo stay device pointers (they
 * are model state, not a step's input).  Copies run on `cuda_stream` inside the call and the
 * call synchronises the stream before returning.  workspace must hold
 * gshard_moe_top2_workspace_bytes(shape,0) + gshard_moe_top2_host_staging_bytes(shape). */
int gshard_moe_top2_forward_host(const gshard_moe_shape* shape, const void* x_host,
                                 const void* wg, const void* wi, const void* wo,
                                 const float* u_host, void* y_host, float* l_aux_host,
                                 const gshard_moe_routing* routing_out, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);

/* Pipelined form of the host-buffer forward for callers that stream batches: nothing is
 * synchronised, the three phases of a step go to three streams so that the host-to-device copy of
 * the next batch, the layer of the current one and the device-to-host copy of the previous one
 * overlap (eq. (1)-(3) / Algorithm 1-2 as in gshard_moe_top2_forward).
 *   staging: device buffer of gshard_moe_top2_host_staging_bytes(shape) bytes holding this SLOT's
 *   copies of x, u, y, l_aux; use two or more slots (staging buffers with their own three events)
 *   in rotation.  workspace: gshard_moe_top2_workspace_bytes(shape, 0) bytes, shared by all slots
 *   (forwards are serialised on compute_stream).  ev_in / ev_done / ev_out: the slot's
 *   cudaEvent_t handles (as void*), created by the caller; the call waits on them where the slot's
 *   previous use must have finished and re-records them, so the same three events are passed every
 *   time the slot is used.  Host buffers must be pinned and stay untouched until ev_out (or
 *   copy_out_stream) has completed; routing_out, if given, must be per slot.  Not for
 *   SAVE_FOR_BACKWARD shapes.  Device-side status: gshard_moe_last_device_status(workspace,
 *   compute_stream). */
int gshard_moe_top2_forward_host_async(const gshard_moe_shape* shape, const void* x_host,
                                       const void* wg, const void* wi, const void* wo,
                                       const float* u_host, void* y_host, float* l_aux_host,
                                       const gshard_moe_routing* routing_out, void* workspace,
                                       size_t workspace_bytes, void* staging, size_t staging_bytes,
                                       void* copy_in_stream, void* compute_stream,
                                       void* copy_out_stream, void* ev_in, void* ev_done,
                                       void* ev_out);

/* Backward of L = <dy, y> + l_aux_weight * l_aux with the routing of the forward call held
 * constant (the paper leaves the backward to automatic differentiation and states that the
 * counts c_e are not differentiable; section 2.2, auxiliary-loss paragraph).
 *   context: the buffer filled by the forward.  dy [G,S,M] dtype.
 *   dx [G,S,M] dtype, dwg [M,E] float, dwi [E,M,H] dtype, dwo [E,H,M] dtype: overwritten. */
int gshard_moe_top2_backward(const gshard_moe_shape* shape, const void* x, const void* wg,
                             const void* wi, const void* wo, const void* context,
                             const void* dy, float l_aux_weight, void* dx, float* dwg,
                             void* dwi, void* dwo, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);

/* ---- the stages of the forward, callable on their own (same conventions) ---------------- */

/* Algorithm 1, gates and top_2: logits = x . wg, softmax in fp32, two largest gates per
 * token (lowest index wins ties), and the mean gates m_e.
 *   expert_idx [G,S,2] int32, gate12 [G,S,2] float (raw softmax values g1, g2), m [G,E] float.
 *   workspace: gshard_moe_top2_workspace_bytes(shape, 0). */
int gshard_moe_gate(const gshard_moe_shape* shape, const void* x, const void* wg,
                    int32_t* expert_idx, float* gate12, float* m, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);

/* Algorithm 1, the two token loops and l_aux, for all groups: positions are the stable rank of
 * a token among the tokens of its group that chose the same expert (first choices before
 * second choices).  Inputs expert_idx, gate12, u, m as produced by gshard_moe_gate.
 * routing_out->expert_idx and ->m are ignored; l_aux may be NULL.
 * workspace: gshard_moe_top2_workspace_bytes(shape, 0). */
int gshard_moe_capacity(const gshard_moe_shape* shape, const int32_t* expert_idx,
                        const float* gate12, const float* u, const float* m,
                        const gshard_moe_routing* routing_out, float* l_aux, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/* gshard_moe_capacity for callers that cannot allocate device memory (the paper has no
 * counterpart: this is an interface variant, not a different computation).
 * Who needs it: code that runs where no device allocation is possible at call time - an operator
 * inside a host runtime that owns the allocator and forbids allocating in its execute hook, a
 * serving loop whose memory pool is frozen after start-up - and that therefore cannot hand over a
 * workspace either.  The per-group statistics scratch of the capacity kernel then lives in a
 * 128 KB array built into the library image (held by every GPU that loads the library until
 * the process exits), which limits this variant to G <= 4096 groups: a larger G returns
 * GSHARD_ERR_UNSUPPORTED_SHAPE and launches nothing.
 * Arguments as gshard_moe_capacity, except that there is no workspace, so routing_out and its
 * slot, weight, flags, first_count, total_count, slot_token and l_aux_group must all be given
 * (stats and l_aux stay optional).  The call allocates nothing and calls no allocating routine.
 * Every call looks up the array's device address for the current device (the device the stream
 * belongs to must be current); the first call on a device also loads the library's module there,
 * so make that first call before any stream capture begins.  All calls on a device share
 * the one array: the kernel rewrites every entry it later reads, so nothing needs clearing
 * between calls, but two calls whose kernels overlap on the GPU (different streams) race on it;
 * keep them on one stream or order them yourself.  Results equal gshard_moe_capacity's. */
int gshard_moe_capacity_static(const gshard_moe_shape* shape, const int32_t* expert_idx,
                               const float* gate12, const float* u, const float* m,
                               const gshard_moe_routing* routing_out, float* l_aux,
                               void* cuda_stream);

/* Algorithm 2 dispatch as an index gather: buf[e, g*C+c, :] = x[g, slot_token[e,g,c], :],
 * zero row for an empty slot.  buf [E, G*C, M] dtype. */
int gshard_moe_dispatch(const gshard_moe_shape* shape, const void* x, const int32_t* slot_token,
                        void* buf, void* cuda_stream);

/* Eq. (2) for every expert: out[e] = relu(buf[e] . wi[e]) . wo[e]; buf, out [E, G*C, M] dtype.
 * workspace holds the hidden activations (gshard_moe_top2_workspace_bytes(shape, 0)). */
int gshard_moe_expert_ffn(const gshard_moe_shape* shape, const void* buf, const void* wi,
                          const void* wo, void* out, void* workspace, size_t workspace_bytes,
                          void* cuda_stream);

/* Eq. (3) / Algorithm 2 combine as a per-token gather:
 * y[g,s,:] = sum over k in {0,1} with slot[g,s,k] >= 0 of weight[g,s,k] * out[e_k, g*C+slot, :]. */
int gshard_moe_combine(const gshard_moe_shape* shape, const void* out, const int32_t* expert_idx,
                       const int32_t* slot, const float* weight, void* y, void* cuda_stream);

/* ---- expert-parallel form over several GPUs ------------------------------------------------
 * The paper's partitioning of the layer (Algorithm 2 and the sharding annotations of the MoE layer
 * in the section on the SPMD partitioner; AllToAll cost in the performance section): groups G split
 * over the devices for gating, capacity assignment, dispatch and combine with wg replicated,
 * experts E split over the devices for the expert FFN, one AllToAll before and one after it.
 * One process per GPU; rank r of `world` owns groups [r*G/world, (r+1)*G/world) and experts
 * [r*E/world, (r+1)*E/world); G and E must be multiples of world. */

/* Where a rank's data lives, as computed on the host by gshard_moe_ep_plan (no GPU needed). */
typedef struct {
  int32_t rank, world;
  int32_t groups_local, experts_local;   /* G/world, E/world                                        */
  int32_t group_begin, expert_begin;     /* first global group / expert of this rank                */
  int32_t rows_local;                    /* groups_local * C: rows of one expert in one rank's slab  */
  size_t row_bytes;                      /* M elements                                               */
  size_t bytes_per_peer;                 /* experts_local * rows_local * row_bytes: one slab         */
  gshard_moe_shape local;                /* shape of the stages that run on the local groups (G = G/world) */
  gshard_moe_shape ffn;                  /* shape of the local expert FFN (E = E/world, all G groups' rows) */
} gshard_moe_ep_layout;

/* The collectives, supplied by the caller (NCCL, torch.distributed, MPI ...).  Both enqueue on
 * cuda_stream (or order themselves after and before it) and return 0 on success.
 *   all_to_all: equal splits; bytes [i*bytes_per_peer, (i+1)*bytes_per_peer) of send go to rank i,
 *     the same range of recv receives from rank i.  send and recv are device buffers inside the
 *     workspace (or, with SAVE_FOR_BACKWARD, the context) of the call and never alias.
 *   all_reduce_sum_f32: in-place sum over the ranks of `count` floats in device memory (the l_aux
 *     scalar in the forward, dwg in the backward). */
typedef struct {
  int (*all_to_all)(void* user, const void* send, void* recv, size_t bytes_per_peer, void* cuda_stream);
  int (*all_reduce_sum_f32)(void* user, float* buf, size_t count, void* cuda_stream);
  void* user;
} gshard_ep_comm;

/* The same collectives through NCCL itself, for callers that hold an ncclComm_t: all_to_all becomes
 * one NCCL group of `world` sends and receives of equal slabs, all_reduce_sum_f32 an ncclAllReduce,
 * both on the call's stream, with no callback into the caller's language.  nccl_comm: an initialised
 * communicator of `world` ranks (an ncclComm_t passed as void*), owned by the caller and outliving
 * `comm`; `state`: storage that `comm` points into, which must outlive it too.  NCCL is not linked:
 * its functions are looked up in the process at run time (GSHARD_ERR_INTERNAL when there is none). */
typedef struct { void* opaque[8]; } gshard_ep_nccl_state;
int gshard_ep_comm_from_nccl(void* nccl_comm, int world, gshard_ep_nccl_state* state, gshard_ep_comm* comm);

/* Host-only: validates the partitioning and fills `layout`.  GSHARD_ERR_UNSUPPORTED_SHAPE when G or
 * E is not a multiple of world. */
int gshard_moe_ep_plan(const gshard_moe_shape* shape, int rank, int world, gshard_moe_ep_layout* layout);

/* Host-only: the permutation between the layout an AllToAll delivers, [world (source rank)]
 * [experts_local][rows_local] rows, and the layout the expert FFN reads, [experts_local]
 * [world * rows_local] rows (one expert's rows from all sources contiguous, in global group order);
 * inverse != 0 goes back.  src and dst are HOST buffers of world * experts_local * rows_local rows of
 * row_bytes bytes.  The device-side regroup inside gshard_moe_top2_forward_ep uses the same index
 * arithmetic; this function lets a CPU-only multi-process test drive it. */
int gshard_moe_ep_regroup_host(const gshard_moe_ep_layout* layout, const void* src, void* dst, size_t row_bytes,
                               int inverse);

size_t gshard_moe_ep_workspace_bytes(const gshard_moe_shape* shape, int world);          /* forward */
size_t gshard_moe_ep_context_bytes(const gshard_moe_shape* shape, int world);
size_t gshard_moe_ep_backward_workspace_bytes(const gshard_moe_shape* shape, int world);

/* Forward of the layer on rank `rank` of `world` (shape is the GLOBAL shape).
 *   x_local, y_local [G/world, S, M], u_local [G/world, S]: this rank's groups; wg [M, E] replicated;
 *   wi_local [E/world, M, H], wo_local [E/world, H, M]: this rank's experts.
 *   l_aux: the layer's loss (mean over ALL groups), identical on every rank after the call.
 *   routing_out: optional outputs for the LOCAL groups (shapes as in gshard_moe_routing with
 *   G = G/world; stats are this rank's).  comm: the collectives; may be NULL when world == 1.
 *   context: with GSHARD_FLAG_SAVE_FOR_BACKWARD, gshard_moe_ep_context_bytes(shape, world) bytes
 *   that receive what gshard_moe_top2_backward_ep needs (routing and softmax statistics of the local
 *   groups; inputs, hidden activations and ReLU mask of the local experts); else NULL.
 * With world == 1 the call runs exactly the kernels of gshard_moe_top2_forward and gives the same
 * bits.  Every received slab lies in this GPU's own memory before a kernel reads it. */
int gshard_moe_top2_forward_ep(const gshard_moe_shape* shape, int rank, int world, const void* x_local,
                               const void* wg, const void* wi_local, const void* wo_local,
                               const float* u_local, void* y_local, float* l_aux,
                               const gshard_moe_routing* routing_out, void* context,
                               const gshard_ep_comm* comm, void* workspace, size_t workspace_bytes,
                               void* cuda_stream);

/* Backward of the expert-parallel layer (same loss and conventions as gshard_moe_top2_backward): the
 * gradients of the expert outputs go to the experts' owners through an AllToAll, the expert FFN
 * backward runs over the local experts, the gradients of the expert inputs come back through a second
 * AllToAll, and the gating backward runs over the local groups.
 *   dy_local, dx_local [G/world, S, M]; dwi_local [E/world, M, H], dwo_local [E/world, H, M]: this
 *   rank's share; dwg [M, E] float: wg is replicated, so every rank ends with the SUM over the ranks
 *   (all_reduce_sum_f32).  context: filled by gshard_moe_top2_forward_ep on this rank.
 *   workspace: gshard_moe_ep_backward_workspace_bytes(shape, world). */
int gshard_moe_top2_backward_ep(const gshard_moe_shape* shape, int rank, int world, const void* x_local,
                                const void* wg, const void* wi_local, const void* wo_local,
                                const void* context, const void* dy_local, float l_aux_weight,
                                void* dx_local, float* dwg, void* dwi_local, void* dwo_local,
                                const gshard_ep_comm* comm, void* workspace, size_t workspace_bytes,
                                void* cuda_stream);

/* The expert-parallel forward with the exchange FUSED into the dispatch and combine kernels (same
 * partitioning and results as gshard_moe_top2_forward_ep).  The dispatch kernel stores each token row
 * directly into the expert owner's input buffer over NVLink, already in the layout the expert FFN
 * reads; the combine kernel loads a token's expert output rows directly from the owners' output
 * buffers.  No AllToAll and no regrouping copy remain; the expert FFN reads and writes only this GPU's
 * own memory; nothing is multicast.
 *   peer_buffers[w]: rank w's exchange buffer (gshard_moe_ep_p2p_buffer_bytes each, 256-byte aligned)
 *   as a device pointer valid in THIS process (peer access enabled / an IPC or symmetric-memory
 *   mapping); entry [rank] is this rank's own buffer.  First half: the FFN input of the rank's experts
 *   [E/world][G*C][M], written by every rank; second half: their output, read by every rank.
 *   rendezvous(user, phase, stream): orders the ranks - it must make this rank's stream publish that
 *   its work enqueued so far has completed AND wait for the same from every other rank (for instance
 *   one interprocess event per rank: record mine, wait on the others').  Called with phase 0 (the
 *   previous use of the buffers is over), 1 (all rows have arrived) and 2 (all expert outputs are
 *   complete); returns 0 on success.  No kernel of this library waits for another rank's kernel.
 *   comm: optional, only its all_reduce_sum_f32 is used (for l_aux; without it l_aux holds this rank's
 *   share, sum of its group losses / G).  workspace: gshard_moe_top2_workspace_bytes of the LOCAL shape
 *   (layout.local) suffices.  Forward only: SAVE_FOR_BACKWARD shapes are refused. */
typedef struct {
  int (*rendezvous)(void* user, int phase, void* cuda_stream);
  void* user;
  void* const* peer_buffers;   /* [world] */
} gshard_ep_p2p;
size_t gshard_moe_ep_p2p_buffer_bytes(const gshard_moe_shape* shape, int world);
int gshard_moe_top2_forward_ep_p2p(const gshard_moe_shape* shape, int rank, int world, const void* x_local,
                                   const void* wg, const void* wi_local, const void* wo_local,
                                   const float* u_local, void* y_local, float* l_aux,
                                   const gshard_moe_routing* routing_out, const gshard_ep_p2p* p2p,
                                   const gshard_ep_comm* comm, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream);

/* The position-wise feed-forward sub-layer of the ordinary Transformer layers that alternate with
 * the MoE layers (section 2.1: every other feed-forward layer is replaced by a MoE layer; the
 * performance section times "MoE layer + adjacent Transformer layer"): y = relu(x . wi) . wo over
 * all tokens, no bias - eq. (2) with a single expert that sees every token, run by the same two
 * grouped tensor-core GEMMs as the expert FFN.
 *   x, y [n_tokens, M], wi [M, H], wo [H, M]: dtype (gshard_dtype); bf16 needs M % 64 == 0 and
 *   H % 64 == 0.  flags: 0, or GSHARD_FLAG_TF32_EXPERTS (fp32 on the tensor cores),
 *   GSHARD_FLAG_ONE_SM_MMA, GSHARD_FLAG_SIMT_CONTRACTIONS with their meaning above.
 *   workspace: gshard_dense_ffn_workspace_bytes() bytes, 256-byte aligned; it holds a
 *   status word (read with gshard_moe_last_device_status) and the hidden activations [n_tokens, H]. */
size_t gshard_dense_ffn_workspace_bytes(int64_t n_tokens, int32_t M, int32_t H, int32_t dtype);
int gshard_dense_ffn_forward(int64_t n_tokens, int32_t M, int32_t H, int32_t dtype, uint32_t flags,
                             const void* x, const void* wi, const void* wo, void* y, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);

/* The check that GSHARD_FLAG_DEBUG_CHECKS runs inside the forward, callable on its own: verifies
 * the invariants Algorithm 1 implies for routing->expert_idx, slot, weight, flags and slot_token
 * (all five required) and records GSHARD_ERR_INTERNAL in the status word of `workspace` (its first
 * word; at least 256 bytes, 256-byte aligned) when one does not hold; read it with
 * gshard_moe_last_device_status.  Indices are bounds-checked before they are used. */
int gshard_moe_check_routing(const gshard_moe_shape* shape, const gshard_moe_routing* routing, void* workspace,
                             void* cuda_stream);

/* Self-test of the give-up path shared by every bounded device-side wait (the paper has no
 * counterpart; this is robustness plumbing).  Launches one small CTA that allocates tensor
 * memory, waits on an mbarrier nothing arrives at with a limit of limit_us microseconds
 * (1..1000), and leaves through the same teardown as the GEMM kernels: abort flag,
 * GSHARD_ERR_TIMEOUT into the status word of `workspace` (its first word; 256-byte aligned, at
 * least 256 bytes), tensor memory released, normal return.  gshard_moe_last_device_status then
 * reports GSHARD_ERR_TIMEOUT and the workspace and the context remain usable. */
int gshard_moe_debug_wait_timeout(void* workspace, uint32_t limit_us, void* cuda_stream);

/* Synchronises `cuda_stream` and returns the device status word of `workspace`
 * (GSHARD_OK, GSHARD_ERR_TIMEOUT, ...) or GSHARD_ERR_CUDA if the stream reported an error. */
int gshard_moe_last_device_status(void* workspace, void* cuda_stream);

/* Number of kernels the last forward/backward/stage call on this thread launched. */
int gshard_moe_last_launch_count(void);

/* Measurement hook: the NEXT gshard_moe_top2_forward call on this thread records start_event
 * before and stop_event after its expert-FFN launches (eq. (2)) on the call's stream
 * (cudaEvent_t handles passed as void*, created with timing enabled, owned by the caller).  The
 * pair is used once; pass two NULLs to disarm.  Lets a benchmark time the dominant kernel inside
 * its timed region instead of in a loop of its own. */
int gshard_moe_time_expert_ffn(void* start_event, void* stop_event);

#ifdef __cplusplus
}
#endif
#endif /* GSHARD_MOE_H_ */
