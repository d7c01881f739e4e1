/*
 * moe.h - C ABI of the B200 (sm_100a) mixture-of-experts FFN layer, forward and backward.
 *
 * The layer is the MoE block of a Qwen3-30B-A3B-style reranker (paper, Section "Expert-Parallel MoE
 * Training": 128 experts, top-8 routing; the LoRA target-group listing names its parts: router.weight,
 * experts.*.linear_fc1, experts.*.linear_fc2).  Every expert is local to the GPU (expert-parallel degree 1).
 *
 *   forward :  l = x W_r (+ b_r)                     fp32 logits
 *              p = softmax(l)                         over all E experts
 *              idx = top-k of l                       lowest index wins ties, stored in pick order
 *              g = p[idx] / sum p[idx]                renormalised gates
 *              rows sorted by (expert, token)         counts, perm
 *              a = silu(x W_gate[e]) * (x W_up[e])    per routed row, SwiGLU
 *              o = a W_down[e]
 *              y[t] = sum_j g[t,j] o[t,j]
 *              aux = E * sum_e (c_e / (T k)) * mean_t p[t,e]
 *   backward:  gradients of  <y, dy> + d_aux * aux  with respect to x, W_r, b_r, W_gate, W_up, W_down,
 *              routing decisions held fixed.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  Tensors are dense row-major.
 *   - bf16 tensors are passed as uint16_t bit patterns.  Pointers must be 16-byte aligned.
 *   - The caller owns every buffer, the workspace included.  No entry point allocates or frees device
 *     memory.
 *   - All work is enqueued on the caller's CUDA stream (passed as void* = cudaStream_t).  Neither
 *     moe_forward nor moe_backward synchronises with the host or copies anything to the host: expert
 *     counts stay on the device and drive the tile schedulers there.
 *   - Errors are return codes.  Argument errors are found before anything is launched.  A device-side
 *     problem (a bounded wait that ran out) sets a status word inside the workspace; the kernels leave
 *     cleanly and moe_poll_status reports it.
 *   - Inputs must be finite.  One moe_ctx serves one stream at a time.
 */
#ifndef MOE_B200_H
#define MOE_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MOE_API __attribute__((visibility("default")))
#else
#define MOE_API
#endif

typedef struct {
  int32_t d;      /* model width,  multiple of 64                                  */
  int32_t E;      /* experts,      1 <= E <= 256                                   */
  int32_t f;      /* expert width, multiple of 64                                  */
  int32_t top_k;  /* experts per token, 1 <= top_k <= E and top_k <= 32            */
  int32_t flags;  /* 0, or one of the MOE_FLAG_* tile flags                        */
} moe_config;

/* Tile shape of the expert GEMMs.  By default the library chooses per GEMM between CTA pairs (256 x 256 tiles,
 * tcgen05 cta_group::2, each CTA staging half of B) and one-CTA 128 x 256 tiles: weight gradients run on pairs when
 * the experts average at least 768 rows, row GEMMs from 512 rows per expert (the dgrad of gate / up with fewer than 64
 * K blocks per tile from 768); an expert with an odd number of 128-row blocks gets a last pair whose second half is
 * empty.  Below those sizes the layer is bound by streaming the weights and one-CTA tiles are used.  The flags force
 * one shape everywhere (same results; for comparison measurements). */
#define MOE_FLAG_CTA_PAIR_TILES 1
#define MOE_FLAG_SINGLE_CTA_TILES 2
/* Row GEMMs run every complete pair of 128-row blocks of an expert on a CTA pair and the leftover block of an odd
 * count on a one-CTA tile (two launches, no half-empty pairs); weight gradients run on pairs. */
#define MOE_FLAG_HYBRID_TILES 16
/* moe_backward normally runs the router's gradient chain (dl, dW_r, db_r, the router term of dx) on a second stream of
 * the context, forked and joined inside the call (the caller's stream sees one ordered call; the pattern is legal
 * inside a stream capture).  This flag keeps everything on the caller's stream. */
#define MOE_FLAG_NO_SIDE_STREAM 8
/* The router weight W_r is passed as fp32 [d,E] instead of bf16 (moe_forward / moe_backward only; E must be a multiple
 * of 8).  Every fp32 value is the exact sum of three bf16 values, so the logits are still an fp32 contraction of exact
 * products: the library splits W_r on the device at every forward call and runs three tensor-core passes. */
#define MOE_FLAG_ROUTER_FP32 32
/* Debug build of the index-driven kernels (permutation scatter, row copies, combine, unpermute, router gradient): every
 * expert index and row index read from the routing tables is checked against its range before it is used; a violation
 * is recorded in the status word (moe_poll_status then returns MOE_ERR_DEVICE_BOUNDS) and the access is skipped or
 * redirected to row 0, so nothing out of range is touched.  For hunting corrupted tables where a memory checker is not
 * available; costs a few percent in those kernels. */
#define MOE_FLAG_DEBUG_CHECKS 64

typedef struct moe_ctx moe_ctx; /* opaque, lives in host memory */

typedef enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = -1,
  MOE_ERR_UNSUPPORTED = -2,
  MOE_ERR_WORKSPACE = -3,   /* workspace_bytes smaller than moe_workspace_bytes(ctx, T) */
  MOE_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed                       */
  MOE_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait ran out                     */
  MOE_ERR_DEVICE_BOUNDS = -6   /* a device-side bounds check failed (MOE_FLAG_DEBUG_CHECKS; moe_ep_plan: rows beyond rows_cap) */
} moe_status;

/* Number of per-stage timers filled by moe_stage_times (see below). */
#define MOE_NUM_STAGES 16

/* Creates a context for one layer shape.  Allocates host memory only.  The first call that launches work binds
 * the context to the device that is current then; later calls with another device current are refused with
 * MOE_ERR_INVALID_ARG (one context per device). */
MOE_API moe_status moe_create(const moe_config* cfg /* host */, moe_ctx** out /* host */);
MOE_API void moe_destroy(moe_ctx* ctx);
/* Device the context is bound to, or -1 while no call has launched work yet (or ctx is NULL). */
MOE_API int moe_ctx_device(const moe_ctx* ctx);

/* Bytes of workspace needed for a call with T tokens (0 if ctx is NULL or T < 0).  The workspace holds
 * the routing tables and the activations that moe_forward saves for moe_backward. */
MOE_API size_t moe_workspace_bytes(const moe_ctx* ctx, int64_t T);

/* Byte offset and size of a named internal buffer inside the workspace, for stage-by-stage tests.
 * Names: "counts" "offsets" "pad_offsets" "logits" "idx" "gates" "inv" "row_gate" "xp" "hg" "hu" "act"
 * "o" "dhg" "dhu" "dxp" "dg" "dl".  Internal row buffers (xp, hg, hu, act, o, dhg, dhu, dxp) are laid out
 * expert-major with every expert's segment padded to a multiple of 128 rows ("pad_offsets"); pad rows
 * are zero.  "act" and "o" are stored already multiplied by the row's gate (so the combine is a plain sum); after
 * moe_backward "o" holds the gathered rows of dy.  Returns MOE_ERR_INVALID_ARG for an unknown name. */
MOE_API moe_status moe_workspace_find(const moe_ctx* ctx, int64_t T, const char* name /* host */,
                              size_t* offset /* host */, size_t* bytes /* host */);

MOE_API const char* moe_status_string(moe_status s);

/* Synchronises the stream and reports the device-side status word of the workspace.  The word is sticky: the
 * first failure a kernel records stays there - no later kernel or call overwrites or clears it - until this call
 * (or moe_step_host_end) has returned it once; reporting acknowledges it, after which the context and the
 * workspace are usable again.  A workspace no call has used yet reports MOE_OK. */
MOE_API moe_status moe_poll_status(moe_ctx* ctx, const void* workspace, void* cuda_stream);

/* Number of kernels the library has launched in this process so far (all contexts; copies and memsets not counted). */
MOE_API long long moe_kernel_launches(void);

/* Exercises the device-side failure path without faulting anything: launches one tiny kernel whose bounded wait
 * (on a barrier nothing signals) runs out after a few thousand polls; the kernel records the timeout in the
 * workspace's status word and returns.  A following moe_poll_status - also one that comes after further
 * moe_forward / moe_backward calls - reports MOE_ERR_DEVICE_TIMEOUT once; the context stays usable.  The layer's kernels bound every wait the same way
 * (about a second); nothing in the library makes a GPU fault, trap or hang on purpose. */
MOE_API moe_status moe_selftest_timeout(moe_ctx* ctx, void* workspace, void* cuda_stream);

/* Per-stage timing.  With enable != 0, moe_forward / moe_backward record CUDA events between their
 * kernels on the caller's stream, one event set per forward+backward pair, in a ring of MOE_PROF_RING sets.
 * moe_stage_times waits for the recorded events, ADDS to ms[s] (host array of MOE_NUM_STAGES floats) the
 * milliseconds stage s took summed over the pairs recorded since the previous call (the last MOE_PROF_RING
 * of them if there were more), stores that number of pairs in *steps, and starts a new window.
 * Stage order: 0 router, 1 permute (histogram, scan, scatter, gather), 2 gate/up GEMM + SwiGLU,
 * 3 down GEMM, 4 combine, 5 combine-bwd (gather of dy rows), 6 dgrad-down + SwiGLU-bwd (+ dg), 7 wgrad-down, 8 dgrad gate/up,
 * 9 wgrad gate/up, 10 router-bwd (dl), 11 dW_r, 12 unpermute-bwd (dx), 13 router term of dx, 14..15 unused.
 * Stages 10, 11 and 13 run on the context's second stream beside stages 7..9 (unless MOE_FLAG_NO_SIDE_STREAM), so the
 * stage times then add up to more than the step. */
#define MOE_PROF_RING 64
MOE_API moe_status moe_set_profiling(moe_ctx* ctx, int enable);
MOE_API moe_status moe_stage_times(moe_ctx* ctx, float* ms /* host */, int32_t* steps /* host */);

/* Forward pass over T tokens (T >= 0).
 *   x          [T,d]   bf16
 *   W_r        [d,E]   bf16 router weight (fp32 with MOE_FLAG_ROUTER_FP32); the contraction accumulates in fp32
 *   b_r        [E]     fp32 additive logit bias, or NULL
 *   logits_in  [T,E]   fp32, or NULL.  When given, routing starts from these logits and the router
 *                      contraction is skipped (test hook: lets a caller construct exact ties).
 *   W_gate,W_up [E,d,f] bf16        W_down [E,f,d] bf16
 * Outputs
 *   y          [T,d]   bf16
 *   topk_idx   [T,k]   int32, pick order (descending logit, ties ascending index)
 *   topk_w     [T,k]   fp32 gates, each row sums to 1
 *   expert_counts [E]  int32
 *   perm       [T*k]   int32 or NULL: perm[r] = t*k + j of the pair in row r of the expert-major order
 *                      (rows sorted by expert, then token)
 *   aux_loss   [1]     fp32, coefficient-free
 *   logits_out [T,E]   fp32 or NULL
 * The workspace must be at least moe_workspace_bytes(ctx, T) bytes and must stay untouched until the
 * matching moe_backward has run. */
MOE_API moe_status moe_forward(moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                       const float* logits_in, const uint16_t* W_gate, const uint16_t* W_up,
                       const uint16_t* W_down, uint16_t* y, int32_t* topk_idx, float* topk_w,
                       int32_t* expert_counts, int32_t* perm, float* aux_loss, float* logits_out,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Forward pass for inference / scoring (the paper's serving use, Section "Evaluation and serving": rerankers score
 * query-passage pairs with forward passes only).  Same arguments and results as moe_forward, but the gate/up GEMM
 * does not store its pre-activations, so 2 * T * top_k * f * 2 bytes less are written, the workspace only needs
 * moe_inference_workspace_bytes(ctx, T) bytes (routing tables, xp, act, o) and it cannot feed moe_backward. */
MOE_API size_t moe_inference_workspace_bytes(const moe_ctx* ctx, int64_t T);
MOE_API moe_status moe_forward_inference(moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r,
                                         const float* b_r, const float* logits_in, const uint16_t* W_gate,
                                         const uint16_t* W_up, const uint16_t* W_down, uint16_t* y,
                                         int32_t* topk_idx, float* topk_w, int32_t* expert_counts, int32_t* perm,
                                         float* aux_loss, float* logits_out, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream);

/* Backward pass of the forward call that filled `workspace`.
 *   dy    [T,d] bf16 upstream gradient of y;  d_aux: host scalar, dLoss/d(aux_loss)
 *   x, W_r, W_gate, W_up, W_down: the forward inputs
 * Outputs (all OVERWRITTEN, not accumulated)
 *   dx [T,d] bf16;  dW_r [d,E] fp32;  db_r [E] fp32 or NULL;
 *   dW_gate, dW_up [E,d,f] bf16;  dW_down [E,f,d] bf16 (zero slabs for experts without tokens).
 * The workspace must be the one a training forward call (moe_forward; moe_lora_forward for moe_lora_backward) filled
 * for the SAME T, untouched in between: its tables drive every index of the backward kernels.  The context remembers
 * what its recent forward calls left in which workspace (the last eight workspaces) and returns MOE_ERR_INVALID_ARG,
 * before any launch, when the workspace was last filled for another T, by moe_forward_inference, or by the other
 * variant of the layer. */
MOE_API moe_status moe_backward(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux, const uint16_t* x,
                        const uint16_t* W_r, const uint16_t* W_gate, const uint16_t* W_up,
                        const uint16_t* W_down, uint16_t* dx, float* dW_r, float* db_r, uint16_t* dW_gate,
                        uint16_t* dW_up, uint16_t* dW_down, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/* Backward pass that ADDS the weight gradients to fp32 buffers instead of overwriting bf16 ones: the gradient
 * accumulation of a training step that is split into micro-batches (the paper's Megatron backend keeps fp32
 * gradient buffers that the distributed optimizer consumes, Section "Megatron backend").
 *   dW_gate, dW_up [E,d,f] fp32, dW_down [E,f,d] fp32, dW_r [d,E] fp32, db_r [E] fp32 or NULL: each is read, the
 *   micro-batch's gradient is added in fp32 (no bf16 rounding of the gradient), and written back.  The caller
 *   zeroes them at the start of an accumulation window.  Slabs of experts without tokens are left untouched.
 *   dx [T,d] bf16 is overwritten as in moe_backward.  All other arguments as in moe_backward. */
MOE_API moe_status moe_backward_accumulate(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux,
                                           const uint16_t* x, const uint16_t* W_r, const uint16_t* W_gate,
                                           const uint16_t* W_up, const uint16_t* W_down, uint16_t* dx, float* dW_r,
                                           float* db_r, float* dW_gate, float* dW_up, float* dW_down,
                                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* moe_backward_accumulate for data-parallel training, where the weight gradients must be summed over the ranks (the
 * paper's Megatron backend: DP = world / (TP x PP), gradients reduced into the distributed optimizer's buffers; Section
 * "Megatron backend").  The two weight-gradient GEMMs run as n_groups launches over consecutive ranges of
 * ceil(E / n_groups) experts, and the library records, on cuda_stream, the caller's events
 *     group_events[g]             when dW_down[range g] is complete           (g = 0 .. n_groups - 1)
 *     group_events[n_groups + g]  when dW_gate[range g] and dW_up[range g] are complete
 * (host array of 2 * n_groups cudaEvent_t handles).  A caller makes its communication stream wait for an event and
 * all-reduces that range's slab while the remaining weight-gradient launches, the dgrad GEMM between them and the
 * router's chain still run: the reduction overlaps the backward pass instead of following it.  Results are those of
 * moe_backward_accumulate (within a range the experts run in index order, not largest first). */
MOE_API moe_status moe_backward_accumulate_grouped(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux,
                                                   const uint16_t* x, const uint16_t* W_r, const uint16_t* W_gate,
                                                   const uint16_t* W_up, const uint16_t* W_down, uint16_t* dx,
                                                   float* dW_r, float* db_r, float* dW_gate, float* dW_up,
                                                   float* dW_down, int32_t n_groups,
                                                   void* const* group_events /* host */, void* workspace,
                                                   size_t workspace_bytes, void* cuda_stream);

/* Expert LoRA: the same layer with frozen expert weights and trainable rank-r adapters on the experts' fc1 (gate | up)
 * and fc2 (down) - the paper's "moe_experts" LoRA target group (experts.*.linear_fc1, experts.*.linear_fc2; Section
 * "LoRA target groups for MoE").  Effective weights:
 *     W_gate' = W_gate + scale * A1 B1_gate,   W_up' = W_up + scale * A1 B1_up,   W_down' = W_down + scale * A2 B2
 * with A1 [E,d,r], B1_gate, B1_up [E,r,f], A2 [E,f,r], B2 [E,r,d], all bf16; r = rank, a multiple of 8 in [8, 64].
 * The effective weights are never formed: the low-rank products (x A1, act A2, ...) are 64-wide row buffers that
 * enter the expert GEMMs as one extra K segment, and the adapter gradients are skinny GEMMs; no gradient of the
 * frozen W_gate / W_up / W_down is computed.  Everything else (routing, outputs, dx, dW_r) is as in moe_forward /
 * moe_backward.  The workspace needs moe_lora_workspace_bytes(ctx, T) bytes.  Gradients dA1, dB1_gate, dB1_up, dA2,
 * dB2 have the adapters' shapes, are bf16 and are overwritten (zero slabs for experts without tokens). */
MOE_API size_t moe_lora_workspace_bytes(const moe_ctx* ctx, int64_t T);
MOE_API moe_status moe_lora_forward(moe_ctx* ctx, int64_t T, int32_t rank, float scale, const uint16_t* x,
                                    const uint16_t* W_r, const float* b_r, const uint16_t* W_gate,
                                    const uint16_t* W_up, const uint16_t* W_down, const uint16_t* A1,
                                    const uint16_t* B1_gate, const uint16_t* B1_up, const uint16_t* A2,
                                    const uint16_t* B2, uint16_t* y, int32_t* topk_idx, float* topk_w,
                                    int32_t* expert_counts, float* aux_loss, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream);
MOE_API moe_status moe_lora_backward(moe_ctx* ctx, int64_t T, int32_t rank, float scale, const uint16_t* dy,
                                     float d_aux, const uint16_t* x, const uint16_t* W_r, const uint16_t* W_gate,
                                     const uint16_t* W_up, const uint16_t* W_down, const uint16_t* A1,
                                     const uint16_t* B1_gate, const uint16_t* B1_up, const uint16_t* A2,
                                     const uint16_t* B2, uint16_t* dx, float* dW_r, uint16_t* dA1, uint16_t* dB1_gate,
                                     uint16_t* dB1_up, uint16_t* dA2, uint16_t* dB2, void* workspace,
                                     size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------------------------------
 * Expert parallelism (EP > 1).  The paper trains its MoE reranker with the experts spread over an EP group (Section
 * "Expert-Parallel MoE Training": EP = 16; "MoE layers dispatch routed tokens only among the ranks within an EP
 * group").  Rank r of `world` ranks owns the experts [r E/world, (r+1) E/world), keeps its own T tokens, and passes
 * only its shard of the expert weights.  Token rows reach the owning rank, and expert outputs come back, through
 * plain stores / loads of this library's kernels into PEER-MAPPED buffers (NVLink): every rank passes the table
 * peer_own_ws[world] of all ranks' owner workspaces as they are mapped into its own address space (entry `rank` is
 * its own; on one GPU the entries are ordinary device pointers).  The caller provides the two group operations the
 * library does not do itself: the all-gather of the per-rank expert counts after moe_ep_route, and a barrier of the
 * group between any two phases, because each phase reads what the previous one wrote on other ranks:
 *
 *   forward :  moe_ep_route | all-gather counts | moe_ep_plan | barrier | moe_ep_dispatch(x) | barrier |
 *              moe_ep_expert_forward | barrier | moe_ep_combine
 *   backward:  moe_ep_dispatch(dy, backward = 1) | barrier | moe_ep_expert_backward | barrier | moe_ep_router_backward
 *
 * Every phase that takes T must name the T of the moe_ep_route call that filled the sender workspace (the context
 * checks this on the host and returns MOE_ERR_INVALID_ARG otherwise).  Results are those of the one-GPU layer applied to the concatenation of the ranks' batches in rank order (same row
 * order inside every expert), except that aux_loss, its gradient and dW_r / db_r are per rank, over the rank's own
 * tokens (each rank is also a data-parallel rank for the router weight; sum dW_r over the group as for any replicated
 * parameter).  Requirements: E a multiple of `world` and of 8, world <= MOE_EP_MAX_RANKS.
 *
 * Workspaces (caller-allocated): the SENDER workspace (moe_ep_send_workspace_bytes(ctx, T): routing state of the
 * rank's tokens) and the OWNER workspace (moe_ep_own_workspace_bytes(ctx): tables and row buffers of the owned
 * experts, sized for rows_cap received rows - the caller's bound on sum over ranks of rows routed to this rank, at
 * most sum_r T_r * min(top_k, E/world); it is the owner workspace that peers map).  rows_cap must be the same on every
 * rank of the group.  A step whose rows do not fit (the rows of the experts of ANY rank, each expert padded to 128,
 * exceed the owner buffers) is refused by moe_ep_plan on every rank alike - every rank sees the same counts: nothing
 * is dispatched, no owner buffer is written, y, dx and the weight gradients of the step come out as zeros, and
 * moe_poll_status on the sender workspace returns MOE_ERR_DEVICE_BOUNDS (once; the context stays usable). */
#define MOE_EP_MAX_RANKS 16
MOE_API moe_status moe_ep_create(const moe_config* cfg /* host */, int32_t world, int32_t rank, int64_t rows_cap,
                                 moe_ctx** out /* host */);
MOE_API size_t moe_ep_send_workspace_bytes(const moe_ctx* ctx, int64_t T);
MOE_API size_t moe_ep_own_workspace_bytes(const moe_ctx* ctx);
/* Named internal buffers, for tests: own_side = 0: sender workspace ("counts" "logits" "idx" "gates" "inv" "dg" "dl"
 * "ep_dest" "status"); own_side = 1: owner workspace (names of moe_workspace_find, E/world experts). */
MOE_API moe_status moe_ep_workspace_find(const moe_ctx* ctx, int64_t T, int own_side, const char* name /* host */,
                                         size_t* offset /* host */, size_t* bytes /* host */);
/* Router over the rank's tokens: x [T,d], W_r [d,E] (all E experts), b_r [E] or NULL -> topk_idx [T,k], topk_w [T,k],
 * counts_local [E] (rows this rank routes to each expert; the caller all-gathers these), aux_loss [1] (local). */
MOE_API moe_status moe_ep_route(moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                                int32_t* topk_idx, float* topk_w, int32_t* counts_local, float* aux_loss,
                                void* send_ws, size_t send_ws_bytes, void* cuda_stream);
/* all_counts [world, E] int32 (device; row r = counts_local of rank r).  Places this rank's rows inside the owners'
 * buffers, builds the tile tables of the owned experts in own_ws and clears what must start at zero there. */
MOE_API moe_status moe_ep_plan(moe_ctx* ctx, int64_t T, const int32_t* all_counts, void* send_ws, size_t send_ws_bytes,
                               void* own_ws, size_t own_ws_bytes, void* cuda_stream);
/* Writes the rank's token rows (src = x with backward = 0, src = dy with backward = 1; [T,d] bf16) into the owners'
 * row buffers; the forward call also stores each row's gate beside it. */
MOE_API moe_status moe_ep_dispatch(moe_ctx* ctx, int64_t T, const uint16_t* src, int backward,
                                   void* const* peer_own_ws /* host array of device pointers */, void* send_ws,
                                   size_t send_ws_bytes, void* cuda_stream);
/* Expert GEMMs over the owned experts: W_gate, W_up [E/world,d,f], W_down [E/world,f,d] are the rank's shards. */
MOE_API moe_status moe_ep_expert_forward(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up,
                                         const uint16_t* W_down, void* own_ws, size_t own_ws_bytes, void* cuda_stream);
/* y [T,d] of the rank's tokens from the owners' output rows. */
MOE_API moe_status moe_ep_combine(moe_ctx* ctx, int64_t T, void* const* peer_own_ws /* host */, const void* send_ws,
                                  size_t send_ws_bytes, uint16_t* y, void* cuda_stream);
/* Backward GEMMs over the owned experts; dW_gate, dW_up [E/world,d,f], dW_down [E/world,f,d] bf16, overwritten. */
MOE_API moe_status moe_ep_expert_backward(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up,
                                          const uint16_t* W_down, uint16_t* dW_gate, uint16_t* dW_up,
                                          uint16_t* dW_down, void* own_ws, size_t own_ws_bytes, void* cuda_stream);
/* The same with the owned experts' weight gradients ADDED into fp32 buffers of the same shapes (the main gradients an
 * expert-parallel rank keeps for its own experts over an accumulation window: they need no reduction inside the group);
 * the caller zeroes them at the start of a window.  Slabs of experts without rows are left untouched. */
MOE_API moe_status moe_ep_expert_backward_accumulate(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up,
                                                     const uint16_t* W_down, float* dW_gate, float* dW_up,
                                                     float* dW_down, void* own_ws, size_t own_ws_bytes,
                                                     void* cuda_stream);
/* Router gradient and dx of the rank's tokens: dx [T,d] bf16, dW_r [d,E] fp32, db_r [E] fp32 or NULL (overwritten). */
MOE_API moe_status moe_ep_router_backward(moe_ctx* ctx, int64_t T, float d_aux, const uint16_t* x, const uint16_t* W_r,
                                          void* const* peer_own_ws /* host */, void* send_ws, size_t send_ws_bytes,
                                          uint16_t* dx, float* dW_r, float* db_r, void* cuda_stream);

/* Listwise training loss on grouped reranker scores (paper, paragraph "Contrastive and distillation losses").
 * scores [n,G] fp32 DEVICE, one row per query (G passages per query).
 *   MOE_LISTWISE_CONTRASTIVE: the positive passage sits at position 0 of every row;
 *       loss = (1/n) sum_g ( logsumexp(s_g) - s_g[0] );  teacher and the temperatures are ignored.
 *   MOE_LISTWISE_DISTILL: teacher [n,G] fp32 DEVICE holds stored teacher scores;
 *       loss = (s_temp^2 / n) sum_g KL( softmax(t_g / t_temp) || softmax(s_g / s_temp) );  s_temp, t_temp > 0.
 * loss [1] fp32 DEVICE is overwritten; dscores [n,G] fp32 DEVICE (or NULL) receives dloss/dscores.  n = 0 gives loss 0.
 * One small kernel on cuda_stream, no workspace, no host synchronisation; the sum over the rows runs in a fixed order
 * (same bits on every run).  Invalid arguments (unknown kind, G < 1, a non-positive temperature, a missing pointer)
 * return MOE_ERR_INVALID_ARG before anything is launched. */
#define MOE_LISTWISE_CONTRASTIVE 0
#define MOE_LISTWISE_DISTILL 1
MOE_API moe_status moe_listwise_loss(int32_t kind, int64_t n, int32_t G, const float* scores, const float* teacher,
                                     float s_temp, float t_temp, float* loss, float* dscores, void* cuda_stream);

/* Host-buffer convenience used for end-to-end timing: every tensor argument is a HOST pointer (pinned
 * memory recommended); the call copies inputs to the device buffers of `dev` (a device scratch of
 * moe_e2e_device_bytes(ctx, T) bytes owned by the caller), runs forward and backward, copies y, dx, aux and
 * the weight gradients back and synchronises the stream.  copy_weights != 0 also uploads the weights and
 * downloads their gradients; with 0 the weights must already be resident from an earlier call.  The copies run on
 * two streams of the context so that dy arrives while forward runs and y leaves while backward runs. */
MOE_API size_t moe_e2e_device_bytes(const moe_ctx* ctx, int64_t T);
/* Byte offset, inside `dev`, of the layer workspace the host-buffer calls use (what moe_poll_status wants). */
MOE_API size_t moe_e2e_workspace_offset(const moe_ctx* ctx, int64_t T);
MOE_API moe_status moe_step_host(moe_ctx* ctx, int64_t T, int copy_weights, const uint16_t* x, const uint16_t* W_r,
                         const uint16_t* W_gate, const uint16_t* W_up, const uint16_t* W_down,
                         const uint16_t* dy, float d_aux, uint16_t* y, float* aux_loss, uint16_t* dx,
                         float* dW_r, uint16_t* dW_gate, uint16_t* dW_up, uint16_t* dW_down,
                         void* dev /* device */, size_t dev_bytes, void* cuda_stream);

/* Pipelined form of moe_step_host for training loops that prefetch the next batch: moe_step_host_begin enqueues one
 * whole step (x, dy in; forward; backward; y, aux, dx out) for slot 0 or 1 and returns without waiting;
 * moe_step_host_end(slot) blocks until that slot's y, aux_loss and dx have arrived in the host buffers.  With both
 * slots in flight (begin(0), begin(1), end(0), begin(0), end(1), ...) the upload of the next batch and the download
 * of the previous results overlap the current step's kernels.  Weights must be resident (one earlier moe_step_host
 * with copy_weights = 1); the weight gradients of the most recent step stay on the device.  Host buffers of a slot
 * must stay untouched between its begin and end.  moe_step_host_end returns MOE_ERR_DEVICE_TIMEOUT (once) when a
 * kernel up to and including that slot's step recorded a failure in the workspace's status word. */
MOE_API moe_status moe_step_host_begin(moe_ctx* ctx, int slot, int64_t T, const uint16_t* x, const uint16_t* dy,
                                       float d_aux, uint16_t* y, float* aux_loss, uint16_t* dx, void* dev,
                                       size_t dev_bytes, void* cuda_stream);
MOE_API moe_status moe_step_host_end(moe_ctx* ctx, int slot);

/* Router weight gradient without any device allocation:  dW_r[d,E] = sum_t x[t,:]^T dl[t,:].
 * (The paper has no counterpart of this call; it exists for integration reasons only.)
 *
 * Who it is for.  moe_backward needs a caller-provided workspace, which in practice means the caller can
 * allocate device memory.  Some callers cannot: a plug-in running inside a host application that handed all device
 * memory to its own pool at start-up, or a service loop that cannot afford the device-wide synchronisation that
 * cudaMalloc and cudaFree imply.  For them this one call keeps its scratch (the per-token-slice partial sums)
 * in a fixed array that is part of the library image, and calls no cudaMalloc, cudaFree or other allocating routine.
 *
 *   x  [T,d] bf16 (device),  dl [T,E] fp32 (device, the router-logit gradient),  dW_r [d,E] fp32 (device, overwritten).
 *   d must be a multiple of 64, 1 <= E <= 256, and d * E <= MOE_STATIC_MAX_DE; larger shapes are refused with
 *   MOE_ERR_UNSUPPORTED before anything is launched (use moe_backward with a workspace instead).
 *
 * Cost and rules.  The scratch is MOE_STATIC_MAX_DE * 8 floats = 8 MiB of device memory on every GPU that loads the
 * library, held until the process ends.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current) and, where the CUDA runtime loads modules lazily, is also the
 * moment the library image with its 8 MiB array is loaded onto that device; make that first call during start-up, ahead
 * of any stream capture.  The address is cached per device for the life of the process: after cudaDeviceReset on a
 * device the cached address is stale and this entry point must not be used on it again.  All calls on one GPU share the array: two calls whose kernels can overlap on the GPU (different streams,
 * different threads) race on it and must be ordered by the caller.  The array keeps whatever the previous call
 * left; that is harmless because each call overwrites every partial it later reads. */
#define MOE_STATIC_MAX_DE 262144
MOE_API moe_status moe_router_wgrad_static(int64_t T, int32_t d, int32_t E, const uint16_t* x, const float* dl,
                                           float* dW_r, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H */
