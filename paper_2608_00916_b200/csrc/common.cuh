// Shared declarations of the MoE layer library: workspace layout, launcher prototypes, small device helpers.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/moe.h"

namespace moe {

constexpr int ROW_PAD = 128;     // every expert's row segment starts and ends on a multiple of this
constexpr int TOK_TILE = 128;    // tokens per tile of the permutation (histogram / scatter blocks: 4 warps x 32); equal to
                                 // the token tile of the tensor-core router, whose epilogue writes the tile histograms
constexpr int TOK_WARPS = TOK_TILE / 32;
constexpr int ROUTER_TOK = 16;   // tokens per block in the router kernel
constexpr int MAX_E = 256;
constexpr int MAX_K = 32;
constexpr int DWR_SPLIT = 8;     // token slices of the dW_r contraction

// status word values written by kernels
constexpr int DEV_OK = 0;
constexpr int DEV_TIMEOUT = 1;
constexpr int DEV_BOUNDS = 2;
// A workspace whose status block carries this pair in words [2], [3] has been initialised by the library; anything
// else is memory the library sees for the first time (its status word is then meaningless and gets cleared).
constexpr int STATUS_COOKIE0 = 0x4D6F4531;
constexpr int STATUS_COOKIE1 = 0x62323030;

struct Shape {
  int d, E, f, k;
};

// Byte offsets of every internal buffer inside the caller's workspace (all 256-byte aligned).
struct WsLayout {
  size_t status;       // int32[16]   [0] device status (first failure sticks), [1] where it happened, [2..3] cookie
  size_t timers;       // int64[GEMM_KINDS][8] cycle counters of the GEMM roles (filled only when MOE_GEMM_TIMERS is set)
  size_t counts;       // int32[E]    rows per expert
  size_t offsets;      // int32[E+1]  exclusive scan of counts (canonical, unpadded)
  size_t pad_offsets;  // int32[E+1]  exclusive scan of counts rounded up to ROW_PAD
  size_t expert_order; // int32[E]    experts sorted by row count, largest first
  size_t sched;        // int32[8]    [0] number of 128-row tiles, [1] padded row total, [2] number of block pairs (odd
                       //             blocks included as half-empty pairs), [3] full pairs, [4] leftover single blocks
  size_t tile_expert;  // int32[max_m_tiles] expert of every 128-row tile
  size_t pair_tab;     // int32[4 * max_m_tiles] pairs of 128-row blocks of one expert: {expert, first row, blocks, 0}
  size_t fpair_tab;    // int32[4 * max_m_tiles] full pairs only (both blocks exist)
  size_t single_tab;   // int32[E] tile index of the last block of every expert with an odd number of blocks
  size_t tile_counts;  // int32[tok_tiles * E] per token-tile histogram, turned into a prefix along tiles
  size_t psum_part;    // float[router_blocks * E] per-block column sums of p
  size_t psum;         // float[E]
  size_t logits;       // float[T*E]
  size_t idx;          // int32[T*k]
  size_t gates;        // float[T*k]
  size_t inv;          // int32[T*k]  padded row of pair (t, j)
  size_t row_gate;     // float[rows_max] gate of a padded row, 0 for pad rows
  size_t dg_part;      // float[2 * ceil(f/256) * rows_max] per-row partial sums of dg, two slices per dgrad-down column tile
  size_t dg;           // float[T*k]
  size_t dl;           // float[T*E]
  size_t dl_hi, dl_lo; // bf16[T*E]   dl split into two bf16 terms (hi + lo) for the tensor-core contractions
  size_t dwr_part;     // float[DWR_SPLIT * d * E]
  size_t wr_split;     // bf16[3 * d * E]  fp32 router weight split into three bf16 terms (MOE_FLAG_ROUTER_FP32)
  size_t xp;           // bf16[rows_max * d]
  size_t hg, hu, act;  // bf16[rows_max * f]
  size_t o;            // bf16[rows_max * d]   gate-scaled o in forward, the gathered dy rows in backward
  size_t dhg, dhu;     // bf16[rows_max * f]
  size_t dxp;          // bf16[rows_max * d]
  size_t dxr;          // bf16[T * d]  router term of dx (dl W_r^T)
  size_t infer_total;  // bytes a forward-only call needs (tables, xp, act, o)
  size_t total;
  // expert-LoRA calls only (beyond `total`): 64-wide row buffers u = s xp A1, v = s act A2, w = s dy B2^T,
  // z = s (dhg B1g^T + dhu B1u^T), bf16 [rows_max, 64], columns beyond the rank are zero
  size_t lora_u, lora_v, lora_w, lora_z;
  size_t lora_total;
  size_t ep_dest;      // int32[E] expert-parallel sender: first row, in the owner's buffers, of this rank's rows of expert e
  int64_t rows_alloc;  // rows the row buffers were actually sized for (0 in a layout without row buffers)
  int64_t rows_max;    // upper bound of the padded row total for T tokens
  int64_t max_m_tiles;
  int64_t tok_tiles;
  int64_t router_blocks;
};

// row_buffers = false: the layout of a rank that only routes and combines (expert-parallel sender side): the
// expert-major row buffers and everything sized by their row count are left out
WsLayout make_layout(const Shape& s, int64_t T, bool row_buffers = true);

struct moe_ctx_impl {
  Shape s;
  int sm_count;
  int device;
  void* encode_fn;  // cuTensorMapEncodeTiled, fetched through the runtime
  int router_fp32;      // W_r is passed as fp32 (MOE_FLAG_ROUTER_FP32)
  int debug_checks;     // MOE_FLAG_DEBUG_CHECKS: index checks in the permutation / combine / router-gradient kernels
  int use_side_stream;  // backward runs the router's gradient chain on s_side, beside the big GEMMs
  int side_created;
  cudaStream_t s_side;
  cudaEvent_t ev_fork, ev_join, ev_b4;
  int tile_mode;    // 0: choose per GEMM, 1: always CTA pairs (odd blocks as half-empty pairs), 2: always one-CTA tiles,
                    // 3: row GEMMs as full pairs + one-CTA tiles for the leftover blocks, weight gradients on pairs
  int gemm_timers;  // MOE_GEMM_TIMERS was set when the context first touched its device
  int row_group_override;  // MOE_ROW_GROUP, if set (measurements of the tile order)
  int b4_pair_override;    // MOE_B4_PAIR = 0 / 1, if set (measurements: dgrad gate/up on one-CTA tiles / CTA pairs); else -1
  // cudaFuncSetAttribute (dynamic shared memory opt-in) is per device: remembered here, for the device the context is
  // bound to, per kernel family (0: one-CTA kernels, 1: CTA-pair kernels) and GEMM kind
  unsigned char attr_done[2][16];
  int profiling;
  cudaEvent_t ev[MOE_PROF_RING][MOE_NUM_STAGES][2];
  unsigned char ev_used[MOE_PROF_RING][MOE_NUM_STAGES];
  int ev_created;
  int64_t prof_step;   // forward+backward pairs recorded so far
  // moe_step_host: copy-in / copy-out streams and the events that order them against the compute stream
  cudaStream_t s_in, s_out;
  cudaEvent_t e2e_ev[6];
  cudaEvent_t pipe_ev[2][5];  // pipelined host steps, per slot: x in, dy in, forward done, backward done, results out
  int pipe_used[2];
  int e2e_created;
  int32_t* pipe_status[2];  // pinned host copies of the device status block, one per slot of the pipelined host steps
  int32_t* pipe_status_dev; // the status block those copies come from
  int64_t prof_read;   // pairs already reported by moe_stage_times
  // expert parallelism (moe_ep_* calls): this rank of ep_world ranks owns experts [ep_rank * E / ep_world, ...);
  // `own` is the context of the owner side (shape with E / ep_world experts), sized for ep_rows_cap received rows
  int ep_world, ep_rank;
  int64_t ep_rows_cap;
  moe_ctx_impl* own;
  // what the most recent forward calls of this context left in which workspace (host-side bookkeeping): a backward call
  // on a workspace found here must name the same token count and variant, else its tables would index out of range
  struct FwdRecord {
    const void* ws;
    int64_t T;
    int kind;  // FWD_TRAINING, FWD_INFERENCE, or FWD_LORA + rank
  } fwd[8];
  int fwd_next;
};
constexpr int FWD_TRAINING = 1, FWD_INFERENCE = 2, FWD_EP = 3, FWD_LORA = 16;
// Host-side record of which forward call (for the expert-parallel path: which moe_ep_route call) filled which workspace.
inline void note_forward(moe_ctx_impl* c, const void* ws, int64_t T, int kind) {
  for (auto& r : c->fwd)
    if (r.ws == ws) {
      r.T = T;
      r.kind = kind;
      return;
    }
  c->fwd[c->fwd_next] = {ws, T, kind};
  c->fwd_next = (c->fwd_next + 1) % 8;
}
// false when `ws` was last filled, by this context, for another token count or another variant of the layer
inline bool forward_matches(const moe_ctx_impl* c, const void* ws, int64_t T, int kind) {
  for (const auto& r : c->fwd)
    if (r.ws == ws) return r.T == T && r.kind == kind;
  return true;  // not on record (filled long ago or never): the caller's word stands
}

// binds the context to the current device on first use (api.cu)
moe_status ensure_device(moe_ctx_impl* c);
// ---- launchers (route.cu)
// first kernel of a forward call: zero row gates, initialise the status block of a workspace seen for the first time
void launch_prepare(const WsLayout& L, char* ws, cudaStream_t st);
void launch_router(const Shape& s, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                   const float* logits_in, float* logits, int32_t* idx, float* gates, int32_t* idx_out,
                   float* gates_out, float* logits_out, float* psum_part, cudaStream_t st);
void launch_permute(const Shape& s, int64_t T, const WsLayout& L, char* ws, const uint16_t* x, int32_t* counts_out,
                    int32_t* perm_out, float* aux_out, int psum_rows, cudaStream_t st, bool tables_only = false,
                    bool histogram_done = false, bool debug = false);
// fp32 [n] -> three bf16 terms hi, mid, lo with hi + mid + lo == w exactly (route.cu)
void launch_split_fp32(const float* w, uint16_t* hi, uint16_t* mid, uint16_t* lo, int64_t n, cudaStream_t st);
// ---- launchers (combine.cu)
// dbg_status (here and below): null, or the workspace's status word - the kernel then checks every row / expert index
// it is about to use, records DEV_BOUNDS and skips or redirects the access instead of touching memory out of range
void launch_combine(const Shape& s, int64_t T, const uint16_t* o, const float* gates, const int32_t* inv,
                    uint16_t* y, cudaStream_t st, int32_t* dbg_status = nullptr, int64_t rows_max = 0);
// rows[inv[t,j],:] = src[t,:] for every (token, slot), pad rows zeroed: xp from x, and the dy rows of backward
void launch_gather_rows(const Shape& s, int64_t T, const WsLayout& L, const char* ws, const uint16_t* src,
                        uint16_t* rows, cudaStream_t st, bool debug = false);
// dg[t,j] = sum over column tiles of dg_part[tile][inv[t,j]], then dl (fp32 and the two-term bf16 split)
void launch_router_bwd(const Shape& s, int64_t T, const float* logits, const int32_t* idx, const float* gates,
                       const float* dg_part, int dg_tiles, int64_t rows_max, const int32_t* inv, float* dg,
                       const int32_t* counts, float d_aux, float* dl, uint16_t* dl_hi, uint16_t* dl_lo,
                       cudaStream_t st, int32_t* dbg_status = nullptr);
// dg_tiles == 0: dg[t,j] has been filled by the caller (expert-parallel path) and is read instead of the partials
// SIMT dW_r (any E) and the shared partial reduction / db_r
void launch_dwr(const Shape& s, int64_t T, const uint16_t* x, const float* dl, float* part, float* dW_r,
                float* db_r, bool partials_ready, cudaStream_t st, bool accumulate = false);
void launch_unpermute_bwd(const Shape& s, int64_t T, const uint16_t* dxp, const int32_t* inv, const float* dl,
                          const uint16_t* W_r, uint16_t* dx, cudaStream_t st);
// dx[t,:] = dxr[t,:] + sum_j dxp[inv[t,j],:]  (router term already contracted on the tensor cores)
void launch_unpermute_sum(const Shape& s, int64_t T, const uint16_t* dxp, const int32_t* inv, const uint16_t* dxr,
                          uint16_t* dx, cudaStream_t st, int32_t* dbg_status = nullptr, int64_t rows_max = 0);
// ---- launchers (gemm.cu); each returns a CUDA / driver error as moe_status
enum GemmKind { GEMM_F3 = 0, GEMM_F4, GEMM_B2, GEMM_B3, GEMM_B4, GEMM_B5, GEMM_RT, GEMM_DX, GEMM_DWR, GEMM_KINDS };
// Caller tensors a grouped-GEMM launch may need besides the workspace.
struct GemmIO {
  bool save_preactivations = true;  // forward: also write hg, hu (needed by backward only)
  const uint16_t* x = nullptr;
  const uint16_t* W_r = nullptr;      // bf16 router weight, or the leading bf16 term of an fp32 one
  const uint16_t* W_r_mid = nullptr;  // fp32 router weight: the second and third bf16 terms (W = hi + mid + lo exactly)
  const uint16_t* W_r_lo = nullptr;
  const float* b_r = nullptr;
  const uint16_t* W_gate = nullptr;
  const uint16_t* W_up = nullptr;
  const uint16_t* W_down = nullptr;
  uint16_t* dW_gate = nullptr;
  uint16_t* dW_up = nullptr;
  uint16_t* dW_down = nullptr;
  uint16_t* dx = nullptr;
  int e_first = 0, e_count = 0;  // weight gradients: e_count > 0 restricts the launch to experts [e_first, e_first + e_count)
  float* dW_gate_acc = nullptr;  // accumulate mode: fp32 buffers the weight gradients are added to
  float* dW_up_acc = nullptr;
  float* dW_down_acc = nullptr;
  int32_t* idx_out = nullptr;
  float* gates_out = nullptr;
  float* logits_out = nullptr;
};
moe_status launch_grouped_gemm(moe_ctx_impl* ctx, GemmKind kind, int64_t T, const WsLayout& L, char* ws,
                               const GemmIO& io, cudaStream_t st);
struct GemmParams;
moe_status launch_pair_gemm(moe_ctx_impl* ctx, GemmKind kind, const GemmParams& p, cudaStream_t st);  // gemm2.cu
// Low-rank adapters of an expert-LoRA call (all device pointers, bf16): A1 [E,d,r], B1g / B1u [E,r,f], A2 [E,f,r],
// B2 [E,r,d]; gradients in the same shapes.
struct LoraArgs {
  int rank = 0;
  float scale = 0.f;
  const uint16_t *A1 = nullptr, *B1g = nullptr, *B1u = nullptr, *A2 = nullptr, *B2 = nullptr;
  uint16_t *dA1 = nullptr, *dB1g = nullptr, *dB1u = nullptr, *dA2 = nullptr, *dB2 = nullptr;
};
enum LoraOp {
  LORA_U = 0,  // u = s xp A1
  LORA_F3,     // [hg|hu] = xp [Wg|Wu] + u [B1g|B1u], SwiGLU epilogue
  LORA_V,      // v = s act A2
  LORA_F4,     // o = act Wd + v B2
  LORA_W,      // w = s dy_rows B2^T
  LORA_B2,     // da = dy_rows Wd^T + w A2^T, SwiGLU-backward epilogue
  LORA_DB2,    // dB2 = v^T dy_rows
  LORA_DA2,    // dA2 = act^T w
  LORA_Z,      // z = s (dhg B1g^T + dhu B1u^T)
  LORA_B4,     // dxp = dhg Wg^T + dhu Wu^T + z A1^T
  LORA_DB1,    // dB1g | dB1u = u^T [dhg | dhu]
  LORA_DA1     // dA1 = xp^T z
};
moe_status launch_lora_gemm(moe_ctx_impl* ctx, LoraOp op, int64_t T, const WsLayout& L, char* ws, const GemmIO& io,
                            const LoraArgs& lo, cudaStream_t st);

// true when the tensor-core router / dW_r / dx kernels apply (their TMA maps need E % 8 == 0)
inline bool router_on_tensor_cores(const Shape& s) { return s.E % 8 == 0; }
// true when that router's epilogue also writes the per-tile histograms of the permutation (its shared-memory form)
inline bool router_writes_histogram(const Shape& s) { return router_on_tensor_cores(s) && s.E <= 128 && s.k <= 16; }
// psum_part rows written by the router: one per warp of a 128-token tile (tensor cores) or per ROUTER_TOK tokens (SIMT)
inline int64_t router_psum_rows(const Shape& s, int64_t T, bool logits_given) {
  return (router_on_tensor_cores(s) && !logits_given) ? 4 * ((T + 127) / 128) : (T + ROUTER_TOK - 1) / ROUTER_TOK;
}

// counts kernel launches of the library (process-wide; read through moe_kernel_launches)
void note_launch(int n = 1);

// ---- device helpers
// Records a device-side failure.  The first failure sticks: later ones do not overwrite it, and no kernel ever resets
// the word (the host acknowledges it after reporting it, see moe_poll_status).
__device__ __forceinline__ void record_status(int32_t* status, int code, int where) {
  if (atomicCAS(status, DEV_OK, code) == DEV_OK) status[1] = where;
}
__device__ __forceinline__ float bf16_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);  // .x = lo (low 16 bits), .y = hi
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi) {
  lo = __uint_as_float(w << 16);
  hi = __uint_as_float(w & 0xFFFF0000u);
}

}  // namespace moe
