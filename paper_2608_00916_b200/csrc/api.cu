// C ABI of the MoE layer library (see include/moe.h): argument checks, workspace layout, kernel sequencing.
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <new>

#include "common.cuh"

namespace moe {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static std::atomic<long long> g_kernel_launches{0};
void note_launch(int n) { g_kernel_launches.fetch_add(n, std::memory_order_relaxed); }

WsLayout make_layout(const Shape& s, int64_t T, bool row_buffers) {
  WsLayout L;
  memset(&L, 0, sizeof(L));
  const int64_t R = T * s.k;
  L.max_m_tiles = (R + ROW_PAD - 1) / ROW_PAD + s.E;
  L.rows_max = L.max_m_tiles * ROW_PAD;
  L.rows_alloc = row_buffers ? L.rows_max : 0;
  L.tok_tiles = (T + TOK_TILE - 1) / TOK_TILE;
  L.router_blocks = (T + ROUTER_TOK - 1) / ROUTER_TOK;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  L.status = take(sizeof(int32_t) * 16);
  L.timers = take(sizeof(long long) * 16 * 8);
  L.counts = take(sizeof(int32_t) * s.E);
  L.offsets = take(sizeof(int32_t) * (s.E + 1));
  L.pad_offsets = take(sizeof(int32_t) * (s.E + 1));
  L.expert_order = take(sizeof(int32_t) * s.E);
  L.sched = take(sizeof(int32_t) * 8);
  L.tile_expert = take(sizeof(int32_t) * L.max_m_tiles);
  L.pair_tab = take(sizeof(int32_t) * 4 * L.max_m_tiles);
  L.fpair_tab = take(sizeof(int32_t) * 4 * L.max_m_tiles);
  L.single_tab = take(sizeof(int32_t) * s.E);
  L.tile_counts = take(sizeof(int32_t) * (L.tok_tiles + 1) * s.E);
  // rows: one per SIMT router block, or four (one per epilogue warp) per 128-token tile of the tensor-core router
  L.psum_part = take(sizeof(float) * (L.router_blocks + 4 * ((T + 127) / 128) + 1) * s.E);
  L.psum = take(sizeof(float) * s.E);
  L.logits = take(sizeof(float) * T * s.E);
  L.idx = take(sizeof(int32_t) * R);
  L.gates = take(sizeof(float) * R);
  L.inv = take(sizeof(int32_t) * R);
  L.ep_dest = take(sizeof(int32_t) * s.E);
  L.row_gate = take(sizeof(float) * L.rows_alloc);
  const size_t rows_d = sizeof(uint16_t) * L.rows_alloc * s.d, rows_f = sizeof(uint16_t) * L.rows_alloc * s.f;
  L.xp = take(rows_d);
  L.act = take(rows_f);
  L.o = take(rows_d);
  L.infer_total = off;  // everything above is all a forward-only call touches
  L.hg = take(rows_f);
  L.hu = take(rows_f);
  L.dg_part = take(sizeof(float) * 2 * ((s.f + 255) / 256) * L.rows_alloc);
  L.dg = take(sizeof(float) * R);
  L.dl = take(sizeof(float) * T * s.E);
  L.dl_hi = take(sizeof(uint16_t) * (T * s.E + 64));
  L.dl_lo = take(sizeof(uint16_t) * (T * s.E + 64));
  L.dwr_part = take(sizeof(float) * DWR_SPLIT * s.d * s.E);
  L.wr_split = take(sizeof(uint16_t) * 3 * (static_cast<size_t>(s.d) * s.E + 64));
  L.dhg = take(rows_f);
  L.dhu = take(rows_f);
  L.dxp = take(rows_d);
  L.dxr = take(sizeof(uint16_t) * T * s.d);
  L.total = off;
  const size_t rows64 = sizeof(uint16_t) * L.rows_alloc * 64;
  L.lora_u = take(rows64);
  L.lora_v = take(rows64);
  L.lora_w = take(rows64);
  L.lora_z = take(rows64);
  L.lora_total = off;
  return L;
}

// The first call that needs the device binds the context to the current one (SM count, tensor-map encoder, the
// per-device kernel attributes); every later call must come with the same device current.
moe_status ensure_device(moe_ctx_impl* c) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_CUDA;
  if (c->encode_fn) return dev == c->device ? MOE_OK : MOE_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return MOE_ERR_CUDA;
  if (prop.major != 10) return MOE_ERR_UNSUPPORTED;  // tcgen05 / TMEM kernels: sm_100a only, no fallback
  c->device = dev;
  c->sm_count = prop.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess)
    return MOE_ERR_CUDA;
  c->encode_fn = fn;
  c->gemm_timers = getenv("MOE_GEMM_TIMERS") != nullptr;
  c->row_group_override = getenv("MOE_ROW_GROUP") ? atoi(getenv("MOE_ROW_GROUP")) : 0;
  c->b4_pair_override = getenv("MOE_B4_PAIR") ? atoi(getenv("MOE_B4_PAIR")) : -1;
  if (c->use_side_stream) {
    if (cudaStreamCreateWithFlags(&c->s_side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_b4, cudaEventDisableTiming) != cudaSuccess)
      return MOE_ERR_CUDA;
    c->side_created = 1;
  }
  memset(c->attr_done, 0, sizeof(c->attr_done));
  return MOE_OK;
}

// Acknowledges a reported failure: the word returns to DEV_OK only if it still holds the code the host has seen.
__global__ void status_ack_kernel(int32_t* status, int seen) {
  if (atomicCAS(status, seen, DEV_OK) == seen) status[1] = 0;
}

static moe_status status_to_code(int v) {
  return v == DEV_OK ? MOE_OK : (v == DEV_BOUNDS ? MOE_ERR_DEVICE_BOUNDS : MOE_ERR_DEVICE_TIMEOUT);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct StageTimer {
  moe_ctx_impl* c;
  cudaStream_t st;
  int stage;
  StageTimer(moe_ctx_impl* c_, cudaStream_t st_, int stage_) : c(c_), st(st_), stage(stage_) {
    if (c->profiling) cudaEventRecord(c->ev[c->prof_step % MOE_PROF_RING][stage][0], st);
  }
  ~StageTimer() {
    if (c->profiling) {
      cudaEventRecord(c->ev[c->prof_step % MOE_PROF_RING][stage][1], st);
      c->ev_used[c->prof_step % MOE_PROF_RING][stage] = 1;
    }
  }
};

}  // namespace moe

using namespace moe;

extern "C" {

moe_status moe_create(const moe_config* cfg, moe_ctx** out) {
  if (!cfg || !out) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->d <= 0 || cfg->f <= 0 || cfg->d % 64 != 0 || cfg->f % 64 != 0) return MOE_ERR_INVALID_ARG;
  if (cfg->E < 1 || cfg->E > MAX_E) return MOE_ERR_INVALID_ARG;
  if (cfg->top_k < 1 || cfg->top_k > cfg->E || cfg->top_k > MAX_K) return MOE_ERR_INVALID_ARG;
  if ((cfg->flags & MOE_FLAG_ROUTER_FP32) && cfg->E % 8 != 0) return MOE_ERR_UNSUPPORTED;  // tensor-core router only
  moe_ctx_impl* c = new (std::nothrow) moe_ctx_impl;
  if (!c) return MOE_ERR_INVALID_ARG;
  memset(c, 0, sizeof(*c));
  c->s = Shape{cfg->d, cfg->E, cfg->f, cfg->top_k};
  c->device = -1;  // bound by the first call that launches work
  c->use_side_stream = (cfg->flags & MOE_FLAG_NO_SIDE_STREAM) ? 0 : 1;
  c->router_fp32 = (cfg->flags & MOE_FLAG_ROUTER_FP32) ? 1 : 0;
  c->debug_checks = (cfg->flags & MOE_FLAG_DEBUG_CHECKS) ? 1 : 0;
  c->tile_mode = (cfg->flags & MOE_FLAG_CTA_PAIR_TILES) ? 1
                 : (cfg->flags & MOE_FLAG_SINGLE_CTA_TILES) ? 2
                 : (cfg->flags & MOE_FLAG_HYBRID_TILES) ? 3 : 0;
  *out = reinterpret_cast<moe_ctx*>(c);
  return MOE_OK;
}

void moe_destroy(moe_ctx* ctx) {
  if (!ctx) return;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (c->ev_created)
    for (int r = 0; r < MOE_PROF_RING; ++r)
      for (int i = 0; i < MOE_NUM_STAGES; ++i) {
        cudaEventDestroy(c->ev[r][i][0]);
        cudaEventDestroy(c->ev[r][i][1]);
      }
  if (c->own) moe_destroy(reinterpret_cast<moe_ctx*>(c->own));
  if (c->side_created) {
    cudaStreamDestroy(c->s_side);
    cudaEventDestroy(c->ev_fork);
    cudaEventDestroy(c->ev_join);
    cudaEventDestroy(c->ev_b4);
  }
  if (c->e2e_created) {
    cudaStreamDestroy(c->s_in);
    cudaStreamDestroy(c->s_out);
    for (int i = 0; i < 6; ++i) cudaEventDestroy(c->e2e_ev[i]);
    for (int sl = 0; sl < 2; ++sl) {
      for (int i = 0; i < 5; ++i) cudaEventDestroy(c->pipe_ev[sl][i]);
      if (c->pipe_status[sl]) cudaFreeHost(c->pipe_status[sl]);
    }
  }
  delete c;
}

size_t moe_workspace_bytes(const moe_ctx* ctx, int64_t T) {
  if (!ctx || T < 0) return 0;
  const moe_ctx_impl* c = reinterpret_cast<const moe_ctx_impl*>(ctx);
  return make_layout(c->s, T).total;
}

moe_status moe_workspace_find(const moe_ctx* ctx, int64_t T, const char* name, size_t* offset, size_t* bytes) {
  if (!ctx || !name || !offset || !bytes || T < 0) return MOE_ERR_INVALID_ARG;
  const moe_ctx_impl* c = reinterpret_cast<const moe_ctx_impl*>(ctx);
  const Shape& s = c->s;
  const WsLayout L = make_layout(s, T);
  const size_t R = static_cast<size_t>(T) * s.k;
  const size_t rows_d = sizeof(uint16_t) * L.rows_max * s.d, rows_f = sizeof(uint16_t) * L.rows_max * s.f;
  struct Ent {
    const char* n;
    size_t off, sz;
  } tab[] = {{"counts", L.counts, sizeof(int32_t) * s.E},
             {"offsets", L.offsets, sizeof(int32_t) * (s.E + 1)},
             {"pad_offsets", L.pad_offsets, sizeof(int32_t) * (s.E + 1)},
             {"logits", L.logits, sizeof(float) * T * s.E},
             {"idx", L.idx, sizeof(int32_t) * R},
             {"gates", L.gates, sizeof(float) * R},
             {"inv", L.inv, sizeof(int32_t) * R},
             {"row_gate", L.row_gate, sizeof(float) * L.rows_max},
             {"xp", L.xp, rows_d},
             {"hg", L.hg, rows_f},
             {"hu", L.hu, rows_f},
             {"act", L.act, rows_f},
             {"o", L.o, rows_d},
             {"dhg", L.dhg, rows_f},
             {"dhu", L.dhu, rows_f},
             {"dxp", L.dxp, rows_d},
             {"dxr", L.dxr, sizeof(uint16_t) * T * s.d},
             {"dg", L.dg, sizeof(float) * R},
             {"dl", L.dl, sizeof(float) * T * s.E},
             {"status", L.status, sizeof(int32_t) * 16},
             {"timers", L.timers, sizeof(long long) * 16 * 8}};
  for (const Ent& e : tab)
    if (strcmp(e.n, name) == 0) {
      *offset = e.off;
      *bytes = e.sz;
      return MOE_OK;
    }
  return MOE_ERR_INVALID_ARG;
}

const char* moe_status_string(moe_status s) {
  switch (s) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_UNSUPPORTED:
      return "unsupported: the device is not sm_100a, or the shape is beyond what this entry point handles";
    case MOE_ERR_WORKSPACE: return "workspace too small";
    case MOE_ERR_CUDA: return "CUDA call failed";
    case MOE_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case MOE_ERR_DEVICE_BOUNDS: return "a device-side bounds check failed (debug checks, or expert-parallel rows beyond the owner buffers)";
  }
  return "unknown status";
}

moe_status moe_poll_status(moe_ctx* ctx, const void* workspace, void* cuda_stream) {
  if (!ctx || !workspace) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  const WsLayout L = make_layout(c->s, 0);
  int32_t st[4] = {0, 0, 0, 0};
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int32_t* dev_status = reinterpret_cast<int32_t*>(const_cast<char*>(static_cast<const char*>(workspace)) + L.status);
  if (cudaMemcpyAsync(st, dev_status, sizeof(st), cudaMemcpyDeviceToHost, s) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return MOE_ERR_CUDA;
  if (st[2] != STATUS_COOKIE0 || st[3] != STATUS_COOKIE1) return MOE_OK;  // no call has used this workspace yet
  if (st[0] == DEV_OK) return MOE_OK;
  // reported: acknowledge, so that the next failure can be recorded
  status_ack_kernel<<<1, 1, 0, s>>>(dev_status, st[0]);
  note_launch();
  if (cudaStreamSynchronize(s) != cudaSuccess) return MOE_ERR_CUDA;
  return status_to_code(st[0]);
}

int moe_ctx_device(const moe_ctx* ctx) {
  return ctx ? reinterpret_cast<const moe_ctx_impl*>(ctx)->device : -1;
}

long long moe_kernel_launches(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

// One CTA waits, with the library's bounded-wait helper cut down to a few thousand polls, on an mbarrier that
// nothing ever signals; the wait gives up, records DEV_TIMEOUT in the status word and the kernel returns normally.
__global__ void selftest_timeout_kernel(int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = static_cast<uint32_t>(__cvta_generic_to_shared(&bar));
  if (threadIdx.x == 0) {
    if (status[2] != STATUS_COOKIE0 || status[3] != STATUS_COOKIE1) {  // workspace not seen before
      status[0] = DEV_OK;
      status[1] = 0;
      status[2] = STATUS_COOKIE0;
      status[3] = STATUS_COOKIE1;
    }
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b) : "memory");
    bool done = false;
    for (int i = 0; i < 4096 && !done; ++i) {
      uint32_t ok;
      asm volatile(
          "{\n\t.reg .pred p;\n\t"
          "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(ok)
          : "r"(b), "r"(0u)
          : "memory");
      done = ok != 0;
    }
    if (!done) record_status(status, DEV_TIMEOUT, 9000);
  }
}

moe_status moe_selftest_timeout(moe_ctx* ctx, void* workspace, void* cuda_stream) {
  if (!ctx || !workspace) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  const WsLayout L = make_layout(c->s, 0);
  selftest_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + L.status));
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_set_profiling(moe_ctx* ctx, int enable) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (enable && !c->ev_created) {
    for (int r = 0; r < MOE_PROF_RING; ++r)
      for (int i = 0; i < MOE_NUM_STAGES; ++i)
        if (cudaEventCreate(&c->ev[r][i][0]) != cudaSuccess || cudaEventCreate(&c->ev[r][i][1]) != cudaSuccess)
          return MOE_ERR_CUDA;
    c->ev_created = 1;
  }
  c->profiling = enable ? 1 : 0;
  c->prof_read = c->prof_step;
  memset(c->ev_used, 0, sizeof(c->ev_used));
  return MOE_OK;
}

moe_status moe_stage_times(moe_ctx* ctx, float* ms, int32_t* steps) {
  if (!ctx || !ms || !steps) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  int64_t first = c->prof_read;
  if (c->prof_step - first > MOE_PROF_RING) first = c->prof_step - MOE_PROF_RING;
  *steps = static_cast<int32_t>(c->prof_step - first);
  for (int64_t sidx = first; sidx < c->prof_step; ++sidx) {
    const int r = static_cast<int>(sidx % MOE_PROF_RING);
    for (int i = 0; i < MOE_NUM_STAGES; ++i) {
      if (!c->ev_used[r][i]) continue;
      c->ev_used[r][i] = 0;
      if (cudaEventSynchronize(c->ev[r][i][1]) != cudaSuccess) return MOE_ERR_CUDA;
      float t = 0.f;
      if (cudaEventElapsedTime(&t, c->ev[r][i][0], c->ev[r][i][1]) != cudaSuccess) return MOE_ERR_CUDA;
      ms[i] += t;
    }
  }
  c->prof_read = c->prof_step;
  return MOE_OK;
}

static moe_status forward_impl(bool training, moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r,
                               const float* b_r, const float* logits_in, const uint16_t* W_gate,
                               const uint16_t* W_up, const uint16_t* W_down, uint16_t* y, int32_t* topk_idx,
                               float* topk_w, int32_t* expert_counts, int32_t* perm, float* aux_loss,
                               float* logits_out, void* workspace, size_t workspace_bytes, void* cuda_stream,
                               const LoraArgs* lora = nullptr) {
  if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  const Shape& s = c->s;
  if (!W_gate || !W_up || !W_down || !expert_counts || !aux_loss || !workspace) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!x || !y || !topk_idx || !topk_w || (!W_r && !logits_in))) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(y) ||
      !aligned16(workspace) || !aligned16(W_r))
    return MOE_ERR_INVALID_ARG;
  if (T * s.k > (int64_t(1) << 30)) return MOE_ERR_UNSUPPORTED;
  const WsLayout L = make_layout(s, T);
  if (workspace_bytes < (lora ? L.lora_total : (training ? L.total : L.infer_total))) return MOE_ERR_WORKSPACE;
  moe_status rc = ensure_device(c);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  GemmIO io;
  io.save_preactivations = training;
  io.x = x; io.W_r = W_r; io.b_r = b_r; io.W_gate = W_gate; io.W_up = W_up; io.W_down = W_down;
  io.idx_out = topk_idx; io.gates_out = topk_w; io.logits_out = logits_out;
  const bool tc_router = router_on_tensor_cores(s) && logits_in == nullptr;
  if (c->router_fp32 && (lora || !training)) return MOE_ERR_UNSUPPORTED;  // fp32 router weight: moe_forward / moe_backward
  launch_prepare(L, ws, st);  // before any kernel that may record a status
  if (c->router_fp32 && W_r) {
    // W_r points at fp32 values: split them into three exact bf16 terms, kept in the workspace for the backward pass
    const int64_t n = static_cast<int64_t>(s.d) * s.E, stride = n + 64;
    uint16_t* sp = reinterpret_cast<uint16_t*>(ws + L.wr_split);
    launch_split_fp32(reinterpret_cast<const float*>(W_r), sp, sp + stride, sp + 2 * stride, n, st);
    io.W_r = sp;
    io.W_r_mid = sp + stride;
    io.W_r_lo = sp + 2 * stride;
  }
  {
    StageTimer tm(c, st, 0);
    if (T > 0 && tc_router) {
      rc = launch_grouped_gemm(c, GEMM_RT, T, L, ws, io, st);
      if (rc != MOE_OK) return rc;
    } else {
      launch_router(s, T, x, W_r, b_r, logits_in, reinterpret_cast<float*>(ws + L.logits),
                    reinterpret_cast<int32_t*>(ws + L.idx), reinterpret_cast<float*>(ws + L.gates), topk_idx, topk_w,
                    logits_out, reinterpret_cast<float*>(ws + L.psum_part), st);
    }
  }
  {
    StageTimer tm(c, st, 1);
    launch_permute(s, T, L, ws, x, expert_counts, perm, aux_loss,
                   static_cast<int>(router_psum_rows(s, T, logits_in != nullptr)), st, /*tables_only=*/false,
                   /*histogram_done=*/tc_router && T > 0 && router_writes_histogram(s), c->debug_checks != 0);
  }
  if (T > 0) {
    {
      StageTimer tm(c, st, 2);
      if (lora) {
        rc = launch_lora_gemm(c, LORA_U, T, L, ws, io, *lora, st);
        if (rc == MOE_OK) rc = launch_lora_gemm(c, LORA_F3, T, L, ws, io, *lora, st);
      } else {
        rc = launch_grouped_gemm(c, GEMM_F3, T, L, ws, io, st);
      }
    }
    if (rc != MOE_OK) return rc;
    {
      StageTimer tm(c, st, 3);
      if (lora) {
        rc = launch_lora_gemm(c, LORA_V, T, L, ws, io, *lora, st);
        if (rc == MOE_OK) rc = launch_lora_gemm(c, LORA_F4, T, L, ws, io, *lora, st);
      } else {
        rc = launch_grouped_gemm(c, GEMM_F4, T, L, ws, io, st);
      }
    }
    if (rc != MOE_OK) return rc;
    {
      StageTimer tm(c, st, 4);
      launch_combine(s, T, reinterpret_cast<const uint16_t*>(ws + L.o), reinterpret_cast<const float*>(ws + L.gates),
                     reinterpret_cast<const int32_t*>(ws + L.inv), y, st,  // o already carries the gates
                     c->debug_checks ? reinterpret_cast<int32_t*>(ws + L.status) : nullptr, L.rows_max);
    }
  }
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  note_forward(c, workspace, T, lora ? FWD_LORA + lora->rank : (training ? FWD_TRAINING : FWD_INFERENCE));
  return MOE_OK;
}

moe_status moe_forward(moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                       const float* logits_in, const uint16_t* W_gate, const uint16_t* W_up,
                       const uint16_t* W_down, uint16_t* y, int32_t* topk_idx, float* topk_w,
                       int32_t* expert_counts, int32_t* perm, float* aux_loss, float* logits_out,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return forward_impl(true, ctx, T, x, W_r, b_r, logits_in, W_gate, W_up, W_down, y, topk_idx, topk_w, expert_counts,
                      perm, aux_loss, logits_out, workspace, workspace_bytes, cuda_stream);
}

moe_status moe_forward_inference(moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                                 const float* logits_in, const uint16_t* W_gate, const uint16_t* W_up,
                                 const uint16_t* W_down, uint16_t* y, int32_t* topk_idx, float* topk_w,
                                 int32_t* expert_counts, int32_t* perm, float* aux_loss, float* logits_out,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return forward_impl(false, ctx, T, x, W_r, b_r, logits_in, W_gate, W_up, W_down, y, topk_idx, topk_w, expert_counts,
                      perm, aux_loss, logits_out, workspace, workspace_bytes, cuda_stream);
}

size_t moe_inference_workspace_bytes(const moe_ctx* ctx, int64_t T) {
  if (!ctx || T < 0) return 0;
  return make_layout(reinterpret_cast<const moe_ctx_impl*>(ctx)->s, T).infer_total;
}

// acc_* non-null: accumulate mode (fp32 weight-gradient buffers are added to; dW_r / db_r are added to as well)
// n_groups > 0 (accumulate mode): the weight gradients are computed in n_groups launches over consecutive ranges of
// experts and group_events[g] / group_events[n_groups + g] are recorded on the stream when the dW_down / the dW_gate and
// dW_up slabs of range g are complete.
static moe_status backward_impl(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux, const uint16_t* x,
                                const uint16_t* W_r, const uint16_t* W_gate, const uint16_t* W_up,
                                const uint16_t* W_down, uint16_t* dx, float* dW_r, float* db_r, uint16_t* dW_gate,
                                uint16_t* dW_up, uint16_t* dW_down, float* acc_gate, float* acc_up, float* acc_down,
                                void* workspace, size_t workspace_bytes, void* cuda_stream,
                                const LoraArgs* lora = nullptr, int n_groups = 0, void* const* group_events = nullptr) {
  const bool accumulate = acc_gate != nullptr;
  if (!ctx || T < 0) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  const Shape& s = c->s;
  if (!W_r || !W_gate || !W_up || !W_down || !dW_r || !workspace) return MOE_ERR_INVALID_ARG;
  if (!lora && (accumulate ? (!acc_up || !acc_down) : (!dW_gate || !dW_up || !dW_down))) return MOE_ERR_INVALID_ARG;
  if (accumulate && (!aligned16(acc_gate) || !aligned16(acc_up) || !aligned16(acc_down))) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!dy || !x || !dx)) return MOE_ERR_INVALID_ARG;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(W_r) || !aligned16(W_gate) || !aligned16(W_up) ||
      !aligned16(W_down) || !aligned16(dx) || !aligned16(dW_gate) || !aligned16(dW_up) || !aligned16(dW_down) ||
      !aligned16(workspace))
    return MOE_ERR_INVALID_ARG;
  const WsLayout L = make_layout(s, T);
  if (workspace_bytes < (lora ? L.lora_total : L.total)) return MOE_ERR_WORKSPACE;
  // the tables in the workspace are the forward call's: another token count or a forward-only / other-variant pass
  // would send the index-driven kernels out of range
  if (!forward_matches(c, workspace, T, lora ? FWD_LORA + lora->rank : FWD_TRAINING)) return MOE_ERR_INVALID_ARG;
  moe_status rc = ensure_device(c);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  float* dl = reinterpret_cast<float*>(ws + L.dl);
  const int32_t* inv = reinterpret_cast<const int32_t*>(ws + L.inv);
  const float* gates = reinterpret_cast<const float*>(ws + L.gates);
  GemmIO io;
  io.x = x; io.W_r = W_r; io.W_gate = W_gate; io.W_up = W_up; io.W_down = W_down;
  if (c->router_fp32) {  // the three bf16 terms the forward call left in the workspace
    if (lora) return MOE_ERR_UNSUPPORTED;
    const int64_t stride = static_cast<int64_t>(s.d) * s.E + 64;
    uint16_t* sp = reinterpret_cast<uint16_t*>(static_cast<char*>(workspace) + L.wr_split);
    io.W_r = sp;
    io.W_r_mid = sp + stride;
    io.W_r_lo = sp + 2 * stride;
  }
  io.dW_gate = dW_gate; io.dW_up = dW_up; io.dW_down = dW_down; io.dx = dx;
  io.dW_gate_acc = acc_gate; io.dW_up_acc = acc_up; io.dW_down_acc = acc_down;
  const bool tc_router = router_on_tensor_cores(s);
  if (T > 0) {
    StageTimer tm(c, st, 5);
    launch_gather_rows(s, T, L, ws, dy, reinterpret_cast<uint16_t*>(ws + L.o), st, c->debug_checks != 0);
  }
  // The router's gradient chain (dl, dW_r, db_r and the router term of dx) needs only the dg partials that the
  // dgrad-down GEMM leaves behind.  It is small and latency-bound, so it runs on a second stream of the context, forked
  // after that GEMM and joined before the final unpermute, where it fills the tails of the three big GEMMs instead of
  // standing in line behind them.  Without tokens, or with MOE_FLAG_NO_SIDE_STREAM, it runs in line.
  bool forked = false;
  auto router_chain = [&]() -> moe_status {
    cudaStream_t rs = st;
    if (T > 0 && c->use_side_stream) {
      if (cudaEventRecord(c->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(c->s_side, c->ev_fork, 0) != cudaSuccess)
        return MOE_ERR_CUDA;
      rs = c->s_side;
      forked = true;
    }
    {
      StageTimer tm(c, rs, 10);
      launch_router_bwd(s, T, reinterpret_cast<const float*>(ws + L.logits), reinterpret_cast<const int32_t*>(ws + L.idx),
                        gates, reinterpret_cast<const float*>(ws + L.dg_part), 2 * ((s.f + 255) / 256), L.rows_max, inv,
                        reinterpret_cast<float*>(ws + L.dg), reinterpret_cast<const int32_t*>(ws + L.counts), d_aux, dl,
                        reinterpret_cast<uint16_t*>(ws + L.dl_hi), reinterpret_cast<uint16_t*>(ws + L.dl_lo), rs,
                        c->debug_checks ? reinterpret_cast<int32_t*>(ws + L.status) : nullptr);
    }
    {
      StageTimer tm(c, rs, 11);
      if (tc_router && T > 0) {
        const moe_status r2 = launch_grouped_gemm(c, GEMM_DWR, T, L, ws, io, rs);
        if (r2 != MOE_OK) return r2;
      }
      launch_dwr(s, T, x, dl, reinterpret_cast<float*>(ws + L.dwr_part), dW_r, db_r, tc_router && T > 0, rs, accumulate);
    }
    if (tc_router && T > 0) {
      StageTimer tm(c, rs, 13);
      const moe_status r2 = launch_grouped_gemm(c, GEMM_DX, T, L, ws, io, rs);
      if (r2 != MOE_OK) return r2;
    }
    return MOE_OK;
  };
  // dx = router term + sum of the dxp rows needs the dgrad gate/up GEMM (dxp) and the router chain (dxr), but not the
  // last weight-gradient GEMM: with the second stream it runs beside that GEMM (it is bandwidth-bound, fits on the SMs
  // next to the GEMM's CTAs and uses the DRAM bandwidth the GEMM leaves idle); the call joins the two streams at its end.
  auto finish_dx = [&](bool after_last_gemm) -> moe_status {
    if (forked == after_last_gemm) return MOE_OK;  // forked: right after the dgrad GEMM; in line: at the very end
    cudaStream_t xs = st;
    if (forked) {
      if (cudaEventRecord(c->ev_b4, st) != cudaSuccess || cudaStreamWaitEvent(c->s_side, c->ev_b4, 0) != cudaSuccess)
        return MOE_ERR_CUDA;
      xs = c->s_side;
    }
    {
      StageTimer tm(c, xs, 12);
      if (tc_router && T > 0) {
        launch_unpermute_sum(s, T, reinterpret_cast<const uint16_t*>(ws + L.dxp), inv,
                             reinterpret_cast<const uint16_t*>(ws + L.dxr), dx, xs,
                             c->debug_checks ? reinterpret_cast<int32_t*>(ws + L.status) : nullptr, L.rows_max);
      } else {
        launch_unpermute_bwd(s, T, reinterpret_cast<const uint16_t*>(ws + L.dxp), inv, dl, W_r, dx, xs);
      }
    }
    if (forked && cudaEventRecord(c->ev_join, c->s_side) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
  };
  if (lora) {
    // base weights frozen: no dW_gate / dW_up / dW_down; the adapter gradients come from skinny GEMMs
    const LoraOp seq[4][2] = {{LORA_W, LORA_B2}, {LORA_DB2, LORA_DA2}, {LORA_Z, LORA_B4}, {LORA_DB1, LORA_DA1}};
    for (int g = 0; g < 4 && rc == MOE_OK; ++g) {
      const bool row_ops = (g == 0 || g == 2);  // row GEMMs have no tiles without tokens; weight gradients zero-fill
      if (!(row_ops && T == 0)) {
        StageTimer tm(c, st, 6 + g);
        rc = launch_lora_gemm(c, seq[g][0], T, L, ws, io, *lora, st);
        if (rc == MOE_OK) rc = launch_lora_gemm(c, seq[g][1], T, L, ws, io, *lora, st);
      }
      if (g == 0 && rc == MOE_OK) rc = router_chain();
      if (g == 2 && rc == MOE_OK) rc = finish_dx(false);
    }
    if (rc != MOE_OK) return rc;
  } else {
    if (T > 0) {
      StageTimer tm(c, st, 6);
      rc = launch_grouped_gemm(c, GEMM_B2, T, L, ws, io, st);
    }
    if (rc != MOE_OK) return rc;
    rc = router_chain();
    if (rc != MOE_OK) return rc;
    // weight gradients: one launch, or one per range of experts with an event after each
    auto wgrad = [&](GemmKind kind, int ev_base) -> moe_status {
      if (n_groups <= 0) return launch_grouped_gemm(c, kind, T, L, ws, io, st);
      const int per = (s.E + n_groups - 1) / n_groups;
      for (int g = 0; g < n_groups; ++g) {
        GemmIO gio = io;
        gio.e_first = g * per;
        gio.e_count = s.E - gio.e_first < per ? s.E - gio.e_first : per;
        if (gio.e_count > 0) {
          const moe_status r2 = launch_grouped_gemm(c, kind, T, L, ws, gio, st);
          if (r2 != MOE_OK) return r2;
        }
        if (cudaEventRecord(static_cast<cudaEvent_t>(group_events[ev_base + g]), st) != cudaSuccess) return MOE_ERR_CUDA;
      }
      return MOE_OK;
    };
    {
      StageTimer tm(c, st, 7);
      rc = wgrad(GEMM_B3, 0);
    }
    if (rc != MOE_OK) return rc;
    if (T > 0) {
      StageTimer tm(c, st, 8);
      rc = launch_grouped_gemm(c, GEMM_B4, T, L, ws, io, st);
    }
    if (rc != MOE_OK) return rc;
    rc = finish_dx(false);
    if (rc != MOE_OK) return rc;
    {
      StageTimer tm(c, st, 9);
      rc = wgrad(GEMM_B5, n_groups);
    }
    if (rc != MOE_OK) return rc;
  }
  rc = finish_dx(true);
  if (rc != MOE_OK) return rc;
  if (forked && cudaStreamWaitEvent(st, c->ev_join, 0) != cudaSuccess) return MOE_ERR_CUDA;
  if (c->profiling) c->prof_step++;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_backward(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux, const uint16_t* x,
                        const uint16_t* W_r, const uint16_t* W_gate, const uint16_t* W_up,
                        const uint16_t* W_down, uint16_t* dx, float* dW_r, float* db_r, uint16_t* dW_gate,
                        uint16_t* dW_up, uint16_t* dW_down, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
  return backward_impl(ctx, T, dy, d_aux, x, W_r, W_gate, W_up, W_down, dx, dW_r, db_r, dW_gate, dW_up, dW_down, nullptr,
                       nullptr, nullptr, workspace, workspace_bytes, cuda_stream);
}

moe_status moe_backward_accumulate(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux, const uint16_t* x,
                                   const uint16_t* W_r, const uint16_t* W_gate, const uint16_t* W_up,
                                   const uint16_t* W_down, uint16_t* dx, float* dW_r, float* db_r, float* dW_gate,
                                   float* dW_up, float* dW_down, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream) {
  if (!dW_gate || !dW_up || !dW_down) return MOE_ERR_INVALID_ARG;
  return backward_impl(ctx, T, dy, d_aux, x, W_r, W_gate, W_up, W_down, dx, dW_r, db_r, nullptr, nullptr, nullptr, dW_gate,
                       dW_up, dW_down, workspace, workspace_bytes, cuda_stream);
}

moe_status moe_backward_accumulate_grouped(moe_ctx* ctx, int64_t T, const uint16_t* dy, float d_aux, const uint16_t* x,
                                           const uint16_t* W_r, const uint16_t* W_gate, const uint16_t* W_up,
                                           const uint16_t* W_down, uint16_t* dx, float* dW_r, float* db_r,
                                           float* dW_gate, float* dW_up, float* dW_down, int32_t n_groups,
                                           void* const* group_events, void* workspace, size_t workspace_bytes,
                                           void* cuda_stream) {
  if (!dW_gate || !dW_up || !dW_down || !ctx || n_groups < 1 || !group_events) return MOE_ERR_INVALID_ARG;
  if (n_groups > reinterpret_cast<moe_ctx_impl*>(ctx)->s.E) return MOE_ERR_INVALID_ARG;
  for (int g = 0; g < 2 * n_groups; ++g)
    if (!group_events[g]) return MOE_ERR_INVALID_ARG;
  return backward_impl(ctx, T, dy, d_aux, x, W_r, W_gate, W_up, W_down, dx, dW_r, db_r, nullptr, nullptr, nullptr, dW_gate,
                       dW_up, dW_down, workspace, workspace_bytes, cuda_stream, nullptr, n_groups, group_events);
}

// ------------------------------------------------------------------------------------------ expert LoRA
static bool lora_args_ok(const moe_ctx_impl* c, int32_t rank, const void* A1, const void* B1g, const void* B1u,
                         const void* A2, const void* B2) {
  (void)c;
  return rank >= 8 && rank <= 64 && rank % 8 == 0 && A1 && B1g && B1u && A2 && B2 && aligned16(A1) && aligned16(B1g) &&
         aligned16(B1u) && aligned16(A2) && aligned16(B2);
}

size_t moe_lora_workspace_bytes(const moe_ctx* ctx, int64_t T) {
  if (!ctx || T < 0) return 0;
  return make_layout(reinterpret_cast<const moe_ctx_impl*>(ctx)->s, T).lora_total;
}

moe_status moe_lora_forward(moe_ctx* ctx, int64_t T, int32_t rank, float scale, const uint16_t* x, const uint16_t* W_r,
                            const float* b_r, const uint16_t* W_gate, const uint16_t* W_up, const uint16_t* W_down,
                            const uint16_t* A1, const uint16_t* B1_gate, const uint16_t* B1_up, const uint16_t* A2,
                            const uint16_t* B2, uint16_t* y, int32_t* topk_idx, float* topk_w, int32_t* expert_counts,
                            float* aux_loss, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !lora_args_ok(reinterpret_cast<moe_ctx_impl*>(ctx), rank, A1, B1_gate, B1_up, A2, B2))
    return MOE_ERR_INVALID_ARG;
  LoraArgs lo;
  lo.rank = rank; lo.scale = scale;
  lo.A1 = A1; lo.B1g = B1_gate; lo.B1u = B1_up; lo.A2 = A2; lo.B2 = B2;
  return forward_impl(true, ctx, T, x, W_r, b_r, nullptr, W_gate, W_up, W_down, y, topk_idx, topk_w, expert_counts,
                      nullptr, aux_loss, nullptr, workspace, workspace_bytes, cuda_stream, &lo);
}

moe_status moe_lora_backward(moe_ctx* ctx, int64_t T, int32_t rank, float scale, const uint16_t* dy, float d_aux,
                             const uint16_t* x, const uint16_t* W_r, const uint16_t* W_gate, const uint16_t* W_up,
                             const uint16_t* W_down, const uint16_t* A1, const uint16_t* B1_gate,
                             const uint16_t* B1_up, const uint16_t* A2, const uint16_t* B2, uint16_t* dx, float* dW_r,
                             uint16_t* dA1, uint16_t* dB1_gate, uint16_t* dB1_up, uint16_t* dA2, uint16_t* dB2,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !lora_args_ok(reinterpret_cast<moe_ctx_impl*>(ctx), rank, A1, B1_gate, B1_up, A2, B2))
    return MOE_ERR_INVALID_ARG;
  if (!dA1 || !dB1_gate || !dB1_up || !dA2 || !dB2 || !aligned16(dA1) || !aligned16(dB1_gate) || !aligned16(dB1_up) ||
      !aligned16(dA2) || !aligned16(dB2))
    return MOE_ERR_INVALID_ARG;
  LoraArgs lo;
  lo.rank = rank; lo.scale = scale;
  lo.A1 = A1; lo.B1g = B1_gate; lo.B1u = B1_up; lo.A2 = A2; lo.B2 = B2;
  lo.dA1 = dA1; lo.dB1g = dB1_gate; lo.dB1u = dB1_up; lo.dA2 = dA2; lo.dB2 = dB2;
  return backward_impl(ctx, T, dy, d_aux, x, W_r, W_gate, W_up, W_down, dx, dW_r, nullptr, nullptr, nullptr, nullptr,
                       nullptr, nullptr, nullptr, workspace, workspace_bytes, cuda_stream, &lo);
}

// ------------------------------------------------------------------------------------------ host-buffer step
struct E2ELayout {
  size_t x, dy, y, dx, W_r, Wg, Wu, Wd, dWr, dWg, dWu, dWd, idx, gates, counts, aux, ws, total;
  size_t x1, dy1, y1, dx1, aux1;  // second slot of the pipelined host steps
};
static E2ELayout e2e_layout(const Shape& s, int64_t T) {
  E2ELayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t td = sizeof(uint16_t) * T * s.d, w = sizeof(uint16_t) * s.E * s.d * s.f;
  L.x = take(td); L.dy = take(td); L.y = take(td); L.dx = take(td);
  L.W_r = take(sizeof(uint16_t) * s.d * s.E);
  L.Wg = take(w); L.Wu = take(w); L.Wd = take(w);
  L.dWr = take(sizeof(float) * s.d * s.E);
  L.dWg = take(w); L.dWu = take(w); L.dWd = take(w);
  L.idx = take(sizeof(int32_t) * T * s.k);
  L.gates = take(sizeof(float) * T * s.k);
  L.counts = take(sizeof(int32_t) * s.E);
  L.aux = take(256);
  L.ws = take(make_layout(s, T).total);
  L.x1 = take(td); L.dy1 = take(td); L.y1 = take(td); L.dx1 = take(td);
  L.aux1 = take(256);
  L.total = off;
  return L;
}

static moe_status e2e_setup(moe_ctx_impl* c) {
  if (c->e2e_created) return MOE_OK;
  if (cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking) != cudaSuccess)
    return MOE_ERR_CUDA;
  for (int i = 0; i < 6; ++i)
    if (cudaEventCreateWithFlags(&c->e2e_ev[i], cudaEventDisableTiming) != cudaSuccess) return MOE_ERR_CUDA;
  for (int sl = 0; sl < 2; ++sl)
    for (int i = 0; i < 5; ++i)
      if (cudaEventCreateWithFlags(&c->pipe_ev[sl][i], cudaEventDisableTiming) != cudaSuccess) return MOE_ERR_CUDA;
  for (int sl = 0; sl < 2; ++sl)
    if (cudaHostAlloc(reinterpret_cast<void**>(&c->pipe_status[sl]), 4 * sizeof(int32_t), cudaHostAllocDefault) !=
        cudaSuccess)
      return MOE_ERR_CUDA;
  c->e2e_created = 1;
  return MOE_OK;
}

size_t moe_e2e_device_bytes(const moe_ctx* ctx, int64_t T) {
  if (!ctx || T < 0) return 0;
  return e2e_layout(reinterpret_cast<const moe_ctx_impl*>(ctx)->s, T).total;
}

size_t moe_e2e_workspace_offset(const moe_ctx* ctx, int64_t T) {
  if (!ctx || T < 0) return 0;
  return e2e_layout(reinterpret_cast<const moe_ctx_impl*>(ctx)->s, T).ws;
}

moe_status moe_step_host(moe_ctx* ctx, int64_t T, int copy_weights, const uint16_t* x, const uint16_t* W_r,
                         const uint16_t* W_gate, const uint16_t* W_up, const uint16_t* W_down,
                         const uint16_t* dy, float d_aux, uint16_t* y, float* aux_loss, uint16_t* dx,
                         float* dW_r, uint16_t* dW_gate, uint16_t* dW_up, uint16_t* dW_down, void* dev,
                         size_t dev_bytes, void* cuda_stream) {
  if (!ctx || T < 0 || !dev || !x || !dy || !y || !dx || !aux_loss) return MOE_ERR_INVALID_ARG;
  if (copy_weights && (!W_r || !W_gate || !W_up || !W_down || !dW_r || !dW_gate || !dW_up || !dW_down))
    return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (c->router_fp32) return MOE_ERR_UNSUPPORTED;  // the host-buffer steps carry a bf16 router weight
  const Shape& s = c->s;
  const E2ELayout L = e2e_layout(s, T);
  if (dev_bytes < L.total) return MOE_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* D = static_cast<char*>(dev);
  const size_t td = sizeof(uint16_t) * T * s.d, w = sizeof(uint16_t) * s.E * s.d * s.f;
  // Copies run on two private streams so that they overlap the compute stream: dy arrives while forward runs,
  // y leaves while backward runs; only the copy of x before forward and of dx after backward are exposed.
  if (e2e_setup(c) != MOE_OK) return MOE_ERR_CUDA;
  cudaEvent_t ev_start = c->e2e_ev[0], ev_x = c->e2e_ev[1], ev_dy = c->e2e_ev[2], ev_fwd = c->e2e_ev[3],
              ev_bwd = c->e2e_ev[4], ev_out = c->e2e_ev[5];
  bool ok = true;
  auto h2d = [&](size_t off, const void* src, size_t n) {
    ok = ok && cudaMemcpyAsync(D + off, src, n, cudaMemcpyHostToDevice, c->s_in) == cudaSuccess;
  };
  auto d2h = [&](void* dst, size_t off, size_t n) {
    ok = ok && cudaMemcpyAsync(dst, D + off, n, cudaMemcpyDeviceToHost, c->s_out) == cudaSuccess;
  };
  // everything already queued on the caller's stream comes first
  ok = ok && cudaEventRecord(ev_start, st) == cudaSuccess && cudaStreamWaitEvent(c->s_in, ev_start, 0) == cudaSuccess;
  if (copy_weights) {
    h2d(L.W_r, W_r, sizeof(uint16_t) * s.d * s.E);
    h2d(L.Wg, W_gate, w);
    h2d(L.Wu, W_up, w);
    h2d(L.Wd, W_down, w);
  }
  h2d(L.x, x, td);
  ok = ok && cudaEventRecord(ev_x, c->s_in) == cudaSuccess;
  h2d(L.dy, dy, td);
  ok = ok && cudaEventRecord(ev_dy, c->s_in) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  const size_t wsb = make_layout(s, T).total;
  auto U = [&](size_t off) { return reinterpret_cast<uint16_t*>(D + off); };
  if (cudaStreamWaitEvent(st, ev_x, 0) != cudaSuccess) return MOE_ERR_CUDA;
  moe_status rc = moe_forward(ctx, T, U(L.x), U(L.W_r), nullptr, nullptr, U(L.Wg), U(L.Wu), U(L.Wd), U(L.y),
                              reinterpret_cast<int32_t*>(D + L.idx), reinterpret_cast<float*>(D + L.gates),
                              reinterpret_cast<int32_t*>(D + L.counts), nullptr, reinterpret_cast<float*>(D + L.aux),
                              nullptr, D + L.ws, wsb, cuda_stream);
  if (rc != MOE_OK) return rc;
  ok = ok && cudaEventRecord(ev_fwd, st) == cudaSuccess && cudaStreamWaitEvent(c->s_out, ev_fwd, 0) == cudaSuccess;
  d2h(y, L.y, td);
  d2h(aux_loss, L.aux, sizeof(float));
  if (!ok || cudaStreamWaitEvent(st, ev_dy, 0) != cudaSuccess) return MOE_ERR_CUDA;
  rc = moe_backward(ctx, T, U(L.dy), d_aux, U(L.x), U(L.W_r), U(L.Wg), U(L.Wu), U(L.Wd), U(L.dx),
                    reinterpret_cast<float*>(D + L.dWr), nullptr, U(L.dWg), U(L.dWu), U(L.dWd), D + L.ws, wsb,
                    cuda_stream);
  if (rc != MOE_OK) return rc;
  ok = ok && cudaEventRecord(ev_bwd, st) == cudaSuccess && cudaStreamWaitEvent(c->s_out, ev_bwd, 0) == cudaSuccess;
  d2h(dx, L.dx, td);
  if (copy_weights) {
    d2h(dW_r, L.dWr, sizeof(float) * s.d * s.E);
    d2h(dW_gate, L.dWg, w);
    d2h(dW_up, L.dWu, w);
    d2h(dW_down, L.dWd, w);
  }
  // the caller's stream continues only after the results have left
  ok = ok && cudaEventRecord(ev_out, c->s_out) == cudaSuccess && cudaStreamWaitEvent(st, ev_out, 0) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MOE_ERR_CUDA;
  return moe_poll_status(ctx, D + L.ws, cuda_stream);
}

// Pipelined host steps: begin enqueues one step (copies in, forward, backward, copies out) for slot 0 or 1 and
// returns; end waits for that slot's results.  With two slots in flight the upload of the next batch and the
// download of the previous results overlap the current step's kernels.
moe_status moe_step_host_begin(moe_ctx* ctx, int slot, int64_t T, const uint16_t* x, const uint16_t* dy, float d_aux,
                               uint16_t* y, float* aux_loss, uint16_t* dx, void* dev, size_t dev_bytes,
                               void* cuda_stream) {
  if (!ctx || T < 0 || (slot != 0 && slot != 1) || !dev || !x || !dy || !y || !dx || !aux_loss) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (c->router_fp32) return MOE_ERR_UNSUPPORTED;
  const Shape& s = c->s;
  const E2ELayout L = e2e_layout(s, T);
  if (dev_bytes < L.total) return MOE_ERR_WORKSPACE;
  if (e2e_setup(c) != MOE_OK) return MOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* D = static_cast<char*>(dev);
  const size_t td = sizeof(uint16_t) * T * s.d;
  const size_t ox = slot ? L.x1 : L.x, ody = slot ? L.dy1 : L.dy, oy = slot ? L.y1 : L.y, odx = slot ? L.dx1 : L.dx,
               oaux = slot ? L.aux1 : L.aux;
  cudaEvent_t* ev = c->pipe_ev[slot];  // 0 x in, 1 dy in, 2 forward done, 3 backward done, 4 results out
  bool ok = true;
  // this slot's device buffers were last read by the slot's previous backward and its previous copy-out
  if (c->pipe_used[slot]) {
    ok = ok && cudaStreamWaitEvent(c->s_in, ev[3], 0) == cudaSuccess && cudaStreamWaitEvent(c->s_in, ev[4], 0) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(D + ox, x, td, cudaMemcpyHostToDevice, c->s_in) == cudaSuccess &&
       cudaEventRecord(ev[0], c->s_in) == cudaSuccess &&
       cudaMemcpyAsync(D + ody, dy, td, cudaMemcpyHostToDevice, c->s_in) == cudaSuccess &&
       cudaEventRecord(ev[1], c->s_in) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  const size_t wsb = make_layout(s, T).total;
  auto U = [&](size_t off) { return reinterpret_cast<uint16_t*>(D + off); };
  if (cudaStreamWaitEvent(st, ev[0], 0) != cudaSuccess) return MOE_ERR_CUDA;
  if (c->pipe_used[slot] && cudaStreamWaitEvent(st, ev[4], 0) != cudaSuccess) return MOE_ERR_CUDA;  // y, dx of this slot are free
  moe_status rc = moe_forward(ctx, T, U(ox), U(L.W_r), nullptr, nullptr, U(L.Wg), U(L.Wu), U(L.Wd), U(oy),
                              reinterpret_cast<int32_t*>(D + L.idx), reinterpret_cast<float*>(D + L.gates),
                              reinterpret_cast<int32_t*>(D + L.counts), nullptr, reinterpret_cast<float*>(D + oaux),
                              nullptr, D + L.ws, wsb, cuda_stream);
  if (rc != MOE_OK) return rc;
  ok = cudaEventRecord(ev[2], st) == cudaSuccess && cudaStreamWaitEvent(c->s_out, ev[2], 0) == cudaSuccess &&
       cudaMemcpyAsync(y, D + oy, td, cudaMemcpyDeviceToHost, c->s_out) == cudaSuccess &&
       cudaMemcpyAsync(aux_loss, D + oaux, sizeof(float), cudaMemcpyDeviceToHost, c->s_out) == cudaSuccess &&
       cudaStreamWaitEvent(st, ev[1], 0) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  rc = moe_backward(ctx, T, U(ody), d_aux, U(ox), U(L.W_r), U(L.Wg), U(L.Wu), U(L.Wd), U(odx),
                    reinterpret_cast<float*>(D + L.dWr), nullptr, U(L.dWg), U(L.dWu), U(L.dWd), D + L.ws, wsb,
                    cuda_stream);
  if (rc != MOE_OK) return rc;
  // the status block of the workspace travels with the slot's results
  c->pipe_status_dev = reinterpret_cast<int32_t*>(D + L.ws + make_layout(s, 0).status);
  ok = cudaEventRecord(ev[3], st) == cudaSuccess && cudaStreamWaitEvent(c->s_out, ev[3], 0) == cudaSuccess &&
       cudaMemcpyAsync(dx, D + odx, td, cudaMemcpyDeviceToHost, c->s_out) == cudaSuccess &&
       cudaMemcpyAsync(c->pipe_status[slot], c->pipe_status_dev, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost,
                       c->s_out) == cudaSuccess &&
       cudaEventRecord(ev[4], c->s_out) == cudaSuccess;
  c->pipe_used[slot] = 1;
  return ok ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_step_host_end(moe_ctx* ctx, int slot) {
  if (!ctx || (slot != 0 && slot != 1)) return MOE_ERR_INVALID_ARG;
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c->e2e_created || !c->pipe_used[slot]) return MOE_ERR_INVALID_ARG;
  if (cudaEventSynchronize(c->pipe_ev[slot][4]) != cudaSuccess) return MOE_ERR_CUDA;
  const int32_t* hs = c->pipe_status[slot];
  if (hs[2] != STATUS_COOKIE0 || hs[3] != STATUS_COOKIE1 || hs[0] == DEV_OK) return MOE_OK;
  // a kernel of this step (or an earlier, not yet reported one) recorded a failure: report it once, then acknowledge
  status_ack_kernel<<<1, 1, 0, c->s_out>>>(c->pipe_status_dev, hs[0]);
  note_launch();
  return status_to_code(hs[0]);
}

}  // extern "C"
