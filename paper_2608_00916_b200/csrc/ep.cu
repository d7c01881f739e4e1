// Expert parallelism (EP > 1): the MoE layer with its experts spread over the ranks of an EP group, each rank keeping
// its own tokens (paper, Section "Expert-Parallel MoE Training": "MoE layers dispatch routed tokens only among the
// ranks within an EP group").
//
// Rank r of W owns the experts [r E/W, (r+1) E/W) and holds, in its OWNER workspace, the expert-major row buffers of
// every row routed to them, from whichever rank the token lives on.  The rows cross the GPUs inside this library's own
// kernels, by plain stores and loads through peer-mapped pointers (NVLink): the dispatch kernel writes each token row
// straight into the owner's buffer, the combine kernels read the owners' output rows back.  Each CTA touches only
// its own rows; there is no multicast and no library kernel is handed a peer pointer.  The only other exchange is the
// W x E table of per-rank expert counts, gathered by the caller (an all-gather of E integers per rank).
//
// Row placement.  Expert e's segment on its owner holds the rows of rank 0 first, then rank 1, ... and the rows of one
// rank in token order, so the order is the one a single GPU would produce for the concatenated batch (rank-major
// tokens).  With tot[e] the sum of the ranks' counts, the segment of e starts, on its owner, at the padded prefix
// (multiples of 128 rows) of the tot[] of that owner's experts before it; rank r's first row in it follows the rows
// of the ranks before r.
//
// Phases of a forward / backward pair (each an entry point; the caller separates them by a barrier of the group,
// because a phase reads what the previous one wrote on OTHER ranks):
//   route            router, local counts                                   -> all-gather of the counts (caller)
//   plan             placement of this rank's rows, tables of the owned experts, cleared pad rows
//   dispatch(x)      rows of x and their gates into the owners' buffers
//   expert_forward   gate/up GEMM + SwiGLU and down GEMM over the owned experts
//   combine          y from the owners' output rows
//   dispatch(dy)     rows of dy into the owners' buffers
//   expert_backward  the four backward GEMMs over the owned experts (dW of the owned experts, dg partials, dxp rows)
//   router_backward  dg from the owners, dl, dW_r, db_r, dx from the owners' dxp rows
#include <string.h>

#include "common.cuh"
#include "tables.cuh"

namespace moe {

struct EpPeers {
  char* ws[MOE_EP_MAX_RANKS];  // owner workspace of every rank of the group, as mapped into this process
};

// ---------------------------------------------------------------------------------------------- plan
// One block.  all_counts[r * E + e]: rows rank r routes to expert e.
// Every rank sees the same table, so every rank reaches the same decision on whether the rows fit: if the padded rows
// of ANY owner exceed the capacity of the owner buffers (own_rows_max rows, the same on every rank of the group), the
// whole step is refused on every rank - all destinations become -1 (nothing is dispatched, combined outputs are zero),
// the owned experts get empty tables, and the sender workspace's status word records DEV_BOUNDS.
__global__ void __launch_bounds__(256) ep_plan_kernel(const int32_t* __restrict__ all_counts, int W, int rank, int E,
                                                      int E_loc, int64_t own_rows_max, int32_t* __restrict__ dest_base,
                                                      const TableOut tabs, int32_t* __restrict__ status) {
  __shared__ int s_tot[MAX_E], s_before[MAX_E], s_cnt[MAX_E];
  __shared__ TableScratch s_tab;
  __shared__ int s_over;
  const int tid = threadIdx.x;
  if (tid == 0) s_over = 0;
  for (int e = tid; e < E; e += blockDim.x) {
    int tot = 0, before = 0;
    for (int r = 0; r < W; ++r) {
      const int c = all_counts[r * E + e];
      tot += c;
      if (r < rank) before += c;
    }
    s_tot[e] = tot;
    s_before[e] = before;
  }
  __syncthreads();
  if (tid < W) {
    int64_t rows = 0;
    for (int q = tid * E_loc; q < (tid + 1) * E_loc; ++q) rows += (s_tot[q] + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
    if (rows > own_rows_max) atomicExch(&s_over, 1);
  }
  __syncthreads();
  const bool over = s_over != 0;
  if (over && tid == 0) record_status(status, DEV_BOUNDS, 601);
  for (int e = tid; e < E; e += blockDim.x) {
    const int first = (e / E_loc) * E_loc;  // first expert of e's owner
    int pad = 0;
    for (int q = first; q < e; ++q) pad += (s_tot[q] + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
    dest_base[e] = over ? -1 : pad + s_before[e];
  }
  for (int el = tid; el < E_loc; el += blockDim.x) s_cnt[el] = over ? 0 : s_tot[rank * E_loc + el];
  __syncthreads();
  build_expert_tables(E_loc, s_cnt, s_tab, tabs);
}

// Pad rows of the owner's xp buffer: one block per owned expert.  (The pad rows of the other row buffers are
// produced as zeros by the GEMMs themselves, from zero xp rows and zero gates.)
__global__ void __launch_bounds__(256) ep_zero_pad_kernel(int d, const int32_t* __restrict__ counts,
                                                          const int32_t* __restrict__ pad_offsets,
                                                          uint16_t* __restrict__ rows) {
  const int e = blockIdx.x;
  const int64_t r0 = static_cast<int64_t>(pad_offsets[e]) + counts[e], r1 = pad_offsets[e + 1];
  uint4* dst = reinterpret_cast<uint4*>(rows + r0 * d);
  const int64_t n = (r1 - r0) * (d / 8);
  for (int64_t i = threadIdx.x; i < n; i += 256) dst[i] = make_uint4(0, 0, 0, 0);
}

// ---------------------------------------------------------------------------------------------- dispatch
// Destination row of every (token, slot) pair of this rank and its gate, stored next to that row on the owner.
// Ranks inside a token tile come from per-warp expert masks and population counts, as in the one-GPU scatter.
__global__ void __launch_bounds__(TOK_TILE) ep_scatter_kernel(int64_t T, int E, int k, int E_loc,
                                                              const int32_t* __restrict__ idx,
                                                              const int32_t* __restrict__ tile_base,
                                                              const int32_t* __restrict__ dest_base,
                                                              const float* __restrict__ gates,
                                                              int32_t* __restrict__ inv, const EpPeers peers,
                                                              size_t row_gate_off) {
  extern __shared__ uint32_t ep_masks[];  // [TOK_WARPS][E]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * TOK_TILE + tid;
  for (int i = tid; i < TOK_WARPS * E; i += TOK_TILE) ep_masks[i] = 0u;
  __syncthreads();
  if (t < T)
    for (int j = 0; j < k; ++j) atomicOr(&ep_masks[warp * E + idx[t * k + j]], 1u << lane);
  __syncthreads();
  if (t >= T) return;
  for (int j = 0; j < k; ++j) {
    const int e = idx[t * k + j];
    if (dest_base[e] < 0) {  // the plan refused the step (the rows do not fit the owner buffers)
      inv[t * k + j] = -1;
      continue;
    }
    int rank = tile_base[static_cast<int64_t>(blockIdx.x) * E + e];
    for (int w = 0; w < warp; ++w) rank += __popc(ep_masks[w * E + e]);
    rank += __popc(ep_masks[warp * E + e] & ((1u << lane) - 1u));
    const int r = dest_base[e] + rank;
    inv[t * k + j] = r;
    reinterpret_cast<float*>(peers.ws[e / E_loc] + row_gate_off)[r] = gates[t * k + j];
  }
}

// rows[owner(idx[t,j])][inv[t,j], :] = src[t, :]: one warp per token, the row is read once and written to its k
// destinations (peer stores for the experts other ranks own).
__global__ void __launch_bounds__(256) ep_scatter_rows_kernel(int64_t T, int d, int k, int E_loc,
                                                              const uint16_t* __restrict__ src,
                                                              const int32_t* __restrict__ idx,
                                                              const int32_t* __restrict__ inv, const EpPeers peers,
                                                              size_t buf_off) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n16 = d / 8;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * 8 + warp;
  if (t >= T) return;
  const uint4* s4 = reinterpret_cast<const uint4*>(src + t * d);
  for (int c0 = 0; c0 < n16; c0 += 256) {
    uint4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (c0 + lane + 32 * i < n16) v[i] = __ldg(s4 + c0 + lane + 32 * i);
    for (int j = 0; j < k; ++j) {
      if (inv[t * k + j] < 0) continue;  // refused step
      uint4* dst = reinterpret_cast<uint4*>(peers.ws[idx[t * k + j] / E_loc] + buf_off) +
                   static_cast<int64_t>(inv[t * k + j]) * n16;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (c0 + lane + 32 * i < n16) dst[c0 + lane + 32 * i] = v[i];
    }
  }
}

// ---------------------------------------------------------------------------------------------- combine
// out[t,:] = (add ? add[t,:] : 0) + sum_j rows[owner(idx[t,j])][inv[t,j], :]   (fp32 sum in slot order, one rounding).
// Forward: rows = the owners' gate-scaled o (y); backward: rows = the owners' dxp, add = the router term of dx.
__global__ void __launch_bounds__(256) ep_gather_sum_kernel(int d, int k, int E_loc, const int32_t* __restrict__ idx,
                                                            const int32_t* __restrict__ inv, const EpPeers peers,
                                                            size_t buf_off, const uint16_t* __restrict__ add,
                                                            uint16_t* __restrict__ out) {
  const int64_t t = blockIdx.x;
  __shared__ const uint16_t* srow[MAX_K];
  if (threadIdx.x < k)
    srow[threadIdx.x] = inv[t * k + threadIdx.x] < 0  // refused step: the row does not exist, it counts as zeros
                            ? nullptr
                            : reinterpret_cast<const uint16_t*>(peers.ws[idx[t * k + threadIdx.x] / E_loc] + buf_off) +
                                  static_cast<int64_t>(inv[t * k + threadIdx.x]) * d;
  __syncthreads();
  for (int c = threadIdx.x * 8; c < d; c += 256 * 8) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    if (add) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(add + t * d + c));
      unpack_bf16x2(v.x, acc[0], acc[1]);
      unpack_bf16x2(v.y, acc[2], acc[3]);
      unpack_bf16x2(v.z, acc[4], acc[5]);
      unpack_bf16x2(v.w, acc[6], acc[7]);
    }
#pragma unroll 8
    for (int j = 0; j < k; ++j) {
      if (!srow[j]) continue;
      const uint4 v = *reinterpret_cast<const uint4*>(srow[j] + c);
      float a, b;
      unpack_bf16x2(v.x, a, b); acc[0] += a; acc[1] += b;
      unpack_bf16x2(v.y, a, b); acc[2] += a; acc[3] += b;
      unpack_bf16x2(v.z, a, b); acc[4] += a; acc[5] += b;
      unpack_bf16x2(v.w, a, b); acc[6] += a; acc[7] += b;
    }
    uint4 w;
    w.x = pack_bf16x2(acc[0], acc[1]);
    w.y = pack_bf16x2(acc[2], acc[3]);
    w.z = pack_bf16x2(acc[4], acc[5]);
    w.w = pack_bf16x2(acc[6], acc[7]);
    *reinterpret_cast<uint4*>(out + t * d + c) = w;
  }
}

// dg[t,j] = sum over the dgrad-down column tiles of the partials the owner left for row inv[t,j] (slice order).
__global__ void __launch_bounds__(256) ep_gather_dg_kernel(int64_t n, int E_loc, const int32_t* __restrict__ idx,
                                                           const int32_t* __restrict__ inv, const EpPeers peers,
                                                           size_t dg_part_off, int dg_tiles, int64_t rows_max,
                                                           float* __restrict__ dg) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (i >= n) return;
  const float* part = reinterpret_cast<const float*>(peers.ws[idx[i] / E_loc] + dg_part_off);
  const int r = inv[i];
  float s = 0.f;
  if (r >= 0)
    for (int nt = 0; nt < dg_tiles; ++nt) s += part[nt * rows_max + r];
  dg[i] = s;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct EpLayouts {
  WsLayout send, own;
  int64_t T_equiv;
};
static EpLayouts ep_layouts(const moe_ctx_impl* c, int64_t T) {
  EpLayouts l;
  l.T_equiv = (c->ep_rows_cap + c->own->s.k - 1) / c->own->s.k;  // tokens that would fill rows_cap rows
  l.send = make_layout(c->s, T, /*row_buffers=*/false);
  l.own = make_layout(c->own->s, l.T_equiv);
  return l;
}
static bool peers_ok(const moe_ctx_impl* c, void* const* peer_ws) {
  if (!peer_ws) return false;
  for (int r = 0; r < c->ep_world; ++r)
    if (!peer_ws[r] || !aligned16(peer_ws[r])) return false;
  return true;
}
static EpPeers make_peers(const moe_ctx_impl* c, void* const* peer_ws) {
  EpPeers p;
  for (int r = 0; r < MOE_EP_MAX_RANKS; ++r) p.ws[r] = r < c->ep_world ? static_cast<char*>(peer_ws[r]) : nullptr;
  return p;
}

}  // namespace moe

using namespace moe;

extern "C" {

moe_status moe_ep_create(const moe_config* cfg, int32_t world, int32_t rank, int64_t rows_cap, moe_ctx** out) {
  if (!cfg || !out) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  if (world < 1 || world > MOE_EP_MAX_RANKS || rank < 0 || rank >= world || rows_cap < 0) return MOE_ERR_INVALID_ARG;
  if (cfg->E % world != 0 || cfg->E % 8 != 0) return MOE_ERR_INVALID_ARG;
  if (cfg->flags & MOE_FLAG_ROUTER_FP32) return MOE_ERR_UNSUPPORTED;  // the expert-parallel path takes a bf16 router weight
  if (rows_cap > (int64_t(1) << 30)) return MOE_ERR_UNSUPPORTED;
  moe_ctx* full = nullptr;
  moe_status rc = moe_create(cfg, &full);
  if (rc != MOE_OK) return rc;
  moe_config own_cfg = *cfg;
  own_cfg.E = cfg->E / world;
  own_cfg.top_k = cfg->top_k < own_cfg.E ? cfg->top_k : own_cfg.E;  // only enters the sizing of the owner workspace
  moe_ctx* own = nullptr;
  rc = moe_create(&own_cfg, &own);
  if (rc != MOE_OK) {
    moe_destroy(full);
    return rc;
  }
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(full);
  c->ep_world = world;
  c->ep_rank = rank;
  c->ep_rows_cap = rows_cap;
  c->own = reinterpret_cast<moe_ctx_impl*>(own);
  *out = full;
  return MOE_OK;
}

size_t moe_ep_send_workspace_bytes(const moe_ctx* ctx, int64_t T) {
  const moe_ctx_impl* c = reinterpret_cast<const moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0) return 0;
  return make_layout(c->s, T, false).total;
}

size_t moe_ep_own_workspace_bytes(const moe_ctx* ctx) {
  const moe_ctx_impl* c = reinterpret_cast<const moe_ctx_impl*>(ctx);
  if (!c || !c->own) return 0;
  return ep_layouts(c, 0).own.total;
}

moe_status moe_ep_workspace_find(const moe_ctx* ctx, int64_t T, int own_side, const char* name, size_t* offset,
                                 size_t* bytes) {
  const moe_ctx_impl* c = reinterpret_cast<const moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0) return MOE_ERR_INVALID_ARG;
  if (own_side) return moe_workspace_find(reinterpret_cast<const moe_ctx*>(c->own), ep_layouts(c, 0).T_equiv, name, offset, bytes);
  if (name && offset && bytes && strcmp(name, "ep_dest") == 0) {
    *offset = make_layout(c->s, T, false).ep_dest;
    *bytes = sizeof(int32_t) * c->s.E;
    return MOE_OK;
  }
  // the sender layout has the same tables as the one-GPU layout, without row buffers
  const WsLayout L = make_layout(c->s, T, false);
  struct Ent { const char* n; size_t off, sz; } tab[] = {
      {"counts", L.counts, sizeof(int32_t) * c->s.E}, {"logits", L.logits, sizeof(float) * T * c->s.E},
      {"idx", L.idx, sizeof(int32_t) * T * c->s.k},   {"gates", L.gates, sizeof(float) * T * c->s.k},
      {"inv", L.inv, sizeof(int32_t) * T * c->s.k},   {"dg", L.dg, sizeof(float) * T * c->s.k},
      {"dl", L.dl, sizeof(float) * T * c->s.E},       {"status", L.status, sizeof(int32_t) * 16}};
  if (!name || !offset || !bytes) return MOE_ERR_INVALID_ARG;
  for (const Ent& e : tab)
    if (strcmp(e.n, name) == 0) {
      *offset = e.off;
      *bytes = e.sz;
      return MOE_OK;
    }
  return MOE_ERR_INVALID_ARG;
}

moe_status moe_ep_route(moe_ctx* ctx, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                        int32_t* topk_idx, float* topk_w, int32_t* counts_local, float* aux_loss, void* send_ws,
                        size_t send_ws_bytes, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0 || !W_r || !counts_local || !aux_loss || !send_ws) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!x || !topk_idx || !topk_w)) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(send_ws)) return MOE_ERR_INVALID_ARG;
  const Shape& s = c->s;
  const WsLayout L = make_layout(s, T, false);
  if (send_ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  moe_status rc = ensure_device(c);
  if (rc == MOE_OK) rc = ensure_device(c->own);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(send_ws);
  launch_prepare(L, ws, st);
  if (T > 0) {
    GemmIO io;
    io.x = x; io.W_r = W_r; io.b_r = b_r;
    io.idx_out = topk_idx; io.gates_out = topk_w;
    rc = launch_grouped_gemm(c, GEMM_RT, T, L, ws, io, st);
    if (rc != MOE_OK) return rc;
  }
  launch_permute(s, T, L, ws, x, counts_local, nullptr, aux_loss, static_cast<int>(router_psum_rows(s, T, false)), st,
                 /*tables_only=*/true, /*histogram_done=*/T > 0 && router_writes_histogram(s));
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  note_forward(c, send_ws, T, FWD_EP);  // the later phases on this sender workspace must name the same T
  return MOE_OK;
}

moe_status moe_ep_plan(moe_ctx* ctx, int64_t T, const int32_t* all_counts, void* send_ws, size_t send_ws_bytes,
                       void* own_ws, size_t own_ws_bytes, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0 || !all_counts || !send_ws || !own_ws || !aligned16(own_ws)) return MOE_ERR_INVALID_ARG;
  const EpLayouts l = ep_layouts(c, T);
  if (send_ws_bytes < l.send.total || own_ws_bytes < l.own.total) return MOE_ERR_WORKSPACE;
  if (!forward_matches(c, send_ws, T, FWD_EP)) return MOE_ERR_INVALID_ARG;
  moe_status rc = ensure_device(c);
  if (rc == MOE_OK) rc = ensure_device(c->own);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ows = static_cast<char*>(own_ws);
  launch_prepare(l.own, ows, st);  // row gates of the owner buffers start at zero; status block
  const int E_loc = c->own->s.E;
  ep_plan_kernel<<<1, 256, 0, st>>>(all_counts, c->ep_world, c->ep_rank, c->s.E, E_loc, l.own.rows_max,
                                    reinterpret_cast<int32_t*>(static_cast<char*>(send_ws) + l.send.ep_dest),
                                    table_pointers(l.own, ows),
                                    reinterpret_cast<int32_t*>(static_cast<char*>(send_ws) + l.send.status));
  note_launch();
  ep_zero_pad_kernel<<<E_loc, 256, 0, st>>>(c->s.d, reinterpret_cast<const int32_t*>(ows + l.own.counts),
                                            reinterpret_cast<const int32_t*>(ows + l.own.pad_offsets),
                                            reinterpret_cast<uint16_t*>(ows + l.own.xp));
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_ep_dispatch(moe_ctx* ctx, int64_t T, const uint16_t* src, int backward, void* const* peer_own_ws,
                           void* send_ws, size_t send_ws_bytes, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0 || !send_ws || !peers_ok(c, peer_own_ws)) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!src || !aligned16(src))) return MOE_ERR_INVALID_ARG;
  const EpLayouts l = ep_layouts(c, T);
  if (send_ws_bytes < l.send.total) return MOE_ERR_WORKSPACE;
  if (!forward_matches(c, send_ws, T, FWD_EP)) return MOE_ERR_INVALID_ARG;
  if (T == 0) return MOE_OK;
  const moe_status rc = ensure_device(c);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(send_ws);
  const Shape& s = c->s;
  const EpPeers peers = make_peers(c, peer_own_ws);
  const int E_loc = c->own->s.E;
  const int32_t* idx = reinterpret_cast<const int32_t*>(ws + l.send.idx);
  int32_t* inv = reinterpret_cast<int32_t*>(ws + l.send.inv);
  if (!backward) {
    ep_scatter_kernel<<<static_cast<unsigned>(l.send.tok_tiles), TOK_TILE, sizeof(uint32_t) * TOK_WARPS * s.E, st>>>(
        T, s.E, s.k, E_loc, idx, reinterpret_cast<const int32_t*>(ws + l.send.tile_counts),
        reinterpret_cast<const int32_t*>(ws + l.send.ep_dest), reinterpret_cast<const float*>(ws + l.send.gates), inv,
        peers, l.own.row_gate);
    note_launch();
  }
  ep_scatter_rows_kernel<<<static_cast<unsigned>((T + 7) / 8), 256, 0, st>>>(T, s.d, s.k, E_loc, src, idx, inv, peers,
                                                                            backward ? l.own.o : l.own.xp);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_ep_expert_forward(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up, const uint16_t* W_down,
                                 void* own_ws, size_t own_ws_bytes, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c || !c->own || !W_gate || !W_up || !W_down || !own_ws) return MOE_ERR_INVALID_ARG;
  if (!aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(own_ws)) return MOE_ERR_INVALID_ARG;
  const EpLayouts l = ep_layouts(c, 0);
  if (own_ws_bytes < l.own.total) return MOE_ERR_WORKSPACE;
  if (c->ep_rows_cap == 0) return MOE_OK;
  moe_status rc = ensure_device(c->own);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  GemmIO io;
  io.W_gate = W_gate; io.W_up = W_up; io.W_down = W_down;
  rc = launch_grouped_gemm(c->own, GEMM_F3, l.T_equiv, l.own, static_cast<char*>(own_ws), io, st);
  if (rc == MOE_OK) rc = launch_grouped_gemm(c->own, GEMM_F4, l.T_equiv, l.own, static_cast<char*>(own_ws), io, st);
  if (rc != MOE_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_ep_combine(moe_ctx* ctx, int64_t T, void* const* peer_own_ws, const void* send_ws, size_t send_ws_bytes,
                          uint16_t* y, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0 || !send_ws || !peers_ok(c, peer_own_ws)) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!y || !aligned16(y))) return MOE_ERR_INVALID_ARG;
  const EpLayouts l = ep_layouts(c, T);
  if (send_ws_bytes < l.send.total) return MOE_ERR_WORKSPACE;
  if (!forward_matches(c, send_ws, T, FWD_EP)) return MOE_ERR_INVALID_ARG;
  if (T == 0) return MOE_OK;
  const char* ws = static_cast<const char*>(send_ws);
  ep_gather_sum_kernel<<<static_cast<unsigned>(T), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      c->s.d, c->s.k, c->own->s.E, reinterpret_cast<const int32_t*>(ws + l.send.idx),
      reinterpret_cast<const int32_t*>(ws + l.send.inv), make_peers(c, peer_own_ws), l.own.o, nullptr, y);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

static moe_status ep_expert_backward_impl(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up,
                                          const uint16_t* W_down, uint16_t* dW_gate, uint16_t* dW_up, uint16_t* dW_down,
                                          float* acc_gate, float* acc_up, float* acc_down, void* own_ws,
                                          size_t own_ws_bytes, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  const bool accumulate = acc_gate != nullptr;
  if (!c || !c->own || !W_gate || !W_up || !W_down || !own_ws) return MOE_ERR_INVALID_ARG;
  if (accumulate ? (!acc_up || !acc_down) : (!dW_gate || !dW_up || !dW_down)) return MOE_ERR_INVALID_ARG;
  if (!aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(dW_gate) || !aligned16(dW_up) ||
      !aligned16(dW_down) || !aligned16(acc_gate) || !aligned16(acc_up) || !aligned16(acc_down) || !aligned16(own_ws))
    return MOE_ERR_INVALID_ARG;
  const EpLayouts l = ep_layouts(c, 0);
  if (own_ws_bytes < l.own.total) return MOE_ERR_WORKSPACE;
  moe_status rc = ensure_device(c->own);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(own_ws);
  GemmIO io;
  io.W_gate = W_gate; io.W_up = W_up; io.W_down = W_down;
  io.dW_gate = dW_gate; io.dW_up = dW_up; io.dW_down = dW_down;
  io.dW_gate_acc = acc_gate; io.dW_up_acc = acc_up; io.dW_down_acc = acc_down;
  const bool rows = c->ep_rows_cap > 0;  // row GEMMs have no tiles without rows; the weight gradients zero-fill
  if (rows) rc = launch_grouped_gemm(c->own, GEMM_B2, l.T_equiv, l.own, ws, io, st);
  if (rc == MOE_OK) rc = launch_grouped_gemm(c->own, GEMM_B3, l.T_equiv, l.own, ws, io, st);
  if (rc == MOE_OK && rows) rc = launch_grouped_gemm(c->own, GEMM_B4, l.T_equiv, l.own, ws, io, st);
  if (rc == MOE_OK) rc = launch_grouped_gemm(c->own, GEMM_B5, l.T_equiv, l.own, ws, io, st);
  if (rc != MOE_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_ep_expert_backward(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up, const uint16_t* W_down,
                                  uint16_t* dW_gate, uint16_t* dW_up, uint16_t* dW_down, void* own_ws,
                                  size_t own_ws_bytes, void* cuda_stream) {
  if (!dW_gate || !dW_up || !dW_down) return MOE_ERR_INVALID_ARG;
  return ep_expert_backward_impl(ctx, W_gate, W_up, W_down, dW_gate, dW_up, dW_down, nullptr, nullptr, nullptr, own_ws,
                                 own_ws_bytes, cuda_stream);
}

moe_status moe_ep_expert_backward_accumulate(moe_ctx* ctx, const uint16_t* W_gate, const uint16_t* W_up,
                                             const uint16_t* W_down, float* dW_gate, float* dW_up, float* dW_down,
                                             void* own_ws, size_t own_ws_bytes, void* cuda_stream) {
  if (!dW_gate || !dW_up || !dW_down) return MOE_ERR_INVALID_ARG;
  return ep_expert_backward_impl(ctx, W_gate, W_up, W_down, nullptr, nullptr, nullptr, dW_gate, dW_up, dW_down, own_ws,
                                 own_ws_bytes, cuda_stream);
}

moe_status moe_ep_router_backward(moe_ctx* ctx, int64_t T, float d_aux, const uint16_t* x, const uint16_t* W_r,
                                  void* const* peer_own_ws, void* send_ws, size_t send_ws_bytes, uint16_t* dx,
                                  float* dW_r, float* db_r, void* cuda_stream) {
  moe_ctx_impl* c = reinterpret_cast<moe_ctx_impl*>(ctx);
  if (!c || !c->own || T < 0 || !W_r || !dW_r || !send_ws || !peers_ok(c, peer_own_ws)) return MOE_ERR_INVALID_ARG;
  if (T > 0 && (!x || !dx)) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(dx) || !aligned16(send_ws)) return MOE_ERR_INVALID_ARG;
  const EpLayouts l = ep_layouts(c, T);
  if (send_ws_bytes < l.send.total) return MOE_ERR_WORKSPACE;
  if (!forward_matches(c, send_ws, T, FWD_EP)) return MOE_ERR_INVALID_ARG;
  moe_status rc = ensure_device(c);
  if (rc != MOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(send_ws);
  const Shape& s = c->s;
  const WsLayout& L = l.send;
  const EpPeers peers = make_peers(c, peer_own_ws);
  const int E_loc = c->own->s.E;
  const int32_t* idx = reinterpret_cast<const int32_t*>(ws + L.idx);
  const int32_t* inv = reinterpret_cast<const int32_t*>(ws + L.inv);
  float* dl = reinterpret_cast<float*>(ws + L.dl);
  const int dg_tiles = 2 * ((s.f + 255) / 256);
  if (T > 0) {
    const int64_t n = T * s.k;
    ep_gather_dg_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
        n, E_loc, idx, inv, peers, l.own.dg_part, dg_tiles, l.own.rows_max, reinterpret_cast<float*>(ws + L.dg));
    note_launch();
  }
  launch_router_bwd(s, T, reinterpret_cast<const float*>(ws + L.logits), idx, reinterpret_cast<const float*>(ws + L.gates),
                    nullptr, 0, 0, inv, reinterpret_cast<float*>(ws + L.dg),
                    reinterpret_cast<const int32_t*>(ws + L.counts), d_aux, dl, reinterpret_cast<uint16_t*>(ws + L.dl_hi),
                    reinterpret_cast<uint16_t*>(ws + L.dl_lo), st);
  GemmIO io;
  io.x = x; io.W_r = W_r;
  if (T > 0) {
    rc = launch_grouped_gemm(c, GEMM_DWR, T, L, ws, io, st);
    if (rc != MOE_OK) return rc;
  }
  launch_dwr(s, T, x, dl, reinterpret_cast<float*>(ws + L.dwr_part), dW_r, db_r, T > 0, st, false);
  if (T > 0) {
    rc = launch_grouped_gemm(c, GEMM_DX, T, L, ws, io, st);
    if (rc != MOE_OK) return rc;
    ep_gather_sum_kernel<<<static_cast<unsigned>(T), 256, 0, st>>>(s.d, s.k, E_loc, idx, inv, peers, l.own.dxp,
                                                                  reinterpret_cast<const uint16_t*>(ws + L.dxr), dx);
    note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // extern "C"
