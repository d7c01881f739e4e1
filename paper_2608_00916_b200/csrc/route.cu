// Router (fp32 logits, softmax, top-k with lowest-index tie-break, renormalised gates) and the
// deterministic token permutation (per-tile histogram, prefix scan, stable scatter, row copy).  The router kernel here
// is the SIMT path (expert counts that are not a multiple of 8, or caller-supplied logits); otherwise the logits are
// contracted on the tensor cores (gemm.cu, kind RT).
#include <algorithm>

#include "common.cuh"
#include "tables.cuh"

namespace moe {

// ------------------------------------------------------------------------------------------ router
// One block routes ROUTER_TOK tokens.  Contraction: thread = (expert, group of 8 tokens), x staged in shared
// memory as fp32 (transposed so that the 8 tokens of a group are two float4), W_r read coalesced over
// experts.  bf16 x bf16 products are exact in fp32, so the logits are fp32 sums of exact terms.
// Then one warp per token: k rounds of (max value, lowest index) warp reduction on the logits, full
// softmax for the auxiliary loss statistics, gates = softmax over the selected logits.
constexpr int RT_CH = 256;  // columns of x staged per step

__global__ void __launch_bounds__(256) router_kernel(int64_t T, int d, int E, int k, const uint16_t* __restrict__ x,
                                                     const uint16_t* __restrict__ W_r, const float* __restrict__ b_r,
                                                     const float* __restrict__ logits_in, float* __restrict__ logits,
                                                     int32_t* __restrict__ idx, float* __restrict__ gates,
                                                     int32_t* __restrict__ idx_out, float* __restrict__ gates_out,
                                                     float* __restrict__ logits_out, float* __restrict__ psum_part) {
  extern __shared__ __align__(16) unsigned char rt_smem[];
  float* xs = reinterpret_cast<float*>(rt_smem);           // [RT_CH][ROUTER_TOK]
  float* ls = xs + RT_CH * ROUTER_TOK;                     // [ROUTER_TOK][E]
  float* pw = ls + ROUTER_TOK * E;                         // [8 warps][E]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * ROUTER_TOK;
  constexpr int TG = ROUTER_TOK / 8;
  const int items = E * TG;

  if (logits_in != nullptr) {
    for (int i = tid; i < ROUTER_TOK * E; i += 256) {
      int tok = i / E, e = i % E;
      int64_t t = t0 + tok;
      ls[i] = (t < T) ? logits_in[t * E + e] : 0.f;
    }
  } else {
    // each thread owns up to 2 items (E <= 256, TG = 2 -> at most 512 items)
    float acc[2][8];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[a][i] = 0.f;
    for (int c0 = 0; c0 < d; c0 += RT_CH) {
      __syncthreads();
      for (int i = tid; i < ROUTER_TOK * RT_CH / 2; i += 256) {
        int tok = i / (RT_CH / 2), cp = i % (RT_CH / 2);
        int64_t t = t0 + tok;
        int c = c0 + 2 * cp;
        float lo = 0.f, hi = 0.f;
        if (t < T && c < d) {
          uint32_t w = *reinterpret_cast<const uint32_t*>(x + t * d + c);
          unpack_bf16x2(w, lo, hi);
        }
        xs[(2 * cp) * ROUTER_TOK + tok] = lo;
        xs[(2 * cp + 1) * ROUTER_TOK + tok] = hi;
      }
      __syncthreads();
      const int cmax = min(RT_CH, d - c0);
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        int item = tid + a * 256;
        if (item < items) {
          int tg = item / E, e = item % E;
          const uint16_t* wp = W_r + static_cast<int64_t>(c0) * E + e;
#pragma unroll 4
          for (int c = 0; c < cmax; ++c) {
            float w = bf16_to_f32(wp[static_cast<int64_t>(c) * E]);
            const float4 xa = *reinterpret_cast<const float4*>(xs + c * ROUTER_TOK + tg * 8);
            const float4 xb = *reinterpret_cast<const float4*>(xs + c * ROUTER_TOK + tg * 8 + 4);
            acc[a][0] = fmaf(xa.x, w, acc[a][0]);
            acc[a][1] = fmaf(xa.y, w, acc[a][1]);
            acc[a][2] = fmaf(xa.z, w, acc[a][2]);
            acc[a][3] = fmaf(xa.w, w, acc[a][3]);
            acc[a][4] = fmaf(xb.x, w, acc[a][4]);
            acc[a][5] = fmaf(xb.y, w, acc[a][5]);
            acc[a][6] = fmaf(xb.z, w, acc[a][6]);
            acc[a][7] = fmaf(xb.w, w, acc[a][7]);
          }
        }
      }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      int item = tid + a * 256;
      if (item < items) {
        int tg = item / E, e = item % E;
        float b = b_r ? b_r[e] : 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) ls[(tg * 8 + i) * E + e] = acc[a][i] + b;
      }
    }
  }
  __syncthreads();

  // ---- per token: selection, softmax, gates (one warp per token)
  const int NQ = (E + 31) / 32;
  float psum_acc[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) psum_acc[q] = 0.f;
  for (int tok = warp; tok < ROUTER_TOK; tok += 8) {
    const int64_t t = t0 + tok;
    if (t >= T) break;  // warp-uniform
    float v[8];
    uint32_t taken = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      int e = lane + 32 * q;
      if (q < NQ && e < E) {
        v[q] = ls[tok * E + e];
        logits[t * E + e] = v[q];
        if (logits_out) logits_out[t * E + e] = v[q];
      } else {
        v[q] = -INFINITY;
        taken |= 1u << q;
      }
    }
    int my_e = 0;
    float my_v = 0.f, vmax = 0.f;
    for (int j = 0; j < k; ++j) {
      float bv = -INFINITY;
      int bi = 0x7FFFFFFF;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (!((taken >> q) & 1u) && (bi == 0x7FFFFFFF || v[q] > bv)) {
          bv = v[q];
          bi = lane + 32 * q;
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
        int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
        bool better = (oi != 0x7FFFFFFF) && (bi == 0x7FFFFFFF || ov > bv || (ov == bv && oi < bi));
        if (better) {
          bv = ov;
          bi = oi;
        }
      }
      if ((bi & 31) == lane) taken |= 1u << (bi >> 5);
      if (lane == j) {
        my_e = bi;
        my_v = bv;
      }
      if (j == 0) vmax = bv;
    }
    // full softmax (statistics for the auxiliary loss)
    float z = 0.f, pe[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      int e = lane + 32 * q;
      pe[q] = (q < NQ && e < E) ? expf(v[q] - vmax) : 0.f;
      z += pe[q];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(0xFFFFFFFFu, z, off);
    const float rz = 1.f / z;
#pragma unroll
    for (int q = 0; q < 8; ++q) psum_acc[q] += pe[q] * rz;
    // gates over the selection
    float ge = (lane < k) ? expf(my_v - vmax) : 0.f;
    float zs = ge;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) zs += __shfl_xor_sync(0xFFFFFFFFu, zs, off);
    if (lane < k) {
      float g = ge / zs;
      idx[t * k + lane] = my_e;
      gates[t * k + lane] = g;
      idx_out[t * k + lane] = my_e;
      gates_out[t * k + lane] = g;
    }
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    int e = lane + 32 * q;
    if (q < NQ && e < E) pw[warp * E + e] = psum_acc[q];
  }
  __syncthreads();
  for (int e = tid; e < E; e += 256) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += pw[w * E + e];
    psum_part[static_cast<int64_t>(blockIdx.x) * E + e] = s;
  }
}

void launch_router(const Shape& s, int64_t T, const uint16_t* x, const uint16_t* W_r, const float* b_r,
                   const float* logits_in, float* logits, int32_t* idx, float* gates, int32_t* idx_out,
                   float* gates_out, float* logits_out, float* psum_part, cudaStream_t st) {
  if (T == 0) return;
  const int blocks = static_cast<int>((T + ROUTER_TOK - 1) / ROUTER_TOK);
  const size_t smem = sizeof(float) * (RT_CH * ROUTER_TOK + ROUTER_TOK * s.E + 8 * s.E);
  router_kernel<<<blocks, 256, smem, st>>>(T, s.d, s.E, s.k, x, W_r, b_r, logits_in, logits, idx, gates, idx_out,
                                           gates_out, logits_out, psum_part);
  note_launch();
}

// ------------------------------------------------------------------------------------------ permutation
// Stable counting sort of the (token, slot) pairs by expert.  A token takes an expert at most once, so
// the order inside an expert is the token order.  Each warp covers 32 consecutive tokens and records, per
// expert, the 32-bit mask of its tokens that chose it (atomicOr: order-free, hence deterministic); ranks
// are population counts of mask prefixes.  Tiles of TOK_TILE tokens are combined by a column scan.
__device__ __forceinline__ void build_masks(uint32_t* masks /* [TOK_WARPS][E] */, const int32_t* __restrict__ idx, int64_t T,
                                            int E, int k, int64_t tile_t0) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < TOK_WARPS * E; i += TOK_TILE) masks[i] = 0u;
  __syncthreads();
  const int64_t t = tile_t0 + tid;
  if (t < T) {
    for (int j = 0; j < k; ++j) {
      int e = idx[t * k + j];
      atomicOr(&masks[warp * E + e], 1u << lane);
    }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(TOK_TILE) hist_kernel(int64_t T, int E, int k, const int32_t* __restrict__ idx,
                                                        int32_t* __restrict__ tile_counts) {
  extern __shared__ uint32_t hist_masks[];
  build_masks(hist_masks, idx, T, E, k, static_cast<int64_t>(blockIdx.x) * TOK_TILE);
  for (int e = threadIdx.x; e < E; e += TOK_TILE) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < TOK_WARPS; ++w) c += __popc(hist_masks[w * E + e]);
    tile_counts[static_cast<int64_t>(blockIdx.x) * E + e] = c;
  }
}

// One block: column scan of tile_counts (in place -> exclusive prefix along tiles), counts, canonical and
// padded offsets, tile -> expert table, and the auxiliary loss from the router's partial column sums of p
// (summed in a fixed order: reproducible).
constexpr int SCAN_THREADS = 1024;
__global__ void __launch_bounds__(SCAN_THREADS) scan_kernel(int64_t T, int E, int k, int tok_tiles, int psum_rows,
                                                            int32_t* __restrict__ tile_counts, const TableOut tabs,
                                                            const float* __restrict__ psum_part,
                                                            float* __restrict__ psum, int32_t* __restrict__ counts_out,
                                                            float* __restrict__ aux_out) {
  __shared__ int s_cnt[MAX_E];
  __shared__ TableScratch s_tab;
  __shared__ float s_term[MAX_E];
  __shared__ float s_ps[SCAN_THREADS];
  __shared__ int s_seg[SCAN_THREADS];
  const int tid = threadIdx.x;
  // column sums of p: G groups of threads stride over the partial rows
  const int G = SCAN_THREADS / E;
  if (tid < G * E) {
    const int g = tid / E, e = tid - g * E;
    // sixteen loads in flight per thread; the partial sums are combined in a fixed order
    float acc[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) acc[u] = 0.f;
    int b = g;
    for (; b + 15 * G < psum_rows; b += 16 * G) {
#pragma unroll
      for (int u = 0; u < 16; ++u) acc[u] += psum_part[static_cast<int64_t>(b + u * G) * E + e];
    }
    for (; b < psum_rows; b += G) acc[0] += psum_part[static_cast<int64_t>(b) * E + e];
#pragma unroll
    for (int st = 8; st >= 1; st >>= 1)
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (u < st) acc[u] += acc[u + st];
    s_ps[tid] = acc[0];
  }
  __syncthreads();
  // exclusive prefix of every expert's column of tile_counts along the tiles.  The G thread groups cut the tiles into G
  // consecutive segments; thread (g, e) sums its segment of column e (lanes of a warp touch consecutive experts, so the
  // accesses are coalesced, sixteen loads in flight), the segment totals are combined through shared memory, and a
  // second sweep over the segment writes the prefixes.  One thread per expert walking all tiles took 4 - 8 dependent
  // rounds of global loads; this takes two.
  {
    const int seg = (tok_tiles + G - 1) / G;
    const int g = tid / E, e = tid - g * E;
    const bool mine = tid < G * E;
    const int t_lo = min(tok_tiles, g * seg), t_hi = min(tok_tiles, t_lo + seg);
    int total = 0;
    if (mine) {
      for (int t0 = t_lo; t0 < t_hi; t0 += 16) {
        int c[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) c[u] = (t0 + u < t_hi) ? tile_counts[static_cast<int64_t>(t0 + u) * E + e] : 0;
#pragma unroll
        for (int u = 0; u < 16; ++u) total += c[u];
      }
      s_seg[tid] = total;
    }
    __syncthreads();
    if (mine) {
      int run = 0;
      for (int q = 0; q < g; ++q) run += s_seg[q * E + e];
      for (int t0 = t_lo; t0 < t_hi; t0 += 16) {
        int c[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) c[u] = (t0 + u < t_hi) ? tile_counts[static_cast<int64_t>(t0 + u) * E + e] : 0;
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          if (t0 + u < t_hi) tile_counts[static_cast<int64_t>(t0 + u) * E + e] = run;
          run += c[u];
        }
      }
      if (g == G - 1) s_cnt[e] = run;  // the last segment ends with the column total (empty segments pass it on)
    }
  }
  __syncthreads();
  for (int e = tid; e < E; e += SCAN_THREADS) {
    const int run = s_cnt[e];
    counts_out[e] = run;
    float ps = 0.f;
    for (int g = 0; g < G; ++g) ps += s_ps[g * E + e];
    psum[e] = ps;
    // aux term: (c_e / (T k)) * (Psum_e / T)
    s_term[e] = (T > 0) ? (static_cast<float>(run) / static_cast<float>(T * k)) * (ps / static_cast<float>(T)) : 0.f;
  }
  __syncthreads();
  if (tid >= 32 && tid < 64) {  // the second warp sums the aux terms in a fixed order while the first one scans
    const int lane = tid - 32;
    float sterm = 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) sterm += (lane * 8 + u < E) ? s_term[lane * 8 + u] : 0.f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sterm += __shfl_xor_sync(0xFFFFFFFFu, sterm, off);
    if (lane == 0) aux_out[0] = sterm * static_cast<float>(E);
  }
  build_expert_tables(E, s_cnt, s_tab, tabs);
}

__global__ void __launch_bounds__(TOK_TILE) scatter_kernel(int64_t T, int E, int k, const int32_t* __restrict__ idx,
                                                           const int32_t* __restrict__ tile_base,
                                                           const int32_t* __restrict__ offsets,
                                                           const int32_t* __restrict__ pad_offsets,
                                                           const float* __restrict__ gates,
                                                           int32_t* __restrict__ inv,
                                                           float* __restrict__ row_gate,
                                                           int32_t* __restrict__ perm_out, int32_t* dbg_status,
                                                           int64_t rows_max) {
  extern __shared__ uint32_t sc_masks[];
  const int64_t tile_t0 = static_cast<int64_t>(blockIdx.x) * TOK_TILE;
  build_masks(sc_masks, idx, T, E, k, tile_t0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t t = tile_t0 + tid;
  if (t >= T) return;
  for (int j = 0; j < k; ++j) {
    const int e = idx[t * k + j];
    if (dbg_status && (e < 0 || e >= E)) {  // debug checks: record and skip instead of touching memory out of range
      record_status(dbg_status, DEV_BOUNDS, 501);
      continue;
    }
    int rank = tile_base[static_cast<int64_t>(blockIdx.x) * E + e];
    for (int w = 0; w < warp; ++w) rank += __popc(sc_masks[w * E + e]);
    rank += __popc(sc_masks[warp * E + e] & ((1u << lane) - 1u));
    const int r = pad_offsets[e] + rank;
    if (dbg_status && (r < 0 || r >= rows_max)) {
      record_status(dbg_status, DEV_BOUNDS, 502);
      continue;
    }
    inv[t * k + j] = r;
    row_gate[r] = gates[t * k + j];
    if (perm_out) perm_out[offsets[e] + rank] = static_cast<int32_t>(t * k + j);
  }
}

// rows[inv[t,j],:] = src[t,:] for every (token, slot), and zero for the pad rows of every expert segment.
// One warp per token: the token's row is read ONCE into registers and written to its k destination rows (a
// gather by destination row re-reads each source row k times at far-apart moments; with the 0.5 GB output stream
// flowing through L2 in between, those re-reads came from DRAM: 328 MB read instead of 67 MB at the Qwen shape).
// Blocks past the token range zero the pad rows, one expert per block.
__global__ void __launch_bounds__(256) scatter_rows_kernel(int64_t T, int d, int k, int E, int tok_blocks,
                                                           const uint16_t* __restrict__ src,
                                                           const int32_t* __restrict__ inv,
                                                           const int32_t* __restrict__ counts,
                                                           const int32_t* __restrict__ pad_offsets,
                                                           uint16_t* __restrict__ rows, int32_t* dbg_status,
                                                           int64_t rows_max) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n16 = d / 8;
  if (static_cast<int>(blockIdx.x) >= tok_blocks) {
    const int e = blockIdx.x - tok_blocks;
    const int64_t r0 = static_cast<int64_t>(pad_offsets[e]) + counts[e], r1 = pad_offsets[e + 1];
    uint4* dst = reinterpret_cast<uint4*>(rows + r0 * d);
    const int64_t n = (r1 - r0) * n16;
    for (int64_t i = threadIdx.x; i < n; i += 256) dst[i] = make_uint4(0, 0, 0, 0);
    return;
  }
  const int64_t t = static_cast<int64_t>(blockIdx.x) * 8 + warp;
  if (t >= T) return;
  const uint4* s4 = reinterpret_cast<const uint4*>(src + t * d);
  for (int c0 = 0; c0 < n16; c0 += 256) {  // 256 x 16 B = 4 KB of the row per pass, 8 pieces per lane
    uint4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (c0 + lane + 32 * i < n16) v[i] = __ldg(s4 + c0 + lane + 32 * i);
    for (int j = 0; j < k; ++j) {
      const int r = inv[t * k + j];
      if (dbg_status && (r < 0 || r >= rows_max)) {
        if (lane == 0) record_status(dbg_status, DEV_BOUNDS, 503);
        continue;
      }
      uint4* dst = reinterpret_cast<uint4*>(rows + static_cast<int64_t>(r) * d);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (c0 + lane + 32 * i < n16) dst[c0 + lane + 32 * i] = v[i];
    }
  }
}

void launch_gather_rows(const Shape& s, int64_t T, const WsLayout& L, const char* ws, const uint16_t* src,
                        uint16_t* rows, cudaStream_t st, bool debug) {
  const int tok_blocks = static_cast<int>((T + 7) / 8);
  scatter_rows_kernel<<<tok_blocks + s.E, 256, 0, st>>>(
      T, s.d, s.k, s.E, tok_blocks, src, reinterpret_cast<const int32_t*>(ws + L.inv),
      reinterpret_cast<const int32_t*>(ws + L.counts), reinterpret_cast<const int32_t*>(ws + L.pad_offsets), rows,
      debug ? reinterpret_cast<int32_t*>(const_cast<char*>(ws) + L.status) : nullptr, L.rows_max);
  note_launch();
}

// First kernel of every forward call: clears the row gates (pad rows must read 0) and makes sure the workspace's status
// block is initialised.  A status block that already carries the cookie is left alone, so a failure recorded by an
// earlier call stays visible until the host has reported it; memory seen for the first time gets a clean block.
__global__ void __launch_bounds__(256) prepare_kernel(int32_t* __restrict__ status, float* __restrict__ row_gate,
                                                      int64_t rows) {
  if (blockIdx.x == 0 && threadIdx.x == 0 && (status[2] != STATUS_COOKIE0 || status[3] != STATUS_COOKIE1)) {
    status[0] = DEV_OK;
    status[1] = 0;
    status[2] = STATUS_COOKIE0;
    status[3] = STATUS_COOKIE1;
  }
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < rows; i += static_cast<int64_t>(gridDim.x) * 256)
    row_gate[i] = 0.f;
}

void launch_prepare(const WsLayout& L, char* ws, cudaStream_t st) {
  const int blocks = static_cast<int>(std::min<int64_t>(296, std::max<int64_t>(1, (L.rows_alloc + 255) / 256)));
  prepare_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<int32_t*>(ws + L.status),
                                         reinterpret_cast<float*>(ws + L.row_gate), L.rows_alloc);
  note_launch();
}

// tables_only: stop after the histogram and the scan (per-tile prefixes, counts, tables, aux loss); the expert-parallel
// path places the rows itself
// An fp32 value is the exact sum of three bf16 values (8 + 8 + 8 significand bits): the router contraction of an
// fp32 weight runs as three bf16 tensor-core products, each exact in fp32.
__global__ void __launch_bounds__(256) split_fp32_kernel(const float* __restrict__ w, uint16_t* __restrict__ hi,
                                                         uint16_t* __restrict__ mid, uint16_t* __restrict__ lo,
                                                         int64_t n) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (i >= n) return;
  const float v = w[i];
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(h);
  const __nv_bfloat16 m = __float2bfloat16_rn(r1);
  const __nv_bfloat16 l = __float2bfloat16_rn(r1 - __bfloat162float(m));
  hi[i] = *reinterpret_cast<const uint16_t*>(&h);
  mid[i] = *reinterpret_cast<const uint16_t*>(&m);
  lo[i] = *reinterpret_cast<const uint16_t*>(&l);
}

void launch_split_fp32(const float* w, uint16_t* hi, uint16_t* mid, uint16_t* lo, int64_t n, cudaStream_t st) {
  if (n == 0) return;
  split_fp32_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(w, hi, mid, lo, n);
  note_launch();
}

void launch_permute(const Shape& s, int64_t T, const WsLayout& L, char* ws, const uint16_t* x, int32_t* counts_out,
                    int32_t* perm_out, float* aux_out, int psum_rows, cudaStream_t st, bool tables_only,
                    bool histogram_done, bool debug) {
  int32_t* idx = reinterpret_cast<int32_t*>(ws + L.idx);
  int32_t* tile_counts = reinterpret_cast<int32_t*>(ws + L.tile_counts);
  const int tiles = static_cast<int>(L.tok_tiles);
  const size_t msm = sizeof(uint32_t) * TOK_WARPS * s.E;
  if (tiles > 0 && !histogram_done) {
    hist_kernel<<<tiles, TOK_TILE, msm, st>>>(T, s.E, s.k, idx, tile_counts);
    note_launch();
  }
  scan_kernel<<<1, SCAN_THREADS, 0, st>>>(T, s.E, s.k, tiles, psum_rows, tile_counts, table_pointers(L, ws),
                                 reinterpret_cast<const float*>(ws + L.psum_part),
                                 reinterpret_cast<float*>(ws + L.psum), counts_out, aux_out);
  note_launch();
  if (tiles > 0 && !tables_only) {
    scatter_kernel<<<tiles, TOK_TILE, msm, st>>>(
        T, s.E, s.k, idx, tile_counts, reinterpret_cast<const int32_t*>(ws + L.offsets),
        reinterpret_cast<const int32_t*>(ws + L.pad_offsets), reinterpret_cast<const float*>(ws + L.gates),
        reinterpret_cast<int32_t*>(ws + L.inv), reinterpret_cast<float*>(ws + L.row_gate), perm_out,
        debug ? reinterpret_cast<int32_t*>(ws + L.status) : nullptr, L.rows_max);
    note_launch();
    launch_gather_rows(s, T, L, ws, x, reinterpret_cast<uint16_t*>(ws + L.xp), st, debug);
  }
}

}  // namespace moe
