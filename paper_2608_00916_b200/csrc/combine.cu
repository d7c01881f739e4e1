// Bandwidth-bound stages around the grouped GEMMs: gate-weighted combine, its backward, the router
// gradient (dl, dW_r, db_r) and the unpermute-backward that assembles dx.
#include "common.cuh"

namespace moe {

// ------------------------------------------------------------------------------------------ combine
// y[t,:] = sum_{j<k} o[inv[t,j],:] where the rows of o already carry their gate (the gate-up epilogue folds it into
// the activation); fp32 accumulation in slot order, one bf16 rounding.
// One block per token; a thread owns 8 consecutive columns (16 bytes) and issues the k row loads back to back.
__global__ void __launch_bounds__(256) combine_kernel(int d, int k, const uint16_t* __restrict__ o,
                                                      const float* __restrict__ gates, const int32_t* __restrict__ inv,
                                                      uint16_t* __restrict__ y, int32_t* dbg_status, int64_t rows_max) {
  const int64_t t = blockIdx.x;
  __shared__ int sr[MAX_K];
  (void)gates;
  if (threadIdx.x < k) {
    int r = inv[t * k + threadIdx.x];
    if (dbg_status && (r < 0 || r >= rows_max)) {  // debug checks: record, and read row 0 instead of out of range
      record_status(dbg_status, DEV_BOUNDS, 504);
      r = 0;
    }
    sr[threadIdx.x] = r;
  }
  __syncthreads();
  for (int c = threadIdx.x * 8; c < d; c += 256 * 8) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll 8
    for (int j = 0; j < k; ++j) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(o + static_cast<int64_t>(sr[j]) * d + c));
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
    *reinterpret_cast<uint4*>(y + t * d + c) = w;
  }
}

void launch_combine(const Shape& s, int64_t T, const uint16_t* o, const float* gates, const int32_t* inv,
                    uint16_t* y, cudaStream_t st, int32_t* dbg_status, int64_t rows_max) {
  if (T == 0) return;
  combine_kernel<<<static_cast<unsigned>(T), 256, 0, st>>>(s.d, s.k, o, gates, inv, y, dbg_status, rows_max);
  note_launch();
}

// ------------------------------------------------------------------------------------------ router backward
// One warp per token.  p is recomputed from the saved logits; dg[t,j] = <dy[t], o_tj> arrives as per-row partial
// sums written by the dgrad-down epilogue (one slice per column tile) and is summed here in slice order.
//   dl[t,e]  = p_e (dp_e - <p, dp>)                       auxiliary loss through P_e, dp_e = d_aux E c_e / (T k) / T
//   dl[t,idx_j] += g_j (dg_j - sum_j' g_j' dg_j')         gates = softmax over the selected logits
__global__ void __launch_bounds__(256) router_bwd_kernel(int64_t T, int E, int k, const float* __restrict__ logits,
                                                         const int32_t* __restrict__ idx,
                                                         const float* __restrict__ gates,
                                                         const float* __restrict__ dg_part, int dg_tiles,
                                                         int64_t rows_max, const int32_t* __restrict__ inv,
                                                         float* __restrict__ dg,
                                                         const int32_t* __restrict__ counts, float d_aux,
                                                         float* __restrict__ dl, uint16_t* __restrict__ dl_hi,
                                                         uint16_t* __restrict__ dl_lo, int32_t* dbg_status) {
  const int lane = threadIdx.x & 31;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (t >= T) return;
  const int NQ = (E + 31) / 32;
  float v[8], dp[8];
  float vmax = -INFINITY;
  const float scale = d_aux * static_cast<float>(E) / (static_cast<float>(T) * static_cast<float>(k)) /
                      static_cast<float>(T);
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    int e = lane + 32 * q;
    bool ok = q < NQ && e < E;
    v[q] = ok ? logits[t * E + e] : -INFINITY;
    dp[q] = ok ? scale * static_cast<float>(counts[e]) : 0.f;
    vmax = fmaxf(vmax, v[q]);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xFFFFFFFFu, vmax, off));
  float z = 0.f, pd = 0.f, p[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    p[q] = (v[q] == -INFINITY) ? 0.f : expf(v[q] - vmax);
    z += p[q];
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(0xFFFFFFFFu, z, off);
  const float rz = 1.f / z;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    p[q] *= rz;
    pd = fmaf(p[q], dp[q], pd);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) pd += __shfl_xor_sync(0xFFFFFFFFu, pd, off);
  float out[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) out[q] = p[q] * (dp[q] - pd);
  // selected slots
  float g = 0.f, dgj = 0.f;
  int ej = -1;
  if (lane < k) {
    g = gates[t * k + lane];
    ej = idx[t * k + lane];
    if (dbg_status && (ej < 0 || ej >= E)) {  // debug checks
      record_status(dbg_status, DEV_BOUNDS, 506);
      ej = 0;
    }
    if (dg_tiles > 0) {
      int r = inv[t * k + lane];
      if (dbg_status && (r < 0 || r >= rows_max)) {
        record_status(dbg_status, DEV_BOUNDS, 507);
        r = 0;
      }
      for (int nt = 0; nt < dg_tiles; ++nt) dgj += dg_part[nt * rows_max + r];
      dg[t * k + lane] = dgj;
    } else {
      dgj = dg[t * k + lane];  // gathered by the caller (expert-parallel path: the partials live on the owner ranks)
    }
  }
  float inner = g * dgj;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) inner += __shfl_xor_sync(0xFFFFFFFFu, inner, off);
  const float mine = g * (dgj - inner);
  for (int j = 0; j < k; ++j) {
    const int e = __shfl_sync(0xFFFFFFFFu, ej, j);
    const float val = __shfl_sync(0xFFFFFFFFu, mine, j);
    if ((e & 31) == lane) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (q == (e >> 5)) out[q] += val;
    }
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    int e = lane + 32 * q;
    if (q < NQ && e < E) {
      dl[t * E + e] = out[q];
      // exact two-term bf16 split (hi + lo reproduces dl to about 2^-17 relative) for the tensor-core contractions
      const __nv_bfloat16 h = __float2bfloat16_rn(out[q]);
      const __nv_bfloat16 l = __float2bfloat16_rn(out[q] - __bfloat162float(h));
      dl_hi[t * E + e] = *reinterpret_cast<const uint16_t*>(&h);
      dl_lo[t * E + e] = *reinterpret_cast<const uint16_t*>(&l);
    }
  }
}

void launch_router_bwd(const Shape& s, int64_t T, const float* logits, const int32_t* idx, const float* gates,
                       const float* dg_part, int dg_tiles, int64_t rows_max, const int32_t* inv, float* dg,
                       const int32_t* counts, float d_aux, float* dl, uint16_t* dl_hi, uint16_t* dl_lo,
                       cudaStream_t st, int32_t* dbg_status) {
  if (T == 0) return;
  router_bwd_kernel<<<static_cast<unsigned>((T + 7) / 8), 256, 0, st>>>(T, s.E, s.k, logits, idx, gates, dg_part,
                                                                        dg_tiles, rows_max, inv, dg, counts, d_aux, dl,
                                                                        dl_hi, dl_lo, dbg_status);
  note_launch();
}

// ------------------------------------------------------------------------------------------ dW_r, db_r
// dW_r[c,e] = sum_t x[t,c] dl[t,e].  Grid (d/64, DWR_SPLIT): a block owns 64 rows of dW_r and one slice of the
// tokens, accumulates a 64 x E tile in registers (thread = 4 rows x E/16... columns) and writes a partial;
// a second kernel adds the DWR_SPLIT partials in fixed order (no atomics, reproducible).
constexpr int DW_BM = 64, DW_BK = 32;

__global__ void __launch_bounds__(256) dwr_partial_kernel(int64_t T, int d, int E, const uint16_t* __restrict__ x,
                                                          const float* __restrict__ dl, float* __restrict__ part) {
  // thread layout: 16 (row groups of 4) x 16 (column groups); columns handled: cg + 16*i for i < E/16 (<= 16)
  __shared__ float xs[DW_BK][DW_BM];        // x^T tile
  extern __shared__ float dls[];            // [DW_BK][E]
  const int tid = threadIdx.x;
  const int rg = tid / 16, cg = tid % 16;
  const int c0 = blockIdx.x * DW_BM;
  const int64_t per = (T + DWR_SPLIT - 1) / DWR_SPLIT;
  const int64_t tb = per * blockIdx.y, te = min(T, tb + per);
  const int NC = (E + 15) / 16;  // <= 16
  float acc[4][16];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 16; ++j) acc[i][j] = 0.f;
  for (int64_t t0 = tb; t0 < te; t0 += DW_BK) {
    __syncthreads();
    for (int i = tid; i < DW_BK * DW_BM / 2; i += 256) {
      int kk = i / (DW_BM / 2), cp = i % (DW_BM / 2);
      int64_t t = t0 + kk;
      float lo = 0.f, hi = 0.f;
      if (t < te) unpack_bf16x2(*reinterpret_cast<const uint32_t*>(x + t * d + c0 + 2 * cp), lo, hi);
      xs[kk][2 * cp] = lo;
      xs[kk][2 * cp + 1] = hi;
    }
    for (int i = tid; i < DW_BK * E; i += 256) {
      int kk = i / E, e = i % E;
      int64_t t = t0 + kk;
      dls[i] = (t < te) ? dl[t * E + e] : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int kk = 0; kk < DW_BK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&xs[kk][rg * 4]);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (j < NC) {
          int e = cg + 16 * j;
          float b = (e < E) ? dls[kk * E + e] : 0.f;
          acc[0][j] = fmaf(a.x, b, acc[0][j]);
          acc[1][j] = fmaf(a.y, b, acc[1][j]);
          acc[2][j] = fmaf(a.z, b, acc[2][j]);
          acc[3][j] = fmaf(a.w, b, acc[3][j]);
        }
      }
    }
  }
  float* dst = part + static_cast<int64_t>(blockIdx.y) * d * E;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      int e = cg + 16 * j;
      if (j < NC && e < E) dst[static_cast<int64_t>(c0 + rg * 4 + i) * E + e] = acc[i][j];
    }
}

__global__ void dwr_reduce_kernel(int64_t n, const float* __restrict__ part, float* __restrict__ dW_r,
                                  int accumulate) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
#pragma unroll
  for (int sl = 0; sl < DWR_SPLIT; ++sl) s += part[sl * n + i];
  dW_r[i] = accumulate ? dW_r[i] + s : s;
}

// db_r[e] = sum_t dl[t,e]: one block per 32 experts, 8 warps stride over the tokens, fixed-order final sum.
__global__ void __launch_bounds__(256) dbr_kernel(int64_t T, int E, const float* __restrict__ dl,
                                                  float* __restrict__ db_r, int accumulate) {
  __shared__ float part[8][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int e = blockIdx.x * 32 + lane;
  float s = 0.f;
  if (e < E)
    for (int64_t t = warp; t < T; t += 8) s += dl[t * E + e];
  part[warp][lane] = s;
  __syncthreads();
  if (warp == 0 && e < E) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) a += part[w][lane];
    db_r[e] = accumulate ? db_r[e] + a : a;
  }
}

void launch_dwr(const Shape& s, int64_t T, const uint16_t* x, const float* dl, float* part, float* dW_r,
                float* db_r, bool partials_ready, cudaStream_t st, bool accumulate) {
  const int64_t n = static_cast<int64_t>(s.d) * s.E;
  if (!partials_ready) {
    dim3 grid(s.d / DW_BM, DWR_SPLIT);
    dwr_partial_kernel<<<grid, 256, sizeof(float) * DW_BK * s.E, st>>>(T, s.d, s.E, x, dl, part);
    note_launch();
  }
  dwr_reduce_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(n, part, dW_r, accumulate ? 1 : 0);
  note_launch();
  if (db_r) {
    dbr_kernel<<<(s.E + 31) / 32, 256, 0, st>>>(T, s.E, dl, db_r, accumulate ? 1 : 0);
    note_launch();
  }
}

// ------------------------------------------------------------------------------------------ unpermute backward
// dx[t,c] = sum_j dxp[inv[t,j], c] + sum_e dl[t,e] W_r[c,e].  A block handles UB_TOK tokens; a thread owns 8
// consecutive columns per pass and reads its W_r rows once for all tokens of the block.
constexpr int UB_TOK = 8;

__global__ void __launch_bounds__(256) unpermute_bwd_kernel(int64_t T, int d, int E, int k,
                                                            const uint16_t* __restrict__ dxp,
                                                            const int32_t* __restrict__ inv,
                                                            const float* __restrict__ dl,
                                                            const uint16_t* __restrict__ W_r,
                                                            uint16_t* __restrict__ dx) {
  extern __shared__ float ub_dl[];  // [UB_TOK][E]
  __shared__ int s_inv[UB_TOK][MAX_K];
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * UB_TOK;
  for (int i = threadIdx.x; i < UB_TOK * E; i += 256) {
    int64_t t = t0 + i / E;
    ub_dl[i] = (t < T) ? dl[t * E + (i % E)] : 0.f;
  }
  for (int i = threadIdx.x; i < UB_TOK * k; i += 256) {
    int64_t t = t0 + i / k;
    s_inv[i / k][i % k] = (t < T) ? inv[t * k + (i % k)] : 0;
  }
  __syncthreads();
  for (int c = threadIdx.x * 8; c < d; c += 256 * 8) {
    float acc[UB_TOK][8];
#pragma unroll
    for (int tk = 0; tk < UB_TOK; ++tk)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[tk][i] = 0.f;
    // router term: rows c..c+7 of W_r, E contiguous bf16 each (vector path needs E % 8 == 0)
    if ((E & 7) != 0) {
      for (int e = 0; e < E; ++e) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float w = bf16_to_f32(W_r[static_cast<int64_t>(c + i) * E + e]);
#pragma unroll
          for (int tk = 0; tk < UB_TOK; ++tk) acc[tk][i] = fmaf(ub_dl[tk * E + e], w, acc[tk][i]);
        }
      }
    } else
    for (int e0 = 0; e0 < E; e0 += 8) {
      float w[8][8];  // [col][e]
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(W_r + static_cast<int64_t>(c + i) * E + e0));
        unpack_bf16x2(v.x, w[i][0], w[i][1]);
        unpack_bf16x2(v.y, w[i][2], w[i][3]);
        unpack_bf16x2(v.z, w[i][4], w[i][5]);
        unpack_bf16x2(v.w, w[i][6], w[i][7]);
      }
#pragma unroll
      for (int tk = 0; tk < UB_TOK; ++tk) {
        const float4 da = *reinterpret_cast<const float4*>(ub_dl + tk * E + e0);
        const float4 db = *reinterpret_cast<const float4*>(ub_dl + tk * E + e0 + 4);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float s = acc[tk][i];
          s = fmaf(da.x, w[i][0], s);
          s = fmaf(da.y, w[i][1], s);
          s = fmaf(da.z, w[i][2], s);
          s = fmaf(da.w, w[i][3], s);
          s = fmaf(db.x, w[i][4], s);
          s = fmaf(db.y, w[i][5], s);
          s = fmaf(db.z, w[i][6], s);
          s = fmaf(db.w, w[i][7], s);
          acc[tk][i] = s;
        }
      }
    }
#pragma unroll
    for (int tk = 0; tk < UB_TOK; ++tk) {
      const int64_t t = t0 + tk;
      if (t < T) {
        for (int j = 0; j < k; ++j) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(dxp + static_cast<int64_t>(s_inv[tk][j]) * d + c));
          float a, b;
          unpack_bf16x2(v.x, a, b); acc[tk][0] += a; acc[tk][1] += b;
          unpack_bf16x2(v.y, a, b); acc[tk][2] += a; acc[tk][3] += b;
          unpack_bf16x2(v.z, a, b); acc[tk][4] += a; acc[tk][5] += b;
          unpack_bf16x2(v.w, a, b); acc[tk][6] += a; acc[tk][7] += b;
        }
        uint4 w4;
        w4.x = pack_bf16x2(acc[tk][0], acc[tk][1]);
        w4.y = pack_bf16x2(acc[tk][2], acc[tk][3]);
        w4.z = pack_bf16x2(acc[tk][4], acc[tk][5]);
        w4.w = pack_bf16x2(acc[tk][6], acc[tk][7]);
        *reinterpret_cast<uint4*>(dx + t * d + c) = w4;
      }
    }
  }
}

// dx[t,:] = dxr[t,:] + sum_j dxp[inv[t,j],:]; one block per token, 16-byte accesses, all row loads in flight at once.
__global__ void __launch_bounds__(256) unpermute_sum_kernel(int d, int k, const uint16_t* __restrict__ dxp,
                                                            const int32_t* __restrict__ inv,
                                                            const uint16_t* __restrict__ dxr,
                                                            uint16_t* __restrict__ dx, int32_t* dbg_status,
                                                            int64_t rows_max) {
  const int64_t t = blockIdx.x;
  __shared__ int sr[MAX_K];
  if (threadIdx.x < k) {
    int r = inv[t * k + threadIdx.x];
    if (dbg_status && (r < 0 || r >= rows_max)) {
      record_status(dbg_status, DEV_BOUNDS, 505);
      r = 0;
    }
    sr[threadIdx.x] = r;
  }
  __syncthreads();
  for (int c = threadIdx.x * 8; c < d; c += 256 * 8) {
    float acc[8];
    {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(dxr + t * d + c));
      unpack_bf16x2(v.x, acc[0], acc[1]);
      unpack_bf16x2(v.y, acc[2], acc[3]);
      unpack_bf16x2(v.z, acc[4], acc[5]);
      unpack_bf16x2(v.w, acc[6], acc[7]);
    }
#pragma unroll 8
    for (int j = 0; j < k; ++j) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(dxp + static_cast<int64_t>(sr[j]) * d + c));
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
    *reinterpret_cast<uint4*>(dx + t * d + c) = w;
  }
}

void launch_unpermute_sum(const Shape& s, int64_t T, const uint16_t* dxp, const int32_t* inv, const uint16_t* dxr,
                          uint16_t* dx, cudaStream_t st, int32_t* dbg_status, int64_t rows_max) {
  if (T == 0) return;
  unpermute_sum_kernel<<<static_cast<unsigned>(T), 256, 0, st>>>(s.d, s.k, dxp, inv, dxr, dx, dbg_status, rows_max);
  note_launch();
}

void launch_unpermute_bwd(const Shape& s, int64_t T, const uint16_t* dxp, const int32_t* inv, const float* dl,
                          const uint16_t* W_r, uint16_t* dx, cudaStream_t st) {
  if (T == 0) return;
  unpermute_bwd_kernel<<<static_cast<unsigned>((T + UB_TOK - 1) / UB_TOK), 256, sizeof(float) * UB_TOK * s.E, st>>>(
      T, s.d, s.E, s.k, dxp, inv, dl, W_r, dx);
  note_launch();
}

}  // namespace moe
