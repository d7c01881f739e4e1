// Grouped GEMMs of the MoE layer on tcgen05 tensor cores (sm_100a).
//
// One persistent, warp-specialised kernel template serves the six contractions of the layer:
//   F3  [hg|hu] = xp  W_gate[e] | W_up[e]          + SwiGLU epilogue (writes hg, hu and act = gate silu(hg) hu)
//   F4  o       = act W_down[e]
//   B2  da      = dy_rows W_down[e]^T               + SwiGLU-backward epilogue (reads hg, hu; writes dhg, dhu, dg partials)
//   B4  dxp     = dhg W_gate[e]^T + dhu W_up[e]^T   (one accumulator, two K segments)
//   B3  dW_down[e]          = act_e^T dy_rows_e     (K = rows of expert e, one CTA owns a whole output tile)
//   B5  dW_gate[e]|dW_up[e] = xp_e^T [dhg_e|dhu_e]
// and the three contractions of the router, whose operands are bf16 (or fp32 split exactly into two bf16 terms),
// so that a bf16 MMA with fp32 accumulation is an fp32 contraction up to summation order:
//   RT  logits = x W_r (+ b_r)                      + routing epilogue (top-k, gates, softmax column sums)
//   DX  dxr    = dl_hi W_r^T + dl_lo W_r^T          (router term of dx; the unpermute kernel adds the dxp rows)
//   DWR dW_r partial[s] = x_s^T (dl_hi + dl_lo)_s   (token slices s; partials are summed by a small kernel)
// Tiles are 128 x 256 with K steps of 64; operands arrive by TMA into 128-byte-swizzled shared memory (4 stages),
// the accumulator lives in tensor memory (2 x 256 columns, so the epilogue of one tile overlaps the main loop
// of the next).  Operand major-ness replaces every transpose: row-major [rows, K] is a K-major operand,
// row-major [K, cols] is an MN-major operand, and the UMMA instruction takes either.
// Row buffers are expert-major with each expert's segment padded to 128 rows of zeros, so an M tile never
// straddles two experts and the ragged K of the weight gradients needs no masking.
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer (owns the TMEM allocation), warps 2..9 epilogue (2..5 for the
// routing kind).  The expert-LoRA variant runs on the same template (launch_lora_gemm at the end of this file).
// Every mbarrier wait is bounded; on a timeout the kernel records it in the status word and leaves.
#include "gemm_common.cuh"

namespace moe {

template <int KIND>
__global__ void __launch_bounds__(KIND == GEMM_RT ? 192 : GEMM_THREADS, 1)
    grouped_gemm_kernel(const __grid_constant__ GemmParams p) {
  using TR = Traits<KIND>;
  constexpr int EPI_WARPS = (KIND == GEMM_RT) ? 4 : 8;
  constexpr int NST = STAGES;
  // The routing kind with E <= 128 stages only 32 KB per K block (16 KB of x, 16 KB of W_r): its stages are packed at
  // that stride and the 96 KB this frees hold the scratch of its routing epilogue (80 KB) and the picks (16 KB).
  constexpr uint32_t RT_STAGE_BYTES = A_BYTES + 2 * CHUNK_BYTES;
  static_assert(STAGES * RT_STAGE_BYTES + ROUTE_SCRATCH_BYTES + 128 * ROUTE_SMEM_MAX_K * 8 <= STAGES * STAGE_BYTES + EPI_BYTES,
                "routing scratch does not fit");
  extern __shared__ unsigned char gemm_smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 5];  // full, empty, accumulator full / empty, drain (failure path)
  __shared__ uint32_t tmem_base_slot;
  __shared__ float s_bias[KIND == GEMM_RT ? MAX_E : 1];  // router bias (zero beyond E)
  __shared__ int s_hist[KIND == GEMM_RT ? 128 : 1];      // picks per expert of the tile (routing epilogue for E <= 128)
  if (KIND == GEMM_RT)
    for (int i = threadIdx.x; i < MAX_E; i += blockDim.x) {
      s_bias[i] = (p.bias && i < p.N_total) ? p.bias[i] : 0.f;
      if (i < 128) s_hist[i] = 0;
    }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(gemm_smem_raw) + 1023u) & ~1023u;
  const uint32_t stage_stride = (KIND == GEMM_RT && p.b_chunks <= 2) ? RT_STAGE_BYTES : STAGE_BYTES;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 32 * EPI_WARPS);
    }
    mbar_init(bar0 + 8u * (2 * STAGES + 4), 1);
    fence_mbar_init();
    tma_prefetch_desc(&p.mapA0);
    tma_prefetch_desc(&p.mapB0);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const int ntiles = total_tiles<KIND>(p);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    uint32_t it = 0;
    bool ok = true;
    long long t_wait = 0, t_begin = clock64();
    for (int rd = 0; rd * static_cast<int>(gridDim.x) < ntiles && ok; ++rd) {
      const int t = tile_of_round<KIND>(rd, blockIdx.x, gridDim.x);
      if (t >= ntiles) continue;
      const Tile tl = get_tile<KIND>(p, t);
      for (int kb = 0; kb < tl.nkb; ++kb, ++it) {
        const int s = it % NST;
        const uint32_t ph = (it / NST) & 1u;
        const long long w0 = clock64();
        if (!mbar_wait(empty_bar(s), ph ^ 1u)) {
          ok = false;
          break;
        }
        t_wait += clock64() - w0;
        const uint32_t sA = smem_base + s * stage_stride;
        if (lane == 0) {
          mbar_expect_tx(full_bar(s), p.stage_tx);
          issue_loads<KIND>(p, tl, kb, sA, sA + A_BYTES, full_bar(s));
        }
        __syncwarp();
      }
    }
    if (p.timers && lane == 0) {
      atomicAdd(p.timers + 0, static_cast<unsigned long long>(clock64() - t_begin));  // producer: total
      atomicAdd(p.timers + 1, static_cast<unsigned long long>(t_wait));               // producer: waiting for a free stage
    }
    if (!ok) {
      // gave up: the copies already issued still land in this CTA's shared memory - wait for them (bounded again)
      // before the CTA may exit
      if (lane == 0) record_status(p.status, DEV_TIMEOUT, 100 + KIND);
      for (uint32_t i = it > static_cast<uint32_t>(NST) ? it - NST : 0; i < it; ++i) mbar_wait(full_bar(i % NST), (i / NST) & 1u);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t idesc = umma_idesc(BM, p.mma_n, TR::A_MN, TR::B_MN);
    constexpr uint32_t A_LBO = TR::A_MN ? CHUNK_BYTES : 0, B_LBO = TR::B_MN ? CHUNK_BYTES : 0;
    constexpr uint32_t A_KSTEP = TR::A_MN ? 2048 : 32, B_KSTEP = TR::B_MN ? 2048 : 32;  // bytes per K = 16
    uint32_t it = 0, tc = 0;
    bool ok = true;
    long long t_acc = 0, t_full = 0, t_begin = clock64();
    for (int rd = 0; rd * static_cast<int>(gridDim.x) < ntiles && ok; ++rd) {
      const int t = tile_of_round<KIND>(rd, blockIdx.x, gridDim.x);
      if (t >= ntiles) continue;
      const Tile tl = get_tile<KIND>(p, t);
      if (tl.nkb == 0) continue;
      const int acc = tc & 1;
      const uint32_t aph = (tc >> 1) & 1u;
      ++tc;
      const long long w0 = clock64();
      if (!mbar_wait(tempty_bar(acc), aph ^ 1u)) {
        ok = false;
        break;
      }
      t_acc += clock64() - w0;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
      for (int kb = 0; kb < tl.nkb; ++kb, ++it) {
        const int s = it % NST;
        const uint32_t ph = (it / NST) & 1u;
        const long long w1 = clock64();
        if (!mbar_wait(full_bar(s), ph)) {
          ok = false;
          break;
        }
        t_full += clock64() - w1;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t sA = smem_base + s * stage_stride;
          const uint32_t sB = sA + A_BYTES;
          const int nks = kb == tl.nkb - 1 ? tl.klast : BK / 16;
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks) {
            if (ks < nks) {
              const uint64_t da = smem_desc(sA + ks * A_KSTEP, A_LBO, 1024);
              const uint64_t db = smem_desc(sB + ks * B_KSTEP, B_LBO, 1024);
              umma_bf16(d_tmem, da, db, idesc, (kb | ks) != 0 ? 1u : 0u);
            }
          }
          umma_commit(empty_bar(s));
        }
        __syncwarp();
      }
      if (ok && lane == 0) umma_commit(tfull_bar(acc));
      __syncwarp();
    }
    if (p.timers && lane == 0) {
      atomicAdd(p.timers + 2, static_cast<unsigned long long>(clock64() - t_begin));  // MMA issuer: total
      atomicAdd(p.timers + 3, static_cast<unsigned long long>(t_acc));                // waiting for a drained accumulator
      atomicAdd(p.timers + 4, static_cast<unsigned long long>(t_full));               // waiting for operands
    }
    if (!ok) {
      // gave up: let every MMA issued so far finish (bounded) before the tensor memory is freed
      if (lane == 0) {
        record_status(p.status, DEV_TIMEOUT, 200 + KIND);
        umma_commit(bar0 + 8u * (2 * STAGES + 4));
      }
      __syncwarp();
      mbar_wait(bar0 + 8u * (2 * STAGES + 4), 0u);
    }
  } else if (warp < 2 + EPI_WARPS) {
    // ------------------------------------------------------------------ epilogue (128 TMEM lanes; two warps per
    // lane quadrant, each draining half of the tile's columns - the routing epilogue needs whole rows and uses one)
    const int ew = warp & 3;           // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;  // which half of the columns
    constexpr int NHALF = EPI_WARPS / 4;
    EpiStage es{smem_base + STAGES * STAGE_BYTES + (warp - 2) * (EPI_UNITS * EPI_UNIT_BYTES), 0u};
    uint32_t tc = 0;
    bool ok = true;
    long long t_idle = 0, t_begin = clock64();
    for (int rd = 0; rd * static_cast<int>(gridDim.x) < ntiles && ok; ++rd) {
      const int t = tile_of_round<KIND>(rd, blockIdx.x, gridDim.x);
      if (t >= ntiles) continue;
      const Tile tl = get_tile<KIND>(p, t);
      const int rin = ew * 32 + lane;  // row inside the tile
      if (tl.nkb == 0) {
        // weight gradient of an expert without tokens: zeros
        if (half != 0) continue;
        if (KIND == GEMM_DWR) {
          const int m = tl.m0 + rin;
          if (m < p.M_total)
            for (int col = tl.n0; col < min(tl.n0 + 128, p.N_total); col += 4)
              *reinterpret_cast<float4*>(p.outf + (static_cast<int64_t>(tl.e) * p.M_total + m) * p.N_total + col) =
                  make_float4(0.f, 0.f, 0.f, 0.f);
        } else if (TR::WGRAD) {
          wgrad_zero_fill<KIND>(p, tl.e, tl.m0 + rin, tl.n0);
        }
        continue;
      }
      const int acc = tc & 1;
      const uint32_t aph = (tc >> 1) & 1u;
      ++tc;
      epilogue_prefetch<KIND>(p, static_cast<int64_t>(tl.row0) + rin, tl.n0, half == 0, tl.e, tl.m0 + rin);
      const long long w0 = clock64();
      if (!mbar_wait(tfull_bar(acc), aph)) {
        ok = false;
        break;
      }
      t_idle += clock64() - w0;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(ew * 32) << 16) + acc * ACC_COLS;
      const int64_t row = static_cast<int64_t>(tl.row0) + rin;
      if (KIND == GEMM_F3 || KIND == GEMM_B2) {
        expert_epilogue<KIND>(p, tl.e, row, (TR::WGRAD ? tl.m0 : tl.row0) + ew * 32, tl.n0, taddr, true,
                              TR::WGRAD ? p.M_total - (tl.m0 + ew * 32) : (KIND == GEMM_DX ? static_cast<int>(p.T - tl.row0 - ew * 32) : 32),
                              es, lane, half, NHALF);
      } else if (KIND == GEMM_RT) {
        if (p.N_total <= 128 && p.top_k <= ROUTE_SMEM_MAX_K)
          routing_epilogue_smem(p, s_bias, s_hist, smem_base + STAGES * RT_STAGE_BYTES,
                                smem_base + STAGES * RT_STAGE_BYTES + ROUTE_SCRATCH_BYTES, row, tl.row0 / BM, ew, taddr,
                                lane);
        else
          routing_epilogue_tmem(p, s_bias, row, tl.row0 / BM, ew, taddr, lane);
      } else if (KIND == GEMM_DWR) {
        // fp32 partial of dW_r for this token slice: hi and lo halves of dl share one accumulator pair
        const int m = tl.m0 + rin;
#pragma unroll 1
        for (int c = 2 * half; c < 2 * half + 2; ++c) {
          uint32_t rh[32], rl[32];
          tmem_ld32(taddr + c * 32, rh);
          tmem_ld32(taddr + 128 + c * 32, rl);
          tmem_ld_wait();
          const int col = tl.n0 + c * 32;
          if (m < p.M_total) {
            float* dst = p.outf + (static_cast<int64_t>(tl.e) * p.M_total + m) * p.N_total + col;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              if (col + i < p.N_total)
                *reinterpret_cast<float4*>(dst + i) = make_float4(
                    __uint_as_float(rh[i]) + __uint_as_float(rl[i]), __uint_as_float(rh[i + 1]) + __uint_as_float(rl[i + 1]),
                    __uint_as_float(rh[i + 2]) + __uint_as_float(rl[i + 2]),
                    __uint_as_float(rh[i + 3]) + __uint_as_float(rl[i + 3]));
            }
          }
        }
      } else {
        expert_epilogue<KIND>(p, tl.e, row, (TR::WGRAD ? tl.m0 : tl.row0) + ew * 32, tl.n0, taddr, true,
                              TR::WGRAD ? p.M_total - (tl.m0 + ew * 32) : (KIND == GEMM_DX ? static_cast<int>(p.T - tl.row0 - ew * 32) : 32),
                              es, lane, half, NHALF);
      }
      tc_fence_before();
      mbar_arrive(tempty_bar(acc));
    }
    if (p.timers && lane == 0 && ew == 0 && half == 0) {
      atomicAdd(p.timers + 5, static_cast<unsigned long long>(clock64() - t_begin));  // epilogue warp: total
      atomicAdd(p.timers + 6, static_cast<unsigned long long>(t_idle));               // waiting for a finished accumulator
      atomicAdd(p.timers + 7, 1ull);                                                  // CTAs counted
    }
    if (!ok && lane == 0) {
      record_status(p.status, DEV_TIMEOUT, 300 + KIND);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 row-major [rows, width] -> 2D map with box {64, box_rows}
static bool map_2d(void* fn, CUtensorMap* m, const void* base, int64_t rows, int64_t width, int box_rows) {
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(width), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(width) * 2};
  cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t es[2] = {1, 1};
  return reinterpret_cast<EncodeTiledFn>(fn)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                                             strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// bf16 [E, rows, width] -> 3D map with box {64, box_rows, 1}
static bool map_3d(void* fn, CUtensorMap* m, const void* base, int64_t E, int64_t rows, int64_t width,
                   int box_rows) {
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(width), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(E)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(width) * 2, static_cast<cuuint64_t>(width) * rows * 2};
  cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
  cuuint32_t es[3] = {1, 1, 1};
  return reinterpret_cast<EncodeTiledFn>(fn)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
                                             strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int KIND>
static moe_status launch_kind(moe_ctx_impl* ctx, const GemmParams& p, cudaStream_t st) {
  if (!ctx->attr_done[0][KIND]) {  // per device: the context is bound to one
    if (cudaFuncSetAttribute(grouped_gemm_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(GEMM_SMEM)) != cudaSuccess)
      return MOE_ERR_CUDA;
    ctx->attr_done[0][KIND] = 1;
  }
  grouped_gemm_kernel<KIND><<<ctx->sm_count, KIND == GEMM_RT ? 192 : GEMM_THREADS, GEMM_SMEM, st>>>(p);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// Row tiles (or pairs) walked together inside a column tile: 1 while the expert's weights are few column tiles wide (they
// stay in L2 between row tiles: Qwen3-30B-A3B shape), 16 for wide experts (coarse shape: at 112 column tiles an expert's
// gate and up slabs are 235 MB and were read from DRAM once per row pair).  MOE_ROW_GROUP overrides (measurements).
static int row_group_for(int n_tiles, const moe_ctx_impl* ctx) {
  if (ctx->row_group_override > 0) return ctx->row_group_override;
  return n_tiles > 12 ? 16 : 1;
}

// One launch of an expert / router contraction.  `pair`: CTA-pair kernel.  `part`: 0 = the whole tile list; row GEMMs
// of the mixed schedule: 1 = the pair kernel over complete pairs of row blocks only, 2 = the one-CTA kernel over the
// leftover blocks.
static moe_status launch_gemm_variant(moe_ctx_impl* ctx, GemmKind kind, int64_t T, const WsLayout& L, char* ws,
                                      const GemmIO& io, cudaStream_t st, bool pair, int part) {
  const uint16_t *W_gate = io.W_gate, *W_up = io.W_up, *W_down = io.W_down;
  uint16_t *dW_gate = io.dW_gate, *dW_up = io.dW_up, *dW_down = io.dW_down;
  const Shape& s = ctx->s;
  const int d = s.d, f = s.f, E = s.E;
  const int64_t R = L.rows_max;
  void* fn = ctx->encode_fn;
  uint16_t* xp = reinterpret_cast<uint16_t*>(ws + L.xp);
  uint16_t* hg = reinterpret_cast<uint16_t*>(ws + L.hg);
  uint16_t* hu = reinterpret_cast<uint16_t*>(ws + L.hu);
  uint16_t* act = reinterpret_cast<uint16_t*>(ws + L.act);
  uint16_t* o = reinterpret_cast<uint16_t*>(ws + L.o);
  uint16_t* dhg = reinterpret_cast<uint16_t*>(ws + L.dhg);
  uint16_t* dhu = reinterpret_cast<uint16_t*>(ws + L.dhu);
  uint16_t* dxp = reinterpret_cast<uint16_t*>(ws + L.dxp);
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.sched = reinterpret_cast<const int32_t*>(ws + L.sched);
  p.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
  p.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
  p.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
  p.pair_tab = reinterpret_cast<const int32_t*>(ws + L.pair_tab);
  p.expert_order = reinterpret_cast<const int32_t*>(ws + L.expert_order);
  p.timers = ctx->gemm_timers ? reinterpret_cast<unsigned long long*>(ws + L.timers) + 8 * kind : nullptr;
  if (part == 1) {
    p.pair_tab = reinterpret_cast<const int32_t*>(ws + L.fpair_tab);
    p.pair_count_slot = 3;
  } else {
    p.pair_count_slot = 2;
  }
  p.oob_row = static_cast<int>(R);
  p.tile_list = part == 2 ? reinterpret_cast<const int32_t*>(ws + L.single_tab) : nullptr;
  p.status = reinterpret_cast<int32_t*>(ws + L.status);
  p.E = E;
  if ((kind == GEMM_B3 || kind == GEMM_B5) && io.e_count > 0) {  // one group of experts, in index order
    p.E = io.e_count;
    p.e_first = io.e_first;
    p.expert_grouped = 1;
  }
  p.b_chunks = 4;
  p.mma_n = BN;
  p.stage_tx = STAGE_BYTES;
  p.nseg = (kind == GEMM_B4 || kind == GEMM_DX) ? 2 : 1;
  p.k_blocks1 = 0;
  p.out_scale = 1.f;
  bool ok = true;
  switch (kind) {
    case GEMM_F3:
      ok = map_2d(fn, &p.mapA0, xp, R, d, 128) && map_3d(fn, &p.mapB0, W_gate, E, d, f, 64) &&
           map_3d(fn, &p.mapB1, W_up, E, d, f, 64);
      p.mapA1 = p.mapA0;
      p.n_tiles = (f + 127) / 128;
      p.k_blocks = d / BK;
      p.N_total = f;
      p.out0 = hg; p.out1 = hu; p.out2 = act;
      p.ld_out = f;
      p.row_gate = reinterpret_cast<const float*>(ws + L.row_gate);
      p.save_pre = io.save_preactivations ? 1 : 0;
      if (!ok) return MOE_ERR_CUDA;
      p.row_group = row_group_for(p.n_tiles, ctx);
      return pair ? launch_pair_gemm(ctx, kind, p, st) : launch_kind<GEMM_F3>(ctx, p, st);
    case GEMM_F4:
      ok = map_2d(fn, &p.mapA0, act, R, f, 128) && map_3d(fn, &p.mapB0, W_down, E, f, d, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.n_tiles = (d + 255) / 256;
      p.k_blocks = f / BK;
      p.N_total = d;
      p.out0 = o;
      p.ld_out = d;
      if (!ok) return MOE_ERR_CUDA;
      p.row_group = row_group_for(p.n_tiles, ctx);
      return pair ? launch_pair_gemm(ctx, kind, p, st) : launch_kind<GEMM_F4>(ctx, p, st);
    case GEMM_B2:
      ok = map_2d(fn, &p.mapA0, o, R, d, 128) && map_3d(fn, &p.mapB0, W_down, E, f, d, pair ? 128 : 256);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.n_tiles = (f + 255) / 256;
      p.k_blocks = d / BK;
      p.N_total = f;
      p.in0 = hg; p.in1 = hu;
      p.out0 = dhg; p.out1 = dhu;
      p.ld_out = f;
      p.row_gate = reinterpret_cast<const float*>(ws + L.row_gate);
      p.outf = reinterpret_cast<float*>(ws + L.dg_part);
      p.rows_max = L.rows_max;
      if (!ok) return MOE_ERR_CUDA;
      p.row_group = row_group_for(p.n_tiles, ctx);
      return pair ? launch_pair_gemm(ctx, kind, p, st) : launch_kind<GEMM_B2>(ctx, p, st);
    case GEMM_B4:
      ok = map_2d(fn, &p.mapA0, dhg, R, f, 128) && map_2d(fn, &p.mapA1, dhu, R, f, 128) &&
           map_3d(fn, &p.mapB0, W_gate, E, d, f, pair ? 128 : 256) &&
           map_3d(fn, &p.mapB1, W_up, E, d, f, pair ? 128 : 256);
      p.n_tiles = (d + 255) / 256;
      p.k_blocks = f / BK;
      p.N_total = d;
      p.out0 = dxp;
      p.ld_out = d;
      if (!ok) return MOE_ERR_CUDA;
      p.row_group = row_group_for(p.n_tiles, ctx);
      return pair ? launch_pair_gemm(ctx, kind, p, st) : launch_kind<GEMM_B4>(ctx, p, st);
    case GEMM_B3:
      ok = map_2d(fn, &p.mapA0, act, R, f, 64) && map_2d(fn, &p.mapB0, o, R, d, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.m_tiles = pair ? (f + 255) / 256 : (f + 127) / 128;
      p.n_tiles = (d + 255) / 256;
      p.M_total = f;
      p.N_total = d;
      p.out0 = dW_down;
      p.accf0 = io.dW_down_acc;
      p.acc_fp32 = io.dW_down_acc != nullptr;
      p.ld_out = d;
      p.expert_stride = static_cast<int64_t>(f) * d;
      if (!ok) return MOE_ERR_CUDA;
      return pair ? launch_pair_gemm(ctx, kind, p, st) : launch_kind<GEMM_B3>(ctx, p, st);
    case GEMM_B5:
      ok = map_2d(fn, &p.mapA0, xp, R, d, 64) && map_2d(fn, &p.mapB0, dhg, R, f, 64) &&
           map_2d(fn, &p.mapB1, dhu, R, f, 64);
      p.mapA1 = p.mapA0;
      p.m_tiles = pair ? (d + 255) / 256 : (d + 127) / 128;
      p.n_tiles = (f + 127) / 128;
      p.M_total = d;
      p.N_total = f;
      p.out0 = dW_gate; p.out1 = dW_up;
      p.accf0 = io.dW_gate_acc; p.accf1 = io.dW_up_acc;
      p.acc_fp32 = io.dW_gate_acc != nullptr;
      p.ld_out = f;
      p.expert_stride = static_cast<int64_t>(d) * f;
      if (!ok) return MOE_ERR_CUDA;
      return pair ? launch_pair_gemm(ctx, kind, p, st) : launch_kind<GEMM_B5>(ctx, p, st);
    case GEMM_RT:
      // logits[T,E] = x[T,d] W_r[d,E]; W_r is read as a one-slab 3D tensor so the weight loaders apply
      ok = map_2d(fn, &p.mapA0, io.x, T, d, 128) && map_3d(fn, &p.mapB0, io.W_r, 1, d, E, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      if (io.W_r_mid) {  // fp32 router weight: x (hi + mid + lo), each product exact in fp32
        ok = ok && map_3d(fn, &p.mapB1, io.W_r_mid, 1, d, E, 64) && map_3d(fn, &p.mapB2, io.W_r_lo, 1, d, E, 64);
        p.nseg = 3;
      }
      p.static_m_tiles = static_cast<int>((T + BM - 1) / BM);
      p.n_tiles = 1;
      p.k_blocks = d / BK;
      p.N_total = E;
      p.b_chunks = (E + 63) / 64;
      p.mma_n = (E + 15) / 16 * 16;
      p.stage_tx = A_BYTES + p.b_chunks * CHUNK_BYTES;
      p.T = T;
      p.top_k = s.k;
      p.bias = io.b_r;
      p.logits = reinterpret_cast<float*>(ws + L.logits);
      p.logits_out = io.logits_out;
      p.idx = reinterpret_cast<int32_t*>(ws + L.idx);
      p.gates = reinterpret_cast<float*>(ws + L.gates);
      p.idx_out = io.idx_out;
      p.gates_out = io.gates_out;
      p.psum_part = reinterpret_cast<float*>(ws + L.psum_part);
      p.tile_counts = reinterpret_cast<int32_t*>(ws + L.tile_counts);  // written by the shared-memory routing epilogue
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_RT>(ctx, p, st);
    case GEMM_DX:
      // dxr[T,d] = dl_hi W_r^T + dl_lo W_r^T
      ok = map_2d(fn, &p.mapA0, ws + L.dl_hi, T, E, 128) && map_2d(fn, &p.mapA1, ws + L.dl_lo, T, E, 128) &&
           map_3d(fn, &p.mapB0, io.W_r, 1, d, E, 256);
      p.mapB1 = p.mapB0;
      if (io.W_r_mid) {  // fp32 router weight: dl_hi W_hi^T + dl_lo W_hi^T + dl_hi W_mid^T (the rest is below 2^-17)
        ok = ok && map_2d(fn, &p.mapA2, ws + L.dl_hi, T, E, 128) && map_3d(fn, &p.mapB2, io.W_r_mid, 1, d, E, 256);
        p.nseg = 3;
      }
      p.static_m_tiles = static_cast<int>((T + BM - 1) / BM);
      p.n_tiles = (d + 255) / 256;
      p.k_blocks = (E + BK - 1) / BK;
      p.N_total = d;
      p.T = T;
      p.top_k = s.k;
      p.out0 = reinterpret_cast<uint16_t*>(ws + L.dxr);
      p.ld_out = d;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_DX>(ctx, p, st);
    case GEMM_DWR: {
      // partial[s][d,E] = x_s^T (dl_hi + dl_lo)_s over token slices of split_rows tokens
      ok = map_2d(fn, &p.mapA0, io.x, T, d, 64) && map_2d(fn, &p.mapB0, ws + L.dl_hi, T, E, 64) &&
           map_2d(fn, &p.mapB1, ws + L.dl_lo, T, E, 64);
      p.mapA1 = p.mapA0;
      const int64_t per = ((T + DWR_SPLIT - 1) / DWR_SPLIT + BK - 1) / BK * BK;
      p.split_rows = static_cast<int>(per);
      p.rows_total = static_cast<int>((T + BK - 1) / BK * BK);
      p.E = DWR_SPLIT;  // slices play the role of experts in the tile list
      p.m_tiles = (d + 127) / 128;
      p.n_tiles = (E + 127) / 128;
      p.M_total = d;
      p.N_total = E;
      p.outf = reinterpret_cast<float*>(ws + L.dwr_part);
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_DWR>(ctx, p, st);
    }
    default:
      break;
  }
  (void)T;
  return MOE_ERR_INVALID_ARG;
}

// Tile shape per GEMM.  A CTA pair (256 x 256 tile, each CTA staging its rows of A and half of B) moves a third
// less operand data from L2 per flop than a one-CTA 128 x 256 tile, and the L2 -> SM feed is what limits these
// kernels: at the Qwen3-30B-A3B shape the pair kernel needs 14 - 18 % fewer cycles per useful flop.  In the
// power-capped steady state the step is bound by energy rather than cycles and the gain shrinks to 1 - 3 %.
// Row GEMMs pair two 128-row blocks of ONE expert, so an expert with an odd block count has a block left over.
// Two ways to deal with it were built and measured in steady state (Qwen shape, ms per step): half-empty pairs
// (the empty half loads no A rows) 4.17; complete pairs on the pair kernel plus the leftover blocks on one-CTA tiles
// in a second launch (MOE_FLAG_HYBRID_TILES) 4.22 - the second launch's ramp and ragged last round cost what the
// empty halves cost; one-CTA tiles throughout 4.39.  Default: half-empty pairs from 512 rows per expert upwards; below
// that there are few complete pairs and the layer is bound by streaming the weights from HBM anyway.
// Weight gradients pair along the weight dimension without leftovers, but their K loop is the expert's row count:
// below ~768 rows per expert the two coupled epilogues bound them and one-CTA tiles are faster.
moe_status launch_grouped_gemm(moe_ctx_impl* ctx, GemmKind kind, int64_t T, const WsLayout& L, char* ws,
                               const GemmIO& io, cudaStream_t st) {
  const bool row_kind = kind == GEMM_F3 || kind == GEMM_F4 || kind == GEMM_B2 || kind == GEMM_B4;
  const bool wgrad_kind = kind == GEMM_B3 || kind == GEMM_B5;
  const double rows_per_expert = static_cast<double>(T) * ctx->s.k / ctx->s.E;
  if (wgrad_kind) {
    const bool pair = ctx->tile_mode == 1 || ctx->tile_mode == 3 || (ctx->tile_mode == 0 && rows_per_expert >= 768.0);
    return launch_gemm_variant(ctx, kind, T, L, ws, io, st, pair, 0);
  }
  if (!row_kind) return launch_gemm_variant(ctx, kind, T, L, ws, io, st, false, 0);
  if (ctx->tile_mode == 1) return launch_gemm_variant(ctx, kind, T, L, ws, io, st, true, 0);
  // dgrad gate/up at short K (2 f / 64 < 64 K blocks per tile) gains from pairs only from 768 rows per expert on
  // (Qwen3-30B-A3B shape, steady state under the power cap: 453 vs 443 us at 512 rows per expert, 838 vs 875 us at
  // 1024, 1590 vs 1709 us at 2048)
  bool long_k = kind != GEMM_B4 || 2 * ctx->s.f / BK >= 64 || rows_per_expert >= 768.0;
  if (kind == GEMM_B4 && ctx->b4_pair_override >= 0) long_k = ctx->b4_pair_override != 0;
  if (ctx->tile_mode == 0 && rows_per_expert >= 512.0 && long_k)
    return launch_gemm_variant(ctx, kind, T, L, ws, io, st, true, 0);
  if (ctx->tile_mode != 3) return launch_gemm_variant(ctx, kind, T, L, ws, io, st, false, 0);
  const moe_status rc = launch_gemm_variant(ctx, kind, T, L, ws, io, st, true, 1);
  if (rc != MOE_OK) return rc;
  return launch_gemm_variant(ctx, kind, T, L, ws, io, st, false, 2);
}

// Backward operations of the expert-LoRA variant (see launch_lora_gemm below, which prepares `p`).
static moe_status launch_lora_gemm_bwd(moe_ctx_impl* ctx, LoraOp op, int64_t T, const WsLayout& L, char* ws,
                                       const GemmIO& io, const LoraArgs& lo, GemmParams p, cudaStream_t st) {
  (void)T;
  const Shape& s = ctx->s;
  const int d = s.d, f = s.f, E = s.E, r = lo.rank;
  const int64_t R = L.rows_max;
  void* fn = ctx->encode_fn;
  auto B16 = [&](size_t off) { return reinterpret_cast<uint16_t*>(ws + off); };
  uint16_t *xp = B16(L.xp), *hg = B16(L.hg), *hu = B16(L.hu), *act = B16(L.act), *dyr = B16(L.o), *dhg = B16(L.dhg),
           *dhu = B16(L.dhu), *dxp = B16(L.dxp), *u = B16(L.lora_u), *v = B16(L.lora_v), *w = B16(L.lora_w),
           *z = B16(L.lora_z);
  const uint32_t skinny_tx = A_BYTES + CHUNK_BYTES;
  bool ok = true;
  switch (op) {
    case LORA_W:  // w[R,64] = s dy_rows B2[e]^T      (B4 kind, one segment, K-major B of 64 rows)
      ok = map_2d(fn, &p.mapA0, dyr, R, d, 128) && map_3d(fn, &p.mapB0, lo.B2, E, r, d, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.n_tiles = 1;
      p.k_blocks = d / BK;
      p.nseg = 1;
      p.mma_n = 64; p.stage_tx = skinny_tx;
      p.N_total = 64;
      p.out0 = w;
      p.ld_out = 64;
      p.out_scale = lo.scale;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B4>(ctx, p, st);
    case LORA_Z:  // z[R,64] = s (dhg B1g[e]^T + dhu B1u[e]^T)   (B4 kind, two segments)
      ok = map_2d(fn, &p.mapA0, dhg, R, f, 128) && map_2d(fn, &p.mapA1, dhu, R, f, 128) &&
           map_3d(fn, &p.mapB0, lo.B1g, E, r, f, 64) && map_3d(fn, &p.mapB1, lo.B1u, E, r, f, 64);
      p.n_tiles = 1;
      p.k_blocks = f / BK;
      p.nseg = 2;
      p.mma_n = 64; p.stage_tx = skinny_tx;
      p.N_total = 64;
      p.out0 = z;
      p.ld_out = 64;
      p.out_scale = lo.scale;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B4>(ctx, p, st);
    case LORA_B2:  // da = dy_rows Wd^T + w A2^T, SwiGLU-backward epilogue
      ok = map_2d(fn, &p.mapA0, dyr, R, d, 128) && map_3d(fn, &p.mapB0, io.W_down, E, f, d, 256) &&
           map_2d(fn, &p.mapA2, w, R, 64, 128) && map_3d(fn, &p.mapB2, lo.A2, E, f, r, 256);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.n_tiles = (f + 255) / 256;
      p.k_blocks = d / BK;
      p.k_blocks1 = 1;
      p.N_total = f;
      p.in0 = hg; p.in1 = hu;
      p.out0 = dhg; p.out1 = dhu;
      p.ld_out = f;
      p.outf = reinterpret_cast<float*>(ws + L.dg_part);
      p.rows_max = L.rows_max;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B2>(ctx, p, st);
    case LORA_B4:  // dxp = dhg Wg^T + dhu Wu^T + z A1^T
      ok = map_2d(fn, &p.mapA0, dhg, R, f, 128) && map_2d(fn, &p.mapA1, dhu, R, f, 128) &&
           map_3d(fn, &p.mapB0, io.W_gate, E, d, f, 256) && map_3d(fn, &p.mapB1, io.W_up, E, d, f, 256) &&
           map_2d(fn, &p.mapA2, z, R, 64, 128) && map_3d(fn, &p.mapB2, lo.A1, E, d, r, 256);
      p.n_tiles = (d + 255) / 256;
      p.k_blocks = f / BK;
      p.nseg = 2;
      p.k_blocks1 = 1;
      p.N_total = d;
      p.out0 = dxp;
      p.ld_out = d;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B4>(ctx, p, st);
    case LORA_DB2:  // dB2[e][r,d] = v_e^T dy_rows_e      (B3 kind, M = rank)
      ok = map_2d(fn, &p.mapA0, v, R, 64, 64) && map_2d(fn, &p.mapB0, dyr, R, d, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.m_tiles = 1;
      p.n_tiles = (d + 255) / 256;
      p.M_total = r;
      p.N_total = d;
      p.out0 = lo.dB2;
      p.ld_out = d;
      p.expert_stride = static_cast<int64_t>(r) * d;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B3>(ctx, p, st);
    case LORA_DA2:  // dA2[e][f,r] = act_e^T w_e           (B3 kind, N = rank)
    case LORA_DA1:  // dA1[e][d,r] = xp_e^T z_e
      ok = map_2d(fn, &p.mapA0, op == LORA_DA2 ? act : xp, R, op == LORA_DA2 ? f : d, 64) &&
           map_2d(fn, &p.mapB0, op == LORA_DA2 ? w : z, R, 64, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.M_total = op == LORA_DA2 ? f : d;
      p.m_tiles = (p.M_total + 127) / 128;
      p.n_tiles = 1;
      p.b_chunks = 1; p.mma_n = 64; p.stage_tx = skinny_tx;
      p.N_total = r;
      p.out0 = op == LORA_DA2 ? lo.dA2 : lo.dA1;
      p.ld_out = r;
      p.expert_stride = static_cast<int64_t>(p.M_total) * r;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B3>(ctx, p, st);
    case LORA_DB1:  // dB1g[e] | dB1u[e] [r,f] = u_e^T [dhg_e | dhu_e]   (B5 kind, M = rank)
      ok = map_2d(fn, &p.mapA0, u, R, 64, 64) && map_2d(fn, &p.mapB0, dhg, R, f, 64) &&
           map_2d(fn, &p.mapB1, dhu, R, f, 64);
      p.mapA1 = p.mapA0;
      p.m_tiles = 1;
      p.n_tiles = (f + 127) / 128;
      p.M_total = r;
      p.N_total = f;
      p.out0 = lo.dB1g; p.out1 = lo.dB1u;
      p.ld_out = f;
      p.expert_stride = static_cast<int64_t>(r) * f;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_B5>(ctx, p, st);
    default:
      break;
  }
  return MOE_ERR_INVALID_ARG;
}

// ------------------------------------------------------------------------------------------ expert LoRA
// The adapted layer reuses the kernels above with different operands: the low-rank path enters each row GEMM as one
// extra 64-deep K segment ([xp | u] [[W]; [B1]], ...), the four 64-wide row buffers u, v, w, z come from skinny
// instances (N = 64) of the F4 / B4 kinds, and the adapter gradients from instances of the B3 / B5 kinds whose M or
// N is the rank.  All on one-CTA tiles.
moe_status launch_lora_gemm(moe_ctx_impl* ctx, LoraOp op, int64_t T, const WsLayout& L, char* ws, const GemmIO& io,
                            const LoraArgs& lo, cudaStream_t st) {
  const Shape& s = ctx->s;
  const int d = s.d, f = s.f, E = s.E, r = lo.rank;
  const int64_t R = L.rows_max;
  void* fn = ctx->encode_fn;
  auto B16 = [&](size_t off) { return reinterpret_cast<uint16_t*>(ws + off); };
  uint16_t *xp = B16(L.xp), *hg = B16(L.hg), *hu = B16(L.hu), *act = B16(L.act), *o = B16(L.o), *dhg = B16(L.dhg),
           *dhu = B16(L.dhu), *dxp = B16(L.dxp), *u = B16(L.lora_u), *v = B16(L.lora_v), *w = B16(L.lora_w),
           *z = B16(L.lora_z);
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.sched = reinterpret_cast<const int32_t*>(ws + L.sched);
  p.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
  p.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
  p.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
  p.pair_tab = reinterpret_cast<const int32_t*>(ws + L.pair_tab);
  p.expert_order = reinterpret_cast<const int32_t*>(ws + L.expert_order);
  p.status = reinterpret_cast<int32_t*>(ws + L.status);
  p.E = E;
  p.b_chunks = 4;
  p.mma_n = BN;
  p.stage_tx = STAGE_BYTES;
  p.nseg = 1;
  p.out_scale = 1.f;
  p.row_gate = reinterpret_cast<const float*>(ws + L.row_gate);
  const uint32_t skinny_tx = A_BYTES + CHUNK_BYTES;  // a 128 x 64 A tile and one 64 x 64 B tile
  bool ok = true;
  switch (op) {
    case LORA_U:  // u[R,64] = s xp A1[e]            (F4 kind, N = 64)
    case LORA_V:  // v[R,64] = s act A2[e]
      ok = map_2d(fn, &p.mapA0, op == LORA_U ? xp : act, R, op == LORA_U ? d : f, 128) &&
           map_3d(fn, &p.mapB0, op == LORA_U ? lo.A1 : lo.A2, E, op == LORA_U ? d : f, r, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.n_tiles = 1;
      p.k_blocks = (op == LORA_U ? d : f) / BK;
      p.b_chunks = 1; p.mma_n = 64; p.stage_tx = skinny_tx;
      p.N_total = 64;
      p.out0 = op == LORA_U ? u : v;
      p.ld_out = 64;
      p.out_scale = lo.scale;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_F4>(ctx, p, st);
    case LORA_F3:  // [hg|hu] = xp [Wg|Wu] + u [B1g|B1u]
      ok = map_2d(fn, &p.mapA0, xp, R, d, 128) && map_3d(fn, &p.mapB0, io.W_gate, E, d, f, 64) &&
           map_3d(fn, &p.mapB1, io.W_up, E, d, f, 64) && map_2d(fn, &p.mapA2, u, R, 64, 128) &&
           map_3d(fn, &p.mapB2, lo.B1g, E, r, f, 64) && map_3d(fn, &p.mapB3, lo.B1u, E, r, f, 64);
      p.mapA1 = p.mapA0;
      p.n_tiles = (f + 127) / 128;
      p.k_blocks = d / BK;
      p.k_blocks1 = 1;
      p.N_total = f;
      p.out0 = hg; p.out1 = hu; p.out2 = act;
      p.ld_out = f;
      p.save_pre = 1;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_F3>(ctx, p, st);
    case LORA_F4:  // o = act Wd + v B2
      ok = map_2d(fn, &p.mapA0, act, R, f, 128) && map_3d(fn, &p.mapB0, io.W_down, E, f, d, 64) &&
           map_2d(fn, &p.mapA2, v, R, 64, 128) && map_3d(fn, &p.mapB2, lo.B2, E, r, d, 64);
      p.mapA1 = p.mapA0; p.mapB1 = p.mapB0;
      p.n_tiles = (d + 255) / 256;
      p.k_blocks = f / BK;
      p.k_blocks1 = 1;
      p.N_total = d;
      p.out0 = o;
      p.ld_out = d;
      if (!ok) return MOE_ERR_CUDA;
      return launch_kind<GEMM_F4>(ctx, p, st);
    default:
      break;
  }
  return launch_lora_gemm_bwd(ctx, op, T, L, ws, io, lo, p, st);
}

}  // namespace moe
