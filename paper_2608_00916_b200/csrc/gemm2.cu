// The six expert contractions on CTA pairs (cluster of 2, tcgen05 cta_group::2).
//
// Why pairs: with one CTA per 128 x 256 tile every SM stages 48 KB of operands per 64-deep K step, and the profile
// of that kernel shows the tensor pipe about half busy with no memory unit saturated - the four-stage ring cannot
// keep enough bytes in flight.  A pair computes a 256 x 256 tile: each CTA stages its own 128 rows of A and only
// HALF of B (128 of the 256 columns); the MMA reads both halves from the two CTAs' shared memories.  Per SM that is
// 32 KB per K step for the same MMA time, and the ring grows to six stages.
//
// Protocol (leader = cluster rank 0).  Both producers issue their own TMA loads, all credited to the LEADER's full
// barrier (the leader's producer posts the expected byte count of both CTAs).  The leader's MMA thread issues
// tcgen05.mma.cta_group::2 and commits to the empty / accumulator-full barriers of BOTH CTAs.  The epilogue warps of
// both CTAs drain their own tensor memory (their 128 rows) and arrive on the leader's accumulator-empty barrier.
// Tensor memory is allocated and freed by one warp of each CTA; cluster barriers bracket the kernel so that no CTA
// leaves while its partner may still touch its shared memory, barriers or tensor memory.
//
// Row GEMMs pair two consecutive 128-row blocks of ONE expert; an expert with an odd number of blocks gets a pair
// whose second half is empty: that CTA stages its half of B, and for A it issues the same TMA copy at a row beyond
// the end of the row buffer, which the copy engine fills with zeros without touching memory - so the unavoidable MMA
// over the empty half multiplies zeros (its power draw depends on the operand data, and the step is power-bound) -
// and nothing of its accumulator half is read or stored.  Weight gradients pair along M.
#include "gemm_common.cuh"

namespace moe {

constexpr int STAGES2 = 6;
constexpr int GEMM2_THREADS = 320;  // warps: 0 TMA producer, 1 MMA issuer, 2..9 epilogue (two per TMEM lane quadrant)
constexpr int BH_BYTES = 128 * BK * 2;              // this CTA's half of B: 16 KB
constexpr int STAGE2_BYTES = A_BYTES + BH_BYTES;    // 32 KB
constexpr size_t GEMM2_SMEM = static_cast<size_t>(STAGES2) * STAGE2_BYTES + EPI_BYTES + 1024;

struct Tile2 {
  int e, row0, m0, n0, nkb;
  int klast;    // K = 16 steps issued in the last K block
  bool write;   // this CTA's 128 rows exist (false: the empty half of an odd expert's last pair)
  bool full;    // both halves of the pair exist
};

template <int KIND>
__device__ __forceinline__ int total_tiles2(const GemmParams& p) {
  if (Traits<KIND>::WGRAD) return p.E * p.m_tiles * p.n_tiles;  // m_tiles = 256-row pairs of the output
  return p.sched[p.pair_count_slot] * p.n_tiles;                // number of row-block pairs in the table in use
}

template <int KIND>
__device__ __forceinline__ Tile2 get_tile2(const GemmParams& p, int t, int rank) {
  Tile2 tl;
  tl.klast = BK / 16;
  if (Traits<KIND>::WGRAD) {
    const int per = p.m_tiles * p.n_tiles;
    const int slot = t / per;
    tl.e = p.expert_grouped ? p.e_first + slot : p.expert_order[slot];  // else: longest K loops first
    const int rem = t - slot * per;
    tl.m0 = (rem / p.n_tiles) * 2 * BM + rank * BM;
    tl.n0 = (rem % p.n_tiles) * Traits<KIND>::N_SPAN;
    tl.row0 = p.pad_offsets[tl.e];
    tl.nkb = (p.counts[tl.e] + BK - 1) / BK;  // the rest of the 128-row padding is zeros
    tl.klast = last_k_steps(p.counts[tl.e]);
    tl.write = true;
    tl.full = true;
  } else {
    int pr, nt;
    row_tile_order(t, p.n_tiles, p.row_group, p.sched[p.pair_count_slot], pr, nt);
    const int4 info = *reinterpret_cast<const int4*>(p.pair_tab + 4 * pr);  // expert, first row, blocks (1 or 2)
    tl.e = info.x;
    tl.row0 = info.y + rank * BM;
    tl.write = rank < info.z;
    tl.full = info.z == 2;
    tl.m0 = 0;
    tl.n0 = nt * Traits<KIND>::N_SPAN;
    tl.nkb = p.k_blocks * p.nseg;
  }
  return tl;
}

// Loads of one K block for the CTA of rank `rank`: its rows of A and its 128-column half of B.
template <int KIND>
__device__ __forceinline__ void issue_loads2(const GemmParams& p, const Tile2& tl, int kb, int rank, uint32_t sA,
                                             uint32_t sB, uint32_t bar) {
  if (KIND == GEMM_F3) {
    tma_load_2d_pair(sA, &p.mapA0, bar, kb * BK, tl.write ? tl.row0 : p.oob_row);
    const CUtensorMap* mb = rank ? &p.mapB1 : &p.mapB0;  // leader: gate columns, partner: the matching up columns
#pragma unroll
    for (int c = 0; c < 2; ++c) tma_load_3d_pair(sB + c * CHUNK_BYTES, mb, bar, tl.n0 + c * 64, kb * BK, tl.e);
  } else if (KIND == GEMM_F4) {
    tma_load_2d_pair(sA, &p.mapA0, bar, kb * BK, tl.write ? tl.row0 : p.oob_row);
#pragma unroll
    for (int c = 0; c < 2; ++c)
      tma_load_3d_pair(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + rank * 128 + c * 64, kb * BK, tl.e);
  } else if (KIND == GEMM_B2) {
    tma_load_2d_pair(sA, &p.mapA0, bar, kb * BK, tl.write ? tl.row0 : p.oob_row);
    tma_load_3d_pair(sB, &p.mapB0, bar, kb * BK, tl.n0 + rank * 128, tl.e);
  } else if (KIND == GEMM_B4) {
    const int seg = kb / p.k_blocks, kk = kb - seg * p.k_blocks;
    tma_load_2d_pair(sA, seg ? &p.mapA1 : &p.mapA0, bar, kk * BK, tl.write ? tl.row0 : p.oob_row);
    tma_load_3d_pair(sB, seg ? &p.mapB1 : &p.mapB0, bar, kk * BK, tl.n0 + rank * 128, tl.e);
  } else if (KIND == GEMM_B3) {
    const int row = tl.row0 + kb * BK;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      tma_load_2d_pair(sA + c * CHUNK_BYTES, &p.mapA0, bar, tl.m0 + c * 64, row);
      tma_load_2d_pair(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + rank * 128 + c * 64, row);
    }
  } else {  // GEMM_B5
    const int row = tl.row0 + kb * BK;
    const CUtensorMap* mb = rank ? &p.mapB1 : &p.mapB0;  // leader: dhg columns, partner: dhu columns
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      tma_load_2d_pair(sA + c * CHUNK_BYTES, &p.mapA0, bar, tl.m0 + c * 64, row);
      tma_load_2d_pair(sB + c * CHUNK_BYTES, mb, bar, tl.n0 + c * 64, row);
    }
  }
}

template <int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM2_THREADS, 1)
    grouped_gemm_pair_kernel(const __grid_constant__ GemmParams p) {
  using TR = Traits<KIND>;
  extern __shared__ unsigned char gemm2_smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * STAGES2 + 5];  // full, empty, accumulator full / empty, drain (failure path)
  __shared__ uint32_t tmem_base_slot;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_ctarank());
  const bool leader = rank == 0;
  const uint32_t smem_base = (smem_u32(gemm2_smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES2 + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES2 + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES2 + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) {
      mbar_init(full_bar(s), 1);   // used in the leader only: its producer's arrive + the bytes of both CTAs
      mbar_init(empty_bar(s), 1);  // one commit from the leader's MMA thread
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);   // one commit from the leader's MMA thread
      mbar_init(tempty_bar(a), 16);  // used in the leader only: 8 epilogue warps of each CTA
    }
    mbar_init(bar0 + 8u * (2 * STAGES2 + 4), 1);
    fence_mbar_init();
    tma_prefetch_desc(&p.mapA0);
    tma_prefetch_desc(&p.mapB0);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_slot), TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();  // barriers of both CTAs are initialised before anyone signals across the pair
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const int ntiles = total_tiles2<KIND>(p);
  const int cid = blockIdx.x >> 1, nclusters = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    uint32_t it = 0;
    bool ok = true;
    long long t_wait = 0, t_begin = clock64();
    for (int rd = 0; rd * nclusters < ntiles && ok; ++rd) {
      const int t = tile_of_round<KIND>(rd, cid, nclusters);
      if (t >= ntiles) continue;
      const Tile2 tl = get_tile2<KIND>(p, t, rank);
      for (int kb = 0; kb < tl.nkb; ++kb, ++it) {
        const int s = it % STAGES2;
        const uint32_t ph = (it / STAGES2) & 1u;
        const long long w0 = clock64();
        if (!mbar_wait(empty_bar(s), ph ^ 1u)) {
          ok = false;
          break;
        }
        t_wait += clock64() - w0;
        if (lane == 0) {
          if (leader) mbar_expect_tx(full_bar(s), 2 * STAGE2_BYTES);
          const uint32_t sA = smem_base + s * STAGE2_BYTES;
          issue_loads2<KIND>(p, tl, kb, rank, sA, sA + A_BYTES, mapa_shared(full_bar(s), 0));
        }
        __syncwarp();
      }
    }
    if (p.timers && lane == 0 && leader) {
      atomicAdd(p.timers + 0, static_cast<unsigned long long>(clock64() - t_begin));
      atomicAdd(p.timers + 1, static_cast<unsigned long long>(t_wait));
    }
    if (!ok) {
      // gave up: the leader waits (bounded) for the copies of BOTH CTAs that were already issued - they are all credited
      // to its full barriers - so that neither CTA exits with copies in flight (the cluster barrier below holds the
      // partner until then)
      if (lane == 0) record_status(p.status, DEV_TIMEOUT, 1100 + KIND);
      if (leader)
        for (uint32_t i = it > static_cast<uint32_t>(STAGES2) ? it - STAGES2 : 0; i < it; ++i)
          mbar_wait(full_bar(i % STAGES2), (i / STAGES2) & 1u);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader) {
      constexpr uint32_t idesc = umma_idesc(2 * BM, BN, TR::A_MN, TR::B_MN);
      constexpr uint32_t A_LBO = TR::A_MN ? CHUNK_BYTES : 0, B_LBO = TR::B_MN ? CHUNK_BYTES : 0;
      constexpr uint32_t A_KSTEP = TR::A_MN ? 2048 : 32, B_KSTEP = TR::B_MN ? 2048 : 32;
      uint32_t it = 0, tc = 0;
      bool ok = true;
      long long t_acc = 0, t_full = 0, t_begin = clock64();
      for (int rd = 0; rd * nclusters < ntiles && ok; ++rd) {
      const int t = tile_of_round<KIND>(rd, cid, nclusters);
      if (t >= ntiles) continue;
        const Tile2 tl = get_tile2<KIND>(p, t, rank);
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
          const int s = it % STAGES2;
          const uint32_t ph = (it / STAGES2) & 1u;
          const long long w1 = clock64();
          if (!mbar_wait(full_bar(s), ph)) {
            ok = false;
            break;
          }
          t_full += clock64() - w1;
          tc_fence_after();
          if (lane == 0) {
            const uint32_t sA = smem_base + s * STAGE2_BYTES;
            const uint32_t sB = sA + A_BYTES;
            const int nks = kb == tl.nkb - 1 ? tl.klast : BK / 16;
#pragma unroll
            for (int ks = 0; ks < BK / 16; ++ks) {
              if (ks < nks) {
                const uint64_t da = smem_desc(sA + ks * A_KSTEP, A_LBO, 1024);
                const uint64_t db = smem_desc(sB + ks * B_KSTEP, B_LBO, 1024);
                umma_bf16_pair(d_tmem, da, db, idesc, (kb | ks) != 0 ? 1u : 0u);
              }
            }
            // the stage is free in both CTAs once these MMAs have read it
            umma_commit_pair_both(empty_bar(s));
          }
          __syncwarp();
        }
        if (ok && lane == 0) {
          umma_commit_pair_both(tfull_bar(acc));
        }
        __syncwarp();
      }
      if (p.timers && lane == 0) {
        atomicAdd(p.timers + 2, static_cast<unsigned long long>(clock64() - t_begin));
        atomicAdd(p.timers + 3, static_cast<unsigned long long>(t_acc));
        atomicAdd(p.timers + 4, static_cast<unsigned long long>(t_full));
      }
      if (!ok) {
        // gave up: let every MMA issued so far finish (bounded) before the pair's tensor memory is freed
        if (lane == 0) {
          record_status(p.status, DEV_TIMEOUT, 1200 + KIND);
          umma_commit_pair_both(bar0 + 8u * (2 * STAGES2 + 4));
        }
        __syncwarp();
        mbar_wait(bar0 + 8u * (2 * STAGES2 + 4), 0u);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps per CTA, own 128 rows:
    // two warps per TMEM lane quadrant, each draining half of the tile's columns)
    const int ew = warp & 3;
    const int half = (warp - 2) >> 2;
    EpiStage es{smem_base + STAGES2 * STAGE2_BYTES + (warp - 2) * (EPI_UNITS * EPI_UNIT_BYTES), 0u};
    uint32_t tc = 0;
    bool ok = true;
    long long t_idle = 0, t_begin = clock64();
    for (int rd = 0; rd * nclusters < ntiles && ok; ++rd) {
      const int t = tile_of_round<KIND>(rd, cid, nclusters);
      if (t >= ntiles) continue;
      const Tile2 tl = get_tile2<KIND>(p, t, rank);
      const int rin = ew * 32 + lane;
      if (tl.nkb == 0) {
        if (TR::WGRAD && half == 0) wgrad_zero_fill<KIND>(p, tl.e, tl.m0 + rin, tl.n0);
        continue;
      }
      const int acc = tc & 1;
      const uint32_t aph = (tc >> 1) & 1u;
      ++tc;
      epilogue_prefetch<KIND>(p, static_cast<int64_t>(tl.row0) + rin, tl.n0, tl.write && half == 0, tl.e, tl.m0 + rin);
      const long long w0 = clock64();
      if (!mbar_wait(tfull_bar(acc), aph)) {
        ok = false;
        break;
      }
      t_idle += clock64() - w0;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(ew * 32) << 16) + acc * ACC_COLS;
      expert_epilogue<KIND>(p, tl.e, static_cast<int64_t>(tl.row0) + rin, (TR::WGRAD ? tl.m0 : tl.row0) + ew * 32, tl.n0, taddr,
                            tl.write, TR::WGRAD ? p.M_total - (tl.m0 + ew * 32) : 32, es, lane, half, 2);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(acc), 0));
    }
    if (p.timers && lane == 0 && ew == 0 && half == 0 && leader) {
      atomicAdd(p.timers + 5, static_cast<unsigned long long>(clock64() - t_begin));
      atomicAdd(p.timers + 6, static_cast<unsigned long long>(t_idle));
      atomicAdd(p.timers + 7, 1ull);
    }
    if (!ok && lane == 0) {
      record_status(p.status, DEV_TIMEOUT, 1300 + KIND);
    }
  }

  tc_fence_before();
  cluster_sync_all();  // the partner has stopped using this CTA's shared memory, barriers and tensor memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

template <int KIND>
static moe_status launch_pair_kind(moe_ctx_impl* ctx, const GemmParams& p, cudaStream_t st) {
  if (!ctx->attr_done[1][KIND]) {  // per device: the context is bound to one
    if (cudaFuncSetAttribute(grouped_gemm_pair_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(GEMM2_SMEM)) != cudaSuccess)
      return MOE_ERR_CUDA;
    ctx->attr_done[1][KIND] = 1;
  }
  const int grid = ctx->sm_count & ~1;  // whole pairs
  grouped_gemm_pair_kernel<KIND><<<grid, GEMM2_THREADS, GEMM2_SMEM, st>>>(p);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status launch_pair_gemm(moe_ctx_impl* ctx, GemmKind kind, const GemmParams& p, cudaStream_t st) {
  switch (kind) {
    case GEMM_F3: return launch_pair_kind<GEMM_F3>(ctx, p, st);
    case GEMM_F4: return launch_pair_kind<GEMM_F4>(ctx, p, st);
    case GEMM_B2: return launch_pair_kind<GEMM_B2>(ctx, p, st);
    case GEMM_B3: return launch_pair_kind<GEMM_B3>(ctx, p, st);
    case GEMM_B4: return launch_pair_kind<GEMM_B4>(ctx, p, st);
    case GEMM_B5: return launch_pair_kind<GEMM_B5>(ctx, p, st);
    default: return MOE_ERR_INVALID_ARG;
  }
}

}  // namespace moe
