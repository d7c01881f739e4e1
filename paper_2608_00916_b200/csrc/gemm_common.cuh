// Shared pieces of the tcgen05 grouped-GEMM kernels: tile geometry, kernel parameters, per-kind traits, the tile
// descriptor and the register-level store / load helpers used by the epilogues.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace moe {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;       // 16 KB
constexpr int B_BYTES = BN * BK * 2;       // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int CHUNK_BYTES = 64 * BK * 2;   // one 64-wide MN chunk of an MN-major tile: 8 KB
constexpr int GEMM_THREADS = 320;  // one-CTA kernel, warps: 0 TMA producer, 1 MMA issuer, 2..9 epilogue (two per TMEM lane
                                   // quadrant, each taking half of the tile's columns)
constexpr int ACC_COLS = 256;
constexpr int TMEM_COLS = 512;
// Epilogue staging: every epilogue warp owns EPI_UNITS units of 32 rows x 32 bf16 columns (64-byte rows, XOR
// swizzle) through which it transposes its results for coalesced global stores.
constexpr int EPI_UNIT_BYTES = 32 * 64;
constexpr int EPI_UNITS = 2;
constexpr int EPI_BYTES = 8 * EPI_UNITS * EPI_UNIT_BYTES;  // up to 8 epilogue warps: 32 KB
constexpr size_t GEMM_SMEM = static_cast<size_t>(STAGES) * STAGE_BYTES + EPI_BYTES + 1024;

struct GemmParams {
  CUtensorMap mapA0, mapA1, mapB0, mapB1;
  CUtensorMap mapA2, mapB2, mapB3;  // operands of the optional extra K segment (low-rank adapter path)
  const int32_t* sched;        // [0] number of 128-row tiles
  const int32_t* tile_expert;  // expert of each 128-row tile
  const int32_t* pad_offsets;  // padded segment starts, E + 1 entries
  const int32_t* counts;       // rows per expert (weight gradients stop their K loop at the last 64-row block with data)
  const int32_t* expert_order; // weight gradients: experts by row count, largest first
  const int32_t* pair_tab;     // CTA-pair kernels: per pair of row blocks {expert, first row, blocks (1|2), 0}
  int pair_count_slot;         // which entry of sched holds the number of entries of pair_tab
  int oob_row;                 // a row index beyond the row buffers: TMA copies from there deliver zeros
  int row_group;               // row GEMMs: consecutive row tiles (or pairs) walked together inside one column tile
  const int32_t* tile_list;    // one-CTA row GEMMs: null = every 128-row tile, else the tiles to compute (sched[4] entries)
  int32_t* status;
  unsigned long long* timers;  // null, or 8 counters of this kind: summed over CTAs (see gemm.cu)
  int n_tiles;   // output tiles along N
  int m_tiles;   // weight gradients: output tiles along M per expert
  int E;         // weight gradients: number of experts this launch covers
  int e_first;   // weight gradients: first expert of the launch when it covers a range (expert_grouped), else unused
  int expert_grouped;  // weight gradients: 1 = experts e_first .. e_first + E - 1 in index order, 0 = all, largest first
  int k_blocks;  // row GEMMs: K blocks per segment
  int nseg;      // row GEMMs: K segments of k_blocks blocks (B4, DX: up to 2)
  int k_blocks1; // row GEMMs: K blocks of the extra segment that follows them (0: none)
  float out_scale;  // plain epilogues multiply the accumulator by this
  int M_total;   // weight gradients: rows of one expert's output
  int N_total;   // columns of the output
  uint16_t* out0;
  uint16_t* out1;
  uint16_t* out2;
  const uint16_t* in0;
  const uint16_t* in1;
  int64_t ld_out;
  int64_t expert_stride;
  // router kinds
  int b_chunks;         // 64-column chunks of an MN-major B tile actually loaded (4 = the whole 256-wide tile)
  int mma_n;            // N of the MMA (256 unless the B tile is narrower)
  uint32_t stage_tx;    // bytes one stage's loads deliver
  int static_m_tiles;   // RT, DX: number of 128-token tiles
  int split_rows;       // DWR: tokens per slice (multiple of 64)
  int rows_total;       // DWR: tokens rounded up to 64
  int top_k;
  int64_t T;
  const float* bias;    // RT: [E] or null
  float* logits;        // RT: [T,E] saved logits
  float* logits_out;    // RT: optional copy for the caller
  int32_t* idx;         // RT: [T,k] (workspace) and idx_out (caller)
  int32_t* idx_out;
  float* gates;
  float* gates_out;
  float* psum_part;     // RT: [4 * tiles, E] per-warp column sums of p
  int32_t* tile_counts; // RT: [tiles, E] histogram of the picks of every 128-token tile (null: not produced here)
  float* outf;          // DWR: [slices, d, E] fp32 partials; B2: [column tiles, rows_max] partial sums of dg
  float* accf0;         // B3, B5 in accumulate mode: fp32 weight-gradient buffers that the tile is ADDED to
  float* accf1;
  int acc_fp32;
  const float* row_gate;  // F3, B2: gate of every padded row (0 for pad rows)
  int save_pre;         // F3: 1 = also store hg, hu (training), 0 = only the activation (forward-only calls)
  int64_t rows_max;     // B2: stride of the dg partial slices
};

template <int KIND>
struct Traits {
  static constexpr bool WGRAD = (KIND == GEMM_B3 || KIND == GEMM_B5 || KIND == GEMM_DWR);
  static constexpr bool STATIC_M = (KIND == GEMM_RT || KIND == GEMM_DX);  // token tiles, no expert lookup
  static constexpr int A_MN = WGRAD ? 1 : 0;
  static constexpr int B_MN = (KIND == GEMM_B2 || KIND == GEMM_B4 || KIND == GEMM_DX) ? 0 : 1;
  // width of output covered by one N tile (F3 / B5 / DWR pair a 128-wide tile with a second 128-wide operand)
  static constexpr int N_SPAN = (KIND == GEMM_F3 || KIND == GEMM_B5 || KIND == GEMM_DWR) ? 128 : 256;
};

// K = 16 steps of the last 64-deep K block that hold any of an expert's `count` rows (the rows after them are zeros).
__device__ __forceinline__ int last_k_steps(int count) { return count > 0 ? ((count - 1) % BK) / 16 + 1 : BK / 16; }

struct Tile {
  int e, row0, m0, n0, nkb;
  int klast = BK / 16;  // K = 16 steps issued in the last K block (weight gradients stop at the expert's last row)
};

// Static tile assignment of the persistent kernels: worker `w` of `nw` takes one tile per round.  Weight-gradient
// tiles are ordered longest first, so odd rounds run through the workers backwards (a snake): the worker that got the
// longest tile of one round gets the shortest of the next, which evens out skewed expert loads.
template <int KIND>
__device__ __forceinline__ int tile_of_round(int round, int w, int nw) {
  return round * nw + ((Traits<KIND>::WGRAD && (round & 1)) ? nw - 1 - w : w);
}

template <int KIND>
__device__ __forceinline__ int total_tiles(const GemmParams& p) {
  if (Traits<KIND>::WGRAD) return p.E * p.m_tiles * p.n_tiles;
  if (Traits<KIND>::STATIC_M) return p.static_m_tiles * p.n_tiles;
  return (p.tile_list ? p.sched[4] : p.sched[0]) * p.n_tiles;
}

// Order of the tiles of a row GEMM.  group == 1: column tiles fastest (the tiles of one row tile are adjacent; right
// when an expert's weights stay in L2 anyway).  group > 1: `group` consecutive row tiles are walked together inside
// one column tile before the next column tile starts, so that a B tile of a wide expert (whose weight slab does not
// fit in L2) is fetched from DRAM once for the whole group instead of once per row tile.
__device__ __forceinline__ void row_tile_order(int t, int n_tiles, int group, int n_rows, int& ri, int& nt) {
  if (group <= 1) {
    ri = t / n_tiles;
    nt = t - ri * n_tiles;
    return;
  }
  const int per = group * n_tiles;
  const int g = t / per, rem = t - g * per;
  const int base = g * group;
  const int gsz = min(group, n_rows - base);  // the last group may be short
  nt = rem / gsz;
  ri = base + rem - nt * gsz;
}

template <int KIND>
__device__ __forceinline__ Tile get_tile(const GemmParams& p, int t) {
  Tile tl;
  if (Traits<KIND>::WGRAD) {
    const int per = p.m_tiles * p.n_tiles;
    tl.e = t / per;
    const int rem = t - tl.e * per;
    tl.m0 = (rem / p.n_tiles) * BM;
    tl.n0 = (rem % p.n_tiles) * Traits<KIND>::N_SPAN;
    if (KIND != GEMM_DWR) tl.e = p.expert_grouped ? p.e_first + tl.e : p.expert_order[tl.e];  // else: longest K loops first
    if (KIND == GEMM_DWR) {  // "expert" = token slice
      tl.row0 = tl.e * p.split_rows;
      tl.nkb = max(0, min(p.split_rows, p.rows_total - tl.row0)) / BK;
    } else {
      tl.row0 = p.pad_offsets[tl.e];
      tl.nkb = (p.counts[tl.e] + BK - 1) / BK;  // the rest of the 128-row padding is zeros
      tl.klast = last_k_steps(p.counts[tl.e]);
    }
  } else if (Traits<KIND>::STATIC_M) {
    const int mt = t / p.n_tiles;
    tl.e = 0;
    tl.row0 = mt * BM;
    tl.m0 = 0;
    tl.n0 = (t % p.n_tiles) * Traits<KIND>::N_SPAN;
    tl.nkb = p.k_blocks * p.nseg + p.k_blocks1;
  } else {
    int ri, nt;
    row_tile_order(t, p.n_tiles, p.row_group, p.tile_list ? p.sched[4] : p.sched[0], ri, nt);
    const int mt = p.tile_list ? p.tile_list[ri] : ri;
    tl.e = p.tile_expert[mt];
    tl.row0 = mt * BM;
    tl.m0 = 0;
    tl.n0 = nt * Traits<KIND>::N_SPAN;
    tl.nkb = p.k_blocks * p.nseg + p.k_blocks1;
  }
  return tl;
}

// Loads of one K block: the A tile and the B tile of the stage, all credited to the stage's full barrier.
// (Issuing A and B from two producer warps was tried: the producer's time is back-pressure from the L2 -> SM
// path, not instruction issue, so it gained nothing.)
template <int KIND>
__device__ __forceinline__ void issue_loads(const GemmParams& p, const Tile& tl, int kb, uint32_t sA, uint32_t sB,
                                            uint32_t bar) {
  if (!Traits<KIND>::WGRAD && kb >= p.k_blocks * p.nseg) {
    // extra K segment of a row GEMM: A = a 64-wide row buffer (x A1, act A2, ... of the low-rank adapters),
    // B = the matching adapter matrix of expert e
    const int kk = kb - p.k_blocks * p.nseg;
    tma_load_2d(sA, &p.mapA2, bar, kk * BK, tl.row0);
    if (KIND == GEMM_F3) {
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        tma_load_3d(sB + c * CHUNK_BYTES, &p.mapB2, bar, tl.n0 + c * 64, kk * BK, tl.e);
        tma_load_3d(sB + (2 + c) * CHUNK_BYTES, &p.mapB3, bar, tl.n0 + c * 64, kk * BK, tl.e);
      }
    } else if (KIND == GEMM_F4) {
#pragma unroll
      for (int c = 0; c < 4; ++c) tma_load_3d(sB + c * CHUNK_BYTES, &p.mapB2, bar, tl.n0 + c * 64, kk * BK, tl.e);
    } else {  // B2, B4: K-major adapter matrix, one box
      tma_load_3d(sB, &p.mapB2, bar, kk * BK, tl.n0, tl.e);
    }
    return;
  }
  if (KIND == GEMM_F3) {
    tma_load_2d(sA, &p.mapA0, bar, kb * BK, tl.row0);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      tma_load_3d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, kb * BK, tl.e);
      tma_load_3d(sB + (2 + c) * CHUNK_BYTES, &p.mapB1, bar, tl.n0 + c * 64, kb * BK, tl.e);
    }
  } else if (KIND == GEMM_RT) {
    // one K segment per bf16 term of the router weight (one term for a bf16 weight, three for an fp32 weight)
    const int seg = kb / p.k_blocks, kk = kb - seg * p.k_blocks;
    const CUtensorMap* mb = seg == 0 ? &p.mapB0 : (seg == 1 ? &p.mapB1 : &p.mapB2);
    tma_load_2d(sA, &p.mapA0, bar, kk * BK, tl.row0);
#pragma unroll
    for (int c = 0; c < 4; ++c)
      if (c < p.b_chunks) tma_load_3d(sB + c * CHUNK_BYTES, mb, bar, tl.n0 + c * 64, kk * BK, tl.e);
  } else if (KIND == GEMM_F4) {
    tma_load_2d(sA, &p.mapA0, bar, kb * BK, tl.row0);
#pragma unroll
    for (int c = 0; c < 4; ++c)
      if (c < p.b_chunks) tma_load_3d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, kb * BK, tl.e);
  } else if (KIND == GEMM_B2) {
    tma_load_2d(sA, &p.mapA0, bar, kb * BK, tl.row0);
    tma_load_3d(sB, &p.mapB0, bar, kb * BK, tl.n0, tl.e);
  } else if (KIND == GEMM_B4 || KIND == GEMM_DX) {
    const int seg = kb / p.k_blocks, kk = kb - seg * p.k_blocks;  // DX: a third segment with an fp32 router weight
    tma_load_2d(sA, seg == 0 ? &p.mapA0 : (seg == 1 ? &p.mapA1 : &p.mapA2), bar, kk * BK, tl.row0);
    tma_load_3d(sB, seg == 0 ? &p.mapB0 : (seg == 1 ? &p.mapB1 : &p.mapB2), bar, kk * BK, tl.n0, tl.e);
  } else if (KIND == GEMM_B3) {
    const int row = tl.row0 + kb * BK;
#pragma unroll
    for (int c = 0; c < 2; ++c) tma_load_2d(sA + c * CHUNK_BYTES, &p.mapA0, bar, tl.m0 + c * 64, row);
#pragma unroll
    for (int c = 0; c < 4; ++c)
      if (c < p.b_chunks) tma_load_2d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, row);
  } else {  // GEMM_B5, GEMM_DWR
    const int row = tl.row0 + kb * BK;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      tma_load_2d(sA + c * CHUNK_BYTES, &p.mapA0, bar, tl.m0 + c * 64, row);
      tma_load_2d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, row);
      tma_load_2d(sB + (2 + c) * CHUNK_BYTES, &p.mapB1, bar, tl.n0 + c * 64, row);
    }
  }
}

__device__ __forceinline__ float fast_sigmoid(float h) { return __fdividef(1.f, 1.f + __expf(-h)); }


// ---------------------------------------------------------------------------------------------- expert epilogues
// One thread owns one accumulator row (TMEM lane) of a 128 x 256 tile; a warp owns a slab of 32 rows.  Results
// leave through shared memory: the warp writes a 32 x 32 bf16 unit (lane = row; 16-byte pieces placed with a
// 64-byte XOR swizzle so both directions are conflict-free), then reads it back transposed - four consecutive lanes
// hold one 64-byte row segment - and stores that to global memory, eight full row segments per instruction.
// Measured alternatives on the Qwen shape: 16-byte stores from each lane to its own row cost one memory wavefront
// per lane (GEMMs at 0.66 of their store-free speed); TMA stores from the same staging queue up behind the
// producer's deep ring of TMA loads and stall the accumulator hand-off (0.72).
struct EpiStage {
  uint32_t base;  // shared address of this warp's two units (2 KB each)
  uint32_t n;     // units written so far
};

__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// out points at (first row of the slab, first of the 32 columns); rows_valid = rows of the slab inside the tensor.
__device__ __forceinline__ void stage_store32(EpiStage& es, uint16_t* out, int64_t ld, int rows_valid,
                                              const float (&v)[32], int lane, int cols_valid = 32) {
  const uint32_t unit = es.base + (es.n & 1u) * EPI_UNIT_BYTES;
  ++es.n;
  const uint32_t rowaddr = unit + lane * 64;
  const uint32_t sw = (lane >> 1) & 3;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    st_shared_v4(rowaddr + ((j ^ sw) << 4), pack_bf16x2(v[8 * j + 0], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                 pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
  __syncwarp();  // also orders this unit's reads of two calls ago before its reuse
  const int ch = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = (lane >> 2) + 8 * i;
    const uint4 w = ld_shared_v4(unit + r * 64 + ((ch ^ ((r >> 1) & 3)) << 4));
    if (r < rows_valid && ch * 8 < cols_valid) *reinterpret_cast<uint4*>(out + r * ld + ch * 8) = w;
  }
}

// fp32 accumulate variant for the weight gradients: out[r, 0..31] += v for the 32 rows of the slab.  The 32 x 32 fp32
// unit (4 KB = both staging units of the warp) is written one row per lane and read back with eight lanes per
// 128-byte row segment, so the global read-modify-write is coalesced.  The old values are loaded by the caller one
// chunk ahead (accum_load) so that their latency overlaps the previous chunk's work.
__device__ __forceinline__ void accum_load(const float* out, int64_t ld, int rows_valid, int lane, float4 (&g)[8]) {
  const int ch = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = (lane >> 3) + 4 * i;
    if (r < rows_valid) g[i] = *reinterpret_cast<const float4*>(out + r * ld + ch * 4);
  }
}
__device__ __forceinline__ void stage_accum32(EpiStage& es, float* out, int64_t ld, int rows_valid,
                                              const float (&v)[32], const float4 (&g)[8], int lane) {
  const uint32_t unit = es.base;
  __syncwarp();  // reads of the previous use are done
  const uint32_t rowaddr = unit + lane * 128;
  const uint32_t sw = lane & 7;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    st_shared_v4(rowaddr + ((j ^ sw) << 4), __float_as_uint(v[4 * j + 0]), __float_as_uint(v[4 * j + 1]),
                 __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
  __syncwarp();
  const int ch = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = (lane >> 3) + 4 * i;
    const uint4 w = ld_shared_v4(unit + r * 128 + ((ch ^ (r & 7)) << 4));
    if (r < rows_valid) {
      float4 a = g[i];
      a.x += __uint_as_float(w.x);
      a.y += __uint_as_float(w.y);
      a.z += __uint_as_float(w.z);
      a.w += __uint_as_float(w.w);
      *reinterpret_cast<float4*>(out + r * ld + ch * 4) = a;
    }
  }
}

// `slab` is the first output row of the warp's 32-row slab (row of the padded row buffers for row GEMMs, row of
// the expert's weight-gradient slab for weight gradients); `row` is the thread's own row (only the SwiGLU-backward
// epilogue reads through it).  `write` (warp-uniform) is false for a tile half whose rows do not exist; `rows_valid`
// clips a slab that overhangs the tensor.  Every tcgen05.ld is executed by all lanes.
template <int KIND>
__device__ __forceinline__ void expert_epilogue(const GemmParams& p, int e, int64_t row, int slab, int n0,
                                                uint32_t taddr, bool write, int rows_valid, EpiStage& es, int lane,
                                                int half = 0, int nhalf = 1) {
  // with two epilogue warps per lane quadrant (nhalf = 2) this warp handles half of the 32-column chunks
  const int c4_lo = half * (4 / nhalf), c4_hi = c4_lo + 4 / nhalf;  // of 4 chunks (F3: gate + up pairs)
  const int c8_lo = half * (8 / nhalf), c8_hi = c8_lo + 8 / nhalf;  // of 8 chunks
  if (KIND == GEMM_F3) {
#pragma unroll 1
    for (int c = c4_lo; c < c4_hi; ++c) {
      uint32_t rg[32], ru[32];
      tmem_ld32(taddr + c * 32, rg);
      tmem_ld32(taddr + 128 + c * 32, ru);
      tmem_ld_wait();
      const int col = n0 + c * 32;
      if (write && col < p.N_total) {
        float t[32];
        const float gate = p.row_gate[row];  // the combine weight is folded into the saved activation
        if (p.save_pre) {
#pragma unroll
          for (int i = 0; i < 32; ++i) t[i] = __uint_as_float(rg[i]);
          stage_store32(es, p.out0 + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid, t, lane);
#pragma unroll
          for (int i = 0; i < 32; ++i) t[i] = __uint_as_float(ru[i]);
          stage_store32(es, p.out1 + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid, t, lane);
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float hg = __uint_as_float(rg[i]);
          t[i] = gate * hg * fast_sigmoid(hg) * __uint_as_float(ru[i]);
        }
        stage_store32(es, p.out2 + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid, t, lane);
      }
    }
  } else if (KIND == GEMM_B2) {
    // hg, hu of the warp's 32 rows x 32 columns arrive one chunk ahead of their use as coalesced pieces (four lanes
    // per 64-byte row segment, eight rows per load instruction) and are transposed through the warp's two staging
    // units so that every thread ends up with its own row.  (A thread fetching its own row directly costs one memory
    // wavefront per lane and load: 256 wavefronts per chunk instead of 64.)
    uint4 nh[4], nu[4];
    const float gate = write ? p.row_gate[row] : 0.f;
    float dgp = 0.f;  // this row's share of dg = <dy, o> = <da, silu(hg) hu> over the tile's columns
    const int pr = lane >> 2, pc = (lane & 3) * 8;  // piece: rows pr + 8 i of the slab, 8 columns from pc
    auto fetch = [&](int col) {
      const uint16_t* qh = p.in0 + (static_cast<int64_t>(slab) + pr) * p.ld_out + col + pc;
      const uint16_t* qu = p.in1 + (static_cast<int64_t>(slab) + pr) * p.ld_out + col + pc;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        nh[i] = __ldg(reinterpret_cast<const uint4*>(qh + static_cast<int64_t>(8 * i) * p.ld_out));
        nu[i] = __ldg(reinterpret_cast<const uint4*>(qu + static_cast<int64_t>(8 * i) * p.ld_out));
      }
    };
    if (write && n0 + c8_lo * 32 < p.N_total) fetch(n0 + c8_lo * 32);
    const uint32_t unit_h = es.base, unit_u = es.base + EPI_UNIT_BYTES;
#pragma unroll 1
    for (int c = c8_lo; c < c8_hi; ++c) {
      const int col = n0 + c * 32;
      const bool live = write && col < p.N_total;
      uint4 ch[4], cu[4];
      if (live) {
        __syncwarp();  // the previous chunk's output reads of both units are done
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = pr + 8 * i;
          const uint32_t a = r * 64 + (((lane & 3) ^ ((r >> 1) & 3)) << 4);
          st_shared_v4(unit_h + a, nh[i].x, nh[i].y, nh[i].z, nh[i].w);
          st_shared_v4(unit_u + a, nu[i].x, nu[i].y, nu[i].z, nu[i].w);
        }
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t a = lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4);
          ch[j] = ld_shared_v4(unit_h + a);
          cu[j] = ld_shared_v4(unit_u + a);
        }
        __syncwarp();  // both units are free for the output staging below
      }
      if (write && c + 1 < c8_hi && col + 32 < p.N_total) fetch(col + 32);
      uint32_t rd[32];
      tmem_ld32(taddr + c * 32, rd);
      tmem_ld_wait();
      if (live) {
        float hg[32], hu[32], t[32];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unpack_bf16x2(ch[i].x, hg[8 * i + 0], hg[8 * i + 1]);
          unpack_bf16x2(ch[i].y, hg[8 * i + 2], hg[8 * i + 3]);
          unpack_bf16x2(ch[i].z, hg[8 * i + 4], hg[8 * i + 5]);
          unpack_bf16x2(ch[i].w, hg[8 * i + 6], hg[8 * i + 7]);
          unpack_bf16x2(cu[i].x, hu[8 * i + 0], hu[8 * i + 1]);
          unpack_bf16x2(cu[i].y, hu[8 * i + 2], hu[8 * i + 3]);
          unpack_bf16x2(cu[i].z, hu[8 * i + 4], hu[8 * i + 5]);
          unpack_bf16x2(cu[i].w, hu[8 * i + 6], hu[8 * i + 7]);
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float sg = fast_sigmoid(hg[i]);
          const float da = __uint_as_float(rd[i]);  // dy W_down^T without the gate
          dgp = fmaf(da, hg[i] * sg * hu[i], dgp);
          const float dag = gate * da;
          hu[i] = dag * hu[i] * sg * (1.f + hg[i] * (1.f - sg));  // dhg
          t[i] = dag * hg[i] * sg;                                 // dhu
        }
        es.n = 0;  // outputs go through unit 0, then unit 1
        stage_store32(es, p.out0 + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid, hu, lane);
        stage_store32(es, p.out1 + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid, t, lane);
      }
    }
    // two partial slices per column tile, one per epilogue warp of the lane quadrant
    if (write) {
      p.outf[static_cast<int64_t>(n0 / 256 * 2 + half) * p.rows_max + row] = dgp;
      if (nhalf == 1) p.outf[static_cast<int64_t>(n0 / 256 * 2 + 1) * p.rows_max + row] = 0.f;
    }
  } else if (Traits<KIND>::WGRAD && KIND != GEMM_DWR && p.acc_fp32) {
    // accumulate mode of the weight gradients: fp32 read-modify-write, old values fetched one chunk ahead
    auto dst_of = [&](int c) -> float* {
      float* fb = (KIND == GEMM_B5 && c >= 4) ? p.accf1 : p.accf0;
      const int col = (KIND == GEMM_B5) ? n0 + (c & 3) * 32 : n0 + c * 32;
      return (write && col < p.N_total) ? fb + e * p.expert_stride + static_cast<int64_t>(slab) * p.ld_out + col : nullptr;
    };
    float4 gn[8];
    float* dn = dst_of(c8_lo);
    if (dn) accum_load(dn, p.ld_out, rows_valid, lane, gn);
#pragma unroll 1
    for (int c = c8_lo; c < c8_hi; ++c) {
      float4 g[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) g[i] = gn[i];
      float* dc = dn;
      dn = c + 1 < c8_hi ? dst_of(c + 1) : nullptr;
      if (dn) accum_load(dn, p.ld_out, rows_valid, lane, gn);
      uint32_t rd[32];
      tmem_ld32(taddr + c * 32, rd);
      tmem_ld_wait();
      float v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(rd[i]);
      if (dc) stage_accum32(es, dc, p.ld_out, rows_valid, v, g, lane);
    }
  } else {
    // plain bf16 store: F4, B4, DX (row GEMMs), B3, B5 (weight gradients)
#pragma unroll 1
    for (int c = c8_lo; c < c8_hi; ++c) {
      uint32_t rd[32];
      tmem_ld32(taddr + c * 32, rd);
      tmem_ld_wait();
      float v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(rd[i]) * p.out_scale;
      uint16_t* base = p.out0;
      int col = n0 + c * 32;
      if (KIND == GEMM_B5) {
        base = (c >= 4) ? p.out1 : p.out0;
        col = n0 + (c & 3) * 32;
      }
      if (Traits<KIND>::WGRAD) {
        if (write && col < p.N_total)
          stage_store32(es, base + e * p.expert_stride + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid,
                        v, lane, p.N_total - col);
      } else {
        if (write && col < p.N_total)
          stage_store32(es, base + static_cast<int64_t>(slab) * p.ld_out + col, p.ld_out, rows_valid, v, lane,
                        p.N_total - col);
      }
    }
  }
}

// Called by an epilogue thread before it starts waiting for the tile's accumulator: the SwiGLU-backward epilogue
// reads hg and hu of its row from global memory, and those rows come straight from DRAM.  Pulling their lines
// into L2 while the tile's main loop still runs keeps the epilogue from stalling on each 32-column chunk (it was
// the slower side of this kernel: accumulators waited for it).
template <int KIND>
__device__ __forceinline__ void epilogue_prefetch(const GemmParams& p, int64_t row, int n0, bool write, int e = 0,
                                                  int m = 0) {
  if ((KIND == GEMM_B3 || KIND == GEMM_B5) && p.acc_fp32 && write && m < p.M_total) {
    // accumulate mode: this thread's row of the fp32 gradient tile (1 KB) will be read by the epilogue
    const int span = KIND == GEMM_B5 ? 128 : 256;
    const int cols = min(span, p.N_total - n0);
    const float* a0 = p.accf0 + e * p.expert_stride + static_cast<int64_t>(m) * p.ld_out + n0;
    for (int c = 0; c < cols; c += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(a0 + c));
    if (KIND == GEMM_B5) {
      const float* a1 = p.accf1 + e * p.expert_stride + static_cast<int64_t>(m) * p.ld_out + n0;
      for (int c = 0; c < cols; c += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(a1 + c));
    }
  }
  if (KIND == GEMM_B2 && write) {
    const int cols = min(256, p.N_total - n0);
    const uint16_t* h = p.in0 + row * p.ld_out + n0;
    const uint16_t* u = p.in1 + row * p.ld_out + n0;
    for (int c = 0; c < cols; c += 64) {
      asm volatile("prefetch.global.L2 [%0];" ::"l"(h + c));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(u + c));
    }
  }
}

// Weight gradient of an expert without tokens: the thread's row of the output tile is zero.
template <int KIND>
__device__ __forceinline__ void wgrad_zero_fill(const GemmParams& p, int e, int m, int n0) {
  if (m >= p.M_total || p.acc_fp32) return;  // accumulate mode: an expert without tokens adds nothing
  constexpr int span = (KIND == GEMM_B5) ? 128 : 256;
  const int cols = min(span, p.N_total - n0);
  for (int c = 0; c < cols; c += 8) {  // 16-byte pieces: the output width is a multiple of 8
    const int64_t off = e * p.expert_stride + static_cast<int64_t>(m) * p.ld_out + n0 + c;
    *reinterpret_cast<uint4*>(p.out0 + off) = make_uint4(0, 0, 0, 0);
    if (KIND == GEMM_B5) *reinterpret_cast<uint4*>(p.out1 + off) = make_uint4(0, 0, 0, 0);
  }
}

// ---------------------------------------------------------------------------------------------- routing epilogues
// One thread per token (TMEM lane).  Pass j picks the largest logit that comes after pick j-1 in the order (value
// descending, index ascending), which is the rule "largest not taken yet, lowest index among equals" without a
// "taken" mask.  Gates are the softmax over the picked logits; the softmax over all E logits is summed per
// column with a butterfly transpose-reduce (lane L ends with column L), one partial row per warp, fixed order.
//
// Generic version (any E <= 256): the row of logits is re-read from tensor memory in every pass.
__device__ __forceinline__ void routing_epilogue_tmem(const GemmParams& p, const float* s_bias, int64_t row, int tile,
                                                      int ew, uint32_t taddr, int lane) {
        const int64_t tok = row;
        const bool valid = tok < p.T;
        const int E = p.N_total, k = p.top_k;
        const int nch = (E + 31) >> 5;
        float selv[MAX_K];
        int seli[MAX_K];
        float pv = INFINITY;
        int pi = -1;
        for (int j = 0; j < k; ++j) {
          float bv = -INFINITY;
          int bi = 0x7FFFFFFF;
          for (int c = 0; c < nch; ++c) {
            uint32_t r[32];
            tmem_ld32(taddr + c * 32, r);
            tmem_ld_wait();
            float val[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) val[i] = __uint_as_float(r[i]) + s_bias[c * 32 + i];
            if (j == 0 && valid) {
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                if (c * 32 + i < E) {
                  const float4 w = make_float4(val[i], val[i + 1], val[i + 2], val[i + 3]);
                  *reinterpret_cast<float4*>(p.logits + tok * E + c * 32 + i) = w;
                  if (p.logits_out) *reinterpret_cast<float4*>(p.logits_out + tok * E + c * 32 + i) = w;
                }
              }
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int e = c * 32 + i;
              const bool after = (val[i] < pv) || (val[i] == pv && e > pi);
              if (e < E && after && val[i] > bv) {
                bv = val[i];
                bi = e;
              }
            }
          }
          selv[j] = bv;
          seli[j] = bi;
          pv = bv;
          pi = bi;
        }
        const float vmax = selv[0];
        float z = 0.f;
        for (int c = 0; c < nch; ++c) {
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c * 32 + i < E) z += expf(__uint_as_float(r[i]) + s_bias[c * 32 + i] - vmax);
        }
        const float rz = valid ? 1.f / z : 0.f;
        for (int c = 0; c < nch; ++c) {
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          tmem_ld_wait();
          float pc[32];
#pragma unroll
          for (int i = 0; i < 32; ++i)
            pc[i] = (c * 32 + i < E) ? expf(__uint_as_float(r[i]) + s_bias[c * 32 + i] - vmax) * rz : 0.f;
          // column sums over the 32 tokens of this warp: butterfly transpose-reduce, lane L ends with column L
#pragma unroll
          for (int off = 16, cnt = 16; off >= 1; off >>= 1, cnt >>= 1) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              if (i < cnt) {
                const bool up = (lane & off) != 0;
                const float send = up ? pc[i] : pc[i + cnt];
                const float keep = up ? pc[i + cnt] : pc[i];
                pc[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
              }
            }
          }
          if (c * 32 + lane < E)
            p.psum_part[(static_cast<int64_t>(tile) * 4 + ew) * E + c * 32 + lane] = pc[0];
        }
        if (valid) {
          float zs = 0.f;
          for (int j = 0; j < k; ++j) zs += expf(selv[j] - vmax);
          const float rzs = 1.f / zs;
          for (int j = 0; j < k; ++j) {
            const float g = expf(selv[j] - vmax) * rzs;
            p.idx[tok * k + j] = seli[j];
            p.gates[tok * k + j] = g;
            p.idx_out[tok * k + j] = seli[j];
            p.gates_out[tok * k + j] = g;
          }
        }
}

// E <= 128, top_k <= 16.  Top-k is a three-level tournament per token: the 128 logits in groups of four, the group
// maxima in "supers" of four groups, the eight super maxima in registers.  A round takes the largest super maximum
// (lowest super among equals), then the group and the column inside it (lowest index among equals at every level,
// which is the lowest-index rule overall because the levels partition the index range in order), removes the column
// and repairs the three maxima above it.  The group of four values and the four group maxima sit in shared memory
// because the group that wins a round is only known at run time; each level is one 16-byte access.
// The code is written as rolled loops on purpose.  A CTA runs this epilogue once (one 128-token tile per CTA), so
// every instruction is fetched cold: the earlier fully unrolled versions (thousands of straight-line instructions)
// were bound by instruction fetch, not by execution - unrolling the k rounds made the epilogue twice as slow.
// Shared-memory layout (per CTA): vals[g][thread] float4 for g < 32 (64 KB), gmax[s][thread] float4 for s < 8 (16 KB),
// picks[j][thread] {value, column} for j < 16 (16 KB, in the unused tail of the first pipeline stage); consecutive
// threads touch consecutive words, so accesses are conflict-free whichever group a thread picks.
constexpr uint32_t ROUTE_SCRATCH_BYTES = 128 * 128 * 4 + 128 * 32 * 4;
constexpr int ROUTE_SMEM_MAX_K = 16;

__device__ __forceinline__ float4 lds_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts_f4(uint32_t addr, float4 v) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ float max4(float4 v) { return fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)); }
// index (0..3) of the first component equal to m
__device__ __forceinline__ int first_eq4(float4 v, float m) { return v.x == m ? 0 : (v.y == m ? 1 : (v.z == m ? 2 : 3)); }

__device__ __forceinline__ void routing_epilogue_smem(const GemmParams& p, const float* s_bias, int* s_hist,
                                                      uint32_t scratch, uint32_t picks_base, int64_t row, int tile,
                                                      int ew, uint32_t taddr, int lane) {
  const int64_t tok = row;
  const bool valid = tok < p.T;
  const int E = p.N_total, k = p.top_k;
  const int tid = ew * 32 + lane;  // token of the tile
  const uint32_t vals = scratch + tid * 16, gmx = scratch + 128 * 128 * 4 + tid * 16, picks = picks_base + tid * 8;
  constexpr uint32_t PITCH = 128 * 16;  // bytes between consecutive groups / supers of one thread
  float sm[8];
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    uint32_t r[32];
    tmem_ld32(taddr + c * 32, r);
    tmem_ld_wait();
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = (c * 32 + i < E) ? __uint_as_float(r[i]) + s_bias[c * 32 + i] : -INFINITY;
    if (valid) {
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        if (c * 32 + i < E) {
          const float4 w = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
          *reinterpret_cast<float4*>(p.logits + tok * E + c * 32 + i) = w;
          if (p.logits_out) *reinterpret_cast<float4*>(p.logits_out + tok * E + c * 32 + i) = w;
        }
      }
    }
    float gm[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 w = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      sts_f4(vals + (c * 8 + q) * PITCH, w);
      gm[q] = max4(w);
    }
    const float4 w0 = make_float4(gm[0], gm[1], gm[2], gm[3]), w1 = make_float4(gm[4], gm[5], gm[6], gm[7]);
    sts_f4(gmx + (c * 2) * PITCH, w0);
    sts_f4(gmx + (c * 2 + 1) * PITCH, w1);
    const float m0 = max4(w0), m1 = max4(w1);
#pragma unroll
    for (int q = 0; q < 8; ++q) sm[q] = (q == 2 * c) ? m0 : ((q == 2 * c + 1) ? m1 : sm[q]);
  }
  float vmax = 0.f, zs = 0.f;
#pragma unroll 1
  for (int j = 0; j < k; ++j) {
    const float best = fmaxf(fmaxf(fmaxf(sm[0], sm[1]), fmaxf(sm[2], sm[3])), fmaxf(fmaxf(sm[4], sm[5]), fmaxf(sm[6], sm[7])));
    int s = 7;
#pragma unroll
    for (int q = 6; q >= 0; --q) s = (sm[q] == best) ? q : s;
    float4 g4 = lds_f4(gmx + s * PITCH);
    const int gi = first_eq4(g4, best);
    const int g = s * 4 + gi;
    float4 v4 = lds_f4(vals + g * PITCH);
    const int ci = first_eq4(v4, best);
    if (j == 0) vmax = best;
    const float ex = __expf(best - vmax);
    zs += ex;
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(picks + j * (128 * 8)), "r"(__float_as_uint(ex)), "r"(g * 4 + ci)
                 : "memory");
    if (valid) atomicAdd(&s_hist[g * 4 + ci], 1);  // the tile's histogram (integer adds: order-free, deterministic)
    v4.x = ci == 0 ? -INFINITY : v4.x;
    v4.y = ci == 1 ? -INFINITY : v4.y;
    v4.z = ci == 2 ? -INFINITY : v4.z;
    v4.w = ci == 3 ? -INFINITY : v4.w;
    sts_f4(vals + g * PITCH, v4);
    const float ng = max4(v4);
    g4.x = gi == 0 ? ng : g4.x;
    g4.y = gi == 1 ? ng : g4.y;
    g4.z = gi == 2 ? ng : g4.z;
    g4.w = gi == 3 ? ng : g4.w;
    sts_f4(gmx + s * PITCH, g4);
    const float ns = max4(g4);
#pragma unroll
    for (int q = 0; q < 8; ++q) sm[q] = (q == s) ? ns : sm[q];
  }
  // the four epilogue warps (128 tokens) have counted their picks: the tile's row of the permutation's histogram
  asm volatile("bar.sync 1, 128;" ::: "memory");
  if (tid < E) {
    p.tile_counts[static_cast<int64_t>(tile) * E + tid] = s_hist[tid];
    s_hist[tid] = 0;  // ready for this CTA's next tile
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  // softmax over all E logits (read again from tensor memory: the shared copy has lost the picks); the exponentials
  // are parked in the shared copy until their sum is known
  float z = 0.f;
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    if (c * 32 < E) {
      uint32_t r[32];
      tmem_ld32(taddr + c * 32, r);
      tmem_ld_wait();
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 w;
        w.x = (c * 32 + 4 * q + 0 < E) ? __expf(__uint_as_float(r[4 * q + 0]) + s_bias[c * 32 + 4 * q + 0] - vmax) : 0.f;
        w.y = (c * 32 + 4 * q + 1 < E) ? __expf(__uint_as_float(r[4 * q + 1]) + s_bias[c * 32 + 4 * q + 1] - vmax) : 0.f;
        w.z = (c * 32 + 4 * q + 2 < E) ? __expf(__uint_as_float(r[4 * q + 2]) + s_bias[c * 32 + 4 * q + 2] - vmax) : 0.f;
        w.w = (c * 32 + 4 * q + 3 < E) ? __expf(__uint_as_float(r[4 * q + 3]) + s_bias[c * 32 + 4 * q + 3] - vmax) : 0.f;
        z += (w.x + w.y) + (w.z + w.w);
        sts_f4(vals + (c * 8 + q) * PITCH, w);
      }
    }
  }
  const float rz = valid ? 1.f / z : 0.f;
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    if (c * 32 < E) {
      float pc[32];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float4 w = lds_f4(vals + (c * 8 + q) * PITCH);
        pc[4 * q + 0] = w.x * rz;
        pc[4 * q + 1] = w.y * rz;
        pc[4 * q + 2] = w.z * rz;
        pc[4 * q + 3] = w.w * rz;
      }
      // column sums over the 32 tokens of this warp: butterfly transpose-reduce, lane L ends with column L
#pragma unroll
      for (int off = 16, cnt = 16; off >= 1; off >>= 1, cnt >>= 1) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          if (i < cnt) {
            const bool up = (lane & off) != 0;
            const float send = up ? pc[i] : pc[i + cnt];
            const float keep = up ? pc[i + cnt] : pc[i];
            pc[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
          }
        }
      }
      if (c * 32 + lane < E) p.psum_part[(static_cast<int64_t>(tile) * 4 + ew) * E + c * 32 + lane] = pc[0];
    }
  }
  if (valid) {
    const float rzs = 1.f / zs;
#pragma unroll 1
    for (int j = 0; j < k; ++j) {
      uint32_t exb, col;
      asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(exb), "=r"(col) : "r"(picks + j * (128 * 8)));
      const float g = __uint_as_float(exb) * rzs;
      p.idx[tok * k + j] = static_cast<int32_t>(col);
      p.gates[tok * k + j] = g;
      p.idx_out[tok * k + j] = static_cast<int32_t>(col);
      p.gates_out[tok * k + j] = g;
    }
  }
}

}  // namespace moe
