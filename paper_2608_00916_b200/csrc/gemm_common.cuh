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
constexpr int GEMM_THREADS = 192;
constexpr int ACC_COLS = 256;
constexpr int TMEM_COLS = 512;
constexpr size_t GEMM_SMEM = static_cast<size_t>(STAGES) * STAGE_BYTES + 1024;

struct GemmParams {
  CUtensorMap mapA0, mapA1, mapB0, mapB1;
  const int32_t* sched;        // [0] number of 128-row tiles
  const int32_t* tile_expert;  // expert of each 128-row tile
  const int32_t* pad_offsets;  // padded segment starts, E + 1 entries
  const int32_t* pair_tab;     // CTA-pair kernels: per pair of row blocks {expert, first row, blocks (1|2), 0}
  int32_t* status;
  int n_tiles;   // output tiles along N
  int m_tiles;   // weight gradients: output tiles along M per expert
  int E;
  int k_blocks;  // row GEMMs: K blocks per segment
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
  float* outf;          // DWR: [slices, d, E] fp32 partials
};

template <int KIND>
struct Traits {
  static constexpr bool WGRAD = (KIND == GEMM_B3 || KIND == GEMM_B5 || KIND == GEMM_DWR);
  static constexpr bool STATIC_M = (KIND == GEMM_RT || KIND == GEMM_DX);  // token tiles, no expert lookup
  static constexpr int A_MN = WGRAD ? 1 : 0;
  static constexpr int B_MN = (KIND == GEMM_B2 || KIND == GEMM_B4 || KIND == GEMM_DX) ? 0 : 1;
  static constexpr int NSEG = (KIND == GEMM_B4 || KIND == GEMM_DX) ? 2 : 1;
  // width of output covered by one N tile (F3 / B5 / DWR pair a 128-wide tile with a second 128-wide operand)
  static constexpr int N_SPAN = (KIND == GEMM_F3 || KIND == GEMM_B5 || KIND == GEMM_DWR) ? 128 : 256;
};

struct Tile {
  int e, row0, m0, n0, nkb;
};

template <int KIND>
__device__ __forceinline__ int total_tiles(const GemmParams& p) {
  if (Traits<KIND>::WGRAD) return p.E * p.m_tiles * p.n_tiles;
  if (Traits<KIND>::STATIC_M) return p.static_m_tiles * p.n_tiles;
  return p.sched[0] * p.n_tiles;
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
    if (KIND == GEMM_DWR) {  // "expert" = token slice
      tl.row0 = tl.e * p.split_rows;
      tl.nkb = max(0, min(p.split_rows, p.rows_total - tl.row0)) / BK;
    } else {
      tl.row0 = p.pad_offsets[tl.e];
      tl.nkb = (p.pad_offsets[tl.e + 1] - tl.row0) / BK;
    }
  } else if (Traits<KIND>::STATIC_M) {
    const int mt = t / p.n_tiles;
    tl.e = 0;
    tl.row0 = mt * BM;
    tl.m0 = 0;
    tl.n0 = (t % p.n_tiles) * Traits<KIND>::N_SPAN;
    tl.nkb = p.k_blocks * Traits<KIND>::NSEG;
  } else {
    const int mt = t / p.n_tiles;
    tl.e = p.tile_expert[mt];
    tl.row0 = mt * BM;
    tl.m0 = 0;
    tl.n0 = (t % p.n_tiles) * Traits<KIND>::N_SPAN;
    tl.nkb = p.k_blocks * Traits<KIND>::NSEG;
  }
  return tl;
}

template <int KIND>
__device__ __forceinline__ void issue_loads(const GemmParams& p, const Tile& tl, int kb, uint32_t sA, uint32_t sB,
                                            uint32_t bar) {
  if (KIND == GEMM_F3) {
    tma_load_2d(sA, &p.mapA0, bar, kb * BK, tl.row0);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      tma_load_3d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, kb * BK, tl.e);
      tma_load_3d(sB + (2 + c) * CHUNK_BYTES, &p.mapB1, bar, tl.n0 + c * 64, kb * BK, tl.e);
    }
  } else if (KIND == GEMM_F4 || KIND == GEMM_RT) {
    tma_load_2d(sA, &p.mapA0, bar, kb * BK, tl.row0);
#pragma unroll
    for (int c = 0; c < 4; ++c) tma_load_3d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, kb * BK, tl.e);
  } else if (KIND == GEMM_B2) {
    tma_load_2d(sA, &p.mapA0, bar, kb * BK, tl.row0);
    tma_load_3d(sB, &p.mapB0, bar, kb * BK, tl.n0, tl.e);
  } else if (KIND == GEMM_B4 || KIND == GEMM_DX) {
    const int seg = kb / p.k_blocks, kk = kb - seg * p.k_blocks;
    tma_load_2d(sA, seg ? &p.mapA1 : &p.mapA0, bar, kk * BK, tl.row0);
    tma_load_3d(sB, seg ? &p.mapB1 : &p.mapB0, bar, kk * BK, tl.n0, tl.e);
  } else if (KIND == GEMM_B3) {
    const int row = tl.row0 + kb * BK;
#pragma unroll
    for (int c = 0; c < 2; ++c) tma_load_2d(sA + c * CHUNK_BYTES, &p.mapA0, bar, tl.m0 + c * 64, row);
#pragma unroll
    for (int c = 0; c < 4; ++c) tma_load_2d(sB + c * CHUNK_BYTES, &p.mapB0, bar, tl.n0 + c * 64, row);
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

__device__ __forceinline__ void store_bf16x32(uint16_t* dst, const float (&v)[32]) {
  uint4* q = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint4 w;
    w.x = pack_bf16x2(v[8 * i + 0], v[8 * i + 1]);
    w.y = pack_bf16x2(v[8 * i + 2], v[8 * i + 3]);
    w.z = pack_bf16x2(v[8 * i + 4], v[8 * i + 5]);
    w.w = pack_bf16x2(v[8 * i + 6], v[8 * i + 7]);
    q[i] = w;
  }
}
__device__ __forceinline__ void load_bf16x32(const uint16_t* src, float (&v)[32]) {
  const uint4* q = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 w = q[i];
    unpack_bf16x2(w.x, v[8 * i + 0], v[8 * i + 1]);
    unpack_bf16x2(w.y, v[8 * i + 2], v[8 * i + 3]);
    unpack_bf16x2(w.z, v[8 * i + 4], v[8 * i + 5]);
    unpack_bf16x2(w.w, v[8 * i + 6], v[8 * i + 7]);
  }
}
__device__ __forceinline__ float fast_sigmoid(float h) { return __fdividef(1.f, 1.f + __expf(-h)); }


// ---------------------------------------------------------------------------------------------- expert epilogues
// One thread owns one accumulator row (TMEM lane) of a 128 x 256 tile.  `taddr` addresses that thread's lane
// quadrant and accumulator buffer; `row` is the row of the padded row buffers (row GEMMs), `m` the row of the
// expert's weight-gradient slab (weight gradients); `write` is false for a tile whose rows do not exist.
// All tcgen05.ld are executed by every lane (they are warp-collective); only the stores are predicated.
template <int KIND>
__device__ __forceinline__ void expert_epilogue(const GemmParams& p, int e, int64_t row, int m, int n0, uint32_t taddr,
                                                bool write) {
  if (KIND == GEMM_F3) {
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      uint32_t rg[32], ru[32];
      tmem_ld32(taddr + c * 32, rg);
      tmem_ld32(taddr + 128 + c * 32, ru);
      tmem_ld_wait();
      const int col = n0 + c * 32;
      if (write && col < p.N_total) {
        float hg[32], hu[32], a[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          hg[i] = __uint_as_float(rg[i]);
          hu[i] = __uint_as_float(ru[i]);
          a[i] = hg[i] * fast_sigmoid(hg[i]) * hu[i];
        }
        const int64_t off = row * p.ld_out + col;
        store_bf16x32(p.out0 + off, hg);
        store_bf16x32(p.out1 + off, hu);
        store_bf16x32(p.out2 + off, a);
      }
    }
  } else if (KIND == GEMM_B2) {
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
      uint32_t rd[32];
      tmem_ld32(taddr + c * 32, rd);
      tmem_ld_wait();
      const int col = n0 + c * 32;
      if (write && col < p.N_total) {
        const int64_t off = row * p.ld_out + col;
        float hg[32], hu[32], dhg[32], dhu[32];
        load_bf16x32(p.in0 + off, hg);
        load_bf16x32(p.in1 + off, hu);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float da = __uint_as_float(rd[i]);
          const float sg = fast_sigmoid(hg[i]);
          dhg[i] = da * hu[i] * sg * (1.f + hg[i] * (1.f - sg));
          dhu[i] = da * hg[i] * sg;
        }
        store_bf16x32(p.out0 + off, dhg);
        store_bf16x32(p.out1 + off, dhu);
      }
    }
  } else {
    // plain bf16 store: F4, B4 (row GEMMs), B3, B5 (weight gradients)
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
      uint32_t rd[32];
      tmem_ld32(taddr + c * 32, rd);
      tmem_ld_wait();
      float v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(rd[i]);
      if (Traits<KIND>::WGRAD) {
        uint16_t* base = p.out0;
        int col = n0 + c * 32;
        if (KIND == GEMM_B5) {
          base = (c >= 4) ? p.out1 : p.out0;
          col = n0 + (c & 3) * 32;
        }
        if (write && m < p.M_total && col < p.N_total)
          store_bf16x32(base + e * p.expert_stride + static_cast<int64_t>(m) * p.ld_out + col, v);
      } else {
        const int col = n0 + c * 32;
        const bool in_rows = (KIND != GEMM_DX) || row < p.T;  // token tiles may overhang T
        if (write && in_rows && col < p.N_total) store_bf16x32(p.out0 + row * p.ld_out + col, v);
      }
    }
  }
}

// Weight gradient of an expert without tokens: the thread's row of the output tile is zero.
template <int KIND>
__device__ __forceinline__ void wgrad_zero_fill(const GemmParams& p, int e, int m, int n0) {
  if (m >= p.M_total) return;
  float z[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) z[i] = 0.f;
  for (int c = 0; c < 8; ++c) {
    uint16_t* base = p.out0;
    int col = n0 + c * 32;
    if (KIND == GEMM_B5) {
      base = (c >= 4) ? p.out1 : p.out0;
      col = n0 + (c & 3) * 32;
    }
    if (col < p.N_total) store_bf16x32(base + e * p.expert_stride + static_cast<int64_t>(m) * p.ld_out + col, z);
  }
}

}  // namespace moe
