// Scheduling tables of the expert GEMMs, built on the device from the per-expert row counts: canonical and padded
// segment offsets, the expert of every 128-row tile, the pairs of row blocks for the CTA-pair kernels and the
// experts ordered by load.  Shared by the permutation's scan kernel (all experts local) and the expert-parallel
// plan kernel (the experts this rank owns).
#pragma once
#include "common.cuh"

namespace moe {

struct TableScratch {
  int pad[MAX_E + 1];     // padded segment starts
  int pair[MAX_E + 1];    // pairs of row blocks before expert e, an odd last block counted as a pair
  int fpair[MAX_E + 1];   // complete pairs before expert e
  int single[MAX_E + 1];  // experts with an odd number of blocks before expert e
};

struct TableOut {
  int32_t *counts, *offsets, *pad_offsets, *sched, *tile_expert, *pair_tab, *fpair_tab, *single_tab, *expert_order;
};

inline TableOut table_pointers(const WsLayout& L, char* ws) {
  auto I = [&](size_t off) { return reinterpret_cast<int32_t*>(ws + off); };
  return TableOut{I(L.counts),   I(L.offsets),   I(L.pad_offsets), I(L.sched),       I(L.tile_expert),
                  I(L.pair_tab), I(L.fpair_tab), I(L.single_tab),  I(L.expert_order)};
}

// Called by every thread of a block (at least 32 threads) after s_cnt[0..E) is complete and the block has synchronised.
__device__ inline void build_expert_tables(int E, const int* s_cnt, TableScratch& sh, const TableOut& o) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  for (int e = tid; e < E; e += nthr) {
    const int run = s_cnt[e];
    o.counts[e] = run;
    // position of e in the order "most rows first" (ties by index): the weight-gradient kernels start with the
    // experts whose K loops are longest so that a skewed load does not leave a long tail
    int rank = 0;
    for (int q = 0; q < E; ++q) rank += (s_cnt[q] > run || (s_cnt[q] == run && q < e)) ? 1 : 0;
    o.expert_order[rank] = e;
  }
  if (tid < 32) {
    // exclusive scans of counts, padded counts and block pairs over the experts: lane L owns experts 8L .. 8L+7
    const int lane = tid;
    int cn[8], pd[8], pr[8], fp[8], sg[8];
    int scn = 0, spd = 0, spr = 0, sfp = 0, ssg = 0;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = lane * 8 + u;
      const int cnt = e < E ? s_cnt[e] : 0;
      const int blocks = (cnt + ROW_PAD - 1) / ROW_PAD;
      cn[u] = scn;
      pd[u] = spd;
      pr[u] = spr;
      fp[u] = sfp;
      sg[u] = ssg;
      scn += cnt;
      spd += blocks * ROW_PAD;
      spr += (blocks + 1) / 2;
      sfp += blocks / 2;
      ssg += blocks & 1;
    }
    int icn = scn, ipd = spd, ipr = spr, ifp = sfp, isg = ssg;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int a = __shfl_up_sync(0xFFFFFFFFu, icn, off), b = __shfl_up_sync(0xFFFFFFFFu, ipd, off),
                c = __shfl_up_sync(0xFFFFFFFFu, ipr, off), d2 = __shfl_up_sync(0xFFFFFFFFu, ifp, off),
                e2 = __shfl_up_sync(0xFFFFFFFFu, isg, off);
      if (lane >= off) {
        icn += a;
        ipd += b;
        ipr += c;
        ifp += d2;
        isg += e2;
      }
    }
    const int bcn = icn - scn, bpd = ipd - spd, bpr = ipr - spr, bfp = ifp - sfp, bsg = isg - ssg;  // exclusive bases
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = lane * 8 + u;
      if (e < E) {
        o.offsets[e] = bcn + cn[u];
        o.pad_offsets[e] = bpd + pd[u];
        sh.pad[e] = bpd + pd[u];
        sh.pair[e] = bpr + pr[u];
        sh.fpair[e] = bfp + fp[u];
        sh.single[e] = bsg + sg[u];
      }
    }
    if (lane == 31) {
      o.offsets[E] = icn;
      o.pad_offsets[E] = ipd;
      sh.pad[E] = ipd;
      sh.pair[E] = ipr;
      sh.fpair[E] = ifp;
      sh.single[E] = isg;
      o.sched[0] = ipd / ROW_PAD;  // 128-row tiles
      o.sched[1] = ipd;            // padded rows
      o.sched[2] = ipr;            // pairs, odd last blocks included
      o.sched[3] = ifp;            // complete pairs
      o.sched[4] = isg;            // leftover single blocks
    }
  }
  __syncthreads();
  for (int e = tid; e < E; e += nthr) {
    for (int m = sh.pad[e] / ROW_PAD; m < sh.pad[e + 1] / ROW_PAD; ++m) o.tile_expert[m] = e;
    // pairs of consecutive 128-row blocks of this expert; the last pair of an odd count has one block
    const int blocks = (sh.pad[e + 1] - sh.pad[e]) / ROW_PAD;
    for (int q = 0; q < sh.pair[e + 1] - sh.pair[e]; ++q)
      *reinterpret_cast<int4*>(o.pair_tab + 4 * (sh.pair[e] + q)) =
          make_int4(e, sh.pad[e] + 2 * q * ROW_PAD, min(2, blocks - 2 * q), 0);
    // the same without half-empty pairs: complete pairs, and the leftover last block of an odd count on its own
    for (int q = 0; q < blocks / 2; ++q)
      *reinterpret_cast<int4*>(o.fpair_tab + 4 * (sh.fpair[e] + q)) = make_int4(e, sh.pad[e] + 2 * q * ROW_PAD, 2, 0);
    if (blocks & 1) o.single_tab[sh.single[e]] = sh.pad[e] / ROW_PAD + blocks - 1;
  }
}

}  // namespace moe
