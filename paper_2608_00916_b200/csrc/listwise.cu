// Listwise training losses on grouped reranker scores (paper, paragraph "Contrastive and distillation losses"):
// scores s [n, G], one row per query.
//   contrastive:  L = (1/n) sum_g ( logsumexp(s_g) - s_g[0] )                 (the positive sits at position 0)
//   distillation: L = (tau_s^2 / n) sum_g KL( softmax(t_g / tau_t) || softmax(s_g / tau_s) )   (stored teacher scores t)
// and dL/ds in the same pass.  The operation is tiny (64 queries x 8 passages per step in the paper's runs), so it is
// one block: a warp per row, lanes striding over the row's G scores, every warp summing the losses of its rows in row
// order and thread 0 adding the 32 warp sums in warp order - the same bits on every run, no scratch memory.
#include "common.cuh"

namespace moe {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

// log-sum-exp of a[0..G) * inv_temp over the lanes of a warp (row maximum subtracted first)
__device__ __forceinline__ float row_lse(const float* __restrict__ a, int G, float inv_temp, int lane) {
  float m = -INFINITY;
  for (int i = lane; i < G; i += 32) m = fmaxf(m, a[i] * inv_temp);
  m = warp_max(m);
  float z = 0.f;
  for (int i = lane; i < G; i += 32) z += expf(a[i] * inv_temp - m);
  return m + logf(warp_sum(z));
}

constexpr int LW_THREADS = 1024;

__global__ void __launch_bounds__(LW_THREADS) listwise_loss_kernel(int kind, int64_t n, int G,
                                                                   const float* __restrict__ scores,
                                                                   const float* __restrict__ teacher, float s_temp,
                                                                   float t_temp, float* __restrict__ loss,
                                                                   float* __restrict__ dscores) {
  __shared__ float s_part[LW_THREADS / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float inv_n = n > 0 ? 1.f / static_cast<float>(n) : 0.f;
  const float inv_s = kind == 1 ? 1.f / s_temp : 1.f, inv_t = kind == 1 ? 1.f / t_temp : 1.f;
  float acc = 0.f;  // identical in all lanes of the warp
  for (int64_t g = warp; g < n; g += LW_THREADS / 32) {
    const float* s = scores + g * G;
    const float lse = row_lse(s, G, inv_s, lane);
    float row = 0.f;
    if (kind == 0) {
      row = lse - s[0];
      if (dscores)
        for (int i = lane; i < G; i += 32) dscores[g * G + i] = (expf(s[i] - lse) - (i == 0 ? 1.f : 0.f)) * inv_n;
    } else {
      const float* t = teacher + g * G;
      const float lse_t = row_lse(t, G, inv_t, lane);
      for (int i = lane; i < G; i += 32) {
        const float lp = t[i] * inv_t - lse_t, lq = s[i] * inv_s - lse;
        const float p = expf(lp);
        if (p > 0.f) row += p * (lp - lq);
        if (dscores) dscores[g * G + i] = (expf(lq) - p) * (s_temp * inv_n);
      }
      row = warp_sum(row);
    }
    acc += row;
  }
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float total = 0.f;
    for (int w = 0; w < LW_THREADS / 32; ++w) total += s_part[w];
    loss[0] = total * inv_n * (kind == 1 ? s_temp * s_temp : 1.f);
  }
}

}  // namespace moe

using namespace moe;

extern "C" moe_status moe_listwise_loss(int32_t kind, int64_t n, int32_t G, const float* scores, const float* teacher,
                                        float s_temp, float t_temp, float* loss, float* dscores, void* cuda_stream) {
  if ((kind != MOE_LISTWISE_CONTRASTIVE && kind != MOE_LISTWISE_DISTILL) || n < 0 || G < 1 || !loss) return MOE_ERR_INVALID_ARG;
  if (n > 0 && !scores) return MOE_ERR_INVALID_ARG;
  if (kind == MOE_LISTWISE_DISTILL && ((n > 0 && !teacher) || !(s_temp > 0.f) || !(t_temp > 0.f))) return MOE_ERR_INVALID_ARG;
  listwise_loss_kernel<<<1, LW_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(kind, n, G, scores, teacher, s_temp,
                                                                                    t_temp, loss, dscores);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
