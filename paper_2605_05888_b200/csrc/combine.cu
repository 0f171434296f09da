// Steps 4+5 of the MoE layer (paper Section II-A, combine and scaling): every token gathers the
// K rows its experts produced (their positions were recorded at dispatch time, the "source
// information" of Section IV-B) and forms y[t,:] = sum_k w[t,k] * rows[slot_of[t,k],:].
//
// HBM-bound gather-reduce: one warp per token; for every 16-byte column chunk the K row loads
// are issued together, the sum runs in fp32 in ascending k (so the result is deterministic),
// and is rounded once to the storage type.
#include "common.cuh"

namespace moehub {

constexpr int kCombThreads = 256;

template <typename XT, int KT>  // KT > 0: K known at compile time; KT == 0: runtime K (<= 32)
__global__ void __launch_bounds__(kCombThreads)
combine_kernel(const uint4* __restrict__ rows, const int* __restrict__ slot_of,
               const float* __restrict__ topk_w, int T, int K_rt, int vec_per_row, uint4* __restrict__ y) {
  constexpr int N = Vec16<XT>::N;
  const int K = KT > 0 ? KT : K_rt;
  const int lane = threadIdx.x % 32;
  const int t = blockIdx.x * (kCombThreads / 32) + threadIdx.x / 32;
  if (t >= T) return;
  // lane k holds slot/weight k; broadcast by shuffle in the loop
  int my_slot = -1;
  float my_w = 0.0f;
  if (lane < K) {
    my_slot = slot_of[(size_t)t * K + lane];
    my_w = topk_w[(size_t)t * K + lane];
  }
  uint4* dst = y + (size_t)t * vec_per_row;
  if (KT > 0) {
    const uint4* src[KT > 0 ? KT : 1];
    float w[KT > 0 ? KT : 1];
#pragma unroll
    for (int k = 0; k < KT; ++k) {
      const int s = __shfl_sync(0xffffffffu, my_slot, k);
      w[k] = __shfl_sync(0xffffffffu, my_w, k);
      src[k] = s >= 0 ? rows + (size_t)s * vec_per_row : nullptr;
    }
    for (int v = lane; v < vec_per_row; v += 32) {
      uint4 r[KT > 0 ? KT : 1];
#pragma unroll
      for (int k = 0; k < KT; ++k) r[k] = src[k] ? __ldcs(src[k] + v) : make_uint4(0, 0, 0, 0);
      float acc[N];
#pragma unroll
      for (int q = 0; q < N; ++q) acc[q] = 0.0f;
#pragma unroll
      for (int k = 0; k < KT; ++k) {
        float f[N];
        Vec16<XT>::unpack(r[k], f);
#pragma unroll
        for (int q = 0; q < N; ++q) acc[q] = __fmaf_rn(w[k], f[q], acc[q]);
      }
      dst[v] = Vec16<XT>::pack(acc);
    }
  } else {
    for (int v0 = 0; v0 < vec_per_row; v0 += 32) {  // warp-uniform trip count: the shuffles need all lanes
      const int v = v0 + lane;
      float acc[N];
#pragma unroll
      for (int q = 0; q < N; ++q) acc[q] = 0.0f;
      for (int k = 0; k < K; ++k) {
        const int s = __shfl_sync(0xffffffffu, my_slot, k);
        const float wk = __shfl_sync(0xffffffffu, my_w, k);
        if (s < 0 || v >= vec_per_row) continue;
        float f[N];
        Vec16<XT>::unpack(__ldcs(rows + (size_t)s * vec_per_row + v), f);
#pragma unroll
        for (int q = 0; q < N; ++q) acc[q] = __fmaf_rn(wk, f[q], acc[q]);
      }
      if (v < vec_per_row) dst[v] = Vec16<XT>::pack(acc);
    }
  }
}

template <typename XT>
static int launch_typed(moe_plan* p, const void* rows, const int* slot_of, const float* topk_w, void* y,
                        cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  const int vec_per_row = c.H * (int)sizeof(XT) / 16;
  const int grid = (c.T + kCombThreads / 32 - 1) / (kCombThreads / 32);
#define MOEHUB_COMBINE(KT)                                                                          \
  combine_kernel<XT, KT><<<grid, kCombThreads, 0, st>>>((const uint4*)rows, slot_of, topk_w, c.T, c.K, \
                                                        vec_per_row, (uint4*)y)
  switch (c.K) {
    case 1: MOEHUB_COMBINE(1); break;
    case 2: MOEHUB_COMBINE(2); break;
    case 4: MOEHUB_COMBINE(4); break;
    case 8: MOEHUB_COMBINE(8); break;
    default: MOEHUB_COMBINE(0); break;
  }
#undef MOEHUB_COMBINE
  p->launches += 1;
  return (int)cudaGetLastError();
}

int launch_combine(moe_plan* p, const void* rows, const int* slot_of, const float* topk_w, void* y,
                   cudaStream_t st) {
  if (p->cfg.T == 0) return 0;
  if (p->cfg.dtype == MOE_DTYPE_BF16) return launch_typed<__nv_bfloat16>(p, rows, slot_of, topk_w, y, st);
  return launch_typed<float>(p, rows, slot_of, topk_w, y, st);
}

}  // namespace moehub
