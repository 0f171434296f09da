// Steps 4+5 of the MoE layer (paper Section II-A, combine and scaling): every token gathers the
// K rows its experts produced (their positions were recorded at dispatch time, the "source
// information" of Section IV-B) and forms y[t,:] = sum_k w[t,k] * rows[slot_of[t,k],:].
//
// HBM-bound gather-reduce.  A warp owns a run of 64 consecutive 16-byte column chunks of one token
// (so a token is spread over several warps and small batches still fill the GPU); lanes 0..K-1 fetch
// the token's slots and weights once and broadcast them by shuffle; for every chunk the K row loads
// are issued together, the sum runs in fp32 in ascending k (so the result is deterministic), and is
// rounded once to the storage type.
#include <climits>

#include "common.cuh"

namespace moehub {

constexpr int kCombThreads = 256;
constexpr int kCombRun = 64;  // 16-byte chunks per warp: two per lane

template <typename XT, int KT>  // KT > 0: K known at compile time; KT == 0: runtime K (<= 32)
__global__ void __launch_bounds__(kCombThreads)
combine_kernel(const uint4* __restrict__ rows, const int* __restrict__ slot_of,
               const float* __restrict__ topk_w, int T, int K_rt, int vec_per_row, int runs_per_row,
               uint4* __restrict__ y, int staged, int row_limit) {
  constexpr int N = Vec16<XT>::N;
  constexpr int KMAX = KT > 0 ? KT : 1;
  const int K = KT > 0 ? KT : K_rt;
  const int lane = threadIdx.x % 32;
  const long long wid = (long long)blockIdx.x * (kCombThreads / 32) + threadIdx.x / 32;
  const int t = (int)(wid / runs_per_row);
  if (t >= T) return;
  const int v_begin = (int)(wid % runs_per_row) * kCombRun;
  pdl_wait();
  pdl_trigger();
  int my_slot = -1;
  float my_w = 0.0f;
  if (lane < K) {
    my_slot = slot_of[(size_t)t * K + lane];
    my_w = topk_w[(size_t)t * K + lane];
    // A slot beyond the rows there are is no slot (what a dispatch that gave up half-way leaves in the entries it
    // never wrote): it adds nothing, like a dropped assignment, and nothing outside the buffer is read.
    if (!staged && my_slot >= row_limit) my_slot = -1;
    // push-style combine: the experts stored assignment (t, k) at row t*K+k themselves; slot_of only says whether it exists
    if (staged && my_slot >= 0) my_slot = t * K + lane;
  }
  uint4* dst = y + (size_t)t * vec_per_row;
  const int v0 = v_begin + lane, v1 = v_begin + 32 + lane;
  const bool ok0 = v0 < vec_per_row, ok1 = v1 < vec_per_row;
  if (KT > 0) {
    uint4 r0[KMAX], r1[KMAX];
    float w[KMAX];
#pragma unroll
    for (int k = 0; k < KT; ++k) {
      const int s = __shfl_sync(0xffffffffu, my_slot, k);
      w[k] = __shfl_sync(0xffffffffu, my_w, k);
      const uint4* src = rows + (size_t)(s >= 0 ? s : 0) * vec_per_row;
      r0[k] = (s >= 0 && ok0) ? __ldcs(src + v0) : make_uint4(0, 0, 0, 0);
      r1[k] = (s >= 0 && ok1) ? __ldcs(src + v1) : make_uint4(0, 0, 0, 0);
    }
    float a0[N], a1[N];
#pragma unroll
    for (int q = 0; q < N; ++q) a0[q] = a1[q] = 0.0f;
#pragma unroll
    for (int k = 0; k < KT; ++k) {
      float f[N];
      Vec16<XT>::unpack(r0[k], f);
#pragma unroll
      for (int q = 0; q < N; ++q) a0[q] = __fmaf_rn(w[k], f[q], a0[q]);
      Vec16<XT>::unpack(r1[k], f);
#pragma unroll
      for (int q = 0; q < N; ++q) a1[q] = __fmaf_rn(w[k], f[q], a1[q]);
    }
    if (ok0) dst[v0] = Vec16<XT>::pack(a0);
    if (ok1) dst[v1] = Vec16<XT>::pack(a1);
  } else {
    float a0[N], a1[N];
#pragma unroll
    for (int q = 0; q < N; ++q) a0[q] = a1[q] = 0.0f;
    for (int k = 0; k < K; ++k) {  // warp-uniform trip count: the shuffles need all lanes
      const int s = __shfl_sync(0xffffffffu, my_slot, k);
      const float wk = __shfl_sync(0xffffffffu, my_w, k);
      if (s < 0) continue;
      const uint4* src = rows + (size_t)s * vec_per_row;
      float f[N];
      if (ok0) {
        Vec16<XT>::unpack(__ldcs(src + v0), f);
#pragma unroll
        for (int q = 0; q < N; ++q) a0[q] = __fmaf_rn(wk, f[q], a0[q]);
      }
      if (ok1) {
        Vec16<XT>::unpack(__ldcs(src + v1), f);
#pragma unroll
        for (int q = 0; q < N; ++q) a1[q] = __fmaf_rn(wk, f[q], a1[q]);
      }
    }
    if (ok0) dst[v0] = Vec16<XT>::pack(a0);
    if (ok1) dst[v1] = Vec16<XT>::pack(a1);
  }
}

template <typename XT>
static int launch_typed(moe_plan* p, const void* rows, const int* slot_of, const float* topk_w, void* y,
                        cudaStream_t st, bool staged) {
  const moe_config_t& c = p->cfg;
  const int vec_per_row = c.H * (int)sizeof(XT) / 16;
  const int runs_per_row = (vec_per_row + kCombRun - 1) / kCombRun;
  const long long warps = (long long)c.T * runs_per_row;
  const int grid = (int)((warps + kCombThreads / 32 - 1) / (kCombThreads / 32));
  const int row_limit = (int)min((long long)p->P * kTileRows, (long long)INT_MAX);
#define MOEHUB_COMBINE(KT)                                                                          \
  launch_pdl(combine_kernel<XT, KT>, dim3(grid), dim3(kCombThreads), 0, st, (const uint4*)rows, slot_of, topk_w, \
             c.T, c.K, vec_per_row, runs_per_row, (uint4*)y, staged ? 1 : 0, row_limit)
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
                   cudaStream_t st, bool staged) {
  if (p->cfg.T == 0) return 0;
  if (p->cfg.dtype == MOE_DTYPE_BF16) return launch_typed<__nv_bfloat16>(p, rows, slot_of, topk_w, y, st, staged);
  return launch_typed<float>(p, rows, slot_of, topk_w, y, st, staged);
}

}  // namespace moehub
