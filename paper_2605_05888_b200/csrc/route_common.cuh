// What every router kernel shares: the selection of the K largest logits of a token with its softmax weights,
// and the side job of resetting the dispatch's per-call state (see PrepArgs).
#pragma once
#include <float.h>

#include "common.cuh"

namespace moehub {

// One warp per token: the token's logits sit in registers (EP/32 per lane); K rounds of a shuffle
// arg-max on (value, lowest index); then the softmax weights of the picks.  ls: [tokens][EP] logits
// in shared memory.
// s_hist (shared memory, [E], or nullptr): every pick is also counted per expert.
template <int EP>
// tp > 1 (expert + tensor parallelism, paper Section VII): every pick is listed once per TP shard, as the
// virtual expert e*tp + s with the pick's weight, so that the dispatch stores the row into every shard's region.
__device__ __forceinline__ void select_topk(const float* ls, int tvalid, int t0, int E, int K, int renorm,
                                            int* __restrict__ topk_idx, float* __restrict__ topk_w, int* s_hist, int tp) {
  constexpr int NJ = (EP + 31) / 32;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  for (int tl = warp; tl < tvalid; tl += blockDim.x / 32) {
    float v[NJ];
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int e = lane + 32 * j;
      v[j] = (e < E) ? ls[tl * EP + e] : -FLT_MAX;
    }
    unsigned taken = 0;
    float my_v = 0.0f;
    int my_e = 0;
    for (int k = 0; k < K; ++k) {
      float bv = -FLT_MAX;
      int be = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int e = lane + 32 * j;
        const bool ok = (e < E) && !((taken >> j) & 1u);
        if (ok && (be == 0x7fffffff || v[j] > bv)) { bv = v[j]; be = e; }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oe = __shfl_xor_sync(0xffffffffu, be, off);
        const bool other = (oe != 0x7fffffff) && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be));
        if (other) { bv = ov; be = oe; }
      }
      if ((be & 31) == lane) taken |= 1u << (be >> 5);
      if (lane == k) { my_v = bv; my_e = be; }
    }
    const float m = __shfl_sync(0xffffffffu, my_v, 0);
    float z = 0.0f;
#pragma unroll
    for (int j = 0; j < NJ; ++j)
      if (lane + 32 * j < E) z += expf(v[j] - m);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
    float p = (lane < K) ? expf(my_v - m) / z : 0.0f;
    if (renorm) {
      float s = p;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
      p = p / s;
    }
    if (lane < K) {
      for (int sh = 0; sh < tp; ++sh) {
        const size_t o = ((size_t)(t0 + tl) * K + lane) * tp + sh;
        topk_idx[o] = my_e * tp + sh;
        topk_w[o] = p;
        if (s_hist != nullptr) atomicAdd(&s_hist[my_e * tp + sh], 1);
      }
    }
  }
}

// The side job of a router that is followed by an ordered dispatch (see PrepArgs): before the chains, clear
// the per-call counters; after the picks, add this CTA's rows per expert to the global counts.
constexpr int kRouteMaxExperts = 256;
__device__ __forceinline__ void route_prep_begin(const PrepArgs& prep, int* s_hist) {
  if (prep.nfill == 0) return;
  for (int e = threadIdx.x; e < kRouteMaxExperts; e += blockDim.x) s_hist[e] = 0;
  prep_reset(prep, blockIdx.x * blockDim.x + threadIdx.x, gridDim.x * blockDim.x);
}
__device__ __forceinline__ void route_prep_end(const PrepArgs& prep, const int* s_hist) {
  if (prep.hist == nullptr) return;
  __syncthreads();
  for (int e = threadIdx.x; e < prep.E; e += blockDim.x)
    if (s_hist[e] != 0) atomicAdd(&prep.hist[e], s_hist[e]);
}

}  // namespace moehub
