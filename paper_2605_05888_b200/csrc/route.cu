// Step 1 of the MoE layer (paper Section II-A, routing): gate logits, softmax, top-K.
//
// Each CTA owns a block of TB tokens and all E experts.  The logit of (token, expert) is ONE
// ascending fp32 FMA chain over h (no split of the h range, no tensor cores), because the
// logit decides which experts are picked and the pick has to be reproducible bit for bit.
// The parallelism is across the T*E independent chains: x and Wr chunks are staged in shared
// memory (16-byte global loads, next chunk prefetched into registers), every thread carries a
// TM x TE register tile of chains.  Afterwards the logits go through shared memory to one warp
// per token, which keeps them in registers (E/32 per lane) and runs K rounds of a shuffle
// arg-max (ties: lowest expert index), then the softmax weights.
#include <float.h>

#include "common.cuh"

namespace moehub {

constexpr int kRouteThreads = 256;
constexpr int kHC = 32;  // h elements per staged chunk

template <typename XT, int ROWS>
struct ChunkRegs {  // the 16-byte vectors one thread holds of a [ROWS][kHC] chunk
  static constexpr int N = Vec16<XT>::N;
  static constexpr int PARTS = kHC / N;
  static constexpr int NVEC = ROWS * PARTS;
  static constexpr int PER_THREAD = (NVEC + kRouteThreads - 1) / kRouteThreads;
  uint4 v[PER_THREAD];

  __device__ __forceinline__ void load(const XT* base, int row0, int nrows_valid, int H, int h0) {
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = threadIdx.x + i * kRouteThreads;
      const int r = idx / PARTS, part = idx % PARTS;
      const int h = h0 + part * N;
      v[i] = make_uint4(0, 0, 0, 0);
      if (idx < NVEC && r < nrows_valid && h < H)
        v[i] = __ldg(reinterpret_cast<const uint4*>(base + (size_t)(row0 + r) * H + h));
    }
  }
  // smem layout [kHC][ROWS + 1] (transposed; the odd width keeps the transposing stores conflict-free)
  __device__ __forceinline__ void store(float* s) const {
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = threadIdx.x + i * kRouteThreads;
      if (idx < NVEC) {
        const int r = idx / PARTS, part = idx % PARTS;
        float f[N];
        Vec16<XT>::unpack(v[i], f);
#pragma unroll
        for (int q = 0; q < N; ++q) s[(part * N + q) * (ROWS + 1) + r] = f[q];
      }
    }
  }
};

template <typename XT, int TX, int TE, int TY, int TM>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(const XT* __restrict__ x, const XT* __restrict__ wr, const float* __restrict__ bias,
             int T, int H, int E, int K, int renorm, int* __restrict__ topk_idx,
             float* __restrict__ topk_w) {
  static_assert(TX * TY == kRouteThreads, "thread layout");
  constexpr int TB = TY * TM, EP = TX * TE;
  constexpr int XW = TB + 1, WW = EP + 1;
  extern __shared__ float smem[];
  float* xs = smem;             // [kHC][XW]
  float* ws = smem + kHC * XW;  // [kHC][WW]
  float* ls = smem;             // [TB][EP], reuses the staging area after the h loop

  const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
  const int t0 = blockIdx.x * TB;
  const int tvalid = min(TB, T - t0);

  float acc[TM][TE];
#pragma unroll
  for (int j = 0; j < TM; ++j)
#pragma unroll
    for (int i = 0; i < TE; ++i) acc[j][i] = 0.0f;

  ChunkRegs<XT, TB> xr;
  ChunkRegs<XT, EP> wrg;
  xr.load(x, t0, tvalid, H, 0);
  wrg.load(wr, 0, E, H, 0);

  for (int h0 = 0; h0 < H; h0 += kHC) {
    __syncthreads();  // previous chunk fully consumed
    xr.store(xs);
    wrg.store(ws);
    __syncthreads();
    if (h0 + kHC < H) {  // prefetch the next chunk while this one is computed
      xr.load(x, t0, tvalid, H, h0 + kHC);
      wrg.load(wr, 0, E, H, h0 + kHC);
    }
    const int hmax = min(kHC, H - h0);
#pragma unroll 4
    for (int hh = 0; hh < hmax; ++hh) {
      float xv[TM], wv[TE];
#pragma unroll
      for (int j = 0; j < TM; ++j) xv[j] = xs[hh * XW + ty + TY * j];
#pragma unroll
      for (int i = 0; i < TE; ++i) wv[i] = ws[hh * WW + tx + TX * i];
#pragma unroll
      for (int j = 0; j < TM; ++j)
#pragma unroll
        for (int i = 0; i < TE; ++i) acc[j][i] = __fmaf_rn(xv[j], wv[i], acc[j][i]);
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < TM; ++j)
#pragma unroll
    for (int i = 0; i < TE; ++i) {
      const int e = tx + TX * i;
      float l = acc[j][i];
      if (bias != nullptr && e < E) l = l + bias[e];
      ls[(ty + TY * j) * EP + e] = l;
    }
  __syncthreads();

  // ---- one warp per token: top-K by K rounds of arg-max, then softmax weights ----
  constexpr int NJ = (EP + 31) / 32;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  for (int tl = warp; tl < tvalid; tl += kRouteThreads / 32) {
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
      topk_idx[(size_t)(t0 + tl) * K + lane] = my_e;
      topk_w[(size_t)(t0 + tl) * K + lane] = p;
    }
  }
}

template <typename XT, int TX, int TE, int TY, int TM>
static int launch_cfg(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                      float* topk_w, cudaStream_t st) {
  constexpr int TB = TY * TM, EP = TX * TE;
  const size_t stage = sizeof(float) * kHC * (TB + 1 + EP + 1);
  const size_t logits = sizeof(float) * TB * EP;
  const size_t smem = stage > logits ? stage : logits;
  auto kern = route_kernel<XT, TX, TE, TY, TM>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
  }
  const moe_config_t& c = p->cfg;
  const int grid = (c.T + TB - 1) / TB;
  kern<<<grid, kRouteThreads, smem, st>>>((const XT*)x, (const XT*)wr, bias, c.T, c.H, c.E, c.K,
                                          c.renormalize, topk_idx, topk_w);
  p->launches += 1;
  return (int)cudaGetLastError();
}

template <typename XT>
static int launch_typed(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                        float* topk_w, cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  if (c.E <= 8) return launch_cfg<XT, 8, 1, 32, 1>(p, x, wr, bias, topk_idx, topk_w, st);
  if (c.E <= 64) return launch_cfg<XT, 16, 4, 16, 1>(p, x, wr, bias, topk_idx, topk_w, st);
  if (c.T >= 2048) return launch_cfg<XT, 32, 8, 8, 8>(p, x, wr, bias, topk_idx, topk_w, st);
  return launch_cfg<XT, 32, 8, 8, 2>(p, x, wr, bias, topk_idx, topk_w, st);
}

int launch_route(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                 float* topk_w, cudaStream_t st) {
  if (p->cfg.T == 0) return 0;
  if (p->cfg.dtype == MOE_DTYPE_BF16)
    return launch_typed<__nv_bfloat16>(p, x, wr, bias, topk_idx, topk_w, st);
  return launch_typed<float>(p, x, wr, bias, topk_idx, topk_w, st);
}

}  // namespace moehub
