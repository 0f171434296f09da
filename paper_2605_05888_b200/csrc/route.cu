// Step 1 of the MoE layer (paper Section II-A, routing): gate logits, softmax, top-K.
//
// Each CTA owns a block of tokens and all E experts.  The logit of (token, expert) is ONE
// ascending fp32 FMA chain over h (no split of the h range, no tensor cores), because the
// logit decides which experts are picked and the pick has to be reproducible bit for bit.
// The parallelism is across the T*E independent chains: x and Wr chunks are staged in shared
// memory as fp32 (16-byte global loads, next chunk prefetched into registers).  Two shapes:
// E <= 64 is bound by the latency of the chain itself - one lane per chain; 64 < E <= 256 is
// bound by fp32 FMA issue - an 8 x 8 register tile of chains per thread.  Afterwards the logits
// go through shared memory to one warp per token, which keeps them in registers (E/32 per lane)
// and runs K rounds of a shuffle arg-max (ties: lowest expert index), then the softmax weights.
#include <float.h>

#include "common.cuh"

namespace moehub {

constexpr int kRouteThreads = 256;

// One warp per token: the token's logits sit in registers (EP/32 per lane); K rounds of a shuffle
// arg-max on (value, lowest index); then the softmax weights of the picks.  ls: [tokens][EP] logits
// in shared memory.
template <int EP>
__device__ __forceinline__ void select_topk(const float* ls, int tvalid, int t0, int E, int K, int renorm,
                                            int* __restrict__ topk_idx, float* __restrict__ topk_w) {
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
      topk_idx[(size_t)(t0 + tl) * K + lane] = my_e;
      topk_w[(size_t)(t0 + tl) * K + lane] = p;
    }
  }
}

// The compute-bound shape (64 < E <= 256): 64 tokens x 256 experts per CTA, 8 x 8 chains per thread,
// every shared-memory read of the inner loop a 16-byte vector: 4 loads feed 64 FMAs.  The staging
// stores are conflict-free because consecutive lanes handle consecutive rows of one 16-byte column
// group.
constexpr int kWideTB = 64, kWideEP = 256, kWideHC = 32;

template <typename XT, int ROWS>
struct WideChunk {
  static constexpr int N = Vec16<XT>::N;
  static constexpr int PARTS = kWideHC / N;
  static constexpr int PER_THREAD = ROWS * PARTS / kRouteThreads;
  uint4 v[PER_THREAD];
  __device__ __forceinline__ void load(const XT* base, int row0, int nrows_valid, int H, int h0) {
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = threadIdx.x + i * kRouteThreads;
      const int r = idx % ROWS, part = idx / ROWS;
      const int h = h0 + part * N;
      v[i] = make_uint4(0, 0, 0, 0);
      if (r < nrows_valid && h < H) v[i] = __ldg(reinterpret_cast<const uint4*>(base + (size_t)(row0 + r) * H + h));
    }
  }
  __device__ __forceinline__ void store(float* s) const {  // s: [kWideHC][ROWS]
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = threadIdx.x + i * kRouteThreads;
      const int r = idx % ROWS, part = idx / ROWS;
      float f[N];
      Vec16<XT>::unpack(v[i], f);
#pragma unroll
      for (int q = 0; q < N; ++q) s[(part * N + q) * ROWS + r] = f[q];
    }
  }
};

template <typename XT>
__global__ void __launch_bounds__(kRouteThreads)
route_wide_kernel(const XT* __restrict__ x, const XT* __restrict__ wr, const float* __restrict__ bias, int T,
                  int H, int E, int K, int renorm, int* __restrict__ topk_idx, float* __restrict__ topk_w) {
  extern __shared__ __align__(16) float smem[];
  float* xs = smem;                      // [32][64]
  float* ws = smem + kWideHC * kWideTB;  // [32][256]
  float* ls = smem;                      // [64][256] after the h loop
  // A warp is an 8 (token groups) x 4 (expert groups) grid of lanes and owns 32 experts for all 64
  // tokens: per h it reads 256 B of x and 128 B of Wr from shared memory for 2048 FMAs.
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int ly = lane / 4, lx = lane % 4;
  const int ebase = 32 * warp + 4 * lx;  // experts ebase..ebase+3 and ebase+16..ebase+19
  const int t0 = blockIdx.x * kWideTB;
  const int tvalid = min(kWideTB, T - t0);

  float acc[8][8];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[j][i] = 0.0f;

  WideChunk<XT, kWideTB> xr;
  WideChunk<XT, kWideEP> wrg;
  pdl_wait();
  pdl_trigger();
  xr.load(x, t0, tvalid, H, 0);
  wrg.load(wr, 0, E, H, 0);
  for (int h0 = 0; h0 < H; h0 += kWideHC) {
    __syncthreads();
    xr.store(xs);
    wrg.store(ws);
    __syncthreads();
    if (h0 + kWideHC < H) {
      xr.load(x, t0, tvalid, H, h0 + kWideHC);
      wrg.load(wr, 0, E, H, h0 + kWideHC);
    }
    const int hmax = min(kWideHC, H - h0);
    // software pipeline: the operands of step hh+1 are loaded while step hh is computed
    float4 xa = *reinterpret_cast<const float4*>(xs + 4 * ly);
    float4 xb = *reinterpret_cast<const float4*>(xs + 32 + 4 * ly);
    float4 wa = *reinterpret_cast<const float4*>(ws + ebase);
    float4 wb = *reinterpret_cast<const float4*>(ws + ebase + 16);
#pragma unroll 2
    for (int hh = 0; hh < hmax; ++hh) {
      const int hn = min(hh + 1, kWideHC - 1);
      const float4 nxa = *reinterpret_cast<const float4*>(xs + hn * kWideTB + 4 * ly);
      const float4 nxb = *reinterpret_cast<const float4*>(xs + hn * kWideTB + 32 + 4 * ly);
      const float4 nwa = *reinterpret_cast<const float4*>(ws + hn * kWideEP + ebase);
      const float4 nwb = *reinterpret_cast<const float4*>(ws + hn * kWideEP + ebase + 16);
      const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
      const float wv[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[j][i] = __fmaf_rn(xv[j], wv[i], acc[j][i]);
      xa = nxa; xb = nxb; wa = nwa; wb = nwb;
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int tl = (j < 4) ? 4 * ly + j : 32 + 4 * ly + (j - 4);
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      const int e0 = ebase + 16 * g;
      float l[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        l[i] = acc[j][g * 4 + i];
        if (bias != nullptr && e0 + i < E) l[i] = l[i] + bias[e0 + i];
      }
      *reinterpret_cast<float4*>(ls + tl * kWideEP + e0) = make_float4(l[0], l[1], l[2], l[3]);
    }
  }
  __syncthreads();
  select_topk<kWideEP>(ls, tvalid, t0, E, K, renorm, topk_idx, topk_w);
}

template <typename XT>
static int launch_wide(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                       float* topk_w, cudaStream_t st) {
  const size_t smem = sizeof(float) * kWideTB * kWideEP;  // the logits tile; the staging area is smaller
  auto kern = route_wide_kernel<XT>;
  static bool attr_done = false;  // per instantiation and process, idempotent
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    attr_done = true;
  }
  const moe_config_t& c = p->cfg;
  p->launches += 1;
  return (int)launch_maybe_pdl(false, kern, dim3((c.T + kWideTB - 1) / kWideTB), dim3(kRouteThreads), smem, st, (const XT*)x,
                         (const XT*)wr, bias, c.T, c.H, c.E, c.K, c.renormalize, topk_idx, topk_w);
}

// The latency-bound shapes (E <= 64): one lane per chain (or two chains for 32 < E <= 64).  A token's
// experts sit on LE consecutive lanes; x and Wr tiles stay in their natural [row][h] layout in shared
// memory (fp32, converted while staging), so a lane reads four consecutive h of its token and of its
// expert with two 16-byte loads and runs its chain over them.  The time is close to the latency of
// the chain itself (4 cycles per h) once the chunk loads are overlapped.
template <typename XT, int ROWS, int HC, int THREADS>
struct NaturalChunk {
  static constexpr int N = Vec16<XT>::N;
  static constexpr int PARTS = HC / N;
  static constexpr int NVEC = ROWS * PARTS;
  static constexpr int PER_THREAD = (NVEC + THREADS - 1) / THREADS;
  static constexpr int PITCH = HC + 4;  // floats; rows land on different banks
  uint4 v[PER_THREAD];
  __device__ __forceinline__ void load(const XT* base, int row0, int nrows_valid, int H, int h0) {
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = threadIdx.x + i * THREADS;
      const int r = idx / PARTS, part = idx % PARTS;
      const int h = h0 + part * N;
      v[i] = make_uint4(0, 0, 0, 0);
      if (idx < NVEC && r < nrows_valid && h < H)
        v[i] = __ldg(reinterpret_cast<const uint4*>(base + (size_t)(row0 + r) * H + h));
    }
  }
  __device__ __forceinline__ void store(float* s) const {  // s: [ROWS][PITCH]
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = threadIdx.x + i * THREADS;
      if (idx < NVEC) {
        const int r = idx / PARTS, part = idx % PARTS;
        float f[N];
        Vec16<XT>::unpack(v[i], f);
        float4* dst = reinterpret_cast<float4*>(s + r * PITCH + part * N);
#pragma unroll
        for (int q = 0; q < N / 4; ++q) dst[q] = make_float4(f[4 * q], f[4 * q + 1], f[4 * q + 2], f[4 * q + 3]);
      }
    }
  }
};

template <typename XT, int LE, int TE, int HC, int THREADS>
__global__ void __launch_bounds__(THREADS)
route_narrow_kernel(const XT* __restrict__ x, const XT* __restrict__ wr, const float* __restrict__ bias, int T,
                    int H, int E, int K, int renorm, int* __restrict__ topk_idx, float* __restrict__ topk_w) {
  constexpr int EP = LE * TE;              // experts covered (padded)
  constexpr int TW = 32 / LE;              // tokens per warp
  constexpr int TB = TW * (THREADS / 32);
  constexpr int PITCH = HC + 4;
  extern __shared__ __align__(16) float smem[];
  float* xs = smem;               // [TB][PITCH]
  float* ws = smem + TB * PITCH;  // [EP][PITCH]
  float* ls = smem;               // [TB][EP] after the h loop
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int tl = warp * TW + lane / LE;  // this lane's token inside the block
  const int le = lane % LE;              // this lane's experts: le + LE*i
  const int t0 = blockIdx.x * TB;
  const int tvalid = min(TB, T - t0);

  float acc[TE];
#pragma unroll
  for (int i = 0; i < TE; ++i) acc[i] = 0.0f;
  NaturalChunk<XT, TB, HC, THREADS> xr;
  NaturalChunk<XT, EP, HC, THREADS> wrg;
  pdl_wait();
  pdl_trigger();
  xr.load(x, t0, tvalid, H, 0);
  wrg.load(wr, 0, E, H, 0);
  for (int h0 = 0; h0 < H; h0 += HC) {
    __syncthreads();
    xr.store(xs);
    wrg.store(ws);
    __syncthreads();
    if (h0 + HC < H) {
      xr.load(x, t0, tvalid, H, h0 + HC);
      wrg.load(wr, 0, E, H, h0 + HC);
    }
    const int hmax = min(HC, H - h0);
    // Groups of 16 h: the next group's operands are loaded while this group's 16-step chain runs, so
    // the shared-memory latency hides behind the chain.  The tail of a short last chunk is zero in
    // shared memory (loads past H are zero-filled) and fma(0, 0, acc) leaves acc's value alone.
    const float* xrow = xs + tl * PITCH;
    const float* wrow = ws + le * PITCH;
    constexpr int G = 4;
    float4 xv[G], wv[TE][G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      xv[g] = *reinterpret_cast<const float4*>(xrow + 4 * g);
#pragma unroll
      for (int i = 0; i < TE; ++i) wv[i][g] = *reinterpret_cast<const float4*>(wrow + LE * i * PITCH + 4 * g);
    }
    for (int hh = 0; hh < hmax; hh += 4 * G) {
      const int hn = min(hh + 4 * G, HC - 4 * G);
      float4 nxv[G], nwv[TE][G];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        nxv[g] = *reinterpret_cast<const float4*>(xrow + hn + 4 * g);
#pragma unroll
        for (int i = 0; i < TE; ++i) nwv[i][g] = *reinterpret_cast<const float4*>(wrow + LE * i * PITCH + hn + 4 * g);
      }
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int i = 0; i < TE; ++i) {
          acc[i] = __fmaf_rn(xv[g].x, wv[i][g].x, acc[i]);
          acc[i] = __fmaf_rn(xv[g].y, wv[i][g].y, acc[i]);
          acc[i] = __fmaf_rn(xv[g].z, wv[i][g].z, acc[i]);
          acc[i] = __fmaf_rn(xv[g].w, wv[i][g].w, acc[i]);
        }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        xv[g] = nxv[g];
#pragma unroll
        for (int i = 0; i < TE; ++i) wv[i][g] = nwv[i][g];
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < TE; ++i) {
    const int e = le + LE * i;
    float l = acc[i];
    if (bias != nullptr && e < E) l = l + bias[e];
    ls[tl * EP + e] = l;
  }
  __syncthreads();
  select_topk<EP>(ls, tvalid, t0, E, K, renorm, topk_idx, topk_w);
}

template <typename XT, int LE, int TE, int HC, int THREADS>
static int launch_narrow(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                         float* topk_w, cudaStream_t st) {
  constexpr int EP = LE * TE, TB = (32 / LE) * (THREADS / 32);
  const size_t smem = sizeof(float) * (TB + EP) * (HC + 4);
  auto kern = route_narrow_kernel<XT, LE, TE, HC, THREADS>;
  static bool attr_done = false;  // per instantiation and process, idempotent
  if (smem > 48 * 1024 && !attr_done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    attr_done = true;
  }
  const moe_config_t& c = p->cfg;
  p->launches += 1;
  return (int)launch_maybe_pdl(false, kern, dim3((c.T + TB - 1) / TB), dim3(THREADS), smem, st, (const XT*)x,
                         (const XT*)wr, bias, c.T, c.H, c.E, c.K, c.renormalize, topk_idx, topk_w);
}

template <typename XT>
static int launch_typed(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                        float* topk_w, cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  // Small E is bound by the latency of the chain: one lane per chain, long chunks; small batches use
  // 128-thread CTAs so that the blocks spread over more SMs.
  const bool small = c.T <= 2048;
  if (c.E <= 8)
    return small ? launch_narrow<XT, 8, 1, 512, 128>(p, x, wr, bias, topk_idx, topk_w, st)
                 : launch_narrow<XT, 8, 1, 512, 256>(p, x, wr, bias, topk_idx, topk_w, st);
  if (c.E <= 16)
    return small ? launch_narrow<XT, 16, 1, 512, 128>(p, x, wr, bias, topk_idx, topk_w, st)
                 : launch_narrow<XT, 16, 1, 512, 256>(p, x, wr, bias, topk_idx, topk_w, st);
  if (c.E <= 32)
    return small ? launch_narrow<XT, 32, 1, 512, 128>(p, x, wr, bias, topk_idx, topk_w, st)
                 : launch_narrow<XT, 32, 1, 512, 256>(p, x, wr, bias, topk_idx, topk_w, st);
  if (c.E <= 64)
    return small ? launch_narrow<XT, 32, 2, 256, 128>(p, x, wr, bias, topk_idx, topk_w, st)
                 : launch_narrow<XT, 32, 2, 256, 256>(p, x, wr, bias, topk_idx, topk_w, st);
  return launch_wide<XT>(p, x, wr, bias, topk_idx, topk_w, st);
}

int launch_route(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                 float* topk_w, cudaStream_t st) {
  if (p->cfg.T == 0) return 0;
  if (p->cfg.dtype == MOE_DTYPE_BF16)
    return launch_typed<__nv_bfloat16>(p, x, wr, bias, topk_idx, topk_w, st);
  return launch_typed<float>(p, x, wr, bias, topk_idx, topk_w, st);
}

}  // namespace moehub
