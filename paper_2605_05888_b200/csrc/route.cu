// Step 1 of the MoE layer (paper Section II-A, routing): gate logits, softmax, top-K.
//
// Each CTA owns a block of tokens and all E experts.  The logit of (token, expert) is ONE
// ascending fp32 FMA chain over h (no split of the h range, no tensor cores), because the
// logit decides which experts are picked and the pick has to be reproducible bit for bit.
// The parallelism is across the T*E independent chains: x and Wr chunks are staged in shared
// memory as fp32 (16-byte global loads, next chunk prefetched into registers).  Two shapes:
// E <= 64 is bound by the shared-memory pipe - one token and two experts per lane; 64 < E <= 256 is
// bound by fp32 FMA issue - a register tile of up to 8 x 16 chains per thread.  In both, some warps only
// stage the operands and the others only compute.  Afterwards the logits
// go through shared memory to one warp per token, which keeps them in registers (E/32 per lane)
// and runs K rounds of a shuffle arg-max (ties: lowest expert index), then the softmax weights.
//
// With more than 64 experts on bf16 data the default is a different pair of kernels (route_filter.cu): tensor
// cores compute approximate logits, and the exact chain runs only for the experts that can still be among the
// K largest - the same picks, a fraction of the chains.  The kernels here remain the path for fp32 data, for
// up to 64 experts, and for route_filter = -1.
#include <float.h>

#include "route_common.cuh"

namespace moehub {


// The compute-bound shape (64 < E <= 256): up to 64 tokens x 256 experts per CTA.  Four compute warps
// hold a TMT x 16 register tile of chains per thread (a warp: 2 token groups by lane % 2, 16 expert
// groups by lane / 2, so that each of its six 16-byte shared-memory loads per h costs the 2-cycle
// minimum) and do nothing but FMAs; four staging warps convert the next chunk of x and Wr into the other
// shared-memory buffer (transposed to [h][token] and [h][expert], fp32) and keep the chunks after it in
// flight from global memory.  One __syncthreads per chunk of 32 h.  TMT (tokens per thread, 4..8) is
// picked at launch so that the CTAs fill the SMs evenly: T = 8192 runs 147 CTAs of 56 tokens.
constexpr int kWideEP = 256, kWideHC = 32, kWideSlots = 64;
constexpr int kWideComputeWarps = 4, kWideFillWarps = 4;
constexpr int kWideThreads = 32 * (kWideComputeWarps + kWideFillWarps);
constexpr int kWideBuf = kWideHC * (kWideSlots + kWideEP);  // floats per buffer

// ROWS rows of the tile (x: token slots, Wr: experts) times kWideHC h, 16 bytes per staging load.
template <typename XT, int ROWS>
struct WideChunk {
  static constexpr int FT = 32 * kWideFillWarps;
  static constexpr int N = Vec16<XT>::N;
  static constexpr int PARTS = kWideHC / N;
  static constexpr int PER_THREAD = ROWS * PARTS / FT;
  uint4 v[PER_THREAD];
  // row_of(r): global row of tile row r, or -1 for a padding row
  template <typename RowOf>
  __device__ __forceinline__ void load(int ft, const XT* base, RowOf row_of, int H, int h0) {
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = ft + i * FT;
      const int r = idx % ROWS, part = idx / ROWS;
      const int h = h0 + part * N;
      const int row = row_of(r);
      v[i] = make_uint4(0, 0, 0, 0);
      if (row >= 0 && h < H) v[i] = __ldg(reinterpret_cast<const uint4*>(base + (size_t)row * H + h));
    }
  }
  __device__ __forceinline__ void store(int ft, float* s) const {  // s: [kWideHC][ROWS]
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = ft + i * FT;
      const int r = idx % ROWS, part = idx / ROWS;
      float f[N];
      Vec16<XT>::unpack(v[i], f);
#pragma unroll
      for (int q = 0; q < N; ++q) s[(part * N + q) * ROWS + r] = f[q];
    }
  }
};

template <typename XT, int TMT>
__global__ void __launch_bounds__(kWideThreads)
route_wide_kernel(const XT* __restrict__ x, const XT* __restrict__ wr, const float* __restrict__ bias, int T,
                  int H, int E, int K, int renorm, int* __restrict__ topk_idx, float* __restrict__ topk_w,
                  const PrepArgs prep, int tp) {
  constexpr int TB = 8 * TMT;  // tokens per CTA: 4 warps x 2 lane groups x TMT
  extern __shared__ __align__(16) float smem[];
  __shared__ int s_hist[kRouteMaxExperts];
  float* ls = smem;  // [TB][256] after the h loop
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const bool computes = warp < kWideComputeWarps;
  const int ft = threadIdx.x - 32 * kWideComputeWarps;
  const int grp = 2 * (computes ? warp : 0) + lane % 2;  // this thread's token group: tokens grp*TMT .. +TMT-1
  const int ebase = 4 * (lane / 2);                       // experts ebase + 64*i + q, i < 4, q < 4
  const int t0 = blockIdx.x * TB;
  const int tvalid = min(TB, T - t0);
  const int nchunks = (H + kWideHC - 1) / kWideHC;
  // The x tile has 8 slots per token group (16-byte aligned for any TMT); slots past TMT stay zero.
  auto x_row = [&](int slot) {
    const int tl = (slot / 8) * TMT + slot % 8;
    return (slot % 8 < TMT && tl < tvalid) ? t0 + tl : -1;
  };
  auto w_row = [&](int e) { return e < E ? e : -1; };

  float acc[TMT][16];
#pragma unroll
  for (int j = 0; j < TMT; ++j)
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[j][i] = 0.0f;

  constexpr int P = sizeof(XT) == 2 ? 2 : 1;  // chunks kept in flight in the staging warps' registers
  WideChunk<XT, kWideSlots> xr[P];
  WideChunk<XT, kWideEP> wrg[P];
  pdl_wait();
  pdl_trigger();
  route_prep_begin(prep, s_hist);
  if (!computes) {  // chunk 0 into buffer 0, chunks 1..P into the registers (slot = chunk % P)
    xr[0].load(ft, x, x_row, H, 0);
    wrg[0].load(ft, wr, w_row, H, 0);
    xr[0].store(ft, smem);
    wrg[0].store(ft, smem + kWideHC * kWideSlots);
#pragma unroll
    for (int j = 1; j <= P; ++j) {  // past H: zero-filled, never stored
      xr[j % P].load(ft, x, x_row, H, j * kWideHC);
      wrg[j % P].load(ft, wr, w_row, H, j * kWideHC);
    }
  }
  for (int c0 = 0; c0 < nchunks; c0 += P) {
#pragma unroll
    for (int p = 0; p < P; ++p) {
      const int c = c0 + p;  // every thread runs the same number of barriers; chunks past the end do nothing
      __syncthreads();       // buffer c&1 holds chunk c; buffer (c+1)&1 is no longer read
      if (!computes) {
        if (c + 1 < nchunks) {
          float* nxt = smem + ((c + 1) & 1) * kWideBuf;
          xr[(p + 1) % P].store(ft, nxt);
          wrg[(p + 1) % P].store(ft, nxt + kWideHC * kWideSlots);
          xr[(p + 1) % P].load(ft, x, x_row, H, (c + 1 + P) * kWideHC);
          wrg[(p + 1) % P].load(ft, wr, w_row, H, (c + 1 + P) * kWideHC);
        }
        continue;
      }
      if (c >= nchunks) continue;
      const float* xs = smem + (c & 1) * kWideBuf + 8 * grp;              // [h][slot]
      const float* ws = smem + (c & 1) * kWideBuf + kWideHC * kWideSlots + ebase;  // [h][expert]
      // software pipeline: the operands of step hh+1 are loaded while step hh is computed.  The tail of
      // a short last chunk is zero in shared memory and fma(0, 0, acc) leaves acc alone.
      float4 xa = *reinterpret_cast<const float4*>(xs);
      float4 xb = *reinterpret_cast<const float4*>(xs + 4);
      float4 wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) wv[i] = *reinterpret_cast<const float4*>(ws + 64 * i);
#pragma unroll 2
      for (int hh = 0; hh < kWideHC; ++hh) {
        const int hn = hh + 1 < kWideHC ? hh + 1 : hh;
        const float4 nxa = *reinterpret_cast<const float4*>(xs + hn * kWideSlots);
        const float4 nxb = *reinterpret_cast<const float4*>(xs + hn * kWideSlots + 4);
        float4 nwv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) nwv[i] = *reinterpret_cast<const float4*>(ws + hn * kWideEP + 64 * i);
        const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
        for (int j = 0; j < TMT; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            acc[j][4 * i + 0] = __fmaf_rn(xv[j], wv[i].x, acc[j][4 * i + 0]);
            acc[j][4 * i + 1] = __fmaf_rn(xv[j], wv[i].y, acc[j][4 * i + 1]);
            acc[j][4 * i + 2] = __fmaf_rn(xv[j], wv[i].z, acc[j][4 * i + 2]);
            acc[j][4 * i + 3] = __fmaf_rn(xv[j], wv[i].w, acc[j][4 * i + 3]);
          }
        xa = nxa;
        xb = nxb;
#pragma unroll
        for (int i = 0; i < 4; ++i) wv[i] = nwv[i];
      }
    }
  }
  __syncthreads();
  if (computes) {
#pragma unroll
    for (int j = 0; j < TMT; ++j) {
      const int tl = grp * TMT + j;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int e0 = ebase + 64 * i;
        float l[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          l[q] = acc[j][4 * i + q];
          if (bias != nullptr && e0 + q < E) l[q] = l[q] + bias[e0 + q];
        }
        *reinterpret_cast<float4*>(ls + tl * kWideEP + e0) = make_float4(l[0], l[1], l[2], l[3]);
      }
    }
  }
  __syncthreads();
  select_topk<kWideEP>(ls, tvalid, t0, E, K, renorm, topk_idx, topk_w, prep.hist ? s_hist : nullptr, tp);
  route_prep_end(prep, s_hist);
}

template <typename XT, int TMT>
static int launch_wide_tmt(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                           float* topk_w, const PrepArgs& prep, cudaStream_t st) {
  constexpr size_t stage = sizeof(float) * 2 * kWideBuf, logits = sizeof(float) * 8 * TMT * kWideEP;
  constexpr size_t smem = stage > logits ? stage : logits;
  auto kern = route_wide_kernel<XT, TMT>;
  static SmemAttrOnce once;  // per instantiation
  if (cudaError_t e = ensure_dynamic_smem(kern, smem, p->device, once)) return (int)e;
  const moe_config_t& c = p->cfg;
  p->launches += 1;
  return (int)launch_maybe_pdl(false, kern, dim3((c.T + 8 * TMT - 1) / (8 * TMT)), dim3(kWideThreads), smem, st,
                               (const XT*)x, (const XT*)wr, bias, c.T, c.H, p->route_E, p->route_K, c.renormalize, topk_idx, topk_w, prep, p->tp);
}

template <typename XT>
static int launch_wide(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                       float* topk_w, const PrepArgs& prep, cudaStream_t st) {
  // Tokens per thread: the time is (waves of CTAs over the SMs) x TMT; ties go to the larger tile.
  const int T = p->cfg.T, sms = p->sm_count > 0 ? p->sm_count : 148;
  int best = 8, best_cost = 1 << 30;
  for (int tmt = 8; tmt >= 4; --tmt) {
    const int ctas = (T + 8 * tmt - 1) / (8 * tmt);
    const int cost = (ctas + sms - 1) / sms * tmt;
    if (cost < best_cost) { best_cost = cost; best = tmt; }
  }
  switch (best) {
    case 4: return launch_wide_tmt<XT, 4>(p, x, wr, bias, topk_idx, topk_w, prep, st);
    case 5: return launch_wide_tmt<XT, 5>(p, x, wr, bias, topk_idx, topk_w, prep, st);
    case 6: return launch_wide_tmt<XT, 6>(p, x, wr, bias, topk_idx, topk_w, prep, st);
    case 7: return launch_wide_tmt<XT, 7>(p, x, wr, bias, topk_idx, topk_w, prep, st);
    default: return launch_wide_tmt<XT, 8>(p, x, wr, bias, topk_idx, topk_w, prep, st);
  }
}

// The latency-bound shapes (E <= 64).  x and Wr tiles stay in their natural [row][h] layout in shared
// memory (fp32, converted while staging); a lane owns one token and two experts, reads four consecutive h
// of its token and of each expert with 16-byte loads and runs its two chains over them.  What bounds the
// kernel is the shared-memory pipe, not the chains (measured on this part): a 16-byte load costs the SM
// 2 pipe cycles when the lanes that share an address are neighbours (lane / 2) or alternate (lane % 2)
// and 4 cycles otherwise, and a warp that has the SM to itself still waits about 8 cycles per load.  So a
// warp is 16 tokens x 2 expert groups (SWAP = false: token by lane / 2, group by lane % 2; 4 experts per
// warp) or 2 tokens x 16 groups (SWAP = true: 32 experts per warp, for many experts), every load a 2-cycle
// one, three loads per 8 FMAs, and enough warps per SM to keep the pipe busy.
//
// The compute warps only run chains.  Four more warps stage: while the compute warps work on one
// shared-memory buffer, the staging warps convert the next chunk (already in their registers) into the
// other buffer and fetch from global memory the chunks after it, so neither the global-memory latency nor
// the conversion sits on the chains' critical path.  One __syncthreads per chunk.
constexpr int kNarrowFillWarps = 4;

// Four elements per staging load (16 bytes of fp32, 8 bytes of bf16): every thread then writes one 16-byte
// vector and consecutive lanes write consecutive vectors, which is free of bank conflicts (eight bf16
// per thread made two vectors 32 bytes apart per lane: a two-way conflict on every store).
template <typename XT> struct Stage4;
template <> struct Stage4<float> {
  typedef uint4 V;
  static __device__ __forceinline__ V zero() { return make_uint4(0, 0, 0, 0); }
  static __device__ __forceinline__ V ld(const float* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  static __device__ __forceinline__ float4 cvt(const V& v) {
    return make_float4(__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w));
  }
};
template <> struct Stage4<__nv_bfloat16> {
  typedef uint2 V;
  static __device__ __forceinline__ V zero() { return make_uint2(0, 0); }
  static __device__ __forceinline__ V ld(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint2*>(p)); }
  static __device__ __forceinline__ float4 cvt(const V& v) {  // bf16 -> fp32 is a 16-bit shift
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                       __uint_as_float(v.y & 0xffff0000u));
  }
};

template <typename XT, int ROWS, int HC>
struct NaturalChunk {
  static constexpr int FT = 32 * kNarrowFillWarps;  // staging threads
  static constexpr int N = 4;
  static constexpr int PARTS = HC / N;
  static constexpr int NVEC = ROWS * PARTS;
  static constexpr int PER_THREAD = (NVEC + FT - 1) / FT;
  static constexpr int PITCH = HC + 4;  // floats; rows land on different banks
  typename Stage4<XT>::V v[PER_THREAD];
  // ft: index of the calling thread among the staging threads
  __device__ __forceinline__ void load(int ft, const XT* base, int row0, int nrows_valid, int H, int h0) {
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = ft + i * FT;
      const int r = idx / PARTS, part = idx % PARTS;
      const int h = h0 + part * N;
      v[i] = Stage4<XT>::zero();
      if (idx < NVEC && r < nrows_valid && h < H) v[i] = Stage4<XT>::ld(base + (size_t)(row0 + r) * H + h);
    }
  }
  __device__ __forceinline__ void store(int ft, float* s) const {  // s: [ROWS][PITCH]
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
      const int idx = ft + i * FT;
      if (idx < NVEC) {
        const int r = idx / PARTS, part = idx % PARTS;
        *reinterpret_cast<float4*>(s + r * PITCH + part * N) = Stage4<XT>::cvt(v[i]);
      }
    }
  }
};

// EW warps side by side cover the experts, TWP warps the tokens of the block.
template <typename XT, bool SWAP, int EW, int TWP, int HC>
__global__ void __launch_bounds__(32 * (EW * TWP + kNarrowFillWarps))
route_narrow_kernel(const XT* __restrict__ x, const XT* __restrict__ wr, const float* __restrict__ bias, int T,
                    int H, int E, int K, int renorm, int* __restrict__ topk_idx, float* __restrict__ topk_w,
                    const PrepArgs prep, int tp) {
  __shared__ int s_hist[kRouteMaxExperts];
  constexpr int TN = 2;                    // experts per lane
  constexpr int G = SWAP ? 16 : 2;         // expert groups per warp
  constexpr int TW = 32 / G;               // tokens per warp
  constexpr int EPW = G * TN;              // experts per warp
  constexpr int EP = EW * EPW;             // experts covered (padded)
  constexpr int TB = TW * TWP;             // tokens per block
  constexpr int CW = EW * TWP;             // compute warps
  constexpr int PITCH = HC + 4;
  constexpr int BUF = (TB + EP) * PITCH;   // floats per buffer: x tile [TB][PITCH], then Wr tile [EP][PITCH]
  extern __shared__ __align__(16) float smem[];
  float* ls = smem;                        // [TB][EP] after the h loop
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const bool computes = warp < CW;
  const int ft = threadIdx.x - 32 * CW;
  const int tl = (computes ? warp / EW : 0) * TW + (SWAP ? lane % 2 : lane / 2);   // this lane's token inside the block
  const int le = (computes ? warp % EW : 0) * EPW + (SWAP ? lane / 2 : lane % 2);  // this lane's experts: le + G*i
  const int t0 = blockIdx.x * TB;
  const int tvalid = min(TB, T - t0);
  const int nchunks = (H + HC - 1) / HC;

  float acc[TN];
#pragma unroll
  for (int i = 0; i < TN; ++i) acc[i] = 0.0f;
  // The staging warps keep P chunks in flight in registers, so that global memory is not waited for.
  constexpr int P = 2;
  NaturalChunk<XT, TB, HC> xr[P];
  NaturalChunk<XT, EP, HC> wrg[P];
  pdl_wait();
  pdl_trigger();
  route_prep_begin(prep, s_hist);
  if (!computes) {  // chunk 0 into buffer 0, chunks 1..P into the registers (slot = chunk % P)
    xr[0].load(ft, x, t0, tvalid, H, 0);
    wrg[0].load(ft, wr, 0, E, H, 0);
    xr[0].store(ft, smem);
    wrg[0].store(ft, smem + TB * PITCH);
#pragma unroll
    for (int j = 1; j <= P; ++j) {  // past H: zero-filled, never stored
      xr[j % P].load(ft, x, t0, tvalid, H, j * HC);
      wrg[j % P].load(ft, wr, 0, E, H, j * HC);
    }
  }
  for (int c0 = 0; c0 < nchunks; c0 += P) {
#pragma unroll
    for (int p = 0; p < P; ++p) {
      const int c = c0 + p;  // every thread runs the same number of barriers; chunks past the end do nothing
      __syncthreads();       // buffer c&1 holds chunk c; buffer (c+1)&1 is no longer read
      float* cur = smem + (c & 1) * BUF;
      if (!computes) {
        if (c + 1 < nchunks) {
          float* nxt = smem + ((c + 1) & 1) * BUF;
          xr[(p + 1) % P].store(ft, nxt);
          wrg[(p + 1) % P].store(ft, nxt + TB * PITCH);
          xr[(p + 1) % P].load(ft, x, t0, tvalid, H, (c + 1 + P) * HC);
          wrg[(p + 1) % P].load(ft, wr, 0, E, H, (c + 1 + P) * HC);
        }
        continue;
      }
      if (c >= nchunks) continue;
      const float* xrow = cur + tl * PITCH;
      const float* wrow = cur + TB * PITCH + le * PITCH;
      // Four h at a time, the operands D steps ahead in flight.  The tail of a short last chunk is zero
      // in shared memory (loads past H are zero-filled) and fma(0, 0, acc) leaves acc alone.
      constexpr int D = 2;
      float4 xv[D], wv[D][TN];
#pragma unroll
      for (int d = 0; d < D; ++d) {
        xv[d] = *reinterpret_cast<const float4*>(xrow + 4 * d);
#pragma unroll
        for (int i = 0; i < TN; ++i) wv[d][i] = *reinterpret_cast<const float4*>(wrow + G * i * PITCH + 4 * d);
      }
#pragma unroll 4
      for (int hh = 0; hh < HC; hh += 4) {
        const int hn = hh + 4 * D < HC ? hh + 4 * D : HC - 4;
        const float4 nxv = *reinterpret_cast<const float4*>(xrow + hn);
        float4 nwv[TN];
#pragma unroll
        for (int i = 0; i < TN; ++i) nwv[i] = *reinterpret_cast<const float4*>(wrow + G * i * PITCH + hn);
#pragma unroll
        for (int i = 0; i < TN; ++i) acc[i] = __fmaf_rn(xv[0].x, wv[0][i].x, acc[i]);
#pragma unroll
        for (int i = 0; i < TN; ++i) acc[i] = __fmaf_rn(xv[0].y, wv[0][i].y, acc[i]);
#pragma unroll
        for (int i = 0; i < TN; ++i) acc[i] = __fmaf_rn(xv[0].z, wv[0][i].z, acc[i]);
#pragma unroll
        for (int i = 0; i < TN; ++i) acc[i] = __fmaf_rn(xv[0].w, wv[0][i].w, acc[i]);
#pragma unroll
        for (int d = 0; d + 1 < D; ++d) {
          xv[d] = xv[d + 1];
#pragma unroll
          for (int i = 0; i < TN; ++i) wv[d][i] = wv[d + 1][i];
        }
        xv[D - 1] = nxv;
#pragma unroll
        for (int i = 0; i < TN; ++i) wv[D - 1][i] = nwv[i];
      }
    }
  }
  __syncthreads();
  if (computes) {
#pragma unroll
    for (int i = 0; i < TN; ++i) {
      const int e = le + G * i;
      float l = acc[i];
      if (bias != nullptr && e < E) l = l + bias[e];
      ls[tl * EP + e] = l;
    }
  }
  __syncthreads();
  select_topk<EP>(ls, tvalid, t0, E, K, renorm, topk_idx, topk_w, prep.hist ? s_hist : nullptr, tp);
  route_prep_end(prep, s_hist);
}

template <typename XT, bool SWAP, int EW, int TWP, int HC>
static int launch_narrow(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                         float* topk_w, const PrepArgs& prep, cudaStream_t st) {
  constexpr int G = SWAP ? 16 : 2, EP = EW * G * 2, TB = (32 / G) * TWP;
  constexpr size_t smem = sizeof(float) * (2 * (TB + EP) * (HC + 4) > TB * EP ? 2 * (TB + EP) * (HC + 4) : TB * EP);
  auto kern = route_narrow_kernel<XT, SWAP, EW, TWP, HC>;
  static SmemAttrOnce once;  // per instantiation
  if (smem > 48 * 1024)
    if (cudaError_t e = ensure_dynamic_smem(kern, smem, p->device, once)) return (int)e;
  const moe_config_t& c = p->cfg;
  p->launches += 1;
  return (int)launch_maybe_pdl(false, kern, dim3((c.T + TB - 1) / TB), dim3(32 * (EW * TWP + kNarrowFillWarps)), smem, st,
                               (const XT*)x, (const XT*)wr, bias, c.T, c.H, p->route_E, p->route_K, c.renormalize, topk_idx, topk_w, prep, p->tp);
}

template <typename XT>
static int launch_typed(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                        float* topk_w, const PrepArgs& prep, cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  // 16 tokens x 2 expert groups per warp, two compute warps per CTA (32 tokens: T = 4096 gives 128
  // CTAs); with many experts 2 tokens x 16 groups, so that the chains still spread over the SMs.
  constexpr int HL = sizeof(XT) == 2 ? 256 : 128;  // h per chunk
  const int E = p->route_E;  // the experts the router scores (the plan's E counts every TP shard of an expert)
  if (E <= 8) return launch_narrow<XT, false, 2, 2, HL>(p, x, wr, bias, topk_idx, topk_w, prep, st);   // 32 tokens per CTA
  if (E <= 16) return launch_narrow<XT, false, 4, 2, HL>(p, x, wr, bias, topk_idx, topk_w, prep, st);  // 32 tokens per CTA
  if (E <= 32) return launch_narrow<XT, true, 1, 4, HL / 2>(p, x, wr, bias, topk_idx, topk_w, prep, st);  // 8 tokens per CTA
  if (E <= 64) return launch_narrow<XT, true, 2, 2, HL / 2>(p, x, wr, bias, topk_idx, topk_w, prep, st);  // 4 tokens per CTA
  return launch_wide<XT>(p, x, wr, bias, topk_idx, topk_w, prep, st);
}

int launch_route(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                 float* topk_w, const PrepArgs* prep_or_null, cudaStream_t st) {
  if (p->cfg.T == 0) return 0;
  PrepArgs prep = {};
  if (prep_or_null != nullptr) prep = *prep_or_null;
  if (route_filter_applies(p)) return launch_route_filter(p, x, wr, bias, topk_idx, topk_w, prep, st);
  if (p->cfg.dtype == MOE_DTYPE_BF16)
    return launch_typed<__nv_bfloat16>(p, x, wr, bias, topk_idx, topk_w, prep, st);
  return launch_typed<float>(p, x, wr, bias, topk_idx, topk_w, prep, st);
}

}  // namespace moehub
