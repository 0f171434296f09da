// Step 1 of the MoE layer (paper Section II-A, routing) for many experts on bf16 data: a tensor-core filter
// in front of the exact chains.
//
// The pick of the K experts is defined on ONE ascending fp32 FMA chain per (token, expert), and it has to
// come out bit for bit.  Only a handful of the E chains of a token decide anything, though.  So:
//
//  (1) route_tc_logits_kernel: approximate logits l~ = x * Wr^T for every (token, expert) with tcgen05 MMAs
//      (128 tokens x 128 experts per CTA, operands by TMA, four fp32 accumulators in tensor memory that take the
//      64-column steps of h in turn and are summed at the end), written to a [T, 256] fp32 scratch.  Products of two bf16 numbers are exact in fp32; only the order and rounding
//      of the additions differ from the chain.  Its idle epilogue warps also compute |w_e|^2 per expert.
//  (2) route_refine_kernel: per token, the K-th largest approximate logit minus twice an error bound is a
//      threshold; every expert at or above it is a candidate and gets its exact chain; the exact values
//      replace the approximate ones and the usual selection runs on the row.
//
// Why the picks are the exact ones.  Error model: every fp32 addition, in whatever order and whether rounded
// to nearest or truncated, is off by at most 2^-23 of a magnitude that never exceeds S = sum_h |x_h * w_eh|.
// A sum of H products has H - 1 additions, so |l~ - exact sum| <= H * 2^-23 * S, and the chain (rounded to
// nearest) is within H * 2^-24 * S of it: |l~ - l| <= eps = 1.5 * H * 2^-23 * S, with S <= |x_t| * max_e |w_e|
// (Cauchy-Schwarz) computed from the data of the call.  The K experts with the largest l~ have l >= kth~ - eps
// and every expert below the threshold kth~ - 2 eps has l < kth~ - eps, so none of those can be among the K
// largest l, ties included.  The kernel checks the model on every candidate (both values are at hand) and
// reports MOE_ERR_INTERNAL if |l~ - l| ever exceeded eps.
//
// The softmax weights use the exact logits of the candidates and the approximate ones of the rest: the rest
// only enters the denominator.  What the accumulation's rounding adds up to grows with the number of additions
// in a row (measured), which is why the approximate logit is the sum of four accumulators.
#include "route_common.cuh"
#include "tc_common.cuh"

namespace moehub {

constexpr int kRfEP = 256;           // experts covered (the accumulator's columns)
constexpr float kRfEps = 1.5f * 1.1920929e-7f;  // 1.5 * 2^-23
constexpr int kRfChunk = 64;         // h per staged chunk: 128 bytes of a row
constexpr int kRfBufs = 3;           // staged chunks in flight
constexpr int kRfWBytes = kRfEP * kRfChunk * 2;  // one chunk of every expert's row: 32 KB
// shared memory of the refine kernel for TPC tokens per CTA (half a warp each): kRfBufs buffers of one chunk of Wr
// and of the tokens' rows of x (written by TMA, 128-byte swizzle), the tokens' logit rows, the list of chains
constexpr size_t rf_smem(int tpc) {
  return 1024 + (size_t)kRfBufs * (kRfWBytes + tpc * kRfChunk * 2) + (size_t)tpc * kRfEP * 4 + (size_t)tpc * kRfEP * 2;
}

// M = 128 tokens, N = 128 experts per MMA
constexpr uint32_t kRfIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

struct RfShared {
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long acc_full;
  unsigned long long drain;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kTcThreads, 1)
route_tc_logits_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                       const __nv_bfloat16* __restrict__ wr, int T, int H, int E, float* __restrict__ logits,
                       float* __restrict__ wnorm2, unsigned long long wait_ns, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* stage_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  RfShared* sh = reinterpret_cast<RfShared*>(stage_base + kStages * kStageBytes);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->acc_full), 1);
    mbar_init(smem_u32(&sh->drain), 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                 "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();
  pdl_trigger();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  volatile int* abort_flag = &sh->abort_flag;
  const int KB = (H + kBK - 1) / kBK;
  const int t0 = blockIdx.x * kTileRows;
  const int e0 = blockIdx.y * 128;  // this CTA's half of the experts
  int fail_site = 0;

  if (warp == 0) {
    if (lane == 0) {  // TMA producer: the tokens' x tile and all experts' Wr block, 64 columns of h per stage
      int stage = 0, armed[kStages];
      uint32_t phase_bit = 0;
#pragma unroll
      for (int s = 0; s < kStages; ++s) armed[s] = 0;
      for (int kb = 0; kb < KB; ++kb) {
        if (!mbar_wait(smem_u32(&sh->empty[stage]), phase_bit ^ 1u, abort_flag, wait_ns)) { fail_site = kWaitMbarTma; break; }
        const uint32_t full = smem_u32(&sh->full[stage]);
        const uint32_t a_dst = smem_u32(stage_base + stage * kStageBytes);
        mbar_expect_tx(full, (uint32_t)(kABytes + kBBytes / 2));
        tma_load_2d(a_dst, &map_x, full, kb * kBK, t0);   // rows past T and columns past H arrive as zeros
        tma_load_2d(a_dst + kABytes, &map_w, full, kb * kBK, e0);  // 128 experts' rows
#pragma unroll
        for (int s = 0; s < kStages; ++s)
          if (s == stage) armed[s] += 1;
        if (++stage == kStages) { stage = 0; phase_bit ^= 1u; }
      }
      if (fail_site || *abort_flag) {  // leave no copy in flight
        sh->abort_flag = 1;
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
          if (armed[s] == 0) continue;
          const unsigned long long ts = globaltimer();
          while (!mbar_try(smem_u32(&sh->full[s]), (uint32_t)((armed[s] - 1) & 1)))
            if (globaltimer() - ts > wait_ns + 1000000ull) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {  // MMA issuer: D[128 tokens, 256 experts] += x tile * Wr block^T
      int stage = 0;
      uint32_t phase_bit = 0;
      for (int kb = 0; kb < KB; ++kb) {
        if (!mbar_wait(smem_u32(&sh->full[stage]), phase_bit, abort_flag, wait_ns)) { fail_site = kWaitMbarMma; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(stage_base + stage * kStageBytes);
        const uint64_t adesc = smem_desc_sw128(a_addr), bdesc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
        // four accumulators that take the steps in turn: a quarter as many additions in a row for each logit
        // (they are summed in the epilogue), and so a quarter of what the accumulation's rounding adds up to
        for (int k = 0; k < kBK / 16; ++k)
          tc_mma(tmem_base + (uint32_t)(kb & 3) * 128u, adesc + 2 * k, bdesc + 2 * k, kRfIdesc, ((kb >> 2) | k) != 0 ? 1u : 0u);
        tc_commit(smem_u32(&sh->empty[stage]));
        if (++stage == kStages) { stage = 0; phase_bit ^= 1u; }
      }
      if (!fail_site) tc_commit(smem_u32(&sh->acc_full));
      if (fail_site) sh->abort_flag = 1;
      if (fail_site || *abort_flag) {  // nothing of this thread's may still run when the CTA frees tensor memory
        tc_commit(smem_u32(&sh->drain));
        const unsigned long long ts = globaltimer();
        while (!mbar_try(smem_u32(&sh->drain), 0u))
          if (globaltimer() - ts > wait_ns + 1000000ull) break;
      }
    }
  } else {
    // While the main loop runs: |w_e|^2 for this CTA's share of the experts (the refine kernel's error bound).
    for (int e = (blockIdx.y * gridDim.x + blockIdx.x) * 4 + (warp - 2); e < E; e += gridDim.x * gridDim.y * 4) {
      const uint4* row = reinterpret_cast<const uint4*>(wr + (size_t)e * H);
      float s = 0.0f;
      for (int v = lane; v < H / 8; v += 32) {
        float f[8];
        Vec16<__nv_bfloat16>::unpack(__ldg(row + v), f);
#pragma unroll
        for (int q = 0; q < 8; ++q) s = fmaf(f[q], f[q], s);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
      if (lane == 0) wnorm2[e] = s;
    }
    // epilogue: the accumulator row of token t0 + 32 * (warp % 4) + lane, 16 experts at a time
    const int quarter = warp & 3;
    if (!mbar_wait(smem_u32(&sh->acc_full), 0u, abort_flag, wait_ns, 200)) {
      fail_site = kWaitMbarEpi;
    } else {
      tc_fence_after();
      const int t = t0 + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
      float* dst = logits + (size_t)t * kRfEP + e0;
      const int nacc = min(KB, 4);  // accumulators that were written at all
#pragma unroll 1
      for (int c = 0; c < 128; c += 16) {
        float f[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) f[q] = 0.0f;
        for (int a = 0; a < nacc; ++a) {
          uint32_t v[16];
          tc_ld16(t_row + (uint32_t)a * 128u + c, v);
          tc_wait_ld();
#pragma unroll
          for (int q = 0; q < 16; ++q) f[q] += __uint_as_float(v[q]);
        }
        if (t < T) {
#pragma unroll
          for (int q = 0; q < 16; q += 4) *reinterpret_cast<float4*>(dst + c + q) = make_float4(f[q], f[q + 1], f[q + 2], f[q + 3]);
        }
      }
    }
    if (fail_site) sh->abort_flag = 1;
  }
  if (fail_site) set_status(status, MOE_ERR_TIMEOUT, fail_site);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}


// ---- (2) candidates, exact chains, selection ----------------------------------------------------------
// A CTA takes TPC tokens, half a warp each (a warp runs two tokens in lockstep) for everything that is per
// token: the row of approximate logits (+ bias) into shared memory; |x_t| from the row of x; the K-th largest
// approximate logit by K rounds of a 16-lane arg-max; the threshold; the candidates.  The chains of all
// tokens of the CTA are then numbered through and thread s runs chain s (so no lane idles because its token
// has few candidates).  A chain reads its expert's row of Wr front to back; threads reading different rows
// straight from global memory would spend their time in the load unit and fetch a row once per (token,
// candidate) pair, so one thread brings in one chunk (64 h: 128 bytes) of EVERY expert's row and of every
// token's row of x per step with two TMA copies, kRfBufs - 1 chunks ahead, and each chain reads its rows from
// shared memory (128-byte swizzle: 16-byte unit u of row r sits at u ^ (r % 8)).  Exact values go back into
// the logit rows; then the common selection.
__device__ __forceinline__ uint4 lds128(uint32_t addr) {  // a shared-memory load by its 32-bit shared address
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

template <int TPC>
__global__ void __launch_bounds__(TPC * 16, 1)
route_refine_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                    const __nv_bfloat16* __restrict__ x, const float* __restrict__ bias, const float* __restrict__ logits,
                    const float* __restrict__ wnorm2, int T, int H, int E, int K, int renorm, int* __restrict__ topk_idx,
                    float* __restrict__ topk_w, const PrepArgs prep, int tp, unsigned long long wait_ns,
                    int* __restrict__ status) {
  constexpr int NT = TPC * 16;
  constexpr int kXBytes = TPC * kRfChunk * 2;
  __shared__ int s_hist[kRouteMaxExperts];
  __shared__ int s_ncand[TPC];
  __shared__ float s_eps[TPC];
  __shared__ unsigned long long s_full[kRfBufs];
  __shared__ unsigned long long s_empty[kRfBufs];  // a buffer may be refilled once every warp has left it
  __shared__ int s_abort;
  extern __shared__ uint8_t rf_dyn[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(rf_dyn) + 1023) & ~(uintptr_t)1023);
  uint8_t* w_stage = base;                                              // [kRfBufs][256 experts][128 bytes]
  uint8_t* x_stage = base + (size_t)kRfBufs * kRfWBytes;                // [kRfBufs][TPC tokens][128 bytes]
  float* ls = reinterpret_cast<float*>(x_stage + (size_t)kRfBufs * kXBytes);  // [TPC][256] logits: approximate, exact where a chain ran
  unsigned short* chains = reinterpret_cast<unsigned short*>(ls + (size_t)TPC * kRfEP);  // [TPC * 256]: token << 8 | expert
  const int t0 = blockIdx.x * TPC;
  const int tvalid = min(TPC, T - t0);
  const int lane = threadIdx.x % 32, l16 = threadIdx.x % 16, half = lane / 16;
  const int tl = threadIdx.x / 16;  // this half-warp's token inside the block
  const bool live = tl < tvalid;
  const unsigned hmask = 0xffffu << (16 * half);
  if (threadIdx.x == 0) {
    for (int b = 0; b < kRfBufs; ++b) {
      mbar_init(smem_u32(&s_full[b]), 1);
      mbar_init(smem_u32(&s_empty[b]), NT / 32);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  pdl_wait();
  pdl_trigger();
  route_prep_begin(prep, s_hist);
  volatile int* abort_flag = &s_abort;

  // the row of approximate logits (16 per lane: experts l16 + 16 j), bias added the way the chain's value gets it
  float v[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int e = l16 + 16 * j;
    float a = -FLT_MAX;
    if (live && e < E) {
      a = logits[(size_t)(t0 + tl) * kRfEP + e];
      if (bias != nullptr) a = a + bias[e];
    }
    v[j] = a;
    ls[tl * kRfEP + e] = a;
  }
  // |x_t|^2 and max_e |w_e|^2
  float xn2 = 0.0f, wm2 = 0.0f;
  if (live) {
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)(t0 + tl) * H);
    for (int q = l16; q < H / 8; q += 16) {
      float f[8];
      Vec16<__nv_bfloat16>::unpack(__ldg(xr + q), f);
#pragma unroll
      for (int i = 0; i < 8; ++i) xn2 = fmaf(f[i], f[i], xn2);
    }
  }
  for (int e = l16; e < E; e += 16) wm2 = fmaxf(wm2, wnorm2[e]);
#pragma unroll
  for (int off = 8; off > 0; off >>= 1) {
    xn2 += __shfl_xor_sync(0xffffffffu, xn2, off);
    wm2 = fmaxf(wm2, __shfl_xor_sync(0xffffffffu, wm2, off));
  }
  // K-th largest approximate logit: K rounds, each removes one maximum (lowest index among equals)
  unsigned taken = 0;
  float kth = -FLT_MAX;
  for (int k = 0; k < K; ++k) {
    float bv = -FLT_MAX;
    int be = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int e = l16 + 16 * j;
      const bool ok = (e < E) && !((taken >> j) & 1u);
      if (ok && (be == 0x7fffffff || v[j] > bv)) { bv = v[j]; be = e; }
    }
#pragma unroll
    for (int off = 8; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
      const int oe = __shfl_xor_sync(0xffffffffu, be, off);
      const bool other = (oe != 0x7fffffff) && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be));
      if (other) { bv = ov; be = oe; }
    }
    if (be != 0x7fffffff && (be & 15) == l16) taken |= 1u << (be >> 4);
    kth = bv;
  }
  // The error bound of this token (a little extra for the two roundings of "+ bias").  First threshold: one bound
  // (plus a sliver) below the K-th largest approximate logit - half the window the proof needs, so about ten
  // candidates instead of twelve and hardly ever more than sixteen.  The missing half is made up afterwards with
  // the exact values: see the end of the round.
  const float eps = kRfEps * (float)H * sqrtf(xn2 * wm2) * 1.0001f + 4.0e-7f * (1.0f + fabsf(kth));
  if (l16 == 0) s_eps[tl] = eps;
  float thr = kth - eps - 1.0e-3f * (1.0f + fabsf(kth));
  unsigned done = 0;  // bit j: the chain of expert l16 + 16 j has been run
  const int nchunk = (H + kRfChunk - 1) / kRfChunk;
  int issued = 0, consumed = 0;  // chunks over all passes: buffer = count % kRfBufs, phase = count / kRfBufs
  bool failed = false;
  // The copies are issued by one thread: the first lane of the last warp, which has chains to run only when the
  // CTA's list is full.  The warps are not held together by a barrier per step: each waits for the step's buffer,
  // runs its chains over it and reports that it has left it; the issuing thread refills a buffer when all have.
  const bool producer = threadIdx.x == NT - 32;
  auto issue = [&](int ch) {  // the producer only
    const int b = issued % kRfBufs;
    if (!mbar_wait(smem_u32(&s_empty[b]), ((uint32_t)(issued / kRfBufs) & 1u) ^ 1u, abort_flag, wait_ns)) {
      failed = true;
      s_abort = 1;
      return;
    }
    const uint32_t bar = smem_u32(&s_full[b]);
    mbar_expect_tx(bar, (uint32_t)(kRfWBytes + kXBytes));
    tma_load_2d(smem_u32(w_stage + (size_t)b * kRfWBytes), &map_w, bar, ch * kRfChunk, 0);   // rows past E, columns past H: zeros
    tma_load_2d(smem_u32(x_stage + (size_t)b * kXBytes), &map_x, bar, ch * kRfChunk, t0);    // rows past T: zeros
    ++issued;
  };
  // candidates of the first round, while the approximate logits are still in registers (later rounds, which are
  // rare, fetch them again: the chains' loop should not have to carry sixteen values it never uses)
  unsigned cand0 = 0;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int e = l16 + 16 * j;
    if (live && e < E && v[j] >= thr) cand0 |= 1u << j;
  }
  for (int round = 0; round < 3; ++round) {  // a second round is rare, a third cannot be needed
    // candidates of this round: at or above the threshold and not yet done; counted, then listed CTA-wide
    unsigned cand = cand0;
    if (round > 0) {
      cand = 0;
      if (live && thr < FLT_MAX) {
        for (int j = 0; j < 16; ++j) {
          const int e = l16 + 16 * j;
          if (e >= E || ((done >> j) & 1u)) continue;
          float a = logits[(size_t)(t0 + tl) * kRfEP + e];
          if (bias != nullptr) a = a + bias[e];
          if (a >= thr) cand |= 1u << j;
        }
      }
    }
    int n_cand = __popc(cand);
#pragma unroll
    for (int off = 8; off > 0; off >>= 1) n_cand += __shfl_xor_sync(0xffffffffu, n_cand, off);
    if (l16 == 0) s_ncand[tl] = n_cand;
    __syncthreads();
    int first = 0, total = 0;
    for (int i = 0; i < TPC; ++i) {
      const int n = s_ncand[i];
      if (i < tl) first += n;
      total += n;
    }
    if (total == 0) break;  // no token of the CTA asks for more (CTA-uniform)
    {  // this token's chains: lanes in order, each lane its experts in order
      int mine = __popc(cand), before = mine;
#pragma unroll
      for (int off = 1; off < 16; off <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, before, off, 16);
        if (l16 >= off) before += o;
      }
      int pos = first + before - mine;
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if ((cand >> j) & 1u) chains[pos++] = (unsigned short)((tl << 8) | (l16 + 16 * j));
      done |= cand;
    }
    __syncthreads();
    const int passes = (total + NT - 1) / NT;
    for (int p = 0; p < passes; ++p) {
      const int sidx = p * NT + threadIdx.x;
      int e = -1, tk = 0;
      if (sidx < total) {
        const unsigned short c = chains[sidx];
        e = c & 0xff;
        tk = c >> 8;
      }
      // shared-memory byte offsets of the eight 16-byte units of this chain's two rows inside a buffer (swizzled)
      uint32_t wo[8], xo[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        wo[q] = (uint32_t)(e >= 0 ? e : 0) * 128u + (((uint32_t)q ^ (uint32_t)(e & 7)) << 4);
        xo[q] = (uint32_t)tk * 128u + (((uint32_t)q ^ (uint32_t)(tk & 7)) << 4);
      }
      const uint32_t w_base = smem_u32(w_stage), x_base = smem_u32(x_stage);
      if (producer)  // (after a wait that ran out nothing more is issued: a buffer may still be in flight)
        for (int ch = 0; ch < kRfBufs - 1 && ch < nchunk && !failed; ++ch) issue(ch);
      float acc = 0.0f;
      for (int ch = 0; ch < nchunk; ++ch) {
        if (producer && !failed && ch + kRfBufs - 1 < nchunk) issue(ch + kRfBufs - 1);
        const int b = consumed % kRfBufs;
        // one lane per warp polls the barrier (a thousand pollers would keep the shared-memory pipe busy)
        if (lane == 0 && !failed && !mbar_wait(smem_u32(&s_full[b]), (uint32_t)(consumed / kRfBufs) & 1u, abort_flag, wait_ns)) {
          failed = true;
          s_abort = 1;
        }
        failed = __shfl_sync(0xffffffffu, (int)failed, 0) != 0;
        ++consumed;
        if (e >= 0 && !failed) {
          const uint32_t wb = w_base + (uint32_t)b * (uint32_t)kRfWBytes, xb = x_base + (uint32_t)b * (uint32_t)kXBytes;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const uint4 xa = lds128(xb + xo[q]);
            const uint4 wa = lds128(wb + wo[q]);
            acc = __fmaf_rn(bf16_lo(xa.x), bf16_lo(wa.x), acc);
            acc = __fmaf_rn(bf16_hi(xa.x), bf16_hi(wa.x), acc);
            acc = __fmaf_rn(bf16_lo(xa.y), bf16_lo(wa.y), acc);
            acc = __fmaf_rn(bf16_hi(xa.y), bf16_hi(wa.y), acc);
            acc = __fmaf_rn(bf16_lo(xa.z), bf16_lo(wa.z), acc);
            acc = __fmaf_rn(bf16_hi(xa.z), bf16_hi(wa.z), acc);
            acc = __fmaf_rn(bf16_lo(xa.w), bf16_lo(wa.w), acc);
            acc = __fmaf_rn(bf16_hi(xa.w), bf16_hi(wa.w), acc);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&s_empty[b]));  // this warp has left the buffer
      }
      if (e >= 0 && !failed) {
        const float exact = bias != nullptr ? acc + bias[e] : acc;
        // the error model, checked where both values are at hand: a miss is an error of this kernel, said aloud
        if (!(fabsf(exact - ls[tk * kRfEP + e]) <= s_eps[tk])) set_status(status, MOE_ERR_INTERNAL, 501);
        ls[tk * kRfEP + e] = exact;
      }
    }
    __syncthreads();
    if (s_abort) break;  // (CTA-uniform: read after the barrier)
    // The K-th largest EXACT logit among the experts done so far.  An expert that is not done has l~ below the
    // threshold, hence l < thr + eps; if that is at most the K-th exact value, none of them belongs to the K
    // largest and the token is finished.  Otherwise the threshold drops to (K-th exact - eps), which is final:
    // more exact values can only raise the K-th one.
    unsigned tkn = 0;
    float kx = -FLT_MAX;
    for (int k = 0; k < K; ++k) {
      float bv = -FLT_MAX;
      int be = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int e = l16 + 16 * j;
        if (!((done >> j) & 1u) || ((tkn >> j) & 1u)) continue;
        const float xv = ls[tl * kRfEP + e];
        if (be == 0x7fffffff || xv > bv) { bv = xv; be = e; }
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oe = __shfl_xor_sync(0xffffffffu, be, off);
        const bool other = (oe != 0x7fffffff) && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be));
        if (other) { bv = ov; be = oe; }
      }
      if (be != 0x7fffffff && (be & 15) == l16) tkn |= 1u << (be >> 4);
      kx = bv;
    }
    thr = (live && thr + eps > kx) ? kx - eps : FLT_MAX;  // FLT_MAX: nothing more to do for this token
  }
  __syncthreads();
  if (s_abort) {
    // A copy that was waited for too long is still on its way: every issued copy has to land before the CTA's
    // shared memory goes away (bounded again; the copies depend on nobody).
    if (producer) {
      for (int g = 0; g < issued; ++g) {
        if (g + kRfBufs < issued) continue;  // an older fill of the same buffer: the later one's phase covers it
        const unsigned long long ts = globaltimer();
        while (!mbar_try(smem_u32(&s_full[g % kRfBufs]), (uint32_t)(g / kRfBufs) & 1u))
          if (globaltimer() - ts > wait_ns + 1000000ull) break;
      }
      set_status(status, MOE_ERR_TIMEOUT, kWaitMbarTma);
    }
    __syncthreads();
    return;
  }
  select_topk<kRfEP>(ls, tvalid, t0, E, K, renorm, topk_idx, topk_w, prep.hist ? s_hist : nullptr, tp);
  route_prep_end(prep, s_hist);
}

// ---- host side ----------------------------------------------------------------------------------------
bool route_filter_applies(const moe_plan* p) {
  return p->cfg.dtype == MOE_DTYPE_BF16 && p->route_E > 64 && p->route_E <= kRfEP && p->cfg.route_filter >= 0 &&
         p->s.route_logits != nullptr;
}

int launch_route_filter(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx, float* topk_w,
                        const PrepArgs& prep, cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  EncodeTiledFn enc;
  int rc = get_encoder(p, &enc);
  if (rc != MOE_OK) return rc;
  CUtensorMap mx, mw;
  if ((rc = make_map_2d(enc, &mx, x, (uint64_t)c.T, (uint64_t)c.H, kTileRows)) != MOE_OK) return rc;
  if ((rc = make_map_2d(enc, &mw, wr, (uint64_t)p->route_E, (uint64_t)c.H, kRfEP)) != MOE_OK) return rc;
  CUtensorMap mwh;  // half of the experts per box, for the filter's CTAs
  if ((rc = make_map_2d(enc, &mwh, wr, (uint64_t)p->route_E, (uint64_t)c.H, 128)) != MOE_OK) return rc;
  static SmemAttrOnce once;
  if (ensure_dynamic_smem(route_tc_logits_kernel, kTcSmem, p->device, once) != cudaSuccess) return MOE_ERR_CUDA;
  const unsigned long long wait_ns = c.wait_limit_ns ? c.wait_limit_ns : kDefaultWaitNs;
  const int grid_a = (c.T + kTileRows - 1) / kTileRows;
  // the first kernel of the layer is launched plainly (see launch_wide_tmt), the second one behind it
  if (launch_maybe_pdl(false, route_tc_logits_kernel, dim3(grid_a, (p->route_E + 127) / 128), dim3(kTcThreads), kTcSmem, st, mx, mwh,
                       (const __nv_bfloat16*)wr, c.T, c.H, p->route_E, p->s.route_logits, p->s.route_wnorm2, wait_ns,
                       p->s.status) != cudaSuccess)
    return MOE_ERR_CUDA;
  // Tokens per CTA: every CTA streams all of Wr once, so as many tokens as still fill the GPU with CTAs.
  static SmemAttrOnce once_b[3];
  auto refine = [&](auto kern, int tpc) -> int {
    CUtensorMap mxb;  // the tokens' rows of x, one CTA's worth per box
    int r = make_map_2d(enc, &mxb, x, (uint64_t)c.T, (uint64_t)c.H, (uint32_t)tpc);
    if (r != MOE_OK) return r;
    if (ensure_dynamic_smem(kern, rf_smem(tpc), p->device, once_b[tpc / 32]) != cudaSuccess) return MOE_ERR_CUDA;
    return launch_pdl(kern, dim3((c.T + tpc - 1) / tpc), dim3(tpc * 16), rf_smem(tpc), st, mw, mxb, (const __nv_bfloat16*)x, bias,
                      (const float*)p->s.route_logits, (const float*)p->s.route_wnorm2, c.T, c.H, p->route_E, p->route_K,
                      c.renormalize, topk_idx, topk_w, prep, p->tp, wait_ns, p->s.status) == cudaSuccess
               ? 0 : MOE_ERR_CUDA;
  };
  const int sms = p->sm_count > 0 ? p->sm_count : 148;
  if (c.T >= 48 * sms) rc = refine(route_refine_kernel<64>, 64);
  else if (c.T >= 24 * sms) rc = refine(route_refine_kernel<32>, 32);
  else rc = refine(route_refine_kernel<16>, 16);
  if (rc != 0) return rc;
  p->launches += 2;
  return 0;
}

}  // namespace moehub
