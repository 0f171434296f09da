// Expert FFN on CTA pairs (paper Section II-A, expert computation; per-tile availability gating as in
// Section IV-D): the cta_group::2 form of the persistent grouped GEMM in ffn_tc.cu.
//
// Why pairs.  With one CTA per tile every 64-wide k-block needs 48 KB of operands per SM for 512
// tensor-pipe cycles, more than the L2 -> SM path sustains; the tensor pipe then idles a quarter of
// the time.  A pair of CTAs (a cluster of two SMs) computes a 256 x 256 accumulator from two 128-row
// tiles of the same expert: each CTA stages its own tile (16 KB) and only HALF of the weight block
// (16 KB), and tcgen05.mma.cta_group::2, issued by the leader CTA alone, reads both halves out of both
// CTAs' shared memory.  32 KB per k-block per SM, six stages in flight.
//
//   GEMM1: the leader stages gate rows Wg[e, f0:f0+128, :], the peer stages up rows Wu[e, f0:f0+128, :];
//          accumulator columns 0-127 are gate, 128-255 up, in each CTA for its own 128 rows.
//   GEMM2: the leader stages Wd[e, h0:h0+128, :], the peer Wd[e, h0+128:h0+256, :].
//
// An expert with an odd number of tiles leaves the peer of its last pair without a tile: that CTA
// stages the pair's first tile again (valid memory) and stores nothing.
//
// Every CTA loads its own bytes with plain per-CTA TMA loads.  Synchronisation: per stage, a "full"
// barrier in the leader (two arrivals + 64 KB of transactions, both CTAs' TMA loads signal it) and an
// "empty" barrier in each CTA (the leader's tcgen05.commit arrives on both); per accumulator, a "full"
// barrier in each CTA (commit to both) and an "empty" barrier in the leader that all eight epilogue
// warps of the pair arrive on.  Every wait is bounded in time.
#include "tc_common.cuh"

namespace moehub {

constexpr int kStages2 = 6;
constexpr int kBHalfBytes = 128 * kBK * 2;                 // 16 KB: this CTA's half of the weight block
constexpr int kStageBytes2 = kABytes + kBHalfBytes;        // 32 KB
constexpr int kTcSmem2 = kStages2 * kStageBytes2 + 1024 + 256;
// Instruction descriptor: bf16 x bf16 -> fp32, A and B K-major, M = 256 (two CTAs x 128), N = 256.
constexpr uint32_t kIdesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) |
                             ((uint32_t)(256 >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c0, int c1,
                                             int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tc2_commit_both(uint32_t bar) {  // arrives on `bar` in both CTAs of the pair
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc2_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

struct Tc2Shared {
  unsigned long long full[kStages2];   // used in the leader
  unsigned long long empty[kStages2];  // used in each CTA
  unsigned long long tmem_full[2];     // used in each CTA
  unsigned long long tmem_empty[2];    // used in the leader
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTcThreads, 1)
ffn_tc2_kernel(const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_bg,
               const __grid_constant__ CUtensorMap map_bu, const __grid_constant__ CUtensorMap map_a2,
               const __grid_constant__ CUtensorMap map_bd, const FfnParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* stage_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Tc2Shared* sh = reinterpret_cast<Tc2Shared*>(stage_base + kStages2 * kStageBytes2);
  __shared__ WorkList wl;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int E = prm.E, F = prm.F, H = prm.H;
  const int nseg = 2 * E;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages2; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 2);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh->tmem_full[a]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[a]), 8);
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // the same warp of both CTAs allocates: 512 columns in each CTA's TMEM
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                 "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  pdl_wait();  // everything above needs no global data and overlaps the predecessor's tail
  build_worklist(wl, prm.tile_expert, prm.P, E, (F + 127) / 128, (H + 255) / 256, prm.lag, prm.fused, 2);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  volatile int* abort_flag = &sh->abort_flag;
  ClockProbe probe(prm.clock_probe);
  const unsigned long long wait_ns = prm.wait_ns;

  const int NB1 = (F + 127) / 128, NB2 = (H + 255) / 256;
  const int KB1 = (H + kBK - 1) / kBK, KB2 = (F + kBK - 1) / kBK;
  int item_begin = 0, item_end = wl.seg_start[nseg];
  if (prm.phase == 1) item_end = wl.n1;
  if (prm.phase == 2) item_begin = wl.n1;
  const int n_clusters = gridDim.x / 2;
  const int first_item = item_begin + blockIdx.x / 2;

  // item -> (type, expert, column block, this CTA's tile); it.tile < 0: this CTA has no tile of its
  // own in the pair and `fill` names the tile it stages instead.
  auto decode = [&](int item, int& fill) {
    int lo = 0, hi = nseg;
    while (hi - lo > 1) {
      const int mid = (lo + hi) / 2;
      if (wl.seg_start[mid] <= item) lo = mid; else hi = mid;
    }
    Item it;
    it.type = wl.seg_info[lo] >> 16;
    it.e = wl.seg_info[lo] & 0xffff;
    const int m = wl.estart[it.e + 1] - wl.estart[it.e];  // tiles of the expert
    const int pairs = (m + 1) / 2;
    const int local = item - wl.seg_start[lo];
    it.nb = local / pairs;
    const int j = local % pairs;
    const int base = wl.estart[it.e] + 2 * j;
    fill = wl.tiles[base];
    it.tile = (2 * j + (int)rank < m) ? wl.tiles[base + rank] : -1;
    if (it.tile >= 0) fill = it.tile;
    return it;
  };

  int fail_site = 0;
  if (warp == 0) {
    // ===================== TMA producer (both CTAs) =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase_bit = 0;
      bool issued = false;
      for (int item = first_item; item < item_end && !fail_site; item += n_clusters) {
        int fill;
        const Item it = decode(item, fill);
        if (it.tile >= 0 && it.type == 0 && prm.tile_count != nullptr) {
          if (ld_acquire(&prm.tile_count[it.tile]) < kTileRows && ld_acquire(prm.rows_done) < prm.total_rows) {
            const unsigned long long t0 = globaltimer();
            while (ld_acquire(&prm.tile_count[it.tile]) < kTileRows && ld_acquire(prm.rows_done) < prm.total_rows) {
              if (*abort_flag || globaltimer() - t0 > wait_ns) { fail_site = kWaitTileReady; break; }
              __nanosleep(64);
            }
            if (fail_site) break;
          }
          asm volatile("fence.proxy.async.global;" ::: "memory");
        }
        if (it.tile >= 0 && it.type == 1) {
          const int need = 4 * NB1;
          if (ld_acquire(&prm.gemm1_done[it.tile]) < need) {
            const unsigned long long t0 = globaltimer();
            while (ld_acquire(&prm.gemm1_done[it.tile]) < need) {
              if (*abort_flag || globaltimer() - t0 > wait_ns) { fail_site = kWaitTileReady; break; }
              __nanosleep(64);
            }
            if (fail_site) break;
          }
          asm volatile("fence.proxy.async.global;" ::: "memory");
        }
        const CUtensorMap* ma = it.type == 0 ? &map_a1 : &map_a2;
        const CUtensorMap* mb = it.type == 0 ? (leader ? &map_bg : &map_bu) : &map_bd;
        const int b_row = it.type == 0 ? it.nb * 128 : it.nb * 256 + (int)rank * 128;
        const int KB = it.type == 0 ? KB1 : KB2;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(smem_u32(&sh->empty[stage]), phase_bit ^ 1u, abort_flag, wait_ns)) { fail_site = kWaitMbarTma; break; }
          const uint32_t full_leader = map_to_cta(smem_u32(&sh->full[stage]), 0);
          const uint32_t a_dst = smem_u32(stage_base + stage * kStageBytes2);
          mbar_expect_tx_cluster(full_leader, kStageBytes2);
          tma2_load_2d(a_dst, ma, full_leader, kb * kBK, fill * kTileRows);
          tma2_load_3d(a_dst + kABytes, mb, full_leader, kb * kBK, b_row, it.e);
          issued = true;
          if (++stage == kStages2) { stage = 0; phase_bit ^= 1u; }
        }
      }
      if (fail_site || *abort_flag) {
        sh->abort_flag = 1;
        if (issued) {  // give copies in flight time to land before this CTA's shared memory goes away
          const unsigned long long t0 = globaltimer();
          while (globaltimer() - t0 < 200000ull) __nanosleep(1000);
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (leader CTA only) =====================
    if (leader && lane == 0) {
      int stage = 0;
      uint32_t phase_bit = 0;
      int local_item = 0;
      for (int item = first_item; item < item_end && !fail_site; item += n_clusters, ++local_item) {
        int fill;
        const Item it = decode(item, fill);
        const int KB = it.type == 0 ? KB1 : KB2;
        const int acc = local_item & 1;
        const uint32_t acc_phase = (uint32_t)(local_item >> 1) & 1u;
        if (!mbar_wait(smem_u32(&sh->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, wait_ns)) { fail_site = kWaitMbarTmemFree; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kUmmaN);
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(smem_u32(&sh->full[stage]), phase_bit, abort_flag, wait_ns)) { fail_site = kWaitMbarMma; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(stage_base + stage * kStageBytes2);
          const uint64_t adesc = smem_desc_sw128(a_addr);
          const uint64_t bdesc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            tc2_mma(d_tmem, adesc + 2 * k, bdesc + 2 * k, kIdesc2, (kb | k) != 0 ? 1u : 0u);
          tc2_commit_both(smem_u32(&sh->empty[stage]));  // both CTAs may refill this stage
          if (++stage == kStages2) { stage = 0; phase_bit ^= 1u; }
        }
        if (fail_site) break;
        tc2_commit_both(smem_u32(&sh->tmem_full[acc]));  // both CTAs' accumulators complete
      }
      if (fail_site) sh->abort_flag = 1;
    }
  } else {
    // ===================== epilogue (both CTAs, own 128 rows) =====================
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    int local_item = 0;
    for (int item = first_item; item < item_end && !fail_site; item += n_clusters, ++local_item) {
      int fill;
      const Item it = decode(item, fill);
      const int acc = local_item & 1;
      const uint32_t acc_phase = (uint32_t)(local_item >> 1) & 1u;
      if (!mbar_wait(smem_u32(&sh->tmem_full[acc]), acc_phase, abort_flag, wait_ns, 500)) { fail_site = kWaitMbarEpi; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kUmmaN);
      if (it.tile >= 0) {
        const size_t row = (size_t)it.tile * kTileRows + row_in_tile;
        if (it.type == 0) {
          __nv_bfloat16* dst = prm.inter + row * F + (size_t)it.nb * 128;
          const int ncols = min(128, F - it.nb * 128);
#pragma unroll 1
          for (int c = 0; c < 128; c += 16) {
            uint32_t g[16], u[16];
            tc_ld16(t_row + c, g);
            tc_ld16(t_row + 128 + c, u);
            tc_wait_ld();
            float s[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float gv = __uint_as_float(g[i]);
              s[i] = silu_mul(gv, __uint_as_float(u[i]));
            }
            if (c + 8 <= ncols) *reinterpret_cast<uint4*>(dst + c) = Vec16<__nv_bfloat16>::pack(s);
            if (c + 16 <= ncols) *reinterpret_cast<uint4*>(dst + c + 8) = Vec16<__nv_bfloat16>::pack(s + 8);
          }
        } else {
          __nv_bfloat16* dst = prm.out + row * H + (size_t)it.nb * 256;
          const int ncols = min(256, H - it.nb * 256);
#pragma unroll 1
          for (int c = 0; c < 256; c += 32) {
            uint32_t r0[16], r1[16];
            tc_ld16(t_row + c, r0);
            tc_ld16(t_row + c + 16, r1);
            tc_wait_ld();
            float f[32];
#pragma unroll
            for (int i = 0; i < 16; ++i) { f[i] = __uint_as_float(r0[i]); f[16 + i] = __uint_as_float(r1[i]); }
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (c + 8 * q + 8 <= ncols) *reinterpret_cast<uint4*>(dst + c + 8 * q) = Vec16<__nv_bfloat16>::pack(f + 8 * q);
          }
        }
      }
      tc_fence_before();
      if (it.tile >= 0 && it.type == 0) {
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_cluster(map_to_cta(smem_u32(&sh->tmem_empty[acc]), 0));  // the leader owns this barrier
        if (it.tile >= 0 && it.type == 0)
          asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(prm.gemm1_done + it.tile) : "memory");
      }
    }
    if (fail_site) sh->abort_flag = 1;
  }
  if (fail_site) set_status(prm.status, MOE_ERR_TIMEOUT, fail_site);

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while its partner may still touch its shared memory or TMEM
  tc_fence_after();
  pdl_trigger();
  probe.finish();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

int launch_ffn_tc2_kernel(const CUtensorMap& a1, const CUtensorMap& bg, const CUtensorMap& bu, const CUtensorMap& a2,
                          const CUtensorMap& bd, const FfnParams& prm, int grid, cudaStream_t st) {
  static SmemAttrOnce once;
  int device = -1;
  cudaGetDevice(&device);
  if (ensure_dynamic_smem(ffn_tc2_kernel, kTcSmem2, device, once) != cudaSuccess) return MOE_ERR_CUDA;
  return launch_pdl(ffn_tc2_kernel, dim3(grid & ~1), dim3(kTcThreads), kTcSmem2, st, a1, bg, bu, a2, bd, prm) ==
                 cudaSuccess ? 0 : MOE_ERR_CUDA;
}

}  // namespace moehub
