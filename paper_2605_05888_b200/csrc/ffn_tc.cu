// Step 3 of the MoE layer (paper Section II-A, expert computation: two GEMMs with an activation
// between them) for bf16 on the 5th-generation tensor cores: a persistent, warp-specialised grouped
// GEMM.  Operands are staged in shared memory by TMA (128-byte swizzle), tcgen05.mma accumulates
// 128 x 256 fp32 tiles in tensor memory, and the epilogue warps read them back with tcgen05.ld.
//
// The unit of work is what the paper's dependency table calls a thread-block group: one 128-row
// tile of one expert's receive region times one block of output columns (Section IV-D, static
// tiling).  Tiles nobody wrote to are not in the work list, so their experts' weights are never
// touched (Section IV-D: thread blocks whose counters stay at zero are never scheduled).
//
//   GEMM1 (SWIGLU): D[128, 256] = A[128, H] * [Wg[e, f0:f0+128, :] ; Wu[e, f0:f0+128, :]]^T
//                   inter[:, f0:f0+128] = bf16( silu(D[:, 0:128]) * D[:, 128:256] )
//   GEMM2         : D[128, 256] = inter[128, F] * Wd[e, h0:h0+256, :]^T ; out = bf16(D)
//
// A tile that is its expert's only one and holds at most 64 rows runs both GEMMs the other way
// round (D^T: 128 weight rows x the tile's rows rounded up to 16, two MMAs per 16 k for the two
// halves of the weight block; the epilogue stores transposed).
//
// Work order is expert-major, then column block, then tile, so that CTAs running at the same time
// share the weight block through L2 and an expert's rows stay L2-resident across its column blocks.
//
// Both GEMMs run in ONE persistent launch.  A GEMM2 item of a tile may start only when all column
// blocks of that tile's intermediate are written: the software form of the paper's data
// availability manager (Section IV-D) - a per-tile status counter bumped (release) by every
// epilogue warp that finished a GEMM1 block, and a consumer that waits (acquire, bounded) for the
// counter to reach its threshold before its TMA loads touch the tile.  The GEMM2 items of an expert
// are placed a few hundred items behind its GEMM1 items, so the wait is normally over before it
// starts.  The same kernel also runs the two GEMMs as two launches (phase 1 / phase 2).
//
// Roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (owns the TMEM allocation),
// warps 2-5 = epilogue (TMEM lane quarter = warp % 4).  Every wait is bounded in time; on expiry
// the CTA records MOE_ERR_TIMEOUT, drains its outstanding TMA copies (bounded), frees its TMEM and
// returns.
#include "dispatch_ordered.cuh"

namespace moehub {

// The producer side of the overlapped form: with ord.x != nullptr the launch has n_dispatch more CTAs than
// SMs; its first n_dispatch CTAs only run the ordered dispatch (dispatch_ordered.cuh) and leave, the others
// are consumers that start on a tile when its status counter reaches the number of rows the tile will hold
// (the last n_dispatch of them become resident as the producers leave).
struct OverlapParams {
  OrderedParams ord;
  int n_dispatch;
  int gate_all;  // consumers wait for the WHOLE dispatch (global counter) instead of their tile's counter
  int* hist_rw;  // [E] the row counts, cleared by the last CTA to leave
};

// ---- the grouped GEMM -----------------------------------------------------------------------
// Items are handed out dynamically: a CTA takes the next unclaimed item of the list, its first one
// included (one global atomicAdd per item, issued by the producer thread while the previous item's
// loads run), so CTAs whose items were short take more of them, and an item that another one waits
// for is never held by a CTA that has not started yet.  The producer
// publishes each item index (-1: no more) to the other roles through a ring in shared memory with one
// mbarrier per slot.  The producer is at most 4 items (one per pipeline stage) ahead of the MMA
// thread and that at most 2 (the accumulators) ahead of the epilogue, so 16 slots never wrap onto an
// unread one.
constexpr int kItemRing = 16;
struct TcShared {
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned long long item_bar[kItemRing];
  unsigned long long drain;  // the MMA thread's last commit when it gives up: nothing of its own is in flight after it
  int item_ring[kItemRing];
  uint32_t tmem_base;
  int abort_flag;
  int last_cta;
};

__global__ void __launch_bounds__(kTcThreads, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap map_a1, const __grid_constant__ CUtensorMap map_bg,
              const __grid_constant__ CUtensorMap map_bu, const __grid_constant__ CUtensorMap map_a2,
              const __grid_constant__ CUtensorMap map_bd, const __grid_constant__ CUtensorMap map_a1t,
              const __grid_constant__ CUtensorMap map_a2t, const FfnParams prm, const OverlapParams ov) {
  const int phase = prm.phase, E = prm.E, F = prm.F, H = prm.H;
  __nv_bfloat16* __restrict__ inter = prm.inter;
  __nv_bfloat16* __restrict__ out = prm.out;
  int* __restrict__ gemm1_done = prm.gemm1_done;
  const int* __restrict__ tile_count = prm.tile_count;
  const int* __restrict__ rows_done = prm.rows_done;
  const int total_rows = prm.total_rows;
  int* __restrict__ status = prm.status;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* stage_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  TcShared* sh = reinterpret_cast<TcShared*>(stage_base + kStages * kStageBytes);
  __shared__ __align__(16) WorkList wl;  // a producer CTA keeps the dispatch's bookkeeping (with its mbarriers) here first

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int nseg = 2 * E;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh->tmem_full[a]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[a]), 4);
    }
    for (int i = 0; i < kItemRing; ++i) mbar_init(smem_u32(&sh->item_bar[i]), 1);
    mbar_init(smem_u32(&sh->drain), 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // the MMA warp owns all 512 TMEM columns: two 128 x 256 fp32 accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                 "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();  // everything above needs no global data and overlaps the predecessor's tail
  const bool producer_cta = ov.ord.x != nullptr && (int)blockIdx.x < ov.n_dispatch;
  if (producer_cta) {
    // A producer CTA: dispatch this CTA's share of the token blocks.  The buffer ring is the stage area and the
    // dispatch's bookkeeping sits in the work list's place; every bulk copy has completed when the call
    // returns.  Afterwards the CTA takes no work item: it only goes through the common tear-down.
    __syncthreads();
    dispatch_ordered_cta<kTcThreads>(ov.ord, *reinterpret_cast<OrdShared*>(&wl), stage_base, (int)blockIdx.x, ov.n_dispatch);
    __syncthreads();
  }
  int* work_counter = prm.work_counter + (phase == 2 ? 1 : 0);
  int first_claim = 0;
  if (threadIdx.x == 0 && !producer_cta) first_claim = atomicAdd(work_counter, 1);  // in flight while the work list is built
  build_worklist(wl, prm.tile_expert, prm.P, E, (F + 127) / 128, (H + 255) / 256, prm.lag, prm.fused, 1, prm.hot_min,
                 prm.hist, prm.hot_first);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  volatile int* abort_flag = &sh->abort_flag;
  ClockProbe probe(prm.clock_probe);
  const unsigned long long wait_ns = prm.wait_ns;

  const int NB1 = (F + 127) / 128, NB2 = (H + 255) / 256;
  const int KB1 = (H + kBK - 1) / kBK, KB2 = (F + kBK - 1) / kBK;
  int item_begin = 0, item_end = wl.seg_start[nseg];
  if (phase == 1) item_end = wl.n1;
  if (phase == 2) item_begin = wl.n1;

  // Interleaving (two launches, skewed load): the launch's items are two runs, hot then cold (see
  // WorkList).  Claim number i is spread evenly over both: floor(i * n_cold / n) of the first i claims
  // are cold ones, so both runs are used up at the same pace and end together.
  const int n_hot = phase == 0 ? -1 : wl.n_hot[phase - 1];
  const long long n_cold = (long long)(item_end - item_begin) - n_hot;
  const long long n_all = item_end - item_begin;

  // item -> (type, expert, column block, tile); inside a segment column-block-major, tile-minor
  // Shared-memory reads are slow while the tensor pipe streams its operands from the same memory
  // (a microsecond for the nine dependent reads of a binary search, measured), so only the first
  // lookup is a search: a thread's items only move forward through each run of the segment list.
  int seg_cursor = -1, seg_cursor_cold = -1;
  auto decode = [&](int item) {
    bool cold = false;
    if (n_hot >= 0 && n_cold > 0) {
      const long long i = item - item_begin;
      const long long before = i * n_cold / n_all;
      cold = (i + 1) * n_cold / n_all > before;
      item = item_begin + (cold ? n_hot + (int)before : (int)(i - before));
    }
    int lo = cold ? seg_cursor_cold : seg_cursor;
    if (lo < 0) {  // largest segment whose first item is <= item
      int hi = nseg;
      lo = 0;
      while (hi - lo > 1) {
        const int mid = (lo + hi) / 2;
        if (wl.seg_start[mid] <= item) lo = mid; else hi = mid;
      }
    } else {
      while (wl.seg_start[lo + 1] <= item) ++lo;  // seg_start[nseg] is the item count, above every item
    }
    if (cold) seg_cursor_cold = lo; else seg_cursor = lo;
    Item it;
    it.type = wl.seg_info[lo] >> 16;
    it.e = wl.seg_info[lo] & 0xffff;
    const int m = wl.estart[it.e + 1] - wl.estart[it.e];
    it.m = m;
    it.cold = m < prm.cold_below;
    const int local = item - wl.seg_start[lo];
    if (prm.band > 0 && m > prm.band) {
      const int per_band = (it.type == 0 ? NB1 : NB2) * prm.band;  // every band but the last is full
      const int j = local / per_band, rem = local - j * per_band;
      const int bz = min(prm.band, m - j * prm.band);
      it.nb = rem / bz;
      it.tile = wl.tiles[wl.estart[it.e] + j * prm.band + rem % bz];
    } else {
      it.nb = local / m;
      it.tile = wl.tiles[wl.estart[it.e] + local % m];
    }
    return it;
  };
  volatile int* item_ring = sh->item_ring;

  int fail_site = 0;
  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase_bit = 0;
      int armed[kStages];
#pragma unroll
      for (int s = 0; s < kStages; ++s) armed[s] = 0;
      int item = item_begin + first_claim;
      const uint64_t pol_stream = l2_policy_evict_first();
      for (int local_item = 0; !fail_site; ++local_item) {
        const int slot = local_item & (kItemRing - 1);
        if (item >= item_end || producer_cta) {
          item_ring[slot] = -1;
          mbar_arrive(smem_u32(&sh->item_bar[slot]));
          break;
        }
        const int next_item = item_begin + atomicAdd(work_counter, 1);  // used after this item's loads
        const Item it = decode(item);
        if (it.tile < 0 || it.tile >= prm.P || it.e < 0 || it.e >= E) {  // own index check on what the work list gave
          set_status(status, MOE_ERR_INTERNAL, 201);
          fail_site = kWaitItem;
          break;
        }
        // Rows the tile will hold, when the work list was built from the experts' row counts: the threshold of
        // its status counter (a partly filled last tile is ready as soon as ITS rows have arrived).
        int tile_rows = -1;
        if (wl.count[it.e] >= 0) tile_rows = min(kTileRows, wl.count[it.e] - (it.tile - wl.estart[it.e]) * kTileRows);
        if (it.type == 0 && tile_count != nullptr && tile_rows >= 0 && ov.gate_all) {
          if (ld_acquire(rows_done) < total_rows) {
            const unsigned long long t0 = globaltimer();
            while (ld_acquire(rows_done) < total_rows) {
              if (*abort_flag || globaltimer() - t0 > wait_ns) { fail_site = kWaitTileReady; break; }
              __nanosleep(64);
            }
            if (fail_site) break;
          }
          asm volatile("fence.proxy.async.global;" ::: "memory");
        } else if (it.type == 0 && tile_count != nullptr && tile_rows >= 0) {
          if (ld_acquire(&tile_count[it.tile]) < tile_rows) {
            const unsigned long long t0 = globaltimer();
            while (ld_acquire(&tile_count[it.tile]) < tile_rows) {
              if (*abort_flag || globaltimer() - t0 > wait_ns) { fail_site = kWaitTileReady; break; }
              __nanosleep(64);
            }
            if (fail_site) break;
          }
          asm volatile("fence.proxy.async.global;" ::: "memory");
        } else if (it.type == 0 && tile_count != nullptr) {
          // Availability of this tile's rows (dispatch side): 128 rows stored, or every assignment of
          // the batch stored (then a partly filled tile is final).
          if (ld_acquire(&tile_count[it.tile]) < kTileRows && ld_acquire(rows_done) < total_rows) {
            const unsigned long long t0 = globaltimer();
            while (ld_acquire(&tile_count[it.tile]) < kTileRows && ld_acquire(rows_done) < total_rows) {
              if (*abort_flag || globaltimer() - t0 > wait_ns) { fail_site = kWaitTileReady; break; }
              __nanosleep(64);
            }
            if (fail_site) break;
          }
          asm volatile("fence.proxy.async.global;" ::: "memory");
        }
        if (it.type == 1) {
          // Availability of this tile's intermediate: every epilogue warp of every GEMM1 block bumps
          // the tile's counter once.  Bounded wait, then order the async proxy behind what was seen.
          const int need = 4 * NB1;
          if (ld_acquire(&gemm1_done[it.tile]) < need) {
            const unsigned long long t0 = globaltimer();
            while (ld_acquire(&gemm1_done[it.tile]) < need) {
              if (*abort_flag || globaltimer() - t0 > wait_ns) { fail_site = kWaitTileReady; break; }
              __nanosleep(64);
            }
            if (fail_site) break;
          }
          asm volatile("fence.proxy.async.global;" ::: "memory");
        }
        // The only tile of an expert with at most 64 rows is computed the other way round: the weight rows
        // are the M side of the MMA and the tile's rows, rounded up to 16, the N side, so the MMA work and
        // the row operand shrink with the rows instead of staying those of 128.  Such an expert's weights
        // are used once, so its items are bound by streaming them, and the narrow form helps (C3 -3.6 %,
        // C4 -4 %); the short last tile of an expert with several tiles stays in the normal form: its
        // weights come from L2, and eight small MMAs per k-block took as long as four full ones
        // (measured: the clock rose 6 %, the step time did not fall).  Such a tile runs the normal form on
        // its first 64 rows only (M = 64 MMAs, the same count of instructions at half the work each: under the
        // power cap the Phi-like layer and C3 gain 1.5 %).  The row count is final here: the tile was
        // declared ready above (GEMM1) or long ago (GEMM2).
        unsigned long long* trace = prm.item_ns ? prm.item_ns + 4 * (size_t)item : nullptr;
        int n16 = 0;
        if (tile_count != nullptr) {
          const int r = tile_rows >= 0 ? tile_rows : tile_count[it.tile];
          if (r <= kThinRows && it.m == 1 && prm.thin) n16 = max(1, (r + 15) / 16);
          else if (r <= kThinRows) n16 = kHalfForm;  // the short last tile of a larger expert: M = 64 MMAs
        }
        item_ring[slot] = item | (n16 << kThinShift);
        mbar_arrive(smem_u32(&sh->item_bar[slot]));  // release: the slot is written before the phase completes
        if (trace) {
          unsigned smid;
          asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
          trace[0] = globaltimer();
          trace[2] = (unsigned long long)it.type | ((unsigned long long)it.cold << 1) | ((unsigned long long)n16 << 2) |
                     ((unsigned long long)it.e << 8) | ((unsigned long long)it.nb << 24) |
                     ((unsigned long long)it.tile << 32) | ((unsigned long long)smid << 52);
        }
        const CUtensorMap* ma = it.type == 0 ? (n16 ? &map_a1t : &map_a1) : (n16 ? &map_a2t : &map_a2);
        const uint32_t stage_tx = n16 ? (uint32_t)(kThinRows * kBK * 2 + kBBytes) : (uint32_t)kStageBytes;
        const int KB = it.type == 0 ? KB1 : KB2;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(smem_u32(&sh->empty[stage]), phase_bit ^ 1u, abort_flag, wait_ns)) { fail_site = kWaitMbarTma; break; }
          const uint32_t full = smem_u32(&sh->full[stage]);
          const uint32_t a_dst = smem_u32(stage_base + stage * kStageBytes);
          const uint32_t b_dst = a_dst + kABytes;
          mbar_expect_tx(full, stage_tx);
          tma_load_2d(a_dst, ma, full, kb * kBK, it.tile * kTileRows);
          if (it.cold) {  // weights that are read this once: first in line for eviction from L2
            if (it.type == 0) {
              tma_load_3d_hint(b_dst, &map_bg, full, kb * kBK, it.nb * 128, it.e, pol_stream);
              tma_load_3d_hint(b_dst + kBBytes / 2, &map_bu, full, kb * kBK, it.nb * 128, it.e, pol_stream);
            } else {
              tma_load_4d_hint(b_dst, &map_bd, full, kb * kBK, it.nb * 256, it.e % prm.tp, it.e / prm.tp, pol_stream);
            }
          } else if (it.type == 0) {
            tma_load_3d(b_dst, &map_bg, full, kb * kBK, it.nb * 128, it.e);
            tma_load_3d(b_dst + kBBytes / 2, &map_bu, full, kb * kBK, it.nb * 128, it.e);
          } else {
            tma_load_4d(b_dst, &map_bd, full, kb * kBK, it.nb * 256, it.e % prm.tp, it.e / prm.tp);
          }
#pragma unroll
          for (int s = 0; s < kStages; ++s)
            if (s == stage) armed[s] += 1;
          if (++stage == kStages) { stage = 0; phase_bit ^= 1u; }
        }
        if (trace) trace[3] = globaltimer();  // every load of the item issued
        item = next_item;
      }
      if (fail_site || *abort_flag) {
        // Leave no copy in flight: wait (bounded) for the last fill of every stage.
        sh->abort_flag = 1;
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
          if (armed[s] == 0) continue;
          const uint32_t par = (uint32_t)((armed[s] - 1) & 1);
          const unsigned long long t0 = globaltimer();
          while (!mbar_try(smem_u32(&sh->full[s]), par))
            if (globaltimer() - t0 > wait_ns) break;
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      int stage = 0;
      uint32_t phase_bit = 0;
      for (int local_item = 0; !fail_site; ++local_item) {
        const int slot = local_item & (kItemRing - 1);
        if (!mbar_wait(smem_u32(&sh->item_bar[slot]), (uint32_t)(local_item / kItemRing) & 1u, abort_flag, wait_ns)) { fail_site = kWaitItem; break; }
        const int entry = item_ring[slot];
        if (entry < 0) break;
        const int item = entry & ((1 << kThinShift) - 1), n16 = entry >> kThinShift;
        const Item it = decode(item);
        const int KB = it.type == 0 ? KB1 : KB2;
        const int acc = local_item & 1;
        const uint32_t acc_phase = (uint32_t)(local_item >> 1) & 1u;
        if (!mbar_wait(smem_u32(&sh->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, wait_ns)) { fail_site = kWaitMbarTmemFree; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kUmmaN);
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(smem_u32(&sh->full[stage]), phase_bit, abort_flag, wait_ns)) { fail_site = kWaitMbarMma; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(stage_base + stage * kStageBytes);
          const uint64_t adesc = smem_desc_sw128(a_addr);
          const uint64_t bdesc = smem_desc_sw128(a_addr + kABytes);
          if (n16 == 0 || n16 == kHalfForm) {
            const uint32_t idesc = n16 == 0 ? kIdesc : kIdescHalf;  // 128 or 64 rows of the tile
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)  // 16 k-elements = 32 bytes = 2 descriptor units per step
              tc_mma(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          } else {
            // thin tile: D[128 weight rows, 16*n16 tile rows], once per half of the weight block (gate / up,
            // or the two 128-row halves of the Wd block), into accumulator columns 0.. and 128..
            const uint32_t idesc = thin_idesc(n16);
            const uint64_t wdesc2 = smem_desc_sw128(a_addr + kABytes + kBBytes / 2);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k) {
              tc_mma(d_tmem, bdesc + 2 * k, adesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
              tc_mma(d_tmem + 128, wdesc2 + 2 * k, adesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            }
          }
          tc_commit(smem_u32(&sh->empty[stage]));  // the stage is free once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase_bit ^= 1u; }
        }
        if (fail_site) break;
        tc_commit(smem_u32(&sh->tmem_full[acc]));  // accumulator complete
      }
      if (fail_site) sh->abort_flag = 1;
      if (fail_site || *abort_flag) {
        // Giving up with MMAs possibly still running: they read the stages and write tensor memory, so wait
        // (bounded) for all of them before the CTA frees either.
        tc_commit(smem_u32(&sh->drain));
        const unsigned long long t0 = globaltimer();
        while (!mbar_try(smem_u32(&sh->drain), 0u))
          if (globaltimer() - t0 > wait_ns + 1000000ull) break;
      }
    }
  } else {
    // ===================== epilogue =====================
    const int quarter = warp & 3;  // TMEM lanes this warp may read
    // 32-byte stores need every row start on a 32-byte boundary
    const bool wide1 = F % 16 == 0 && (reinterpret_cast<uintptr_t>(inter) & 31) == 0;
    const bool wide2 = H % 16 == 0 && (reinterpret_cast<uintptr_t>(out) & 31) == 0;
    const int row_in_tile = quarter * 32 + lane;
    for (int local_item = 0; !fail_site; ++local_item) {
      const int slot = local_item & (kItemRing - 1);
      if (!mbar_wait(smem_u32(&sh->item_bar[slot]), (uint32_t)(local_item / kItemRing) & 1u, abort_flag, wait_ns)) { fail_site = kWaitItem; break; }
      const int entry = item_ring[slot];
      if (entry < 0) break;
      const int item = entry & ((1 << kThinShift) - 1), n16 = entry >> kThinShift;
      const Item it = decode(item);
      const int acc = local_item & 1;
      const uint32_t acc_phase = (uint32_t)(local_item >> 1) & 1u;
      if (!mbar_wait(smem_u32(&sh->tmem_full[acc]), acc_phase, abort_flag, wait_ns, 500)) { fail_site = kWaitMbarEpi; break; }
      tc_fence_after();
      if (prm.item_ns && warp == 2 && lane == 0) prm.item_ns[4 * (size_t)item + 1] = globaltimer();  // MMAs complete
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kUmmaN);
      size_t row = (size_t)it.tile * kTileRows + row_in_tile;
      bool row_live = true;
      if (n16 == kHalfForm) {
        // An M = 64 accumulator keeps 16 rows in each quadrant of the 128 lanes: row r sits in lane
        // 32 * (r / 16) + r % 16 (checked against the oracle; rows in lanes 0-63 is not the layout).
        row_live = lane < 16;
        row = (size_t)it.tile * kTileRows + quarter * 16 + lane;
      }
      if (n16 != 0 && n16 != kHalfForm) {
        // thin tile: this lane owns a weight row (an F or H column of the result), the accumulator's
        // columns are the tile's rows; a warp's 32 lanes write 64 contiguous bytes of one output row.
        const size_t row0 = (size_t)it.tile * kTileRows;
        if (it.type == 0) {
          const int f = it.nb * 128 + row_in_tile;
#pragma unroll 1
          for (int c = 0; c < 16 * n16; c += 16) {
            uint32_t g[16], u[16];
            tc_ld16(t_row + c, g);
            tc_ld16(t_row + 128 + c, u);
            tc_wait_ld();
            if (f < F) {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                inter[(row0 + c + i) * F + f] = __float2bfloat16_rn(silu_mul(__uint_as_float(g[i]), __uint_as_float(u[i])));
            }
          }
        } else {
#pragma unroll 1
          for (int half = 0; half < 2; ++half) {
            const int h = it.nb * 256 + half * 128 + row_in_tile;
#pragma unroll 1
            for (int c = 0; c < 16 * n16; c += 16) {
              uint32_t v[16];
              tc_ld16(t_row + half * 128 + c, v);
              tc_wait_ld();
              if (h < H) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  long long orow = (long long)(row0 + c + i);
                  if (prm.push_src != nullptr) {  // the row's own token position; anything else (a stale word after a
                    orow = __ldcg(prm.push_src + row0 + c + i);  // dispatch that gave up) is no position
                    if (orow >= total_rows) orow = -1;
                  }
                  if (orow >= 0) out[(size_t)orow * H + h] = __float2bfloat16_rn(__uint_as_float(v[i]));
                }
              }
            }
          }
        }
      } else if (it.type == 0) {
        __nv_bfloat16* dst = inter + row * F + (size_t)it.nb * 128;
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
          if (!row_live) continue;
          if (wide1 && c + 16 <= ncols) {
            st_global_32B(dst + c, Vec16<__nv_bfloat16>::pack(s), Vec16<__nv_bfloat16>::pack(s + 8));
          } else {
            if (c + 8 <= ncols) *reinterpret_cast<uint4*>(dst + c) = Vec16<__nv_bfloat16>::pack(s);
            if (c + 16 <= ncols) *reinterpret_cast<uint4*>(dst + c + 8) = Vec16<__nv_bfloat16>::pack(s + 8);
          }
        }
      } else {
        // Push-style combine (paper Section IV-B, all-to-all combine): the expert reads the row's source
        // information after its final GEMM and stores the result straight to the token's position.
        if (prm.push_src != nullptr) {
          const int src = __ldcg(prm.push_src + row);
          if (src < 0 || src >= total_rows) row_live = false;  // an empty slot (or no position at all): nothing to return
          else row = (size_t)src;
        }
        __nv_bfloat16* dst = out + row * H + (size_t)it.nb * 256;
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
          if (!row_live) continue;
          if (wide2 && c + 32 <= ncols) {
            st_global_32B(dst + c, Vec16<__nv_bfloat16>::pack(f), Vec16<__nv_bfloat16>::pack(f + 8));
            st_global_32B(dst + c + 16, Vec16<__nv_bfloat16>::pack(f + 16), Vec16<__nv_bfloat16>::pack(f + 24));
          } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (c + 8 * q + 8 <= ncols) *reinterpret_cast<uint4*>(dst + c + 8 * q) = Vec16<__nv_bfloat16>::pack(f + 8 * q);
          }
        }
      }
      tc_fence_before();
      if (it.type == 0) {
        // This warp's part of the block is written: make it visible (also to the async proxy, which
        // is how the GEMM2 producer will read it) and bump the tile's status counter.
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&sh->tmem_empty[acc]));
        if (it.type == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(gemm1_done + it.tile) : "memory");
      }
    }
    if (fail_site) sh->abort_flag = 1;
  }
  if (fail_site) set_status(status, MOE_ERR_TIMEOUT, fail_site);

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_trigger();
  probe.finish();
  if (threadIdx.x == 0) {
    // Every CTA has taken its last item index by now; the last one to leave puts the counters back to
    // zero, so a launch never depends on the host having cleared them.
    int* exit_counter = work_counter + 2;
    const bool last = atomicAdd(exit_counter, 1) == (int)gridDim.x - 1;
    if (last) {
      *work_counter = 0;
      *exit_counter = 0;
    }
    sh->last_cta = last ? 1 : 0;
  }
  __syncthreads();
  if (sh->last_cta && phase != 1) {
    // The last CTA of the launch that ran the GEMM2 items: every wait on the per-tile GEMM1 counters is
    // over, so they go back to zero too.  A later call on the same tiles (another set of weights on one
    // dispatch result) then waits for ITS OWN GEMM1 blocks instead of finding the old counts.
    for (int pt = threadIdx.x; pt < prm.P; pt += kTcThreads) gemm1_done[pt] = 0;
  }
  if (sh->last_cta && ov.ord.x != nullptr) {
    // the launch that carried the dispatch: every CTA has read the row counts; clear them for the next call
    for (int e = threadIdx.x; e < E; e += kTcThreads) ov.hist_rw[e] = 0;
  }
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// ---- host side ------------------------------------------------------------------------------
// bf16 tensor [E, rows, cols], box [1, box_rows, 64].
static int make_map_3d(EncodeTiledFn enc, CUtensorMap* m, const void* base, uint64_t E, uint64_t rows, uint64_t cols,
                       uint32_t box_rows) {
  cuuint64_t dims[3] = {cols, rows, E};
  cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
  cuuint32_t box[3] = {(cuuint32_t)kBK, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MOE_OK : MOE_ERR_CUDA;
}

OrderedParams make_ordered_params(moe_plan* p, const void* x, const int* topk_idx, void* recv, int* expert_count,
                                  int* tile_expert, int* src_info, int* slot_of, int* tile_count, int* rows_done);

// overlap_x / overlap_idx != nullptr: the overlapped form - the launch that runs the GEMM1 items also
// dispatches x (ordered scheme, into recv and the plan's own dispatch outputs) on its first CTAs.
// The down matrices [E, H, F*tp] seen as [E, tp, H, F]: shard s of an expert is the column slice [s*F, (s+1)*F).
// Box [1, 1, box_rows, 64].
static int make_map_wd(EncodeTiledFn enc, CUtensorMap* m, const void* base, uint64_t experts, uint64_t tp, uint64_t rows,
                       uint64_t cols, uint32_t box_rows) {
  cuuint64_t dims[4] = {cols, rows, tp, experts};
  cuuint64_t strides[3] = {cols * tp * 2, cols * 2, rows * cols * tp * 2};
  cuuint32_t box[4] = {(cuuint32_t)kBK, box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MOE_OK : MOE_ERR_CUDA;
}

int launch_ffn_tc(moe_plan* p, const void* recv, const int* tile_expert, const void* wg, const void* wu,
                  const void* wd, void* out_rows, const int* tile_count, const int* rows_done, cudaStream_t st,
                  const void* overlap_x, const int* overlap_idx, const int* push_src) {
  const moe_config_t& c = p->cfg;
  if (p->P == 0 || c.T == 0) return 0;
  EncodeTiledFn enc;
  int rc = get_encoder(p, &enc);
  if (rc != MOE_OK) return rc;
  const uint64_t pool_rows = (uint64_t)p->P * kTileRows;
  CUtensorMap a1, bg, bu, a2, bd;
  if ((rc = make_map_2d(enc, &a1, recv, pool_rows, c.H, kTileRows)) != MOE_OK) return rc;
  if ((rc = make_map_3d(enc, &bg, wg, c.E, c.F, c.H, 128)) != MOE_OK) return rc;
  if ((rc = make_map_3d(enc, &bu, wu, c.E, c.F, c.H, 128)) != MOE_OK) return rc;
  if ((rc = make_map_2d(enc, &a2, p->s.inter, pool_rows, c.F, kTileRows)) != MOE_OK) return rc;
  if (c.ffn_kernel == 2) {  // the pair kernel: 3-D map, no TP shards
    if (p->tp != 1) return MOE_ERR_UNSUPPORTED;
    if ((rc = make_map_3d(enc, &bd, wd, c.E, c.H, c.F, 128)) != MOE_OK) return rc;
  } else if ((rc = make_map_wd(enc, &bd, wd, c.E / p->tp, p->tp, c.H, c.F, 256)) != MOE_OK) {
    return rc;
  }
  CUtensorMap a1t, a2t;  // the first kThinRows rows of a tile, for tiles computed the other way round
  if ((rc = make_map_2d(enc, &a1t, recv, pool_rows, c.H, kThinRows)) != MOE_OK) return rc;
  if ((rc = make_map_2d(enc, &a2t, p->s.inter, pool_rows, c.F, kThinRows)) != MOE_OK) return rc;

  static SmemAttrOnce once;
  if (ensure_dynamic_smem(ffn_tc_kernel, kTcSmem, p->device, once) != cudaSuccess) return MOE_ERR_CUDA;
  const int grid = p->sm_count;
  const int NB1 = (c.F + 127) / 128, NB2 = (c.H + 255) / 256;
  // One launch for both GEMMs, or one per GEMM.  With many small experts (E = 256 under Zipf routing)
  // the single launch measures 2-3 % slower than two, also with items handed out dynamically, so the
  // default splits there.
  const int fused = c.ffn_split == 2 ? 1 : (c.ffn_split == 1 ? 0 : (c.E <= 64 ? 1 : 0));
  const bool pairs = c.ffn_kernel == 2;  // opt-in: the CTA-pair kernel
  if (pairs && push_src != nullptr) return MOE_ERR_UNSUPPORTED;
  const int workers = pairs ? grid / 2 : grid;
  if (p->P > kMaxListTiles) return MOE_ERR_UNSUPPORTED;  // the work list lives in the kernel's shared memory
  if ((long long)p->P * (NB1 + NB2) >= (1ll << kThinShift)) return MOE_ERR_UNSUPPORTED;  // item index field of the ring
  // The one-CTA kernel puts its counters back to zero itself; the pair kernel has static item assignment
  // and no last-one-out step, so its GEMM1 counters are cleared here (also for a call without counters,
  // which no dispatch preceded).
  if ((tile_count == nullptr || pairs) &&
      cudaMemsetAsync(p->s.gemm1_done, 0, sizeof(int) * (size_t)(p->P + 4), st) != cudaSuccess)
    return MOE_ERR_CUDA;
  mark(p, 3, st);
  FfnParams prm;
  prm.tile_expert = tile_expert;
  prm.P = (int)p->P;
  prm.lag = 2 * workers;
  prm.fused = fused;
  // Interleaving (opt-in, two-launch form only).  Measured on the DeepSeek-like layer it changes nothing:
  // every kind of item there takes 57-75 us whether the kinds are mixed or not, because none of them is
  // bound by HBM bandwidth alone.
  prm.hot_min = (fused || pairs || c.ffn_hot_min_tiles <= 0) ? 0 : c.ffn_hot_min_tiles;
  prm.cold_below = prm.hot_min > 0 ? prm.hot_min : 3;
  prm.thin = c.ffn_thin_tiles >= 0;
  prm.tp = p->tp;
  prm.E = c.E;
  prm.F = c.F;
  prm.H = c.H;
  prm.inter = (__nv_bfloat16*)p->s.inter;
  prm.out = (__nv_bfloat16*)out_rows;
  prm.gemm1_done = p->s.gemm1_done;
  prm.work_counter = p->s.gemm1_done + p->P;
  prm.tile_count = tile_count;
  prm.rows_done = rows_done;
  prm.wait_ns = c.wait_limit_ns ? c.wait_limit_ns : kDefaultWaitNs;
  prm.total_rows = c.T * c.K;
  prm.status = p->s.status;
  prm.clock_probe = reinterpret_cast<unsigned long long*>(p->s.clock_probe);
  prm.item_ns = (p->trace && !pairs) ? p->s.item_ns : nullptr;
  prm.hist = nullptr;
  prm.hot_first = 0;
  prm.band = 0;
  prm.push_src = push_src;
  OverlapParams ov = {};
  const bool overlap = overlap_x != nullptr && !pairs;
  if (overlap) {
    Scratch& s = p->s;
    ov.ord = make_ordered_params(p, overlap_x, overlap_idx, s.recv, s.expert_count, s.tile_expert, s.src_info, s.slot_of,
                                 s.tile_count, s.rows_done);
    ov.ord.ring_bytes = kStages * kStageBytes;
    // Producer CTAs: enough of them to keep HBM busy with the row copies (half of the SMs move about 85 % of
    // what all of them do), the rest start on expert tiles at once.
    ov.gate_all = c.overlap < 0 ? 1 : 0;
    ov.n_dispatch = c.overlap > 1 ? min(c.overlap, grid - 1) : grid / 2;
    ov.n_dispatch = max(1, min(ov.n_dispatch, ov.ord.nblk));
    ov.hist_rw = s.hist;
  }
  auto launch = [&](int phase) -> int {
    prm.phase = phase;
    if (pairs) return launch_ffn_tc2_kernel(a1, bg, bu, a2, bd, prm, grid, st);
    OverlapParams ovp = {};
    if (overlap && phase != 2) {
      // The launch that carries the dispatch: its work list comes from the row counts (no tile owner is
      // written yet), hottest experts first.  One CTA per SM and CTAs start in index order, so the producer
      // CTAs (the lowest indices) are resident before any consumer waits for their rows; a consumer's wait is
      // bounded in any case.
      ovp = ov;
      prm.hist = p->s.hist;
      prm.hot_first = 1;
      // Bands re-read an expert's gate and up matrices once per band: only where they stay in L2 meanwhile
      // (58.7 MB on the DeepSeek-like layer; the Mixtral-like layer's 235 MB would be streamed again and again).
      prm.band = (size_t)2 * c.F * c.H * 2 <= ((size_t)64 << 20) ? 4 : 0;
      return launch_pdl(ffn_tc_kernel, dim3(grid + ov.n_dispatch), dim3(kTcThreads), kTcSmem, st, a1, bg, bu, a2, bd, a1t, a2t, prm,
                        ovp) == cudaSuccess ? 0 : MOE_ERR_CUDA;
    }
    prm.hist = nullptr;
    prm.hot_first = 0;
    prm.band = 0;
    return launch_pdl(ffn_tc_kernel, dim3(grid), dim3(kTcThreads), kTcSmem, st, a1, bg, bu, a2, bd, a1t, a2t, prm, ovp) == cudaSuccess
               ? 0 : MOE_ERR_CUDA;
  };
  if (fused) {
    if ((rc = launch(0)) != 0) return rc;
    mark(p, 4, st);  // timed runs: the whole launch is booked on the GEMM1 stage, the GEMM2 stage is empty
    p->launches += 1;
  } else {
    if ((rc = launch(1)) != 0) return rc;
    mark(p, 4, st);
    if ((rc = launch(2)) != 0) return rc;
    p->launches += 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : MOE_ERR_CUDA;
}

}  // namespace moehub
