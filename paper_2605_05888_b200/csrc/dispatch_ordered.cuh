// Destination-agnostic dispatch as a persistent, token-ordered producer (dispatch mode 3).
//
// Paper hooks.  Section IV-B: a row is sent as soon as its expert id is known and the consumer side hands
// out the next free row of the expert's region (allocation pointer table, RowPointer).  Section IV-C: the
// packet scheduler sends the smallest RowID first, so that whole rows - and with them whole tiles -
// complete early instead of all at the end.  Section IV-D: every stored row raises the status counter of
// the thread-block group that depends on it; the group is released when the counter reaches its
// threshold.
//
// What this file does with them.  A fixed set of CTAs walks the token blocks in ONE global ascending
// order (CTA w takes blocks w, w + n, w + 2n, ...), so LocalRowIDs are handed out in near token order and
// tile i of an expert is complete once its first 128 (i + 1) rows have been emitted.  The experts' row
// counts are known when the kernel starts (the router, or a counting pass, left them in hist[E]), so the
// region of expert e is the run of tiles [tile_base[e], tile_base[e + 1]) of the pool, tile_base being the
// exclusive scan of ceil(hist[e] / 128) that every CTA computes for itself: no tile table, no wait for
// another CTA anywhere in the dispatch.  Only the order of rows inside a region is decided at run time,
// by one aggregated atomicAdd per touched expert per token block.
//
// Rows move with plain bulk asynchronous copies (global to shared and back, no tensor map): one thread per
// CTA loads a row (or a 16 KB chunk of it) into a ring of shared-memory buffers and stores it from there
// to each of its K slots; the copies do not depend on resident warps or registers, loads run a few units
// ahead of the stores, and up to 8 x K row stores are in flight per CTA.  A second warp raises the
// availability counters: a row is counted as stored (red.release on its tile's counter) once the copy
// thread has seen its bulk stores complete.  (The copy thread must not do this itself: a release, or a
// proxy fence, issued by the thread that has bulk stores in flight waits for all of them, and the copy
// pipeline then runs at 3.3 instead of 5.5 TB/s.)  The remaining warps do the index work of the next
// token blocks and stage the slots in shared memory.
#pragma once
#include "tc_common.cuh"

namespace moehub {

constexpr int kOrdRingMax = 24;     // most chunk buffers per CTA; as many as fit into kOrdRingBytes are used
constexpr int kOrdRingBytes = 192 * 1024;
constexpr int kOrdStoreSlack = 4;   // buffers not holding a load in flight: loads run (ring - 4) units ahead of the stores
constexpr int kOrdMaxLag = 32;      // most units whose stores may be awaiting completion (see signal lag below)
constexpr int kOrdChunk = 16384;    // largest chunk of a row that is moved in one piece (bytes)
constexpr int kOrdSlotRing = 12;    // token blocks whose slots may be staged at the same time
constexpr int kOrdMaxAssign = 128;  // assignments (token, k) per token block
static_assert(kOrdStoreSlack - 1 == 3, "the wait_group.read immediate below follows this");
__host__ __device__ inline int ord_buf_bytes(int row_bytes) { return ((row_bytes < kOrdChunk ? row_bytes : kOrdChunk) + 127) & ~127; }
__host__ __device__ inline int ord_ring(int row_bytes, int ring_bytes = kOrdRingBytes) {
  const int r = ring_bytes / ord_buf_bytes(row_bytes);
  return r > kOrdRingMax ? kOrdRingMax : (r < kOrdStoreSlack + 1 ? kOrdStoreSlack + 1 : r);
}

// cp.async.bulk.wait_group takes an immediate: at most n of this thread's bulk groups still pending.
__device__ __forceinline__ void bulk_wait_group(int n) {
  switch (n) {
#define MOEHUB_WG(N) case N: asm volatile("cp.async.bulk.wait_group " #N ";" ::: "memory"); break;
    MOEHUB_WG(0) MOEHUB_WG(1) MOEHUB_WG(2) MOEHUB_WG(3) MOEHUB_WG(4) MOEHUB_WG(5) MOEHUB_WG(6) MOEHUB_WG(7)
    MOEHUB_WG(8) MOEHUB_WG(9) MOEHUB_WG(10) MOEHUB_WG(11) MOEHUB_WG(12) MOEHUB_WG(13) MOEHUB_WG(14) MOEHUB_WG(15)
    MOEHUB_WG(16) MOEHUB_WG(17) MOEHUB_WG(18) MOEHUB_WG(19) MOEHUB_WG(20) MOEHUB_WG(21) MOEHUB_WG(22) MOEHUB_WG(23)
    MOEHUB_WG(24) MOEHUB_WG(25) MOEHUB_WG(26) MOEHUB_WG(27) MOEHUB_WG(28) MOEHUB_WG(29) MOEHUB_WG(30) MOEHUB_WG(31)
    default: asm volatile("cp.async.bulk.wait_group 32;" ::: "memory"); break;
#undef MOEHUB_WG
  }
}

struct OrderedParams {
  const uint8_t* x;        // [T, row_bytes]
  const int* topk_idx;     // [T, K]
  int T, E, K, P;
  int row_bytes;           // H * element size, a multiple of 16
  int tok_per_blk, nblk;
  int ring_bytes;          // shared memory the caller gave to the buffer ring
  const int* hist;         // [E] rows per expert, complete before the kernel starts
  int* row_pointer;        // [E] next free LocalRowID per expert, zero at the start
  uint8_t* recv;           // [P * 128, row_bytes]
  int* src_info;           // [P * 128]
  int* slot_of;            // [T, K]
  int* expert_count;       // [E]  written by worker 0
  int* tile_expert;        // [P]  written by worker 0
  int* tile_count;         // [P]  rows stored per tile (zero at the start)
  int* rows_done;          // [1]
  int* status;
  unsigned long long* avail_ns;  // availability trace or nullptr
  unsigned long long wait_ns;    // bound on every wait
};

struct OrdShared {
  unsigned long long load_full[kOrdRingMax];
  unsigned long long slot_full[kOrdSlotRing];
  unsigned long long slot_free[kOrdSlotRing];
  int slots[kOrdSlotRing][kOrdMaxAssign];
  int tile_base[kMaxExperts + 1];
  int cnt[kMaxExperts];
  int base[kMaxExperts];
  int done_units;   // units whose stores the copy thread has seen complete (read by the signalling warp)
  int abort_flag;   // set by whichever role gave up; ends the other roles' waits early
  int index_abort;  // written by index thread 0 only, read by all index threads after a barrier (uniform decision)
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

// Exclusive scan of the experts' tile counts, by warp 0; every thread of the CTA must call (it synchronises).
__device__ __forceinline__ void ordered_tile_base(int* tile_base, const int* __restrict__ hist, int E) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int c[kMaxExperts / 32], sum = 0;
#pragma unroll
    for (int i = 0; i < kMaxExperts / 32; ++i) {
      const int e = lane * (kMaxExperts / 32) + i;
      c[i] = e < E ? (hist[e] + kTileRows - 1) / kTileRows : 0;
      sum += c[i];
    }
    int incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += n;
    }
    int run = incl - sum;
#pragma unroll
    for (int i = 0; i < kMaxExperts / 32; ++i) {
      const int e = lane * (kMaxExperts / 32) + i;
      if (e < E) tile_base[e] = run;
      run += c[i];
    }
    if (lane == 31) tile_base[E] = incl;
  }
  __syncthreads();
}

// Walks units (token block, token, chunk) of one worker in order.
struct OrdCursor {
  int q, blk, tl, c;  // local block number, global block, token inside the block, chunk inside the row
  __device__ __forceinline__ void init(int worker) { q = 0; blk = worker; tl = 0; c = 0; }
  __device__ __forceinline__ int ntok(const OrderedParams& p) const { return min(p.tok_per_blk, p.T - blk * p.tok_per_blk); }
  __device__ __forceinline__ void advance(const OrderedParams& p, int nchunk, int n_workers) {
    if (++c < nchunk) return;
    c = 0;
    if (++tl < ntok(p)) return;
    tl = 0;
    ++q;
    blk += n_workers;
  }
};

// The dispatch of one worker CTA.  All NT threads of the CTA call it; ring: ord_ring(row_bytes) buffers of
// ord_buf_bytes(row_bytes) bytes, 128-byte aligned, in shared memory.
// Returns false if a bounded wait ran out (status is set).
template <int NT>
__device__ __forceinline__ bool dispatch_ordered_cta(const OrderedParams& p, OrdShared& sh, uint8_t* ring, int worker,
                                                     int n_workers) {
  constexpr int NI = NT - 64;  // index threads: warps 2 ..
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kOrdRingMax; ++i) mbar_init(smem_u32(&sh.load_full[i]), 1);
    for (int i = 0; i < kOrdSlotRing; ++i) {
      mbar_init(smem_u32(&sh.slot_full[i]), 1);
      mbar_init(smem_u32(&sh.slot_free[i]), 1);
    }
    sh.abort_flag = 0;
    sh.index_abort = 0;
    sh.done_units = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (p.avail_ns != nullptr) atomicMin(p.avail_ns, globaltimer());
  }
  ordered_tile_base(sh.tile_base, p.hist, p.E);  // synchronises the CTA
  volatile int* abort_flag = &sh.abort_flag;
  const int nchunk = (p.row_bytes + kOrdChunk - 1) / kOrdChunk;
  const int buf_bytes = ord_buf_bytes(p.row_bytes);
  const int ring_n = ord_ring(p.row_bytes, p.ring_bytes), load_ahead = ring_n - kOrdStoreSlack;
  int my_blocks = 0, my_units = 0, my_assign = 0;
  for (int blk = worker; blk < p.nblk; blk += n_workers) {
    const int nt = min(p.tok_per_blk, p.T - blk * p.tok_per_blk);
    ++my_blocks;
    my_units += nt * nchunk;
    my_assign += nt * p.K;
  }
  int fail = 0;

  if (warp == 0) {
    // ===================== copy engine: one thread =====================
    if (lane == 0) {
      OrdCursor cl, cs;  // load and store cursors
      cl.init(worker);
      cs.init(worker);
      volatile int* done_units = &sh.done_units;
      auto chunk_bytes = [&](int c) { return min(kOrdChunk, p.row_bytes - c * kOrdChunk); };
      // Signal lag: a unit is reported complete `lag` units after its stores were issued.  Completion of a
      // store takes microseconds, so the stores in flight must add up to several hundred KB (small rows or
      // few copies per token: more units), and the slots of all those units must still be staged.
      const int unit_store_bytes = max(1, p.K * min(p.row_bytes, kOrdChunk));
      int lag = (640 * 1024 + unit_store_bytes - 1) / unit_store_bytes;
      lag = max(6, min(lag, min(kOrdMaxLag, (kOrdSlotRing - 3) * p.tok_per_blk * nchunk)));
      int signalled = 0, loaded = 0, stored = 0;
      for (int step = 0; step < my_units + load_ahead && !fail; ++step) {
        if (step < my_units) {  // (A) load unit `step`
          const int b = step % ring_n;
          // the buffer's last occupant was unit step - ring, stored at step - 4: at most the 3 groups after it may still be reading
          if (step >= ring_n) asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
          const uint32_t bytes = (uint32_t)chunk_bytes(cl.c);
          const uint32_t bar = smem_u32(&sh.load_full[b]);
          const int tok = cl.blk * p.tok_per_blk + cl.tl;
          if (tok < 0 || tok >= p.T || (size_t)(b + 1) * buf_bytes > (size_t)p.ring_bytes) {  // own index check: never read outside x or the ring
            set_status(p.status, MOE_ERR_INTERNAL, 101);
            fail = kWaitMbarTma;
            break;
          }
          mbar_expect_tx(bar, bytes);
          bulk_load(smem_u32(ring + (size_t)b * buf_bytes), p.x + (size_t)tok * p.row_bytes + (size_t)cl.c * kOrdChunk, bytes, bar);
          cl.advance(p, nchunk, n_workers);
          ++loaded;
        }
        const int v = step - load_ahead;
        if (v >= 0) {  // (B) store unit v to the token's K slots
          const int b = v % ring_n;
          if (cs.tl == 0 && cs.c == 0 &&
              !mbar_wait(smem_u32(&sh.slot_full[cs.q % kOrdSlotRing]), (uint32_t)(cs.q / kOrdSlotRing) & 1u, abort_flag, p.wait_ns)) {
            fail = kWaitItem;
            break;
          }
          if (!mbar_wait(smem_u32(&sh.load_full[b]), (uint32_t)(v / ring_n) & 1u, abort_flag, p.wait_ns)) { fail = kWaitMbarTma; break; }
          const int* slots = sh.slots[cs.q % kOrdSlotRing] + cs.tl * p.K;
          const uint32_t src = smem_u32(ring + (size_t)b * buf_bytes);
          const uint32_t bytes = (uint32_t)chunk_bytes(cs.c);
          for (int k = 0; k < p.K; ++k) {
            const int slot = slots[k];
            if (slot >= p.P * kTileRows) {  // own index check: never store outside the pool
              set_status(p.status, MOE_ERR_INTERNAL, 102);
              continue;
            }
            if (slot >= 0) bulk_store(p.recv + (size_t)slot * p.row_bytes + (size_t)cs.c * kOrdChunk, src, bytes);
          }
          bulk_commit();  // group number v (empty if every assignment of the token was dropped)
          cs.advance(p, nchunk, n_workers);
          ++stored;
          if (v >= lag) {  // (C) group v - lag and all older ones are complete: tell the signalling warp
            bulk_wait_group(lag);
            asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(&sh.done_units)), "r"(++signalled) : "memory");
          }
        }
      }
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // bulk copies complete on their own: not a wait on anyone
      if (!fail) {
        asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(&sh.done_units)), "r"(my_units) : "memory");
      } else {
        sh.abort_flag = 1;
        // loads in flight must land before the buffers go away: wait (bounded) for those not yet consumed
        for (int u = stored; u < loaded; ++u) {
          const unsigned long long t0 = globaltimer();
          while (!mbar_try(smem_u32(&sh.load_full[u % ring_n]), (uint32_t)(u / ring_n) & 1u))
            if (globaltimer() - t0 > 1000000ull) break;
        }
      }
    }
  } else if (warp == 1) {
    // ===================== signalling: lane k raises the counter of the tile that holds the token's k-th row =====================
    OrdCursor cg;
    cg.init(worker);
    int seen = 0;
    for (int u = 0; u < my_units && !fail; ++u) {
      if (seen <= u) {
        const unsigned long long t0 = globaltimer();
        for (;;) {
          asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(seen) : "r"(smem_u32(&sh.done_units)) : "memory");
          if (seen > u) break;
          if (*abort_flag || globaltimer() - t0 > p.wait_ns) { fail = kWaitItem; break; }
          __nanosleep(200);
        }
        fail = __shfl_sync(0xffffffffu, fail, 0);  // lanes may read the clock differently: lane 0 decides
        seen = __shfl_sync(0xffffffffu, seen, 0);
        if (fail) break;
        // One fence for every unit reported since the last look (the rows were written by the async proxy, seen
        // complete by the copy thread, and that knowledge reached this warp through done_units); the counter
        // updates that follow are relaxed: fence + relaxed atomic is a release, and a fence per row would cost
        // most of a microsecond each.
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
      }
      if (cg.c == nchunk - 1) {  // the token's last chunk: its rows are complete
        const int slot = lane < p.K ? sh.slots[cg.q % kOrdSlotRing][cg.tl * p.K + lane] : -1;
        if (slot >= 0) {
          int* ctr = p.tile_count + slot / kTileRows;
          if (p.avail_ns == nullptr) {
            asm volatile("red.relaxed.gpu.global.add.s32 [%0], 1;" ::"l"(ctr) : "memory");
          } else {
            int old;
            asm volatile("atom.relaxed.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(ctr) : "memory");
            if (old + 1 == kTileRows) p.avail_ns[2 + slot / kTileRows] = globaltimer();
          }
        }
        __syncwarp();
        if (cg.tl == cg.ntok(p) - 1 && lane == 0) mbar_arrive(smem_u32(&sh.slot_free[cg.q % kOrdSlotRing]));  // the block's slots are no longer needed
      }
      cg.advance(p, nchunk, n_workers);
    }
    if (!fail && lane == 0) {
      if (p.avail_ns == nullptr) {
        asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p.rows_done), "r"(my_assign) : "memory");
      } else {
        int old;
        asm volatile("atom.release.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p.rows_done), "r"(my_assign) : "memory");
        if (old < p.T * p.K && old + my_assign >= p.T * p.K) p.avail_ns[1] = globaltimer();
      }
    }
    if (fail) sh.abort_flag = 1;
  } else {
    // ===================== index workers =====================
    const int ti = threadIdx.x - 64;
    if (worker == 0) {
      // what does not depend on arrival order: counts, tile owners, and the source info of slots that stay empty
      for (int e = ti; e < p.E; e += NI) {
        const int c = p.hist[e];
        p.expert_count[e] = c;
        const int first = sh.tile_base[e], last = sh.tile_base[e + 1];
        for (int t = first; t < last; ++t) p.tile_expert[t] = e;
        for (int r = c; r < (last - first) * kTileRows; ++r) p.src_info[(size_t)first * kTileRows + r] = -1;
      }
      for (int t = sh.tile_base[p.E] + ti; t < p.P; t += NI) p.tile_expert[t] = -1;
      for (long long s = (long long)sh.tile_base[p.E] * kTileRows + ti; s < (long long)p.P * kTileRows; s += NI) p.src_info[s] = -1;
    }
    int q = 0;
    for (int blk = worker; blk < p.nblk && !fail; blk += n_workers, ++q) {
      const int sidx = q % kOrdSlotRing;
      // Only one thread waits (bounded) for the slot buffer and every index thread reads its verdict after the
      // barrier, so that all of them leave the loop together (a named barrier has no time limit).
      if (q >= kOrdSlotRing && ti == 0 &&
          !mbar_wait(smem_u32(&sh.slot_free[sidx]), (uint32_t)(q / kOrdSlotRing - 1) & 1u, abort_flag, p.wait_ns))
        sh.index_abort = 1;
      const int t0 = blk * p.tok_per_blk;
      const int na = min(p.tok_per_blk, p.T - t0) * p.K;
      for (int e = ti; e < p.E; e += NI) sh.cnt[e] = 0;
      asm volatile("bar.sync 1, %0;" ::"n"(NI) : "memory");
      if (sh.index_abort) {
        fail = kWaitItem;
        break;
      }
      int e = -1, lrank = 0;
      if (ti < na) {
        e = p.topk_idx[(size_t)t0 * p.K + ti];
        if (e < 0 || e >= p.E) {  // not an expert: reported, dropped
          set_status(p.status, MOE_ERR_ARG, t0 + ti / p.K);
          e = -1;
        }
      }
      {  // rank inside the block: warp-aggregated shared-memory atomics
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        const int leader = __ffs(peers) - 1;
        int base = 0;
        if (e >= 0 && lane == leader) base = atomicAdd(&sh.cnt[e], __popc(peers));
        base = __shfl_sync(0xffffffffu, base, leader);
        lrank = base + __popc(peers & ((1u << lane) - 1u));
      }
      asm volatile("bar.sync 1, %0;" ::"n"(NI) : "memory");
      // one global atomicAdd per touched expert: the block's rows get LocalRowIDs [base, base + n)
      for (int ee = ti; ee < p.E; ee += NI) {
        const int n = sh.cnt[ee];
        if (n != 0) sh.base[ee] = atomicAdd(&p.row_pointer[ee], n);
      }
      asm volatile("bar.sync 1, %0;" ::"n"(NI) : "memory");
      if (ti < na) {
        int slot = -1;
        if (e >= 0) {
          const int local_row = sh.base[e] + lrank;
          // address = Base + LocalRowID * RowSize, Base = the expert's first tile
          if (local_row < (sh.tile_base[e + 1] - sh.tile_base[e]) * kTileRows) slot = sh.tile_base[e] * kTileRows + local_row;
          else set_status(p.status, MOE_ERR_OVERFLOW, e);  // the counts did not describe this topk_idx
        }
        sh.slots[sidx][ti] = slot;
        p.slot_of[(size_t)t0 * p.K + ti] = slot;
        if (slot >= 0) p.src_info[slot] = t0 * p.K + ti;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(NI) : "memory");
      if (ti == 0) mbar_arrive(smem_u32(&sh.slot_full[sidx]));
    }
    if (fail) sh.abort_flag = 1;
  }
  if (fail) set_status(p.status, MOE_ERR_TIMEOUT, fail);
  __syncthreads();
  return sh.abort_flag == 0;
}

}  // namespace moehub
