// Step 2 of the MoE layer (paper Section II-A, dispatch) with both address-resolution schemes.
//
// Mode 0, the conventional software mediation (Section III-A): per token-block histogram ->
// exclusive scan over (expert, block) and over experts (tile-padded) -> stable scatter.  Three
// kernels, and no row moves before every count is known.  The layout is the canonical one: an
// expert's rows are in (token, k) order.
//
// Modes 1/2, destination-agnostic (Section IV-A/IV-B): one kernel.  As soon as a token block
// knows its expert ids it takes rows from the experts' row pointers with one aggregated atomicAdd
// per touched expert (the software stand-in of the allocation pointer table's self-incrementing
// RowPointer) and stores each row at Base + LocalRowID*RowSize.  Mode 1 gives every expert a
// static region (the paper's conservative pre-allocation); mode 2 pages 128-row tiles out of one
// pool on demand (the paging-style manager the paper allows behind rowspMalloc): the block whose
// rows open a new tile takes it from the pool and publishes it in the expert's tile table, the
// others look it up with a bounded wait.
//
// Row movement is the same in every mode: one warp per token reads the row once with 16-byte
// vectors (several in flight per lane) and stores it to its K slots; the slot indices are staged
// in shared memory first so the copy loop has no dependent index loads.
#include "dispatch_ordered.cuh"

namespace moehub {

constexpr int kDispThreads = 256;
constexpr int kMaxAssign = 256;  // assignments (token,k pairs) per CTA

// ------------------------------------------------------------------------------------------------
// Row copy: the block's rows are cut into runs of 32*UNROLL 16-byte vectors; the warps take runs
// round-robin, so a block with a single token still uses all its warps.  A run is read once and
// stored to the token's K slots.
template <int UNROLL>
__device__ __forceinline__ void copy_rows(const uint4* __restrict__ x, uint4* __restrict__ recv,
                                          const int* s_slot, int t0, int ntok, int K, int vec_per_row) {
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  constexpr int RUN = 32 * UNROLL;
  const int runs = (vec_per_row + RUN - 1) / RUN;
  for (int u = warp; u < ntok * runs; u += kDispThreads / 32) {
    const int tl = u / runs, v0 = (u % runs) * RUN;
    const uint4* src = x + (size_t)(t0 + tl) * vec_per_row;
    const int* slots = s_slot + tl * K;
    uint4 r[UNROLL];
#pragma unroll
    for (int i = 0; i < UNROLL; ++i) {
      const int v = v0 + i * 32 + lane;
      if (v < vec_per_row) r[i] = __ldg(src + v);
    }
    for (int k = 0; k < K; ++k) {
      const int slot = slots[k];
      if (slot < 0) continue;
      uint4* dst = recv + (size_t)slot * vec_per_row;
#pragma unroll
      for (int i = 0; i < UNROLL; ++i) {
        const int v = v0 + i * 32 + lane;
        if (v < vec_per_row) __stcs(dst + v, r[i]);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Availability signalling (the software form of the paper's data availability manager, Section
// IV-D): after a block's rows are stored, every 128-row tile it wrote into gets its status counter
// raised by the number of rows (release), and the global counter by the block's assignments.  A
// consumer may read a tile once its counter shows 128 rows, or once the global counter shows all
// T*K assignments (partly filled last tiles are then final; tiles at zero never become work).
// With avail_ns given (measurement only) the counters are raised with atomics that return the old value,
// and the thread that completes a tile, or the batch, writes the time: avail_ns[0] earliest start of a
// dispatch CTA, [1] the moment the global counter reached all T*K assignments, [2 + tile] the moment the
// tile's counter reached 128 (0: the tile never filled).
__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void signal_rows(const int* s_slot, int na, int* __restrict__ tile_count,
                                            int* __restrict__ rows_done, unsigned long long* __restrict__ avail_ns,
                                            int total_rows) {
  asm volatile("fence.proxy.async.global;" ::: "memory");  // consumers read the rows through TMA
  __threadfence();
  __syncthreads();
  const int a = threadIdx.x;
  const int slot = a < na ? s_slot[a] : -1;
  const int tile = slot >= 0 ? slot / kTileRows : -1;
  const unsigned peers = __match_any_sync(0xffffffffu, tile);
  const bool first = tile >= 0 && (threadIdx.x % 32) == __ffs(peers) - 1;
  if (avail_ns == nullptr) {
    if (first)
      asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(tile_count + tile), "r"(__popc(peers)) : "memory");
    if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(rows_done), "r"(na) : "memory");
    return;
  }
  if (first) {
    int old;
    const int n = __popc(peers);
    asm volatile("atom.release.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(tile_count + tile), "r"(n) : "memory");
    if (old < kTileRows && old + n >= kTileRows) avail_ns[2 + tile] = now_ns();
  }
  if (threadIdx.x == 0) {
    int old;
    asm volatile("atom.release.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(rows_done), "r"(na) : "memory");
    if (old < total_rows && old + na >= total_rows) avail_ns[1] = now_ns();
  }
}

// ------------------------------------------------------------------------------------------------
// Mode 0, kernel 1: histogram of one token block.  cta_count[blk][e].
__global__ void __launch_bounds__(kDispThreads)
hist_kernel(const int* __restrict__ topk_idx, int T, int E, int K, int tok_per_blk,
            int* __restrict__ cta_count, int* __restrict__ status, unsigned long long* __restrict__ avail_ns) {
  extern __shared__ int s_cnt[];  // [E]
  for (int e = threadIdx.x; e < E; e += kDispThreads) s_cnt[e] = 0;
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  if (avail_ns != nullptr && threadIdx.x == 0) atomicMin(avail_ns, now_ns());
  const int t0 = blockIdx.x * tok_per_blk;
  const int na = min(tok_per_blk, T - t0) * K;
  for (int a = threadIdx.x; a < na; a += kDispThreads) {
    const int e = topk_idx[(size_t)t0 * K + a];
    if (e >= 0 && e < E) atomicAdd(&s_cnt[e], 1);
    else set_status(status, MOE_ERR_ARG, t0 + a / K);  // an expert id outside [0, E): the assignment is dropped
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += kDispThreads) cta_count[(size_t)blockIdx.x * E + e] = s_cnt[e];
}

// Mode 0, kernel 2: CTA e scans expert e's per-block counts (exclusive) -> cta_base[blk][e] and
// expert_count[e]; the last CTA to finish scans ceil(count/128) over the experts -> tile_base,
// tile_expert.
__global__ void __launch_bounds__(kDispThreads)
scan_kernel(const int* __restrict__ cta_count, int nblk, int E, int P, int* __restrict__ cta_base,
            int* __restrict__ expert_count, int* __restrict__ tile_base, int* __restrict__ tile_expert,
            int* __restrict__ ticket) {
  __shared__ int s_warp[kDispThreads / 32];
  __shared__ int s_carry;
  __shared__ int s_last;
  const int e = blockIdx.x;
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  if (threadIdx.x == 0) s_carry = 0;
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  for (int b0 = 0; b0 < nblk; b0 += kDispThreads) {
    const int b = b0 + threadIdx.x;
    const int c = (b < nblk) ? cta_count[(size_t)b * E + e] : 0;
    int incl = c;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int wbase = 0;
    for (int w = 0; w < warp; ++w) wbase += s_warp[w];
    const int carry = s_carry;
    if (b < nblk) cta_base[(size_t)b * E + e] = carry + wbase + incl - c;
    __syncthreads();
    if (threadIdx.x == kDispThreads - 1) s_carry = carry + wbase + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    expert_count[e] = s_carry;
    __threadfence();
    s_last = (atomicAdd(ticket, 1) == E - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // Exclusive scan of tiles-per-expert over the experts (E <= 256: one element per thread).
  int tiles = 0;
  if (threadIdx.x < E) tiles = (ld_acquire(&expert_count[threadIdx.x]) + kTileRows - 1) / kTileRows;
  int incl = tiles;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += n;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  int wbase = 0;
  for (int w = 0; w < warp; ++w) wbase += s_warp[w];
  const int first = wbase + incl - tiles;
  if (threadIdx.x < E) {
    tile_base[threadIdx.x] = first;
    for (int i = 0; i < tiles; ++i)
      if (first + i < P) tile_expert[first + i] = threadIdx.x;
  }
  if (threadIdx.x == E - 1) tile_base[E] = first + tiles;
}

// Mode 0, kernel 3: stable scatter.  The rank of an assignment inside its block is the number of
// earlier assignments (in (token,k) order) of the same expert.
__global__ void __launch_bounds__(kDispThreads)
scatter_kernel(const uint4* __restrict__ x, const int* __restrict__ topk_idx, int T, int E, int K,
               int tok_per_blk, int vec_per_row, const int* __restrict__ cta_base,
               const int* __restrict__ tile_base, uint4* __restrict__ recv, int* __restrict__ src_info,
               int* __restrict__ slot_of, int* __restrict__ tile_count, int* __restrict__ rows_done,
               unsigned long long* __restrict__ avail_ns) {
  extern __shared__ int smem_i[];
  int* s_wcnt = smem_i;                          // [8][E] per-warp counts
  int* s_slot = smem_i + (kDispThreads / 32) * E;  // [kMaxAssign]
  const int t0 = blockIdx.x * tok_per_blk;
  const int ntok = min(tok_per_blk, T - t0);
  const int na = ntok * K;
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  for (int i = threadIdx.x; i < (kDispThreads / 32) * E; i += kDispThreads) s_wcnt[i] = 0;
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  if (avail_ns != nullptr && threadIdx.x == 0) atomicMin(avail_ns, now_ns());
  const int a = threadIdx.x;  // one assignment per thread, na <= 256
  int e = -1, wrank = 0;
  if (a < na) e = topk_idx[(size_t)t0 * K + a];
  if (e >= E) e = -1;  // reported by the histogram kernel; dropped here
  {
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    wrank = __popc(peers & ((1u << lane) - 1u));
    if (e >= 0 && wrank == 0) s_wcnt[warp * E + e] = __popc(peers);
  }
  __syncthreads();
  if (a < na) {
    int slot = -1;
    if (e >= 0) {
      int before = 0;
      for (int w = 0; w < warp; ++w) before += s_wcnt[w * E + e];
      slot = tile_base[e] * kTileRows + cta_base[(size_t)blockIdx.x * E + e] + before + wrank;
      src_info[slot] = t0 * K + a;
    }
    s_slot[a] = slot;
    slot_of[(size_t)t0 * K + a] = slot;
  }
  __syncthreads();
  copy_rows<4>(x, recv, s_slot, t0, ntok, K, vec_per_row);
  signal_rows(s_slot, na, tile_count, rows_done, avail_ns, T * K);
}

// ------------------------------------------------------------------------------------------------
// Modes 1/2: destination-agnostic dispatch in one kernel.
template <bool PAGED>
__global__ void __launch_bounds__(kDispThreads)
dispatch_atomic_kernel(const uint4* __restrict__ x, const int* __restrict__ topk_idx, int T, int E, int K,
                       int tok_per_blk, int vec_per_row, int cap_rows, int P, int tiles_per_expert,
                       unsigned long long spin_limit, int* __restrict__ row_pointer,
                       int* __restrict__ tile_table, int* __restrict__ pool_next,
                       int* __restrict__ tile_expert, uint4* __restrict__ recv, int* __restrict__ src_info,
                       int* __restrict__ slot_of, int* __restrict__ status, int* __restrict__ tile_count,
                       int* __restrict__ rows_done, unsigned long long* __restrict__ avail_ns) {
  extern __shared__ int smem_i[];
  int* s_cnt = smem_i;        // [E] rows this block sends to expert e
  int* s_base = smem_i + E;   // [E] first LocalRowID this block got from expert e's row pointer
  int* s_slot = smem_i + 2 * E;  // [kMaxAssign] physical row per assignment
  const int t0 = blockIdx.x * tok_per_blk;
  const int ntok = min(tok_per_blk, T - t0);
  const int na = ntok * K;
  const int lane = threadIdx.x % 32;
  for (int e = threadIdx.x; e < E; e += kDispThreads) s_cnt[e] = 0;
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  if (avail_ns != nullptr && threadIdx.x == 0) atomicMin(avail_ns, now_ns());

  // (a) rank inside the block: warp-aggregated shared-memory atomics
  const int a = threadIdx.x;
  int e = -1, lrank = 0;
  if (a < na) {
    e = topk_idx[(size_t)t0 * K + a];
    if (e < 0 || e >= E) {  // not an expert: report it, drop the assignment, touch no table with it
      set_status(status, MOE_ERR_ARG, t0 + a / K);
      e = -1;
    }
  }
  {
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int leader = __ffs(peers) - 1;
    int base = 0;
    if (e >= 0 && lane == leader) base = atomicAdd(&s_cnt[e], __popc(peers));
    base = __shfl_sync(0xffffffffu, base, leader);
    lrank = base + __popc(peers & ((1u << lane) - 1u));
  }
  __syncthreads();

  // (b) one global atomicAdd per touched expert: the block's rows get LocalRowIDs
  //     [base, base+n).  The block whose range opens a tile (a multiple of 128) claims it.
  for (int ee = threadIdx.x; ee < E; ee += kDispThreads) {
    const int n = s_cnt[ee];
    if (n == 0) continue;
    const int base = atomicAdd(&row_pointer[ee], n);
    s_base[ee] = base;
    const int first_tile = (base + kTileRows - 1) / kTileRows;  // tiles whose row 0 lies in [base, base+n)
    const int last_tile = (base + n - 1) / kTileRows;
    for (int lt = first_tile; lt <= last_tile; ++lt) {
      if (PAGED) {
        if (lt >= tiles_per_expert) { set_status(status, MOE_ERR_OVERFLOW, ee); continue; }
        const int tile = atomicAdd(pool_next, 1);
        if (tile >= P) { set_status(status, MOE_ERR_OVERFLOW, ee); continue; }
        tile_expert[tile] = ee;
        st_release(&tile_table[(size_t)ee * tiles_per_expert + lt], tile);
      } else {
        if ((lt + 1) * kTileRows <= cap_rows) tile_expert[ee * (cap_rows / kTileRows) + lt] = ee;
      }
    }
  }
  __syncthreads();

  // (c) LocalRowID -> physical row (address = Base + LocalRowID*RowSize), staged in shared memory
  if (a < na) {
    const int local_row = e >= 0 ? s_base[e] + lrank : 0;
    int slot = -1;
    if (e < 0) {
      // dropped above
    } else if (PAGED) {
      const int lt = local_row / kTileRows;
      if (lt < tiles_per_expert) {
        const int* entry = &tile_table[(size_t)e * tiles_per_expert + lt];
        int tile = ld_acquire(entry);
        unsigned long long spins = 0;
        while (tile < 0) {  // bounded wait for the block that opened this tile
          const int seen = ld_acquire(status);  // an overflow means the opener may never publish; a bad id elsewhere does not
          if ((seen != 0 && seen != MOE_ERR_ARG) || ++spins > spin_limit) {
            set_status(status, MOE_ERR_TIMEOUT, kWaitTileTable);
            break;
          }
          __nanosleep(32);
          tile = ld_acquire(entry);
        }
        if (tile >= 0) slot = tile * kTileRows + local_row % kTileRows;
      }
    } else {
      if (local_row < cap_rows) slot = e * cap_rows + local_row;
      else set_status(status, MOE_ERR_OVERFLOW, e);
    }
    s_slot[a] = slot;
    slot_of[(size_t)t0 * K + a] = slot;
    if (slot >= 0) src_info[slot] = t0 * K + a;  // the row's source information
  }
  __syncthreads();
  copy_rows<4>(x, recv, s_slot, t0, ntok, K, vec_per_row);
  if (tile_count != nullptr) signal_rows(s_slot, na, tile_count, rows_done, avail_ns, T * K);
}

// ------------------------------------------------------------------------------------------------
// The per-call start state of every dispatch scheme (counters, tile owners, source info, tile table: see
// make_prep) and, for the ordered scheme, the rows per expert.  When a dispatch is called on its own this
// small pass does it; inside moe_layer the router does it on the side and this launch does not exist.
__global__ void __launch_bounds__(kDispThreads)
prep_count_kernel(const PrepArgs prep, const int* __restrict__ topk_idx, int n_assign, int K) {
  __shared__ int s_hist[kMaxExperts];
  for (int e = threadIdx.x; e < kMaxExperts; e += kDispThreads) s_hist[e] = 0;
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  const int gtid = blockIdx.x * kDispThreads + threadIdx.x, gthreads = gridDim.x * kDispThreads;
  prep_reset(prep, gtid, gthreads);
  if (prep.hist == nullptr) return;
  for (int a = gtid; a < n_assign; a += gthreads) {
    const int e = topk_idx[a];
    if (e >= 0 && e < prep.E) atomicAdd(&s_hist[e], 1);  // ids that are no expert are reported by the dispatch itself
  }
  __syncthreads();
  for (int e = threadIdx.x; e < prep.E; e += kDispThreads)
    if (s_hist[e] != 0) atomicAdd(&prep.hist[e], s_hist[e]);
}

__global__ void __launch_bounds__(kDispThreads, 2)
dispatch_ordered_kernel(const OrderedParams prm, int* __restrict__ hist_rw, int* __restrict__ exit_counter) {
  extern __shared__ uint8_t ord_smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ord_smem_raw) + 127) & ~(uintptr_t)127);
  __shared__ OrdShared sh;
  pdl_wait();
  pdl_trigger();
  dispatch_ordered_cta<kDispThreads>(prm, sh, ring, blockIdx.x, gridDim.x);
  // Every CTA has read hist by now; the last one to leave clears it for the next call's counting.
  if (threadIdx.x == 0) sh.index_abort = atomicAdd(exit_counter, 1) == (int)gridDim.x - 1;
  __syncthreads();
  if (sh.index_abort) {
    for (int e = threadIdx.x; e < prm.E; e += kDispThreads) hist_rw[e] = 0;
    if (threadIdx.x == 0) *exit_counter = 0;
  }
}

PrepArgs make_prep(moe_plan* p, int* expert_count, int* tile_expert, int* src_info, int* tile_count, int* rows_done) {
  const moe_config_t& c = p->cfg;
  const int P = (int)p->P;
  PrepArgs a = {};
  auto add = [&](int* ptr, long long n, int value) {
    if (ptr != nullptr && n > 0) a.fill[a.nfill++] = PrepArgs::Fill{ptr, (int)n, value};
  };
  add(p->s.status, (long long)(p->counters_bytes / sizeof(int)), 0);  // status, pool cursor, scan ticket, global counter
  add(rows_done, 1, 0);
  add(tile_count, P, 0);
  add(p->s.gemm1_done, P + 4, 0);
  if (c.dispatch_mode == MOE_DISPATCH_ATOMIC_ORDERED && c.T > 0) {
    add(p->s.row_pointer, c.E, 0);  // expert_count, tile_expert and the empty slots' source info are written by the dispatch
    a.hist = p->s.hist;
  } else {  // (an empty batch in the ordered scheme launches no dispatch: its outputs get their start state here)
    add(expert_count, c.E, 0);
    add(tile_expert, P, -1);
    add(src_info, (long long)P * kTileRows, -1);
    if (c.dispatch_mode == MOE_DISPATCH_ATOMIC_PAGED) add(p->s.tile_table, (long long)c.E * p->tiles_per_expert, -1);
  }
  a.E = c.E;
  a.avail_ns = p->trace ? p->s.avail_ns : nullptr;
  a.avail_n = P + 2;
  return a;
}

OrderedParams make_ordered_params(moe_plan* p, const void* x, const int* topk_idx, void* recv, int* expert_count,
                                  int* tile_expert, int* src_info, int* slot_of, int* tile_count, int* rows_done) {
  const moe_config_t& c = p->cfg;
  OrderedParams q;
  q.x = (const uint8_t*)x;
  q.topk_idx = topk_idx;
  q.T = c.T;
  q.E = c.E;
  q.K = c.K;
  q.P = (int)p->P;
  q.row_bytes = c.H * (c.dtype == MOE_DTYPE_BF16 ? 2 : 4);
  q.tok_per_blk = p->ord_tokens;
  q.nblk = p->ord_nblk;
  q.ring_bytes = kOrdRingBytes;
  q.hist = p->s.hist;
  q.row_pointer = p->s.row_pointer;
  q.recv = (uint8_t*)recv;
  q.src_info = src_info;
  q.slot_of = slot_of;
  q.expert_count = expert_count;
  q.tile_expert = tile_expert;
  q.tile_count = tile_count;
  q.rows_done = rows_done;
  q.status = p->s.status;
  q.avail_ns = p->trace ? p->s.avail_ns : nullptr;
  q.wait_ns = c.wait_limit_ns ? c.wait_limit_ns : kDefaultWaitNs;
  return q;
}

static int launch_dispatch_ordered(moe_plan* p, const void* x, const int* topk_idx, void* recv, int* expert_count,
                                   int* tile_expert, int* src_info, int* slot_of, int* tile_count, int* rows_done,
                                   cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  OrderedParams q = make_ordered_params(p, x, topk_idx, recv, expert_count, tile_expert, src_info, slot_of, tile_count,
                                        rows_done);
  // Two CTAs per SM, each with half of the shared memory for its ring: one thread per CTA issues the bulk
  // copies, and two issuing threads per SM move small rows faster than one.
  q.ring_bytes = 96 * 1024;
  const size_t smem = (size_t)ord_ring(q.row_bytes, q.ring_bytes) * ord_buf_bytes(q.row_bytes) + 128;
  static SmemAttrOnce once;
  if (ensure_dynamic_smem(dispatch_ordered_kernel, smem, p->device, once) != cudaSuccess) return (int)cudaErrorInvalidValue;
  const int grid = max(1, min(2 * p->sm_count, q.nblk));
  launch_pdl(dispatch_ordered_kernel, dim3(grid), dim3(kDispThreads), smem, st, q, p->s.hist, p->s.ord_exit);
  p->launches += 1;
  return (int)cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
int launch_dispatch(moe_plan* p, const void* x, const int* topk_idx, void* recv, int* expert_count,
                    int* tile_expert, int* src_info, int* slot_of, int* tile_count, int* rows_done,
                    bool prepared, cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  const int eb = c.dtype == MOE_DTYPE_BF16 ? 2 : 4;
  const int vec_per_row = c.H * eb / 16;
  // Per-call start state (and, for the ordered scheme, the rows per expert): done by the kernel before this
  // call when `prepared`, else by one small launch here.
  if (!prepared) {
    const PrepArgs prep = make_prep(p, expert_count, tile_expert, src_info, tile_count, rows_done);
    const long long work = max((long long)p->P * kTileRows, (long long)c.T * c.K);
    const int grid = (int)max(1ll, min((long long)4 * p->sm_count, (work + 4 * kDispThreads - 1) / (4 * kDispThreads)));
    launch_pdl(prep_count_kernel, dim3(grid), dim3(kDispThreads), 0, st, prep, topk_idx, c.T * c.K, c.K);
    p->launches += 1;
  }
  if (c.T == 0) return 0;
  if (c.dispatch_mode == MOE_DISPATCH_ATOMIC_ORDERED)
    return launch_dispatch_ordered(p, x, topk_idx, recv, expert_count, tile_expert, src_info, slot_of, tile_count,
                                   rows_done, st);
  const int nblk = p->nblk, tpb = p->dispatch_tokens;
  if (c.dispatch_mode == MOE_DISPATCH_SCAN) {
    launch_maybe_pdl(false, hist_kernel, dim3(nblk), dim3(kDispThreads), sizeof(int) * c.E, st, topk_idx, c.T, c.E, c.K, tpb,
               p->s.cta_count, p->s.status, p->trace ? p->s.avail_ns : nullptr);
    launch_maybe_pdl(false, scan_kernel, dim3(c.E), dim3(kDispThreads), 0, st, p->s.cta_count, nblk, c.E, (int)p->P, p->s.cta_base,
               expert_count, p->s.tile_base, tile_expert, p->s.scan_ticket);
    const size_t smem = sizeof(int) * ((kDispThreads / 32) * c.E + kMaxAssign);
    launch_maybe_pdl(false, scatter_kernel, dim3(nblk), dim3(kDispThreads), smem, st, (const uint4*)x, topk_idx, c.T, c.E, c.K, tpb,
               vec_per_row, p->s.cta_base, p->s.tile_base, (uint4*)recv, src_info, slot_of, tile_count, rows_done,
               p->trace ? p->s.avail_ns : nullptr);
    p->launches += 3;
  } else {
    const size_t smem = sizeof(int) * (2 * c.E + kMaxAssign);
    const unsigned long long spin = c.spin_limit ? c.spin_limit : (1ull << 22);
    auto kern = c.dispatch_mode == MOE_DISPATCH_ATOMIC_PAGED ? dispatch_atomic_kernel<true> : dispatch_atomic_kernel<false>;
    launch_pdl(kern, dim3(nblk), dim3(kDispThreads), smem, st, (const uint4*)x, topk_idx, c.T, c.E, c.K, tpb, vec_per_row,
               (int)p->cap_rows, (int)p->P, p->tiles_per_expert, spin, expert_count, p->s.tile_table, p->s.pool_next,
               tile_expert, (uint4*)recv, src_info, slot_of, p->s.status, tile_count, rows_done,
               p->trace ? p->s.avail_ns : nullptr);
    p->launches += 1;
  }
  return (int)cudaGetLastError();
}

}  // namespace moehub

// ------------------------------------------------------------------------------------------------
// moe_dispatch_noalloc: the paged destination-agnostic dispatch for callers that cannot allocate.
//
// Its scratch (the pool cursor and the per-expert tile table) lives in the file-scope device array
// below instead of a caller-supplied workspace, so the call needs no plan and no device allocation
// of any kind.  Every GPU that loads this library carries the array (about 129 KB) until exit.
#include <mutex>

namespace {

constexpr int kNoAllocMaxTokens = MOE_NOALLOC_MAX_TOKENS;
constexpr int kNoAllocMaxExperts = 256;
constexpr int kNoAllocTilesPerExpert = kNoAllocMaxTokens / MOE_TILE_ROWS;
// layout: [0] pool cursor, [64 ...] tile table [E][tiles_per_expert]
constexpr int kNoAllocTableOffset = 64;
constexpr int kNoAllocInts = kNoAllocTableOffset + kNoAllocMaxExperts * kNoAllocTilesPerExpert;

static __device__ __align__(256) int g_noalloc_scratch[kNoAllocInts];

// In host code the array's name is only a handle for the runtime, not a device address.  The
// address is looked up once per device, with that device current, and kept here.
constexpr int kMaxDevices = 64;
int* g_noalloc_ptr[kMaxDevices];
std::mutex g_noalloc_mutex;

int noalloc_scratch_for_current_device(int** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOE_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (g_noalloc_ptr[dev] == nullptr) {
    int* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return MOE_ERR_CUDA;
    g_noalloc_ptr[dev] = ptr;
  }
  *out = g_noalloc_ptr[dev];
  return MOE_OK;
}

}  // namespace

extern "C" int moe_dispatch_noalloc(const moe_config_t* cfg, const void* d_x, const int32_t* d_topk_idx,
                                    void* d_recv, int32_t* d_expert_count, int32_t* d_tile_expert,
                                    int32_t* d_src_info, int32_t* d_slot_of, int32_t* d_status, void* stream) {
  using namespace moehub;
  if (!cfg || !d_recv || !d_expert_count || !d_tile_expert || !d_src_info || !d_status) return MOE_ERR_ARG;
  const moe_config_t& c = *cfg;
  if (c.T < 0 || c.H <= 0 || c.E <= 0 || c.R <= 0 || c.K <= 0 || c.K > c.E || c.E % c.R != 0) return MOE_ERR_ARG;
  if (c.dtype != MOE_DTYPE_FP32 && c.dtype != MOE_DTYPE_BF16) return MOE_ERR_ARG;
  if (c.T > 0 && (!d_x || !d_topk_idx || !d_slot_of)) return MOE_ERR_ARG;
  if (c.K > 32) return MOE_ERR_UNSUPPORTED;
  if (c.T > kNoAllocMaxTokens || c.E > kNoAllocMaxExperts) return MOE_ERR_TOO_LARGE;
  const int eb = c.dtype == MOE_DTYPE_BF16 ? 2 : 4;
  if (((int64_t)c.H * eb) % 16 != 0) return MOE_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_recv)) & 15) return MOE_ERR_ALIGN;

  int* scratch = nullptr;
  int rc = noalloc_scratch_for_current_device(&scratch);
  if (rc != MOE_OK) return rc;
  int* pool_next = scratch;
  int* tile_table = scratch + kNoAllocTableOffset;

  cudaStream_t st = (cudaStream_t)stream;
  const int64_t P = (int64_t)c.T * c.K / kTileRows + c.E;
  int tiles_per_expert = (c.T + kTileRows - 1) / kTileRows;
  if (tiles_per_expert == 0) tiles_per_expert = 1;
  int tpb = 256 / c.K;
  if (tpb > 16) tpb = 16;
  while (tpb > 1 && (c.T + tpb - 1) / tpb < 2 * 148) tpb /= 2;
  const int nblk = (c.T + tpb - 1) / tpb;
  // The array keeps whatever the previous call left: reset the cursor and the part of the table
  // this call reads, and the caller's counters, before the kernel runs.
  if (cudaMemsetAsync(pool_next, 0, sizeof(int), st) != cudaSuccess ||
      cudaMemsetAsync(tile_table, 0xff, sizeof(int) * (size_t)c.E * tiles_per_expert, st) != cudaSuccess ||
      cudaMemsetAsync(d_status, 0, sizeof(int) * 2, st) != cudaSuccess ||
      cudaMemsetAsync(d_expert_count, 0, sizeof(int) * c.E, st) != cudaSuccess ||
      cudaMemsetAsync(d_tile_expert, 0xff, sizeof(int) * P, st) != cudaSuccess ||
      cudaMemsetAsync(d_src_info, 0xff, sizeof(int) * P * kTileRows, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (c.T == 0) return MOE_OK;
  const size_t smem = sizeof(int) * (2 * c.E + kMaxAssign);
  const unsigned long long spin = c.spin_limit ? c.spin_limit : (1ull << 22);
  dispatch_atomic_kernel<true><<<nblk, kDispThreads, smem, st>>>(
      (const uint4*)d_x, d_topk_idx, c.T, c.E, c.K, tpb, c.H * eb / 16, 0, (int)P, tiles_per_expert, spin,
      d_expert_count, tile_table, pool_next, d_tile_expert, (uint4*)d_recv, d_src_info, d_slot_of, d_status,
      nullptr, nullptr, nullptr);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
