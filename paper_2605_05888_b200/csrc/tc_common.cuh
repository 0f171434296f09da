// PTX wrappers and constants shared by the tcgen05 expert-FFN kernels (one-CTA and CTA-pair forms).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace moehub {

constexpr int kTcThreads = 192;
constexpr int kStages = 4;
constexpr int kBK = 64;                       // k elements per stage (128 bytes of bf16)
constexpr int kUmmaN = 256;
constexpr int kABytes = kTileRows * kBK * 2;  // 16 KB
constexpr int kBBytes = kUmmaN * kBK * 2;     // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTcSmem = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers, item ring*/;
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;  // default bound on any single wait: 2 s

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the time limit ran out or another role already gave up.
// sleep_ns > 0 backs off between polls: for waits that are long by design (an epilogue warp waiting
// for a whole main loop) polling at full rate only burns power the tensor pipe could use.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns, unsigned sleep_ns = 0) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  for (unsigned it = 1;; ++it) {
    if (sleep_ns) __nanosleep(sleep_ns);
    if (mbar_try(bar, parity)) return true;
    if ((it & 31u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer() - t0 > limit_ns) return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
// The same load with an L2 eviction-priority hint (a policy made by l2_policy_evict_first/_last).
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// One 32-byte store (a whole L2 sector) per lane.  The epilogues write a row per lane, so a 16-byte
// store covers half a sector and the L2 has to merge the halves; whole sectors need no merge.
__device__ __forceinline__ void st_global_32B(void* p, const uint4& lo, const uint4& hi) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(lo.x), "r"(lo.y), "r"(lo.z),
               "r"(lo.w), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
}

// silu(g) * u in fp32.  The quotient is the approximate divide (2 ulp, far inside the bf16 rounding that
// follows): the IEEE divide leaves its fast path for NaN, infinite and very large operands, and the
// padding rows of a partly filled tile hold whatever the pool held before, so a single such lane
// sends its whole warp through the slow subroutine (measured: 21 us instead of 2 us per 128 x 128 block
// when three quarters of a tile's rows are padding).
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) in the
// 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fff);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                  // leading byte offset (unused with swizzle, K-major)
  d |= (uint64_t)(1024 >> 4) << 32;        // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                  // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                  // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A and B K-major, M = 128, N = 256.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kUmmaN >> 3) << 17) |
                            ((uint32_t)(kTileRows >> 4) << 24);

// Thin tiles (at most kThinRows rows): the MMA is M = 128 weight rows x N = 16*n16 tile rows.
constexpr int kThinRows = 64;
constexpr int kThinShift = 24;  // an item-ring entry is item | n16 << kThinShift
__host__ __device__ constexpr uint32_t thin_idesc(int n16) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n16 * 16 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// Short last tile of an expert with several tiles: M = 64 MMAs on the tile's first 64 rows.
constexpr int kHalfForm = 8;  // value of the n16 field for this form (thin tiles use 1..4)
constexpr uint32_t kIdescHalf = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kUmmaN >> 3) << 17) | ((uint32_t)(64 >> 4) << 24);

constexpr int kMaxExperts = 256;

struct Item {
  int type;   // 0: GEMM1 (+SwiGLU), 1: GEMM2
  int e, nb, tile;
  int m;      // tiles of expert e
  bool cold;  // item of the weight-streaming-bound run (interleaved work list)
};

// The work list, built by every CTA for itself in shared memory from tile_expert[P] (the same
// deterministic result in every CTA, so no launch and no global round trip is spent on it).
//   tiles[estart[e] .. estart[e+1])  the used tiles of expert e, in ascending tile order;
//   the item sequence is at most 2E segments, segment = all GEMM1 items or all GEMM2 items of one
//   expert: seg_start[i] first item of segment i (seg_start[2E] = number of items), seg_info[i] =
//   expert | type << 16 (type 0: GEMM1, 1: GEMM2); n1 = items before the first GEMM2 item when the
//   two GEMMs are separate launches.
//   With hot_min > 0 (separate launches only) each GEMM's segments are ordered "hot" experts first
//   (at least hot_min tiles: their items are bound by the tensor pipe, the weights come out of L2),
//   then "cold" ones (fewer tiles: bound by streaming the expert's weights from HBM once), both in
//   ascending expert order, and n_hot[g] counts the hot items of GEMM g: the kernel walks the two
//   runs interleaved, so that at any moment some SMs pull weights from HBM while the others run MMAs.
constexpr int kMaxListTiles = 4608;
struct WorkList {
  int estart[kMaxExperts + 1];
  int seg_start[2 * kMaxExperts + 1];
  int seg_info[2 * kMaxExperts];
  int cursor[kMaxExperts];
  int order[kMaxExperts];  // the experts in the order their segments are placed
  int count[kMaxExperts];  // rows per expert when the list was built from row counts, else -1
  int n1;
  int n_hot[2];
  int tiles[kMaxListTiles];
};

// All threads of the CTA call this (it synchronises the CTA).  pair = 2 counts one item per PAIR of
// tiles.  fused: the GEMM2 segment of an expert follows once at least `lag` items were placed after its
// GEMM1 segment, as long as `lag` GEMM2 items stay in reserve for the end of the list; otherwise all
// GEMM1 segments come first.
// hist != nullptr: the list is built from the experts' row counts instead of tile_expert - expert e then
// owns the consecutive tiles [estart[e], estart[e + 1]) (the layout of the ordered dispatch), which is known
// before a single row has been dispatched.  hot_first: experts are placed by descending row count (the
// experts whose first tiles fill earliest come first) instead of by index.
__device__ __forceinline__ void build_worklist(WorkList& wl, const int* __restrict__ tile_expert, int P, int E,
                                               int NB1, int NB2, int lag, int fused, int pair, int hot_min = 0,
                                               const int* __restrict__ hist = nullptr, int hot_first = 0) {
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid % 32;
  for (int e = tid; e < kMaxExperts; e += nthr) {
    wl.cursor[e] = (hist != nullptr && e < E) ? (hist[e] + kTileRows - 1) / kTileRows : 0;
    wl.count[e] = (hist != nullptr && e < E) ? hist[e] : -1;
    wl.order[e] = e;
  }
  __syncthreads();
  if (hist == nullptr) {
    for (int p = tid; p < P; p += nthr) {
      const int e = tile_expert[p];
      if (e >= 0 && e < E) atomicAdd(&wl.cursor[e], 1);
    }
  } else if (hot_first) {
    // position of expert e = experts with more rows, or as many and a lower index
    for (int e = tid; e < E; e += nthr) {
      const int c = wl.count[e];
      int rank = 0;
      for (int o = 0; o < E; ++o) {
        const int co = wl.count[o];
        rank += (co > c || (co == c && o < e)) ? 1 : 0;
      }
      wl.order[rank] = e;
    }
  }
  __syncthreads();
  if (tid < 32) {  // exclusive scan of the per-expert tile counts: 8 experts per lane
    int c[kMaxExperts / 32], sum = 0;
#pragma unroll
    for (int i = 0; i < kMaxExperts / 32; ++i) {
      const int e = lane * (kMaxExperts / 32) + i;
      c[i] = e < E ? wl.cursor[e] : 0;
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
      if (e < E) {
        wl.estart[e] = run;
        wl.cursor[e] = run;
      }
      run += c[i];
    }
    if (lane == 31) wl.estart[E] = incl;
    __syncwarp();
    if (hist != nullptr) {
      const int total = min(__shfl_sync(0xffffffffu, incl, 31), kMaxListTiles);
      for (int t = lane; t < total; t += 32) wl.tiles[t] = t;  // regions are consecutive tiles
    } else {
      // stable scatter, 32 tiles at a time: the same list in every CTA
      for (int p0 = 0; p0 < P; p0 += 32) {
        const int p = p0 + lane;
        int e = p < P ? tile_expert[p] : -1;
        if (e >= E) e = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        if (e >= 0) wl.tiles[wl.cursor[e] + __popc(peers & ((1u << lane) - 1u))] = p;
        __syncwarp();
        if (e >= 0 && lane == __ffs(peers) - 1) wl.cursor[e] += __popc(peers);
        __syncwarp();
      }
    }
    __syncwarp();
    auto tiles_of = [&](int e) { return wl.estart[e + 1] - wl.estart[e]; };
    if (lane == 0 && !fused && hot_min > 0) {
      // two passes per GEMM: hot experts, then cold ones
      int pos = 0, nseg = 0;
      for (int g = 0; g < 2; ++g) {
        const int nb = g == 0 ? NB1 : NB2;
        const int begin = pos;
        for (int cold = 0; cold < 2; ++cold) {
          for (int e = 0; e < E; ++e) {
            const int m = tiles_of(e);
            if ((m >= hot_min ? 0 : 1) != cold) continue;
            wl.seg_start[nseg] = pos;
            wl.seg_info[nseg++] = e | (g << 16);
            pos += (m + pair - 1) / pair * nb;
          }
          if (cold == 0) wl.n_hot[g] = pos - begin;
        }
        if (g == 0) wl.n1 = pos;
      }
      wl.seg_start[nseg] = pos;  // nseg == 2E
    } else if (lane == 0) {
      wl.n_hot[0] = wl.n_hot[1] = -1;  // no interleaving
      int pos = 0, nseg = 0, q = 0;  // i, q: positions in wl.order
      // GEMM2 items of the experts at positions q+1 .. E-2: what would still stand between the last expert's
      // GEMM1 and its GEMM2 if the GEMM2 segment of position q were placed now.  Keeping `lag` items in that
      // reserve gives the last experts the same distance as the first ones (without it their GEMM2 items
      // waited up to half an item for the intermediate).
      int reserve = 0;
      for (int j = 1; j + 1 < E; ++j) reserve += (tiles_of(wl.order[j]) + pair - 1) / pair * NB2;
      for (int i = 0; i < E; ++i) {
        const int e = wl.order[i];
        wl.seg_start[nseg] = pos;
        wl.seg_info[nseg++] = e;
        pos += (tiles_of(e) + pair - 1) / pair * NB1;
        wl.cursor[i] = pos;  // end of the GEMM1 items of position i
        while (fused && q < i && pos - wl.cursor[q] >= lag && reserve >= lag) {
          wl.seg_start[nseg] = pos;
          wl.seg_info[nseg++] = wl.order[q] | (1 << 16);
          pos += (tiles_of(wl.order[q]) + pair - 1) / pair * NB2;
          ++q;
          if (q + 1 < E) reserve -= (tiles_of(wl.order[q]) + pair - 1) / pair * NB2;
        }
      }
      wl.n1 = fused ? 0 : pos;
      for (; q < E; ++q) {
        wl.seg_start[nseg] = pos;
        wl.seg_info[nseg++] = wl.order[q] | (1 << 16);
        pos += (tiles_of(wl.order[q]) + pair - 1) / pair * NB2;
      }
      wl.seg_start[nseg] = pos;  // nseg == 2E
    }
  }
  __syncthreads();
}

// Everything the expert-FFN kernels take.
struct FfnParams {
  const int* tile_expert;  // [P]
  int P, lag, fused;
  int hot_min;  // > 0: interleave tensor-bound and weight-streaming-bound items (see WorkList)
  const int* push_src;  // push-style combine: the source info t*K+k of every pool row - the GEMM2 epilogue stores row r
                        // of the pool at row push_src[r] of `out` (the token's own position) and skips rows whose
                        // source is negative (empty slots); nullptr: rows stay where they are
  const int* hist;  // rows per expert (the ordered dispatch's counts): the work list is built from them, or nullptr
  int hot_first;    // with hist: experts are walked by descending row count
  int band;         // > 0 (the launch that carries the dispatch): an expert's items go band by band of this many tiles
                    // (column-block-major inside a band), so the first items need only the expert's first tiles,
                    // which the token-ordered dispatch completes first; 0: column-block-major over all its tiles
  int thin;         // the narrow (transposed) form for single tiles of at most 64 rows is in use
  int cold_below;   // experts with fewer tiles than this stream their weights once: their loads are evict-first
  int phase, E, F, H;
  int tp;  // TP shards per expert: expert index e of the work list is shard e % tp of expert e / tp (the down matrix's map is 4-D)
  __nv_bfloat16* inter;
  __nv_bfloat16* out;
  int* gemm1_done;
  int* work_counter;  // [4] items handed out beyond the first one per CTA: [0] phases 0 and 1, [1] phase 2 (zero at launch; the
                      // last CTA to leave zeroes it again); [2], [3]: CTAs that left
  const int* tile_count;
  const int* rows_done;
  int total_rows;
  unsigned long long wait_ns;  // bound on every wait inside the kernel
  int* status;
  unsigned long long* clock_probe;  // [2]: SM cycles and nanoseconds CTA 0 spent in the kernel (accumulated)
  unsigned long long* item_ns;      // work-item timeline (measurement; nullptr: off): 4 words per position of the item list
};

// Effective SM clock while a kernel runs: CTA 0 adds its elapsed %clock64 and %globaltimer.
struct ClockProbe {
  unsigned long long* out;
  long long c0;
  unsigned long long t0;
  __device__ explicit ClockProbe(unsigned long long* o) : out(o), c0(0), t0(0) {
    if (out != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
      c0 = clock64();
      t0 = globaltimer();
    }
  }
  __device__ void finish() {
    if (out != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
      atomicAdd(out, (unsigned long long)(clock64() - c0));
      atomicAdd(out + 1, globaltimer() - t0);
    }
  }
};

// The CTA-pair (cta_group::2) kernel lives in ffn_tc2.cu.
int launch_ffn_tc2_kernel(const CUtensorMap& a1, const CUtensorMap& bg, const CUtensorMap& bu, const CUtensorMap& a2,
                          const CUtensorMap& bd, const FfnParams& prm, int grid, cudaStream_t st);

// ---- tensor maps (host side) ---------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline int get_encoder(moe_plan* p, EncodeTiledFn* fn) {
  if (!p->encode_tiled) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || !sym ||
        q != cudaDriverEntryPointSuccess)
      return MOE_ERR_CUDA;
    p->encode_tiled = sym;
  }
  *fn = (EncodeTiledFn)p->encode_tiled;
  return MOE_OK;
}

// bf16 matrix [rows, cols] (row-major, cols contiguous), box [box_rows, 64 cols], 128-byte swizzle.
inline int make_map_2d(EncodeTiledFn enc, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                       uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace moehub
