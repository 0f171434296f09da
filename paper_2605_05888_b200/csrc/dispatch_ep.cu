// Destination-agnostic dispatch across GPUs (real expert parallelism): the paper's actual setting
// (Section III-B and IV-B).  Rank r holds a contiguous share of the tokens and the experts
// [r*E/R, (r+1)*E/R).  A producer rank does NOT learn counts or offsets from anybody: for every token block
// it takes LocalRowIDs straight from the CONSUMER's allocation pointers - one system-scope atomicAdd per
// touched expert on the owning rank's row_pointer, through a peer mapping - and stores the rows into the
// owner's region at Base + LocalRowID * RowSize with plain 16-byte peer stores.  After the stores it raises
// the owner's per-tile status counters and global counter with system-scope release atomics (Section IV-D),
// so the consumer can start a tile as soon as its rows are there.  Regions are static, `cap_rows` per expert
// (the paper's conservative pre-allocation); a full region is reported, never overrun.
//
// Only plain loads, stores and atomics touch another GPU's memory here: no TMA or bulk copy, no multicast,
// no library kernel.  The kernel waits for nobody, so ranks never depend on running at the same time.
// Not measured on more than one GPU yet: on one GPU the test runs the ranks one after the other with every
// "peer" pointer in local memory.
#include "common.cuh"

namespace moehub {

constexpr int kEpThreads = 256;
constexpr int kEpMaxAssign = 256;
constexpr int kEpMaxRanks = MOE_EP_MAX_RANKS;

struct EpPeers {
  uint4* recv[kEpMaxRanks];
  int* row_pointer[kEpMaxRanks];
  int* tile_count[kEpMaxRanks];
  int* src_info[kEpMaxRanks];
  int* rows_done[kEpMaxRanks];
};

__global__ void __launch_bounds__(kEpThreads)
dispatch_ep_kernel(const uint4* __restrict__ x, const int* __restrict__ topk_idx, int T, int E, int R, int K, int rank,
                   int tok_per_blk, int vec_per_row, int cap_rows, const EpPeers peers, int* __restrict__ slot_of,
                   int* __restrict__ status) {
  extern __shared__ int smem_i[];
  int* s_cnt = smem_i;           // [E] rows this block sends to expert e
  int* s_base = smem_i + E;      // [E] first LocalRowID this block got from the owner's row pointer
  int* s_slot = smem_i + 2 * E;  // [kEpMaxAssign] owner-local physical row per assignment, -1: dropped
  int* s_owner = s_slot + kEpMaxAssign;
  const int epr = E / R;         // experts per rank
  const int t0 = blockIdx.x * tok_per_blk;
  const int ntok = min(tok_per_blk, T - t0);
  const int na = ntok * K;
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  for (int e = threadIdx.x; e < E; e += kEpThreads) s_cnt[e] = 0;
  __syncthreads();
  // (a) rank inside the block
  const int a = threadIdx.x;
  int e = -1, lrank = 0;
  if (a < na) {
    e = topk_idx[(size_t)t0 * K + a];
    if (e < 0 || e >= E) {
      set_status(status, MOE_ERR_ARG, t0 + a / K);
      e = -1;
    }
  }
  {
    const unsigned peers_mask = __match_any_sync(0xffffffffu, e);
    const int leader = __ffs(peers_mask) - 1;
    int base = 0;
    if (e >= 0 && lane == leader) base = atomicAdd(&s_cnt[e], __popc(peers_mask));
    base = __shfl_sync(0xffffffffu, base, leader);
    lrank = base + __popc(peers_mask & ((1u << lane) - 1u));
  }
  __syncthreads();
  // (b) one system-scope atomicAdd per touched expert on the OWNER's allocation pointer
  for (int ee = threadIdx.x; ee < E; ee += kEpThreads) {
    const int n = s_cnt[ee];
    if (n != 0) s_base[ee] = atomicAdd_system(&peers.row_pointer[ee / epr][ee % epr], n);
  }
  __syncthreads();
  // (c) LocalRowID -> address in the owner's region
  if (a < na) {
    int slot = -1, owner = 0;
    if (e >= 0) {
      owner = e / epr;
      const int local_row = s_base[e] + lrank;
      if (local_row < cap_rows) slot = (e % epr) * cap_rows + local_row;
      else set_status(status, MOE_ERR_OVERFLOW, e);
    }
    s_slot[a] = slot;
    s_owner[a] = owner;
    // the combine side finds the row again through (owner, row): one global row number
    slot_of[(size_t)t0 * K + a] = slot >= 0 ? owner * epr * cap_rows + slot : -1;
    if (slot >= 0) peers.src_info[owner][slot] = (rank * T + t0) * K + a;  // source information: (source rank, token, k)
  }
  __syncthreads();
  // (d) the rows: read once, stored to each of the K owners with 16-byte peer stores
  constexpr int RUN = 32 * 4;
  const int runs = (vec_per_row + RUN - 1) / RUN;
  for (int u = warp; u < ntok * runs; u += kEpThreads / 32) {
    const int tl = u / runs, v0 = (u % runs) * RUN;
    const uint4* src = x + (size_t)(t0 + tl) * vec_per_row;
    uint4 r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int v = v0 + i * 32 + lane;
      if (v < vec_per_row) r[i] = __ldg(src + v);
    }
    for (int k = 0; k < K; ++k) {
      const int slot = s_slot[tl * K + k];
      if (slot < 0) continue;
      uint4* dst = peers.recv[s_owner[tl * K + k]] + (size_t)slot * vec_per_row;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int v = v0 + i * 32 + lane;
        if (v < vec_per_row) dst[v] = r[i];
      }
    }
  }
  // (e) availability: the owner's status counters, after this block's stores are visible system-wide
  __threadfence_system();
  __syncthreads();
  if (a < na && s_slot[a] >= 0) {
    int* ctr = peers.tile_count[s_owner[a]] + s_slot[a] / kTileRows;
    asm volatile("red.release.sys.global.add.s32 [%0], 1;" ::"l"(ctr) : "memory");
  }
  // every assignment is counted at its owner (a dropped one too: the consumer must not wait for it forever)
  if (a < na) {
    const int owner = e >= 0 ? e / epr : 0;
    asm volatile("red.release.sys.global.add.s32 [%0], 1;" ::"l"(peers.rows_done[owner]) : "memory");
  }
}

// The owner's tile table from its allocation pointers, once every producer has finished: region e holds
// min(row_pointer[e], cap_rows) rows in its first tiles; the other tiles of the region are unused.
__global__ void ep_tiles_kernel(const int* __restrict__ row_pointer, int epr, int cap_rows, int* __restrict__ expert_count,
                                int* __restrict__ tile_expert) {
  const int tiles_per = cap_rows / kTileRows;
  const int tile = blockIdx.x * blockDim.x + threadIdx.x;
  if (tile >= epr * tiles_per) return;
  const int e = tile / tiles_per, i = tile % tiles_per;
  const int cnt = max(0, min(row_pointer[e], cap_rows));
  tile_expert[tile] = i * kTileRows < cnt ? e : -1;
  if (i == 0) expert_count[e] = cnt;
}

// The combine direction (Section IV-B, all-to-all combine): the owner reads every result row's source
// information (source rank, token, k) and stores the row at the token's own position, row t*K+k of the source
// rank's staging buffer [T*K, H] - plain 16-byte peer stores again.  After a CTA's stores are visible
// system-wide it raises the source rank's counter of returned rows by the rows it sent there, so that rank
// knows its T*K rows (minus dropped ones) are back without hearing from anybody.
struct EpStaging {
  uint4* staging[kEpMaxRanks];
  int* rows_back[kEpMaxRanks];
};

__global__ void __launch_bounds__(kEpThreads)
combine_ep_kernel(const uint4* __restrict__ out_rows, const int* __restrict__ src_info, const int* __restrict__ expert_count,
                  int cap_rows, int vec_per_row, int rows_per_rank /* T*K */, int R, const EpStaging peers,
                  int* __restrict__ status) {
  __shared__ int s_sent[kEpMaxRanks];
  const int tiles_per = cap_rows / kTileRows;
  const int e = blockIdx.x / tiles_per, i = blockIdx.x % tiles_per;
  const int rows = min(kTileRows, expert_count[e] - i * kTileRows);
  if (rows <= 0) return;
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  if (threadIdx.x < kEpMaxRanks) s_sent[threadIdx.x] = 0;
  __syncthreads();
  const size_t row0 = (size_t)e * cap_rows + (size_t)i * kTileRows;
  for (int r = warp; r < rows; r += kEpThreads / 32) {
    const int src = src_info[row0 + r];
    const int dst = src / rows_per_rank;
    if (src < 0 || dst >= R) {  // a row nobody registered: report it, send nothing
      if (lane == 0) set_status(status, MOE_ERR_INTERNAL, 301);
      continue;
    }
    const uint4* from = out_rows + (row0 + r) * vec_per_row;
    uint4* to = peers.staging[dst] + (size_t)(src % rows_per_rank) * vec_per_row;
    for (int v = lane; v < vec_per_row; v += 32) to[v] = __ldg(from + v);
    if (lane == 0) atomicAdd(&s_sent[dst], 1);
  }
  __threadfence_system();
  __syncthreads();
  if (threadIdx.x < R && s_sent[threadIdx.x] != 0)
    asm volatile("red.release.sys.global.add.s32 [%0], %1;" ::"l"(peers.rows_back[threadIdx.x]), "r"(s_sent[threadIdx.x]) : "memory");
}

}  // namespace moehub

extern "C" int moe_ep_tiles(int32_t experts_local, int64_t cap_rows, const int32_t* d_row_pointer, int32_t* d_expert_count,
                            int32_t* d_tile_expert, void* stream) {
  using namespace moehub;
  if (experts_local <= 0 || cap_rows <= 0 || cap_rows % kTileRows != 0) return MOE_ERR_ARG;
  if (!d_row_pointer || !d_expert_count || !d_tile_expert) return MOE_ERR_ARG;
  if ((int64_t)experts_local * cap_rows >= (1ll << 31)) return MOE_ERR_UNSUPPORTED;
  const int tiles = experts_local * (int)(cap_rows / kTileRows);
  ep_tiles_kernel<<<(tiles + 127) / 128, 128, 0, (cudaStream_t)stream>>>(d_row_pointer, experts_local, (int)cap_rows,
                                                                        d_expert_count, d_tile_expert);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

extern "C" int moe_combine_ep(const moe_config_t* cfg, void* const* h_staging, int32_t* const* h_rows_back, int64_t cap_rows,
                              const void* d_out_rows, const int32_t* d_src_info, const int32_t* d_expert_count,
                              int32_t* d_status, void* stream) {
  using namespace moehub;
  if (!cfg || !h_staging || !h_rows_back || !d_status) return MOE_ERR_ARG;
  const moe_config_t& c = *cfg;
  if (c.T < 0 || c.H <= 0 || c.E <= 0 || c.R <= 0 || c.K <= 0 || c.E % c.R != 0) return MOE_ERR_ARG;
  if (cap_rows <= 0 || cap_rows % kTileRows != 0) return MOE_ERR_ARG;
  if (c.dtype != MOE_DTYPE_FP32 && c.dtype != MOE_DTYPE_BF16) return MOE_ERR_ARG;
  if (c.R > kEpMaxRanks) return MOE_ERR_UNSUPPORTED;
  if (!d_out_rows || !d_src_info || !d_expert_count) return MOE_ERR_ARG;
  const int eb = c.dtype == MOE_DTYPE_BF16 ? 2 : 4;
  if (((int64_t)c.H * eb) % 16 != 0 || (reinterpret_cast<uintptr_t>(d_out_rows) & 15)) return MOE_ERR_ALIGN;
  if ((int64_t)c.R * c.T * c.K >= (1ll << 31) || (int64_t)(c.E / c.R) * cap_rows >= (1ll << 31)) return MOE_ERR_UNSUPPORTED;
  EpStaging peers = {};
  for (int r = 0; r < c.R; ++r) {
    if (!h_staging[r] || !h_rows_back[r]) return MOE_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(h_staging[r]) & 15) return MOE_ERR_ALIGN;
    peers.staging[r] = (uint4*)h_staging[r];
    peers.rows_back[r] = h_rows_back[r];
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(d_status, 0, 2 * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
  if (c.T == 0) return MOE_OK;  // with no tokens per rank nothing was dispatched
  const int tiles = (c.E / c.R) * (int)(cap_rows / kTileRows);
  combine_ep_kernel<<<tiles, kEpThreads, 0, st>>>((const uint4*)d_out_rows, d_src_info, d_expert_count, (int)cap_rows,
                                                  c.H * eb / 16, c.T * c.K, c.R, peers, d_status);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

extern "C" int moe_dispatch_ep(const moe_config_t* cfg, int32_t rank, const moe_ep_peer_t* h_peers, int64_t cap_rows,
                               const void* d_x, const int32_t* d_topk_idx, int32_t* d_slot_of, int32_t* d_status,
                               void* stream) {
  using namespace moehub;
  if (!cfg || !h_peers || !d_status) return MOE_ERR_ARG;
  const moe_config_t& c = *cfg;
  if (c.T < 0 || c.H <= 0 || c.E <= 0 || c.R <= 0 || c.K <= 0 || c.K > c.E || c.E % c.R != 0) return MOE_ERR_ARG;
  if (rank < 0 || rank >= c.R || cap_rows <= 0 || cap_rows % kTileRows != 0) return MOE_ERR_ARG;
  if (c.dtype != MOE_DTYPE_FP32 && c.dtype != MOE_DTYPE_BF16) return MOE_ERR_ARG;
  if (c.R > kEpMaxRanks || c.E > 256 || c.K > 32) return MOE_ERR_UNSUPPORTED;
  if (c.T > 0 && (!d_x || !d_topk_idx || !d_slot_of)) return MOE_ERR_ARG;
  const int eb = c.dtype == MOE_DTYPE_BF16 ? 2 : 4;
  if (((int64_t)c.H * eb) % 16 != 0 || (reinterpret_cast<uintptr_t>(d_x) & 15)) return MOE_ERR_ALIGN;
  if ((int64_t)c.R * c.T * c.K >= (1ll << 31) || (int64_t)c.E * cap_rows >= (1ll << 31)) return MOE_ERR_UNSUPPORTED;
  EpPeers peers = {};
  for (int r = 0; r < c.R; ++r) {
    const moe_ep_peer_t& q = h_peers[r];
    if (!q.recv || !q.row_pointer || !q.tile_count || !q.src_info || !q.rows_done) return MOE_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(q.recv) & 15) return MOE_ERR_ALIGN;
    peers.recv[r] = (uint4*)q.recv;
    peers.row_pointer[r] = q.row_pointer;
    peers.tile_count[r] = q.tile_count;
    peers.src_info[r] = q.src_info;
    peers.rows_done[r] = q.rows_done;
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(d_status, 0, 2 * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
  if (c.T == 0) return MOE_OK;
  int tpb = kEpMaxAssign / c.K;
  if (tpb > 16) tpb = 16;
  if (tpb < 1) tpb = 1;
  const int nblk = (c.T + tpb - 1) / tpb;
  const size_t smem = sizeof(int) * (2 * c.E + 2 * kEpMaxAssign);
  dispatch_ep_kernel<<<nblk, kEpThreads, smem, st>>>((const uint4*)d_x, d_topk_idx, c.T, c.E, c.R, c.K, rank, tpb,
                                                     c.H * eb / 16, (int)cap_rows, peers, d_slot_of, d_status);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
