// Shared declarations of the sm_100a MoE hot path: the plan, the launchers each .cu file
// exports to api.cu, and small device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moehub.h"

namespace moehub {

constexpr int kTileRows = MOE_TILE_ROWS;

// Device status word: [0] code, [1] detail.  First error wins.
__device__ __forceinline__ void set_status(int* status, int code, int detail) {
  if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// Wait sites reported in the detail word of MOE_ERR_TIMEOUT.
enum WaitSite { kWaitTileTable = 1, kWaitMbarTma = 3, kWaitMbarMma = 4,
                kWaitMbarEpi = 5, kWaitMbarTmemFree = 6, kWaitTileReady = 7, kWaitItem = 8 };

struct Scratch {          // device pointers carved out of the caller's workspace
  int* status;            // [4]
  int* pool_next;         // [1]   paged mode: next free tile
  int* scan_ticket;       // [1]   mode 0: CTAs of the scan kernel that finished
  int* rows_done;         // [1]   assignments whose rows are stored (global completion counter)
  int* tile_count;        // [P]   rows stored per tile (per-tile status counter)
  int* tile_table;        // [E * tiles_per_expert] paged mode: expert-local tile -> pool tile
  int* cta_count;         // [nblk * E] mode 0: per token-block histogram
  int* cta_base;          // [nblk * E] mode 0: exclusive prefix inside the expert
  int* tile_base;         // [E + 1]    mode 0: first pool tile of each expert
  int* hist;              // [E]   mode 3: rows per expert, counted by the router (or a counting pass) before the dispatch;
                          //       zero between calls (the dispatch puts it back)
  int* row_pointer;       // [E]   mode 3: next free LocalRowID per expert
  int* ord_exit;          // [2]   mode 3: CTAs that left the dispatch kernel / the fused kernel
  unsigned long long* clock_probe;  // [2] cycles, nanoseconds of CTA 0 inside the tensor-core kernels
  unsigned long long* avail_ns;  // [P+2] availability trace (measurement): dispatch start, all-ready time, per-tile ready time
  unsigned long long* item_ns;   // [4 * P * (NB1 + NB2)] work-item timeline of the tensor-core expert kernel (measurement)
  int* gemm1_done;        // [P+4]  per-tile status counter: GEMM1 blocks finished (x4 epilogue warps); [P..P+1] item counters, [P+2..P+3] exit counters of the expert kernel's launches
  void* inter;            // [P*128, F] SwiGLU intermediate
  float* route_logits;    // [T, 256] approximate router logits of the tensor-core filter (wide router, bf16)
  float* route_wnorm2;    // [256]    squared norms of the router's weight rows, recomputed by every call
  // moe_layer's internal buffers
  int* topk_idx;
  float* topk_w;
  void* recv;
  void* out_rows;
  int* expert_count;
  int* tile_expert;
  int* src_info;
  int* slot_of;
  void* x_stage[2];       // [T,H] device copies of host x (moe_layer_host; two for the pipelined form)
  void* y_stage[2];       // [T,H]
};

}  // namespace moehub

namespace moehub {
// What the kernel that runs right before a dispatch does on the side (inside moe_layer that kernel is the
// router, so no reset launch stands between the two): it puts the per-call counters and tables into their
// start state and, for the ordered scheme, adds its part of the experts' row counts to hist.
struct PrepArgs {
  struct Fill { int* ptr; int n; int value; };
  Fill fill[9];
  int nfill;                     // 0: nothing to do
  unsigned long long* avail_ns;  // [avail_n] availability trace to re-arm, or nullptr
  int avail_n;
  int* hist;                     // [E] rows per expert (ordered dispatch), or nullptr
  int E;
};
__device__ __forceinline__ void prep_reset(const PrepArgs& a, int gtid, int gthreads) {
  for (int j = 0; j < a.nfill; ++j)
    for (int i = gtid; i < a.fill[j].n; i += gthreads) a.fill[j].ptr[i] = a.fill[j].value;
  if (a.avail_ns != nullptr)
    for (int i = gtid; i < a.avail_n; i += gthreads) a.avail_ns[i] = i == 0 ? ~0ull : 0ull;
}
}  // namespace moehub

struct moe_plan {
  moe_config_t cfg;          // the EFFECTIVE configuration: with tp_shards = S, E, K and F here are E*S, K*S and F/S
                             // (every expert's S shards are S virtual experts, every pick S assignments)
  int tp;                    // TP shards per expert (1: none)
  int route_E, route_K;      // what the router works with: the experts it scores and the picks per token
  int64_t P;                 // pool tiles
  int64_t cap_rows;          // mode 1: rows per expert
  int tiles_per_expert;      // paged tile-table width
  int dispatch_tokens;       // tokens per dispatch CTA
  int nblk;                  // dispatch CTAs
  int ord_tokens, ord_nblk;  // mode 3: tokens per token block, token blocks
  int device;
  int sm_count;
  int launches;
  size_t counters_bytes;     // leading part of the workspace cleared by dispatch
  moehub::Scratch s;
  void* encode_tiled;        // cuTensorMapEncodeTiled entry point (driver API), looked up once
  // moe_layer_host_submit / _wait: copy streams and per-buffer events (host resources, made on first use)
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_in[2], ev_done[2], ev_out[2];
  long long submitted;       // steps submitted so far
  int cuda_error;            // last CUDA error a call of this plan met (cudaError_t), 0 if none
  int cuda_error_step;       // which step of moe_layer met it: 1 router, 2 dispatch, 3 experts, 4 combine
  int timing;                // moe_layer_timed: record an event after every kernel of the layer
  int trace;                 // moe_availability_trace: the dispatch kernels write avail_ns
  cudaEvent_t tev[MOE_STAGE_COUNT + 1];
};

namespace moehub {

// Timing marks of moe_layer_timed: mark i closes stage i-1.
inline void mark(moe_plan* p, int i, cudaStream_t st) {
  if (p->timing) cudaEventRecord(p->tev[i], st);
}

// Launch with the programmatic-stream-serialization attribute (see pdl_wait / pdl_trigger).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_maybe_pdl(bool pdl, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  return launch_maybe_pdl(true, kern, grid, block, smem, st, static_cast<Args&&>(args)...);
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) applies to the CURRENT device only, so the "already
// set" flag of a kernel is kept per device (a process may hold plans on several GPUs).  Setting it twice
// is harmless, so concurrent first calls need no lock.
struct SmemAttrOnce {
  size_t set[64] = {};  // bytes the attribute was last set to, per device
};
template <typename Kern>
inline cudaError_t ensure_dynamic_smem(Kern kern, size_t bytes, int device, SmemAttrOnce& once) {
  if (device >= 0 && device < 64 && once.set[device] >= bytes) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && device >= 0 && device < 64) once.set[device] = bytes;
  return e;
}

// ---- launchers (defined in the other .cu files); each returns a cudaError_t as int ------------
// prep: the per-call resets and the row counts of an ordered dispatch that follows (nullptr: none).
int launch_route(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx,
                 float* topk_w, const PrepArgs* prep, cudaStream_t st);
// the tensor-core filter in front of the exact chains (many experts, bf16): see route_filter.cu
bool route_filter_applies(const moe_plan* p);
int launch_route_filter(moe_plan* p, const void* x, const void* wr, const float* bias, int* topk_idx, float* topk_w,
                        const PrepArgs& prep, cudaStream_t st);
// prepared: the kernel before this call has already done what make_prep() describes.
int launch_dispatch(moe_plan* p, const void* x, const int* topk_idx, void* recv, int* expert_count,
                    int* tile_expert, int* src_info, int* slot_of, int* tile_count, int* rows_done,
                    bool prepared, cudaStream_t st);
PrepArgs make_prep(moe_plan* p, int* expert_count, int* tile_expert, int* src_info, int* tile_count, int* rows_done);
// staged: rows holds assignment (t, k) at row t*K+k (push-style combine); slot_of then only tells dropped assignments.
int launch_combine(moe_plan* p, const void* rows, const int* slot_of, const float* topk_w, void* y,
                   cudaStream_t st, bool staged = false);
int launch_ffn_simt(moe_plan* p, const void* recv, const int* tile_expert, const void* wg,
                    const void* wu, const void* wd, void* out_rows, cudaStream_t st);
// tile_count / rows_done: availability counters the GEMM1 producer waits on before it reads a tile
// (nullptr: the rows are complete when the kernel starts).
int launch_ffn_tc(moe_plan* p, const void* recv, const int* tile_expert, const void* wg,
                  const void* wu, const void* wd, void* out_rows, const int* tile_count,
                  const int* rows_done, cudaStream_t st, const void* overlap_x = nullptr,
                  const int* overlap_idx = nullptr, const int* push_src = nullptr);

// ---- element helpers ---------------------------------------------------------------------------
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

// Unpack one 16-byte vector of T into floats (4 for fp32, 8 for bf16).
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                      __float_as_uint(f[3]));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ uint4 pack(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// Programmatic dependent launch: the kernels of the layer (all but the first, the router: starting
// it while the previous layer call drains measured slower) are launched so that they may start while
// their predecessor in the stream is still draining.  pdl_wait() blocks until the predecessor has
// completed and its writes are visible; nothing before it may touch global memory.  pdl_trigger()
// lets the successor begin launching.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

}  // namespace moehub
