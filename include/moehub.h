/*
 * moehub.h — C ABI of the B200 (sm_100a) MoE-layer hot path.
 *
 * The path is the five-step MoE layer of Section II-A of the paper "MoE-Hub" (routing,
 * all-to-all dispatch, expert computation, all-to-all combine, scaling) on ONE GPU, where the
 * E experts are partitioned over R logical expert-parallel ranks that are buffer partitions
 * only (expert e lives on rank e / (E/R)).  The paper's destination-agnostic dispatch
 * (Section IV-A/IV-B: a producer sends a row as soon as its expert id is known and the consumer
 * side hands out the next free row of that expert's region, address =
 * BaseAddr + LocalRowID*RowSize + RowOffset) is realised in software: slot allocation by
 * aggregated atomics on per-expert row pointers.  The conventional "software mediation"
 * (Section III-A: counts -> scan -> offsets -> shuffle) is kept as dispatch mode 0, the
 * baseline it is shown against.
 *
 * General rules
 *  - Every pointer named d_* is DEVICE memory owned by the caller; h_* is HOST memory.  The
 *    library allocates no device memory: its scratch is the caller's workspace (see
 *    moe_workspace_bytes / moe_plan_create).  A plan owns host-side metadata only.  The one
 *    exception to this rule and to "no global state" below is moe_dispatch_noalloc, which keeps
 *    its scratch in a device array that is part of the library image (see its declaration).
 *  - dtype 0: fp32, dtype 1: bf16.  It is the type of x, the router weight, the expert
 *    weights, the receive buffers, the expert outputs and y.  Routing weights are fp32,
 *    indices int32.  All matrices are row-major and dense.
 *  - Alignment: H*elem and F*elem must be multiples of 16 bytes; device pointers must be
 *    16-byte aligned (cudaMalloc / torch allocations are).
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default
 *    stream).  Return value: 0 = MOE_OK, negative = error found on the host before anything
 *    was launched.  Errors found on the device (region overflow, a bounded wait that ran out,
 *    an expert id outside [0, E) in a caller-supplied topk_idx) are left in a device status
 *    word: read it with moe_last_status.
 *  - A plan is used by one host thread / one stream at a time.  No global state.
 *  - Receive-buffer geometry: rows live in a pool of P tiles of 128 rows
 *    (moe_pool_tiles).  tile_expert[p] names the expert that owns tile p (-1: unused).  An
 *    expert's rows are dense inside its tiles (only its last tile may be partly filled).
 *    Physical row = tile*128 + row-in-tile.  Within one expert the order of rows is
 *    unspecified in the atomic modes (arrival order, Section IV-B) and is (token, k) order in
 *    mode 0.  In mode 3 an expert's tiles are consecutive pool tiles, experts in ascending order.
 */
#ifndef MOEHUB_H_
#define MOEHUB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOE_OK 0
#define MOE_ERR_ARG (-1)         /* null pointer, non-positive size, K > E, E % R != 0, ... */
#define MOE_ERR_ALIGN (-2)       /* H or F row pitch not a multiple of 16 bytes, misaligned pointer */
#define MOE_ERR_UNSUPPORTED (-3) /* outside what the kernels cover (E > 256, K > 32, ...) */
#define MOE_ERR_CUDA (-4)        /* a CUDA runtime/driver call failed */
#define MOE_ERR_OVERFLOW (-5)    /* device status: an expert's region (mode 1) or the pool is full */
#define MOE_ERR_TIMEOUT (-6)     /* device status: a bounded device-side wait ran out */
#define MOE_ERR_WORKSPACE (-7)   /* workspace too small or misaligned */
#define MOE_ERR_TOO_LARGE (-8)   /* moe_dispatch_noalloc: T or E beyond its fixed built-in scratch */
#define MOE_ERR_INTERNAL (-9)    /* device status: a kernel's own index check failed (the access was
                                    skipped); detail names the check */

#define MOE_DTYPE_FP32 0
#define MOE_DTYPE_BF16 1

#define MOE_DISPATCH_SCAN 0          /* baseline: histogram -> exclusive scan -> stable scatter */
#define MOE_DISPATCH_ATOMIC_STATIC 1 /* row-pointer atomics, one static region per expert   */
#define MOE_DISPATCH_ATOMIC_PAGED 2  /* row-pointer atomics, 128-row tiles paged on demand  */
#define MOE_DISPATCH_ATOMIC_ORDERED 3 /* row-pointer atomics; persistent CTAs emit the tokens in one
                                        ascending order (Section IV-C: smallest RowID first), regions
                                        sized by the rows per expert that the router counted, rows
                                        moved by bulk asynchronous copies                           */

#define MOE_TILE_ROWS 128

typedef struct moe_plan moe_plan_t; /* opaque */

typedef struct {
  int32_t T, H, E, R, K, F;     /* tokens, hidden, experts, logical ranks, top-K, FFN width   */
  int32_t dtype;                /* MOE_DTYPE_*                                               */
  int32_t renormalize;          /* 0: w = softmax prob. of the picked experts; 1: / their sum */
  int32_t dispatch_mode;        /* MOE_DISPATCH_*                                            */
  int32_t identity_experts;     /* 1: moe_layer skips the FFN (expert output = expert input)  */
  int32_t ffn_kernel;           /* 0: tensor-core (tcgen05) kernel, one CTA per tile, for bf16,
                                   SIMT for fp32; 1: SIMT fp32-FMA kernel for either dtype
                                   (check path); 2: tensor-core kernel on CTA pairs
                                   (cta_group::2, two tiles per MMA; bf16)                    */
  int32_t ffn_split;            /* 1: one launch per expert GEMM; 2: both GEMMs in one persistent
                                   launch (per-tile status counters gate GEMM2); 0: choose
                                   (one launch when E <= 64; with more, smaller experts two
                                   launches measure faster)                                   */
  int32_t ffn_hot_min_tiles;    /* two-launch form of the tensor-core kernel: > 0 = experts with at
                                   least this many tiles count as tensor-bound, the others as
                                   bound by streaming their weights, and the kernel walks the two
                                   kinds of work interleaved; 0 (default) = one expert after the
                                   other                                                       */
  int32_t ffn_thin_tiles;       /* tensor-core kernel: 0 = an expert's only tile, if it holds at
                                   most 64 rows, is computed in the transposed narrow form;
                                   negative = never (such a tile runs M = 64 MMAs instead)      */
  int32_t overlap;              /* moe_layer, dispatch mode 3, bf16, tensor-core kernel: != 0 =
                                   dispatch and expert computation in ONE launch: n producer CTAs
                                   (1: half as many as SMs, n > 1: n) only dispatch, and as many
                                   consumer CTAs as there are SMs compute every tile as soon as
                                   its status counter has reached its threshold (Section IV-D);
                                   negative: the same launch, but the consumers wait for the whole
                                   dispatch (for comparison); 0 = stream-ordered launches        */
  int32_t combine_mode;         /* moe_layer: 0 = gather (the combine kernel fetches every token's K
                                   expert rows from the pool through slot_of); 1 = push (Section
                                   IV-B, all-to-all combine: the expert kernel's final epilogue
                                   reads each row's source information and stores the result at
                                   the token's own position [t*K+k], the combine kernel then reads
                                   K consecutive rows per token).  Push needs bf16 and the
                                   one-CTA-per-tile tensor-core kernel (ffn_kernel 0)            */
  int32_t tp_shards;            /* expert + tensor parallelism (Section VII): S > 1 cuts every expert's
                                   FFN into S slices of its width F (gate/up rows [s*F/S, (s+1)*F/S),
                                   the matching columns of the down matrix), gives every slice a
                                   receive region of its own (one registration per TP shard) and
                                   stores every row to all S of them.  Every stage then sees E*S
                                   experts and K*S assignments per token: topk_idx / topk_w /
                                   slot_of are [T, K*S] with entry k*S+s = (expert*S + s, the
                                   pick's weight), expert_count is [E*S], the pool has
                                   floor(T*K*S/128) + E*S tiles, and the combine step adds the
                                   K*S partial rows.  Needs F % S == 0, E*S <= 256, K*S <= 32;
                                   0 or 1 = none                                               */
  int32_t route_filter;         /* router with more than 64 experts on bf16 data: 0 = tensor-core filter
                                   (approximate logits by tcgen05 MMAs, then the exact fp32 chain only
                                   for the experts that can still be among the K largest: the picks
                                   are the exact ones, bit for bit); -1 = every chain computed        */
  int64_t capacity_rows;        /* mode 1: rows per expert region, multiple of 128, 0 = T
                                   rounded up (overflow-free); modes 0/2: ignored            */
  uint64_t spin_limit;          /* bound (iterations) on the dispatch kernels' waits, 0 = 1<<22 */
  uint64_t wait_limit_ns;       /* bound (nanoseconds) on every wait inside the tensor-core
                                   expert kernels, 0 = 2 s                                   */
} moe_config_t;

/* Number P of 128-row tiles in the receive pool for this configuration:
 * modes 0/2/3: floor(T*K/128) + E;  mode 1: E * capacity_rows/128. */
int moe_pool_tiles(const moe_config_t* cfg, int64_t* out_tiles);

/* Bytes of device workspace moe_plan_create needs (scratch counters, tile tables, the SwiGLU
 * intermediate, and the internal buffers moe_layer uses between its stages). */
int moe_workspace_bytes(const moe_config_t* cfg, size_t* out_bytes);

/* Analogue of the paper's rowspMalloc (Section IV-A, runtime API): registers the receive
 * regions (base, row size, tile pool) once.  d_workspace: device memory, 256-byte aligned,
 * at least moe_workspace_bytes() long, owned by the caller, must outlive the plan's queued
 * work.  Runs on the current CUDA device.  *out is freed by moe_plan_destroy. */
int moe_plan_create(const moe_config_t* cfg, void* d_workspace, size_t bytes, moe_plan_t** out);
int moe_plan_destroy(moe_plan_t* plan);

/* Step 1 (Section II-A, routing): logits l[t,e] = sum_h x[t,h]*Wr[e,h] (+bias[e]) as one
 * ascending fp32 FMA chain, softmax over the E experts, the K largest logits (lowest index
 * wins ties), in descending order.  (With more than 64 experts on bf16 data the chain is evaluated only for
 * the experts that a tensor-core pass and an error bound derived from the data leave in question; the picks are
 * those of the chains of all experts, bit for bit - see route_filter in moe_config_t.)
 * d_x [T,H], d_wr [E,H] (dtype); d_bias [E] fp32 or NULL;
 * out: d_topk_idx [T,K] int32, d_topk_w [T,K] fp32.
 * An empty batch (T = 0) is legal in every call of this header: the per-token pointers may then be NULL,
 * no kernel touches a row, and the dispatch outputs get their start state (counts 0, no tile owned). */
int moe_route(moe_plan_t* plan, const void* d_x, const void* d_wr, const float* d_bias,
              int32_t* d_topk_idx, float* d_topk_w, void* stream);

/* Step 2 (Section II-A dispatch; address resolution per Section III-A in mode 0, per
 * Section IV-B in modes 1/2): copies x[t,:] to one slot of each of its K experts.
 * in: d_x [T,H], d_topk_idx [T,K].
 * out: d_recv [P*128,H] (dtype; rows of unused slots are left untouched),
 *      d_expert_count [E] rows per expert, d_tile_expert [P] owner of each tile or -1,
 *      d_src_info [P*128] = t*K+k of the row in that slot, -1 for an empty slot (the source
 *      information of Section IV-B, combine), d_slot_of [T,K] physical row of assignment
 *      (t,k), or -1 if it was dropped by an overflow (status MOE_ERR_OVERFLOW) or because
 *      topk_idx[t,k] is not in [0, E) (status MOE_ERR_ARG, detail = the token; no table is
 *      indexed with such an id and the assignment's row is not stored);
 *      availability counters (Section IV-D, data availability manager), both or neither,
 *      NULL = kept in the plan's workspace: d_tile_count [P] rows stored so far in each tile,
 *      d_rows_done [1] assignments whose rows are stored; both raised with release semantics
 *      after the rows they count are written, so a consumer that reads tile_count[p] >= 128
 *      or rows_done == T*K with acquire semantics may read the tile. */
int moe_dispatch(moe_plan_t* plan, const void* d_x, const int32_t* d_topk_idx, void* d_recv,
                 int32_t* d_expert_count, int32_t* d_tile_expert, int32_t* d_src_info,
                 int32_t* d_slot_of, int32_t* d_tile_count, int32_t* d_rows_done, void* stream);

/* Step 3 (Section II-A, expert computation: two GEMMs with an activation between them, here
 * SwiGLU): for every used tile p of expert e = tile_expert[p]:
 *   S = silu(A*Wg[e]^T) .* (A*Wu[e]^T),  O = S*Wd[e]^T,  A = the tile's 128 rows of d_recv.
 * Unused tiles are skipped and their experts' weights never read (Section IV-D: thread
 * blocks whose counters stay zero are never scheduled).
 * in: d_recv [P*128,H], d_tile_expert [P], d_wg/d_wu [E,F,H], d_wd [E,H,F] (dtype);
 *     d_tile_count [P], d_rows_done [1]: the availability counters of moe_dispatch, both or
 *     neither.  When given, the tensor-core kernel waits before it reads a tile until
 *     tile_count[p] >= 128 or rows_done >= T*K (bounded by wait_limit_ns; on expiry the status
 *     word reads MOE_ERR_TIMEOUT and the kernel returns).  NULL: the rows are complete when the
 *     call is reached in stream order.  The SIMT kernel ignores them (stream order).  The
 *     counters also tell the kernel how many rows a tile holds: with them, an expert whose only
 *     tile holds at most 64 rows is computed in a narrower form (same result, less work);
 *     without them every tile is computed as 128 rows.
 * out: d_out_rows [P*128,H] (dtype); rows of empty slots hold unspecified values.
 * The tensor-core kernels keep their work list in shared memory: P <= 4608 tiles (T*K <= 557 056 rows at
 * E = 256), MOE_ERR_UNSUPPORTED beyond. */
int moe_expert_ffn(moe_plan_t* plan, const void* d_recv, const int32_t* d_tile_expert,
                   const void* d_wg, const void* d_wu, const void* d_wd, void* d_out_rows,
                   const int32_t* d_tile_count, const int32_t* d_rows_done, void* stream);

/* Dispatch without any allocation (the paper has no counterpart: this entry point exists for
 * the callers described here, not for a step of the method).  Some callers cannot give this
 * library a workspace because they cannot allocate device memory at the point of the call: a
 * serving process that handed the whole GPU to its own pool at start-up, a plug-in that has no
 * access to its host's allocator, a latency-critical loop that must not risk the device-wide
 * synchronisation an allocation can cause.  For them this variant of moe_dispatch keeps its
 * scratch (pool cursor + tile table, about 129 KB) in a fixed device array built into the
 * library; every GPU that loads the library holds that array until the process exits.  It takes
 * no plan, calls no cudaMalloc/cudaFree or any other allocating routine, and always uses the
 * paged destination-agnostic scheme (cfg->dispatch_mode, capacity_rows and F are ignored).
 *
 * Limits: T <= MOE_NOALLOC_MAX_TOKENS and E <= 256, otherwise MOE_ERR_TOO_LARGE is returned and
 * nothing is launched.  Arguments and outputs are those of moe_dispatch, with the pool size
 * P = floor(T*K/128) + E, plus d_status: [2] int32 in device memory owned by the caller, which
 * receives the device status (code, detail) that moe_last_status would report.
 *
 * The first call on each device looks up the array's device address (that device must be
 * current); make that first call outside any stream capture.  With the CUDA runtime's lazy module
 * loading, that first call (or the first kernel of this library on the device) is also when the
 * driver loads the library's device image and places the array, so "allocates nothing" holds from
 * the second call on: issue one warm-up call at start-up, while allocation is still permitted.  All calls on a device share the
 * one array, which still holds the previous call's contents: each call clears what it needs on
 * `stream` before its kernel, so calls issued to the same stream are safe back to back, but two
 * calls that can overlap on the GPU (different streams, no dependency) race on it. */
#define MOE_NOALLOC_MAX_TOKENS 16384
int moe_dispatch_noalloc(const moe_config_t* cfg, const void* d_x, const int32_t* d_topk_idx,
                         void* d_recv, int32_t* d_expert_count, int32_t* d_tile_expert,
                         int32_t* d_src_info, int32_t* d_slot_of, int32_t* d_status, void* stream);

/* Step 3 with the push-style return of Section IV-B (all-to-all combine: the expert reads the source
 * information that travelled with each row and stores its output at the row's origin): as
 * moe_expert_ffn, but the result of the row in pool slot r goes to d_staged[d_src_info[r], :] - the
 * position t*K+k of its assignment - and slots whose source is -1 produce nothing.
 * in: as moe_expert_ffn, plus d_src_info [P*128] from moe_dispatch.  out: d_staged [T*K,H] (dtype);
 * rows of dropped assignments keep their old contents.  bf16 with ffn_kernel 0 only
 * (MOE_ERR_UNSUPPORTED otherwise). */
int moe_expert_ffn_push(moe_plan_t* plan, const void* d_recv, const int32_t* d_tile_expert,
                        const int32_t* d_src_info, const void* d_wg, const void* d_wu, const void* d_wd,
                        void* d_staged, const int32_t* d_tile_count, const int32_t* d_rows_done, void* stream);

/* Steps 4+5 after moe_expert_ffn_push: y[t,:] = sum_k w[t,k]*staged[t*K+k,:], k ascending, fp32
 * accumulation, one rounding: the same arithmetic as moe_combine, hence the same bytes in y.
 * d_slot_of is only looked at to skip dropped assignments (slot -1). */
int moe_combine_staged(moe_plan_t* plan, const void* d_staged, const int32_t* d_slot_of,
                       const float* d_topk_w, void* d_y, void* stream);

/* Dispatch across GPUs - real expert parallelism, the paper's own setting (Section III-B: producers send
 * without knowing the destination's layout; Section IV-B: the CONSUMER's allocation pointers hand out the
 * rows).  Rank r of cfg->R holds cfg->T tokens (its share of the batch) and the experts
 * [r*E/R, (r+1)*E/R); cfg->E counts all experts.  Every rank owns, in its own memory, one static region of
 * cap_rows rows per local expert plus the counters below, and makes them reachable by the other ranks
 * (CUDA IPC, a symmetric-memory allocator, or - on one GPU - plain local pointers).  The call dispatches THIS
 * rank's tokens: for every token block one system-scope atomicAdd per touched expert on the owner's
 * row_pointer, the rows by plain 16-byte stores into the owner's region, then system-scope release
 * increments of the owner's tile and global counters.  Nothing but ordinary loads, stores and atomics
 * touches another GPU's memory (no TMA, no bulk copy, no multicast, no library kernel), and the kernel waits
 * for nobody, so no two ranks need to run at the same time.
 *
 * Before any rank dispatches, every rank clears ITS OWN row_pointer, tile_count and rows_done and fills its
 * src_info with -1, and the ranks synchronise (host barrier or events): that start state is the caller's job.
 * h_peers: HOST array [R] of device pointers valid on the calling GPU, entry r describing rank r's buffers:
 *   recv [E/R * cap_rows, H] (dtype), row_pointer [E/R], tile_count [E/R * cap_rows/128],
 *   src_info [E/R * cap_rows] (receives (source rank * T + t) * K + k), rows_done [1] (assignments addressed
 *   to this rank, dropped ones included).
 * cap_rows: multiple of 128; an assignment beyond it is dropped and reported (MOE_ERR_OVERFLOW).
 * out: d_slot_of [T,K] = owner rank * (E/R * cap_rows) + row in the owner's regions, or -1;
 *      d_status [2] device status (code, detail) of this call.
 * Limits: R <= MOE_EP_MAX_RANKS, E <= 256, K <= 32.  Not yet measured on more than one GPU. */
#define MOE_EP_MAX_RANKS 32
typedef struct {
  void* recv;
  int32_t* row_pointer;
  int32_t* tile_count;
  int32_t* src_info;
  int32_t* rows_done;
} moe_ep_peer_t;
int moe_dispatch_ep(const moe_config_t* cfg, int32_t rank, const moe_ep_peer_t* h_peers, int64_t cap_rows,
                    const void* d_x, const int32_t* d_topk_idx, int32_t* d_slot_of, int32_t* d_status,
                    void* stream);

/* After every rank's moe_dispatch_ep has completed (host barrier): the owner's tile table from its allocation
 * pointers, in the form moe_expert_ffn takes for static regions of cap_rows rows - expert e of this rank holds
 * min(row_pointer[e], cap_rows) rows in the first tiles of region e, the region's other tiles are unused.
 * in: d_row_pointer [experts_local].  out: d_expert_count [experts_local], d_tile_expert
 * [experts_local * cap_rows/128] (local expert index, or -1).  One small launch on `stream`. */
int moe_ep_tiles(int32_t experts_local, int64_t cap_rows, const int32_t* d_row_pointer,
                 int32_t* d_expert_count, int32_t* d_tile_expert, void* stream);

/* The combine direction across GPUs (Section IV-B, all-to-all combine): the owner reads the source
 * information of every result row and stores the row at the token's own position - row t*K+k of the SOURCE
 * rank's staging buffer [T*K, H] - with plain 16-byte peer stores, then raises that rank's counter of returned
 * rows with a system-scope release add.  The source rank then runs moe_combine_staged on its staging buffer
 * (after a host barrier, or once rows_back has reached the number of its assignments that were not dropped).
 * cfg as for moe_dispatch_ep (T = tokens per rank, E = all experts).  h_staging, h_rows_back: HOST arrays [R]
 * of device pointers valid on the calling GPU (rank r's staging buffer; its int32 counter, zero before the
 * step).  in: d_out_rows [E/R * cap_rows, H] (this rank's expert outputs, same rows as its receive regions),
 * d_src_info [E/R * cap_rows], d_expert_count [E/R] (from moe_ep_tiles).  out: d_status [2]; a row without
 * valid source information is reported as MOE_ERR_INTERNAL and not sent.  Same rule as the dispatch: only
 * ordinary loads, stores and atomics touch peer memory, and the kernel waits for nobody.  Not yet measured on
 * more than one GPU. */
int moe_combine_ep(const moe_config_t* cfg, void* const* h_staging, int32_t* const* h_rows_back,
                   int64_t cap_rows, const void* d_out_rows, const int32_t* d_src_info,
                   const int32_t* d_expert_count, int32_t* d_status, void* stream);

/* Steps 4+5 (Section II-A, combine and scaling): y[t,:] = sum_k w[t,k]*rows[slot_of[t,k],:],
 * k ascending, fp32 accumulation, rounded once to dtype.  Assignments with slot -1 add 0.
 * in: d_rows [P*128,H] (dtype), d_slot_of [T,K], d_topk_w [T,K].  out: d_y [T,H] (dtype). */
int moe_combine(moe_plan_t* plan, const void* d_rows, const int32_t* d_slot_of,
                const float* d_topk_w, void* d_y, void* stream);

/* The whole layer, steps 1-5, on device buffers: route -> dispatch -> experts -> combine,
 * intermediate buffers in the plan's workspace. */
int moe_layer(moe_plan_t* plan, const void* d_x, const void* d_wr, const float* d_bias,
              const void* d_wg, const void* d_wu, const void* d_wd, void* d_y, void* stream);

/* The whole layer with the activations in HOST memory: copies h_x [T,H] to the device,
 * runs moe_layer, copies y back to h_y [T,H] and synchronises the stream.  Weights stay
 * device-resident (they are parameters, not per-step inputs).  Pinned host memory makes the
 * copies asynchronous to the host but the call still returns only when h_y is complete. */
int moe_layer_host(moe_plan_t* plan, const void* h_x, const void* d_wr, const float* d_bias,
                   const void* d_wg, const void* d_wu, const void* d_wd, void* h_y, void* stream);

/* Pipelined form of moe_layer_host for a stream of batches.  submit() enqueues one step and returns
 * at once with a ticket: the copy of h_x goes to a copy-in stream, the layer to `stream`, the copy of
 * y to a copy-out stream, chained by events, with two sets of staging buffers, so that step n+1's
 * host-to-device copy and step n-1's device-to-host copy run under step n's kernels.  wait(ticket)
 * blocks the host until that step's h_y is complete.  Keep at most two steps in flight (wait for
 * ticket n-1 before submitting n+1), leave h_x and h_y alone until their step is waited for, and use
 * pinned host memory: pageable memory makes the copies synchronous.  Device errors: moe_last_status. */
int moe_layer_host_submit(moe_plan_t* plan, const void* h_x, const void* d_wr, const float* d_bias,
                          const void* d_wg, const void* d_wu, const void* d_wd, void* h_y, void* stream,
                          int64_t* ticket);
int moe_layer_host_wait(moe_plan_t* plan, int64_t ticket);

/* moe_layer with a CUDA event recorded after every kernel: runs the layer once, synchronises the
 * stream and writes the device time of each stage, in milliseconds, to h_stage_ms
 * [MOE_STAGE_COUNT] (host): route, dispatch (all its kernels and counter resets), FFN set-up (host-side
 * descriptor encoding only: the work list is built inside the expert kernel), FFN GEMM1 (+SwiGLU), FFN GEMM2,
 * combine.  With ffn_split = 0 both GEMMs are one launch: its
 * time is reported under GEMM1 and GEMM2 reads 0.  For measurement only. */
#define MOE_STAGE_ROUTE 0
#define MOE_STAGE_DISPATCH 1
#define MOE_STAGE_WORKLIST 2
#define MOE_STAGE_GEMM1 3
#define MOE_STAGE_GEMM2 4
#define MOE_STAGE_COMBINE 5
#define MOE_STAGE_COUNT 6
int moe_layer_timed(moe_plan_t* plan, const void* d_x, const void* d_wr, const float* d_bias,
                    const void* d_wg, const void* d_wu, const void* d_wd, void* d_y, void* stream,
                    float* h_stage_ms);

/* Device pointers of moe_layer's intermediate results inside the workspace (valid after a
 * moe_layer call completes): which = 0 topk_idx, 1 topk_w, 2 recv, 3 expert_count,
 * 4 tile_expert, 5 src_info, 6 slot_of, 7 out_rows, 8 the availability trace, 9 the work-item
 * timeline (both below). */
int moe_layer_buffer(moe_plan_t* plan, int which, void** out_ptr);

/* Availability trace (Section IV-D: when does a consumer learn that a tile is ready), for
 * measurement.  While enabled, the dispatch kernels of this plan (moe_dispatch, moe_layer) raise the
 * availability counters with value-returning atomics and write %globaltimer nanoseconds into a
 * uint64 array [P + 2] in the workspace (moe_layer_buffer, which = 8): [0] the earliest start of a
 * dispatch CTA, [1] the moment the global counter reached all T*K assignments, [2 + p] the moment
 * tile p's counter reached 128 rows (0: the tile never filled).  Disabled (the default) the kernels
 * are unchanged.  The flag is host-side state of the plan.
 * While enabled, the tensor-core expert kernel (one CTA per tile, bf16) also writes a timeline of its
 * work items: uint64 [P * (ceil(F/128) + ceil(H/256))][4] (moe_layer_buffer, which = 9), one entry
 * per position of its item list in the order the items were claimed: [0] the moment the item's
 * producer had seen its tile ready and began to load, [1] the moment its MMAs were complete, [2] what
 * it was (bit 0: 0 = GEMM1 block, 1 = GEMM2 block; bit 1: an expert bound by streaming its weights;
 * bits 2-5 the narrow form used; bits 8-23 expert, 24-31 column block, 32-51 tile, 52-63 SM),
 * [3] the moment its last load was issued.  Entries of positions that were not claimed keep their
 * old contents. */
int moe_availability_trace(moe_plan_t* plan, int enable);

/* Effective SM clock inside the tensor-core expert kernels since the last reset: one CTA of every
 * launch accumulates its elapsed SM cycles and nanoseconds; *out_mhz = cycles / time (0 if none ran).
 * Synchronises `stream` when out_mhz is given; reset != 0 clears the accumulators afterwards.
 * For measurement: tells a kernel slowed by a power-capped clock from one that waits for data. */
int moe_ffn_clock_mhz(moe_plan_t* plan, void* stream, int reset, float* out_mhz);

/* Number of kernels the last stage call (or moe_layer) launched. */
int moe_last_launch_count(moe_plan_t* plan, int32_t* out);

/* Synchronises `stream` and reads the device status word: *code is MOE_OK, MOE_ERR_OVERFLOW,
 * MOE_ERR_TIMEOUT or MOE_ERR_ARG; *detail says where (expert id for an overflow, wait site for
 * a timeout, token index for an expert id outside [0, E)).  The first error of a call wins. */
int moe_last_status(moe_plan_t* plan, void* stream, int32_t* code, int32_t* detail);

/* After moe_layer returned MOE_ERR_CUDA: which of its steps met the CUDA error (1 router, 2 dispatch,
 * 3 experts, 4 combine; 0: none so far) and the error's name as the CUDA runtime spells it (a static
 * string).  Kernel launches are asynchronous, so an error raised while a kernel RUNS is reported by a
 * later step (or by the next synchronising call) unless launches are made blocking. */
int moe_last_cuda_error(moe_plan_t* plan, int32_t* step, const char** name);

const char* moe_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MOEHUB_H_ */
