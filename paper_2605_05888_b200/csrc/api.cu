// The C ABI declared in include/moehub.h: argument checks, workspace carving, stage launches.
// No device memory is allocated here; every buffer is the caller's.
#include <new>
#include <string.h>

#include "common.cuh"

using namespace moehub;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Geometry {
  moe_config_t eff;  // the effective configuration (TP shards folded into E, K and F: see moe_plan)
  int tp;
  int64_t P, cap_rows;
  int tiles_per_expert, dispatch_tokens, nblk, eb;
  int ord_tokens, ord_nblk;
};

int check_config(const moe_config_t* user, Geometry* g) {
  if (!user) return MOE_ERR_ARG;
  if (user->T < 0 || user->H <= 0 || user->E <= 0 || user->R <= 0 || user->K <= 0) return MOE_ERR_ARG;
  if (user->K > user->E || user->E % user->R != 0) return MOE_ERR_ARG;
  // Expert + tensor parallelism (paper Section VII): an expert's FFN is cut into tp_shards slices of its
  // width F, every slice has a receive region of its own and every row is stored to all of them.  From
  // here on shard s of expert e is the virtual expert e*S + s of a layer with E*S experts, K*S picks per
  // token and FFN width F/S (SwiGLU and the down projection are sums over F, so the S partial results of a
  // pick add up to the expert's output; the combine step adds them with the pick's weight).
  const int tp = user->tp_shards > 1 ? user->tp_shards : 1;
  if (user->tp_shards < 0) return MOE_ERR_ARG;
  if (tp > 1 && (user->identity_experts || user->F % tp != 0)) return MOE_ERR_ARG;
  if (tp > 1 && user->ffn_kernel == 2) return MOE_ERR_UNSUPPORTED;
  g->eff = *user;
  g->eff.E = user->E * tp;
  g->eff.K = user->K * tp;
  if (!user->identity_experts) g->eff.F = user->F / tp;
  g->eff.R = user->R;  // a rank keeps its experts' shards: E*S % R == 0 follows
  g->tp = tp;
  const moe_config_t* c = &g->eff;
  if (c->dtype != MOE_DTYPE_FP32 && c->dtype != MOE_DTYPE_BF16) return MOE_ERR_ARG;
  if (c->dispatch_mode < 0 || c->dispatch_mode > 3) return MOE_ERR_ARG;
  if (!c->identity_experts && c->F <= 0) return MOE_ERR_ARG;
  if (c->E > 256 || c->K > 32) return MOE_ERR_UNSUPPORTED;
  if (c->combine_mode < 0 || c->combine_mode > 1) return MOE_ERR_ARG;
  if (c->route_filter < -1 || c->route_filter > 0) return MOE_ERR_ARG;
  if (c->combine_mode == 1 && (c->dtype != MOE_DTYPE_BF16 || c->ffn_kernel != 0 || c->identity_experts))
    return MOE_ERR_UNSUPPORTED;
  const int eb = c->dtype == MOE_DTYPE_BF16 ? 2 : 4;
  if (((int64_t)c->H * eb) % 16 != 0) return MOE_ERR_ALIGN;
  if (!c->identity_experts && ((int64_t)c->F * eb) % 16 != 0) return MOE_ERR_ALIGN;
  if ((int64_t)c->T * c->K >= (1ll << 31) / 2) return MOE_ERR_UNSUPPORTED;
  g->eb = eb;
  const int64_t rows = (int64_t)c->T * c->K;
  if (c->dispatch_mode == MOE_DISPATCH_ATOMIC_STATIC) {
    int64_t cap = c->capacity_rows > 0 ? c->capacity_rows : (c->T + kTileRows - 1) / kTileRows * kTileRows;
    if (cap % kTileRows != 0) return MOE_ERR_ARG;
    if (cap == 0) cap = kTileRows;
    g->cap_rows = cap;
    g->P = (int64_t)c->E * (cap / kTileRows);
  } else {
    g->cap_rows = 0;
    g->P = rows / kTileRows + c->E;
  }
  if (g->P * kTileRows >= (1ll << 31)) return MOE_ERR_UNSUPPORTED;
  g->tiles_per_expert = (c->T + kTileRows - 1) / kTileRows;
  if (g->tiles_per_expert == 0) g->tiles_per_expert = 1;
  int tpb = 256 / c->K;  // at most 256 assignments per dispatch CTA
  if (tpb > 16) tpb = 16;
  if (tpb < 1) tpb = 1;
  while (tpb > 1 && (c->T + tpb - 1) / tpb < 2 * 148) tpb /= 2;  // small batches: enough CTAs to fill the GPU
  g->dispatch_tokens = tpb;
  g->nblk = (c->T + tpb - 1) / tpb;
  // ordered dispatch: at most 128 assignments per token block, smaller blocks while there are fewer blocks than SMs
  int otb = 128 / c->K;
  // Stream-ordered launches: 16-token blocks (fastest: 0.80 of the copy rate on the DeepSeek-like layer).  The
  // overlapped launch: 4-token blocks, so that the token order is followed more closely and the first tiles are
  // complete after a tenth of the dispatch (with 16: a fifth) - there a consumer is waiting for them.
  const int otb_cap = c->overlap != 0 ? 4 : 16;
  if (otb > otb_cap) otb = otb_cap;
  if (otb < 1) otb = 1;
  while (otb > 1 && (c->T + otb - 1) / otb < 148) otb /= 2;
  g->ord_tokens = otb;
  g->ord_nblk = (c->T + otb - 1) / otb;
  return MOE_OK;
}

// Lays the scratch out in the workspace; with base == nullptr only measures it.
size_t carve(const moe_config_t& c, const Geometry& g, char* base, Scratch* s, size_t* counters_bytes) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    char* ptr = base ? base + off : nullptr;
    off += align_up(bytes);
    return ptr;
  };
  Scratch t;
  memset(&t, 0, sizeof t);
  // leading block, cleared by every dispatch: status, pool_next, scan_ticket, rows_done
  t.status = (int*)take(sizeof(int) * 4);
  t.pool_next = (int*)take(sizeof(int));
  t.scan_ticket = (int*)take(sizeof(int));
  t.rows_done = (int*)take(sizeof(int));
  if (counters_bytes) *counters_bytes = off;
  t.tile_count = (int*)take(sizeof(int) * (size_t)(g.P > 0 ? g.P : 1));
  t.tile_table = (int*)take(sizeof(int) * (size_t)c.E * g.tiles_per_expert);
  t.cta_count = (int*)take(sizeof(int) * (size_t)(g.nblk > 0 ? g.nblk : 1) * c.E);
  t.cta_base = (int*)take(sizeof(int) * (size_t)(g.nblk > 0 ? g.nblk : 1) * c.E);
  t.tile_base = (int*)take(sizeof(int) * (size_t)(c.E + 1));
  t.hist = (int*)take(sizeof(int) * (size_t)c.E);
  t.row_pointer = (int*)take(sizeof(int) * (size_t)c.E);
  t.ord_exit = (int*)take(sizeof(int) * 2);
  t.clock_probe = (unsigned long long*)take(sizeof(unsigned long long) * 2);
  t.avail_ns = (unsigned long long*)take(sizeof(unsigned long long) * (size_t)((g.P > 0 ? g.P : 1) + 2));
  if (!c.identity_experts && c.dtype == MOE_DTYPE_BF16) {
    const size_t items = (size_t)(g.P > 0 ? g.P : 1) * ((c.F + 127) / 128 + (c.H + 255) / 256);
    t.item_ns = (unsigned long long*)take(sizeof(unsigned long long) * 4 * items);
  }
  t.gemm1_done = (int*)take(sizeof(int) * (size_t)((g.P > 0 ? g.P : 1) + 4));  // + the expert kernel's item and exit counters
  const size_t pool_rows = (size_t)g.P * kTileRows;
  if (!c.identity_experts) t.inter = take(pool_rows * c.F * g.eb);
  const bool filter = c.dtype == MOE_DTYPE_BF16 && c.E / g.tp > 64 && c.route_filter >= 0;  // c.E counts every TP shard
  t.route_logits = filter ? (float*)take(sizeof(float) * (size_t)(c.T > 0 ? c.T : 1) * 256) : nullptr;
  t.route_wnorm2 = filter ? (float*)take(sizeof(float) * 256) : nullptr;
  t.topk_idx = (int*)take(sizeof(int) * (size_t)c.T * c.K);
  t.topk_w = (float*)take(sizeof(float) * (size_t)c.T * c.K);
  t.recv = take(pool_rows * c.H * g.eb);
  t.out_rows = c.identity_experts ? t.recv : take(pool_rows * c.H * g.eb);
  t.expert_count = (int*)take(sizeof(int) * (size_t)c.E);
  t.tile_expert = (int*)take(sizeof(int) * (size_t)g.P);
  t.src_info = (int*)take(sizeof(int) * pool_rows);
  t.slot_of = (int*)take(sizeof(int) * (size_t)c.T * c.K);
  for (int b = 0; b < 2; ++b) {
    t.x_stage[b] = take((size_t)c.T * c.H * g.eb);
    t.y_stage[b] = take((size_t)c.T * c.H * g.eb);
  }
  if (s) *s = t;
  return off;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

}  // namespace

extern "C" {

int moe_pool_tiles(const moe_config_t* cfg, int64_t* out_tiles) {
  Geometry g;
  if (!out_tiles) return MOE_ERR_ARG;
  int rc = check_config(cfg, &g);
  if (rc != MOE_OK) return rc;
  *out_tiles = g.P;
  return MOE_OK;
}

int moe_workspace_bytes(const moe_config_t* cfg, size_t* out_bytes) {
  Geometry g;
  if (!out_bytes) return MOE_ERR_ARG;
  int rc = check_config(cfg, &g);
  if (rc != MOE_OK) return rc;
  *out_bytes = carve(g.eff, g, nullptr, nullptr, nullptr);
  return MOE_OK;
}

int moe_plan_create(const moe_config_t* cfg, void* d_workspace, size_t bytes, moe_plan_t** out) {
  Geometry g;
  if (!out) return MOE_ERR_ARG;
  *out = nullptr;
  int rc = check_config(cfg, &g);
  if (rc != MOE_OK) return rc;
  if (!d_workspace) return MOE_ERR_ARG;
  if (reinterpret_cast<uintptr_t>(d_workspace) % kAlign != 0) return MOE_ERR_WORKSPACE;
  if (bytes < carve(g.eff, g, nullptr, nullptr, nullptr)) return MOE_ERR_WORKSPACE;
  moe_plan* p = new (std::nothrow) moe_plan();
  if (!p) return MOE_ERR_ARG;
  p->cfg = g.eff;
  p->tp = g.tp;
  p->route_E = cfg->E;
  p->route_K = cfg->K;
  p->P = g.P;
  p->cap_rows = g.cap_rows;
  p->tiles_per_expert = g.tiles_per_expert;
  p->dispatch_tokens = g.dispatch_tokens;
  p->nblk = g.nblk;
  p->ord_tokens = g.ord_tokens;
  p->ord_nblk = g.ord_nblk;
  p->launches = 0;
  p->cuda_error = 0;
  p->cuda_error_step = 0;
  p->encode_tiled = nullptr;
  p->timing = 0;
  for (int i = 0; i <= MOE_STAGE_COUNT; ++i) p->tev[i] = nullptr;
  p->copy_in = p->copy_out = nullptr;
  p->submitted = 0;
  for (int b = 0; b < 2; ++b) p->ev_in[b] = p->ev_done[b] = p->ev_out[b] = nullptr;
  carve(g.eff, g, (char*)d_workspace, &p->s, &p->counters_bytes);
  if (cudaGetDevice(&p->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device) != cudaSuccess) {
    delete p;
    return MOE_ERR_CUDA;
  }
  // The status word must start clean even if a stage other than dispatch is called first.
  if (cudaMemset(p->s.status, 0, p->counters_bytes) != cudaSuccess ||
      cudaMemset(p->s.hist, 0, sizeof(int) * (size_t)g.eff.E) != cudaSuccess ||
      cudaMemset(p->s.ord_exit, 0, sizeof(int) * 2) != cudaSuccess ||
      cudaMemset(p->s.gemm1_done, 0, sizeof(int) * (size_t)(g.P + 4)) != cudaSuccess ||
      cudaMemset(p->s.clock_probe, 0, 2 * sizeof(unsigned long long)) != cudaSuccess) {
    delete p;
    return MOE_ERR_CUDA;
  }
  *out = p;
  return MOE_OK;
}

int moe_plan_destroy(moe_plan_t* plan) {
  if (plan) {
    for (int i = 0; i <= MOE_STAGE_COUNT; ++i)
      if (plan->tev[i]) cudaEventDestroy(plan->tev[i]);
    for (int b = 0; b < 2; ++b) {
      if (plan->ev_in[b]) cudaEventDestroy(plan->ev_in[b]);
      if (plan->ev_done[b]) cudaEventDestroy(plan->ev_done[b]);
      if (plan->ev_out[b]) cudaEventDestroy(plan->ev_out[b]);
    }
    if (plan->copy_in) cudaStreamDestroy(plan->copy_in);
    if (plan->copy_out) cudaStreamDestroy(plan->copy_out);
  }
  delete plan;
  return MOE_OK;
}

int moe_route(moe_plan_t* p, const void* d_x, const void* d_wr, const float* d_bias, int32_t* d_topk_idx,
              float* d_topk_w, void* stream) {
  if (!p || !d_wr) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!d_x || !d_topk_idx || !d_topk_w)) return MOE_ERR_ARG;  // an empty batch has no rows to point at
  if (misaligned(d_x) || misaligned(d_wr)) return MOE_ERR_ALIGN;
  p->launches = 0;
  return launch_route(p, d_x, d_wr, d_bias, d_topk_idx, d_topk_w, nullptr, (cudaStream_t)stream) ? MOE_ERR_CUDA : MOE_OK;
}

int moe_dispatch(moe_plan_t* p, const void* d_x, const int32_t* d_topk_idx, void* d_recv,
                 int32_t* d_expert_count, int32_t* d_tile_expert, int32_t* d_src_info, int32_t* d_slot_of,
                 int32_t* d_tile_count, int32_t* d_rows_done, void* stream) {
  if (!p || !d_recv || !d_expert_count || !d_tile_expert || !d_src_info) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!d_x || !d_topk_idx || !d_slot_of)) return MOE_ERR_ARG;
  if (misaligned(d_x) || misaligned(d_recv)) return MOE_ERR_ALIGN;
  p->launches = 0;
  if ((d_tile_count == nullptr) != (d_rows_done == nullptr)) return MOE_ERR_ARG;
  return launch_dispatch(p, d_x, d_topk_idx, d_recv, d_expert_count, d_tile_expert, d_src_info, d_slot_of,
                         d_tile_count ? d_tile_count : p->s.tile_count, d_rows_done ? d_rows_done : p->s.rows_done,
                         false, (cudaStream_t)stream) ? MOE_ERR_CUDA : MOE_OK;
}

static int ffn_dispatch(moe_plan* p, const void* recv, const int* tile_expert, const void* wg, const void* wu,
                        const void* wd, void* out_rows, const int* tile_count, const int* rows_done,
                        cudaStream_t st) {
  if (p->cfg.dtype == MOE_DTYPE_BF16 && p->cfg.ffn_kernel != 1)
    return launch_ffn_tc(p, recv, tile_expert, wg, wu, wd, out_rows, tile_count, rows_done, st);
  return launch_ffn_simt(p, recv, tile_expert, wg, wu, wd, out_rows, st);
}

int moe_expert_ffn(moe_plan_t* p, const void* d_recv, const int32_t* d_tile_expert, const void* d_wg,
                   const void* d_wu, const void* d_wd, void* d_out_rows, const int32_t* d_tile_count,
                   const int32_t* d_rows_done, void* stream) {
  if (!p || !d_recv || !d_tile_expert || !d_wg || !d_wu || !d_wd || !d_out_rows) return MOE_ERR_ARG;
  if (p->cfg.identity_experts) return MOE_ERR_ARG;
  if (misaligned(d_recv) || misaligned(d_wg) || misaligned(d_wu) || misaligned(d_wd) || misaligned(d_out_rows))
    return MOE_ERR_ALIGN;
  p->launches = 0;
  if ((d_tile_count == nullptr) != (d_rows_done == nullptr)) return MOE_ERR_ARG;
  int rc = ffn_dispatch(p, d_recv, d_tile_expert, d_wg, d_wu, d_wd, d_out_rows, d_tile_count, d_rows_done,
                        (cudaStream_t)stream);
  return rc == 0 ? MOE_OK : (rc < 0 ? rc : MOE_ERR_CUDA);
}

int moe_expert_ffn_push(moe_plan_t* p, const void* d_recv, const int32_t* d_tile_expert, const int32_t* d_src_info,
                        const void* d_wg, const void* d_wu, const void* d_wd, void* d_staged,
                        const int32_t* d_tile_count, const int32_t* d_rows_done, void* stream) {
  if (!p || !d_recv || !d_tile_expert || !d_src_info || !d_wg || !d_wu || !d_wd || !d_staged) return MOE_ERR_ARG;
  if (p->cfg.identity_experts) return MOE_ERR_ARG;
  if (p->cfg.dtype != MOE_DTYPE_BF16 || p->cfg.ffn_kernel != 0) return MOE_ERR_UNSUPPORTED;
  if (misaligned(d_recv) || misaligned(d_wg) || misaligned(d_wu) || misaligned(d_wd) || misaligned(d_staged))
    return MOE_ERR_ALIGN;
  if ((d_tile_count == nullptr) != (d_rows_done == nullptr)) return MOE_ERR_ARG;
  p->launches = 0;
  int rc = launch_ffn_tc(p, d_recv, d_tile_expert, d_wg, d_wu, d_wd, d_staged, d_tile_count, d_rows_done,
                         (cudaStream_t)stream, nullptr, nullptr, d_src_info);
  return rc == 0 ? MOE_OK : (rc < 0 ? rc : MOE_ERR_CUDA);
}

int moe_combine_staged(moe_plan_t* p, const void* d_staged, const int32_t* d_slot_of, const float* d_topk_w, void* d_y,
                       void* stream) {
  if (!p) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!d_staged || !d_slot_of || !d_topk_w || !d_y)) return MOE_ERR_ARG;
  if (misaligned(d_staged) || misaligned(d_y)) return MOE_ERR_ALIGN;
  p->launches = 0;
  return launch_combine(p, d_staged, d_slot_of, d_topk_w, d_y, (cudaStream_t)stream, true) ? MOE_ERR_CUDA : MOE_OK;
}

int moe_combine(moe_plan_t* p, const void* d_rows, const int32_t* d_slot_of, const float* d_topk_w, void* d_y,
                void* stream) {
  if (!p) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!d_rows || !d_slot_of || !d_topk_w || !d_y)) return MOE_ERR_ARG;
  if (misaligned(d_rows) || misaligned(d_y)) return MOE_ERR_ALIGN;
  p->launches = 0;
  return launch_combine(p, d_rows, d_slot_of, d_topk_w, d_y, (cudaStream_t)stream) ? MOE_ERR_CUDA : MOE_OK;
}

int moe_layer(moe_plan_t* p, const void* d_x, const void* d_wr, const float* d_bias, const void* d_wg,
              const void* d_wu, const void* d_wd, void* d_y, void* stream) {
  if (!p || !d_wr) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!d_x || !d_y)) return MOE_ERR_ARG;
  if (!p->cfg.identity_experts && (!d_wg || !d_wu || !d_wd)) return MOE_ERR_ARG;
  if (misaligned(d_x) || misaligned(d_wr) || misaligned(d_wg) || misaligned(d_wu) || misaligned(d_wd) ||
      misaligned(d_y))
    return MOE_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  Scratch& s = p->s;
  p->launches = 0;
  mark(p, 0, st);
  // The router puts the dispatch's counters and tables into their start state on the side (and counts the
  // rows per expert for the ordered scheme), so no reset launch stands between it and the dispatch.
  const bool prepared = p->cfg.T > 0;
  const PrepArgs prep = make_prep(p, s.expert_count, s.tile_expert, s.src_info, s.tile_count, s.rows_done);
  auto cuda_failed = [&](int step) {
    p->cuda_error = (int)cudaGetLastError();
    p->cuda_error_step = step;
    return MOE_ERR_CUDA;
  };
  if (launch_route(p, d_x, d_wr, d_bias, s.topk_idx, s.topk_w, prepared ? &prep : nullptr, st)) return cuda_failed(1);
  mark(p, 1, st);
  // Overlapped form: the dispatch runs inside the expert kernel's launch (ordered scheme, tensor-core kernel).
  const moe_config_t& c = p->cfg;
  const bool overlap = c.overlap != 0 && prepared && c.dispatch_mode == MOE_DISPATCH_ATOMIC_ORDERED &&
                       !c.identity_experts && c.dtype == MOE_DTYPE_BF16 && c.ffn_kernel == 0;
  if (!overlap && launch_dispatch(p, d_x, s.topk_idx, s.recv, s.expert_count, s.tile_expert, s.src_info, s.slot_of,
                                  s.tile_count, s.rows_done, prepared, st))
    return cuda_failed(2);
  mark(p, 2, st);
  const bool push = c.combine_mode == 1;  // the expert kernel returns every row to its token's position itself
  if (overlap || push) {
    int rc = launch_ffn_tc(p, s.recv, s.tile_expert, d_wg, d_wu, d_wd, s.out_rows, s.tile_count, s.rows_done, st,
                           overlap ? d_x : nullptr, overlap ? s.topk_idx : nullptr, push ? s.src_info : nullptr);
    if (rc != 0) return rc < 0 && rc != MOE_ERR_CUDA ? rc : cuda_failed(3);
  } else if (!p->cfg.identity_experts) {
    int rc = ffn_dispatch(p, s.recv, s.tile_expert, d_wg, d_wu, d_wd, s.out_rows, s.tile_count, s.rows_done, st);
    if (rc != 0) return rc < 0 && rc != MOE_ERR_CUDA ? rc : cuda_failed(3);
  } else {
    mark(p, 3, st);
    mark(p, 4, st);
  }
  mark(p, 5, st);
  if (launch_combine(p, s.out_rows, s.slot_of, s.topk_w, d_y, st, push)) return cuda_failed(4);
  mark(p, 6, st);
  return MOE_OK;
}

int moe_last_cuda_error(moe_plan_t* p, int32_t* step, const char** name) {
  if (!p) return MOE_ERR_ARG;
  if (step) *step = p->cuda_error_step;
  if (name) *name = cudaGetErrorName((cudaError_t)p->cuda_error);
  return MOE_OK;
}

int moe_layer_timed(moe_plan_t* p, const void* d_x, const void* d_wr, const float* d_bias, const void* d_wg,
                    const void* d_wu, const void* d_wd, void* d_y, void* stream, float* h_stage_ms) {
  if (!p || !h_stage_ms) return MOE_ERR_ARG;
  for (int i = 0; i <= MOE_STAGE_COUNT; ++i)
    if (!p->tev[i] && cudaEventCreate(&p->tev[i]) != cudaSuccess) return MOE_ERR_CUDA;
  p->timing = 1;
  int rc = moe_layer(p, d_x, d_wr, d_bias, d_wg, d_wu, d_wd, d_y, stream);
  p->timing = 0;
  if (rc != MOE_OK) return rc;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MOE_ERR_CUDA;
  for (int i = 0; i < MOE_STAGE_COUNT; ++i)
    if (cudaEventElapsedTime(&h_stage_ms[i], p->tev[i], p->tev[i + 1]) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

int moe_layer_host(moe_plan_t* p, const void* h_x, const void* d_wr, const float* d_bias, const void* d_wg,
                   const void* d_wu, const void* d_wd, void* h_y, void* stream) {
  if (!p) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!h_x || !h_y)) return MOE_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t bytes = (size_t)p->cfg.T * p->cfg.H * (p->cfg.dtype == MOE_DTYPE_BF16 ? 2 : 4);
  if (bytes && cudaMemcpyAsync(p->s.x_stage[0], h_x, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  int rc = moe_layer(p, p->s.x_stage[0], d_wr, d_bias, d_wg, d_wu, d_wd, p->s.y_stage[0], stream);
  if (rc != MOE_OK) return rc;
  if (bytes && cudaMemcpyAsync(h_y, p->s.y_stage[0], bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_layer_host_submit(moe_plan_t* p, const void* h_x, const void* d_wr, const float* d_bias, const void* d_wg,
                          const void* d_wu, const void* d_wd, void* h_y, void* stream, int64_t* ticket) {
  if (!p || !ticket) return MOE_ERR_ARG;
  if (p->cfg.T > 0 && (!h_x || !h_y)) return MOE_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (!p->copy_in) {
    if (cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking) != cudaSuccess)
      return MOE_ERR_CUDA;
    for (int b = 0; b < 2; ++b)
      if (cudaEventCreateWithFlags(&p->ev_in[b], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&p->ev_done[b], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&p->ev_out[b], cudaEventDisableTiming) != cudaSuccess)
        return MOE_ERR_CUDA;
  }
  const int b = (int)(p->submitted & 1);
  const bool reuse = p->submitted >= 2;  // buffer b was used by step n-2
  const size_t bytes = (size_t)p->cfg.T * p->cfg.H * (p->cfg.dtype == MOE_DTYPE_BF16 ? 2 : 4);
  // copy-in stream: x_stage[b] is free once step n-2's layer has run
  if (reuse && cudaStreamWaitEvent(p->copy_in, p->ev_done[b], 0) != cudaSuccess) return MOE_ERR_CUDA;
  if (bytes && cudaMemcpyAsync(p->s.x_stage[b], h_x, bytes, cudaMemcpyHostToDevice, p->copy_in) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (cudaEventRecord(p->ev_in[b], p->copy_in) != cudaSuccess) return MOE_ERR_CUDA;
  // compute stream: needs this step's x, and y_stage[b] drained by step n-2's copy-out
  if (cudaStreamWaitEvent(st, p->ev_in[b], 0) != cudaSuccess) return MOE_ERR_CUDA;
  if (reuse && cudaStreamWaitEvent(st, p->ev_out[b], 0) != cudaSuccess) return MOE_ERR_CUDA;
  int rc = moe_layer(p, p->s.x_stage[b], d_wr, d_bias, d_wg, d_wu, d_wd, p->s.y_stage[b], stream);
  if (rc != MOE_OK) return rc;
  if (cudaEventRecord(p->ev_done[b], st) != cudaSuccess) return MOE_ERR_CUDA;
  // copy-out stream
  if (cudaStreamWaitEvent(p->copy_out, p->ev_done[b], 0) != cudaSuccess) return MOE_ERR_CUDA;
  if (bytes && cudaMemcpyAsync(h_y, p->s.y_stage[b], bytes, cudaMemcpyDeviceToHost, p->copy_out) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (cudaEventRecord(p->ev_out[b], p->copy_out) != cudaSuccess) return MOE_ERR_CUDA;
  *ticket = p->submitted++;
  return MOE_OK;
}

int moe_layer_host_wait(moe_plan_t* p, int64_t ticket) {
  if (!p || ticket < 0 || ticket >= p->submitted) return MOE_ERR_ARG;
  if (ticket < p->submitted - 2) return MOE_OK;  // its buffer has been reused: that step finished long ago
  return cudaEventSynchronize(p->ev_out[ticket & 1]) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_layer_buffer(moe_plan_t* p, int which, void** out_ptr) {
  if (!p || !out_ptr) return MOE_ERR_ARG;
  Scratch& s = p->s;
  void* tab[10] = {s.topk_idx, s.topk_w, s.recv, s.expert_count, s.tile_expert, s.src_info, s.slot_of, s.out_rows,
                   s.avail_ns, s.item_ns};
  if (which < 0 || which >= 10) return MOE_ERR_ARG;
  *out_ptr = tab[which];
  return MOE_OK;
}

int moe_availability_trace(moe_plan_t* p, int enable) {
  if (!p) return MOE_ERR_ARG;
  p->trace = enable ? 1 : 0;
  return MOE_OK;
}

int moe_ffn_clock_mhz(moe_plan_t* p, void* stream, int reset, float* out_mhz) {
  if (!p) return MOE_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned long long host[2] = {0, 0};
  if (out_mhz) {
    if (cudaMemcpyAsync(host, p->s.clock_probe, sizeof host, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
      return MOE_ERR_CUDA;
    *out_mhz = host[1] ? (float)(1e3 * (double)host[0] / (double)host[1]) : 0.0f;
  }
  if (reset && cudaMemsetAsync(p->s.clock_probe, 0, sizeof host, st) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

int moe_last_launch_count(moe_plan_t* p, int32_t* out) {
  if (!p || !out) return MOE_ERR_ARG;
  *out = p->launches;
  return MOE_OK;
}

int moe_last_status(moe_plan_t* p, void* stream, int32_t* code, int32_t* detail) {
  if (!p || !code) return MOE_ERR_ARG;
  int host[2] = {0, 0};
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(host, p->s.status, sizeof host, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MOE_ERR_CUDA;
  *code = host[0];
  if (detail) *detail = host[1];
  return MOE_OK;
}

const char* moe_strerror(int code) {
  switch (code) {
    case MOE_OK: return "ok";
    case MOE_ERR_ARG: return "bad argument";
    case MOE_ERR_ALIGN: return "row pitch or pointer not 16-byte aligned";
    case MOE_ERR_UNSUPPORTED: return "configuration outside what the kernels cover";
    case MOE_ERR_CUDA: return "CUDA call failed";
    case MOE_ERR_OVERFLOW: return "receive region overflow";
    case MOE_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case MOE_ERR_WORKSPACE: return "workspace too small or misaligned";
    case MOE_ERR_TOO_LARGE: return "T or E beyond the fixed scratch of moe_dispatch_noalloc";
    case MOE_ERR_INTERNAL: return "a kernel's own index check failed";
    default: return "unknown error";
  }
}

}  // extern "C"
