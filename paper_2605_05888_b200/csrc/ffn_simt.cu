// Step 3 of the MoE layer (paper Section II-A, expert computation) on plain fp32 FMA units.
//
// Used for dtype fp32 (a tensor-core tf32 product cannot meet the 1e-4 error bound) and as a
// second, independent device implementation to check the tcgen05 kernel against.  Two launches:
// S = silu(A*Wg^T) .* (A*Wu^T) into the intermediate buffer, then O = S*Wd^T.  A CTA owns one
// 128-row tile of one expert and 64 output columns; tiles without an owner exit at once, so the
// weights of experts that received no rows are never read.
#include "common.cuh"

namespace moehub {

constexpr int kSimtThreads = 256;
constexpr int kSimtBN = 64;
constexpr int kSimtBK = 16;

template <typename XT, bool SWIGLU>
__global__ void __launch_bounds__(kSimtThreads)
ffn_simt_kernel(const XT* __restrict__ A, int lda, const int* __restrict__ tile_expert,
                const XT* __restrict__ B1, const XT* __restrict__ B2, size_t expert_stride, int tp,
                size_t shard_offset, int ldb, int N, int Kd, XT* __restrict__ C, int ldc, int E) {
  const int p = blockIdx.y;
  pdl_wait();
  pdl_trigger();
  const int e = tile_expert[p];
  if (e < 0 || e >= E) return;  // no owner, or no expert at all (a caller's own table): nothing of the weights is read
  const int n0 = blockIdx.x * kSimtBN;
  const size_t row0 = (size_t)p * kTileRows;
  // e is a virtual expert: shard e % tp of expert e / tp (tp = 1: the expert itself)
  const size_t base = (size_t)(e / tp) * expert_stride + (size_t)(e % tp) * shard_offset;
  const XT* b1 = B1 + base;
  const XT* b2 = SWIGLU ? B2 + base : nullptr;
  __shared__ float As[kSimtBK][kTileRows + 1];
  __shared__ float Bs[kSimtBK][kSimtBN + 1];
  __shared__ float Bs2[SWIGLU ? kSimtBK : 1][kSimtBN + 1];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[8][4], acc2[SWIGLU ? 8 : 1][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      acc[i][j] = 0.0f;
      if (SWIGLU) acc2[i][j] = 0.0f;
    }
  for (int k0 = 0; k0 < Kd; k0 += kSimtBK) {
#pragma unroll
    for (int i = 0; i < kTileRows * kSimtBK / kSimtThreads; ++i) {
      const int idx = threadIdx.x + i * kSimtThreads;
      const int r = idx / kSimtBK, kk = idx % kSimtBK;
      As[kk][r] = (k0 + kk < Kd) ? to_float(A[(row0 + r) * lda + k0 + kk]) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < kSimtBN * kSimtBK / kSimtThreads; ++i) {
      const int idx = threadIdx.x + i * kSimtThreads;
      const int r = idx / kSimtBK, kk = idx % kSimtBK;
      const bool ok = (n0 + r < N) && (k0 + kk < Kd);
      Bs[kk][r] = ok ? to_float(b1[(size_t)(n0 + r) * ldb + k0 + kk]) : 0.0f;
      if (SWIGLU) Bs2[kk][r] = ok ? to_float(b2[(size_t)(n0 + r) * ldb + k0 + kk]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSimtBK; ++kk) {
      float a[8], b[4], c[4];
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] = As[kk][ty + 16 * i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = Bs[kk][tx + 16 * j];
        if (SWIGLU) c[j] = Bs2[kk][tx + 16 * j];
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = __fmaf_rn(a[i], b[j], acc[i][j]);
          if (SWIGLU) acc2[i][j] = __fmaf_rn(a[i], c[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx + 16 * j;
      if (n >= N) continue;
      float v = acc[i][j];
      if (SWIGLU) v = v / (1.0f + expf(-v)) * acc2[i][j];
      C[(row0 + ty + 16 * i) * ldc + n] = from_float<XT>(v);
    }
}

template <typename XT>
static int launch_typed(moe_plan* p, const void* recv, const int* tile_expert, const void* wg,
                        const void* wu, const void* wd, void* out_rows, cudaStream_t st) {
  const moe_config_t& c = p->cfg;
  // c.F is a shard's width; a whole expert's matrices are tp times that.  Gate/up rows of a shard are
  // contiguous ([F/tp, H] at offset s*F/tp*H); a shard of the down matrix is a column slice of it (row pitch: the full width).
  const int tp = p->tp;
  const size_t stride = (size_t)c.F * tp * c.H;
  mark(p, 3, st);
  dim3 g1((c.F + kSimtBN - 1) / kSimtBN, (unsigned)p->P);
  launch_pdl(ffn_simt_kernel<XT, true>, g1, dim3(kSimtThreads), 0, st, (const XT*)recv, c.H, tile_expert,
             (const XT*)wg, (const XT*)wu, stride, tp, (size_t)c.F * c.H, c.H, c.F, c.H, (XT*)p->s.inter, c.F, c.E);
  mark(p, 4, st);
  dim3 g2((c.H + kSimtBN - 1) / kSimtBN, (unsigned)p->P);
  launch_pdl(ffn_simt_kernel<XT, false>, g2, dim3(kSimtThreads), 0, st, (const XT*)p->s.inter, c.F, tile_expert,
             (const XT*)wd, (const XT*)nullptr, stride, tp, (size_t)c.F, c.F * tp, c.H, c.F, (XT*)out_rows, c.H, c.E);
  p->launches += 2;
  return (int)cudaGetLastError();
}

int launch_ffn_simt(moe_plan* p, const void* recv, const int* tile_expert, const void* wg, const void* wu,
                    const void* wd, void* out_rows, cudaStream_t st) {
  if (p->P == 0 || p->cfg.T == 0) return 0;
  if (p->cfg.dtype == MOE_DTYPE_BF16)
    return launch_typed<__nv_bfloat16>(p, recv, tile_expert, wg, wu, wd, out_rows, st);
  return launch_typed<float>(p, recv, tile_expert, wg, wu, wd, out_rows, st);
}

}  // namespace moehub
