// Dense projections, fp32 FMA path: a strided tiled GEMM used for every
// projection and its two gradient products when math_mode is TGNN_MATH_FP32,
// and for the small products in every mode.
#include <cstdio>

#include "tgnn_internal.cuh"

namespace tgnn {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4, NT = 256;

// grid: (ceil(N/BN), ceil(M/BM), split_k)
__global__ void __launch_bounds__(NT) gemm_fp32_kernel(GemmArgs g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int M = g.dev_M ? min(*g.dev_M, g.M) : g.M;
  const int K = g.dev_K ? min(*g.dev_K, g.K) : g.K;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M || n0 >= g.N) return;
  const int kchunk = ((K + g.split_k - 1) / g.split_k + BK - 1) / BK * BK;
  const int kbeg = blockIdx.z * kchunk;
  const int kend = min(K, kbeg + kchunk);
  if (kbeg >= kend && !(blockIdx.z == 0 && g.bias)) return;

  const int tid = threadIdx.x;
  const int tx = tid % (BN / TN), ty = tid / (BN / TN);
  float acc[TM][TN] = {};
  float rsum[TM] = {};
  const bool do_rowsum = g.rowsum_out != nullptr && blockIdx.x == 0 && tx == 0;
  // loader mappings: along the unit-stride direction of each operand
  const bool a_k_contig = g.a_cs == 1;
  const bool b_n_contig = g.b_cs == 1;

  for (int k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
    for (int i = 0; i < (BM * BK) / NT; ++i) {
      int e = tid + i * NT, mm, kk;
      if (a_k_contig) { kk = e % BK; mm = e / BK; } else { mm = e % BM; kk = e / BM; }
      const int gm = m0 + mm, gk = k0 + kk;
      As[kk][mm] = (gm < M && gk < kend) ? g.A[(int64_t)gm * g.a_rs + (int64_t)gk * g.a_cs] : 0.f;
    }
#pragma unroll
    for (int i = 0; i < (BN * BK) / NT; ++i) {
      int e = tid + i * NT, nn, kk;
      if (b_n_contig) { nn = e % BN; kk = e / BN; } else { kk = e % BK; nn = e / BK; }
      const int gn = n0 + nn, gk = k0 + kk;
      Bs[kk][nn] = (gn < g.N && gk < kend) ? g.B[(int64_t)gk * g.b_rs + (int64_t)gn * g.b_cs] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], b[TN];
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * TM]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * TN]);
      a[0] = av.x; a[1] = av.y; a[2] = av.z; a[3] = av.w;
      b[0] = bv.x; b[1] = bv.y; b[2] = bv.z; b[3] = bv.w;
#pragma unroll
      for (int i = 0; i < TM; ++i) {
        if (do_rowsum) rsum[i] += a[i];
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int gm = m0 + ty * TM + i;
    if (gm >= M) continue;
    if (do_rowsum) atomicAdd(&g.rowsum_out[gm], rsum[i]);
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int gn = n0 + tx * TN + j;
      if (gn >= g.N) continue;
      float v = acc[i][j];
      if (g.bias && blockIdx.z == 0) v += g.bias[gn];
      float* c = &g.C[(int64_t)gm * g.ldc + gn];
      if (g.accumulate) {
        atomicAdd(c, v);
      } else {
        if (g.relu) v = fmaxf(v, 0.f);
        *c = v;
      }
    }
  }
}

}  // namespace

int launch_gemm(tgnn_ctx* ctx, const GemmArgs& g, const char* name, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0) return TGNN_OK;
  if (g.split_k > 1 && !g.accumulate) return set_error(ctx, TGNN_EINVAL, "gemm %s: split_k needs accumulate", name);
  if (ctx->cfg.math_mode != TGNN_MATH_FP32) {
    GemmArgs gp = g;
    if (ctx->cfg.math_mode != TGNN_MATH_TF32_FAST) gp.precise = 1;
    const int rc = launch_gemm_tf32(ctx, gp, name, s);
    if (rc != 1) return rc;  // 1: shape not handled by the tensor-core kernel, use the FMA tiles
    // not an error, but not silent either: the note stays in tgnn_last_error and the launches are counted
    ctx->fma_fallbacks++;
    snprintf(ctx->err, sizeof(ctx->err), "note: product %s (M=%d N=%d K=%d) does not fit the tensor-core kernel and ran on the "
             "fp32 FMA tiles (%lld such launches so far)", name, g.M, g.N, g.K, (long long)ctx->fma_fallbacks);
  }
  if (g.a_idx) return set_error(ctx, TGNN_EINVAL, "gemm %s: row-indirect A needs the tensor-core path", name);
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.split_k < 1 ? 1 : g.split_k);
  GemmArgs a = g;
  if (a.split_k < 1) a.split_k = 1;
  {
    KernelScope scope__(ctx, name, s);
    gemm_fp32_kernel<<<grid, NT, 0, s>>>(a);
  }
  TGNN_LAUNCH_OK(ctx, name);
  return TGNN_OK;
}

}  // namespace tgnn
