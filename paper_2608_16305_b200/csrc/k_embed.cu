// Step (5): single-layer multi-head temporal attention over the <= k sampled neighbors.
#include "tgnn_internal.cuh"
#include "tgnn_device.cuh"

namespace tgnn {
namespace {

constexpr unsigned FULL = 0xffffffffu;

// One warp per row.  Rows [0, n*k): neighbor rows z = [m_nbr || x_eid || Phi(t - ts)] (zero if the slot
// is empty).  Rows [n*k, n*k + n): per root, z_q = [m_root || Phi(0)] and the memory half of cat_o.
__global__ void __launch_bounds__(256) gather_z_kernel(const float* __restrict__ memory, const void* __restrict__ efeat,
                                                       int feat_bf16, const float* __restrict__ time_w,
                                                       const float* __restrict__ time_b, int d, int de, int k,
                                                       const int32_t* __restrict__ nodes, const double* __restrict__ times,
                                                       int n, const int32_t* __restrict__ nbr,
                                                       const int32_t* __restrict__ eid, const double* __restrict__ ts,
                                                       int ld, float* __restrict__ Z, float* __restrict__ z_dt,
                                                       float* __restrict__ Zsin,
                                                       float* __restrict__ Zq, float* __restrict__ cat_o) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int nb_rows = n * k;
  const int dkv = 2 * d + de;
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < nb_rows + n; r += warps) {
    if (r < nb_rows) {
      float* row = Z + (int64_t)r * ld;
      const int nb = nbr[r];
      if (nb < 0) {
        for (int q = lane; q < ld; q += 32) row[q] = 0.f;
        for (int q = lane; q < d; q += 32) Zsin[(int64_t)r * d + q] = 0.f;
        if (lane == 0) z_dt[r] = 0.f;
        continue;
      }
      const float dtf = (float)(times[r / k] - ts[r]);
      warp_copy_f32(row, memory + (int64_t)nb * d, d, lane);
      warp_copy_feat(row + d, efeat, feat_bf16, eid[r], de, lane);
      float* phi = row + d + de;
      for (int q = lane; q < d; q += 32) time_encode_sc(time_w[q], time_b[q], dtf, &phi[q], &Zsin[(int64_t)r * d + q]);
      for (int q = dkv + lane; q < ld; q += 32) row[q] = 0.f;
      if (lane == 0) z_dt[r] = dtf;
    } else {
      const int i = r - nb_rows;
      const float* m = memory + (int64_t)nodes[i] * d;
      warp_copy_f32(Zq + (int64_t)i * 2 * d, m, d, lane);
      warp_copy_f32(cat_o + (int64_t)i * 2 * d + d, m, d, lane);
      for (int q = lane; q < d; q += 32) Zq[(int64_t)i * 2 * d + d + q] = time_encode(time_w[q], time_b[q], 0.f);
    }
  }
}

// One warp per root: logits, softmax over the valid slots, weighted sum of V into cat_o[:, :d].
// Dynamic shared memory: warps_per_block * H * k floats.
__global__ void __launch_bounds__(256) attention_fwd_kernel(const float* __restrict__ Q, const float* __restrict__ KV,
                                                            const int32_t* __restrict__ cnt, int n, int d, int H, int k,
                                                            float* __restrict__ alpha, float* __restrict__ cat_o) {
  extern __shared__ float sm[];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int i = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (i >= n) return;
  float* al = sm + wib * H * k;
  const int dh = d / H;
  const int c = cnt[i];
  const float scale = rsqrtf((float)dh);
  const float* q = Q + (int64_t)i * d;
  for (int h = 0; h < H; ++h) {
    float mx = -INFINITY;
    for (int s = 0; s < c; ++s) {
      const float* kr = KV + ((int64_t)i * k + s) * 2 * d + h * dh;
      float a = 0.f;
      for (int e = lane; e < dh; e += 32) a = fmaf(q[h * dh + e], kr[e], a);
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(FULL, a, o);
      a *= scale;
      if (lane == 0) al[h * k + s] = a;
      mx = fmaxf(mx, a);
    }
    __syncwarp();
    float den = 0.f;
    for (int s = 0; s < c; ++s) den += expf(al[h * k + s] - mx);
    __syncwarp();
    if (lane < c) al[h * k + lane] = expf(al[h * k + lane] - mx) / den;
    if (lane >= c && lane < k) al[h * k + lane] = 0.f;
    __syncwarp();
    if (lane < k) alpha[((int64_t)i * H + h) * k + lane] = al[h * k + lane];
  }
  for (int e = lane; e < d; e += 32) {
    const int h = e / dh;
    float a = 0.f;
    for (int s = 0; s < c; ++s) a = fmaf(al[h * k + s], KV[((int64_t)i * k + s) * 2 * d + d + e], a);
    cat_o[(int64_t)i * 2 * d + e] = a;
  }
}

}  // namespace

int launch_embed(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, const int32_t* nbr,
                 const int32_t* eid, const double* ts, const int32_t* cnt, float* h_out, cudaStream_t s) {
  if (n == 0) return TGNN_OK;
  const tgnn_config& c = ctx->cfg;
  const ParamLayout& L = ctx->L;
  Workspace& w = ctx->ws;
  const int d = c.d, k = c.k, H = c.heads;
  const int rows = n * k + n;
  {
    KernelScope scope__(ctx, "gather_z", s);
    gather_z_kernel<<<(rows + 7) / 8, 256, 0, s>>>(ctx->memory, ctx->efeat, c.feat_dtype == TGNN_BF16,
                                                   ctx->params + L.time_w, ctx->params + L.time_b, d, c.d_e, k, nodes,
                                                   times, n, nbr, eid, ts, ctx->ld_kv, w.Z, w.z_dt, w.Zsin, w.Zq, w.cat_o);
  }
  TGNN_LAUNCH_OK(ctx, "gather_z");
  GemmArgs g = {};
  g.A = w.Z; g.a_rs = ctx->ld_kv; g.a_cs = 1;
  g.B = ctx->params + L.wk; g.b_rs = 1; g.b_cs = L.dkv;  // rows of [W_k; W_v]
  g.C = w.KV; g.ldc = 2 * d; g.M = n * k; g.N = 2 * d; g.K = (int)L.dkv;
  g.bias = ctx->params + L.bk; g.split_k = 1;
  int rc = fork_to(ctx, s, ctx->side[0]);  // the query projection runs beside the key/value projection
  if (rc) return rc;
  rc = launch_gemm(ctx, g, "kv_proj", s);
  if (rc) return rc;
  g = GemmArgs{};
  g.A = w.Zq; g.a_rs = 2 * d; g.a_cs = 1;
  g.B = ctx->params + L.wq; g.b_rs = 1; g.b_cs = 2 * d;
  g.C = w.Q; g.ldc = d; g.M = n; g.N = d; g.K = 2 * d; g.bias = ctx->params + L.bq; g.split_k = 1;
  rc = launch_gemm(ctx, g, "q_proj", ctx->side[0]);
  if (rc) return rc;
  rc = fork_to(ctx, ctx->side[0], s);
  if (rc) return rc;
  const int wpb = 8;
  {
    KernelScope scope__(ctx, "attention_fwd", s);
    attention_fwd_kernel<<<(n + wpb - 1) / wpb, wpb * 32, wpb * H * k * sizeof(float), s>>>(w.Q, w.KV, cnt, n, d, H, k,
                                                                                           w.alpha, w.cat_o);
  }
  TGNN_LAUNCH_OK(ctx, "attention_fwd");
  g = GemmArgs{};
  g.A = w.cat_o; g.a_rs = 2 * d; g.a_cs = 1;
  g.B = ctx->params + L.wo; g.b_rs = 1; g.b_cs = 2 * d;
  g.C = h_out; g.ldc = d; g.M = n; g.N = d; g.K = 2 * d; g.bias = ctx->params + L.bo; g.relu = 1; g.split_k = 1;
  return launch_gemm(ctx, g, "out_proj", s);
}

}  // namespace tgnn
