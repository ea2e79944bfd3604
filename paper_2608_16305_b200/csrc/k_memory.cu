// Memory path: Message of Eq. 1 (step 2) and Update of Eq. 2 as a GRU cell with
// scatter write-back (step 4).
#include "tgnn_internal.cuh"
#include "tgnn_device.cuh"

namespace tgnn {
namespace {

// Writes one message row [m_self || m_other || x || Phi(dt)] (dm floats) with the lanes of a warp.
__device__ __forceinline__ void write_message_row(float* __restrict__ row, const float* __restrict__ memory,
                                                  const void* __restrict__ efeat, int feat_bf16,
                                                  const float* __restrict__ time_w, const float* __restrict__ time_b,
                                                  int d, int de, int self, int other, int eid, float dtf, int lane,
                                                  float* __restrict__ sin_row) {
  warp_copy_f32(row, memory + (int64_t)self * d, d, lane);
  warp_copy_f32(row + d, memory + (int64_t)other * d, d, lane);
  warp_copy_feat(row + 2 * d, efeat, feat_bf16, eid, de, lane);
  float* phi = row + 2 * d + de;
  if (sin_row == nullptr) {
    for (int q = lane; q < d; q += 32) phi[q] = time_encode(time_w[q], time_b[q], dtf);
  } else {
    for (int q = lane; q < d; q += 32) time_encode_sc(time_w[q], time_b[q], dtf, &phi[q], &sin_row[q]);
  }
}

// One warp per message j = 2i + role.
__global__ void __launch_bounds__(256) build_messages_kernel(const float* __restrict__ memory,
                                                             const double* __restrict__ last_update,
                                                             const void* __restrict__ efeat, int feat_bf16,
                                                             const float* __restrict__ time_w,
                                                             const float* __restrict__ time_b, int d, int de,
                                                             const int32_t* __restrict__ src,
                                                             const int32_t* __restrict__ dst, const double* __restrict__ t,
                                                             const int32_t* __restrict__ eid,
                                                             const uint8_t* __restrict__ keep, int n, int64_t N, int64_t E,
                                                             int32_t* status, float* __restrict__ msg_out,
                                                             int32_t* __restrict__ msg_node_out) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int dm = 3 * d + de;
  for (int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; j < 2 * n; j += warps) {
    const int i = j >> 1, role = j & 1;
    bool kept = keep == nullptr || keep[i] != 0;
    const int self = role ? dst[i] : src[i];
    const int other = role ? src[i] : dst[i];
    // an event naming a node or a feature row that does not exist is reported and sends no message
    if (kept) {
      int32_t* st = lane == 0 ? status : nullptr;
      kept = index_ok(self, N, st) & index_ok(other, N, st) & (de == 0 || index_ok(eid[i], E, st));
    }
    if (lane == 0) msg_node_out[j] = kept ? self : -1;
    if (msg_out == nullptr) continue;
    float* row = msg_out + (int64_t)j * dm;
    if (!kept) {
      for (int q = lane; q < dm; q += 32) row[q] = 0.f;
      continue;
    }
    const float dtf = (float)(t[i] - last_update[self]);
    write_message_row(row, memory, efeat, feat_bf16, time_w, time_b, d, de, self, other, eid[i], dtf, lane, nullptr);
  }
}

// One warp per unique node u: the winner's message row into X (leading dimension ld), its dt and timestamp.
__global__ void __launch_bounds__(256) gather_winner_kernel(const float* __restrict__ memory,
                                                            const double* __restrict__ last_update,
                                                            const void* __restrict__ efeat, int feat_bf16,
                                                            const float* __restrict__ time_w,
                                                            const float* __restrict__ time_b, int d, int de,
                                                            const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                                                            const double* __restrict__ t, const int32_t* __restrict__ eid,
                                                            const float* __restrict__ msg, const int32_t* __restrict__ uniq,
                                                            const int32_t* __restrict__ winner,
                                                            const int32_t* __restrict__ n_uniq, int u_cap, int n_msg, int64_t N,
                                                            int64_t E, int32_t* status, int ld,
                                                            float* __restrict__ X, float* __restrict__ x_dt,
                                                            float* __restrict__ Xsin, double* __restrict__ win_t) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  if (blockIdx.x == 0 && threadIdx.x == 0) index_ok(*n_uniq, (long long)u_cap + 1, status);   // a count beyond the capacity
  const int U = max(0, min(*n_uniq, u_cap));
  const int dm = 3 * d + de;
  for (int u = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < U; u += warps) {
    float* row = X + (int64_t)u * ld;
    float* sin_row = Xsin + (int64_t)u * d;
    int32_t* st = lane == 0 ? status : nullptr;
    const int j = winner[u];
    bool good = index_ok(j, n_msg, st);
    const int i = good ? j >> 1 : 0, role = j & 1;
    const int self = good ? (role ? dst[i] : src[i]) : 0;
    const int other = good ? (role ? src[i] : dst[i]) : 0;
    good = good && index_ok(self, N, st) && index_ok(other, N, st) && (de == 0 || msg != nullptr || index_ok(eid[i], E, st));
    if (!good) {   // reported; the row is zero and the node's update starts from a zero message
      for (int q = lane; q < ld; q += 32) row[q] = 0.f;
      for (int q = lane; q < d; q += 32) sin_row[q] = 0.f;
      if (lane == 0) { x_dt[u] = 0.f; win_t[u] = 0.0; }
      continue;
    }
    const double ti = t[i];
    const float dtf = (float)(ti - last_update[self]);
    if (msg != nullptr) {
      warp_copy_f32(row, msg + (int64_t)j * dm, dm, lane);
      for (int q = lane; q < d; q += 32) sin_row[q] = sinf(time_arg(time_w[q], time_b[q], dtf));
    } else {
      write_message_row(row, memory, efeat, feat_bf16, time_w, time_b, d, de, self, other, eid[i], dtf, lane, sin_row);
    }
    for (int q = dm + lane; q < ld; q += 32) row[q] = 0.f;
    if (lane == 0) { x_dt[u] = dtf; win_t[u] = ti; }
  }
}

// Gates of the GRU cell and write-back.  Gi = W_i x + b_i, Gh = W_h h + b_h are given.
__global__ void __launch_bounds__(256) gru_gate_kernel(const float* __restrict__ Gi, const float* __restrict__ Gh,
                                                       const float* __restrict__ X, int ld, int d,
                                                       const int32_t* __restrict__ uniq, const double* __restrict__ win_t,
                                                       const int32_t* __restrict__ n_uniq, int u_cap,
                                                       float* __restrict__ g_r, float* __restrict__ g_z,
                                                       float* __restrict__ g_n, float* __restrict__ g_hn,
                                                       float* __restrict__ memory, double* __restrict__ last_update,
                                                       int64_t N, int32_t* status) {
  const int U = max(0, min(*n_uniq, u_cap));
  const int64_t total = (int64_t)U * d;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int u = (int)(e / d), q = (int)(e % d);
    const float* gi = Gi + (int64_t)u * 3 * d;
    const float* gh = Gh + (int64_t)u * 3 * d;
    const float r = sigmoidf_(gi[q] + gh[q]);
    const float z = sigmoidf_(gi[d + q] + gh[d + q]);
    const float hn = gh[2 * d + q];
    const float nn = tanhf(fmaf(r, hn, gi[2 * d + q]));
    const float h = X[(int64_t)u * ld + q];
    const float hnew = fmaf(z, h - nn, nn);  // (1 - z) n + z h
    g_r[e] = r; g_z[e] = z; g_n[e] = nn; g_hn[e] = hn;
    const int node = uniq[u];
    if (!index_ok(node, N, q == 0 ? status : nullptr)) continue;   // reported, nothing written
    memory[(int64_t)node * d + q] = hnew;
    if (q == 0) last_update[node] = win_t[u];
  }
}

// The plain recurrent cell and write-back: m' = tanh(Gi + Gh) with Gi = W_i x + b_i, Gh = W_h h + b_h
// (row pitch d).  The new row is kept in g_n for the backward pass (d tanh = 1 - m'^2).
__global__ void __launch_bounds__(256) rnn_gate_kernel(const float* __restrict__ Gi, const float* __restrict__ Gh, int d,
                                                       const int32_t* __restrict__ uniq, const double* __restrict__ win_t,
                                                       const int32_t* __restrict__ n_uniq, int u_cap,
                                                       float* __restrict__ g_n, float* __restrict__ memory,
                                                       double* __restrict__ last_update, int64_t N, int32_t* status) {
  const int U = max(0, min(*n_uniq, u_cap));
  const int64_t total = (int64_t)U * d;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int u = (int)(e / d), q = (int)(e % d);
    const float hnew = tanhf(Gi[e] + Gh[e]);
    g_n[e] = hnew;
    const int node = uniq[u];
    if (!index_ok(node, N, q == 0 ? status : nullptr)) continue;
    memory[(int64_t)node * d + q] = hnew;
    if (q == 0) last_update[node] = win_t[u];
  }
}

}  // namespace

int launch_build_messages(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const double* t, const int32_t* eid,
                          const uint8_t* keep, int n, float* msg_out, int32_t* msg_node_out, cudaStream_t s) {
  if (n == 0) return TGNN_OK;
  const tgnn_config& c = ctx->cfg;
  const int warps = 2 * n;
  const int blocks = msg_out ? (warps + 7) / 8 : (warps + 8 * 32 - 1) / (8 * 32) + 1;
  {
    KernelScope scope__(ctx, "build_messages", s);
    build_messages_kernel<<<blocks, 256, 0, s>>>(ctx->memory, ctx->last_update, ctx->efeat, c.feat_dtype == TGNN_BF16,
                                                 ctx->params + ctx->L.time_w, ctx->params + ctx->L.time_b, c.d, c.d_e, src,
                                                 dst, t, eid, keep, n, c.num_nodes, ctx->num_events, ctx->ws.status, msg_out,
                                                 msg_node_out);
  }
  TGNN_LAUNCH_OK(ctx, "build_messages");
  return TGNN_OK;
}

int launch_memory_update(tgnn_ctx* ctx, const float* msg, const int32_t* uniq, const int32_t* winner,
                         const int32_t* n_uniq, cudaStream_t s) {
  const tgnn_config& c = ctx->cfg;
  const ParamLayout& L = ctx->L;
  Workspace& w = ctx->ws;
  const int d = c.d, U_cap = min(ctx->U_cap, 2 * ctx->m_n);
  const int gd = (int)L.gates * d;  // rows of the cell's matrices: 3d (GRU) or d (plain cell)
  if (U_cap == 0) return TGNN_OK;
  {
    KernelScope scope__(ctx, "gather_winner", s);
    gather_winner_kernel<<<(U_cap + 7) / 8, 256, 0, s>>>(ctx->memory, ctx->last_update, ctx->efeat,
                                                         c.feat_dtype == TGNN_BF16, ctx->params + L.time_w,
                                                         ctx->params + L.time_b, d, c.d_e, ctx->m_src, ctx->m_dst, ctx->m_t,
                                                         ctx->m_eid, msg, uniq, winner, n_uniq, U_cap, 2 * ctx->m_n, c.num_nodes,
                                                         ctx->num_events, w.status, ctx->ld_msg, w.X, w.x_dt, w.Xsin, w.win_t);
  }
  TGNN_LAUNCH_OK(ctx, "gather_winner");
  GemmArgs g = {};
  g.A = w.X; g.a_rs = ctx->ld_msg; g.a_cs = 1;
  g.B = ctx->params + L.gru_wi; g.b_rs = 1; g.b_cs = L.dmsg;  // B(k,n) = W_i[n,k]
  g.C = w.Gi; g.ldc = gd; g.M = U_cap; g.N = gd; g.K = (int)L.dmsg; g.dev_M = n_uniq;
  g.bias = ctx->params + L.gru_bi;
  // few rows, long contraction: split the contraction over CTAs and accumulate into a cleared Gi
  g.accumulate = 1; g.split_k = 4; g.site = SITE_GI + 1;
  TGNN_CUDA_OK(ctx, cudaMemsetAsync(w.Gi, 0, sizeof(float) * (size_t)U_cap * gd, s));
  int rc = fork_to(ctx, s, ctx->side[0]);  // the hidden-state product runs beside the input product
  if (rc) return rc;
  rc = launch_gemm(ctx, g, "gru_gi", s);
  if (rc) return rc;
  g.B = ctx->params + L.gru_wh; g.b_cs = d; g.C = w.Gh; g.K = d; g.bias = ctx->params + L.gru_bh;
  g.accumulate = 0; g.split_k = 1; g.site = SITE_GH + 1;
  rc = launch_gemm(ctx, g, "gru_gh", ctx->side[0]);
  if (rc) return rc;
  rc = fork_to(ctx, ctx->side[0], s);
  if (rc) return rc;
  const int64_t total = (int64_t)U_cap * d;
  if (c.model == TGNN_MODEL_JODIE) {
    {
      KernelScope scope__(ctx, "rnn_gate", s);
      rnn_gate_kernel<<<(int)((total + 255) / 256), 256, 0, s>>>(w.Gi, w.Gh, d, uniq, w.win_t, n_uniq, U_cap, w.g_n,
                                                                 ctx->memory, ctx->last_update, c.num_nodes, w.status);
    }
    TGNN_LAUNCH_OK(ctx, "rnn_gate");
    return TGNN_OK;
  }
  {
    KernelScope scope__(ctx, "gru_gate", s);
    gru_gate_kernel<<<(int)((total + 255) / 256), 256, 0, s>>>(w.Gi, w.Gh, w.X, ctx->ld_msg, d, uniq, w.win_t, n_uniq,
                                                               U_cap, w.g_r, w.g_z, w.g_n, w.g_hn, ctx->memory,
                                                               ctx->last_update, c.num_nodes, w.status);
  }
  TGNN_LAUNCH_OK(ctx, "gru_gate");
  return TGNN_OK;
}

}  // namespace tgnn
