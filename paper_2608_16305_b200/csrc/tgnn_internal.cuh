// Internal declarations shared by the CUDA translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "../../include/tgnn.h"

namespace tgnn {

// Offsets of the parameter tensors in the flat vector (order fixed by the public header).
struct ParamLayout {
  int64_t d, de, dmsg, dkv, dq;
  int64_t gates;  // rows of the update cell's matrices in units of d: 3 (GRU) or 1 (plain recurrent cell)
  int64_t time_w, time_b, gru_wi, gru_wh, gru_bi, gru_bh, wq, bq, wk, wv, bk, bv, wo, bo, proj_w, proj_b, w1, b1, w2, b2,
      total;
};
ParamLayout make_layout(int d, int d_e, int model);

// Workspace: everything the step keeps between entry points.  Row-major, fp32 unless noted.
struct Workspace {
  // step (0)
  int32_t* hist;  // [N] zero between calls
  // step (3)
  unsigned long long* best_t;   // [N] zero between calls
  unsigned long long* best_id;  // [N] zero between calls
  int32_t* win_msg;             // [N]
  int32_t* node2slot;           // [N], -1 except for the nodes updated by the last memory update
  int32_t* prev_uniq;           // [2*max_events] nodes whose node2slot entry is set
  int32_t* prev_n_uniq;         // [1]
  // internal copies used by tgnn_train_step
  int32_t* msg_node;  // [2*max_events]
  int32_t* uniq;      // [2*max_events]
  int32_t* winner;    // [2*max_events]
  int32_t* n_uniq;    // [1]
  int32_t* r_node;    // [max_roots]
  double* r_time;     // [max_roots]
  int32_t* nb_node;   // [max_roots*k]
  int32_t* nb_eid;    // [max_roots*k]
  double* nb_ts;      // [max_roots*k]
  int32_t* nb_cnt;    // [max_roots]
  float* h;           // [max_roots, d]
  // host-input staging for tgnn_train_step_host
  int32_t *st_u_src, *st_u_dst, *st_u_eid, *st_q_src, *st_q_dst, *st_q_neg;
  double *st_u_t, *st_q_t;
  uint8_t *st_u_keep, *st_mask;
  float* st_scalars;  // [4] loss accumulator, spare, loss, gradient norm
  // step (4) activations
  float* X;        // [U_cap, ld_msg] winners' message rows (first d columns = the node's own memory)
  float* x_dt;     // [U_cap] fp32 dt inside Phi of the winner message
  float* Xsin;     // [U_cap, d] sin of the time-encoding arguments of the winner messages
  double* win_t;   // [U_cap]
  float* Gi;       // [U_cap, 3d]
  float* Gh;       // [U_cap, 3d]
  float *g_r, *g_z, *g_n, *g_hn;  // [U_cap, d]
  // step (5) activations
  float* Z;      // [NB_cap, ld_kv]
  float* z_dt;   // [NB_cap]
  float* KV;     // [NB_cap, 2d]  (K | V)
  float* Zq;     // [R_cap, 2d]
  float* Q;      // [R_cap, d]
  float* alpha;  // [R_cap, H, k]
  float* cat_o;  // [R_cap, 2d]  (a | m_root)
  // step (6)
  float* head_wT; // [2d, up4(d)] W_1's two halves transposed ([c][j]) for the tile head, rewritten with the weight images
  float* cat1;    // [2*nq_cap, 2d]
  float* hid1;    // [2*nq_cap, d]  ReLU(pre1); overwritten by dpre1
  uint8_t* hid_gate;  // [2*nq_cap, d] 1 where the head's hidden unit was active
  float* dcat1;   // [2*nq_cap, 2d]
  float* dpre_o;  // [R_cap, d]
  float* dcat_o;  // [R_cap, 2d]
  float* dQ;      // [R_cap, d]
  float* dzq;     // [R_cap, 2d]
  float* dKV;     // [NB_cap, 2d]
  float* dZmp;    // [NB_cap, 2d] grad wrt the memory part (cols [0,d)) and the time-encoding part (cols [d,2d)) of Z
  float* dMemU;   // [U_cap, d]   grad wrt the rows written by the memory update
  float* dGi;     // [U_cap, 3d]
  float* dGh;     // [U_cap, 3d]
  float* dXp;     // [U_cap, d]   grad wrt the time-encoding part of the winners' messages
  float* dWkv_pad;  // [2d, ld_wkv] W_kv's gradient (and, in column dkv, its bias gradient) with 16-byte aligned rows
  float* grads;   // [P]
  double* red;    // [4] sum of squares, spare
  double* tg_acc; // [2d] fp64 sums of the time-encoder gradient (dw | db)
  float* adam_sc; // [4] bias corrections 1/(1-b1^t), 1/(1-b2^t)
  unsigned int* counters;  // [4] "last block" tickets
  int32_t* status;         // [1] device status word
};

// Optional per-kernel timing (tgnn_profile_begin / tgnn_profile_report): an event pair around
// every launch while enabled.  Off by default; nothing is recorded or allocated then.
struct ProfEntry {
  const char* name;
  cudaEvent_t a, b;
};
struct Profiler {
  bool on = false;
  std::vector<ProfEntry> entries;  // events are created once and reused
  size_t used = 0;
};

// A weight matrix in its role as the B operand of one projection, with the tiling the tensor-core
// kernel will use for it.  Once per step the weights are written out as "images": for every n-tile and
// contraction block the exact bytes of the shared-memory B tile (TF32 head, then TF32 tail, already
// swizzled), so that a CTA fetches a stage's B operand with one bulk asynchronous copy instead of
// loading, splitting and storing it through registers in every CTA.
enum WeightSiteId {
  SITE_GI = 0, SITE_GH, SITE_KV, SITE_Q, SITE_OUT, SITE_HEAD,   // forward: B(k,n) = W[n*ld + k]
  SITE_DCAT1, SITE_DCATO, SITE_DZQ, SITE_DZ, SITE_DXPHI,        // input gradients: B(k,n) = W[k*ld + col(n)]
  SITE_COUNT
};
struct WeightSite {
  int64_t w_off, ld;
  int major;                 // 0: K-major (forward), 1: MN-major (input gradient)
  int N, K;                  // columns of C, contraction length
  int col0, n_split, col1;   // MN-major: col(n) = n < n_split ? col0 + n : col1 + (n - n_split)
  int precise;
  int n_tiles, bn, bn_t, nkb;
  int64_t image_off;         // byte offset of the site's images in the image buffer
  int64_t chunks;            // 16-byte chunks the preparation kernel writes for this site
};

// An fp32 matrix stored as two 16-bit planes of the same row-major shape: hi = r16(scale * x) at `hi`,
// lo = r16(scale * x - hi) at hi + plane_stride (in elements), r16 rounding to fp16 (fp16 = 1: 22 mantissa bits
// together, values must stay inside fp16's range, hence the power-of-two `scale` for gradients) or to bf16
// (fp16 = 0: 16 bits, any range).  ld and plane_stride are multiples of 8, `hi` is 16-byte aligned.
struct SplitMat {
  void* hi;
  int64_t ld, plane_stride;
  int64_t rows, cols;
  int fp16;
  float scale;
  int planes;   // 2: hi and lo planes (three passes per product); 1: only the hi plane is read (one pass, 11-bit operands)
};

}  // namespace tgnn

struct tgnn_ctx {
  tgnn_config cfg;
  tgnn::ParamLayout L;
  int U_cap, R_cap, NB_cap, nq_cap;
  int ld_msg, ld_kv;  // padded leading dimensions of X and Z
  int ld_wkv;         // row pitch of the padded W_kv gradient: dkv + 1 rounded up to a multiple of 4
  // borrowed
  const int64_t* indptr;
  const int32_t *g_nbr, *g_eid;
  const double* g_ts;
  int64_t n_entries;
  const void* efeat;
  int64_t num_events;
  float* memory;
  double* last_update;
  float *params, *adam_m, *adam_v;
  int64_t* step;
  // event arrays recorded by the last tgnn_build_messages
  const int32_t *m_src, *m_dst, *m_eid;
  const double* m_t;
  const uint8_t* m_keep;
  int m_n;
  // arrays recorded by the last tgnn_embed
  const int32_t *e_nodes, *e_nbr, *e_eid, *e_cnt;
  const double *e_times, *e_ts;
  int e_n;
  const float* e_h;
  // device count / capacity of the rows written by the last tgnn_memory_update
  const int32_t* upd_n_uniq;
  int upd_cap;
  bool have_update, have_embed;
  // tgnn_step_mixed_host: the mixed batch of the current call stays on the device (two slots, used
  // alternately) because it is the update batch of the next call; host inputs travel as one packed
  // block through two pinned buffers.
  struct MixedSlot {
    int32_t *src, *dst, *eid;
    double* t;
    uint8_t *aux, *keep;
    int n;
  };
  MixedSlot mixed[2];
  int mixed_cur;              // slot written by the last call (-1: none yet)
  unsigned char* pack_host[2];
  cudaEvent_t pack_done[2];
  unsigned char* pack_dev;
  size_t pack_bytes;
  int32_t* heavy_dev;
  tgnn::WeightSite sites[tgnn::SITE_COUNT];
  tgnn::WeightSite* sites_dev;   // device copy
  unsigned char* images;         // device buffer of all sites' images
  size_t images_bytes;
  bool images_fresh;             // images match the current parameters (set by the step, cleared by Adam)
  // TGNN_MATH_F16X3: the attention inputs Z (with a column of ones after the last input column), the gradient
  // of the key/value rows and the key/value weights in their two roles, each as two fp16 planes
  void* split_buf;
  tgnn::SplitMat zs, dkvs, wkv_s, wz_s;
  bool z_split;       // the attention inputs of the current step are (being) written as fp16 planes
  bool z_static_done; // tgnn_train_step already gathered the memory-independent part of the attention inputs
  bool grads_zeroed;  // tgnn_train_step cleared the gradient block ahead of the backward pass
  tgnn::Workspace ws;
  void* arena;
  size_t arena_bytes;
  // Internal streams for kernels that do not lie on the step's critical chain (weight-gradient
  // products, the neighbor search next to the memory update, ...).  They are forked from and joined
  // back into the caller's stream with events, so the caller still sees one ordered stream of work.
  cudaStream_t side[4];   // [2]: the time-encoder sum over the neighbor rows in the split mode (it must not queue behind
                          // products that wait for a whole SM's shared memory); [3]: the update cell's input-weight
                          // gradient in that mode (it must not queue behind the persistent weight gradient on [0])
  cudaEvent_t ev[32];
  // tgnn_train_step's side stream, recorded after the neighbor search and after everything else it carries (the static
  // half of the attention inputs, the clear of the gradient block); the embedding waits for each where it first
  // needs it (side_pending: recorded and not yet waited for)
  cudaEvent_t ev_search, ev_side_done;
  bool side_pending;
  int ev_next;
  // Replay of a whole training step as a CUDA graph: tgnn_train_step copies its inputs into the
  // fixed staging buffers and, for a shape signature it has already run once, captures the launch
  // sequence on the caller's stream and replays it from then on.
  struct StepGraph {
    int n_u, n_q, has_keep, has_mask;
    float *loss_out, *gradnorm_out;
    int seen;
    int64_t kernels;
    cudaGraphExec_t exec;
  };
  StepGraph graphs[8];
  int n_graphs;
  int graphs_enabled;
  // Gradient synchronisation across workers: the step stops after the gradient, the caller reduces
  // the buffer and tgnn_apply_gradient finishes the step.
  int defer_adam;
  bool grad_pending;
  int64_t launches;
  int64_t fma_fallbacks;   // products that a tensor-core mode had to run on the fp32 FMA tiles
  tgnn::Profiler prof;
  char err[256];
};

namespace tgnn {

int set_error(tgnn_ctx* ctx, int code, const char* fmt, ...);
#define TGNN_CUDA_OK(ctx, expr)                                                              \
  do {                                                                                       \
    cudaError_t e__ = (expr);                                                                \
    if (e__ != cudaSuccess) return tgnn::set_error(ctx, TGNN_ECUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)
#define TGNN_LAUNCH_OK(ctx, name)                                                            \
  do {                                                                                       \
    (ctx)->launches++;                                                                       \
    cudaError_t e__ = cudaGetLastError();                                                    \
    if (e__ != cudaSuccess) return tgnn::set_error(ctx, TGNN_ECUDA, "launch %s: %s", name, cudaGetErrorString(e__)); \
  } while (0)

// cudaFuncAttributeMaxDynamicSharedMemorySize is a setting per device (and the library may serve several devices
// from several threads of one process): each kernel keeps one of these to remember what it has raised where.
struct SmemLimit {
  int bytes[64] = {};
  std::mutex lock;
};
template <typename F>
inline int raise_smem_limit(tgnn_ctx* ctx, F kernel, int bytes, SmemLimit& st) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
    return set_error(ctx, TGNN_ECUDA, "cudaGetDevice failed or device index above 63");
  std::lock_guard<std::mutex> g(st.lock);
  if (st.bytes[dev] >= bytes) return TGNN_OK;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return set_error(ctx, TGNN_ECUDA, "cudaFuncSetAttribute(%d bytes): %s", bytes, cudaGetErrorString(e));
  st.bytes[dev] = bytes;
  return TGNN_OK;
}

// side[i] waits for everything enqueued so far on `from`.
inline int fork_to(tgnn_ctx* ctx, cudaStream_t from, cudaStream_t to) {
  cudaEvent_t e = ctx->ev[ctx->ev_next];
  ctx->ev_next = (ctx->ev_next + 1) % 32;
  if (cudaEventRecord(e, from) != cudaSuccess || cudaStreamWaitEvent(to, e, 0) != cudaSuccess)
    return set_error(ctx, TGNN_ECUDA, "stream fork/join failed: %s", cudaGetErrorString(cudaGetLastError()));
  return TGNN_OK;
}

// The two halves of fork_to, for a dependency that is recorded now and waited for later.
inline cudaEvent_t mark_stream(tgnn_ctx* ctx, cudaStream_t on) {
  cudaEvent_t e = ctx->ev[ctx->ev_next];
  ctx->ev_next = (ctx->ev_next + 1) % 32;
  return cudaEventRecord(e, on) == cudaSuccess ? e : nullptr;
}
inline int wait_mark(tgnn_ctx* ctx, cudaStream_t waiter, cudaEvent_t e) {
  if (!e || cudaStreamWaitEvent(waiter, e, 0) != cudaSuccess)
    return set_error(ctx, TGNN_ECUDA, "stream fork/join failed: %s", cudaGetErrorString(cudaGetLastError()));
  return TGNN_OK;
}

// Brackets one kernel launch with events when profiling is on.
struct KernelScope {
  tgnn_ctx* c;
  cudaStream_t s;
  long idx;
  KernelScope(tgnn_ctx* ctx, const char* name, cudaStream_t stream) : c(ctx), s(stream), idx(-1) {
    Profiler& p = ctx->prof;
    if (!p.on) return;
    if (p.used == p.entries.size()) {
      ProfEntry e{name, nullptr, nullptr};
      if (cudaEventCreate(&e.a) != cudaSuccess || cudaEventCreate(&e.b) != cudaSuccess) return;
      p.entries.push_back(e);
    }
    idx = (long)p.used++;
    p.entries[idx].name = name;
    cudaEventRecord(p.entries[idx].a, s);
  }
  ~KernelScope() {
    if (idx >= 0) cudaEventRecord(c->prof.entries[idx].b, s);
  }
};

// ---- integer kernels (k_index.cu) ----
int launch_prune_mask(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const int32_t* eid, const uint8_t* is_aux,
                      int n, int force_heavy, uint32_t drop_q32, uint64_t seed, int64_t batch_idx, uint8_t* keep_out,
                      int32_t* heavy_out, cudaStream_t s);
int launch_sample_recent(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, int32_t* nbr_out,
                         int32_t* eid_out, double* ts_out, int32_t* cnt_out, cudaStream_t s);
int launch_reduce_latest(tgnn_ctx* ctx, const int32_t* msg_node, const double* t, const int32_t* eid, int n_msg,
                         int32_t* uniq_out, int32_t* winner_out, int32_t* n_uniq_out, cudaStream_t s);
int launch_reduce_latest_events(tgnn_ctx* ctx, const int32_t* msg_node, const int32_t* src, const int32_t* dst,
                                const uint8_t* keep, const double* t, const int32_t* eid, int n_msg, int32_t* uniq_out,
                                int32_t* winner_out, int32_t* n_uniq_out, cudaStream_t s);
int launch_stage_inputs(tgnn_ctx* ctx, const int32_t* u_src, const int32_t* u_dst, const double* u_t,
                        const int32_t* u_eid, const uint8_t* u_keep, int n_u, const int32_t* q_src, const int32_t* q_dst,
                        const int32_t* q_neg, const double* q_t, int n_q, const uint8_t* loss_mask, cudaStream_t s);
int launch_unpack_mixed(tgnn_ctx* ctx, const unsigned char* packed, int n, int n_q, bool with_mask, int slot,
                        cudaStream_t s);
int launch_make_roots(tgnn_ctx* ctx, const int32_t* q_src, const int32_t* q_dst, const int32_t* q_neg,
                      const double* q_t, int n_q, cudaStream_t s);

// ---- memory path (k_memory.cu) ----
int launch_build_messages(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const double* t, const int32_t* eid,
                          const uint8_t* keep, int n, float* msg_out, int32_t* msg_node_out, cudaStream_t s);
int launch_memory_update(tgnn_ctx* ctx, const float* msg, const int32_t* uniq, const int32_t* winner,
                         const int32_t* n_uniq, cudaStream_t s);

// ---- embedding (k_embed.cu) ----
int launch_embed(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, const int32_t* nbr,
                 const int32_t* eid, const double* ts, const int32_t* cnt, float* h_out, cudaStream_t s);

int launch_embed_static(tgnn_ctx* ctx, const double* times, int n, const int32_t* nbr, const int32_t* eid,
                        const double* ts, cudaStream_t s);

// ---- backward + Adam (k_backward.cu) ----
int launch_apply_gradient(tgnn_ctx* ctx, float gscale, float* gradnorm_out, cudaStream_t s);
int launch_backward(tgnn_ctx* ctx, int n_q, const uint8_t* loss_mask, float* loss_out, float* gradnorm_out,
                    cudaStream_t s);

int launch_get_gates(tgnn_ctx* ctx, uint8_t* h_gate_out, uint8_t* hid_gate_out, cudaStream_t s);

// ---- dense projections (k_gemm.cu) ----
// C[M,N] (+)= sum_k A(m,k) B(k,n) (+ bias[n]) (ReLU);  A(m,k) = A[m*a_rs + k*a_cs], B(k,n) = B[k*b_rs + n*b_cs].
struct GemmArgs {
  const float* A; int64_t a_rs, a_cs;
  const float* B; int64_t b_rs, b_cs;
  float* C; int64_t ldc;
  int M, N, K;            // capacities when the matching device count is given
  const int32_t* dev_M;   // optional device-side row count (<= M)
  const int32_t* dev_K;   // optional device-side contraction length (<= K)
  const float* bias;      // optional [N], added once
  float* rowsum_out;      // optional [M]: += sum_k A(m,k) (bias gradient of a transposed product)
  int relu;               // apply ReLU in the epilogue (store mode only)
  int accumulate;         // atomicAdd into C (C must hold valid data); required when split_k > 1
  int split_k;            // >= 1
  const int32_t* a_idx;   // optional (tensor-core path, K-major A): leading a_tab_cols columns of row m come from
  const float* a_tab;     //   a_tab[a_idx[m] * a_tab_cols + k] (zero row if a_idx[m] < 0) instead of A
  int a_tab_cols;
  int64_t a_tab_rows;     //   rows of a_tab: an index at or beyond it reads as a zero row
  int site;               // WeightSiteId + 1 when B is that weight matrix (0: none); lets the kernel use its image
  int precise;            // tensor-core mode only: 3xTF32 head/tail split, close to fp32 accuracy
  int tail_slack;         // both operands live in the workspace arena: a tiled load may read up to 124 bytes past
                          //   the end of a matrix whose width is not a multiple of 32 (the arena ends in slack)
};
int launch_gemm(tgnn_ctx* ctx, const GemmArgs& g, const char* name, cudaStream_t s);
int launch_gemm_tf32(tgnn_ctx* ctx, const GemmArgs& g, const char* name, cudaStream_t s);  // k_gemm_tc.cu
// ---- split-operand projections (k_gemm_split.cu) ----
int launch_prep_split_weights(tgnn_ctx* ctx, cudaStream_t s);
int launch_split_rows(tgnn_ctx* ctx, const float* X, int64_t ld_in, int64_t rows, int cols, const int32_t* dev_rows,
                      const SplitMat& out, int ones_col, const char* name, cudaStream_t s);   // honours out.fp16, out.scale
int launch_gemm_split(tgnn_ctx* ctx, const SplitMat& A, const SplitMat& B, int mn_major, float* C, int64_t ldc, int M, int N,
                      int K, const float* bias, int relu, int accumulate, int split_k, const char* name, cudaStream_t s,
                      int debug_withhold = 0, unsigned spin_limit = 0, int extra_col = -1, float* extra_out = nullptr, long long* trace = nullptr,
                      int single = -1, int launches = 1, int pair = -1);
size_t plan_weight_sites(tgnn_ctx* ctx);                       // fills ctx->sites, returns the image bytes needed
int launch_prep_weights(tgnn_ctx* ctx, cudaStream_t s);        // writes all images from the current parameters
int launch_prep_head(tgnn_ctx* ctx, cudaStream_t s);           // k_backward.cu: W_1 transposed for the tile head

}  // namespace tgnn
