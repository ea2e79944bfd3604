/*
 * tgnn.h -- C ABI of the B200 (sm_100a) training-step library for a TGN-style
 * memory-based temporal graph network.
 *
 * One chronological training step over a mixed event batch (target events plus
 * flagged auxiliary replay events), as framed by the paper:
 *   events e=(u,v,t,x) sorted by t, node memory m_u(t)         Section III-A
 *   Message / Update recursion                                   Eq. 1, Eq. 2
 *   mixed batch with an event-type mask                          Eq. 5
 *   pruning set and pruned batch                                 Eq. 10, Eq. 11
 *   target mask and masked loss                                  Eq. 12, Eq. 13
 *   per-batch order (prune, execute in timestamp order, masked
 *   loss, backprop + gradient norm g_r, parameter update)        Algorithm 2
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer BORROWED from the caller unless the
 *     parameter name ends in `_host`.  The library owns only the workspace it
 *     allocates in tgnn_create (sized from the capacities in tgnn_config) and
 *     never allocates afterwards.
 *   - All work is enqueued on the caller's stream (`stream` is a cudaStream_t
 *     passed as void*); no call synchronises the device unless documented.
 *   - Every function returns TGNN_OK or a negative error code; the message of
 *     the last error of a context is available from tgnn_last_error.  Invalid
 *     arguments are rejected on the host before anything is launched.
 *   - A context is used from one host thread at a time, on one stream.
 *   - Node ids are int32 in [0, num_nodes); event ids are int32 positions in
 *     the time-sorted stream; timestamps are fp64 wherever they are compared
 *     or subtracted.
 *
 * Model (the paper leaves internals open; these are the textbook forms)
 *   d = memory = time-encoding = embedding dimension, d_e = edge-feature
 *   dimension, d_msg = 3d + d_e, d_kv = 2d + d_e, heads H, k neighbors.
 *   Phi(dt)_c = cos(fmaf(w_c, (float)dt, b_c)), dt formed in fp64, argument in fp32.
 *   Parameters live in ONE flat fp32 vector, matrices [out, in] row-major, in
 *   this order (tgnn_param_layout reports the offsets):
 *     time_w[d] time_b[d]
 *     gru_w_i[3d,d_msg] gru_w_h[3d,d] gru_b_i[3d] gru_b_h[3d]     gates r,z,n
 *     w_q[d,2d] b_q[d]  w_k[d,d_kv] w_v[d,d_kv] b_k[d] b_v[d]  w_o[d,2d] b_o[d]
 *     w_1[d,2d] b_1[d] w_2[d] b_2[1]
 */
#ifndef TGNN_H_
#define TGNN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  TGNN_OK = 0,
  TGNN_EINVAL = -1,    /* null pointer or value out of range */
  TGNN_ESHAPE = -2,    /* dimensions inconsistent with the configuration */
  TGNN_ECAPACITY = -3, /* n exceeds a capacity given at tgnn_create */
  TGNN_ESTATE = -4,    /* call out of order (graph/state not set, no forward before backward ...) */
  TGNN_ECUDA = -5,     /* a CUDA runtime call failed; see tgnn_last_error */
  TGNN_ETIMEOUT = -6,  /* a bounded device-side wait expired (reported through tgnn_status) */
  TGNN_EBOUNDS = -7    /* a device-side index check failed (reported through tgnn_status) */
};

enum { TGNN_F32 = 0, TGNN_BF16 = 1 };

/* math_mode: how the dense projections are computed.  Gates, softmax, loss, the
 * time encoding and Adam are always fp32. */
enum {
  TGNN_MATH_FP32 = 0,     /* fp32 FMA tiles */
  TGNN_MATH_TF32 = 1,     /* tcgen05 tensor cores: every operand is split into a TF32 head and a TF32
                             tail (3 MMAs per product, fp32 accumulation in TMEM), close to fp32 accuracy */
  TGNN_MATH_F16X3 = 3,    /* as TGNN_MATH_TF32, except that the three products over the sampled-neighbor rows (key/value
                             projection, its input gradient and its weight gradient) hold each fp32 operand as two fp16
                             numbers (hi + lo, 22 mantissa bits; gradients are scaled by a power of two into fp16's
                             range) and run as three fp16 tensor-core passes with fp32 accumulation: the accuracy of
                             the TF32 split at half its tensor time.  Edge features and memory values must stay below
                             fp16's largest number (65504) in magnitude.  With a bf16 edge-feature table (tolerance
                             1e-2) the weight gradient of the key/value projection, a leaf of the backward pass, reads
                             only the hi numbers (one pass) */
  TGNN_MATH_TF32_FAST = 2 /* tcgen05 tensor cores, single TF32 pass in the forward projections (the gradient
                             products keep the split).  Outputs stay within 2e-3, but gradient tensors whose
                             terms cancel (time encoder, W_k) can be off by ~1e-2 of their largest entry. */
};

/* model: which memory-based model the step trains.  Steps (0)-(3), the head, the loss and Adam are
 * shared; steps (4)-(5) and their backward differ. */
enum {
  TGNN_MODEL_TGN = 0,   /* GRU memory update + one temporal attention layer over the k most recent neighbors */
  TGNN_MODEL_JODIE = 1  /* plain recurrent cell  m' = tanh(W_i msg + b_i + W_h m + b_h)  and the
                           time-projected embedding  h(n, t) = m_n * (1 + dt w_p + b_p),
                           dt = fp32(t - last_update[n]); no neighbor sampling, no attention */
};

#if defined(__GNUC__)
#define TGNN_API __attribute__((visibility("default")))
#else
#define TGNN_API
#endif

typedef struct tgnn_ctx tgnn_ctx;

typedef struct {
  int64_t num_nodes;
  int32_t d;          /* memory / time / embedding dimension, <= 256, multiple of 4 and of heads */
  int32_t d_e;        /* edge-feature dimension, >= 0, even */
  int32_t k;          /* neighbors per root, 1..32 */
  int32_t heads;      /* attention heads */
  int32_t feat_dtype; /* TGNN_F32 or TGNN_BF16 */
  int32_t max_events; /* capacity: events in one mixed batch */
  int32_t max_roots;  /* capacity: roots in one tgnn_embed call (3 per target event) */
  int32_t math_mode;  /* TGNN_MATH_* */
  float lr, beta1, beta2, eps; /* Adam */
  int32_t model;      /* TGNN_MODEL_* */
  int32_t embed_aux;  /* 0: tgnn_step_mixed_host embeds and scores the target events only (auxiliary events
                         carry loss weight 0, so their embeddings cannot change the result);
                         1: it embeds and scores EVERY event of the mixed batch and applies the target
                         mask of Eq. 12 in the loss (Eq. 13), the cost model of the workload analysis
                         in which auxiliary events pay the forward pass too.  Loss, gradients and
                         state are the same either way up to summation order. */
} tgnn_config;

/* ---- life cycle --------------------------------------------------------- */

/* Allocates the context and all device workspace on the current device.
 * cfg_host is read during the call only.  On failure *out is NULL. */
TGNN_API int tgnn_create(const tgnn_config* cfg_host, tgnn_ctx** out);
/* Frees the workspace.  Synchronises the device.  NULL is accepted. */
TGNN_API int tgnn_destroy(tgnn_ctx* ctx);
/* Message of the last error recorded in ctx (static string if ctx is NULL). Never NULL. */
TGNN_API const char* tgnn_last_error(const tgnn_ctx* ctx);

/* Number of fp32 parameters, and the offsets of the 20 tensors followed by the total (out21_host has
 * 21 entries): time_w, time_b, update-cell W_i [g*d, d_msg], W_h [g*d, d], b_i, b_h (g = 3 gates for
 * the GRU, 1 for the plain cell), W_q, b_q, W_k, W_v, b_k, b_v, W_o, b_o, W_1, b_1, w_2, b_2, then the
 * projection's w_p, b_p.  Tensors a model does not have are empty (the attention block for
 * TGNN_MODEL_JODIE, the projection for TGNN_MODEL_TGN); in memory w_p, b_p sit between b_o and W_1.
 * Pure host computations. */
TGNN_API int64_t tgnn_param_count(const tgnn_config* cfg_host);
TGNN_API int tgnn_param_layout(const tgnn_config* cfg_host, int64_t* out21_host);

/* Time-sorted adjacency (T-CSR) of the whole stream, both directions of every
 * event: node n owns entries [indptr[n], indptr[n+1]) sorted by (ts, eid).
 * indptr:int64[num_nodes+1], nbr,eid:int32[n_entries], ts:f64[n_entries].
 * Borrowed until replaced or the context is destroyed. */
TGNN_API int tgnn_set_graph(tgnn_ctx* ctx, const int64_t* indptr, const int32_t* nbr, const int32_t* eid, const double* ts,
                   int64_t n_entries);
/* Edge-feature table [num_events, d_e] row-major, fp32 or bf16 per dtype (must
 * equal cfg.feat_dtype); may be NULL when d_e == 0.  Borrowed. */
TGNN_API int tgnn_set_edge_features(tgnn_ctx* ctx, const void* efeat, int dtype, int64_t num_events, int d_e);
/* Model state, mutated in place by tgnn_memory_update and tgnn_backward_step:
 * memory:f32[num_nodes,d], last_update:f64[num_nodes], params/adam_m/adam_v:
 * f32[param_count], step:int64[1] (Adam step counter, device).  Borrowed.
 * Call again after changing params from outside (cached operand copies are refreshed). */
TGNN_API int tgnn_set_state(tgnn_ctx* ctx, float* memory, double* last_update, float* params, float* adam_m, float* adam_v,
                   int64_t* step);

/* ---- the step ------------------------------------------------------------ */

/* Step (0): load-aware pruning of auxiliary replay events (Eq. 10-11) on a
 * mixed batch (Eq. 5).  cnt[v] = endpoint occurrences of node v among the n
 * events, T = number of nodes with cnt > 0; heavy = (max cnt * T > 8 n), i.e.
 * "max > 4 x mean over touched nodes", unless force_heavy is 0 or 1, in which
 * case the caller's flag H (e.g. the batch-time EMA rule of Eq. 9) is used.
 * keep_out[i] = 1 for every target event (is_aux[i] == 0; targets are never
 * pruned).  A replay event is dropped iff heavy and (drop_q32 == 0xFFFFFFFF,
 * meaning all of them as in Eq. 11, or hash32(seed, batch_idx, eid[i]) <
 * drop_q32), where hash32 = top 32 bits of the SplitMix64 finaliser applied to
 * seed ^ batch_idx*0x9E3779B97F4A7C15 ^ (uint32)eid*0xC2B2AE3D27D4EB4F.
 * src,dst,eid:int32[n], is_aux:uint8[n] -> keep_out:uint8[n], heavy_out:int32[1]. */
TGNN_API int tgnn_prune_mask(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const int32_t* eid, const uint8_t* is_aux,
                    int n, int force_heavy, uint32_t drop_q32, uint64_t seed, int64_t batch_idx, uint8_t* keep_out,
                    int32_t* heavy_out, void* stream);

/* Step (1): most-recent-k temporal neighbor search ("temporal neighborhood
 * aggregation", Section VI-A model description).  For root i, p = first index
 * of node nodes[i]'s T-CSR slice with ts[p] >= times[i]; cnt = min(k, p -
 * indptr[node]); slot s < cnt is entry p-1-s (slot 0 most recent); unused
 * slots hold nbr = eid = -1, ts = 0.
 * nodes:int32[n], times:f64[n] -> nbr_out,eid_out:int32[n,k], ts_out:f64[n,k], cnt_out:int32[n]. */
TGNN_API int tgnn_sample_recent(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, int32_t* nbr_out,
                       int32_t* eid_out, double* ts_out, int32_t* cnt_out, void* stream);

/* Step (2): Message of Eq. 1 for the n update events (the previous kept mixed
 * batch): message 2i goes to src[i] (role 0), 2i+1 to dst[i] (role 1), layout
 * [m_self || m_other || x_eid || Phi(t - last_update[self])], memory and
 * last_update as they stand when the kernel runs.  keep may be NULL (all kept);
 * events with keep[i] == 0 give msg_node = -1 and zero rows.
 * msg_node_out:int32[2n] is always written.  msg_out:f32[2n,d_msg] may be NULL:
 * the rows then stay virtual and tgnn_memory_update gathers the winners' rows
 * itself from the event arrays, which must stay valid until that call is enqueued. */
TGNN_API int tgnn_build_messages(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const double* t, const int32_t* eid,
                        const uint8_t* keep, int n, float* msg_out, int32_t* msg_node_out, void* stream);

/* Step (3): per-node latest-event reduction.  Message j belongs to event j>>1
 * with role j&1; t,eid are per event ([n_msg/2]).  For every node with a
 * message (msg_node >= 0) the winner is the message with the lexicographically
 * largest (t, eid, role).  uniq_out:int32[<=n_msg] touched nodes ascending,
 * winner_out:int32[<=n_msg] message index per unique node, n_uniq_out:int32[1]. */
TGNN_API int tgnn_reduce_latest(tgnn_ctx* ctx, const int32_t* msg_node, const double* t, const int32_t* eid, int n_msg,
                       int32_t* uniq_out, int32_t* winner_out, int32_t* n_uniq_out, void* stream);

/* Step (4): Update of Eq. 2 as a GRU cell (gate order r,z,n; r multiplies the
 * hidden candidate pre-activation including its bias; TGNN_MODEL_JODIE: the plain tanh cell) on the winners:
 * memory[uniq[u]] <- GRU(msg[winner[u]], memory[uniq[u]]), last_update[uniq[u]]
 * <- t[winner[u]>>1]; every new row is computed from pre-call memory before any
 * row is written.  msg may be NULL if tgnn_build_messages ran with msg_out NULL
 * (rows are gathered from its event arrays).  Activations are kept in the
 * workspace for tgnn_backward_step.  n_uniq is a device scalar. */
TGNN_API int tgnn_memory_update(tgnn_ctx* ctx, const float* msg, const int32_t* uniq, const int32_t* winner,
                       const int32_t* n_uniq, void* stream);

/* Step (5): one multi-head temporal attention layer.  For root i: query from
 * [m_root || Phi(0)], keys/values from [m_nbr || x_eid || Phi(times[i] - ts)] of
 * its cnt[i] valid neighbor slots, softmax over valid slots of q.k/sqrt(d/H) per
 * head (zero vector if cnt = 0), h = ReLU(W_o [a || m_root] + b_o).
 * Inputs as produced by tgnn_sample_recent -> h_out:f32[n,d].  Activations are
 * kept for tgnn_backward_step; the neighbor arrays must stay valid until then.
 * TGNN_MODEL_JODIE: h[i] = memory[nodes[i]] * (1 + dt w_p + b_p) with dt = fp32(times[i] -
 * last_update[nodes[i]]); nbr, eid, ts, cnt are ignored and may be NULL. */
TGNN_API int tgnn_embed(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, const int32_t* nbr, const int32_t* eid,
               const double* ts, const int32_t* cnt, float* h_out, void* stream);

/* Step (6): masked link-prediction loss (Eq. 13) on the rows of the last
 * tgnn_embed call, laid out as [src | dst | neg] blocks of n_q rows:
 *   score(a,b) = w_2 . ReLU(W_1 [a || b] + b_1) + b_2,
 *   l_j = softplus(-score(src_j,dst_j)) + softplus(score(src_j,neg_j)),
 *   L = sum_j M_j l_j / sum_j M_j, or 0 if no event has M_j = 1,
 * loss_mask:uint8[n_q] (NULL = all ones) being the target mask of Eq. 12; then
 * the exact gradient w.r.t. all parameters (rows written by the last
 * tgnn_memory_update depend on the GRU and time-encoder parameters, all other
 * table reads are constants), the gradient norm g_r = ||grad||_2 (Algorithm 2,
 * "compute gradient norm") and one Adam step (step += 1, bias-corrected, no
 * weight decay).  loss_out, gradnorm_out: f32 device scalars (may be NULL). */
TGNN_API int tgnn_backward_step(tgnn_ctx* ctx, int n_q, const uint8_t* loss_mask, float* loss_out, float* gradnorm_out,
                       void* stream);

/* ---- whole step, one call ------------------------------------------------- */

/* Runs steps (1)-(6) in lag-one order on device-resident event arrays:
 * the update events (previous kept batch: u_src..u_keep, n_u, may be 0) refresh
 * memory, then the n_q target events (q_src,q_dst,q_neg:int32[n_q], q_t:f64[n_q])
 * are sampled, embedded, scored and trained on.  Equivalent to calling the six
 * entry points above with workspace-owned intermediates.  The inputs are first
 * copied into fixed staging buffers by the first kernel of the step; treat them
 * as borrowed until the stream has passed that kernel.
 * Graph replay: the second call with the same (n_u, n_q, keep / mask presence,
 * output pointers) records the step's launch sequence with CUDA stream capture
 * on `stream` (which therefore must not be the legacy default stream; if capture
 * is refused the library silently keeps launching kernel by kernel) and later
 * calls replay the instantiated graph.  tgnn_set_graph_replay(ctx, 0) turns this
 * off.  Profiling (tgnn_profile_begin) always uses plain launches. */
TGNN_API int tgnn_train_step(tgnn_ctx* ctx, const int32_t* u_src, const int32_t* u_dst, const double* u_t, const int32_t* u_eid,
                    const uint8_t* u_keep, int n_u, const int32_t* q_src, const int32_t* q_dst, const int32_t* q_neg,
                    const double* q_t, int n_q, const uint8_t* loss_mask, float* loss_out, float* gradnorm_out,
                    void* stream);

TGNN_API int tgnn_set_graph_replay(tgnn_ctx* ctx, int enable);

/* ---- gradient synchronisation across workers (Algorithm 2: the gradient norm g_r "is computed from
 * the synchronised model gradients") ------------------------------------------------------------
 * tgnn_set_grad_sync(ctx, 1): from now on tgnn_backward_step / tgnn_train_step and the host forms stop
 * after the gradient: the complete fp32 gradient of the step is left in the context's gradient buffer,
 * the loss is written, gradnorm_out receives the norm of the LOCAL gradient, and parameters, Adam
 * moments and the step counter are untouched.  The caller reduces the buffer across workers in stream
 * order (e.g. an NCCL all-reduce on the same stream) and calls tgnn_apply_gradient, which multiplies the
 * buffer by `scale` (1 / workers for a mean; the product is stored), computes g_r = ||gradient||_2 into
 * gradnorm_out (f32 device scalar, may be NULL) and performs the Adam step (step += 1).  A new step
 * before the pending gradient is applied is refused with TGNN_ESTATE.  tgnn_set_grad_sync(ctx, 0)
 * returns to the fused form; switching drops recorded step graphs (they are recorded again).
 * tgnn_grad_buffer: *grads_dev_out = the buffer (device, param_count floats, owned by the context and
 * valid for its lifetime; layout = the parameter layout), *count_out = param_count.  Both host pointers. */
TGNN_API int tgnn_set_grad_sync(tgnn_ctx* ctx, int defer);
TGNN_API int tgnn_grad_buffer(tgnn_ctx* ctx, float** grads_dev_out, int64_t* count_out);
TGNN_API int tgnn_apply_gradient(tgnn_ctx* ctx, float scale, float* gradnorm_out, void* stream);

/* The same step with HOST inputs and outputs: the event arrays are copied to
 * workspace staging buffers with cudaMemcpyAsync (pin them for overlap), and
 * loss / gradient norm are copied back to loss_host / gradnorm_host (may be
 * NULL).  The call returns after enqueueing; synchronise the stream before
 * reading the two scalars or reusing the host buffers. */
TGNN_API int tgnn_train_step_host(tgnn_ctx* ctx, const int32_t* u_src_host, const int32_t* u_dst_host, const double* u_t_host,
                         const int32_t* u_eid_host, const uint8_t* u_keep_host, int n_u, const int32_t* q_src_host,
                         const int32_t* q_dst_host, const int32_t* q_neg_host, const double* q_t_host, int n_q,
                         const uint8_t* loss_mask_host, float* loss_host, float* gradnorm_host, void* stream);

/* The streaming form of the step, host inputs: one call per mixed batch (Eq. 5), in stream order.
 * The call copies the batch to the device as one packed block, computes its prune mask (step 0,
 * arguments as in tgnn_prune_mask) beside the rest of the step, and trains on its target events
 * (is_aux == 0, in batch order; neg_host holds one negative destination per target event; with
 * cfg.embed_aux = 1 every event of the batch is embedded and scored under the mask 1 - is_aux, neg_host
 * holds one negative per EVENT and max_roots must cover 3 n) after the
 * PREVIOUS call's batch, as kept by its mask, has updated memory (lag-one order).  The batch then
 * stays on the device for the next call.  tgnn_set_state restarts the sequence (no previous batch).
 * Host arrays may be pageable and are free for reuse when the call returns; loss_host /
 * gradnorm_host (may be NULL) are written by asynchronous copies: synchronise the stream first. */
TGNN_API int tgnn_step_mixed_host(tgnn_ctx* ctx, const int32_t* src_host, const int32_t* dst_host, const double* t_host,
                                  const int32_t* eid_host, const uint8_t* is_aux_host, int n, const int32_t* neg_host,
                                  int force_heavy, uint32_t drop_q32, uint64_t seed, int64_t batch_idx,
                                  float* loss_host, float* gradnorm_host, void* stream);

/* ---- debug / parity -------------------------------------------------------- */

/* Copies the parameter gradient of the last tgnn_backward_step to grads_out:f32[param_count]. */
TGNN_API int tgnn_debug_get_grads(tgnn_ctx* ctx, float* grads_out, void* stream);
/* Copies the embeddings h of the last tgnn_embed call (or of the last whole step) to h_out:f32[n_roots, d]. */
TGNN_API int tgnn_debug_get_embeddings(tgnn_ctx* ctx, float* h_out, void* stream);
/* The ReLU branch each unit took in the last tgnn_embed / tgnn_backward_step pair, as bytes:
 * h_gate_out:uint8[n_roots, d] (1 where h > 0), hid_gate_out:uint8[2 n_q, d] (hidden layer of the
 * link-prediction head, positive pairs first).  A parity check needs them because the derivative
 * of ReLU jumps at zero: a pre-activation closer to zero than the arithmetic resolves may fall on
 * either side, and the reference must differentiate the branch the kernel took. */
TGNN_API int tgnn_debug_get_gates(tgnn_ctx* ctx, uint8_t* h_gate_out, uint8_t* hid_gate_out, void* stream);
/* The dense-projection kernel on its own (the one the configured math_mode selects), for
 * parity tests: C[M,N] (+)= sum_k A(m,k) B(k,n) (+ bias[n]) (ReLU), with element strides
 * A(m,k) = A[m*a_rs + k*a_cs], B(k,n) = B[k*b_rs + n*b_cs], C row-major with leading
 * dimension ldc.  dev_M / dev_K (device int32, may be NULL) cap M / K at run time; bias [N]
 * and rowsum_out [M] (+= sum_k A(m,k), the bias gradient of a transposed product) may be
 * NULL; accumulate != 0 adds into C atomically and is required when split_k > 1; precise != 0
 * selects the 3xTF32 head/tail split in the tensor-core mode (ignored in the fp32 mode). */
TGNN_API int tgnn_debug_gemm(tgnn_ctx* ctx, const float* A, int64_t a_rs, int64_t a_cs, const float* B, int64_t b_rs,
                             int64_t b_cs, float* C, int64_t ldc, int M, int N, int K, const int32_t* dev_M,
                             const int32_t* dev_K, const float* bias, float* rowsum_out, int relu, int accumulate,
                             int split_k, int precise, void* stream);
/* Device status word (0 or the first TGNN_ETIMEOUT / TGNN_EBOUNDS recorded by a
 * kernel) copied to *status_host.  Synchronises the stream. */
TGNN_API int tgnn_status(tgnn_ctx* ctx, int32_t* status_host, void* stream);
/* Resets the device status word to 0 (enqueued on `stream`): after a recorded TGNN_ETIMEOUT / TGNN_EBOUNDS
 * has been read and dealt with, so that the next one can be seen. */
TGNN_API int tgnn_clear_status(tgnn_ctx* ctx, void* stream);
/* Number of kernels this context has launched since creation (host counter). */
TGNN_API int64_t tgnn_kernel_launches(const tgnn_ctx* ctx);

/* The split-operand projection kernel on its own, for parity tests (sm_100 tensor cores, any math_mode): the
 * fp32 operands are first split into two fp16 planes each (hi = fp16(x), lo = fp16(x - hi), 22 mantissa bits
 * together) inside `scratch` (device, 256-byte aligned, >= 2 * 2 * (rows * ceil8(cols)) bytes per operand plus
 * 256), then C[M,N] (+)= A B (+ bias[n]) (ReLU) runs as three fp16 passes with fp32 accumulation.  Strides as in
 * tgnn_debug_gemm, with the restriction that either both operands have the contraction index contiguous
 * (a_cs = 1, b_rs = 1) or both have the other index contiguous (a_rs = 1, b_cs = 1: C = A^T B over matrix rows).
 * accumulate / split_k as in tgnn_debug_gemm.  debug_withhold > 0 makes the kernel keep that many shared-memory
 * slots to itself instead of handing them back, and spin_limit > 0 shortens its bounded waits: together they let
 * a test make a wait run out (the kernel then records TGNN_ETIMEOUT, stores nothing further, frees its tensor
 * memory and returns; the context stays usable).  Both 0 in normal use.  Environment switches read by this call
 * only: TGNN_GEMM_PAIR=0|1 forces the one-CTA-per-tile form or the CTA-pair form (one 256-row MMA across two SMs,
 * each loading half of the B tile; default: pairs for K-major products of 32 row tiles and more),
 * TGNN_GEMM_SINGLE=0|1 the walk by pairs of row tiles or by single tiles, TGNN_GEMM_BF16=1 bf16 planes,
 * TGNN_GEMM_SCALE=s a scale of 2^s on A, TGNN_GEMM_PASSES=1 only the hi planes (one pass, 11-bit operands: the
 * form the step uses for the key/value weight gradient when the feature table is bf16). */
TGNN_API int tgnn_debug_gemm_split(tgnn_ctx* ctx, const float* A, int64_t a_rs, int64_t a_cs, const float* B, int64_t b_rs,
                                   int64_t b_cs, float* C, int64_t ldc, int M, int N, int K, const float* bias, int relu,
                                   int accumulate, int split_k, void* scratch, int64_t scratch_bytes, int debug_withhold,
                                   uint32_t spin_limit, void* stream);

/* ---- for callers that cannot allocate --------------------------------------- */

/* The paper has no counterpart to this entry point; it exists for hosts that
 * keep every byte of device memory under their own plan -- a serving process
 * with a fixed memory budget, a framework sandbox that hands an operator only
 * the buffers it was given -- where a cudaMalloc made by a library either is
 * forbidden, fails against the budget, or stalls the device while it runs.
 * Such a host cannot use tgnn_create (it allocates the workspace), so this is
 * step (3), the per-node latest-event reduction, with the same semantics as
 * tgnn_reduce_latest but no context: its per-node scratch tables live in an
 * array compiled into the library (20 bytes per node, TGNN_STATIC_MAX_NODES
 * nodes = 1.25 MiB, held by every GPU that loads the library until the process
 * exits).  Nothing is allocated or freed, by the library or on its behalf.
 *   msg_node:int32[n_msg], t:f64[n_msg/2], eid:int32[n_msg/2] (message j belongs
 *   to event j>>1 with role j&1; msg_node < 0 = dropped) -> uniq_out, winner_out:
 *   int32[<= min(n_msg, num_nodes)], n_uniq_out:int32[1]; all device pointers
 *   borrowed for the call; stream is a cudaStream_t.
 * num_nodes above TGNN_STATIC_MAX_NODES is refused with TGNN_ECAPACITY.  On any
 * failure a message is written to err_host (host buffer of err_size bytes, may
 * be NULL).  A message whose node id is >= num_nodes is skipped on the device
 * without being used as an index, and the call then reports it by writing -1 to
 * n_uniq_out (uniq_out / winner_out are undefined in that case); there is no
 * status word here, so check n_uniq_out.
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current) and keeps it for the life of
 * the process; make that first call before any stream capture begins.  The kept
 * address does not survive a cudaDeviceReset of that device: a process that
 * resets a device must not call this entry point on it afterwards.
 * All calls share the one array and it keeps what the last call left, so the
 * kernel clears the entries it uses before it starts; two calls that overlap
 * on the same GPU (different streams, or two threads) race on it and give
 * wrong results -- serialise them. */
#define TGNN_STATIC_MAX_NODES 65536
TGNN_API int tgnn_reduce_latest_static(const int32_t* msg_node, const double* t, const int32_t* eid, int n_msg,
                                       int64_t num_nodes, int32_t* uniq_out, int32_t* winner_out, int32_t* n_uniq_out,
                                       void* stream, char* err_host, int err_size);

/* Per-kernel timing for benchmarks (no counterpart in the paper beyond its
 * per-phase time breakdown, Table 5).  After tgnn_profile_begin every kernel
 * launch is bracketed by a CUDA event pair on the caller's stream until
 * tgnn_profile_report, which synchronises the device, writes one line per kernel
 * name ("name launches total_ms\n", NUL-terminated, truncated to size bytes)
 * into buf_host and switches profiling off.  Creates events on first use. */
TGNN_API int tgnn_profile_begin(tgnn_ctx* ctx);
TGNN_API int tgnn_profile_report(tgnn_ctx* ctx, char* buf_host, int64_t size);
/* Same recording, reported launch by launch in issue order: "name start_us duration_us\n", start
 * relative to the first recorded launch (the internal side streams make launches overlap). */
TGNN_API int tgnn_profile_timeline(tgnn_ctx* ctx, char* buf_host, int64_t size);

/* ---- adaptive runtime controller (Eq. 6-9, Algorithm 2): host-side, no GPU work -------------
 * Keeps the exponential moving averages of the gradient norm g_r (Eq. 6, factor alpha) and of
 * the measured batch time c_r (Eq. 8, factor beta) and takes the two per-batch decisions of
 * Algorithm 2.  An average that is exactly 0 restarts from the next sample.  All arithmetic is
 * fp64.  Every pointer is a HOST pointer; the object is owned by the caller between create and
 * destroy and is not thread-safe.
 *
 * tgnn_controller_create   alpha, beta in (0, 1]; tau_g, tau_c > 0; K >= 1 (candidate cache-refresh
 *                          boundaries are the batches r with r % K == 0); else TGNN_EINVAL
 *                          (TGNN_ECAPACITY if the host allocation fails).
 * tgnn_controller_begin_batch   the decisions before batch r (r >= 0) runs:
 *     *boundary_out = 1 if r is a candidate boundary, else 0;
 *     *sync_out     = S_r of Eq. 7 at a boundary (0: skip the refresh, when r > 0, the gradient
 *                     average is > 0 and the last norm is < tau_g * average; else 1), -1 elsewhere;
 *     *heavy_out    = H_r of Eq. 9 (1 when r > 0, the time average is > 0 and the last batch time
 *                     is > tau_c * average; else 0) -- pass it as force_heavy, with
 *                     drop_q32 = 0xFFFFFFFF, to prune every pure replay event of the batch (Eq. 10-11).
 *     On one GPU there is no remote cache: S_r is reported for the log only.
 * tgnn_controller_end_batch     folds g_r (>= 0) and c_r (>= 0, any unit) into the averages after
 *                          the batch; NaN or negative values are refused with TGNN_EINVAL.
 * tgnn_controller_state    out_host[4] = {g average, last g, c average, last c}. */
typedef struct tgnn_controller tgnn_controller;
TGNN_API int tgnn_controller_create(double alpha, double beta, double tau_g, double tau_c, int K, tgnn_controller** out);
TGNN_API int tgnn_controller_destroy(tgnn_controller* ctl);
TGNN_API int tgnn_controller_begin_batch(tgnn_controller* ctl, int64_t r, int* boundary_out, int* sync_out,
                                         int* heavy_out);
TGNN_API int tgnn_controller_end_batch(tgnn_controller* ctl, double g_r, double c_r);
TGNN_API int tgnn_controller_state(const tgnn_controller* ctl, double* out_host);

/* ---- offline preprocessing: backward dependency scan and mixed batches (Algorithm 1, Eq. 5) ----
 * Stateless (no context); every pointer is a DEVICE pointer borrowed for the call unless named
 * *_host; work is enqueued on `stream` (a cudaStream_t) and nothing is allocated.  On failure a
 * message is written to err_host (host buffer of err_size bytes, may be NULL).
 *
 * The stream is src/dst[num_events] in timestamp order, cut into global batches of `batch` events
 * (the last may be short); window W_q holds batches qK .. qK+K-1 (the last may hold fewer); owner[n]
 * in [0, P) is the node ownership map pi.  nb = ceil(num_events / batch), Q = ceil(nb / K).
 *
 * tgnn_backward_scan runs Algorithm 1 for every worker p and window q:
 *   role_out[p * num_events + e] = 1 if e is a target event of worker p (pi(src) = p), 2 if it is an
 *       auxiliary replay event of p in its window, 0 if p's mixed batches do not contain it;
 *   n_sync_out[p * Q + q]        = |N_sync| of (p, q), the candidate boundary refresh set;
 *   sync_out[(p * Q + q) * num_nodes + n] = 1 if n is in that set, else 0 (may be NULL);
 *   scratch  int32[tgnn_backward_scan_scratch(...)]: per-block node tables, contents undefined after;
 *   status_out  device int32: zeroed by the call, set to 1 if a window's relaxation did not settle
 *       within its event count (cannot happen; the loop is bounded all the same).
 * Within a batch the walk is reverse chronological as between batches; the target events' remote
 * destinations enter the frontier before their batch is walked, as in the listing.
 * Errors: TGNN_EINVAL (null pointer, size < 1), TGNN_ECAPACITY (K * batch or P * Q out of int range),
 * TGNN_ECUDA.  num_events = 0 is a no-op. */
#define TGNN_SCAN_MAX_BLOCKS 592
TGNN_API int64_t tgnn_backward_scan_scratch(int64_t num_events, int batch, int K, int64_t num_nodes, int P);
TGNN_API int tgnn_backward_scan(const int32_t* src, const int32_t* dst, int64_t num_events, int batch, int K,
                                const int32_t* owner, int64_t num_nodes, int P, uint8_t* role_out,
                                int32_t* n_sync_out, uint8_t* sync_out, int32_t* scratch, int32_t* status_out,
                                void* stream, char* err_host, int64_t err_size);

/* tgnn_build_mixed forms one worker's mixed batches (Eq. 5) from its row of role_out: for every global
 * batch s the events with role != 0, in timestamp order, with the event-type mask, and the target
 * events among them.
 *   role            uint8[num_events], one worker's row;   neg  int32[num_events] negatives per event or NULL;
 *   mb_off_out      int32[nb + 1]: mixed batch s occupies [mb_off[s], mb_off[s+1]) of mb_src, mb_dst, mb_t,
 *                   mb_eid (stream position of the event), mb_aux (1 = auxiliary replay event);
 *   tgt_off_out     int32[nb + 1]: the targets of batch s occupy [tgt_off[s], tgt_off[s+1]) of tgt_src,
 *                   tgt_dst, tgt_t, tgt_neg (may be NULL; -1 where neg is NULL), tgt_eid;
 *   cap_mixed, cap_tgt  elements available in the mb_* / tgt_* arrays (num_events always suffices);
 *   status_out      device int32: zeroed by the call, set to 2 if a capacity was too small (the events
 *                   beyond it are not written).
 * Errors: TGNN_EINVAL, TGNN_ECAPACITY (num_events beyond int32), TGNN_ECUDA. */
TGNN_API int tgnn_build_mixed(const int32_t* src, const int32_t* dst, const double* t, const int32_t* neg,
                              int64_t num_events, int batch, const uint8_t* role, int32_t* mb_off_out,
                              int32_t* tgt_off_out, int64_t cap_mixed, int64_t cap_tgt, int32_t* mb_src, int32_t* mb_dst,
                              double* mb_t, int32_t* mb_eid, uint8_t* mb_aux, int32_t* tgt_src, int32_t* tgt_dst,
                              double* tgt_t, int32_t* tgt_neg, int32_t* tgt_eid, int32_t* status_out, void* stream,
                              char* err_host, int64_t err_size);

/* ---- boundary cache refresh (dynamic cache synchronisation: at an executed boundary, S_r = 1, worker p
 * fetches the state of every node in N_sync[p] from the worker that owns it) -------------------------
 * Stateless, device pointers, work enqueued on `stream`, nothing allocated; errors as above.  The
 * exchange between the workers' processes is the caller's (one all-to-all of packed rows); these
 * entry points compute who sends what and move the rows on each GPU.  A node's state is its memory
 * row and its last-update time; a packed row is d + 2 floats (the row, then the low and high halves
 * of the fp64 time), so d must be even and memory / packed 8-byte aligned.
 *
 * tgnn_refresh_plan: worker `me`'s plan for every window from tgnn_backward_scan's sync_out flags
 *   (uint8[P, Q, num_nodes]) and the ownership map:
 *   recv_nodes[q * cap + i], recv_off[q * (P + 1) + o]: the nodes of N_sync[me] in window q, grouped by
 *       owner o (group o occupies [recv_off[o], recv_off[o + 1])), ascending ids within a group;
 *   send_nodes / send_off: the nodes owned by `me` that worker r requests, grouped by r, ascending;
 *       group r of `me`'s send list equals group `me` of worker r's receive list, element by element.
 *   cap = elements per window in recv_nodes / send_nodes (the sum of the window's N_sync sizes over
 *       all workers always suffices); status_out: device int32, zeroed by the call, 2 if cap was too
 *       small (the excess is not written), 3 if a worker's N_sync names a node it owns (skipped).
 * tgnn_pack_rows:   packed[i] = state of nodes[i]      (n rows; what an owner sends)
 * tgnn_unpack_rows: state of nodes[i] = packed[i]      (n rows; what a requester received; nodes must be
 *       distinct or the result for a repeated node is one of its rows)
 *   status: device int32, NOT zeroed by these two; 4 is recorded for a node id outside [0, num_nodes)
 *   (packed as zeros / not written). */
TGNN_API int tgnn_refresh_plan(const uint8_t* sync, const int32_t* owner, int64_t num_nodes, int P, int Q, int me,
                               int64_t cap, int32_t* recv_nodes, int32_t* recv_off, int32_t* send_nodes,
                               int32_t* send_off, int32_t* status_out, void* stream, char* err_host, int64_t err_size);
TGNN_API int tgnn_pack_rows(const float* memory, const double* last_update, int64_t num_nodes, int d,
                            const int32_t* nodes, int n, float* packed, int32_t* status, void* stream, char* err_host,
                            int64_t err_size);
TGNN_API int tgnn_unpack_rows(float* memory, double* last_update, int64_t num_nodes, int d, const int32_t* nodes, int n,
                              const float* packed, int32_t* status, void* stream, char* err_host, int64_t err_size);

#ifdef __cplusplus
}
#endif
#endif /* TGNN_H_ */
