// C ABI: context life cycle, argument checks, and the sequencing of one training step.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>
#include <string>

#include "tgnn_internal.cuh"

namespace tgnn {

ParamLayout make_layout(int d_, int de_, int model) {
  ParamLayout L;
  const int64_t d = d_, de = de_;
  const bool jodie = model == TGNN_MODEL_JODIE;
  const int64_t g = jodie ? 1 : 3, att = jodie ? 0 : 1, prj = jodie ? 1 : 0;
  L.d = d; L.de = de; L.dmsg = 3 * d + de; L.dkv = 2 * d + de; L.dq = 2 * d; L.gates = g;
  int64_t o = 0;
  L.time_w = o; o += d;
  L.time_b = o; o += d;
  L.gru_wi = o; o += g * d * L.dmsg;
  L.gru_wh = o; o += g * d * d;
  L.gru_bi = o; o += g * d;
  L.gru_bh = o; o += g * d;
  L.wq = o; o += att * d * L.dq;
  L.bq = o; o += att * d;
  L.wk = o; o += att * d * L.dkv;
  L.wv = o; o += att * d * L.dkv;
  L.bk = o; o += att * d;
  L.bv = o; o += att * d;
  L.wo = o; o += att * d * 2 * d;
  L.bo = o; o += att * d;
  L.proj_w = o; o += prj * d;
  L.proj_b = o; o += prj * d;
  L.w1 = o; o += d * 2 * d;
  L.b1 = o; o += d;
  L.w2 = o; o += d;
  L.b2 = o; o += 1;
  L.total = o;
  return L;
}

int set_error(tgnn_ctx* ctx, int code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

namespace {

int check_config(const tgnn_config* c) {
  if (!c) return TGNN_EINVAL;
  if (c->num_nodes <= 0 || c->num_nodes > 0x7fffffff) return TGNN_EINVAL;
  if (c->d <= 0 || c->d > 256 || c->d % 4 != 0 || c->heads <= 0 || c->d % c->heads != 0) return TGNN_ESHAPE;
  if (c->d_e < 0 || c->d_e % 2 != 0) return TGNN_ESHAPE;
  if (c->k < 1 || c->k > 32 || c->heads * c->k > 1024) return TGNN_ESHAPE;
  if (c->feat_dtype != TGNN_F32 && c->feat_dtype != TGNN_BF16) return TGNN_EINVAL;
  if (c->max_events < 1 || c->max_roots < 3 || c->max_events > (1 << 24) || c->max_roots > (1 << 24)) return TGNN_EINVAL;
  if (c->math_mode != TGNN_MATH_FP32 && c->math_mode != TGNN_MATH_TF32 && c->math_mode != TGNN_MATH_TF32_FAST &&
      c->math_mode != TGNN_MATH_F16X3) return TGNN_EINVAL;
  if (c->model != TGNN_MODEL_TGN && c->model != TGNN_MODEL_JODIE) return TGNN_EINVAL;
  if (c->embed_aux != 0 && c->embed_aux != 1) return TGNN_EINVAL;
  if (!(c->lr >= 0.f) || !(c->beta1 >= 0.f && c->beta1 < 1.f) || !(c->beta2 >= 0.f && c->beta2 < 1.f) || !(c->eps > 0.f))
    return TGNN_EINVAL;
  return TGNN_OK;
}

struct Carver {
  char* base;
  size_t off;
  template <typename T>
  void take(T*& p, size_t count) {
    off = (off + 255) & ~(size_t)255;
    p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
  }
  // no alignment gap: keeps a group of buffers contiguous for a single memset
  template <typename T>
  void take_packed(T*& p, size_t count) {
    off = (off + 15) & ~(size_t)15;
    p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
  }
};

size_t carve(tgnn_ctx* ctx, char* base) {
  const tgnn_config& c = ctx->cfg;
  Workspace& w = ctx->ws;
  const size_t N = (size_t)c.num_nodes, d = c.d, k = c.k, H = c.heads;
  const size_t ne = c.max_events, U = ctx->U_cap, R = ctx->R_cap, NB = ctx->NB_cap, nq = ctx->nq_cap;
  Carver cv{base, 0};
  cv.take(w.hist, N);
  cv.take(w.best_t, N);
  cv.take(w.best_id, N);
  cv.take(w.win_msg, N);
  cv.take(w.node2slot, N);
  cv.take(w.prev_uniq, U);
  cv.take(w.prev_n_uniq, 4);
  cv.take(w.msg_node, U);
  cv.take(w.uniq, U);
  cv.take(w.winner, U);
  cv.take(w.n_uniq, 4);
  cv.take(w.r_node, R);
  cv.take(w.r_time, R);
  cv.take(w.nb_node, NB);
  cv.take(w.nb_eid, NB);
  cv.take(w.nb_ts, NB);
  cv.take(w.nb_cnt, R);
  cv.take(w.h, R * d);
  cv.take(w.st_u_src, ne); cv.take(w.st_u_dst, ne); cv.take(w.st_u_eid, ne);
  cv.take(w.st_q_src, nq); cv.take(w.st_q_dst, nq); cv.take(w.st_q_neg, nq);
  cv.take(w.st_u_t, ne); cv.take(w.st_q_t, nq);
  cv.take(w.st_u_keep, ne); cv.take(w.st_mask, nq);
  cv.take(w.X, U * ctx->ld_msg);
  cv.take(w.x_dt, U);
  cv.take(w.Xsin, U * d);
  cv.take(w.win_t, U);
  cv.take(w.Gi, U * 3 * d);
  cv.take(w.Gh, U * 3 * d);
  cv.take(w.g_r, U * d); cv.take(w.g_z, U * d); cv.take(w.g_n, U * d); cv.take(w.g_hn, U * d);
  cv.take(w.Z, NB * ctx->ld_kv);
  cv.take(w.z_dt, NB);
  cv.take(w.KV, NB * 2 * d);
  cv.take(w.Zq, R * 2 * d);
  cv.take(w.Q, R * d);
  cv.take(w.alpha, R * H * k);
  cv.take(w.cat_o, R * 2 * d);
  cv.take(w.head_wT, 2 * d * ((d + 3) / 4 * 4));
  cv.take(w.cat1, 2 * nq * 2 * d);
  cv.take(w.hid1, 2 * nq * d);
  cv.take(w.hid_gate, 2 * nq * d);
  cv.take(w.dcat1, 2 * nq * 2 * d);
  cv.take(w.dpre_o, R * d);
  cv.take(w.dcat_o, R * 2 * d);
  cv.take(w.dQ, R * d);
  cv.take(w.dzq, R * 2 * d);
  cv.take(w.dKV, NB * 2 * d);
  cv.take(w.dZmp, NB * 2 * d);
  cv.take(w.dGi, U * 3 * d);
  cv.take(w.dGh, U * 3 * d);
  cv.take(w.dXp, U * d);
  cv.take(w.adam_sc, 4);
  cv.take(w.counters, 4);
  cv.take(w.status, 4);
  // cleared together at the start of every backward pass: keep these six adjacent and in this order
  cv.take(w.grads, (size_t)ctx->L.total);
  cv.take_packed(w.dWkv_pad, (size_t)2 * d * ctx->ld_wkv);
  cv.take_packed(w.dMemU, U * d);
  cv.take_packed(w.red, 4);
  cv.take_packed(w.tg_acc, 4 * d);  // time encoder dw | db, time projection dw_p | db_p
  cv.take_packed(w.st_scalars, 4);
  // 256 bytes of slack: a tiled load of a transposed operand may run up to 124 bytes past the end of its matrix
  return ((cv.off + 255) & ~(size_t)255) + 256;
}

inline cudaStream_t S(void* stream) { return reinterpret_cast<cudaStream_t>(stream); }

// Recorded step graphs have the borrowed pointers (state, graph, feature table) and the launch sequence of
// the current mode baked into their kernel arguments: whenever one of those changes they are dropped and
// the next steps record new ones.
void drop_step_graphs(tgnn_ctx* ctx) {
  for (int i = 0; i < ctx->n_graphs; ++i)
    if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
  ctx->n_graphs = 0;
}

}  // namespace
}  // namespace tgnn

using namespace tgnn;

#define NEED(ctx, cond, code, ...)                       \
  do {                                                   \
    if (!(cond)) return set_error(ctx, code, __VA_ARGS__); \
  } while (0)

extern "C" {

int64_t tgnn_param_count(const tgnn_config* cfg) {
  if (check_config(cfg) != TGNN_OK) return -1;
  return make_layout(cfg->d, cfg->d_e, cfg->model).total;
}

int tgnn_param_layout(const tgnn_config* cfg, int64_t* out) {
  const int rc = check_config(cfg);
  if (rc != TGNN_OK) return rc;
  if (!out) return TGNN_EINVAL;
  const ParamLayout L = make_layout(cfg->d, cfg->d_e, cfg->model);
  const int64_t v[21] = {L.time_w, L.time_b, L.gru_wi, L.gru_wh, L.gru_bi, L.gru_bh, L.wq, L.bq, L.wk, L.wv, L.bk,
                         L.bv, L.wo, L.bo, L.w1, L.b1, L.w2, L.b2, L.proj_w, L.proj_b, L.total};
  for (int i = 0; i < 21; ++i) out[i] = v[i];
  return TGNN_OK;
}

int tgnn_create(const tgnn_config* cfg, tgnn_ctx** out) {
  if (!out) return TGNN_EINVAL;
  *out = nullptr;
  const int rc = check_config(cfg);
  if (rc != TGNN_OK) return rc;
  int dev = 0, cc_major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TGNN_ECUDA;
  if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TGNN_ECUDA;
  if (cc_major != 10) return TGNN_ECUDA;  // kernels are built for sm_100a only
  tgnn_ctx* ctx = new (std::nothrow) tgnn_ctx();
  if (!ctx) return TGNN_ECUDA;
  ctx->cfg = *cfg;
  ctx->L = make_layout(cfg->d, cfg->d_e, cfg->model);
  ctx->U_cap = 2 * cfg->max_events;
  ctx->R_cap = cfg->max_roots;
  ctx->NB_cap = cfg->max_roots * cfg->k;
  ctx->nq_cap = cfg->max_roots / 3;
  ctx->ld_msg = (int)((ctx->L.dmsg + 31) / 32 * 32);
  ctx->ld_kv = (int)((ctx->L.dkv + 31) / 32 * 32);
  ctx->ld_wkv = (int)((ctx->L.dkv + 1 + 3) / 4 * 4);
  ctx->arena_bytes = carve(ctx, nullptr);
  if (cudaMalloc(&ctx->arena, ctx->arena_bytes) != cudaSuccess) {
    cudaGetLastError();
    delete ctx;
    return TGNN_ECUDA;
  }
  carve(ctx, (char*)ctx->arena);
  bool ok = cudaMemset(ctx->arena, 0, ctx->arena_bytes) == cudaSuccess;
  ok = ok && cudaMemset(ctx->ws.node2slot, 0xff, sizeof(int32_t) * (size_t)cfg->num_nodes) == cudaSuccess;
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    cudaFree(ctx->arena);
    delete ctx;
    return TGNN_ECUDA;
  }
  {
    const size_t ne = (size_t)cfg->max_events, nq = (size_t)ctx->nq_cap;
    ctx->pack_bytes = (8 * ne + 8 * nq + 12 * ne + 12 * nq + ne + nq + 63) & ~(size_t)63;
    const size_t slot_bytes = (((12 + 8 + 2) * ne) + 255) & ~(size_t)255;
    unsigned char* base = nullptr;
    ctx->mixed_cur = -1;
    ctx->pack_dev = nullptr; ctx->pack_host[0] = ctx->pack_host[1] = nullptr; ctx->heavy_dev = nullptr;
    ok = ok && cudaMalloc((void**)&ctx->pack_dev, ctx->pack_bytes + 2 * slot_bytes + 256) == cudaSuccess;
    if (ok) {
      base = ctx->pack_dev + ctx->pack_bytes;
      for (int i = 0; i < 2; ++i) {
        unsigned char* p = base + i * slot_bytes;
        ctx->mixed[i].t = (double*)p; p += 8 * ne;
        ctx->mixed[i].src = (int32_t*)p; p += 4 * ne;
        ctx->mixed[i].dst = (int32_t*)p; p += 4 * ne;
        ctx->mixed[i].eid = (int32_t*)p; p += 4 * ne;
        ctx->mixed[i].aux = p; p += ne;
        ctx->mixed[i].keep = p;
        ctx->mixed[i].n = 0;
      }
      ctx->heavy_dev = (int32_t*)(base + 2 * slot_bytes);
    }
    for (int i = 0; ok && i < 2; ++i)
      ok = cudaHostAlloc((void**)&ctx->pack_host[i], ctx->pack_bytes, cudaHostAllocDefault) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->pack_done[i], cudaEventDisableTiming) == cudaSuccess;
  }
  ctx->images = nullptr; ctx->sites_dev = nullptr; ctx->images_fresh = false;
  if (ok && cfg->math_mode != TGNN_MATH_FP32) {
    ctx->images_bytes = plan_weight_sites(ctx);
    ok = cudaMalloc((void**)&ctx->images, ctx->images_bytes) == cudaSuccess &&
         cudaMemset(ctx->images, 0, ctx->images_bytes) == cudaSuccess &&
         cudaMalloc((void**)&ctx->sites_dev, sizeof(ctx->sites)) == cudaSuccess &&
         cudaMemcpy(ctx->sites_dev, ctx->sites, sizeof(ctx->sites), cudaMemcpyHostToDevice) == cudaSuccess;
  }
  ctx->split_buf = nullptr;
  if (ok && cfg->math_mode == TGNN_MATH_F16X3 && cfg->model == TGNN_MODEL_TGN) {
    const int64_t d = cfg->d, dkv = ctx->L.dkv, NB = ctx->NB_cap;
    // every operand as two fp16 numbers (22 mantissa bits); the gradient rows, whose entries are far below fp16's
    // normal range, multiplied by 2^12 first (the products divide it out again)
    const int planes = 2;   // hi and lo (a product that can do with one pass reads the hi planes alone)
    // Row pitches are multiples of 64 elements (128 bytes): a tile copy's 128-byte row pieces then never straddle two
    // cache lines (measured on the key/value projection's shape: 73 us with a 784-byte pitch, 66 us with 768).
    const auto up64 = [](int64_t x) { return (x + 63) / 64 * 64; };
    ctx->zs = SplitMat{nullptr, up64(dkv + 1), 0, NB, dkv + 1, 1, 1.f, planes};
    ctx->dkvs = SplitMat{nullptr, up64(2 * d), 0, NB, 2 * d, 1, 4096.f, planes};
    ctx->wkv_s = SplitMat{nullptr, up64(dkv), 0, 2 * d, dkv, 1, 1.f, planes};
    ctx->wz_s = SplitMat{nullptr, up64(2 * d), 0, 2 * d, 2 * d, 1, 1.f, planes};
    SplitMat* ms[4] = {&ctx->zs, &ctx->dkvs, &ctx->wkv_s, &ctx->wz_s};
    size_t off = 0;
    for (SplitMat* m : ms) {
      m->plane_stride = (m->rows * m->ld + 127) / 128 * 128;
      off += (size_t)(planes * m->plane_stride * 2);
    }
    off += 256;   // a chunked tile copy may read up to 126 bytes past the last plane (values that reach no stored output)
    ok = cudaMalloc(&ctx->split_buf, off) == cudaSuccess && cudaMemset(ctx->split_buf, 0, off) == cudaSuccess;
    off = 0;
    for (SplitMat* m : ms) {
      m->hi = (char*)ctx->split_buf + off;
      off += (size_t)(planes * m->plane_stride * 2);
    }
  }
  ctx->ev_next = 0;
  ctx->n_graphs = 0;
  ctx->graphs_enabled = 1;
  ctx->defer_adam = 0;
  ctx->grad_pending = false;
  {
    // the side streams carry work that is off the step's critical chain: lowest priority, so that a kernel of the
    // chain (the caller's stream) gets the next free SM slots when both have blocks waiting
    int least = 0, greatest = 0;
    ok = ok && cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess;
    for (int i = 0; ok && i < 4; ++i)
      ok = cudaStreamCreateWithPriority(&ctx->side[i], cudaStreamNonBlocking, least) == cudaSuccess;
  }
  for (int i = 0; ok && i < 32; ++i) ok = cudaEventCreateWithFlags(&ctx->ev[i], cudaEventDisableTiming) == cudaSuccess;
  ctx->side_pending = false;
  ok = ok && cudaEventCreateWithFlags(&ctx->ev_search, cudaEventDisableTiming) == cudaSuccess &&
       cudaEventCreateWithFlags(&ctx->ev_side_done, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    cudaFree(ctx->images);
    cudaFree(ctx->split_buf);
    cudaFree(ctx->sites_dev);
    cudaFree(ctx->pack_dev);
    for (int i = 0; i < 2; ++i) if (ctx->pack_host[i]) cudaFreeHost(ctx->pack_host[i]);
    cudaFree(ctx->arena);
    delete ctx;
    return TGNN_ECUDA;
  }
  snprintf(ctx->err, sizeof(ctx->err), "no error");
  *out = ctx;
  return TGNN_OK;
}

int tgnn_destroy(tgnn_ctx* ctx) {
  if (!ctx) return TGNN_OK;
  cudaDeviceSynchronize();
  for (ProfEntry& e : ctx->prof.entries) {
    cudaEventDestroy(e.a);
    cudaEventDestroy(e.b);
  }
  for (int i = 0; i < ctx->n_graphs; ++i)
    if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
  for (int i = 0; i < 4; ++i) cudaStreamDestroy(ctx->side[i]);
  for (int i = 0; i < 32; ++i) cudaEventDestroy(ctx->ev[i]);
  cudaEventDestroy(ctx->ev_search); cudaEventDestroy(ctx->ev_side_done);
  cudaFree(ctx->images);
  cudaFree(ctx->split_buf);
  cudaFree(ctx->sites_dev);
  cudaFree(ctx->pack_dev);
  for (int i = 0; i < 2; ++i) {
    if (ctx->pack_host[i]) cudaFreeHost(ctx->pack_host[i]);
    cudaEventDestroy(ctx->pack_done[i]);
  }
  cudaFree(ctx->arena);
  delete ctx;
  return TGNN_OK;
}

const char* tgnn_last_error(const tgnn_ctx* ctx) { return ctx ? ctx->err : "null context"; }

int64_t tgnn_kernel_launches(const tgnn_ctx* ctx) { return ctx ? ctx->launches : 0; }

int tgnn_set_graph(tgnn_ctx* ctx, const int64_t* indptr, const int32_t* nbr, const int32_t* eid, const double* ts,
                   int64_t n_entries) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, indptr && n_entries >= 0, TGNN_EINVAL, "set_graph: null indptr or negative size");
  NEED(ctx, n_entries == 0 || (nbr && eid && ts), TGNN_EINVAL, "set_graph: null adjacency arrays");
  if (ctx->indptr != indptr || ctx->g_nbr != nbr || ctx->g_eid != eid || ctx->g_ts != ts) drop_step_graphs(ctx);
  ctx->indptr = indptr; ctx->g_nbr = nbr; ctx->g_eid = eid; ctx->g_ts = ts; ctx->n_entries = n_entries;
  return TGNN_OK;
}

int tgnn_set_edge_features(tgnn_ctx* ctx, const void* efeat, int dtype, int64_t num_events, int d_e) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, d_e == ctx->cfg.d_e, TGNN_ESHAPE, "set_edge_features: d_e %d != configured %d", d_e, ctx->cfg.d_e);
  NEED(ctx, dtype == ctx->cfg.feat_dtype, TGNN_EINVAL, "set_edge_features: dtype differs from the configuration");
  NEED(ctx, d_e == 0 || efeat, TGNN_EINVAL, "set_edge_features: null table");
  NEED(ctx, num_events >= 0, TGNN_EINVAL, "set_edge_features: negative size");
  NEED(ctx, ((uintptr_t)efeat & 3) == 0, TGNN_EINVAL, "set_edge_features: table must be 4-byte aligned");
  if (ctx->efeat != efeat) drop_step_graphs(ctx);
  ctx->efeat = efeat; ctx->num_events = num_events;
  return TGNN_OK;
}

int tgnn_set_state(tgnn_ctx* ctx, float* memory, double* last_update, float* params, float* adam_m, float* adam_v,
                   int64_t* step) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, memory && last_update && params && adam_m && adam_v && step, TGNN_EINVAL, "set_state: null pointer");
  if (ctx->memory != memory || ctx->last_update != last_update || ctx->params != params || ctx->adam_m != adam_m ||
      ctx->adam_v != adam_v || ctx->step != step)
    drop_step_graphs(ctx);
  ctx->memory = memory; ctx->last_update = last_update; ctx->params = params;
  ctx->adam_m = adam_m; ctx->adam_v = adam_v; ctx->step = step;
  ctx->have_update = false; ctx->have_embed = false; ctx->grads_zeroed = false; ctx->images_fresh = false;
  ctx->grad_pending = false;
  ctx->mixed_cur = -1;
  return TGNN_OK;
}

int tgnn_prune_mask(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const int32_t* eid, const uint8_t* is_aux,
                    int n, int force_heavy, uint32_t drop_q32, uint64_t seed, int64_t batch_idx, uint8_t* keep_out,
                    int32_t* heavy_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, n >= 0, TGNN_EINVAL, "prune_mask: negative n");
  NEED(ctx, n <= ctx->cfg.max_events, TGNN_ECAPACITY, "prune_mask: n %d > max_events %d", n, ctx->cfg.max_events);
  NEED(ctx, heavy_out && (n == 0 || (src && dst && eid && is_aux && keep_out)), TGNN_EINVAL, "prune_mask: null pointer");
  NEED(ctx, force_heavy >= -1 && force_heavy <= 1, TGNN_EINVAL, "prune_mask: force_heavy must be -1, 0 or 1");
  return launch_prune_mask(ctx, src, dst, eid, is_aux, n, force_heavy, drop_q32, seed, batch_idx, keep_out, heavy_out,
                           S(stream));
}

int tgnn_sample_recent(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, int32_t* nbr_out,
                       int32_t* eid_out, double* ts_out, int32_t* cnt_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, ctx->indptr, TGNN_ESTATE, "sample_recent: tgnn_set_graph has not been called");
  NEED(ctx, n >= 0, TGNN_EINVAL, "sample_recent: negative n");
  NEED(ctx, n == 0 || (nodes && times && nbr_out && eid_out && ts_out && cnt_out), TGNN_EINVAL,
       "sample_recent: null pointer");
  return launch_sample_recent(ctx, nodes, times, n, nbr_out, eid_out, ts_out, cnt_out, S(stream));
}

int tgnn_build_messages(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const double* t, const int32_t* eid,
                        const uint8_t* keep, int n, float* msg_out, int32_t* msg_node_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, ctx->memory, TGNN_ESTATE, "build_messages: tgnn_set_state has not been called");
  NEED(ctx, ctx->cfg.d_e == 0 || ctx->efeat, TGNN_ESTATE, "build_messages: tgnn_set_edge_features has not been called");
  NEED(ctx, n >= 0, TGNN_EINVAL, "build_messages: negative n");
  NEED(ctx, n <= ctx->cfg.max_events, TGNN_ECAPACITY, "build_messages: n %d > max_events %d", n, ctx->cfg.max_events);
  NEED(ctx, n == 0 || (src && dst && t && eid && msg_node_out), TGNN_EINVAL, "build_messages: null pointer");
  ctx->m_src = src; ctx->m_dst = dst; ctx->m_t = t; ctx->m_eid = eid; ctx->m_keep = keep; ctx->m_n = n;
  return launch_build_messages(ctx, src, dst, t, eid, keep, n, msg_out, msg_node_out, S(stream));
}

int tgnn_reduce_latest(tgnn_ctx* ctx, const int32_t* msg_node, const double* t, const int32_t* eid, int n_msg,
                       int32_t* uniq_out, int32_t* winner_out, int32_t* n_uniq_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, n_msg >= 0 && n_msg % 2 == 0, TGNN_EINVAL, "reduce_latest: n_msg must be even and non-negative");
  NEED(ctx, n_msg <= ctx->U_cap, TGNN_ECAPACITY, "reduce_latest: n_msg %d > 2*max_events", n_msg);
  NEED(ctx, n_uniq_out && (n_msg == 0 || (msg_node && t && eid && uniq_out && winner_out)), TGNN_EINVAL,
       "reduce_latest: null pointer");
  return launch_reduce_latest(ctx, msg_node, t, eid, n_msg, uniq_out, winner_out, n_uniq_out, S(stream));
}

int tgnn_memory_update(tgnn_ctx* ctx, const float* msg, const int32_t* uniq, const int32_t* winner,
                       const int32_t* n_uniq, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, ctx->memory, TGNN_ESTATE, "memory_update: tgnn_set_state has not been called");
  NEED(ctx, ctx->m_src || ctx->m_n == 0, TGNN_ESTATE, "memory_update: tgnn_build_messages has not been called");
  NEED(ctx, n_uniq && (ctx->m_n == 0 || (uniq && winner)), TGNN_EINVAL, "memory_update: null pointer");
  ctx->upd_n_uniq = n_uniq;
  ctx->upd_cap = ctx->U_cap < 2 * ctx->m_n ? ctx->U_cap : 2 * ctx->m_n;
  ctx->have_update = ctx->upd_cap > 0;
  return launch_memory_update(ctx, msg, uniq, winner, n_uniq, S(stream));
}

int tgnn_embed(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, const int32_t* nbr, const int32_t* eid,
               const double* ts, const int32_t* cnt, float* h_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, ctx->memory, TGNN_ESTATE, "embed: tgnn_set_state has not been called");
  NEED(ctx, ctx->cfg.d_e == 0 || ctx->efeat, TGNN_ESTATE, "embed: tgnn_set_edge_features has not been called");
  NEED(ctx, n >= 0, TGNN_EINVAL, "embed: negative n");
  NEED(ctx, n <= ctx->R_cap, TGNN_ECAPACITY, "embed: n %d > max_roots %d", n, ctx->R_cap);
  const bool needs_nbrs = ctx->cfg.model == TGNN_MODEL_TGN;
  NEED(ctx, n == 0 || (nodes && times && h_out && (!needs_nbrs || (nbr && eid && ts && cnt))), TGNN_EINVAL,
       "embed: null pointer");
  ctx->e_nodes = nodes; ctx->e_times = times; ctx->e_nbr = nbr; ctx->e_eid = eid; ctx->e_ts = ts; ctx->e_cnt = cnt;
  ctx->e_n = n; ctx->e_h = h_out; ctx->have_embed = true;
  return launch_embed(ctx, nodes, times, n, nbr, eid, ts, cnt, h_out, S(stream));
}

int tgnn_backward_step(tgnn_ctx* ctx, int n_q, const uint8_t* loss_mask, float* loss_out, float* gradnorm_out,
                       void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, ctx->have_embed, TGNN_ESTATE, "backward_step: no tgnn_embed call to differentiate");
  NEED(ctx, n_q >= 0 && 3 * n_q == ctx->e_n, TGNN_ESHAPE, "backward_step: the last embed call had %d rows, expected 3*n_q = %d",
       ctx->e_n, 3 * n_q);
  NEED(ctx, !ctx->grad_pending, TGNN_ESTATE, "backward_step: the previous step's gradient has not been applied (tgnn_apply_gradient)");
  const int rc = launch_backward(ctx, n_q, loss_mask, loss_out, gradnorm_out, S(stream));
  ctx->grad_pending = ctx->defer_adam != 0 && rc == TGNN_OK;
  ctx->have_embed = false;
  ctx->have_update = false;
  ctx->grads_zeroed = false;
  ctx->images_fresh = false;  // Adam has changed the parameters
  return rc;
}

namespace {

// The launch sequence of one step on fixed (staging) input addresses.
int step_body(tgnn_ctx* ctx, int n_u, bool has_keep, int n_q, bool has_mask, float* loss_out, float* gradnorm_out,
              void* stream) {
  Workspace& w = ctx->ws;
  int rc;
  ctx->have_update = false;
  // While per-kernel timing is on, everything is issued on the caller's stream: the event pair around a
  // launch then times that kernel alone instead of the kernel plus whatever shares the machine with it.
  struct SideGuard {
    tgnn_ctx* c;
    cudaStream_t s0, s1, s2, s3;
    SideGuard(tgnn_ctx* c_, cudaStream_t main) : c(c_), s0(c_->side[0]), s1(c_->side[1]), s2(c_->side[2]), s3(c_->side[3]) {
      if (c->prof.on) c->side[0] = c->side[1] = c->side[2] = c->side[3] = main;
    }
    ~SideGuard() { c->side[0] = s0; c->side[1] = s1; c->side[2] = s2; c->side[3] = s3; }
  } side_guard(ctx, S(stream));
  // the weights' B-operand images for this step's projections: written beside the first kernels
  const bool prep = ctx->images != nullptr;
  ctx->z_split = ctx->split_buf != nullptr && prep;   // the weight planes will be fresh by the time the embedding runs
  if (prep) {
    rc = fork_to(ctx, S(stream), ctx->side[0]);
    if (rc) return rc;
    rc = launch_prep_weights(ctx, ctx->side[0]);
    if (rc) return rc;
  }
  // the neighbor search reads only the static graph: it runs beside the memory update
  cudaStream_t side = ctx->side[1];
  rc = fork_to(ctx, S(stream), side);
  if (rc) return rc;
  rc = launch_make_roots(ctx, w.st_q_src, w.st_q_dst, w.st_q_neg, w.st_q_t, n_q, side);
  if (rc) return rc;
  NEED(ctx, ctx->cfg.d_e == 0 || ctx->efeat, TGNN_ESTATE, "train_step: tgnn_set_edge_features has not been called");
  TGNN_CUDA_OK(ctx, cudaEventRecord(ctx->ev_search, side));
  if (ctx->cfg.model == TGNN_MODEL_TGN) {  // the time-projected embedding samples no neighbors
    rc = tgnn_sample_recent(ctx, w.r_node, w.r_time, 3 * n_q, w.nb_node, w.nb_eid, w.nb_ts, w.nb_cnt, side);
    if (rc) return rc;
    TGNN_CUDA_OK(ctx, cudaEventRecord(ctx->ev_search, side));
    // edge features and time encodings of the sampled neighbors do not depend on memory either
    rc = launch_embed_static(ctx, w.r_time, 3 * n_q, w.nb_node, w.nb_eid, w.nb_ts, side);
    if (rc) return rc;
    ctx->z_static_done = true;
  }
  {  // clear the gradient block off the critical chain (grads | dMemU | red | tg_acc | scalars, contiguous); the
     // backward pass is its first reader, so it goes behind the gathers, which the embedding waits for
    const size_t zero_bytes = (size_t)((char*)(w.st_scalars + 4) - (char*)w.grads);
    TGNN_CUDA_OK(ctx, cudaMemsetAsync(w.grads, 0, zero_bytes, side));
    ctx->grads_zeroed = true;
  }
  TGNN_CUDA_OK(ctx, cudaEventRecord(ctx->ev_side_done, side));
  ctx->side_pending = true;
  if (n_u > 0) {
    // messages stay virtual: the reduction reads the event arrays, the memory update gathers the winners
    ctx->m_src = w.st_u_src; ctx->m_dst = w.st_u_dst; ctx->m_t = w.st_u_t; ctx->m_eid = w.st_u_eid;
    ctx->m_keep = has_keep ? w.st_u_keep : nullptr; ctx->m_n = n_u;
    rc = launch_reduce_latest_events(ctx, nullptr, w.st_u_src, w.st_u_dst, ctx->m_keep, w.st_u_t, w.st_u_eid, 2 * n_u,
                                     w.uniq, w.winner, w.n_uniq, S(stream));
    if (rc) return rc;
    if (prep) {
      rc = fork_to(ctx, ctx->side[0], S(stream));
      if (rc) return rc;
      ctx->images_fresh = true;
    }
    rc = tgnn_memory_update(ctx, nullptr, w.uniq, w.winner, w.n_uniq, stream);
    if (rc) return rc;
  } else if (prep) {
    rc = fork_to(ctx, ctx->side[0], S(stream));
    if (rc) return rc;
    ctx->images_fresh = true;
  }
  // the embedding waits for the side stream's pieces where it first needs each: roots and neighbor lists here, the
  // static half of its inputs before the key/value projection
  TGNN_CUDA_OK(ctx, cudaStreamWaitEvent(S(stream), ctx->ev_search, 0));
  rc = tgnn_embed(ctx, w.r_node, w.r_time, 3 * n_q, w.nb_node, w.nb_eid, w.nb_ts, w.nb_cnt, w.h, stream);
  if (rc) return rc;
  return tgnn_backward_step(ctx, n_q, has_mask ? w.st_mask : nullptr, loss_out, gradnorm_out, stream);
}

// Host-side bookkeeping that step_body leaves behind, reproduced after a graph replay.
void after_replay(tgnn_ctx* ctx, int n_u, bool has_keep, int n_q) {
  Workspace& w = ctx->ws;
  ctx->m_src = w.st_u_src; ctx->m_dst = w.st_u_dst; ctx->m_t = w.st_u_t; ctx->m_eid = w.st_u_eid;
  ctx->m_keep = has_keep ? w.st_u_keep : nullptr; ctx->m_n = n_u;
  ctx->upd_n_uniq = w.n_uniq;
  ctx->upd_cap = ctx->U_cap < 2 * n_u ? ctx->U_cap : 2 * n_u;
  ctx->e_nodes = w.r_node; ctx->e_times = w.r_time; ctx->e_nbr = w.nb_node; ctx->e_eid = w.nb_eid;
  ctx->e_ts = w.nb_ts; ctx->e_cnt = w.nb_cnt; ctx->e_n = 3 * n_q; ctx->e_h = w.h;
  ctx->have_embed = false; ctx->have_update = false; ctx->grads_zeroed = false; ctx->images_fresh = false;
  ctx->grad_pending = ctx->defer_adam != 0;
}

}  // namespace

int tgnn_set_grad_sync(tgnn_ctx* ctx, int defer) {
  if (!ctx) return TGNN_EINVAL;
  if ((defer != 0) == (ctx->defer_adam != 0)) return TGNN_OK;
  // recorded steps end with the fused norm + Adam launch of the other mode: drop them
  drop_step_graphs(ctx);
  ctx->defer_adam = defer ? 1 : 0;
  ctx->grad_pending = false;
  return TGNN_OK;
}

int tgnn_grad_buffer(tgnn_ctx* ctx, float** grads_dev_out, int64_t* count_out) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, grads_dev_out && count_out, TGNN_EINVAL, "grad_buffer: null pointer");
  *grads_dev_out = ctx->ws.grads;
  *count_out = ctx->L.total;
  return TGNN_OK;
}

int tgnn_apply_gradient(tgnn_ctx* ctx, float scale, float* gradnorm_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, ctx->defer_adam, TGNN_ESTATE, "apply_gradient: the context applies Adam inside the step (tgnn_set_grad_sync(ctx, 1) first)");
  NEED(ctx, ctx->grad_pending, TGNN_ESTATE, "apply_gradient: no step has left a gradient to apply");
  NEED(ctx, scale == scale && scale != 0.f, TGNN_EINVAL, "apply_gradient: scale must be a non-zero number");
  const int rc = launch_apply_gradient(ctx, scale, gradnorm_out, S(stream));
  ctx->grad_pending = false;
  ctx->images_fresh = false;  // Adam has changed the parameters
  return rc;
}

int tgnn_set_graph_replay(tgnn_ctx* ctx, int enable) {
  if (!ctx) return TGNN_EINVAL;
  ctx->graphs_enabled = enable ? 1 : 0;
  return TGNN_OK;
}

int tgnn_train_step(tgnn_ctx* ctx, const int32_t* u_src, const int32_t* u_dst, const double* u_t, const int32_t* u_eid,
                    const uint8_t* u_keep, int n_u, const int32_t* q_src, const int32_t* q_dst, const int32_t* q_neg,
                    const double* q_t, int n_q, const uint8_t* loss_mask, float* loss_out, float* gradnorm_out,
                    void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, n_u >= 0 && n_q >= 0, TGNN_EINVAL, "train_step: negative size");
  NEED(ctx, n_u <= ctx->cfg.max_events, TGNN_ECAPACITY, "train_step: n_u %d > max_events %d", n_u, ctx->cfg.max_events);
  NEED(ctx, n_q <= ctx->nq_cap, TGNN_ECAPACITY, "train_step: n_q %d > max_roots/3 = %d", n_q, ctx->nq_cap);
  NEED(ctx, n_u == 0 || (u_src && u_dst && u_t && u_eid), TGNN_EINVAL, "train_step: null update arrays");
  NEED(ctx, n_q == 0 || (q_src && q_dst && q_neg && q_t), TGNN_EINVAL, "train_step: null target arrays");
  NEED(ctx, ctx->memory && ctx->indptr, TGNN_ESTATE, "train_step: tgnn_set_state / tgnn_set_graph have not been called");
  NEED(ctx, !ctx->grad_pending, TGNN_ESTATE, "train_step: the previous step's gradient has not been applied (tgnn_apply_gradient)");
  const bool has_keep = n_u > 0 && u_keep != nullptr, has_mask = n_q > 0 && loss_mask != nullptr;
  int rc = launch_stage_inputs(ctx, u_src, u_dst, u_t, u_eid, u_keep, n_u, q_src, q_dst, q_neg, q_t, n_q, loss_mask,
                               S(stream));
  if (rc) return rc;
  if (!ctx->graphs_enabled || ctx->prof.on)
    return step_body(ctx, n_u, has_keep, n_q, has_mask, loss_out, gradnorm_out, stream);

  tgnn_ctx::StepGraph* e = nullptr;
  for (int i = 0; i < ctx->n_graphs; ++i) {
    tgnn_ctx::StepGraph& c = ctx->graphs[i];
    if (c.n_u == n_u && c.n_q == n_q && c.has_keep == (int)has_keep && c.has_mask == (int)has_mask &&
        c.loss_out == loss_out && c.gradnorm_out == gradnorm_out) { e = &c; break; }
  }
  if (!e) {
    if (ctx->n_graphs == 8) return step_body(ctx, n_u, has_keep, n_q, has_mask, loss_out, gradnorm_out, stream);
    e = &ctx->graphs[ctx->n_graphs++];
    *e = tgnn_ctx::StepGraph{n_u, n_q, (int)has_keep, (int)has_mask, loss_out, gradnorm_out, 0, 0, nullptr};
  }
  if (e->exec) {
    TGNN_CUDA_OK(ctx, cudaGraphLaunch(e->exec, S(stream)));
    ctx->launches += e->kernels;
    after_replay(ctx, n_u, has_keep, n_q);
    return TGNN_OK;
  }
  if (e->seen++ == 0)  // first time: plain launches (also performs one-time kernel attribute set-up)
    return step_body(ctx, n_u, has_keep, n_q, has_mask, loss_out, gradnorm_out, stream);
  // second time: record the launches into a graph, then run it
  if (cudaStreamBeginCapture(S(stream), cudaStreamCaptureModeRelaxed) != cudaSuccess) {
    cudaGetLastError();  // e.g. the legacy default stream cannot capture: stay with plain launches
    ctx->graphs_enabled = 0;
    return step_body(ctx, n_u, has_keep, n_q, has_mask, loss_out, gradnorm_out, stream);
  }
  const int64_t l0 = ctx->launches;
  rc = step_body(ctx, n_u, has_keep, n_q, has_mask, loss_out, gradnorm_out, stream);
  cudaGraph_t graph = nullptr;
  const cudaError_t ce = cudaStreamEndCapture(S(stream), &graph);
  if (rc != TGNN_OK || ce != cudaSuccess || !graph) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    ctx->graphs_enabled = 0;
    if (rc != TGNN_OK) return rc;
    return set_error(ctx, TGNN_ECUDA, "train_step: stream capture failed: %s", cudaGetErrorString(ce));
  }
  e->kernels = ctx->launches - l0;
  cudaGraphExec_t exec = nullptr;
  // node priorities as captured (side-stream kernels low, the caller's stream as it is) instead of one priority for all
  // (the attention model only: in the short chain of the time-projection model the side streams' kernels are on the
  // critical path themselves, and ranking them below the chain cost 9 % there)
  const cudaError_t ie = cudaGraphInstantiate(&exec, graph, ctx->cfg.model == TGNN_MODEL_TGN ? cudaGraphInstantiateFlagUseNodePriority : 0);
  cudaGraphDestroy(graph);
  if (ie != cudaSuccess || !exec) {
    cudaGetLastError();
    ctx->graphs_enabled = 0;
    return set_error(ctx, TGNN_ECUDA, "train_step: graph instantiation failed: %s", cudaGetErrorString(ie));
  }
  e->exec = exec;
  TGNN_CUDA_OK(ctx, cudaGraphLaunch(e->exec, S(stream)));
  after_replay(ctx, n_u, has_keep, n_q);
  return TGNN_OK;
}

int tgnn_step_mixed_host(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const double* t, const int32_t* eid,
                         const uint8_t* is_aux, int n, const int32_t* neg, int force_heavy, uint32_t drop_q32,
                         uint64_t seed, int64_t batch_idx, float* loss_host, float* gradnorm_host, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, n >= 0, TGNN_EINVAL, "step_mixed_host: negative n");
  NEED(ctx, n <= ctx->cfg.max_events, TGNN_ECAPACITY, "step_mixed_host: n %d > max_events %d", n, ctx->cfg.max_events);
  NEED(ctx, n == 0 || (src && dst && t && eid && is_aux), TGNN_EINVAL, "step_mixed_host: null batch arrays");
  NEED(ctx, force_heavy >= -1 && force_heavy <= 1, TGNN_EINVAL, "step_mixed_host: force_heavy must be -1, 0 or 1");
  const bool all = ctx->cfg.embed_aux != 0;  // every event is a root; the loss mask is 1 - is_aux
  int n_q = 0;
  for (int i = 0; i < n; ++i) n_q += all || is_aux[i] == 0;
  NEED(ctx, n_q <= ctx->nq_cap, TGNN_ECAPACITY, "step_mixed_host: %d scored events > max_roots/3 = %d", n_q, ctx->nq_cap);
  NEED(ctx, n_q == 0 || neg, TGNN_EINVAL, "step_mixed_host: null negatives");
  cudaStream_t s = S(stream);
  const int slot = ctx->mixed_cur < 0 ? 0 : 1 - ctx->mixed_cur;
  // pack: one block, one copy
  unsigned char* pk = ctx->pack_host[slot];
  TGNN_CUDA_OK(ctx, cudaEventSynchronize(ctx->pack_done[slot]));  // the copy that last used this buffer has finished
  double* p_t = reinterpret_cast<double*>(pk);
  double* p_qt = p_t + n;
  int32_t* p_i = reinterpret_cast<int32_t*>(p_qt + n_q);
  int32_t* p_q = p_i + 3 * (size_t)n;
  uint8_t* p_aux = reinterpret_cast<uint8_t*>(p_q + 3 * (size_t)n_q);
  uint8_t* p_mask = p_aux + n;  // [n_q], present only when every event is scored
  memcpy(p_t, t, sizeof(double) * n);
  memcpy(p_i, src, sizeof(int32_t) * n);
  memcpy(p_i + n, dst, sizeof(int32_t) * n);
  memcpy(p_i + 2 * (size_t)n, eid, sizeof(int32_t) * n);
  memcpy(p_aux, is_aux, n);
  for (int i = 0, j = 0; i < n; ++i)
    if (all || !is_aux[i]) {
      p_qt[j] = t[i]; p_q[j] = src[i]; p_q[n_q + j] = dst[i]; p_q[2 * (size_t)n_q + j] = neg[j];
      if (all) p_mask[j] = is_aux[i] ? 0 : 1;
      ++j;
    }
  const size_t bytes = (size_t)(p_aux + n + (all ? n_q : 0) - pk);
  if (bytes > 0) TGNN_CUDA_OK(ctx, cudaMemcpyAsync(ctx->pack_dev, pk, bytes, cudaMemcpyHostToDevice, s));
  TGNN_CUDA_OK(ctx, cudaEventRecord(ctx->pack_done[slot], s));
  // the previous call's prune ran on a side stream: its keep mask is needed from here on
  int rc = fork_to(ctx, ctx->side[1], s);
  if (rc) return rc;
  rc = launch_unpack_mixed(ctx, ctx->pack_dev, n, n_q, all, slot, s);
  if (rc) return rc;
  ctx->mixed[slot].n = n;
  if (n > 0) {  // step (0) for this batch, beside the step: its result is first read by the next call
    rc = fork_to(ctx, s, ctx->side[1]);
    if (rc) return rc;
    const tgnn_ctx::MixedSlot& m = ctx->mixed[slot];
    rc = launch_prune_mask(ctx, m.src, m.dst, m.eid, m.aux, n, force_heavy, drop_q32, seed, batch_idx, m.keep,
                           ctx->heavy_dev, ctx->side[1]);
    if (rc) return rc;
  }
  const tgnn_ctx::MixedSlot* u = ctx->mixed_cur >= 0 ? &ctx->mixed[ctx->mixed_cur] : nullptr;
  Workspace& w = ctx->ws;
  rc = tgnn_train_step(ctx, u ? u->src : nullptr, u ? u->dst : nullptr, u ? u->t : nullptr, u ? u->eid : nullptr,
                       u ? u->keep : nullptr, u ? u->n : 0, w.st_q_src, w.st_q_dst, w.st_q_neg, w.st_q_t, n_q,
                       all ? w.st_mask : nullptr, nullptr, nullptr, stream);
  if (rc) return rc;
  ctx->mixed_cur = slot;
  if (loss_host) TGNN_CUDA_OK(ctx, cudaMemcpyAsync(loss_host, w.st_scalars + 2, sizeof(float), cudaMemcpyDeviceToHost, s));
  if (gradnorm_host)
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(gradnorm_host, w.st_scalars + 3, sizeof(float), cudaMemcpyDeviceToHost, s));
  return TGNN_OK;
}

int tgnn_train_step_host(tgnn_ctx* ctx, const int32_t* u_src, const int32_t* u_dst, const double* u_t,
                         const int32_t* u_eid, const uint8_t* u_keep, int n_u, const int32_t* q_src,
                         const int32_t* q_dst, const int32_t* q_neg, const double* q_t, int n_q,
                         const uint8_t* loss_mask, float* loss_host, float* gradnorm_host, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, n_u >= 0 && n_q >= 0, TGNN_EINVAL, "train_step_host: negative size");
  NEED(ctx, n_u <= ctx->cfg.max_events, TGNN_ECAPACITY, "train_step_host: n_u %d > max_events", n_u);
  NEED(ctx, n_q <= ctx->nq_cap, TGNN_ECAPACITY, "train_step_host: n_q %d > max_roots/3", n_q);
  NEED(ctx, n_u == 0 || (u_src && u_dst && u_t && u_eid), TGNN_EINVAL, "train_step_host: null update arrays");
  NEED(ctx, n_q == 0 || (q_src && q_dst && q_neg && q_t), TGNN_EINVAL, "train_step_host: null target arrays");
  Workspace& w = ctx->ws;
  cudaStream_t s = S(stream);
  const cudaMemcpyKind H2D = cudaMemcpyHostToDevice;
  if (n_u > 0) {
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_u_src, u_src, sizeof(int32_t) * n_u, H2D, s));
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_u_dst, u_dst, sizeof(int32_t) * n_u, H2D, s));
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_u_t, u_t, sizeof(double) * n_u, H2D, s));
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_u_eid, u_eid, sizeof(int32_t) * n_u, H2D, s));
    if (u_keep) TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_u_keep, u_keep, n_u, H2D, s));
  }
  if (n_q > 0) {
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_q_src, q_src, sizeof(int32_t) * n_q, H2D, s));
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_q_dst, q_dst, sizeof(int32_t) * n_q, H2D, s));
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_q_neg, q_neg, sizeof(int32_t) * n_q, H2D, s));
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_q_t, q_t, sizeof(double) * n_q, H2D, s));
    if (loss_mask) TGNN_CUDA_OK(ctx, cudaMemcpyAsync(w.st_mask, loss_mask, n_q, H2D, s));
  }
  const int rc = tgnn_train_step(ctx, w.st_u_src, w.st_u_dst, w.st_u_t, w.st_u_eid, u_keep ? w.st_u_keep : nullptr, n_u,
                                 w.st_q_src, w.st_q_dst, w.st_q_neg, w.st_q_t, n_q, loss_mask ? w.st_mask : nullptr,
                                 nullptr, nullptr, stream);
  if (rc) return rc;
  if (loss_host) TGNN_CUDA_OK(ctx, cudaMemcpyAsync(loss_host, w.st_scalars + 2, sizeof(float), cudaMemcpyDeviceToHost, s));
  if (gradnorm_host)
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(gradnorm_host, w.st_scalars + 3, sizeof(float), cudaMemcpyDeviceToHost, s));
  return TGNN_OK;
}

int tgnn_debug_get_grads(tgnn_ctx* ctx, float* grads_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, grads_out, TGNN_EINVAL, "debug_get_grads: null pointer");
  TGNN_CUDA_OK(ctx, cudaMemcpyAsync(grads_out, ctx->ws.grads, sizeof(float) * (size_t)ctx->L.total,
                                    cudaMemcpyDeviceToDevice, S(stream)));
  return TGNN_OK;
}

int tgnn_debug_get_embeddings(tgnn_ctx* ctx, float* h_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, h_out, TGNN_EINVAL, "debug_get_embeddings: null pointer");
  NEED(ctx, ctx->e_h, TGNN_ESTATE, "debug_get_embeddings: no embedding recorded");
  if (ctx->e_n > 0)
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(h_out, ctx->e_h, sizeof(float) * (size_t)ctx->e_n * ctx->cfg.d,
                                      cudaMemcpyDeviceToDevice, S(stream)));
  return TGNN_OK;
}

int tgnn_debug_get_gates(tgnn_ctx* ctx, uint8_t* h_gate_out, uint8_t* hid_gate_out, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, h_gate_out && hid_gate_out, TGNN_EINVAL, "debug_get_gates: null pointer");
  NEED(ctx, ctx->e_h && ctx->e_n % 3 == 0, TGNN_ESTATE, "debug_get_gates: no embedding / backward pass recorded");
  return launch_get_gates(ctx, h_gate_out, hid_gate_out, S(stream));
}

int tgnn_debug_gemm(tgnn_ctx* ctx, const float* A, int64_t a_rs, int64_t a_cs, const float* B, int64_t b_rs, int64_t b_cs,
                    float* C, int64_t ldc, int M, int N, int K, const int32_t* dev_M, const int32_t* dev_K,
                    const float* bias, float* rowsum_out, int relu, int accumulate, int split_k, int precise,
                    void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, A && B && C && M >= 0 && N >= 0 && K >= 0, TGNN_EINVAL, "debug_gemm: null pointer or negative size");
  GemmArgs g = {};
  g.A = A; g.a_rs = a_rs; g.a_cs = a_cs; g.B = B; g.b_rs = b_rs; g.b_cs = b_cs; g.C = C; g.ldc = ldc;
  g.M = M; g.N = N; g.K = K; g.dev_M = dev_M; g.dev_K = dev_K; g.bias = bias; g.rowsum_out = rowsum_out;
  g.relu = relu; g.accumulate = accumulate; g.split_k = split_k < 1 ? 1 : split_k; g.precise = precise;
  return launch_gemm(ctx, g, "debug_gemm", S(stream));
}

int tgnn_debug_gemm_split(tgnn_ctx* ctx, const float* A, int64_t a_rs, int64_t a_cs, const float* B, int64_t b_rs,
                          int64_t b_cs, float* C, int64_t ldc, int M, int N, int K, const float* bias, int relu,
                          int accumulate, int split_k, void* scratch, int64_t scratch_bytes, int debug_withhold,
                          uint32_t spin_limit, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, A && B && C && scratch && M > 0 && N > 0 && K > 0, TGNN_EINVAL, "debug_gemm_split: null pointer or empty product");
  int mn;
  int64_t lda, ldb, a_rows, a_cols, b_rows, b_cols;
  if (a_cs == 1 && b_rs == 1) { mn = 0; lda = a_rs; ldb = b_cs; a_rows = M; a_cols = K; b_rows = N; b_cols = K; }
  else if (a_rs == 1 && b_cs == 1) { mn = 1; lda = a_cs; ldb = b_rs; a_rows = K; a_cols = M; b_rows = K; b_cols = N; }
  else return set_error(ctx, TGNN_ESHAPE, "debug_gemm_split: operands must both have the contraction index contiguous, or both the other one");
  const auto up8 = [](int64_t x) { return (x + 7) / 8 * 8; };
  // TGNN_GEMM_BF16=1 (debugging aid): bf16 planes instead of fp16 planes; TGNN_GEMM_SCALE=s: A is scaled by 2^s
  const int f16 = getenv("TGNN_GEMM_BF16") && atoi(getenv("TGNN_GEMM_BF16")) ? 0 : 1;
  const float sc = getenv("TGNN_GEMM_SCALE") ? ldexpf(1.f, atoi(getenv("TGNN_GEMM_SCALE"))) : 1.f;
  // TGNN_GEMM_PASSES=1 (debugging aid): hi planes only, one pass
  const int planes = getenv("TGNN_GEMM_PASSES") && atoi(getenv("TGNN_GEMM_PASSES")) == 1 ? 1 : 2;
  SplitMat a{nullptr, up8(a_cols), 0, a_rows, a_cols, f16, sc, planes}, b{nullptr, up8(b_cols), 0, b_rows, b_cols, f16, 1.f, planes};
  a.plane_stride = a.rows * a.ld;
  b.plane_stride = b.rows * b.ld;
  const int64_t a_bytes = (2 * a.plane_stride * 2 + 255) / 256 * 256, b_bytes = 2 * b.plane_stride * 2;
  NEED(ctx, scratch_bytes >= a_bytes + b_bytes + 256, TGNN_ECAPACITY, "debug_gemm_split: scratch of %lld bytes, %lld needed",
       (long long)scratch_bytes, (long long)(a_bytes + b_bytes));
  NEED(ctx, ((uintptr_t)scratch & 255) == 0, TGNN_EINVAL, "debug_gemm_split: scratch must be 256-byte aligned");
  a.hi = scratch;
  b.hi = (char*)scratch + a_bytes;
  int rc = launch_split_rows(ctx, A, lda, a.rows, (int)a.cols, nullptr, a, -1, "split_a", S(stream));
  if (rc) return rc;
  rc = launch_split_rows(ctx, B, ldb, b.rows, (int)b.cols, nullptr, b, -1, "split_b", S(stream));
  if (rc) return rc;
  // TGNN_GEMM_TRACE=1 (debugging aid): the first 4 KB of scratch receive clock stamps of CTA 0 instead of nothing
  static const bool trace_on = getenv("TGNN_GEMM_TRACE") != nullptr;
  long long* trace = nullptr;
  if (trace_on && scratch_bytes >= a_bytes + b_bytes + 256 + 4096 + 256)
    trace = reinterpret_cast<long long*>((char*)scratch + ((a_bytes + b_bytes + 256 + 255) / 256 * 256));
  return launch_gemm_split(ctx, a, b, mn, C, ldc, M, N, K, bias, relu, accumulate, split_k < 1 ? 1 : split_k, "debug_gemm_split",
                           S(stream), debug_withhold, spin_limit, -1, nullptr, trace,
                           getenv("TGNN_GEMM_SINGLE") ? atoi(getenv("TGNN_GEMM_SINGLE")) : -1, 1,
                           getenv("TGNN_GEMM_PAIR") ? atoi(getenv("TGNN_GEMM_PAIR")) : -1);
}

int tgnn_status(tgnn_ctx* ctx, int32_t* status_host, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, status_host, TGNN_EINVAL, "status: null pointer");
  TGNN_CUDA_OK(ctx, cudaMemcpyAsync(status_host, ctx->ws.status, sizeof(int32_t), cudaMemcpyDeviceToHost, S(stream)));
  TGNN_CUDA_OK(ctx, cudaStreamSynchronize(S(stream)));
  return TGNN_OK;
}

int tgnn_clear_status(tgnn_ctx* ctx, void* stream) {
  if (!ctx) return TGNN_EINVAL;
  TGNN_CUDA_OK(ctx, cudaMemsetAsync(ctx->ws.status, 0, sizeof(int32_t), S(stream)));
  return TGNN_OK;
}

int tgnn_profile_begin(tgnn_ctx* ctx) {
  if (!ctx) return TGNN_EINVAL;
  ctx->prof.used = 0;
  ctx->prof.on = true;
  return TGNN_OK;
}

int tgnn_profile_timeline(tgnn_ctx* ctx, char* buf, int64_t size) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, buf && size > 0, TGNN_EINVAL, "profile_timeline: null buffer");
  ctx->prof.on = false;
  TGNN_CUDA_OK(ctx, cudaDeviceSynchronize());
  std::string out;
  char line[160];
  for (size_t i = 0; i < ctx->prof.used; ++i) {
    const ProfEntry& e = ctx->prof.entries[i];
    float t0 = 0.f, dt = 0.f;
    if (cudaEventElapsedTime(&t0, ctx->prof.entries[0].a, e.a) != cudaSuccess ||
        cudaEventElapsedTime(&dt, e.a, e.b) != cudaSuccess) { cudaGetLastError(); continue; }
    snprintf(line, sizeof(line), "%s %.3f %.3f\n", e.name, t0 * 1e3, dt * 1e3);
    out += line;
  }
  snprintf(buf, (size_t)size, "%s", out.c_str());
  ctx->prof.used = 0;
  return TGNN_OK;
}

int tgnn_profile_report(tgnn_ctx* ctx, char* buf, int64_t size) {
  if (!ctx) return TGNN_EINVAL;
  NEED(ctx, buf && size > 0, TGNN_EINVAL, "profile_report: null buffer");
  ctx->prof.on = false;
  TGNN_CUDA_OK(ctx, cudaDeviceSynchronize());
  std::map<std::string, std::pair<long, double>> agg;
  std::vector<std::string> order;
  for (size_t i = 0; i < ctx->prof.used; ++i) {
    const ProfEntry& e = ctx->prof.entries[i];
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e.a, e.b) != cudaSuccess) { cudaGetLastError(); continue; }
    auto it = agg.find(e.name);
    if (it == agg.end()) { order.push_back(e.name); it = agg.emplace(e.name, std::make_pair(0L, 0.0)).first; }
    it->second.first += 1;
    it->second.second += ms;
  }
  std::string out;
  char line[160];
  for (const std::string& n : order) {
    snprintf(line, sizeof(line), "%s %ld %.6f\n", n.c_str(), agg[n].first, agg[n].second);
    out += line;
  }
  snprintf(buf, (size_t)size, "%s", out.c_str());
  ctx->prof.used = 0;
  return TGNN_OK;
}

}  // extern "C"
