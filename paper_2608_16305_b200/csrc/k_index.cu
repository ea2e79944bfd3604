// Integer kernels: pruning mask (step 0), most-recent-k neighbor search
// (step 1), per-node latest-event reduction (step 3).  All results are unique,
// so they are bit-exact whatever the thread interleaving.
#include "tgnn_internal.cuh"
#include "tgnn_device.cuh"

namespace tgnn {
namespace {

constexpr unsigned FULL = 0xffffffffu;

// ---------------------------------------------------------------- step (0) --
__device__ __forceinline__ uint64_t mix64(uint64_t z) {  // SplitMix64 finaliser
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
__device__ __forceinline__ uint32_t hash32(uint64_t seed, int64_t batch_idx, int32_t eid) {
  const uint64_t x =
      seed ^ ((uint64_t)batch_idx * 0x9E3779B97F4A7C15ULL) ^ ((uint64_t)(uint32_t)eid * 0xC2B2AE3D27D4EB4FULL);
  return (uint32_t)(mix64(x) >> 32);
}

// One occurrence count per endpoint, warp-aggregated so a hub costs one atomic per warp.
__device__ __forceinline__ void hist_add(int32_t* hist, int node, bool valid) {
  const unsigned act = __ballot_sync(FULL, valid);
  if (!valid) return;
  const unsigned peers = __match_any_sync(act, node);
  if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[node], __popc(peers));
}

constexpr int FIRST_VISIT = 0x40000000;

// Single CTA: the batch has a few thousand events and the histogram lives in L2.
__global__ void __launch_bounds__(1024) prune_mask_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                                                          const int32_t* __restrict__ eid,
                                                          const uint8_t* __restrict__ is_aux, int n, int N,
                                                          int32_t* status, int32_t* hist, int force_heavy, uint32_t drop_q32, uint64_t seed,
                                                          int64_t batch_idx, uint8_t* __restrict__ keep_out,
                                                          int32_t* __restrict__ heavy_out) {
  __shared__ int s_max, s_touched, s_heavy;
  if (threadIdx.x == 0) { s_max = 0; s_touched = 0; }
  const int n_round = (n + 31) / 32 * 32;
  for (int i = threadIdx.x; i < n_round; i += blockDim.x) {
    // an endpoint outside [0, N) is reported and left out of the counts
    const int a = i < n ? src[i] : 0, b = i < n ? dst[i] : 0;
    hist_add(hist, a, i < n && index_ok(a, N, status));
    hist_add(hist, b, i < n && index_ok(b, N, status));
  }
  __syncthreads();
  // max count and number of touched nodes: the first visitor of a node counts it
  int lmax = 0, ltouched = 0;
  for (int i = threadIdx.x; i < 2 * n; i += blockDim.x) {
    const int node = (i & 1) ? dst[i >> 1] : src[i >> 1];
    if (node < 0 || node >= N) continue;
    const int old = atomicOr(&hist[node], FIRST_VISIT);
    lmax = max(lmax, old & (FIRST_VISIT - 1));
    ltouched += (old & FIRST_VISIT) ? 0 : 1;
  }
  for (int o = 16; o > 0; o >>= 1) {
    lmax = max(lmax, __shfl_xor_sync(FULL, lmax, o));
    ltouched += __shfl_xor_sync(FULL, ltouched, o);
  }
  if ((threadIdx.x & 31) == 0) { atomicMax(&s_max, lmax); atomicAdd(&s_touched, ltouched); }
  __syncthreads();
  if (threadIdx.x == 0) {
    int heavy = ((int64_t)s_max * (int64_t)s_touched > 8ll * n) ? 1 : 0;
    if (force_heavy == 0 || force_heavy == 1) heavy = force_heavy;
    s_heavy = heavy;
    *heavy_out = heavy;
  }
  __syncthreads();
  const int heavy = s_heavy;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    bool keep = true;
    if (is_aux[i] && heavy) keep = !(drop_q32 == 0xFFFFFFFFu || hash32(seed, batch_idx, eid[i]) < drop_q32);
    keep_out[i] = keep ? 1 : 0;
    if (src[i] >= 0 && src[i] < N) hist[src[i]] = 0;  // leave the histogram clean for the next call
    if (dst[i] >= 0 && dst[i] < N) hist[dst[i]] = 0;
  }
}

// ---------------------------------------------------------------- step (1) --
// One warp per root.  The lower bound is found by a 32-way search: each round
// the lanes probe 32 spread positions of the remaining range with independent
// loads and a ballot picks the sub-range, so a hub slice of 2*10^7 entries
// needs 5 dependent memory round trips instead of 25.
__global__ void __launch_bounds__(256) sample_recent_kernel(const int64_t* __restrict__ indptr,
                                                            const int32_t* __restrict__ g_nbr,
                                                            const int32_t* __restrict__ g_eid,
                                                            const double* __restrict__ g_ts,
                                                            const int32_t* __restrict__ nodes,
                                                            const double* __restrict__ times, int n, int k, int N,
                                                            int32_t* status, int32_t* __restrict__ nbr_out,
                                                            int32_t* __restrict__ eid_out, double* __restrict__ ts_out,
                                                            int32_t* __restrict__ cnt_out) {
  const int lane = threadIdx.x & 31;
  const int root = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (root >= n) return;
  const int node = nodes[root];
  if (!index_ok(node, N, lane == 0 ? status : nullptr)) {   // a root outside the graph: reported, no neighbors
    if (lane == 0) cnt_out[root] = 0;
    if (lane < k) {
      const int64_t o = (int64_t)root * k + lane;
      nbr_out[o] = -1; eid_out[o] = -1; ts_out[o] = 0.0;
    }
    return;
  }
  const double t = times[root];
  const int64_t base = indptr[node];
  int64_t lo = base, hi = indptr[node + 1];  // the answer p lies in [lo, hi]
  while (hi - lo > 32) {
    const int64_t len = hi - lo;
    const int64_t idx = lo + ((int64_t)(lane + 1) * len) / 33;  // in [lo, hi), non-decreasing in lane
    const bool below = g_ts[idx] < t;                           // p > idx
    const int c = __popc(__ballot_sync(FULL, below));
    const int64_t idx_hi = __shfl_sync(FULL, idx, c < 32 ? c : 31);       // first probe with ts >= t
    const int64_t idx_lo = __shfl_sync(FULL, idx, c > 0 ? c - 1 : 0);     // last probe with ts < t
    if (c < 32) hi = idx_hi;
    if (c > 0) lo = idx_lo + 1;
  }
  {
    const int len = (int)(hi - lo);
    const bool below = lane < len && g_ts[lo + lane] < t;
    lo += __popc(__ballot_sync(FULL, below));
  }
  const int64_t p = lo;
  const int cnt = (int)min((int64_t)k, p - base);
  if (lane == 0) cnt_out[root] = cnt;
  if (lane < k) {
    const int64_t o = (int64_t)root * k + lane;
    if (lane < cnt) {
      const int64_t e = p - 1 - lane;
      nbr_out[o] = g_nbr[e];
      eid_out[o] = g_eid[e];
      ts_out[o] = g_ts[e];
    } else {
      nbr_out[o] = -1;
      eid_out[o] = -1;
      ts_out[o] = 0.0;
    }
  }
}

__global__ void make_roots_kernel(const int32_t* __restrict__ q_src, const int32_t* __restrict__ q_dst,
                                  const int32_t* __restrict__ q_neg, const double* __restrict__ q_t, int n_q,
                                  int32_t* __restrict__ r_node, double* __restrict__ r_time) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= 3 * n_q) return;
  const int j = i % n_q, blk = i / n_q;
  r_node[i] = blk == 0 ? q_src[j] : (blk == 1 ? q_dst[j] : q_neg[j]);
  r_time[i] = q_t[j];
}

// Copies one step's event arrays into the context's fixed staging buffers (so that the rest of the
// step always sees the same addresses).  Sources equal to their destination are skipped.
struct StageArgs {
  const int32_t *u_src, *u_dst, *u_eid, *q_src, *q_dst, *q_neg;
  const double *u_t, *q_t;
  const uint8_t *u_keep, *mask;
  int32_t *d_u_src, *d_u_dst, *d_u_eid, *d_q_src, *d_q_dst, *d_q_neg;
  double *d_u_t, *d_q_t;
  uint8_t *d_u_keep, *d_mask;
  int n_u, n_q;
};
// All loads are issued before the first store (the pointers may alias as far as the compiler knows, so
// written one array after the other every load would wait for the store before it).
__global__ void __launch_bounds__(256) stage_inputs_kernel(StageArgs a) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const bool u = i < a.n_u, q = i < a.n_q;
  // an array that is already in place is not copied
  const bool c0 = u && a.u_src != a.d_u_src, c1 = u && a.u_dst != a.d_u_dst, c2 = u && a.u_eid != a.d_u_eid;
  const bool c3 = u && a.u_t != a.d_u_t, c4 = u && a.u_keep && a.u_keep != a.d_u_keep;
  const bool e0 = q && a.q_src != a.d_q_src, e1 = q && a.q_dst != a.d_q_dst, e2 = q && a.q_neg != a.d_q_neg;
  const bool e3 = q && a.q_t != a.d_q_t, e4 = q && a.mask && a.mask != a.d_mask;
  const int32_t s0 = c0 ? a.u_src[i] : 0, s1 = c1 ? a.u_dst[i] : 0, s2 = c2 ? a.u_eid[i] : 0;
  const double s3 = c3 ? a.u_t[i] : 0.0;
  const uint8_t s4 = c4 ? a.u_keep[i] : 0;
  const int32_t t0 = e0 ? a.q_src[i] : 0, t1 = e1 ? a.q_dst[i] : 0, t2 = e2 ? a.q_neg[i] : 0;
  const double t3 = e3 ? a.q_t[i] : 0.0;
  const uint8_t t4 = e4 ? a.mask[i] : 0;
  if (c0) a.d_u_src[i] = s0;
  if (c1) a.d_u_dst[i] = s1;
  if (c2) a.d_u_eid[i] = s2;
  if (c3) a.d_u_t[i] = s3;
  if (c4) a.d_u_keep[i] = s4;
  if (e0) a.d_q_src[i] = t0;
  if (e1) a.d_q_dst[i] = t1;
  if (e2) a.d_q_neg[i] = t2;
  if (e3) a.d_q_t[i] = t3;
  if (e4) a.d_mask[i] = t4;
}

// Packed host block of tgnn_step_mixed_host: [t f64 n][q_t f64 nq][src,dst,eid i32 n each]
// [q_src,q_dst,q_neg i32 nq each][is_aux u8 n][loss mask u8 nq, only if q_mask != nullptr].  Scattered into
// the mixed-batch slot and the target staging.
__global__ void __launch_bounds__(256) unpack_mixed_kernel(const unsigned char* __restrict__ pk, int n, int nq,
                                                           int32_t* src, int32_t* dst, int32_t* eid, double* t,
                                                           uint8_t* aux, uint8_t* keep, int32_t* q_src, int32_t* q_dst,
                                                           int32_t* q_neg, double* q_t, uint8_t* q_mask) {
  const double* p_t = reinterpret_cast<const double*>(pk);
  const double* p_qt = p_t + n;
  const int32_t* p_i = reinterpret_cast<const int32_t*>(p_qt + nq);
  const int32_t* p_q = p_i + 3 * (size_t)n;
  const uint8_t* p_aux = reinterpret_cast<const uint8_t*>(p_q + 3 * (size_t)nq);
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    t[i] = p_t[i]; src[i] = p_i[i]; dst[i] = p_i[n + i]; eid[i] = p_i[2 * n + i];
    aux[i] = p_aux[i]; keep[i] = 1;
  }
  if (i < nq) {
    q_t[i] = p_qt[i]; q_src[i] = p_q[i]; q_dst[i] = p_q[nq + i]; q_neg[i] = p_q[2 * nq + i];
    if (q_mask) q_mask[i] = p_aux[n + i];
  }
}

// ---------------------------------------------------------------- step (3) --
// fp64 -> uint64 preserving order (0 is left free as "empty" for every finite value)
__device__ __forceinline__ unsigned long long orderable(double x) {
  unsigned long long u = (unsigned long long)__double_as_longlong(x);
  return (u >> 63) ? ~u : (u | 0x8000000000000000ULL);
}

// max over the lanes of `peers` (a __match_any_sync mask all of whose lanes call this)
__device__ __forceinline__ unsigned long long peer_max(unsigned peers, unsigned long long v) {
  unsigned long long m = v;
  unsigned rest = peers;
  while (rest) {
    const int l = __ffs(rest) - 1;
    rest &= rest - 1;
    const unsigned long long o = __shfl_sync(peers, v, l);
    m = o > m ? o : m;
  }
  return m;
}

// Single CTA.  Key order (t, eid, role) is resolved in two atomicMax passes over
// per-node tables (time first, then eid/role among the messages that tie on
// time); a hub's thousands of messages are pre-reduced inside each warp.
// Then the touched nodes are compacted in ascending id order by a block scan.
// msg_node may be null: the node of message j is then read from the event arrays (src for role 0,
// dst for role 1, none if keep[j>>1] == 0), which saves materialising it.
// An event that names a node outside [0, N) (or, when E > 0, a feature row outside [0, E)) is reported and sends
// no message at all, exactly as if its keep flag were 0.
__device__ __forceinline__ int message_node(const int32_t* __restrict__ msg_node, const int32_t* __restrict__ src,
                                            const int32_t* __restrict__ dst, const uint8_t* __restrict__ keep,
                                            const int32_t* __restrict__ eid, int j, int N, int64_t E, int32_t* status) {
  if (msg_node) {
    const int node = msg_node[j];
    if (node < 0) return -1;
    return index_ok(node, N, status) ? node : -1;
  }
  const int i = j >> 1;
  if (keep && !keep[i]) return -1;
  const int a = src[i], b = dst[i];
  if (!(index_ok(a, N, status) & index_ok(b, N, status) & (E <= 0 || index_ok(eid[i], E, status)))) return -1;
  return (j & 1) ? b : a;
}

__global__ void __launch_bounds__(1024) reduce_latest_kernel(const int32_t* __restrict__ msg_node,
                                                             const int32_t* __restrict__ ev_src,
                                                             const int32_t* __restrict__ ev_dst,
                                                             const uint8_t* __restrict__ ev_keep,
                                                             const double* __restrict__ t,
                                                             const int32_t* __restrict__ eid, int n_msg, int N,
                                                             unsigned long long* best_t, unsigned long long* best_id,
                                                             int32_t* win_msg, int32_t* node2slot, int32_t* prev_uniq,
                                                             int32_t* prev_n_uniq, int32_t* __restrict__ uniq_out,
                                                             int32_t* __restrict__ winner_out,
                                                             int32_t* __restrict__ n_uniq_out, int smem_nodes,
                                                             int32_t* status, int64_t E) {
  extern __shared__ int s_last[];  // [smem_nodes]: last message index per node (fast path)
  __shared__ int s_warp[32];
  __shared__ int s_total;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  // forget the previous step's node -> slot map
  const int pn = *prev_n_uniq;
  for (int i = tid; i < pn; i += blockDim.x) node2slot[prev_uniq[i]] = -1;
  // Fast path.  A mixed batch arrives sorted by (t, eid) (Eq. 5), and then the key order of the
  // messages is their index order: the winner of a node is simply its last message.  One shared-memory
  // atomicMax per warp and node replaces the two global passes.  Unsorted input takes the general path.
  if (smem_nodes >= N) {
    bool sorted = true;
    const int n_ev = n_msg >> 1;
    for (int i = tid; i + 1 < n_ev; i += blockDim.x)
      sorted = sorted && (t[i] < t[i + 1] || (t[i] == t[i + 1] && eid[i] < eid[i + 1]));
    if (__syncthreads_and(sorted)) {
      for (int v = tid; v < N; v += blockDim.x) s_last[v] = -1;
      __syncthreads();
      const int n_round = (n_msg + 31) / 32 * 32;
      for (int j = tid; j < n_round; j += blockDim.x) {
        const int node = j < n_msg ? message_node(msg_node, ev_src, ev_dst, ev_keep, eid, j, N, E, status) : -1;
        const bool v = node >= 0;
        const unsigned act = __ballot_sync(FULL, v);
        if (v) {
          const unsigned peers = __match_any_sync(act, node);
          if (lane == 31 - __clz(peers)) atomicMax(&s_last[node], j);  // the highest lane holds the largest j
        }
      }
      __syncthreads();
      const int chunk = (N + blockDim.x - 1) / blockDim.x;
      const int nb = min(N, tid * chunk), ne = min(N, nb + chunk);
      int mine = 0;
      for (int v = nb; v < ne; ++v) mine += s_last[v] >= 0;
      int incl = mine;
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += y;
      }
      if (lane == 31) s_warp[wid] = incl;
      __syncthreads();
      if (wid == 0) {
        const int w = lane < (int)(blockDim.x >> 5) ? s_warp[lane] : 0;
        int wi = w;
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(FULL, wi, o);
          if (lane >= o) wi += y;
        }
        s_warp[lane] = wi - w;
        if (lane == 31) s_total = wi;
      }
      __syncthreads();
      int pos = s_warp[wid] + incl - mine;
      for (int v = nb; v < ne; ++v) {
        const int j = s_last[v];
        if (j >= 0) {
          uniq_out[pos] = v;
          winner_out[pos] = j;
          prev_uniq[pos] = v;
          node2slot[v] = pos;
          ++pos;
        }
      }
      if (tid == 0) { *n_uniq_out = s_total; *prev_n_uniq = s_total; }
      return;
    }
  }
  const int n_round = (n_msg + 31) / 32 * 32;
  for (int j = tid; j < n_round; j += blockDim.x) {
    const int node = j < n_msg ? message_node(msg_node, ev_src, ev_dst, ev_keep, eid, j, N, E, status) : -1;
    const bool v = node >= 0;
    const unsigned act = __ballot_sync(FULL, v);
    if (v) {
      const unsigned peers = __match_any_sync(act, node);
      const unsigned long long m = peer_max(peers, orderable(t[j >> 1]));
      if (lane == __ffs(peers) - 1) atomicMax(&best_t[node], m);
    }
  }
  __syncthreads();
  for (int j = tid; j < n_round; j += blockDim.x) {
    const int node = j < n_msg ? message_node(msg_node, ev_src, ev_dst, ev_keep, eid, j, N, E, status) : -1;
    const bool v = node >= 0 && orderable(t[j >> 1]) == best_t[node];
    const unsigned act = __ballot_sync(FULL, v);
    if (v) {
      const unsigned peers = __match_any_sync(act, node);
      const unsigned long long key = (((unsigned long long)(uint32_t)eid[j >> 1]) << 1 | (unsigned)(j & 1)) + 1ULL;
      const unsigned long long m = peer_max(peers, key);
      if (lane == __ffs(peers) - 1) atomicMax(&best_id[node], m);
    }
  }
  __syncthreads();
  for (int j = tid; j < n_msg; j += blockDim.x) {
    const int node = message_node(msg_node, ev_src, ev_dst, ev_keep, eid, j, N, E, status);
    if (node < 0) continue;
    const unsigned long long key = (((unsigned long long)(uint32_t)eid[j >> 1]) << 1 | (unsigned)(j & 1)) + 1ULL;
    if (orderable(t[j >> 1]) == best_t[node] && key == best_id[node]) win_msg[node] = j;
  }
  __syncthreads();
  // ascending compaction: thread i owns a contiguous chunk of node ids
  const int chunk = (N + blockDim.x - 1) / blockDim.x;
  const int nb = min(N, tid * chunk), ne = min(N, nb + chunk);
  int mine = 0;
  for (int v = nb; v < ne; ++v) mine += best_id[v] != 0ULL;
  int incl = mine;
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(FULL, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_warp[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    int w = lane < (int)(blockDim.x >> 5) ? s_warp[lane] : 0;
    int wi = w;
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(FULL, wi, o);
      if (lane >= o) wi += y;
    }
    s_warp[lane] = wi - w;  // exclusive prefix of the warp totals
    if (lane == 31) s_total = wi;
  }
  __syncthreads();
  int pos = s_warp[wid] + incl - mine;
  for (int v = nb; v < ne; ++v) {
    if (best_id[v] != 0ULL) {
      uniq_out[pos] = v;
      winner_out[pos] = win_msg[v];
      prev_uniq[pos] = v;
      node2slot[v] = pos;
      best_t[v] = 0ULL;
      best_id[v] = 0ULL;
      ++pos;
    }
  }
  if (tid == 0) { *n_uniq_out = s_total; *prev_n_uniq = s_total; }
}

}  // namespace

int launch_prune_mask(tgnn_ctx* ctx, const int32_t* src, const int32_t* dst, const int32_t* eid, const uint8_t* is_aux,
                      int n, int force_heavy, uint32_t drop_q32, uint64_t seed, int64_t batch_idx, uint8_t* keep_out,
                      int32_t* heavy_out, cudaStream_t s) {
  {
    KernelScope scope__(ctx, "prune_mask", s);
    prune_mask_kernel<<<1, 1024, 0, s>>>(src, dst, eid, is_aux, n, (int)ctx->cfg.num_nodes, ctx->ws.status, ctx->ws.hist, force_heavy, drop_q32, seed, batch_idx,
                                         keep_out, heavy_out);
  }
  TGNN_LAUNCH_OK(ctx, "prune_mask");
  return TGNN_OK;
}

int launch_sample_recent(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, int32_t* nbr_out,
                         int32_t* eid_out, double* ts_out, int32_t* cnt_out, cudaStream_t s) {
  if (n == 0) return TGNN_OK;
  const int warps_per_block = 8;
  {
    KernelScope scope__(ctx, "sample_recent", s);
    sample_recent_kernel<<<(n + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, s>>>(
        ctx->indptr, ctx->g_nbr, ctx->g_eid, ctx->g_ts, nodes, times, n, ctx->cfg.k, (int)ctx->cfg.num_nodes, ctx->ws.status,
        nbr_out, eid_out, ts_out, cnt_out);
  }
  TGNN_LAUNCH_OK(ctx, "sample_recent");
  return TGNN_OK;
}

int launch_stage_inputs(tgnn_ctx* ctx, const int32_t* u_src, const int32_t* u_dst, const double* u_t,
                        const int32_t* u_eid, const uint8_t* u_keep, int n_u, const int32_t* q_src, const int32_t* q_dst,
                        const int32_t* q_neg, const double* q_t, int n_q, const uint8_t* loss_mask, cudaStream_t s) {
  const int n = n_u > n_q ? n_u : n_q;
  if (n == 0) return TGNN_OK;
  Workspace& w = ctx->ws;
  StageArgs a = {u_src, u_dst, u_eid, q_src, q_dst, q_neg, u_t, q_t, u_keep, loss_mask,
                 w.st_u_src, w.st_u_dst, w.st_u_eid, w.st_q_src, w.st_q_dst, w.st_q_neg, w.st_u_t, w.st_q_t,
                 w.st_u_keep, w.st_mask, n_u, n_q};
  {
    KernelScope scope__(ctx, "stage_inputs", s);
    stage_inputs_kernel<<<(n + 255) / 256, 256, 0, s>>>(a);
  }
  TGNN_LAUNCH_OK(ctx, "stage_inputs");
  return TGNN_OK;
}

int launch_unpack_mixed(tgnn_ctx* ctx, const unsigned char* packed, int n, int n_q, bool with_mask, int slot,
                        cudaStream_t s) {
  const int m = n > n_q ? n : n_q;
  if (m == 0) return TGNN_OK;
  Workspace& w = ctx->ws;
  tgnn_ctx::MixedSlot& ms = ctx->mixed[slot];
  {
    KernelScope scope__(ctx, "unpack_mixed", s);
    unpack_mixed_kernel<<<(m + 255) / 256, 256, 0, s>>>(packed, n, n_q, ms.src, ms.dst, ms.eid, ms.t, ms.aux, ms.keep,
                                                        w.st_q_src, w.st_q_dst, w.st_q_neg, w.st_q_t,
                                                        with_mask ? w.st_mask : nullptr);
  }
  TGNN_LAUNCH_OK(ctx, "unpack_mixed");
  return TGNN_OK;
}

int launch_make_roots(tgnn_ctx* ctx, const int32_t* q_src, const int32_t* q_dst, const int32_t* q_neg,
                      const double* q_t, int n_q, cudaStream_t s) {
  if (n_q == 0) return TGNN_OK;
  {
    KernelScope scope__(ctx, "make_roots", s);
    make_roots_kernel<<<(3 * n_q + 255) / 256, 256, 0, s>>>(q_src, q_dst, q_neg, q_t, n_q, ctx->ws.r_node, ctx->ws.r_time);
  }
  TGNN_LAUNCH_OK(ctx, "make_roots");
  return TGNN_OK;
}

int launch_reduce_latest(tgnn_ctx* ctx, const int32_t* msg_node, const double* t, const int32_t* eid, int n_msg,
                         int32_t* uniq_out, int32_t* winner_out, int32_t* n_uniq_out, cudaStream_t s) {
  return launch_reduce_latest_events(ctx, msg_node, nullptr, nullptr, nullptr, t, eid, n_msg, uniq_out, winner_out,
                                     n_uniq_out, s);
}

int launch_reduce_latest_events(tgnn_ctx* ctx, const int32_t* msg_node, const int32_t* src, const int32_t* dst,
                                const uint8_t* keep, const double* t, const int32_t* eid, int n_msg, int32_t* uniq_out,
                                int32_t* winner_out, int32_t* n_uniq_out, cudaStream_t s) {
  Workspace& w = ctx->ws;
  // shared-memory table of the fast path: 4 bytes per node, when it fits
  const int N = (int)ctx->cfg.num_nodes;
  const int smem_nodes = (size_t)N * 4 <= 200 * 1024 ? N : 0;
  static SmemLimit smem_limit;
  if (smem_nodes * 4 > 48 * 1024) {
    const int rc = raise_smem_limit(ctx, reduce_latest_kernel, smem_nodes * 4, smem_limit);
    if (rc) return rc;
  }
  {
    KernelScope scope__(ctx, "reduce_latest", s);
    reduce_latest_kernel<<<1, 1024, (size_t)smem_nodes * 4, s>>>(msg_node, src, dst, keep, t, eid, n_msg, N, w.best_t,
                                                                 w.best_id, w.win_msg, w.node2slot, w.prev_uniq,
                                                                 w.prev_n_uniq, uniq_out, winner_out, n_uniq_out,
                                                                 smem_nodes, w.status,
                                                                 ctx->cfg.d_e > 0 && src != nullptr ? ctx->num_events : 0);
  }
  TGNN_LAUNCH_OK(ctx, "reduce_latest");
  return TGNN_OK;
}

}  // namespace tgnn
