// Offline preprocessing of the event stream: the source-based backward dependency scan
// (Algorithm 1) for every worker and synchronisation window at once, and the construction of one
// worker's mixed batches (Eq. 5) from the scan's result.
//
// The listing is a sequential backward walk whose frontier F grows as it goes.  Here each
// (worker, window) pair is one thread block that computes the same sets as a least fixed point:
//   position i   = index of an event in the walk (0 = last event of the window, counting backward);
//   entry[x]     = position from which node x is in F: the first position of batch s for the remote
//                  destinations of the batch's target events (they enter before the batch is walked),
//                  i + 1 for the remote endpoints of an auxiliary event at position i;
//   an event at position i whose source is remote is auxiliary iff min(entry[u], entry[v]) <= i.
// All events of the window are relaxed together (atomicMin on entry[]) until a sweep changes
// nothing.  What an event decides depends only on entries set at smaller positions, so the fixed
// point is unique and equals what the walk produces; the number of sweeps is the length of the
// longest chain of events pulling one another in, bounded by the window's event count.
#include <cstdarg>
#include <cstdio>

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tgnn.h"

namespace {

constexpr unsigned FULL = 0xffffffffu;
constexpr int kInf = 0x3fffffff;
constexpr int kMaxBlocks = TGNN_SCAN_MAX_BLOCKS;

int fail(char* err, int64_t size, int code, const char* fmt, ...) {
  if (err && size > 0) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(err, (size_t)size, fmt, ap);
    va_end(ap);
  }
  return code;
}

__global__ void __launch_bounds__(256) backward_scan_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                                                            int64_t E, int batch, int K,
                                                            const int32_t* __restrict__ owner, int64_t N, int P, int Q,
                                                            uint8_t* __restrict__ role, int32_t* __restrict__ n_sync,
                                                            uint8_t* __restrict__ sync, int32_t* scratch,
                                                            int32_t* status) {
  __shared__ int s_changed;
  __shared__ int s_count;
  const int tid = threadIdx.x;
  int32_t* entry = scratch + (int64_t)blockIdx.x * N;
  for (int64_t pq = blockIdx.x; pq < (int64_t)P * Q; pq += gridDim.x) {
    const int p = (int)(pq / Q), q = (int)(pq % Q);
    const int64_t lo = (int64_t)q * K * batch;
    const int64_t hi = min(E, lo + (int64_t)K * batch);
    const int n = (int)(hi - lo);
    uint8_t* rl = role + (int64_t)p * E;
    for (int64_t x = tid; x < N; x += blockDim.x) entry[x] = kInf;
    if (tid == 0) s_count = 0;
    __syncthreads();
    // target events, and their remote destinations at the first position of their batch
    for (int64_t e = lo + tid; e < hi; e += blockDim.x) {
      const int u = src[e], v = dst[e];
      const bool tar = owner[u] == p;
      rl[e] = tar ? 1 : 0;
      if (tar && owner[v] != p) {
        const int64_t s_end = min(hi, (e / batch + 1) * batch);  // one past the batch's last event
        atomicMin(&entry[v], (int)(hi - s_end));
      }
    }
    __syncthreads();
    bool converged = false;
    for (int sweep = 0; sweep <= n; ++sweep) {
      if (tid == 0) s_changed = 0;
      __syncthreads();
      for (int64_t e = lo + tid; e < hi; e += blockDim.x) {
        const int u = src[e], v = dst[e];
        const bool ru = owner[u] != p;
        if (!ru) continue;
        const int i = (int)(hi - 1 - e);
        const int m = min(atomicMin(&entry[u], kInf), atomicMin(&entry[v], kInf));  // current values
        if (m <= i) {
          bool ch = false;
          if (rl[e] != 2) { rl[e] = 2; ch = true; }
          if (atomicMin(&entry[u], i + 1) > i + 1) ch = true;
          if (owner[v] != p && atomicMin(&entry[v], i + 1) > i + 1) ch = true;
          if (ch) s_changed = 1;
        }
      }
      __syncthreads();
      const int changed = s_changed;
      __syncthreads();
      if (!changed) { converged = true; break; }
    }
    if (!converged && tid == 0) atomicExch(status, 1);
    // N_sync = the frontier after the walk
    int c = 0;
    for (int64_t x = tid; x < N; x += blockDim.x) {
      const bool in = entry[x] < kInf;
      c += in;
      if (sync) sync[pq * N + x] = in ? 1 : 0;
    }
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(FULL, c, o);
    if ((tid & 31) == 0 && c) atomicAdd(&s_count, c);
    __syncthreads();
    if (tid == 0) n_sync[pq] = s_count;
    __syncthreads();
  }
}

// ---- mixed batches of one worker --------------------------------------------------------------
// off[s + 1] = events of batch s with role != 0, toff[s + 1] = with role == 1 (one block per batch)
__global__ void __launch_bounds__(256) mixed_count_kernel(const uint8_t* __restrict__ role, int64_t E, int batch,
                                                          int32_t* __restrict__ off, int32_t* __restrict__ toff) {
  __shared__ int s_a, s_t;
  const int s = blockIdx.x;
  if (threadIdx.x == 0) { s_a = 0; s_t = 0; }
  __syncthreads();
  const int64_t lo = (int64_t)s * batch, hi = min(E, lo + batch);
  int a = 0, t = 0;
  for (int64_t e = lo + threadIdx.x; e < hi; e += blockDim.x) {
    const uint8_t r = role[e];
    a += r != 0;
    t += r == 1;
  }
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(FULL, a, o);
    t += __shfl_xor_sync(FULL, t, o);
  }
  if ((threadIdx.x & 31) == 0) { atomicAdd(&s_a, a); atomicAdd(&s_t, t); }
  __syncthreads();
  if (threadIdx.x == 0) { off[s + 1] = s_a; toff[s + 1] = s_t; }
}

// In-place inclusive prefix sums of off[1..nb] and toff[1..nb] (off[0] = toff[0] = 0): one block, chunks of 1024.
__global__ void __launch_bounds__(1024) mixed_offsets_kernel(int32_t* off, int32_t* toff, int nb) {
  __shared__ int s_warp[2][32];
  __shared__ int s_carry[2];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) { off[0] = 0; toff[0] = 0; s_carry[0] = 0; s_carry[1] = 0; }
  __syncthreads();
  for (int base = 0; base < nb; base += 1024) {
    const int j = base + tid;
    int a = j < nb ? off[j + 1] : 0, t = j < nb ? toff[j + 1] : 0;
    for (int o = 1; o < 32; o <<= 1) {
      const int a2 = __shfl_up_sync(FULL, a, o), t2 = __shfl_up_sync(FULL, t, o);
      if (lane >= o) { a += a2; t += t2; }
    }
    if (lane == 31) { s_warp[0][wid] = a; s_warp[1][wid] = t; }
    __syncthreads();
    if (wid == 0) {
      int wa = s_warp[0][lane], wt = s_warp[1][lane];
      for (int o = 1; o < 32; o <<= 1) {
        const int a2 = __shfl_up_sync(FULL, wa, o), t2 = __shfl_up_sync(FULL, wt, o);
        if (lane >= o) { wa += a2; wt += t2; }
      }
      s_warp[0][lane] = wa; s_warp[1][lane] = wt;
    }
    __syncthreads();
    const int pa = (wid ? s_warp[0][wid - 1] : 0) + s_carry[0], pt = (wid ? s_warp[1][wid - 1] : 0) + s_carry[1];
    if (j < nb) { off[j + 1] = a + pa; toff[j + 1] = t + pt; }
    __syncthreads();
    if (tid == 1023) { s_carry[0] = a + pa; s_carry[1] = t + pt; }
    __syncthreads();
  }
}

// Stable compaction of batch s: events with role != 0 in stream (= timestamp) order into the mixed-batch
// arrays at off[s], the targets among them into the target arrays at toff[s].
__global__ void __launch_bounds__(256) mixed_fill_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                                                         const double* __restrict__ t, const int32_t* __restrict__ neg,
                                                         const uint8_t* __restrict__ role, int64_t E, int batch,
                                                         const int32_t* __restrict__ off, const int32_t* __restrict__ toff,
                                                         int64_t cap_mixed, int64_t cap_tgt, int32_t* __restrict__ mb_src,
                                                         int32_t* __restrict__ mb_dst, double* __restrict__ mb_t,
                                                         int32_t* __restrict__ mb_eid, uint8_t* __restrict__ mb_aux,
                                                         int32_t* __restrict__ tg_src, int32_t* __restrict__ tg_dst,
                                                         double* __restrict__ tg_t, int32_t* __restrict__ tg_neg,
                                                         int32_t* __restrict__ tg_eid, int32_t* status) {
  __shared__ int s_wa[8], s_wt[8];
  __shared__ int s_base_a, s_base_t;
  const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int64_t lo = (int64_t)s * batch, hi = min(E, lo + batch);
  if (tid == 0) { s_base_a = off[s]; s_base_t = toff[s]; }
  __syncthreads();
  for (int64_t base = lo; base < hi; base += blockDim.x) {
    const int64_t e = base + tid;
    const uint8_t r = e < hi ? role[e] : 0;
    const unsigned ba = __ballot_sync(FULL, r != 0), bt = __ballot_sync(FULL, r == 1);
    if (lane == 0) { s_wa[wid] = __popc(ba); s_wt[wid] = __popc(bt); }
    __syncthreads();
    int pa = s_base_a, pt = s_base_t;
    for (int w = 0; w < wid; ++w) { pa += s_wa[w]; pt += s_wt[w]; }
    const unsigned below = (1u << lane) - 1u;
    if (r != 0) {
      const int64_t o = pa + __popc(ba & below);
      if (o < cap_mixed) {
        mb_src[o] = src[e]; mb_dst[o] = dst[e]; mb_t[o] = t[e]; mb_eid[o] = (int32_t)e; mb_aux[o] = r == 2;
      } else {
        atomicExch(status, 2);
      }
    }
    if (r == 1) {
      const int64_t o = pt + __popc(bt & below);
      if (o < cap_tgt) {
        tg_src[o] = src[e]; tg_dst[o] = dst[e]; tg_t[o] = t[e]; tg_eid[o] = (int32_t)e;
        if (tg_neg) tg_neg[o] = neg ? neg[e] : -1;
      } else {
        atomicExch(status, 2);
      }
    }
    __syncthreads();
    if (tid == 0) {
      int a = 0, tt = 0;
      for (int w = 0; w < 8; ++w) { a += s_wa[w]; tt += s_wt[w]; }
      s_base_a += a; s_base_t += tt;
    }
    __syncthreads();
  }
}

}  // namespace

extern "C" {

int64_t tgnn_backward_scan_scratch(int64_t num_events, int batch, int K, int64_t num_nodes, int P) {
  if (num_events < 0 || batch < 1 || K < 1 || num_nodes < 1 || P < 1) return -1;
  const int64_t nb = (num_events + batch - 1) / batch;
  const int64_t Q = (nb + K - 1) / K;
  const int64_t blocks = P * Q < kMaxBlocks ? P * Q : kMaxBlocks;
  return (blocks > 0 ? blocks : 1) * num_nodes;
}

int tgnn_backward_scan(const int32_t* src, const int32_t* dst, int64_t num_events, int batch, int K,
                       const int32_t* owner, int64_t num_nodes, int P, uint8_t* role_out, int32_t* n_sync_out,
                       uint8_t* sync_out, int32_t* scratch, int32_t* status_out, void* stream, char* err_host,
                       int64_t err_size) {
  if (num_events < 0 || batch < 1 || K < 1 || num_nodes < 1 || P < 1)
    return fail(err_host, err_size, TGNN_EINVAL, "tgnn_backward_scan: size out of range");
  if ((int64_t)K * batch > 0x3ffffff0)
    return fail(err_host, err_size, TGNN_ECAPACITY, "tgnn_backward_scan: window of %lld events exceeds the position range",
                (long long)K * batch);
  if (num_events == 0) return TGNN_OK;
  if (!src || !dst || !owner || !role_out || !n_sync_out || !scratch || !status_out)
    return fail(err_host, err_size, TGNN_EINVAL, "tgnn_backward_scan: null pointer");
  const int64_t nb = (num_events + batch - 1) / batch;
  const int64_t Q = (nb + K - 1) / K;
  if (Q > 0x7fffffff / P) return fail(err_host, err_size, TGNN_ECAPACITY, "tgnn_backward_scan: too many windows");
  const int64_t pairs = (int64_t)P * Q;
  const int blocks = (int)(pairs < kMaxBlocks ? pairs : kMaxBlocks);
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemsetAsync(status_out, 0, sizeof(int32_t), s) != cudaSuccess)
    return fail(err_host, err_size, TGNN_ECUDA, "tgnn_backward_scan: %s", cudaGetErrorString(cudaGetLastError()));
  backward_scan_kernel<<<blocks, 256, 0, s>>>(src, dst, num_events, batch, K, owner, num_nodes, P, (int)Q, role_out,
                                              n_sync_out, sync_out, scratch, status_out);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(err_host, err_size, TGNN_ECUDA, "tgnn_backward_scan: %s", cudaGetErrorString(e));
  return TGNN_OK;
}

int tgnn_build_mixed(const int32_t* src, const int32_t* dst, const double* t, const int32_t* neg, int64_t num_events,
                     int batch, const uint8_t* role, int32_t* mb_off_out, int32_t* tgt_off_out, int64_t cap_mixed,
                     int64_t cap_tgt, int32_t* mb_src, int32_t* mb_dst, double* mb_t, int32_t* mb_eid, uint8_t* mb_aux,
                     int32_t* tgt_src, int32_t* tgt_dst, double* tgt_t, int32_t* tgt_neg, int32_t* tgt_eid,
                     int32_t* status_out, void* stream, char* err_host, int64_t err_size) {
  if (num_events < 0 || batch < 1 || cap_mixed < 0 || cap_tgt < 0)
    return fail(err_host, err_size, TGNN_EINVAL, "tgnn_build_mixed: size out of range");
  if (num_events > 0x7fffffff) return fail(err_host, err_size, TGNN_ECAPACITY, "tgnn_build_mixed: event ids exceed int32");
  if (!mb_off_out || !tgt_off_out || !status_out) return fail(err_host, err_size, TGNN_EINVAL, "tgnn_build_mixed: null pointer");
  const int64_t nb = (num_events + batch - 1) / batch;
  if (nb > 0x7ffffff0) return fail(err_host, err_size, TGNN_ECAPACITY, "tgnn_build_mixed: too many batches");
  if (num_events > 0 && (!src || !dst || !t || !role || !mb_src || !mb_dst || !mb_t || !mb_eid || !mb_aux || !tgt_src ||
                         !tgt_dst || !tgt_t || !tgt_eid))
    return fail(err_host, err_size, TGNN_EINVAL, "tgnn_build_mixed: null pointer");
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemsetAsync(status_out, 0, sizeof(int32_t), s) != cudaSuccess)
    return fail(err_host, err_size, TGNN_ECUDA, "tgnn_build_mixed: %s", cudaGetErrorString(cudaGetLastError()));
  if (nb > 0) mixed_count_kernel<<<(unsigned)nb, 256, 0, s>>>(role, num_events, batch, mb_off_out, tgt_off_out);
  mixed_offsets_kernel<<<1, 1024, 0, s>>>(mb_off_out, tgt_off_out, (int)nb);
  if (nb > 0)
    mixed_fill_kernel<<<(unsigned)nb, 256, 0, s>>>(src, dst, t, neg, role, num_events, batch, mb_off_out, tgt_off_out,
                                                   cap_mixed, cap_tgt, mb_src, mb_dst, mb_t, mb_eid, mb_aux, tgt_src,
                                                   tgt_dst, tgt_t, tgt_neg, tgt_eid, status_out);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(err_host, err_size, TGNN_ECUDA, "tgnn_build_mixed: %s", cudaGetErrorString(e));
  return TGNN_OK;
}

}  // extern "C"
