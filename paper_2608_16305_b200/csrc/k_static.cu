// tgnn_reduce_latest_static: the per-node latest-event reduction for callers that must not
// allocate device memory.  Its per-node scratch tables live in a fixed array that is part of
// the library image instead of a workspace obtained from cudaMalloc.
#include <cstdarg>
#include <cstdio>
#include <mutex>

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tgnn.h"

namespace {

constexpr unsigned FULL = 0xffffffffu;
constexpr int64_t kMaxNodes = TGNN_STATIC_MAX_NODES;

// Per node: best time key (8 B), best (eid, role) key (8 B), winning message index (4 B).
// 20 B x 65 536 nodes = 1.25 MiB, resident on every GPU that loads the library until exit.
constexpr size_t kScratchBytes = (size_t)kMaxNodes * (8 + 8 + 4);
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address each device gave the array is looked up once per device and cached here.
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

__device__ __forceinline__ unsigned long long orderable(double x) {
  unsigned long long u = (unsigned long long)__double_as_longlong(x);
  return (u >> 63) ? ~u : (u | 0x8000000000000000ULL);
}

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

// Same algorithm as the workspace-backed reduction: two order-independent atomicMax passes
// (time, then eid/role among the messages tying on time), then an ascending compaction.
// The tables hold whatever the previous call left, so the first thing the kernel does is
// clear the N entries it is going to use.
__global__ void __launch_bounds__(1024) reduce_latest_static_kernel(const int32_t* __restrict__ msg_node,
                                                                    const double* __restrict__ t,
                                                                    const int32_t* __restrict__ eid, int n_msg, int N,
                                                                    unsigned char* scratch,
                                                                    int32_t* __restrict__ uniq_out,
                                                                    int32_t* __restrict__ winner_out,
                                                                    int32_t* __restrict__ n_uniq_out) {
  unsigned long long* best_t = reinterpret_cast<unsigned long long*>(scratch);
  unsigned long long* best_id = best_t + kMaxNodes;
  int32_t* win_msg = reinterpret_cast<int32_t*>(best_id + kMaxNodes);
  __shared__ int s_warp[32];
  __shared__ int s_total;
  __shared__ int s_bad;  // a message named a node outside [0, N): it is skipped, never used as an index
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) s_bad = 0;
  for (int v = tid; v < N; v += blockDim.x) { best_t[v] = 0ULL; best_id[v] = 0ULL; }
  __syncthreads();
  const int n_round = (n_msg + 31) / 32 * 32;
  for (int j = tid; j < n_round; j += blockDim.x) {
    const int node = j < n_msg ? msg_node[j] : -1;
    if (node >= N) s_bad = 1;
    const bool v = node >= 0 && node < N;
    const unsigned act = __ballot_sync(FULL, v);
    if (v) {
      const unsigned peers = __match_any_sync(act, node);
      const unsigned long long m = peer_max(peers, orderable(t[j >> 1]));
      if (lane == __ffs(peers) - 1) atomicMax(&best_t[node], m);
    }
  }
  __syncthreads();
  for (int j = tid; j < n_round; j += blockDim.x) {
    const int node = j < n_msg ? msg_node[j] : -1;
    const bool v = node >= 0 && node < N && orderable(t[j >> 1]) == best_t[node];
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
    const int node = msg_node[j];
    if (node < 0 || node >= N) continue;
    const unsigned long long key = (((unsigned long long)(uint32_t)eid[j >> 1]) << 1 | (unsigned)(j & 1)) + 1ULL;
    if (orderable(t[j >> 1]) == best_t[node] && key == best_id[node]) win_msg[node] = j;
  }
  __syncthreads();
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
    if (best_id[v] != 0ULL) {
      uniq_out[pos] = v;
      winner_out[pos] = win_msg[v];
      ++pos;
    }
  }
  if (tid == 0) *n_uniq_out = s_bad ? -1 : s_total;
}

int fail(char* err, int err_size, int code, const char* fmt, ...) {
  if (err && err_size > 0) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(err, (size_t)err_size, fmt, ap);
    va_end(ap);
  }
  return code;
}

}  // namespace

extern "C" int tgnn_reduce_latest_static(const int32_t* msg_node, const double* t, const int32_t* eid, int n_msg,
                                         int64_t num_nodes, int32_t* uniq_out, int32_t* winner_out,
                                         int32_t* n_uniq_out, void* stream, char* err_host, int err_size) {
  if (err_host && err_size > 0) err_host[0] = '\0';
  if (num_nodes < 1 || num_nodes > kMaxNodes)
    return fail(err_host, err_size, TGNN_ECAPACITY,
                "reduce_latest_static: num_nodes %lld is outside 1..%lld (TGNN_STATIC_MAX_NODES, the size of the "
                "built-in scratch array); use tgnn_reduce_latest with a context for larger graphs",
                (long long)num_nodes, (long long)kMaxNodes);
  if (n_msg < 0 || n_msg % 2 != 0 || n_msg > (1 << 25))
    return fail(err_host, err_size, TGNN_EINVAL, "reduce_latest_static: n_msg %lld must be even and in 0..%lld",
                (long long)n_msg, (long long)(1 << 25));
  if (!n_uniq_out || (n_msg > 0 && (!msg_node || !t || !eid || !uniq_out || !winner_out)))
    return fail(err_host, err_size, TGNN_EINVAL, "reduce_latest_static: null pointer");
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail(err_host, err_size, TGNN_ECUDA, "reduce_latest_static: cudaGetDevice failed (%lld) or device index %lld unsupported",
                (long long)e, (long long)dev);
  void* scratch = nullptr;
  {
    // Once per device, with that device current: ask the runtime where this device keeps the array.
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || !p) {
        cudaGetLastError();
        return fail(err_host, err_size, TGNN_ECUDA, "reduce_latest_static: cudaGetSymbolAddress failed (%lld) on device %lld",
                    (long long)e, (long long)dev);
      }
      g_scratch_addr[dev] = p;
    }
    scratch = g_scratch_addr[dev];
  }
  reduce_latest_static_kernel<<<1, 1024, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      msg_node, t, eid, n_msg, (int)num_nodes, static_cast<unsigned char*>(scratch), uniq_out, winner_out, n_uniq_out);
  e = cudaGetLastError();
  if (e != cudaSuccess)
    return fail(err_host, err_size, TGNN_ECUDA, "reduce_latest_static: kernel launch failed (%lld)", (long long)e);
  return TGNN_OK;
}
