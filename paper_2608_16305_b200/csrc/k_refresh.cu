// Boundary cache refresh (dynamic cache synchronisation, Algorithm 2): at an executed window boundary
// worker p fetches the state of every node of N_sync[p] -- memory row and last-update time -- from the
// worker that owns it.  The exchange itself is one all-to-all between the workers' processes; this file
// holds what runs on each GPU around it:
//   * the exchange plan of one worker for every window, computed once from the scan's N_sync flags:
//     which nodes it receives from each owner and which of its own nodes it sends to each requester,
//     both in ascending node order so that the two sides of a transfer agree without talking;
//   * packing the rows to send into one contiguous buffer, and writing received rows into the table.
// A packed row is d + 2 floats: the memory row, then the two halves of the fp64 time.
//
// Both row kernels move 2 x (4 d + 8) bytes per row and nothing else: they are bound by HBM (and by the
// row-granular access pattern on the table side: one 4d-byte segment per node, wherever it lies).
#include <cstdarg>
#include <cstdio>

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tgnn.h"

namespace {

constexpr unsigned FULL = 0xffffffffu;

int fail(char* err, int64_t size, int code, const char* fmt, ...) {
  if (err && size > 0) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(err, (size_t)size, fmt, ap);
    va_end(ap);
  }
  return code;
}

// Block (q, dir): dir 0 builds worker `me`'s receive list of window q (its N_sync nodes grouped by owner),
// dir 1 its send list (its own nodes grouped by the worker that asks for them).  Within a group the
// nodes ascend: the block sweeps the node range once per peer and appends the hits in order (ballot +
// warp prefix, then a prefix over the warps).
__global__ void __launch_bounds__(1024) refresh_plan_kernel(const uint8_t* __restrict__ sync, const int32_t* __restrict__ owner,
                                                            int64_t N, int P, int Q, int me, int64_t cap,
                                                            int32_t* __restrict__ recv_nodes, int32_t* __restrict__ recv_off,
                                                            int32_t* __restrict__ send_nodes, int32_t* __restrict__ send_off,
                                                            int32_t* status) {
  __shared__ int s_warp[32];
  __shared__ int s_base;
  const int q = blockIdx.x >> 1, dir = blockIdx.x & 1;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  int32_t* out = (dir ? send_nodes : recv_nodes) + (int64_t)q * cap;
  int32_t* off = (dir ? send_off : recv_off) + (int64_t)q * (P + 1);
  if (tid == 0) { s_base = 0; off[0] = 0; }
  __syncthreads();
  for (int peer = 0; peer < P; ++peer) {
    // receive: my flags, nodes owned by `peer`;  send: peer's flags, nodes owned by me
    const uint8_t* fl = sync + ((int64_t)(dir ? peer : me) * Q + q) * N;
    const int want_owner = dir ? me : peer;
    for (int64_t x0 = 0; x0 < N; x0 += blockDim.x) {
      const int64_t x = x0 + tid;
      bool hit = false;
      if (x < N && fl[x]) {
        const int o = owner[x];
        if (!dir && o == me) {
          if (peer == 0) atomicMax(status, 3);   // a worker never requests a node it owns
        } else {
          hit = (o == want_owner) && (peer != me);
        }
      }
      const unsigned b = __ballot_sync(FULL, hit);
      if (lane == 0) s_warp[wid] = __popc(b);
      __syncthreads();
      int before = 0, total = 0;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
        const int c = s_warp[w];
        if (w < wid) before += c;
        total += c;
      }
      const int base = s_base;
      if (hit) {
        const int64_t pos = (int64_t)base + before + __popc(b & ((1u << lane) - 1u));
        if (pos < cap) out[pos] = (int32_t)x;
        else atomicMax(status, 2);
      }
      __syncthreads();
      if (tid == 0) s_base = base + total;
      __syncthreads();
    }
    if (tid == 0) off[peer + 1] = s_base;
  }
}

// A warp moves ROWS rows at a time in 8-byte pieces (a packed row starts on an 8-byte boundary: d is
// even): all pieces of all its rows are loaded before the first is stored, so that ROWS x J independent
// loads per lane are in flight.  J = ceil((d / 2 + 1) / 32) pieces per lane and row; piece d / 2 is the time.
constexpr int ROWS = 4;

template <int J>
__global__ void __launch_bounds__(256) pack_rows_kernel(const float* __restrict__ memory, const double* __restrict__ last_update,
                                                        int64_t N, int d, const int32_t* __restrict__ nodes, int n,
                                                        float* __restrict__ packed, int32_t* status) {
  const int row0 = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * ROWS;
  const int lane = threadIdx.x & 31;
  if (row0 >= n) return;
  const int h = d >> 1;
  int my = (lane < ROWS && row0 + lane < n) ? nodes[row0 + lane] : -1;
  if (lane < ROWS && row0 + lane < n && (my < 0 || my >= N)) {
    atomicMax(status, 4);
    my = -1;
  }
  float2 v[ROWS][J];
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    const int node = __shfl_sync(FULL, my, r);
    const float2* src = reinterpret_cast<const float2*>(memory + (int64_t)(node < 0 ? 0 : node) * d);
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int c = lane + 32 * j;
      v[r][j] = make_float2(0.f, 0.f);
      if (node >= 0) {
        if (c < h) {
          v[r][j] = src[c];
        } else if (c == h) {
          const long long bits = __double_as_longlong(last_update[node]);
          v[r][j] = make_float2(__int_as_float((int)(bits & 0xffffffffll)), __int_as_float((int)(bits >> 32)));
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    if (row0 + r >= n) break;
    float2* dst = reinterpret_cast<float2*>(packed + (int64_t)(row0 + r) * (d + 2));
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int c = lane + 32 * j;
      if (c <= h) dst[c] = v[r][j];      // an out-of-range node id packs as zeros
    }
  }
}

template <int J>
__global__ void __launch_bounds__(256) unpack_rows_kernel(float* __restrict__ memory, double* __restrict__ last_update,
                                                          int64_t N, int d, const int32_t* __restrict__ nodes, int n,
                                                          const float* __restrict__ packed, int32_t* status) {
  const int row0 = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * ROWS;
  const int lane = threadIdx.x & 31;
  if (row0 >= n) return;
  const int h = d >> 1;
  int my = (lane < ROWS && row0 + lane < n) ? nodes[row0 + lane] : -1;
  if (lane < ROWS && row0 + lane < n && (my < 0 || my >= N)) {
    atomicMax(status, 4);
    my = -1;
  }
  float2 v[ROWS][J];
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    const float2* src = reinterpret_cast<const float2*>(packed + (int64_t)(row0 + r) * (d + 2));
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int c = lane + 32 * j;
      v[r][j] = (row0 + r < n && c <= h) ? src[c] : make_float2(0.f, 0.f);
    }
  }
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    const int node = __shfl_sync(FULL, my, r);
    if (node < 0) continue;             // beyond n, or an id outside the table: not written
    float2* dst = reinterpret_cast<float2*>(memory + (int64_t)node * d);
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int c = lane + 32 * j;
      if (c < h) {
        dst[c] = v[r][j];
      } else if (c == h) {
        const long long bits = ((long long)__float_as_int(v[r][j].y) << 32) | (unsigned int)__float_as_int(v[r][j].x);
        last_update[node] = __longlong_as_double(bits);
      }
    }
  }
}

constexpr int kMaxD = 32 * 2 * 8 - 2;   // J <= 8 pieces per lane

template <bool PACK>
cudaError_t launch_rows(const float* memory_in, float* memory_out, const double* lu_in, double* lu_out, int64_t N, int d,
                        const int32_t* nodes, int n, const float* packed_in, float* packed_out, int32_t* status,
                        cudaStream_t s) {
  const int J = (d / 2 + 1 + 31) / 32;
  const int grid = (n + 8 * ROWS - 1) / (8 * ROWS);
#define TGNN_ROWS_CASE(JJ)                                                                                              \
  case JJ:                                                                                                              \
    if (PACK) pack_rows_kernel<JJ><<<grid, 256, 0, s>>>(memory_in, lu_in, N, d, nodes, n, packed_out, status);         \
    else unpack_rows_kernel<JJ><<<grid, 256, 0, s>>>(memory_out, lu_out, N, d, nodes, n, packed_in, status);           \
    break;
  switch (J) {
    TGNN_ROWS_CASE(1) TGNN_ROWS_CASE(2) TGNN_ROWS_CASE(3) TGNN_ROWS_CASE(4) TGNN_ROWS_CASE(5) TGNN_ROWS_CASE(6)
    TGNN_ROWS_CASE(7) TGNN_ROWS_CASE(8)
    default: return cudaErrorInvalidValue;
  }
#undef TGNN_ROWS_CASE
  return cudaGetLastError();
}

}  // namespace

extern "C" {

int tgnn_refresh_plan(const uint8_t* sync, const int32_t* owner, int64_t num_nodes, int P, int Q, int me, int64_t cap,
                      int32_t* recv_nodes, int32_t* recv_off, int32_t* send_nodes, int32_t* send_off, int32_t* status_out,
                      void* stream, char* err_host, int64_t err_size) {
  if (num_nodes < 1 || P < 1 || Q < 0 || me < 0 || me >= P || cap < 0)
    return fail(err_host, err_size, TGNN_EINVAL, "tgnn_refresh_plan: size out of range");
  if (num_nodes > 0x7fffffff || cap > 0x7fffffff || Q > 0x3fffffff)
    return fail(err_host, err_size, TGNN_ECAPACITY, "tgnn_refresh_plan: node ids, capacity or windows exceed int32");
  if (!status_out || (Q > 0 && (!sync || !owner || !recv_off || !send_off || (cap > 0 && (!recv_nodes || !send_nodes)))))
    return fail(err_host, err_size, TGNN_EINVAL, "tgnn_refresh_plan: null pointer");
  cudaStream_t s = (cudaStream_t)stream;
  if (cudaMemsetAsync(status_out, 0, sizeof(int32_t), s) != cudaSuccess)
    return fail(err_host, err_size, TGNN_ECUDA, "tgnn_refresh_plan: %s", cudaGetErrorString(cudaGetLastError()));
  if (Q > 0)
    refresh_plan_kernel<<<(unsigned)(2 * Q), 1024, 0, s>>>(sync, owner, num_nodes, P, Q, me, cap, recv_nodes, recv_off,
                                                           send_nodes, send_off, status_out);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(err_host, err_size, TGNN_ECUDA, "tgnn_refresh_plan: %s", cudaGetErrorString(e));
  return TGNN_OK;
}

static int check_rows(const char* who, const void* memory, const void* last_update, int64_t num_nodes, int d,
                      const void* nodes, int n, const void* packed, const void* status, char* err_host, int64_t err_size) {
  if (num_nodes < 1 || d < 2 || (d & 1) || d > kMaxD || n < 0)
    return fail(err_host, err_size, TGNN_EINVAL, "%s: size out of range (d must be even and at most %d)", who, kMaxD);
  if (!status || !memory || !last_update || (n > 0 && (!nodes || !packed)))
    return fail(err_host, err_size, TGNN_EINVAL, "%s: null pointer", who);
  if ((((uintptr_t)memory | (uintptr_t)packed) & 7) != 0)
    return fail(err_host, err_size, TGNN_EINVAL, "%s: memory and packed must be 8-byte aligned", who);
  return TGNN_OK;
}

int tgnn_pack_rows(const float* memory, const double* last_update, int64_t num_nodes, int d, const int32_t* nodes, int n,
                   float* packed, int32_t* status, void* stream, char* err_host, int64_t err_size) {
  const int rc = check_rows("tgnn_pack_rows", memory, last_update, num_nodes, d, nodes, n, packed, status, err_host, err_size);
  if (rc) return rc;
  if (n == 0) return TGNN_OK;
  const cudaError_t e = launch_rows<true>(memory, nullptr, last_update, nullptr, num_nodes, d, nodes, n, nullptr, packed, status,
                                          (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(err_host, err_size, TGNN_ECUDA, "tgnn_pack_rows: %s", cudaGetErrorString(e));
  return TGNN_OK;
}

int tgnn_unpack_rows(float* memory, double* last_update, int64_t num_nodes, int d, const int32_t* nodes, int n,
                     const float* packed, int32_t* status, void* stream, char* err_host, int64_t err_size) {
  const int rc = check_rows("tgnn_unpack_rows", memory, last_update, num_nodes, d, nodes, n, packed, status, err_host, err_size);
  if (rc) return rc;
  if (n == 0) return TGNN_OK;
  const cudaError_t e = launch_rows<false>(nullptr, memory, nullptr, last_update, num_nodes, d, nodes, n, packed, nullptr, status,
                                           (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(err_host, err_size, TGNN_ECUDA, "tgnn_unpack_rows: %s", cudaGetErrorString(e));
  return TGNN_OK;
}

}  // extern "C"
