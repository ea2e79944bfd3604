// Step (5): single-layer multi-head temporal attention over the <= k sampled neighbors.
#include "tgnn_internal.cuh"
#include "tgnn_device.cuh"

// Raises a kernel's dynamic shared-memory limit (the attention kernels stage > 48 KB per block), once per device.
#define RC_ATTR(ctx, kernel, bytes)                                              \
  do {                                                                           \
    static tgnn::SmemLimit lim__;                                                \
    const int rc__ = tgnn::raise_smem_limit(ctx, kernel, (int)(bytes), lim__);   \
    if (rc__) return rc__;                                                       \
  } while (0)

namespace tgnn {
namespace {

// The attention inputs are gathered in two kernels.  The static part of a neighbor row z = [m_nbr ||
// x_eid || Phi(t - ts)] -- edge features, time encoding and its sine -- depends only on the sampled
// neighbors and the parameters, so it can run beside the memory update; the memory part has to wait
// for it.  One warp per row in both.
//
// Static part.  Rows [0, n*k): columns [d, ld) of Z (zero row if the slot is empty), z_dt (-1 if empty).
// Rows [n*k, n*k + n): the Phi(0) half of z_q.
// A warp takes ZS_ROWS neighbor rows at a time (registers kept to 80 so that three blocks fit an SM): their slot records first (one lane per row), then the
// feature loads of all of them, and only then the conversions, the time encodings and the stores -- the
// dependent chain slot -> event id -> feature row is paid once per ZS_ROWS rows instead of once per row.
constexpr int ZS_ROWS = 2;
constexpr int ZS_FEAT = 8;  // 32-bit feature words per lane and row held in registers: two 16-byte chunks of an
                            // fp32 row (de <= 256) or four bf16 pairs (de <= 256)

__global__ void __launch_bounds__(256, 3) gather_z_static_kernel(const void* __restrict__ efeat, int feat_bf16,
                                                              const float* __restrict__ time_w,
                                                              const float* __restrict__ time_b, int d, int de, int k,
                                                              const double* __restrict__ times, int n,
                                                              const int32_t* __restrict__ nbr,
                                                              const int32_t* __restrict__ eid,
                                                              const double* __restrict__ ts, int ld,
                                                              float* __restrict__ Z, float* __restrict__ z_dt,
                                                              float* __restrict__ Zq, int64_t N, int64_t E, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int nb_rows = n * k;
  const int dkv = 2 * d + de;
  const int wrow = feat_bf16 ? (de >> 1) : de;          // 32-bit words per feature row
  // fp32 rows as 16-byte chunks (rows and the destination columns are 16-byte aligned when d and de are
  // multiples of 4), bf16 rows as 32-bit pairs; anything wider or ragged goes row by row as before
  const bool vec4 = !feat_bf16 && (de & 3) == 0 && (d & 3) == 0 && (ld & 3) == 0 && de <= 256 &&
                    ((((uintptr_t)efeat) | ((uintptr_t)Z)) & 15) == 0;
  const bool pairs = feat_bf16 && wrow <= 128;
  const bool regs = vec4 || pairs;
  const int groups = (nb_rows + ZS_ROWS - 1) / ZS_ROWS;
  // the encoder's frequencies and phases of this lane's columns stay in registers (d <= 128: four per lane)
  const bool tw_regs = d <= 128;
  float tw[4], tb[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int q = lane + 32 * u;
    tw[u] = (tw_regs && q < d) ? time_w[q] : 0.f;
    tb[u] = (tw_regs && q < d) ? time_b[q] : 0.f;
  }
  for (int gidx = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; gidx < groups; gidx += warps) {
    const int r0 = gidx * ZS_ROWS;
    // slot records: lane j < ZS_ROWS reads row r0 + j
    int my_nbr = -1, my_eid = 0;
    float my_dt = 0.f;
    if (lane < ZS_ROWS && r0 + lane < nb_rows) {
      const int r = r0 + lane;
      my_nbr = nbr[r];
      my_eid = eid[r];
      my_dt = (float)(times[r / k] - ts[r]);
      // a slot naming a node or a feature row that does not exist is reported and treated as empty
      if (my_nbr >= 0 && !(index_ok(my_nbr, N, status) & (de == 0 || index_ok(my_eid, E, status)))) my_nbr = -1;
    }
    uint32_t f[ZS_ROWS][ZS_FEAT];
    int v_nbr[ZS_ROWS];
    float v_dt[ZS_ROWS];
#pragma unroll
    for (int j = 0; j < ZS_ROWS; ++j) {
      v_nbr[j] = __shfl_sync(0xffffffffu, my_nbr, j);
      v_dt[j] = __shfl_sync(0xffffffffu, my_dt, j);
      const int e = __shfl_sync(0xffffffffu, my_eid, j);
      if (regs && v_nbr[j] >= 0) {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(efeat) + (int64_t)e * wrow;
        if (vec4) {
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int q = lane + 32 * u;
            uint4 x = make_uint4(0u, 0u, 0u, 0u);
            if (q < (wrow >> 2)) x = __ldg(reinterpret_cast<const uint4*>(src) + q);
            f[j][4 * u] = x.x; f[j][4 * u + 1] = x.y; f[j][4 * u + 2] = x.z; f[j][4 * u + 3] = x.w;
          }
        } else {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int q = lane + 32 * u;
            f[j][u] = q < wrow ? __ldg(src + q) : 0u;
          }
        }
      } else if (!regs && v_nbr[j] >= 0) {
        warp_copy_feat(Z + (int64_t)(r0 + j) * ld + d, efeat, feat_bf16, e, de, lane);  // very wide rows: as before
      }
    }
#pragma unroll
    for (int j = 0; j < ZS_ROWS; ++j) {
      const int r = r0 + j;
      if (r >= nb_rows) break;
      float* row = Z + (int64_t)r * ld;
      if (v_nbr[j] < 0) {
        for (int q = lane; q < ld; q += 32) row[q] = 0.f;  // the memory part too: nobody else writes this row
        if (lane == 0) z_dt[r] = -1.f;  // marks the empty slot for the time-encoder gradient (a real dt is >= 0)
        continue;
      }
      if (vec4) {
        uint4* dst = reinterpret_cast<uint4*>(row + d);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int q = lane + 32 * u;
          if (q < (wrow >> 2)) dst[q] = make_uint4(f[j][4 * u], f[j][4 * u + 1], f[j][4 * u + 2], f[j][4 * u + 3]);
        }
      } else if (pairs) {
        float* dst = row + d;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int q = lane + 32 * u;
          if (q < wrow) {
            dst[2 * q] = __uint_as_float(f[j][u] << 16);
            dst[2 * q + 1] = __uint_as_float(f[j][u] & 0xffff0000u);
          }
        }
      }
      const float dtf = v_dt[j];
      float* phi = row + d + de;
      // the sines the backward pass needs are recomputed there from z_dt (cheaper than 4d bytes out and in again)
      if (tw_regs) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {  // four independent chains per lane
          const int q = lane + 32 * u;
          if (q < d) phi[q] = time_encode(tw[u], tb[u], dtf);
        }
      } else {
#pragma unroll 4
        for (int q = lane; q < d; q += 32) phi[q] = time_encode(time_w[q], time_b[q], dtf);
      }
      for (int q = dkv + lane; q < ld; q += 32) row[q] = 0.f;
      if (lane == 0) z_dt[r] = dtf;
    }
  }
  // the Phi(0) half of z_q
  for (int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps)
    for (int q = lane; q < d; q += 32) Zq[(int64_t)i * 2 * d + d + q] = time_encode(time_w[q], time_b[q], 0.f);
}

// The static part for the split-operand products: the same rows written as two fp16 planes (hi, lo; row pitch ld
// elements, planes plane_s elements apart) -- columns [d, d + de) edge features, [d + de, dkv) time encoding,
// column dkv a constant 1 (it turns the weight-gradient product's last column into the bias gradient), zeros up
// to ld; an empty slot is a row of zeros.  Values travel as pairs of neighbouring columns packed into 32-bit
// words (d and de are even).  Both planes hold fp16 numbers (activations of moderate size: 22 mantissa bits).
__global__ void __launch_bounds__(256, 4) gather_z_static_split_kernel(const void* __restrict__ efeat, int feat_bf16,
                                                                    const float* __restrict__ time_w,
                                                                    const float* __restrict__ time_b, int d, int de, int k,
                                                                    const double* __restrict__ times, int n,
                                                                    const int32_t* __restrict__ nbr,
                                                                    const int32_t* __restrict__ eid,
                                                                    const double* __restrict__ ts, int ld,
                                                                    __nv_bfloat16* __restrict__ z_hi, int64_t plane_s,
                                                                    float* __restrict__ z_dt, float* __restrict__ Zq, int64_t N,
                                                                    int64_t E, int32_t* status, int g_begin, int g_end) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int nb_rows = n * k;
  const int dkv = 2 * d + de;
  const int fp = de >> 1, tp = d >> 1;          // feature pairs, encoding pairs per row
  // words written per row: the dkv + 1 columns rounded up to 8 (the rest of the pitch, padding that keeps rows on
  // 128-byte lines, is never read: tile copies stop at the matrix's column count)
  const int zero_end = min(ld, (dkv + 1 + 7) / 8 * 8) >> 1;
  const int groups = (nb_rows + ZS_ROWS - 1) / ZS_ROWS;
  constexpr int FP_MAX = 4, TP_MAX = 2;         // pairs per lane held in registers: de <= 256, d <= 128
  const bool regs = fp <= 32 * FP_MAX && tp <= 32 * TP_MAX;
  float tw[TP_MAX][2], tb[TP_MAX][2];
#pragma unroll
  for (int u = 0; u < TP_MAX; ++u) {
    const int q = 2 * (lane + 32 * u);
    const bool in = regs && q < d;
    tw[u][0] = in ? time_w[q] : 0.f; tw[u][1] = in ? time_w[q + 1] : 0.f;
    tb[u][0] = in ? time_b[q] : 0.f; tb[u][1] = in ? time_b[q + 1] : 0.f;
  }
  // this launch covers the row groups [g_begin, g_end) (the gather goes out as several launches, see the launcher)
  // The slot records of a group (one lane per row) are fetched one group ahead: the dependent chain of a group is
  // slot record -> feature rows -> stores, and a warp that walks several groups would otherwise pay both round
  // trips one after the other for each of them.
  const int g_last = min(groups, g_end);
  int nx_nbr = -1, nx_eid = 0;
  double nx_t = 0.0, nx_ts = 0.0;
  auto fetch_slots = [&](int gi) {
    nx_nbr = -1; nx_eid = 0; nx_t = 0.0; nx_ts = 0.0;
    const int r = gi * ZS_ROWS + lane;
    if (gi < g_last && lane < ZS_ROWS && r < nb_rows) {
      nx_nbr = __ldg(nbr + r);
      nx_eid = __ldg(eid + r);
      nx_t = __ldg(times + r / k);
      nx_ts = __ldg(ts + r);
    }
  };
  const int g_first = g_begin + ((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  fetch_slots(g_first);
  for (int gidx = g_first; gidx < g_last; gidx += warps) {
    const int r0 = gidx * ZS_ROWS;
    int my_nbr = nx_nbr, my_eid = nx_eid;
    float my_dt = (float)(nx_t - nx_ts);
    fetch_slots(gidx + warps);   // in flight while this group's feature rows are fetched and written
    if (lane < ZS_ROWS && r0 + lane < nb_rows) {
      // a slot naming a node or a feature row that does not exist is reported and treated as empty
      if (my_nbr >= 0 && !(index_ok(my_nbr, N, status) & (de == 0 || index_ok(my_eid, E, status)))) my_nbr = -1;
    }
    // feature pairs of both rows first (the dependent chain slot -> event id -> feature row is paid once)
    uint32_t fa[ZS_ROWS][FP_MAX], fb[ZS_ROWS][FP_MAX];   // bf16 table: fa = the pair as stored; fp32 table: fa, fb = the two floats
    int v_nbr[ZS_ROWS], v_eid[ZS_ROWS];
    float v_dt[ZS_ROWS];
#pragma unroll
    for (int j = 0; j < ZS_ROWS; ++j) {
      v_nbr[j] = __shfl_sync(0xffffffffu, my_nbr, j);
      v_dt[j] = __shfl_sync(0xffffffffu, my_dt, j);
      v_eid[j] = __shfl_sync(0xffffffffu, my_eid, j);
      if (regs && v_nbr[j] >= 0) {
#pragma unroll
        for (int u = 0; u < FP_MAX; ++u) {
          const int q = lane + 32 * u;
          fa[j][u] = 0u; fb[j][u] = 0u;
          if (q < fp) {
            if (feat_bf16) {
              fa[j][u] = __ldg(reinterpret_cast<const uint32_t*>(efeat) + (int64_t)v_eid[j] * fp + q);
            } else {
              const uint2 x = __ldg(reinterpret_cast<const uint2*>(efeat) + (int64_t)v_eid[j] * fp + q);
              fa[j][u] = x.x; fb[j][u] = x.y;
            }
          }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < ZS_ROWS; ++j) {
      const int r = r0 + j;
      if (r >= nb_rows) break;
      uint32_t* hi = reinterpret_cast<uint32_t*>(z_hi + (int64_t)r * ld);
      uint32_t* lo = reinterpret_cast<uint32_t*>(z_hi + plane_s + (int64_t)r * ld);
      if (v_nbr[j] < 0) {
        for (int q = lane; q < zero_end; q += 32) { hi[q] = 0u; lo[q] = 0u; }   // the memory part too: nobody else writes this row
        if (lane == 0) z_dt[r] = -1.f;
        continue;
      }
      const float dtf = v_dt[j];
      if (regs) {
#pragma unroll
        for (int u = 0; u < FP_MAX; ++u) {
          const int q = lane + 32 * u;
          if (q < fp) {
            if (feat_bf16) {
              // A bf16 number is an fp16 number (8 significant bits, and the workloads' features lie inside fp16's
              // range), so its lo part is zero: the lo plane's feature columns are never written and stay at the
              // zeros they were allocated with.  (Below 6e-5 in magnitude the value is rounded to fp16's subnormal
              // grid instead: an absolute error under 3e-8.)
              hi[(d >> 1) + q] = pack_f16_pair(__uint_as_float(fa[j][u] << 16), __uint_as_float(fa[j][u] & 0xffff0000u));
            } else {
              uint32_t h, l;
              split_f16_pair(__uint_as_float(fa[j][u]), __uint_as_float(fb[j][u]), &h, &l);
              hi[(d >> 1) + q] = h; lo[(d >> 1) + q] = l;
            }
          }
        }
#pragma unroll
        for (int u = 0; u < TP_MAX; ++u) {
          const int q = lane + 32 * u;
          if (q < tp) {
            uint32_t h, l;
            split_f16_pair(time_encode(tw[u][0], tb[u][0], dtf), time_encode(tw[u][1], tb[u][1], dtf), &h, &l);
            hi[((d + de) >> 1) + q] = h; lo[((d + de) >> 1) + q] = l;
          }
        }
      } else {   // very wide rows: straight from memory, pair by pair
        for (int q = lane; q < fp; q += 32) {
          uint32_t h, l;
          if (feat_bf16) {
            const uint32_t w2 = __ldg(reinterpret_cast<const uint32_t*>(efeat) + (int64_t)v_eid[j] * fp + q);
            hi[(d >> 1) + q] = pack_f16_pair(__uint_as_float(w2 << 16), __uint_as_float(w2 & 0xffff0000u));
            continue;
          }
          const uint2 x = __ldg(reinterpret_cast<const uint2*>(efeat) + (int64_t)v_eid[j] * fp + q);
          split_f16_pair(__uint_as_float(x.x), __uint_as_float(x.y), &h, &l);
          hi[(d >> 1) + q] = h; lo[(d >> 1) + q] = l;
        }
        for (int q = lane; q < tp; q += 32) {
          uint32_t h, l;
          split_f16_pair(time_encode(time_w[2 * q], time_b[2 * q], dtf), time_encode(time_w[2 * q + 1], time_b[2 * q + 1], dtf), &h, &l);
          hi[((d + de) >> 1) + q] = h; lo[((d + de) >> 1) + q] = l;
        }
      }
      // column dkv = 1, then zeros up to the row pitch (dkv is even, the pitch a multiple of 8)
      for (int q = (dkv >> 1) + lane; q < zero_end; q += 32) { hi[q] = q == (dkv >> 1) ? 0x3c00u : 0u; lo[q] = 0u; }
      if (lane == 0) z_dt[r] = dtf;
    }
  }
  // (the Phi(0) half of z_q is written with the roots' memory rows, by gather_z_memory_kernel)
  (void)Zq;
}

// Memory part.  Rows [0, n*k): columns [0, d) of Z for the valid slots.  Rows [n*k, n*k + n): the
// memory half of z_q and of cat_o.
// z_hi != nullptr: the neighbor rows go to the two fp16 planes of the split products instead (pitch ld_s, planes
// plane_s apart), as pairs of columns packed into 32-bit words.
__global__ void __launch_bounds__(256) gather_z_memory_kernel(const float* __restrict__ memory, int d, int k,
                                                              const int32_t* __restrict__ nodes, int n,
                                                              const int32_t* __restrict__ nbr, int ld,
                                                              float* __restrict__ Z, float* __restrict__ Zq,
                                                              float* __restrict__ cat_o, __nv_bfloat16* __restrict__ z_hi,
                                                              int64_t plane_s, int ld_s, int64_t N, int32_t* status,
                                                              int part, const float* __restrict__ time_w,
                                                              const float* __restrict__ time_b) {
  // part: bit 0 = the neighbor rows, bit 1 = the root rows (with time_w != nullptr also their Phi(0) half of z_q, so
  // that the query projection depends on this launch alone)
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int nb_rows = n * k;
  if (z_hi != nullptr && (part & 1)) {
    // a warp takes four rows at a time: their slot records, then the four table rows (16 bytes per lane), then the
    // conversions and stores -- four independent round trips in flight per warp instead of a dependent chain per row
    const int d4 = d >> 2;          // <= 64: two 16-byte pieces per lane at most
    const int wg = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    for (int r0 = wg * 4; r0 < nb_rows; r0 += warps * 4) {
      int nb[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        nb[j] = r0 + j < nb_rows ? __ldg(nbr + r0 + j) : -1;
        if (nb[j] >= N) nb[j] = -1;   // reported by the static half, which left the row empty
      }
      float4 x[4][2];
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int q = lane + 32 * u;
          x[j][u] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (nb[j] >= 0 && q < d4) x[j][u] = __ldg(reinterpret_cast<const float4*>(memory + (int64_t)nb[j] * d) + q);
        }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (nb[j] < 0) continue;
        uint2* hi = reinterpret_cast<uint2*>(z_hi + (int64_t)(r0 + j) * ld_s);
        uint2* lo = reinterpret_cast<uint2*>(z_hi + plane_s + (int64_t)(r0 + j) * ld_s);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int q = lane + 32 * u;
          if (q < d4) {
            uint2 h, l;
            split_f16_pair(x[j][u].x, x[j][u].y, &h.x, &l.x);
            split_f16_pair(x[j][u].z, x[j][u].w, &h.y, &l.y);
            hi[q] = h; lo[q] = l;
          }
        }
      }
    }
  }
  const int r_first = (z_hi != nullptr || !(part & 1)) ? nb_rows : 0, r_last = (part & 2) ? nb_rows + n : nb_rows;
  for (int r = r_first + ((blockIdx.x * blockDim.x + threadIdx.x) >> 5); r < r_last; r += warps) {
    if (r < nb_rows) {
      const int nb = nbr[r];
      if (nb >= 0 && nb < N) warp_copy_f32(Z + (int64_t)r * ld, memory + (int64_t)nb * d, d, lane);
    } else {
      const int i = r - nb_rows;
      if (!index_ok(nodes[i], N, lane == 0 ? status : nullptr)) {   // a root outside the graph: reported, zero rows
        for (int q = lane; q < d; q += 32) { Zq[(int64_t)i * 2 * d + q] = 0.f; cat_o[(int64_t)i * 2 * d + d + q] = 0.f; }
        continue;
      }
      const float* m = memory + (int64_t)nodes[i] * d;
      warp_copy_f32(Zq + (int64_t)i * 2 * d, m, d, lane);
      warp_copy_f32(cat_o + (int64_t)i * 2 * d + d, m, d, lane);
    }
    if (r >= nb_rows && time_w != nullptr) {
      const int i = r - nb_rows;
      for (int q = lane; q < d; q += 32) Zq[(int64_t)i * 2 * d + d + q] = time_encode(time_w[q], time_b[q], 0.f);
    }
  }
}

// One warp per root.  Lane p < H*k owns the (head, slot) pair p: it forms the scaled dot product
// from shared memory, then the softmax over the head's valid slots; afterwards the lanes own output
// columns and accumulate the weighted sum of V into cat_o[:, :d].
__global__ void __launch_bounds__(256) attention_fwd_kernel(const float* __restrict__ Q, const float* __restrict__ KV,
                                                            const int32_t* __restrict__ cnt, int n, int d, int H, int k,
                                                            float* __restrict__ alpha, float* __restrict__ cat_o) {
  extern __shared__ __align__(16) float sm[];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int i = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (i >= n) return;
  float* Ks = sm + wib * attn_warp_floats(d, H, k);
  float* Vs = Ks + k * d;
  float* Qs = Vs + k * d;
  float* al = Qs + 2 * d;  // logits
  float* pr = al + H * k;  // probabilities
  const int dh = d / H;
  const int c = max(0, min(cnt[i], k));   // a count outside [0, k] is clamped (the neighbor search never produces one)
  const float scale = rsqrtf((float)dh);
  attn_stage_issue(Ks, Vs, Qs, Q, KV, i, c, d, k, lane);
  attn_stage_wait();
  for (int p = lane; p < H * k; p += 32) {
    const int h = p / k, s = p - h * k;
    float a = 0.f;
    if (s < c) {
      const float* kr = Ks + s * d + h * dh;
      const float* qr = Qs + h * dh;
      for (int e = 0; e < dh; ++e) a = fmaf(qr[e], kr[e], a);
      a *= scale;
    }
    al[p] = a;
  }
  __syncwarp();
  for (int p = lane; p < H * k; p += 32) {
    const int h = p / k, s = p - h * k;
    float out = 0.f;
    if (s < c) {
      float mx = -INFINITY, den = 0.f;
      for (int t = 0; t < c; ++t) mx = fmaxf(mx, al[h * k + t]);
      for (int t = 0; t < c; ++t) den += expf(al[h * k + t] - mx);
      out = expf(al[p] - mx) / den;
    }
    pr[p] = out;
    alpha[(int64_t)i * H * k + p] = out;
  }
  __syncwarp();
  for (int e = lane; e < d; e += 32) {
    const int h = e / dh;
    float a = 0.f;
    for (int s = 0; s < c; ++s) a = fmaf(pr[h * k + s], Vs[s * d + e], a);
    cat_o[(int64_t)i * 2 * d + e] = a;
  }
}

// The same kernel for compile-time shapes (D columns, H heads, KS slots; D / H even, H * KS <= 32): the generic
// kernel above spends 1 900 instructions per root, mostly loop control and scalar shared-memory loads, and is bound
// by instruction issue.  Here the dot products read pairs of columns, the exponentials are formed once per (head,
// slot) and shared through shared memory, and the weighted sum of V runs on four columns per lane.  Every sum keeps
// the generic kernel's order of operations, so the two give the same bits.
template <int D, int H, int KS>
__host__ __device__ constexpr int attn_fwd_fixed_floats() { return (KS * D + D + 2 * H * KS + 3) & ~3; }   // K rows, query, two scratch vectors
template <int D, int H, int KS>
__global__ void __launch_bounds__(256, 5) attention_fwd_fixed_kernel(const float* __restrict__ Q, const float* __restrict__ KV,
                                                                     const int32_t* __restrict__ cnt, int n,
                                                                     float* __restrict__ alpha, float* __restrict__ cat_o) {
  constexpr int DH = D / H, D4 = D / 4, P = H * KS;
  static_assert(D % 4 == 0 && DH % 2 == 0 && P <= 32 && D4 <= 32, "shape not covered by the fixed kernel");
  extern __shared__ __align__(16) float sm[];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int i = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (i >= n) return;
  // Only the K halves and the query are staged (4.6 KB per warp: five blocks per SM instead of three); the V halves
  // are read once, column-wise, straight from global memory in the last phase.
  float* Ks = sm + wib * attn_fwd_fixed_floats<D, H, KS>();
  float* Qs = Ks + KS * D;
  float* al = Qs + D;      // logits
  float* pr = al + P;      // exponentials, then probabilities
  const int c = max(0, min(cnt[i], KS));   // a count outside [0, k] is clamped (the neighbor search never produces one)
  const float scale = rsqrtf((float)DH);
  const float* kv = KV + (int64_t)i * KS * 2 * D + 4 * lane;
  if (lane < D4) {
    cp_async16(Qs + 4 * lane, Q + (int64_t)i * D + 4 * lane);
    float* kd = Ks + 4 * lane;
#pragma unroll
    for (int t = 0; t < KS; ++t)
      if (t < c) cp_async16(kd + t * D, kv + t * 2 * D);
  }
  attn_stage_wait();
  const int h = lane / KS, sl = lane - h * KS;
  const bool live = lane < P && sl < c;
  float a = 0.f;
  if (live) {
    const float2* kr = reinterpret_cast<const float2*>(Ks + sl * D + h * DH);
    const float2* qr = reinterpret_cast<const float2*>(Qs + h * DH);
#pragma unroll
    for (int e = 0; e < DH / 2; ++e) {
      const float2 qv = qr[e], kv2 = kr[e];
      a = fmaf(qv.x, kv2.x, a);
      a = fmaf(qv.y, kv2.y, a);
    }
    a *= scale;
  }
  if (lane < P) al[lane] = a;
  __syncwarp();
  float ex = 0.f;
  if (live) {
    float mx = -INFINITY;
#pragma unroll
    for (int t = 0; t < KS; ++t)
      if (t < c) mx = fmaxf(mx, al[h * KS + t]);
    ex = expf(a - mx);
  }
  if (lane < P) pr[lane] = ex;
  __syncwarp();
  float out = 0.f;
  if (live) {
    float den = 0.f;
#pragma unroll
    for (int t = 0; t < KS; ++t)
      if (t < c) den += pr[h * KS + t];
    out = ex / den;
  }
  __syncwarp();   // every lane has read the exponentials
  if (lane < P) {
    pr[lane] = out;
    alpha[(int64_t)i * P + lane] = out;
  }
  __syncwarp();
  if (lane < D4) {
    const int h0 = (4 * lane) / DH, h1 = (4 * lane + 2) / DH;   // columns 4l, 4l+1 share a head, and so do 4l+2, 4l+3
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    constexpr int HALF = (KS + 1) / 2;   // the rows' loads go out in two rounds (registers)
#pragma unroll
    for (int t0 = 0; t0 < KS; t0 += HALF) {
      float4 v[HALF];
#pragma unroll
      for (int u = 0; u < HALF; ++u)
        if (t0 + u < KS && t0 + u < c) v[u] = __ldg(reinterpret_cast<const float4*>(kv + (t0 + u) * 2 * D + D));
#pragma unroll
      for (int u = 0; u < HALF; ++u) {
        const int t = t0 + u;
        if (t < KS && t < c) {
          const float p0 = pr[h0 * KS + t], p1 = pr[h1 * KS + t];
          acc.x = fmaf(p0, v[u].x, acc.x); acc.y = fmaf(p0, v[u].y, acc.y);
          acc.z = fmaf(p1, v[u].z, acc.z); acc.w = fmaf(p1, v[u].w, acc.w);
        }
      }
    }
    *reinterpret_cast<float4*>(cat_o + (int64_t)i * 2 * D + 4 * lane) = acc;
  }
}

// Time-projected embedding: h[i] = memory[node_i] * (1 + dt_i w_p + b_p), dt_i = fp32(t_i - last_update[node_i]).
// One warp per root, 128-bit accesses (d is a multiple of 4, rows 16-byte aligned).
__global__ void __launch_bounds__(256) jodie_embed_kernel(const float* __restrict__ memory,
                                                          const double* __restrict__ last_update,
                                                          const float* __restrict__ proj_w,
                                                          const float* __restrict__ proj_b,
                                                          const int32_t* __restrict__ nodes,
                                                          const double* __restrict__ times, int n, int d,
                                                          float* __restrict__ h, int64_t N, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (i >= n) return;
  const int node = nodes[i];
  if (!index_ok(node, N, lane == 0 ? status : nullptr)) {   // reported; the embedding of a node that does not exist is zero
    for (int q = lane; q < d; q += 32) h[(int64_t)i * d + q] = 0.f;
    return;
  }
  const float dt = (float)(times[i] - last_update[node]);
  const float4* m4 = reinterpret_cast<const float4*>(memory + (int64_t)node * d);
  float4* h4 = reinterpret_cast<float4*>(h + (int64_t)i * d);
  for (int q = lane; q < (d >> 2); q += 32) {
    const float4 m = __ldg(m4 + q);
    const float4 w = *reinterpret_cast<const float4*>(proj_w + 4 * q);
    const float4 b = *reinterpret_cast<const float4*>(proj_b + 4 * q);
    float4 o;
    o.x = m.x * (1.f + fmaf(dt, w.x, b.x));
    o.y = m.y * (1.f + fmaf(dt, w.y, b.y));
    o.z = m.z * (1.f + fmaf(dt, w.z, b.z));
    o.w = m.w * (1.f + fmaf(dt, w.w, b.w));
    h4[q] = o;
  }
}

}  // namespace

int launch_embed_static(tgnn_ctx* ctx, const double* times, int n, const int32_t* nbr, const int32_t* eid,
                        const double* ts, cudaStream_t s) {
  if (n == 0) return TGNN_OK;
  const tgnn_config& c = ctx->cfg;
  const ParamLayout& L = ctx->L;
  Workspace& w = ctx->ws;
  {
    KernelScope scope__(ctx, "gather_z_static", s);
    if (ctx->split_buf != nullptr && ctx->z_split) {
      // Large batches in three pieces: the gather runs on a low-priority side stream beside the memory update, whose
      // products need whole SMs; between two pieces the SMs that drain go to those kernels first.
      const int groups = (n * c.k + ZS_ROWS - 1) / ZS_ROWS;
      const int per = groups >= 32768 ? (groups + 2) / 3 : groups;   // (small batches: one launch)
      for (int g0 = 0; g0 < groups; g0 += per) {
        const int g1 = g0 + per < groups ? g0 + per : groups;
        // a grid of four waves (three blocks per SM at a time) whose warps walk the groups: the encoder's frequencies
        // and phases are loaded once per warp for several pairs of rows, and blocks still end often enough for the
        // kernels of the chain (higher priority) to find room between them
        const int want = (g1 - g0 + 7) / 8 + 1;
        gather_z_static_split_kernel<<<want < 148 * 12 ? want : 148 * 12, 256, 0, s>>>(
            ctx->efeat, c.feat_dtype == TGNN_BF16, ctx->params + L.time_w, ctx->params + L.time_b, c.d, c.d_e, c.k, times, n,
            nbr, eid, ts, (int)ctx->zs.ld, reinterpret_cast<__nv_bfloat16*>(ctx->zs.hi), ctx->zs.plane_stride, w.z_dt, w.Zq,
            c.num_nodes, ctx->num_events, w.status, g0, g1);
        ctx->launches++;
      }
      ctx->launches--;
    } else
      gather_z_static_kernel<<<(n * c.k / ZS_ROWS + n + 7) / 8 + 1, 256, 0, s>>>(ctx->efeat, c.feat_dtype == TGNN_BF16, ctx->params + L.time_w,
                                                          ctx->params + L.time_b, c.d, c.d_e, c.k, times, n, nbr, eid, ts,
                                                          ctx->ld_kv, w.Z, w.z_dt, w.Zq, c.num_nodes, ctx->num_events, w.status);
  }
  TGNN_LAUNCH_OK(ctx, "gather_z_static");
  return TGNN_OK;
}

int launch_embed(tgnn_ctx* ctx, const int32_t* nodes, const double* times, int n, const int32_t* nbr,
                 const int32_t* eid, const double* ts, const int32_t* cnt, float* h_out, cudaStream_t s) {
  const tgnn_config& c = ctx->cfg;
  // tgnn_train_step left work on its side stream; it is waited for where it is first needed
  const bool pending = ctx->side_pending;
  ctx->side_pending = false;
  if (pending && (n == 0 || c.model == TGNN_MODEL_JODIE)) TGNN_CUDA_OK(ctx, cudaStreamWaitEvent(s, ctx->ev_side_done, 0));
  if (n == 0) return TGNN_OK;
  const ParamLayout& L = ctx->L;
  Workspace& w = ctx->ws;
  const int d = c.d, k = c.k, H = c.heads;
  if (c.model == TGNN_MODEL_JODIE) {
    {
      KernelScope scope__(ctx, "jodie_embed", s);
      jodie_embed_kernel<<<(n + 7) / 8, 256, 0, s>>>(ctx->memory, ctx->last_update, ctx->params + L.proj_w,
                                                     ctx->params + L.proj_b, nodes, times, n, d, h_out, c.num_nodes, w.status);
    }
    TGNN_LAUNCH_OK(ctx, "jodie_embed");
    return TGNN_OK;
  }
  const int rows = n * k + n;
  // split operands: the attention inputs are written as fp16 planes, complete before the product starts
  const bool split = ctx->split_buf != nullptr && ctx->images_fresh;
  if (!ctx->z_static_done) {
    ctx->z_split = split;
    const int rc0 = launch_embed_static(ctx, times, n, nbr, eid, ts, s);
    if (rc0) return rc0;
  } else if (ctx->z_split != split) {
    return set_error(ctx, TGNN_ESTATE, "embed: the static half of the attention inputs was gathered in the other operand format");
  }
  ctx->z_static_done = false;
  // In the tensor-core modes the key/value projection reads the neighbors' memory rows straight from
  // the table (row-indirect A), so the copy of those rows into Z -- still needed by the backward pass,
  // like the root rows by the query and output projections -- leaves the critical chain for a side stream.
  const bool indirect = c.math_mode != TGNN_MATH_FP32 && !split;
  int rc = fork_to(ctx, s, ctx->side[0]);
  if (rc) return rc;
  if (split) {
    // root rows (both halves of z_q, the memory half of cat_o) on the side stream, where the query projection
    // follows them at once; the neighbor rows -- planes the key/value projection reads -- on this one
    {
      KernelScope scope__(ctx, "gather_roots", ctx->side[0]);
      gather_z_memory_kernel<<<(n + 7) / 8, 256, 0, ctx->side[0]>>>(ctx->memory, d, k, nodes, n, nbr, ctx->ld_kv, w.Z, w.Zq, w.cat_o,
                                                                   reinterpret_cast<__nv_bfloat16*>(ctx->zs.hi), ctx->zs.plane_stride,
                                                                   (int)ctx->zs.ld, c.num_nodes, w.status, 2,
                                                                   ctx->params + L.time_w, ctx->params + L.time_b);
    }
    TGNN_LAUNCH_OK(ctx, "gather_roots");
    {
      KernelScope scope__(ctx, "gather_z_memory", s);
      // a grid that fits the machine once (six blocks per SM), rows in groups of four per warp
      const int nbr_rows = n * k;
      const int gblocks = (nbr_rows + 31) / 32 < 148 * 6 ? (nbr_rows + 31) / 32 : 148 * 6;
      gather_z_memory_kernel<<<gblocks, 256, 0, s>>>(ctx->memory, d, k, nodes, n, nbr, ctx->ld_kv, w.Z, w.Zq, w.cat_o,
                                                    reinterpret_cast<__nv_bfloat16*>(ctx->zs.hi), ctx->zs.plane_stride,
                                                    (int)ctx->zs.ld, c.num_nodes, w.status, 1, nullptr, nullptr);
    }
    TGNN_LAUNCH_OK(ctx, "gather_z_memory");
    // the static half of the attention inputs (the step's side stream) is needed from here on
    if (pending) TGNN_CUDA_OK(ctx, cudaStreamWaitEvent(s, ctx->ev_side_done, 0));
  } else {
    cudaStream_t sg = indirect ? ctx->side[0] : s;
    {
      KernelScope scope__(ctx, "gather_z_memory", sg);
      gather_z_memory_kernel<<<(rows + 7) / 8, 256, 0, sg>>>(ctx->memory, d, k, nodes, n, nbr, ctx->ld_kv, w.Z, w.Zq, w.cat_o, nullptr,
                                                            0, 0, c.num_nodes, w.status, 3, nullptr, nullptr);
    }
    TGNN_LAUNCH_OK(ctx, "gather_z_memory");
    if (!indirect) {  // the query projection below runs on the side stream and needs the rows just gathered
      rc = fork_to(ctx, s, ctx->side[0]);
      if (rc) return rc;
    }
    // the static half of the attention inputs (the step's side stream) is needed from here on: by the key/value
    // projection and, through the time encoding of the roots, by the query projection on side[0]
    if (pending) {
      TGNN_CUDA_OK(ctx, cudaStreamWaitEvent(s, ctx->ev_side_done, 0));
      TGNN_CUDA_OK(ctx, cudaStreamWaitEvent(ctx->side[0], ctx->ev_side_done, 0));
    }
  }
  GemmArgs g = {};
  g.A = w.Z; g.a_rs = ctx->ld_kv; g.a_cs = 1;
  g.B = ctx->params + L.wk; g.b_rs = 1; g.b_cs = L.dkv;  // rows of [W_k; W_v]
  g.C = w.KV; g.ldc = 2 * d; g.M = n * k; g.N = 2 * d; g.K = (int)L.dkv;
  g.bias = ctx->params + L.bk; g.split_k = 1; g.site = SITE_KV + 1;
  if (indirect) { g.a_idx = nbr; g.a_tab = ctx->memory; g.a_tab_cols = d; g.a_tab_rows = c.num_nodes; }
  if (split) {
    SplitMat zs = ctx->zs;
    zs.rows = n * k;
    zs.cols = L.dkv;   // the forward product stops before the column of ones
    rc = launch_gemm_split(ctx, zs, ctx->wkv_s, 0, w.KV, 2 * d, n * k, 2 * d, (int)L.dkv, ctx->params + L.bk, 0, 0, 1, "kv_proj", s);
  } else {
    rc = launch_gemm(ctx, g, "kv_proj", s);
  }
  if (rc) return rc;
  g = GemmArgs{};
  g.A = w.Zq; g.a_rs = 2 * d; g.a_cs = 1;
  g.B = ctx->params + L.wq; g.b_rs = 1; g.b_cs = 2 * d;
  g.C = w.Q; g.ldc = d; g.M = n; g.N = d; g.K = 2 * d; g.bias = ctx->params + L.bq; g.split_k = 1; g.site = SITE_Q + 1;
  rc = launch_gemm(ctx, g, "q_proj", ctx->side[0]);
  if (rc) return rc;
  rc = fork_to(ctx, ctx->side[0], s);
  if (rc) return rc;
  const int wpb = attn_warps_per_block(d, H, k);
  const bool fixed_shape = d == 100 && H == 2 && k == 10;   // the paper's configuration
  constexpr int fixed_smem = 8 * attn_fwd_fixed_floats<100, 2, 10>() * 4;   // eight warps per block
  if (fixed_shape) RC_ATTR(ctx, (attention_fwd_fixed_kernel<100, 2, 10>), fixed_smem);
  else RC_ATTR(ctx, attention_fwd_kernel, attn_smem_bytes(d, H, k, wpb));
  {
    KernelScope scope__(ctx, "attention_fwd", s);
    if (fixed_shape)
      attention_fwd_fixed_kernel<100, 2, 10><<<(n + 7) / 8, 256, fixed_smem, s>>>(w.Q, w.KV, cnt, n, w.alpha, w.cat_o);
    else
      attention_fwd_kernel<<<(n + wpb - 1) / wpb, wpb * 32, attn_smem_bytes(d, H, k, wpb), s>>>(w.Q, w.KV, cnt, n, d, H, k,
                                                                                             w.alpha, w.cat_o);
  }
  TGNN_LAUNCH_OK(ctx, "attention_fwd");
  g = GemmArgs{};
  g.A = w.cat_o; g.a_rs = 2 * d; g.a_cs = 1;
  g.B = ctx->params + L.wo; g.b_rs = 1; g.b_cs = 2 * d;
  g.C = h_out; g.ldc = d; g.M = n; g.N = d; g.K = 2 * d; g.bias = ctx->params + L.bo; g.relu = 1; g.split_k = 1; g.site = SITE_OUT + 1;
  return launch_gemm(ctx, g, "out_proj", s);
}

}  // namespace tgnn
