// Step (6): masked link-prediction loss (Eq. 13), exact backward of steps (4)-(5),
// gradient norm g_r and the Adam update.
#include "tgnn_internal.cuh"
#include "tgnn_device.cuh"

namespace tgnn {
namespace {

constexpr unsigned FULL = 0xffffffffu;

// cat1[p] = [h_src || h_dst] for p < nq (positive pairs), [h_src || h_neg] for p >= nq.
__global__ void __launch_bounds__(256) head_gather_kernel(const float* __restrict__ h, int nq, int d,
                                                          float* __restrict__ cat1) {
  const int64_t total = (int64_t)2 * nq * 2 * d;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int p = (int)(e / (2 * d)), q = (int)(e % (2 * d));
    const int j = p < nq ? p : p - nq;
    const int row = q < d ? j : (p < nq ? nq + j : 2 * nq + j);
    cat1[e] = h[(int64_t)row * d + (q < d ? q : q - d)];
  }
}

// One warp per target event: both scores, the event's loss term, d loss / d score, then
// hid1 is overwritten by d loss / d pre1.  Accumulates dw_2, db_2 and the loss.
__global__ void __launch_bounds__(256) head_loss_kernel(float* __restrict__ hid1, const float* __restrict__ w2,
                                                        const float* __restrict__ b2,
                                                        const uint8_t* __restrict__ loss_mask, int nq, int d,
                                                        float* __restrict__ g_w2, float* __restrict__ g_b2,
                                                        float* __restrict__ loss_acc, uint8_t* __restrict__ hid_gate) {
  extern __shared__ float s_gw2[];  // [d]
  __shared__ float s_msum;
  __shared__ float s_gb2, s_loss;
  const int lane = threadIdx.x & 31;
  for (int q = threadIdx.x; q < d; q += blockDim.x) s_gw2[q] = 0.f;
  if (threadIdx.x == 0) { s_msum = 0.f; s_gb2 = 0.f; s_loss = 0.f; }
  __syncthreads();
  {  // every block counts the whole mask (a few KB)
    int c = 0;
    for (int j = threadIdx.x; j < nq; j += blockDim.x) c += loss_mask ? (loss_mask[j] != 0) : 1;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(FULL, c, o);
    if (lane == 0 && c) atomicAdd(&s_msum, (float)c);
  }
  __syncthreads();
  const float msum = s_msum;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  for (int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; j < nq; j += warps) {
    const float m = (loss_mask ? (loss_mask[j] != 0) : 1) ? 1.f : 0.f;
    const float wj = msum > 0.f ? m / msum : 0.f;
    float* hp = hid1 + (int64_t)j * d;
    float* hn = hid1 + (int64_t)(nq + j) * d;
    float sp = 0.f, sn = 0.f;
    for (int q = lane; q < d; q += 32) {
      sp = fmaf(w2[q], hp[q], sp);
      sn = fmaf(w2[q], hn[q], sn);
    }
    for (int o = 16; o > 0; o >>= 1) {
      sp += __shfl_xor_sync(FULL, sp, o);
      sn += __shfl_xor_sync(FULL, sn, o);
    }
    sp += b2[0];
    sn += b2[0];
    const float dsp = -wj * sigmoidf_(-sp);
    const float dsn = wj * sigmoidf_(sn);
    if (lane == 0) {
      atomicAdd(&s_loss, wj * (softplusf_(-sp) + softplusf_(sn)));
      atomicAdd(&s_gb2, dsp + dsn);
    }
    for (int q = lane; q < d; q += 32) {
      const float a = hp[q], b = hn[q];
      if (wj != 0.f) atomicAdd(&s_gw2[q], dsp * a + dsn * b);
      hp[q] = a > 0.f ? dsp * w2[q] : 0.f;
      hn[q] = b > 0.f ? dsn * w2[q] : 0.f;
      hid_gate[(int64_t)j * d + q] = a > 0.f;
      hid_gate[(int64_t)(nq + j) * d + q] = b > 0.f;
    }
  }
  __syncthreads();
  for (int q = threadIdx.x; q < d; q += blockDim.x)
    if (s_gw2[q] != 0.f) atomicAdd(&g_w2[q], s_gw2[q]);
  if (threadIdx.x == 0) {
    if (s_gb2 != 0.f) atomicAdd(g_b2, s_gb2);
    if (s_loss != 0.f) atomicAdd(loss_acc, s_loss);
  }
}

// d loss / d pre_o = ReLU'(h) * d loss / d h, where dh collects the head's input gradients.
__global__ void __launch_bounds__(256) dh_kernel(const float* __restrict__ dcat1, const float* __restrict__ h, int nq,
                                                 int d, float* __restrict__ dpre_o, int relu_out) {
  const int64_t total = (int64_t)3 * nq * d;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int i = (int)(e / d), q = (int)(e % d);
    float g;
    if (i < nq)
      g = dcat1[(int64_t)i * 2 * d + q] + dcat1[(int64_t)(nq + i) * 2 * d + q];
    else if (i < 2 * nq)
      g = dcat1[(int64_t)(i - nq) * 2 * d + d + q];
    else
      g = dcat1[(int64_t)(i - nq) * 2 * d + d + q];
    dpre_o[e] = (!relu_out || h[e] > 0.f) ? g : 0.f;
  }
}

// The whole link-prediction head for a group of 4 target events (8 pairs: 4 positive, 4 negative) in one
// block: gather [h_a || h_b], hidden layer, scores, the masked loss (Eq. 13), and the backward pass down to
// d loss / d pre_o of the 12 embedding rows involved.  W_1 stays in shared memory (row pitch 2d+1: both the
// forward sweep, threads over hidden units, and the backward sweep, threads over input columns, are free
// of bank conflicts) while the block walks over its groups.  Also leaves what the leaves of the chain
// need: cat1 and d loss / d pre1 (for dW_1, db_1), the hidden gates, and the sums for dw_2, db_2 and the loss.
// Rows of hsT: 0-3 source, 4-7 destination, 8-11 negative.  Dynamic shared memory: head_fused_smem(d) bytes.
// relu_out: the embedding rows are outputs of a ReLU layer (attention model) and dpre_o is masked by it;
// otherwise dpre_o is the plain gradient with respect to the embedding rows.
// Two teams of 512 threads share the block's copy of W_1 and work on two groups side by side (their phases
// are latency-bound, so the teams overlap almost for free, and a batch of 600 events -- 150 groups -- fits
// 75 blocks with nothing left over for a second round).  Team barriers are the named barriers 1 and 2.
constexpr int HF_EV = 4, HF_TEAM = 512, HF_TEAMS = 2, HF_THREADS = HF_TEAM * HF_TEAMS;
__host__ __device__ inline int head_fused_w_floats(int d) { return (d * (2 * d + 1) + 3) & ~3; }
inline size_t head_fused_smem(int d) {
  return (size_t)(head_fused_w_floats(d) + HF_TEAMS * (12 * d + 12 * d + 8 * d + 8 * 2 * d) + d) * sizeof(float);
}

__global__ void __launch_bounds__(HF_THREADS) head_fused_kernel(const float* __restrict__ h, const float* __restrict__ W1,
                                                                const float* __restrict__ b1,
                                                                const float* __restrict__ w2, const float* __restrict__ b2,
                                                                const uint8_t* __restrict__ loss_mask, int nq, int d,
                                                                float* __restrict__ cat1, float* __restrict__ dpre1,
                                                                uint8_t* __restrict__ hid_gate,
                                                                float* __restrict__ dpre_o, float* __restrict__ g_w2,
                                                                float* __restrict__ g_b2, float* __restrict__ loss_acc,
                                                                int relu_out) {
  extern __shared__ __align__(16) float sm[];
  __shared__ float s_msum, s_gb2, s_loss;
  const int PW = 2 * d + 1;
  const int tid = threadIdx.x, lane = tid & 31;
  const int team = tid / HF_TEAM, tt = tid - team * HF_TEAM, wid = tt >> 5;  // team, thread and warp within the team
  float* W1s = sm;                                                         // [d][2d+1]  (shared by the teams)
  float* gw2 = W1s + head_fused_w_floats(d);                               // [d]        (shared)
  float* hsT = gw2 + d + team * (12 * d + 12 * d + 8 * d + 16 * d);        // [d][12]   embedding rows, transposed
  float* part = hsT + 12 * d;                   // [d][12]   W_1a h_src | W_1b h_dst | W_1b h_neg per event
  float* dh1T = part + 12 * d;                  // [d][8]    d loss / d pre1, transposed
  float* dc = dh1T + 8 * d;                     // [2d][8]   partial input gradients of the lower half of j
  auto team_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "n"(HF_TEAM) : "memory"); };
  {  // W_1 [d][2d] -> padded rows; 2d is a multiple of 4 and the parameter block is 16-byte aligned
    const int n4 = d * 2 * d / 4, row4 = 2 * d / 4;
    const bool vec = (((uintptr_t)W1) & 15) == 0;
    for (int e = tid; e < n4; e += blockDim.x) {
      const int j = e / row4, c = 4 * (e - j * row4);
      float4 v;
      if (vec) v = __ldg(reinterpret_cast<const float4*>(W1) + e);
      else v = make_float4(W1[4 * e], W1[4 * e + 1], W1[4 * e + 2], W1[4 * e + 3]);
      float* dst = W1s + j * PW + c;
      dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    }
  }
  for (int q = tid; q < d; q += blockDim.x) gw2[q] = 0.f;
  if (tid == 0) { s_msum = 0.f; s_gb2 = 0.f; s_loss = 0.f; }
  __syncthreads();
  {  // every block counts the whole mask (a few KB)
    int c = 0;
    for (int j = tid; j < nq; j += blockDim.x) c += loss_mask ? (loss_mask[j] != 0) : 1;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(FULL, c, o);
    if (lane == 0 && c) atomicAdd(&s_msum, (float)c);
  }
  __syncthreads();
  const float msum = s_msum;
  const float bias2 = b2[0];
  const int groups = (nq + HF_EV - 1) / HF_EV;
  for (int grp = blockIdx.x * HF_TEAMS + team; grp < groups; grp += gridDim.x * HF_TEAMS) {
    const int ev0 = grp * HF_EV;
    for (int e = tt; e < 12 * d; e += HF_TEAM) {
      const int r = e / d, q = e - r * d;
      const int ev = ev0 + (r & 3), blk = r >> 2;
      float v = 0.f;
      if (ev < nq) {
        v = h[((int64_t)blk * nq + ev) * d + q];
        if (blk == 0) {
          cat1[(int64_t)ev * 2 * d + q] = v;
          cat1[(int64_t)(nq + ev) * 2 * d + q] = v;
        } else if (blk == 1) {
          cat1[(int64_t)ev * 2 * d + d + q] = v;
        } else {
          cat1[(int64_t)(nq + ev) * 2 * d + d + q] = v;
        }
      }
      hsT[q * 12 + r] = v;
    }
    team_sync();
    // hidden layer in three parts: a thread owns hidden unit j and one block of 4 embedding rows (the
    // source rows serve the positive and the negative pair of their event, so their part is formed once)
    for (int it = tt; it < 3 * d; it += HF_TEAM) {
      const int blk = it / d, j = it - blk * d;
      const float* wr = W1s + j * PW + (blk ? d : 0);
      const float* hb = hsT + 4 * blk;
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 4
      for (int c = 0; c < d; ++c) {
        const float x = wr[c];
        const float4 v = *reinterpret_cast<const float4*>(hb + c * 12);
        a0 = fmaf(x, v.x, a0); a1 = fmaf(x, v.y, a1); a2 = fmaf(x, v.z, a2); a3 = fmaf(x, v.w, a3);
      }
      *reinterpret_cast<float4*>(part + j * 12 + 4 * blk) = make_float4(a0, a1, a2, a3);
    }
    team_sync();
    // scores, loss terms and d loss / d pre1: one warp per pair
    for (int p = wid; p < 8; p += (HF_TEAM >> 5)) {
      const int half = p >> 2, e4 = p & 3, ev = ev0 + e4;
      const bool valid = ev < nq;
      const int o_col = 4 + 4 * half + e4;  // the pair's second row: destination or negative
      float sc = 0.f;
      for (int q = lane; q < d; q += 32) {
        const float a = fmaxf(part[q * 12 + e4] + part[q * 12 + o_col] + b1[q], 0.f);
        sc = fmaf(w2[q], a, sc);
      }
      for (int o = 16; o > 0; o >>= 1) sc += __shfl_xor_sync(FULL, sc, o);
      sc += bias2;
      const float m = valid && (loss_mask ? (loss_mask[ev] != 0) : true) ? 1.f : 0.f;
      const float wj = msum > 0.f ? m / msum : 0.f;
      const float ds = half == 0 ? -wj * sigmoidf_(-sc) : wj * sigmoidf_(sc);
      if (lane == 0 && wj != 0.f) {
        atomicAdd(&s_loss, wj * (half == 0 ? softplusf_(-sc) : softplusf_(sc)));
        atomicAdd(&s_gb2, ds);
      }
      const int64_t row = (int64_t)half * nq + ev;
      for (int q = lane; q < d; q += 32) {
        const float a = fmaxf(part[q * 12 + e4] + part[q * 12 + o_col] + b1[q], 0.f);
        if (wj != 0.f) atomicAdd(&gw2[q], ds * a);
        const float dv = a > 0.f ? ds * w2[q] : 0.f;
        dh1T[q * 8 + p] = dv;
        if (valid) {
          dpre1[row * d + q] = dv;
          hid_gate[row * d + q] = a > 0.f;
        }
      }
    }
    team_sync();
    // input gradient: a thread owns column c of [h_a || h_b] for all 8 pairs over one half of the hidden
    // units; the lower half parks its sums in shared memory, the upper half adds them and folds the pairs
    // into the embedding rows (the source row collects its positive and its negative pair)
    const int jh = (d + 1) / 2;
    for (int base = 0; base < 4 * d; base += HF_TEAM) {  // items [0, 2d): lower half of j, [2d, 4d): upper half
      const int it = base + tt;
      const bool act = it < 4 * d;
      const int hi = act ? it / (2 * d) : 0, c = act ? it - hi * 2 * d : 0;
      float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (act) {
        const int j0 = hi ? jh : 0, j1 = hi ? d : jh;
#pragma unroll 4
        for (int j = j0; j < j1; ++j) {
          const float x = W1s[j * PW + c];
          const float4 u = *reinterpret_cast<const float4*>(dh1T + j * 8);
          const float4 v = *reinterpret_cast<const float4*>(dh1T + j * 8 + 4);
          a[0] = fmaf(x, u.x, a[0]); a[1] = fmaf(x, u.y, a[1]); a[2] = fmaf(x, u.z, a[2]); a[3] = fmaf(x, u.w, a[3]);
          a[4] = fmaf(x, v.x, a[4]); a[5] = fmaf(x, v.y, a[5]); a[6] = fmaf(x, v.z, a[6]); a[7] = fmaf(x, v.w, a[7]);
        }
        if (hi == 0) {
          *reinterpret_cast<float4*>(dc + c * 8) = make_float4(a[0], a[1], a[2], a[3]);
          *reinterpret_cast<float4*>(dc + c * 8 + 4) = make_float4(a[4], a[5], a[6], a[7]);
        }
      }
      team_sync();
      if (act && hi == 1) {
        const float4 u = *reinterpret_cast<const float4*>(dc + c * 8);
        const float4 v = *reinterpret_cast<const float4*>(dc + c * 8 + 4);
        a[0] += u.x; a[1] += u.y; a[2] += u.z; a[3] += u.w;
        a[4] += v.x; a[5] += v.y; a[6] += v.z; a[7] += v.w;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int ev = ev0 + e;
          if (ev >= nq) break;
          if (c < d) {
            dpre_o[(int64_t)ev * d + c] = (!relu_out || hsT[c * 12 + e] > 0.f) ? a[e] + a[4 + e] : 0.f;
          } else {
            const int q = c - d;
            dpre_o[((int64_t)nq + ev) * d + q] = (!relu_out || hsT[q * 12 + 4 + e] > 0.f) ? a[e] : 0.f;
            dpre_o[((int64_t)2 * nq + ev) * d + q] = (!relu_out || hsT[q * 12 + 8 + e] > 0.f) ? a[4 + e] : 0.f;
          }
        }
      }
    }
    team_sync();
  }
  __syncthreads();  // both teams are through: the block's sums are complete
  for (int q = tid; q < d; q += blockDim.x)
    if (gw2[q] != 0.f) atomicAdd(&g_w2[q], gw2[q]);
  if (tid == 0) {
    if (s_gb2 != 0.f) atomicAdd(g_b2, s_gb2);
    if (s_loss != 0.f) atomicAdd(loss_acc, s_loss);
  }
}

// W_1 [d][2d] -> WT[c2][j] = W_1[j][c2] (row pitch ldw): both halves transposed, the layout head_tile_kernel keeps in
// shared memory.  A warp owns four hidden units, its lanes walk the columns.
__global__ void __launch_bounds__(256) prep_head_wt_kernel(const float* __restrict__ W1, int d, int ldw, float* __restrict__ WT) {
  const int lane = threadIdx.x & 31, wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nw = (gridDim.x * blockDim.x) >> 5;
  for (int j4 = wid; j4 < (d >> 2); j4 += nw) {
    const float* w0 = W1 + (int64_t)(4 * j4) * 2 * d;
    for (int c2 = lane; c2 < 2 * d; c2 += 32) {
      float4 v;
      v.x = __ldg(w0 + c2); v.y = __ldg(w0 + 2 * d + c2); v.z = __ldg(w0 + 4 * d + c2); v.w = __ldg(w0 + 6 * d + c2);
      *reinterpret_cast<float4*>(WT + (size_t)c2 * ldw + 4 * j4) = v;
    }
  }
}

// The same head on tiles of TE events per block with register-blocked products (the form used when the model's
// width allows: d a multiple of 4 and both halves of W_1, transposed, fit in shared memory beside the tile).
// Rows of a tile: [0, TE) sources, [TE, 2TE) destinations, [2TE, 3TE) negatives; pairs: [0, TE) positive, [TE, 2TE)
// negative.  Shared memory, all c-major / j-major so that the inner loops read 16 bytes per operand:
//   WaT[c][j] = W_1[j][c], WbT[c][j] = W_1[j][d + c]   (pitch LDW)
//   HT[c][r]   embedding rows, transposed             (pitch RP = 3 TE + 4)
//   PT[j][r]   W_1a h_r (sources) or W_1b h_r         (pitch RP)
//   D1T[j][p]  d loss / d pre1, transposed            (pitch PP = 2 TE + 4)
// Hidden layer: a thread owns a 4 x 4 block of (hidden unit, row) and walks the d input columns (two 16-byte loads
// per 16 FMAs).  Input gradient: a thread owns 4 events x {positive, negative} x 4 input columns and walks the hidden
// units four at a time; it holds both pairs of its two events, so the source rows' two contributions meet in
// registers.  Everything else (scores, loss, dw_2, db_2, gate bytes) as in head_fused_kernel.
template <int TE>
struct HeadTile {
  static constexpr int ROWS = 3 * TE, PAIRS = 2 * TE, RP = ROWS + 4, PP = PAIRS + 4;
  static constexpr int THREADS = 832;   // 26 warps: the products' loops wait on shared-memory loads, and more warps hide that
  static __host__ __device__ int ldw(int d) { return (d + 3) & ~3; }
  static __host__ __device__ size_t smem_floats(int d) { return (size_t)2 * d * ldw(d) + (size_t)2 * d * RP + (size_t)d * PP + 3 * (size_t)ldw(d); }
};

template <int TE>
__global__ void __launch_bounds__(HeadTile<TE>::THREADS) head_tile_kernel(const float* __restrict__ h, const float* __restrict__ WT,
                                                                        const float* __restrict__ b1, const float* __restrict__ w2,
                                                                        const float* __restrict__ b2,
                                                                        const uint8_t* __restrict__ loss_mask, int nq, int d,
                                                                        float* __restrict__ cat1, float* __restrict__ dpre1,
                                                                        uint8_t* __restrict__ hid_gate, float* __restrict__ dpre_o,
                                                                        float* __restrict__ g_w2, float* __restrict__ g_b2,
                                                                        float* __restrict__ loss_acc, int relu_out) {
  using HT_ = HeadTile<TE>;
  constexpr int ROWS = HT_::ROWS, PAIRS = HT_::PAIRS, RP = HT_::RP, PP = HT_::PP, T = HT_::THREADS;
  extern __shared__ __align__(16) float sm[];
  __shared__ float s_msum, s_gb2, s_loss;
  const int LDW = HT_::ldw(d);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  float* WaT = sm;
  float* WbT = WaT + (size_t)d * LDW;
  float* HTs = WbT + (size_t)d * LDW;
  float* PTs = HTs + (size_t)d * RP;
  float* D1T = PTs + (size_t)d * RP;
  float* b1s = D1T + (size_t)d * PP;
  float* w2s = b1s + LDW;
  float* gw2 = w2s + LDW;
  {  // both transposed halves of W_1 (prepared once per step in this layout): a straight 16-byte copy
    const int n4 = (2 * d * LDW) >> 2;
    const float4* src = reinterpret_cast<const float4*>(WT);
    float4* dst = reinterpret_cast<float4*>(WaT);
    for (int i = tid; i < n4; i += T) dst[i] = __ldg(src + i);
  }
  for (int q = tid; q < d; q += T) { b1s[q] = b1[q]; w2s[q] = w2[q]; gw2[q] = 0.f; }
  if (tid == 0) { s_msum = 0.f; s_gb2 = 0.f; s_loss = 0.f; }
  __syncthreads();
  {  // every block counts the whole mask (a few KB)
    int c = 0;
    for (int j = tid; j < nq; j += T) c += loss_mask ? (loss_mask[j] != 0) : 1;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(FULL, c, o);
    if (lane == 0 && c) atomicAdd(&s_msum, (float)c);
  }
  __syncthreads();
  const float msum = s_msum;
  const float bias2 = b2[0];
  const int tiles = (nq + TE - 1) / TE;
  for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const int ev0 = tile * TE;
    // ---- embedding rows -> HT (transposed) and cat1 ----
    // a warp owns rows r = wid, wid + warps, ...; its lanes walk the d columns (up to eight loads per lane in flight)
    for (int r = wid; r < ROWS; r += (T >> 5)) {
      const int blk = r / TE, ev = ev0 + (r - blk * TE);   // (TE is a compile-time constant)
      const bool in = ev < nq;
      const float* src = h + ((int64_t)blk * nq + (in ? ev : 0)) * d;
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c = lane + 32 * u;
        v[u] = (in && c < d) ? __ldg(src + c) : 0.f;
      }
      float* o0 = nullptr;   // where this row goes in cat1 (sources go to two rows)
      float* o1 = nullptr;
      if (in) {
        if (blk == 0) { o0 = cat1 + (int64_t)ev * 2 * d; o1 = cat1 + (int64_t)(nq + ev) * 2 * d; }
        else if (blk == 1) o0 = cat1 + (int64_t)ev * 2 * d + d;
        else o0 = cat1 + (int64_t)(nq + ev) * 2 * d + d;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c = lane + 32 * u;
        if (c < d) {
          if (o0) o0[c] = v[u];
          if (o1) o1[c] = v[u];
          HTs[c * RP + r] = v[u];
        }
      }
    }
    __syncthreads();
    // ---- hidden layer: PT[j][r] = sum_c W[j][c] h_r[c] ----
    {
      const int ntj = d >> 2, ntr = ROWS >> 2;
      for (int t = tid; t < ntj * ntr; t += T) {
        const int tj = t % ntj, tr = t / ntj;
        const float* Wp = (4 * tr < TE ? WaT : WbT) + 4 * tj;   // (TE is a multiple of 4: a row block lies in one part)
        const float* Hp = HTs + 4 * tr;
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
        for (int c = 0; c < d; ++c) {
          const float4 wv = *reinterpret_cast<const float4*>(Wp + (size_t)c * LDW);
          const float4 hv = *reinterpret_cast<const float4*>(Hp + c * RP);
          const float wj[4] = {wv.x, wv.y, wv.z, wv.w};
          const float hr[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(wj[a], hr[b], acc[a][b]);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
          *reinterpret_cast<float4*>(PTs + (4 * tj + a) * RP + 4 * tr) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
      }
    }
    __syncthreads();
    // ---- scores, loss terms, d loss / d pre1: one warp per pair ----
    {
      float gw2r[8];   // this lane's hidden units j = lane + 32 u (d <= 256)
#pragma unroll
      for (int u = 0; u < 8; ++u) gw2r[u] = 0.f;
      for (int p = wid; p < PAIRS; p += (T >> 5)) {
        const int half = p / TE, e = p - half * TE, ev = ev0 + e;
        const bool valid = ev < nq;
        const int s_col = e, o_col = TE + TE * half + e;
        float sc = 0.f;
        for (int q = lane; q < d; q += 32) {
          const float a = fmaxf(PTs[q * RP + s_col] + PTs[q * RP + o_col] + b1s[q], 0.f);
          sc = fmaf(w2s[q], a, sc);
        }
        for (int o = 16; o > 0; o >>= 1) sc += __shfl_xor_sync(FULL, sc, o);
        sc += bias2;
        const float m = valid && (loss_mask ? (loss_mask[ev] != 0) : true) ? 1.f : 0.f;
        const float wj = msum > 0.f ? m / msum : 0.f;
        const float ds = half == 0 ? -wj * sigmoidf_(-sc) : wj * sigmoidf_(sc);
        if (lane == 0 && wj != 0.f) {
          atomicAdd(&s_loss, wj * (half == 0 ? softplusf_(-sc) : softplusf_(sc)));
          atomicAdd(&s_gb2, ds);
        }
        const int64_t row = (int64_t)half * nq + ev;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int q = lane + 32 * u;
          if (q < d) {
            const float a = fmaxf(PTs[q * RP + s_col] + PTs[q * RP + o_col] + b1s[q], 0.f);
            gw2r[u] = fmaf(ds, a, gw2r[u]);
            const float dv = a > 0.f ? ds * w2s[q] : 0.f;
            D1T[q * PP + p] = dv;
            if (valid) {
              dpre1[row * d + q] = dv;
              hid_gate[row * d + q] = a > 0.f;
            }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int q = lane + 32 * u;
        if (q < d && gw2r[u] != 0.f) atomicAdd(&gw2[q], gw2r[u]);
      }
    }
    __syncthreads();
    // ---- input gradient: dC[p][c2] = sum_j dh1[p][j] W_1[j][c2], both pairs of 2 events x 4 columns per thread ----
    {
      const int ntp = TE >> 1, ntc = (2 * d) >> 2;
      for (int t = tid; t < ntp * ntc; t += T) {
        const int tp = t % ntp, tc = t / ntp;
        const int c2 = 4 * tc;
        const bool lower = c2 < d;
        const float* Wp = lower ? WaT + (size_t)c2 * LDW : WbT + (size_t)(c2 - d) * LDW;
        const float* Dp = D1T + 2 * tp;
        float aP[2][4], aN[2][4];   // [event][column]
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) { aP[a][b] = 0.f; aN[a][b] = 0.f; }
        for (int j0 = 0; j0 < d; j0 += 4) {
          float4 w4[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) w4[i] = *reinterpret_cast<const float4*>(Wp + (size_t)i * LDW + j0);
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const float2 dp = *reinterpret_cast<const float2*>(Dp + (j0 + jj) * PP);
            const float2 dn = *reinterpret_cast<const float2*>(Dp + (j0 + jj) * PP + TE);
            const float de[2] = {dp.x, dp.y};
            const float dm[2] = {dn.x, dn.y};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float wv = jj == 0 ? w4[i].x : (jj == 1 ? w4[i].y : (jj == 2 ? w4[i].z : w4[i].w));
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                aP[e][i] = fmaf(de[e], wv, aP[e][i]);
                aN[e][i] = fmaf(dm[e], wv, aN[e][i]);
              }
            }
          }
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int el = 2 * tp + e, ev = ev0 + el;
          if (ev >= nq) continue;
          if (lower) {   // source rows collect their positive and their negative pair
            float o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              o[i] = (!relu_out || HTs[(c2 + i) * RP + el] > 0.f) ? aP[e][i] + aN[e][i] : 0.f;
            *reinterpret_cast<float4*>(dpre_o + (int64_t)ev * d + c2) = make_float4(o[0], o[1], o[2], o[3]);
          } else {
            const int cc = c2 - d;
            float o[4], n[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              o[i] = (!relu_out || HTs[(cc + i) * RP + TE + el] > 0.f) ? aP[e][i] : 0.f;
              n[i] = (!relu_out || HTs[(cc + i) * RP + 2 * TE + el] > 0.f) ? aN[e][i] : 0.f;
            }
            *reinterpret_cast<float4*>(dpre_o + ((int64_t)nq + ev) * d + cc) = make_float4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<float4*>(dpre_o + ((int64_t)2 * nq + ev) * d + cc) = make_float4(n[0], n[1], n[2], n[3]);
          }
        }
      }
    }
    __syncthreads();
  }
  for (int q = tid; q < d; q += T)
    if (gw2[q] != 0.f) atomicAdd(&g_w2[q], gw2[q]);
  if (tid == 0) {
    if (s_gb2 != 0.f) atomicAdd(g_b2, s_gb2);
    if (s_loss != 0.f) atomicAdd(loss_acc, s_loss);
  }
}

// One warp per root: backward of the weighted sum, the softmax and the scaled dot products, on the
// root's K | V rows staged in shared memory.  Lane p < H*k owns the (head, slot) pair p for the
// probability and logit gradients; afterwards the lanes own columns and write dQ and the dK | dV rows.
// SPLIT: the key/value gradient rows are written as two fp16 planes (hi, lo; row pitch ld_s, plane_s elements
// apart), multiplied by the power of two gscale so that they sit inside fp16's range, for the split products that
// consume them (which divide it out again), instead of as fp32 rows.
template <bool SPLIT>
__global__ void __launch_bounds__(256) attention_bwd_kernel(const float* __restrict__ Q, const float* __restrict__ KV,
                                                            const float* __restrict__ alpha,
                                                            const float* __restrict__ dcat_o,
                                                            const int32_t* __restrict__ cnt, int n, int d, int H, int k,
                                                            float* __restrict__ dQ, float* __restrict__ dKV,
                                                            __nv_bfloat16* __restrict__ dkv_hi, int64_t plane_s, int ld_s,
                                                            float gscale) {
  extern __shared__ __align__(16) float sm[];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int i = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (i >= n) return;
  float* Ks = sm + wib * attn_warp_floats(d, H, k);
  float* Vs = Ks + k * d;
  float* Qs = Vs + k * d;
  float* das = Qs + d;       // d loss / d a
  float* al = das + d;       // probabilities
  float* dal = al + H * k;   // d loss / d probability
  float* dl = dal + H * k;   // d loss / d logit, already scaled
  const int dh = d / H;
  const int c = max(0, min(cnt[i], k));
  const float scale = rsqrtf((float)dh);
  attn_stage_issue(Ks, Vs, Qs, Q, KV, i, c, d, k, lane);
  {
    const float* g = dcat_o + (int64_t)i * 2 * d;
    for (int e = lane; e < (d >> 2); e += 32) cp_async16(das + 4 * e, g + 4 * e);
    for (int p = lane; p < H * k; p += 32) al[p] = alpha[(int64_t)i * H * k + p];
  }
  attn_stage_wait();
  for (int p = lane; p < H * k; p += 32) {
    const int h = p / k, s = p - h * k;
    float a = 0.f;
    if (s < c) {
      const float* vr = Vs + s * d + h * dh;
      const float* gr = das + h * dh;
      for (int e = 0; e < dh; ++e) a = fmaf(gr[e], vr[e], a);
    }
    dal[p] = a;
  }
  __syncwarp();
  for (int p = lane; p < H * k; p += 32) {
    const int h = p / k, s = p - h * k;
    float g = 0.f;
    if (s < c) {
      float dot = 0.f;
      for (int t = 0; t < c; ++t) dot = fmaf(al[h * k + t], dal[h * k + t], dot);
      g = al[p] * (dal[p] - dot) * scale;
    }
    dl[p] = g;
  }
  __syncwarp();
  if (!SPLIT) {
    for (int e = lane; e < d; e += 32) {
      const int h = e / dh;
      const float qe = Qs[e], dae = das[e];
      float dq = 0.f;
      for (int s = 0; s < k; ++s) {
        float* row = dKV + ((int64_t)i * k + s) * 2 * d;
        if (s < c) {
          const float g = dl[h * k + s];
          dq = fmaf(g, Ks[s * d + e], dq);
          row[e] = g * qe;
          row[d + e] = al[h * k + s] * dae;
        } else {
          row[e] = 0.f;
          row[d + e] = 0.f;
        }
      }
      dQ[(int64_t)i * d + e] = dq;
    }
  } else {
    // a lane owns two neighbouring columns (d is even): each (hi, lo) pair goes out as one 32-bit word per plane
    for (int e = 2 * lane; e < d; e += 64) {
      const int h0 = e / dh, h1 = (e + 1) / dh;
      const float q0 = Qs[e], q1 = Qs[e + 1], a0 = das[e], a1 = das[e + 1];
      float dq0 = 0.f, dq1 = 0.f;
      for (int s = 0; s < k; ++s) {
        uint32_t* hi = reinterpret_cast<uint32_t*>(dkv_hi + ((int64_t)i * k + s) * ld_s);
        uint32_t* lo = reinterpret_cast<uint32_t*>(dkv_hi + plane_s + ((int64_t)i * k + s) * ld_s);
        uint32_t kh = 0u, kl = 0u, vh = 0u, vl = 0u;
        if (s < c) {
          const float g0 = dl[h0 * k + s], g1 = dl[h1 * k + s];
          dq0 = fmaf(g0, Ks[s * d + e], dq0);
          dq1 = fmaf(g1, Ks[s * d + e + 1], dq1);
          split_f16_pair(g0 * q0 * gscale, g1 * q1 * gscale, &kh, &kl);
          split_f16_pair(al[h0 * k + s] * a0 * gscale, al[h1 * k + s] * a1 * gscale, &vh, &vl);
        }
        hi[e >> 1] = kh; lo[e >> 1] = kl;
        hi[(d + e) >> 1] = vh; lo[(d + e) >> 1] = vl;
      }
      dQ[(int64_t)i * d + e] = dq0;
      dQ[(int64_t)i * d + e + 1] = dq1;
    }
  }
}

// The split form of the kernel above for compile-time shapes (D columns, H heads, KS slots; D / H even, H * KS <= 32,
// D <= 128).  The generic kernel is bound by instruction issue (2 800 instructions per root: loop control, scalar
// shared-memory loads, 32-bit plane stores); here the dot products read pairs of columns, a lane owns four
// neighbouring columns of the key / value gradient rows and writes them as one 64-bit word per plane and row.  Every
// sum keeps the generic kernel's order of operations.
template <int D, int H, int KS>
__global__ void __launch_bounds__(256) attention_bwd_fixed_kernel(const float* __restrict__ Q, const float* __restrict__ KV,
                                                                  const float* __restrict__ alpha,
                                                                  const float* __restrict__ dcat_o,
                                                                  const int32_t* __restrict__ cnt, int n,
                                                                  float* __restrict__ dQ, __nv_bfloat16* __restrict__ dkv_hi,
                                                                  int64_t plane_s, int ld_s, float gscale) {
  constexpr int DH = D / H, D4 = D / 4, P = H * KS;
  static_assert(D % 4 == 0 && DH % 2 == 0 && P <= 32 && D4 <= 32, "shape not covered by the fixed kernel");
  extern __shared__ __align__(16) float sm[];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int i = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
  if (i >= n) return;
  float* Ks = sm + wib * attn_warp_floats(D, H, KS);
  float* Vs = Ks + KS * D;
  float* Qs = Vs + KS * D;
  float* das = Qs + D;       // d loss / d a
  float* al = das + D;       // probabilities
  float* dal = al + P;       // d loss / d probability
  float* dl = dal + P;       // d loss / d logit, already scaled
  const int c = max(0, min(cnt[i], KS));
  const float scale = rsqrtf((float)DH);
  {
    const float* q = Q + (int64_t)i * D;
    const float* g = dcat_o + (int64_t)i * 2 * D;
    if (lane < D4) {
      cp_async16(Qs + 4 * lane, q + 4 * lane);
      cp_async16(das + 4 * lane, g + 4 * lane);
    }
    // lane l < D / 4 copies chunk l of every valid row's K half and V half: constant offsets from two pointers
    const float* kv = KV + (int64_t)i * KS * 2 * D + 4 * lane;
    float* kd = Ks + 4 * lane;
    if (lane < D4) {
#pragma unroll
      for (int t = 0; t < KS; ++t) {
        if (t < c) {
          cp_async16(kd + t * D, kv + t * 2 * D);
          cp_async16(kd + (KS + t) * D, kv + t * 2 * D + D);   // (Vs = Ks + KS * D)
        }
      }
    }
    if (lane < P) al[lane] = alpha[(int64_t)i * P + lane];
  }
  attn_stage_wait();
  const int h = lane / KS, sl = lane - h * KS;
  const bool live = lane < P && sl < c;
  float a = 0.f;
  if (live) {
    const float2* vr = reinterpret_cast<const float2*>(Vs + sl * D + h * DH);
    const float2* gr = reinterpret_cast<const float2*>(das + h * DH);
#pragma unroll
    for (int e = 0; e < DH / 2; ++e) {
      const float2 gv = gr[e], vv = vr[e];
      a = fmaf(gv.x, vv.x, a);
      a = fmaf(gv.y, vv.y, a);
    }
  }
  if (lane < P) dal[lane] = a;
  __syncwarp();
  float gl = 0.f;
  if (live) {
    float dot = 0.f;
#pragma unroll
    for (int t = 0; t < KS; ++t)
      if (t < c) dot = fmaf(al[h * KS + t], dal[h * KS + t], dot);
    gl = al[lane] * (a - dot) * scale;
  }
  if (lane < P) dl[lane] = gl;
  __syncwarp();
  if (lane < D4) {
    const int h0 = (4 * lane) / DH, h1 = (4 * lane + 2) / DH;   // columns 4l, 4l+1 share a head, and so do 4l+2, 4l+3
    const float4 q4 = *reinterpret_cast<const float4*>(Qs + 4 * lane);
    const float4 a4 = *reinterpret_cast<const float4*>(das + 4 * lane);
    float4 dq = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int t = 0; t < KS; ++t) {
      __nv_bfloat16* hi_row = dkv_hi + ((int64_t)i * KS + t) * ld_s + 4 * lane;
      __nv_bfloat16* lo_row = hi_row + plane_s;
      uint2 kh = make_uint2(0u, 0u), kl = kh, vh = kh, vl = kh;
      if (t < c) {
        const float g0 = dl[h0 * KS + t], g1 = dl[h1 * KS + t];
        const float p0 = al[h0 * KS + t], p1 = al[h1 * KS + t];
        const float4 kv4 = *reinterpret_cast<const float4*>(Ks + t * D + 4 * lane);
        dq.x = fmaf(g0, kv4.x, dq.x); dq.y = fmaf(g0, kv4.y, dq.y);
        dq.z = fmaf(g1, kv4.z, dq.z); dq.w = fmaf(g1, kv4.w, dq.w);
        split_f16_pair(g0 * q4.x * gscale, g0 * q4.y * gscale, &kh.x, &kl.x);
        split_f16_pair(g1 * q4.z * gscale, g1 * q4.w * gscale, &kh.y, &kl.y);
        split_f16_pair(p0 * a4.x * gscale, p0 * a4.y * gscale, &vh.x, &vl.x);
        split_f16_pair(p1 * a4.z * gscale, p1 * a4.w * gscale, &vh.y, &vl.y);
      }
      *reinterpret_cast<uint2*>(hi_row) = kh;
      *reinterpret_cast<uint2*>(lo_row) = kl;
      *reinterpret_cast<uint2*>(hi_row + D) = vh;
      *reinterpret_cast<uint2*>(lo_row + D) = vl;
    }
    *reinterpret_cast<float4*>(dQ + (int64_t)i * D + 4 * lane) = dq;
  }
}

// Gradient rows flowing into memory rows that the last memory update wrote: one warp per
// source row, added into dMemU[node2slot[node]].  Rows [0, nb_rows): dZm with node = nbr;
// rows [nb_rows, nb_rows + n): the root's own row, dcat_o[:, d:] + dzq[:, :d].
__global__ void __launch_bounds__(256) scatter_dmem_kernel(const float* __restrict__ dZm, const float* __restrict__ dcat_o,
                                                           const float* __restrict__ dzq,
                                                           const int32_t* __restrict__ nbr,
                                                           const int32_t* __restrict__ nodes, int n, int k, int d,
                                                           const int32_t* __restrict__ node2slot,
                                                           float* __restrict__ dMemU, int64_t N) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int nb_rows = n * k;
  const int d4 = d >> 2;  // <= 64: at most two 16-byte pieces per lane
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < nb_rows + n; r += warps) {
    // the row's gradient is requested before it is known whether its node was updated (most were not):
    // the index chain node -> slot and the row loads overlap
    const bool isn = r < nb_rows;
    const int i = r - nb_rows;
    float4 g[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int q4 = lane + 32 * u;
      g[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (q4 < d4) {
        if (isn) {
          g[u] = __ldg(reinterpret_cast<const float4*>(dZm + (int64_t)r * 2 * d) + q4);  // memory half of the row
        } else {
          const float4 a = __ldg(reinterpret_cast<const float4*>(dcat_o + (int64_t)i * 2 * d + d) + q4);
          const float4 b = __ldg(reinterpret_cast<const float4*>(dzq + (int64_t)i * 2 * d) + q4);
          g[u] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
        }
      }
    }
    const int node = isn ? nbr[r] : nodes[i];
    if (node < 0 || node >= N) continue;   // (an id beyond the graph was reported by the forward pass)
    const int slot = node2slot[node];
    if (slot < 0) continue;
    float4* out = reinterpret_cast<float4*>(dMemU + (int64_t)slot * d);
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int q4 = lane + 32 * u;
      if (q4 < d4) atomicAdd(out + q4, g[u]);
    }
  }
}

// The same scatter for batches in which many rows hit few nodes (hub nodes: tens of thousands of rows onto one
// updated row serialise on its atomics).  A block takes SC_ROWS consecutive rows.  One thread per row first
// resolves row -> node -> slot and files the row under one of SC_WAYS lists (a list belongs to the first slot that
// claims it by compare-and-swap; a row whose list belongs to another slot goes to a list of singles).  The lists
// are then laid end to end, so that rows of one slot are neighbours, and every warp walks an equal share of that
// sequence, 6 / U row loads in flight: it sums in registers while the slot stays the same and adds the sum to
// dMemU when it changes.  Rows whose node was not updated are never read.
constexpr int SC_ROWS = 256, SC_WAYS = 32;  // 256 rows, 256 threads: the whole batch is one wave of blocks
template <int U>  // 16-byte pieces of a row per lane: 1 (d <= 128) or 2
__global__ void __launch_bounds__(256, 5) scatter_dmem_cached_kernel(const float* __restrict__ dZm,
                                                                     const float* __restrict__ dcat_o,
                                                                     const float* __restrict__ dzq,
                                                                     const int32_t* __restrict__ nbr,
                                                                     const int32_t* __restrict__ nodes, int n, int k, int d,
                                                                     const int32_t* __restrict__ node2slot,
                                                                     float* __restrict__ dMemU, int64_t N) {
  static_assert(SC_WAYS == 32, "one lane per list in the offset scan");
  static_assert(SC_ROWS == 256, "one thread per row, row numbers kept in a byte");
  __shared__ int s_id[SC_WAYS], s_cnt[SC_WAYS + 1], s_off[SC_WAYS + 1], s_slot[SC_ROWS];
  __shared__ unsigned char s_seq[SC_ROWS];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int nb_rows = n * k, total = nb_rows + n;
  const int d4 = d >> 2;  // <= 32 U
  const int r_base = blockIdx.x * SC_ROWS;
  if (threadIdx.x < SC_WAYS) s_id[threadIdx.x] = -1;
  if (threadIdx.x <= SC_WAYS) s_cnt[threadIdx.x] = 0;  // (entry SC_WAYS: the singles)
  __syncthreads();
  int way = -1, pos = 0;
  if (r_base + threadIdx.x < total) {
    const int r = r_base + threadIdx.x;
    const int node = r < nb_rows ? nbr[r] : nodes[r - nb_rows];
    int slot = -1;
    if (node >= 0 && node < N) slot = node2slot[node];  // (an id beyond the graph was reported by the forward pass)
    s_slot[threadIdx.x] = slot;
    if (slot >= 0) {
      way = slot % SC_WAYS;
      const int owner = atomicCAS(&s_id[way], -1, slot);
      if (owner != -1 && owner != slot) way = SC_WAYS;
      pos = atomicAdd(&s_cnt[way], 1);
    }
  }
  __syncthreads();
  if (wid == 0) {  // exclusive scan of the list lengths
    const int c = s_cnt[lane];
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(FULL, incl, o);
      if (lane >= o) incl += t;
    }
    s_off[lane] = incl - c;
    if (lane == 31) s_off[SC_WAYS] = incl;
  }
  __syncthreads();
  if (way >= 0) s_seq[s_off[way] + pos] = (unsigned char)threadIdx.x;
  __syncthreads();
  const int n_live = s_off[SC_WAYS] + s_cnt[SC_WAYS];
  const int share = (n_live + 7) >> 3;
  const int e_end = min(n_live, (wid + 1) * share);
  constexpr int V = 6 / U;  // (48 registers: five blocks share an SM, or fewer beside a persistent product)
  int cur = -1;
  float4 acc[U];
#pragma unroll
  for (int u = 0; u < U; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  auto flush = [&]() {
    if (cur < 0) return;
    float4* out = reinterpret_cast<float4*>(dMemU + (int64_t)cur * d);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int q4 = lane + 32 * u;
      if (q4 < d4) atomicAdd(out + q4, acc[u]);
      acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  for (int e = wid * share; e < e_end; e += V) {
    float4 g[V][U];
    int t[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
      t[v] = e + v < e_end ? (int)s_seq[e + v] : -1;
      if (t[v] < 0) continue;
      const int r = r_base + t[v];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int q4 = lane + 32 * u;
        g[v][u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q4 < d4) {
          if (r < nb_rows) {
            g[v][u] = __ldg(reinterpret_cast<const float4*>(dZm + (int64_t)r * 2 * d) + q4);  // memory half of the row
          } else {
            const int i = r - nb_rows;
            const float4 a = __ldg(reinterpret_cast<const float4*>(dcat_o + (int64_t)i * 2 * d + d) + q4);
            const float4 b = __ldg(reinterpret_cast<const float4*>(dzq + (int64_t)i * 2 * d) + q4);
            g[v][u] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
          }
        }
      }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
      if (t[v] < 0) continue;  // (uniform over the warp)
      const int slot = s_slot[t[v]];
      if (slot != cur) { flush(); cur = slot; }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        acc[u].x += g[v][u].x; acc[u].y += g[v][u].y; acc[u].z += g[v][u].z; acc[u].w += g[v][u].w;
      }
    }
  }
  flush();
}

// Time-encoder gradient: G[r, col0 + c] is d loss / d Phi(dt_r)_c and S[r, c] = sin(arg) was kept by
// the forward pass (S == nullptr: every row has dt = 0, sin(arg) = sin(b_c)).
//   dw_c += -S dt_r G,   db_c += -S G
// The terms are large (dt reaches the time span of the stream) and cancel, so they are summed in
// fp64.  Block = 8 warps over rows_per_block rows; lanes own columns c = lane + 32 j; the warps' partial sums
// meet in shared memory and leave as one pair of fp64 atomics per block and column into acc[0:d]
// (dw) and acc[d:2d] (db).  Dynamic shared memory: 8 * 2 * d doubles.
constexpr int TG_MAXJ = 8;
// Rows per block: every block ends with one fp64 atomic per column onto the same 2d addresses, and those
// serialise, so the grid is kept to about two blocks per SM, as many as fit at once (rows per block a multiple
// of the 8 warps); inside a block each warp walks its rows three at a time so that their loads overlap.
constexpr int TG_U = 3;   // rows a warp has in flight (four spill at the 128 registers that let two blocks share an SM)
inline int tg_rows_per_block(int rows) {
  const int r = (rows + 295) / 296;
  return r < 8 ? 8 : (r + 7) / 8 * 8;
}
template <int V>  // 16-byte column pieces per lane: 1 (d <= 128: half the registers, four blocks share an SM) or 2
__global__ void __launch_bounds__(256, V == 1 ? 4 : 2) time_grad_kernel(const float* __restrict__ G, int64_t ldg, int col0,
                                                        const float* __restrict__ S, const float* __restrict__ dt,
                                                        int rows, const int32_t* __restrict__ dev_rows, int d,
                                                        const float* __restrict__ time_w,
                                                        const float* __restrict__ time_b, double* __restrict__ acc,
                                                        int rows_per_block) {
  extern __shared__ double s_part[];  // [8][2][d]
  const int R = dev_rows ? min(*dev_rows, rows) : rows;
  const int r0 = blockIdx.x * rows_per_block, r1 = min(R, r0 + rows_per_block);
  if (r0 >= r1) return;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  // a lane owns columns 4 (lane + 32 v) .. + 3, v < V (d <= 128 V): 128-bit loads of G and S (d, ldg and col0 are
  // multiples of 4 and the rows 16-byte aligned)
  // Sines: saved rows S; or (S null, dt given) recomputed from the row's dt exactly as the forward pass formed
  // them -- a row with dt < 0 is an empty slot and contributes nothing; or (both null) the constant sin(b) of dt = 0.
  double gw[V][4], gb[V][4];
  float4 sb[V], wv[V], bv[V];
  const bool recompute = S == nullptr && dt != nullptr;
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const int c = 4 * (lane + 32 * v);
#pragma unroll
    for (int e = 0; e < 4; ++e) { gw[v][e] = 0.0; gb[v][e] = 0.0; }
    sb[v] = wv[v] = bv[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (S == nullptr && c < d) {
      bv[v] = make_float4(time_b[c], time_b[c + 1], time_b[c + 2], time_b[c + 3]);
      if (recompute) wv[v] = make_float4(time_w[c], time_w[c + 1], time_w[c + 2], time_w[c + 3]);
      else sb[v] = make_float4(sinf(bv[v].x), sinf(bv[v].y), sinf(bv[v].z), sinf(bv[v].w));
    }
  }
  for (int rb = r0 + wid; rb < r1; rb += 8 * TG_U) {  // rows rb, rb + 8, ...: loads first, sums after
    float4 g[TG_U][V], sn[TG_U][V];
    float dtr[TG_U];
#pragma unroll
    for (int u = 0; u < TG_U; ++u) {
      const int r = rb + 8 * u;
      const bool in = r < r1;
      dtr[u] = (in && dt) ? dt[r] : 0.f;
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const int c = 4 * (lane + 32 * v);
        const bool ok = in && c < d;
        g[u][v] = ok ? __ldg(reinterpret_cast<const float4*>(G + (int64_t)r * ldg + col0 + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
        sn[u][v] = ok ? (S ? __ldg(reinterpret_cast<const float4*>(S + (int64_t)r * d + c)) : sb[v]) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (recompute) {
#pragma unroll
      for (int u = 0; u < TG_U; ++u) {
        const bool live = rb + 8 * u < r1 && dtr[u] >= 0.f;
#pragma unroll
        for (int v = 0; v < V; ++v) {
          const int c = 4 * (lane + 32 * v);
          float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
          if (live && c < d) {
            q.x = __sinf(reduce_two_pi(time_arg(wv[v].x, bv[v].x, dtr[u])));
            q.y = __sinf(reduce_two_pi(time_arg(wv[v].y, bv[v].y, dtr[u])));
            q.z = __sinf(reduce_two_pi(time_arg(wv[v].z, bv[v].z, dtr[u])));
            q.w = __sinf(reduce_two_pi(time_arg(wv[v].w, bv[v].w, dtr[u])));
          }
          sn[u][v] = q;
        }
        if (!live) dtr[u] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < TG_U; ++u) {
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const float ge[4] = {g[u][v].x, g[u][v].y, g[u][v].z, g[u][v].w};
        const float se[4] = {sn[u][v].x, sn[u][v].y, sn[u][v].z, sn[u][v].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const double t = -(double)se[e] * (double)ge[e];
          gw[v][e] = fma(t, (double)dtr[u], gw[v][e]);
          gb[v][e] += t;
        }
      }
    }
  }
#pragma unroll
  for (int v = 0; v < V; ++v) {
    const int c = 4 * (lane + 32 * v);
    if (c < d) {
#pragma unroll
      for (int e = 0; e < 4; ++e) { s_part[(wid * 2 + 0) * d + c + e] = gw[v][e]; s_part[(wid * 2 + 1) * d + c + e] = gb[v][e]; }
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 2 * d; e += blockDim.x) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += s_part[w * 2 * d + e];
    if (t != 0.0) atomicAdd(&acc[e], t);
  }
}

inline void time_grad_launch(int grid, size_t smem, cudaStream_t st, const float* G, int64_t ldg, int col0, const float* S,
                             const float* dt, int rows, const int32_t* dev_rows, int d, const float* time_w,
                             const float* time_b, double* acc, int rows_per_block) {
  if (d <= 128)
    time_grad_kernel<1><<<grid, 256, smem, st>>>(G, ldg, col0, S, dt, rows, dev_rows, d, time_w, time_b, acc, rows_per_block);
  else
    time_grad_kernel<2><<<grid, 256, smem, st>>>(G, ldg, col0, S, dt, rows, dev_rows, d, time_w, time_b, acc, rows_per_block);
}

// Backward of the time-projected embedding h = m * (1 + dt w_p + b_p), one warp per root:
//   dw_p += dh m dt,  db_p += dh m   (fp64 block sums, then one pair of fp64 atomics per block and column into
//                                     acc[0:d] and acc[d:2d]: dt spans the stream and the terms cancel)
//   dm = dh (1 + dt w_p + b_p) is added to the row's slot of dMemU when the node's memory row was written
//   by this step's update (all other table rows are constants).
// Dynamic shared memory: 8 * 2 * d doubles.
__global__ void __launch_bounds__(256) jodie_embed_bwd_kernel(const float* __restrict__ dh, const float* __restrict__ memory,
                                                              const double* __restrict__ last_update,
                                                              const float* __restrict__ proj_w,
                                                              const float* __restrict__ proj_b,
                                                              const int32_t* __restrict__ nodes,
                                                              const double* __restrict__ times, int n, int d,
                                                              const int32_t* __restrict__ node2slot, int have_update,
                                                              float* __restrict__ dMemU, double* __restrict__ acc, int64_t N) {
  extern __shared__ double s_part[];  // [8][2][d]
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  double gw[TG_MAXJ], gb[TG_MAXJ];
#pragma unroll
  for (int j = 0; j < TG_MAXJ; ++j) { gw[j] = 0.0; gb[j] = 0.0; }
  const int warps = (gridDim.x * blockDim.x) >> 5;
  for (int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps) {
    const int node = nodes[i];
    if (node < 0 || node >= N) continue;   // reported by the forward pass; its embedding was zero
    const float dt = (float)(times[i] - last_update[node]);
    const int slot = have_update ? node2slot[node] : -1;
#pragma unroll
    for (int j = 0; j < TG_MAXJ; ++j) {
      const int c = lane + 32 * j;
      if (c < d) {
        const float g = dh[(int64_t)i * d + c];
        const float m = memory[(int64_t)node * d + c];
        const double t = (double)g * (double)m;
        gw[j] = fma(t, (double)dt, gw[j]);
        gb[j] += t;
        if (slot >= 0) atomicAdd(&dMemU[(int64_t)slot * d + c], g * (1.f + fmaf(dt, proj_w[c], proj_b[c])));
      }
    }
  }
#pragma unroll
  for (int j = 0; j < TG_MAXJ; ++j) {
    const int c = lane + 32 * j;
    if (c < d) { s_part[(wid * 2 + 0) * d + c] = gw[j]; s_part[(wid * 2 + 1) * d + c] = gb[j]; }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 2 * d; e += blockDim.x) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += s_part[w * 2 * d + e];
    if (t != 0.0) atomicAdd(&acc[e], t);
  }
}

// Backward of the plain recurrent cell for the rows the memory update wrote: d pre = dm' (1 - m'^2).
__global__ void __launch_bounds__(256) rnn_bwd_gate_kernel(const float* __restrict__ dMemU, const float* __restrict__ g_n,
                                                           const int32_t* __restrict__ n_uniq, int u_cap, int d,
                                                           float* __restrict__ dG) {
  const int U = min(*n_uniq, u_cap);
  const int64_t total = (int64_t)U * d;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const float m = g_n[e];
    dG[e] = dMemU[e] * (1.f - m * m);
  }
}

// Backward of the GRU gates for the rows the memory update wrote.
__global__ void __launch_bounds__(256) gru_bwd_gate_kernel(const float* __restrict__ dMemU, const float* __restrict__ X,
                                                           int ld, int d, const float* __restrict__ g_r,
                                                           const float* __restrict__ g_z, const float* __restrict__ g_n,
                                                           const float* __restrict__ g_hn,
                                                           const int32_t* __restrict__ n_uniq, int u_cap,
                                                           float* __restrict__ dGi, float* __restrict__ dGh) {
  const int U = min(*n_uniq, u_cap);
  const int64_t total = (int64_t)U * d;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int u = (int)(e / d), q = (int)(e % d);
    const float g = dMemU[e];
    const float r = g_r[e], z = g_z[e], nn = g_n[e];
    const float h = X[(int64_t)u * ld + q];
    const float dn = g * (1.f - z);
    const float dz = g * (h - nn);
    const float dpn = dn * (1.f - nn * nn);
    const float dpz = dz * z * (1.f - z);
    const float dpr = dpn * g_hn[e] * r * (1.f - r);
    float* gi = dGi + (int64_t)u * 3 * d;
    float* gh = dGh + (int64_t)u * 3 * d;
    gi[q] = dpr; gi[d + q] = dpz; gi[2 * d + q] = dpn;
    gh[q] = dpr; gh[d + q] = dpz; gh[2 * d + q] = dpn * r;
  }
}

// Gradient norm g_r and the Adam update in one pass over the parameters.  Adam does not depend on the
// norm (no clipping), so each thread squares its gradient entries into the block's partial sum and
// updates the same entries; the last block to finish turns the sum into g_r and bumps the step counter
// (every block has read the counter before it takes its ticket).
// The time-encoder entries [t_off, t_off + t_n) and the time projection's [p_off, p_off + p_n) are taken
// from their fp64 sums tg_acc (rounded once) and written into grads, where the debug export finds them.
// apply = 0 stops after the gradient and its norm (parameters, moments and the step counter stay): the
// caller synchronises the gradient across workers and comes back with t_n = p_n = 0 and gscale = 1 / workers;
// a gscale other than 1 multiplies every gradient entry first and stores the product.
__global__ void __launch_bounds__(256) gradnorm_adam_kernel(float* __restrict__ grads, int64_t P,
                                                            const double* __restrict__ tg_acc, int64_t t_off, int t_n,
                                                            int64_t p_off, int p_n, double* red, unsigned int* ticket, int64_t* step,
                                                            float* __restrict__ p, float* __restrict__ m,
                                                            float* __restrict__ v, float lr, float beta1, float beta2,
                                                            float eps, const float* __restrict__ loss_acc, float* scalars,
                                                            float* loss_out, float* gradnorm_out, float gscale, int apply) {
  __shared__ double s_part[8];
  __shared__ float s_c1, s_c2;
  if (threadIdx.x == 0) {
    const double t = (double)(step[0] + 1);
    s_c1 = (float)(1.0 / (1.0 - pow((double)beta1, t)));
    s_c2 = (float)(1.0 / (1.0 - pow((double)beta2, t)));
  }
  __syncthreads();
  const float c1 = s_c1, c2 = s_c2;
  // 1 - beta formed in fp64 from the configured fp32 value, then rounded once
  const float omb1 = (float)(1.0 - (double)beta1), omb2 = (float)(1.0 - (double)beta2);
  double acc = 0.0;
  // one parameter: gradient (from the fp64 sums where those exist), sum of squares, Adam
  auto one = [&](int64_t e, float ge, float& pe, float& me, float& ve) {
    acc = fma((double)ge, (double)ge, acc);
    if (!apply) return;
    me = fmaf(beta1, me, omb1 * ge);
    ve = fmaf(beta2, ve, omb2 * ge * ge);
    pe -= lr * (me * c1) / (sqrtf(ve * c2) + eps);
  };
  // groups of four consecutive parameters with 128-bit accesses (the arrays are 16-byte aligned; the ranges
  // taken from the fp64 sums start and end on multiples of four because d is one), then the last P % 4
  const bool vec = ((((uintptr_t)grads | (uintptr_t)p | (uintptr_t)m | (uintptr_t)v) & 15) == 0) && (t_off % 4 == 0) &&
                   (t_n % 4 == 0) && (p_off % 4 == 0) && (p_n % 4 == 0);
  const int64_t P4 = vec ? P / 4 : 0;
  for (int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; q < P4; q += (int64_t)gridDim.x * blockDim.x) {
    const int64_t e = 4 * q;
    float4 g4;
    if (e >= t_off && e < t_off + t_n) {
      const double* a = tg_acc + (e - t_off);
      g4 = make_float4((float)a[0], (float)a[1], (float)a[2], (float)a[3]);
      reinterpret_cast<float4*>(grads)[q] = g4;
    } else if (e >= p_off && e < p_off + p_n) {  // the projection's w_p | b_p, summed in fp64 behind the time encoder's
      const double* a = tg_acc + t_n + (e - p_off);
      g4 = make_float4((float)a[0], (float)a[1], (float)a[2], (float)a[3]);
      reinterpret_cast<float4*>(grads)[q] = g4;
    } else {
      g4 = reinterpret_cast<const float4*>(grads)[q];
    }
    if (gscale != 1.f) {
      g4 = make_float4(g4.x * gscale, g4.y * gscale, g4.z * gscale, g4.w * gscale);
      reinterpret_cast<float4*>(grads)[q] = g4;
    }
    float4 p4 = make_float4(0.f, 0.f, 0.f, 0.f), m4 = p4, v4 = p4;
    if (apply) { p4 = reinterpret_cast<float4*>(p)[q]; m4 = reinterpret_cast<float4*>(m)[q]; v4 = reinterpret_cast<float4*>(v)[q]; }
    one(e, g4.x, p4.x, m4.x, v4.x);
    one(e + 1, g4.y, p4.y, m4.y, v4.y);
    one(e + 2, g4.z, p4.z, m4.z, v4.z);
    one(e + 3, g4.w, p4.w, m4.w, v4.w);
    if (apply) {
      reinterpret_cast<float4*>(p)[q] = p4;
      reinterpret_cast<float4*>(m)[q] = m4;
      reinterpret_cast<float4*>(v)[q] = v4;
    }
  }
  for (int64_t e = 4 * P4 + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < P; e += (int64_t)gridDim.x * blockDim.x) {
    float ge;
    if (e >= t_off && e < t_off + t_n) {
      ge = (float)tg_acc[e - t_off];
      grads[e] = ge;
    } else if (e >= p_off && e < p_off + p_n) {
      ge = (float)tg_acc[t_n + (e - p_off)];
      grads[e] = ge;
    } else {
      ge = grads[e];
    }
    if (gscale != 1.f) {
      ge *= gscale;
      grads[e] = ge;
    }
    float pe = 0.f, me = 0.f, ve = 0.f;
    if (apply) { pe = p[e]; me = m[e]; ve = v[e]; }
    one(e, ge, pe, me, ve);
    if (apply) { p[e] = pe; m[e] = me; v[e] = ve; }
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(FULL, acc, o);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double b = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) b += s_part[w];
    atomicAdd(&red[0], b);
    __threadfence();
    const unsigned int done = atomicAdd(ticket, 1u);
    if (done == gridDim.x - 1) {
      __threadfence();
      const double ss = atomicAdd(&red[0], 0.0);
      const float gn = (float)sqrt(ss);
      if (apply) step[0] = step[0] + 1;
      const float loss = *loss_acc;
      scalars[0] = loss;
      scalars[1] = gn;
      if (loss_out) *loss_out = loss;
      if (gradnorm_out) *gradnorm_out = gn;
      *ticket = 0u;
    }
  }
}

__global__ void gate_bytes_kernel(const float* __restrict__ h, int64_t n, uint8_t* __restrict__ out) {
  const int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (e < n) out[e] = h[e] > 0.f;
}

int pick_split(int M, int N, int K) {
  const int tiles = ((M + 63) / 64) * ((N + 63) / 64);
  int s = (4 * 148 + tiles - 1) / tiles;
  const int max_s = (K + 127) / 128;
  if (s > max_s) s = max_s;
  return s < 1 ? 1 : s;
}

// dW[N_out, K_in] += dY^T A  (+ db[N_out] += column sums of dY): a transposed product with the
// contraction over rows (optionally a device-side count).
int grad_w(tgnn_ctx* ctx, const float* dY, int64_t ld_dy, const float* A, int64_t ld_a, int rows, const int32_t* dev_rows,
           int n_out, int k_in, float* dW, float* db, const char* name, cudaStream_t s) {
  GemmArgs g = {};
  g.A = dY; g.a_rs = 1; g.a_cs = ld_dy;  // A(m,k) = dY[k, m]
  g.B = A; g.b_rs = ld_a; g.b_cs = 1;    // B(k,n) = A[k, n]
  g.C = dW; g.ldc = k_in; g.M = n_out; g.N = k_in; g.K = rows; g.dev_K = dev_rows;
  g.rowsum_out = db; g.accumulate = 1; g.split_k = pick_split(n_out, k_in, rows); g.precise = 1;
  g.tail_slack = 1;  // dY and the saved activations are workspace buffers
  return launch_gemm(ctx, g, name, s);
}

// dA[rows, n_cols] = dY[rows, n_out] W[:, col0 : col0 + n_cols]   (W is [n_out, ld_w] row-major)
int grad_in(tgnn_ctx* ctx, const float* dY, int64_t ld_dy, const float* W, int64_t ld_w, int col0, int rows,
            const int32_t* dev_rows, int n_out, int n_cols, float* dA, int64_t ld_da, const char* name, cudaStream_t s,
            int site = 0) {
  GemmArgs g = {};
  g.A = dY; g.a_rs = ld_dy; g.a_cs = 1;
  g.B = W + col0; g.b_rs = ld_w; g.b_cs = 1;
  g.C = dA; g.ldc = ld_da; g.M = rows; g.N = n_cols; g.K = n_out; g.dev_M = dev_rows; g.split_k = 1; g.precise = 1;
  g.site = site;
  return launch_gemm(ctx, g, name, s);
}

}  // namespace

int launch_prep_head(tgnn_ctx* ctx, cudaStream_t s) {
  const int d = ctx->cfg.d;
  if (d % 4 != 0 || d > 256) return TGNN_OK;   // (the tile head is not used for such widths)
  {
    KernelScope scope__(ctx, "prep_head", s);
    prep_head_wt_kernel<<<(d / 4 + 7) / 8, 256, 0, s>>>(ctx->params + ctx->L.w1, d, (d + 3) / 4 * 4, ctx->ws.head_wT);
  }
  TGNN_LAUNCH_OK(ctx, "prep_head");
  return TGNN_OK;
}

int launch_get_gates(tgnn_ctx* ctx, uint8_t* h_gate_out, uint8_t* hid_gate_out, cudaStream_t s) {
  const int64_t n = (int64_t)ctx->e_n * ctx->cfg.d;
  if (n > 0) {
    gate_bytes_kernel<<<(int)((n + 255) / 256), 256, 0, s>>>(ctx->e_h, n, h_gate_out);
    TGNN_LAUNCH_OK(ctx, "gate_bytes");
    const size_t m = (size_t)2 * (ctx->e_n / 3) * ctx->cfg.d;
    TGNN_CUDA_OK(ctx, cudaMemcpyAsync(hid_gate_out, ctx->ws.hid_gate, m, cudaMemcpyDeviceToDevice, s));
  }
  return TGNN_OK;
}

// G[wk + r * dkv + c] += pad[r * ld + c] for c < dkv, G[bk + r] += pad[r * ld + dkv]: the weight gradient of the
// key/value projection is accumulated in a copy with 16-byte aligned rows (vector atomics from every contraction
// split instead of four scalar ones) and folded into the flat gradient once.
__global__ void __launch_bounds__(256) fold_dwkv_kernel(const float* __restrict__ pad, int ld, int rows, int dkv,
                                                        float* __restrict__ g_w, float* __restrict__ g_b) {
  const int total = rows * (dkv + 1);
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
    const int r = e / (dkv + 1), c = e - r * (dkv + 1);
    const float v = pad[(int64_t)r * ld + c];
    if (c < dkv) g_w[(int64_t)r * dkv + c] += v;
    else g_b[r] += v;
  }
}

#define RC(x)            \
  do {                   \
    int rc__ = (x);      \
    if (rc__) return rc__; \
  } while (0)

int launch_backward(tgnn_ctx* ctx, int n_q, const uint8_t* loss_mask, float* loss_out, float* gradnorm_out,
                    cudaStream_t s) {
  const tgnn_config& c = ctx->cfg;
  const ParamLayout& L = ctx->L;
  Workspace& w = ctx->ws;
  const int d = c.d, k = c.k, H = c.heads, de = c.d_e;
  const int R = 3 * n_q, NB = R * k;
  float* P = ctx->params;
  float* G = w.grads;
  // The chain loss -> head -> output projection -> attention -> inputs -> memory rows -> GRU is
  // sequential and stays on the caller's stream s.  Weight-gradient products and time-encoder sums
  // are leaves of that chain: they go to the two side streams as soon as their operands exist and
  // are joined back before the gradient norm.
  cudaStream_t sa = ctx->side[0], sb = ctx->side[1], sc = ctx->side[2], sd = ctx->side[3];
  // grads | dMemU | red | tg_acc | st_scalars are contiguous in the arena: one memset clears them all
  if (!ctx->grads_zeroed) {
    const size_t zero_bytes = (size_t)((char*)(w.st_scalars + 4) - (char*)w.grads);
    TGNN_CUDA_OK(ctx, cudaMemsetAsync(w.grads, 0, zero_bytes, s));
  }

  if (n_q > 0) {
    // One block does the head forward and backward for 4 events at a time when W_1 fits in shared memory
    // beside the staging rows; wider models take the projections through the GEMM path instead.
    const int relu_out = c.model == TGNN_MODEL_TGN ? 1 : 0;
    const size_t hf_smem = head_fused_smem(d);
    // Large batches: tiles of TE events per block with register-blocked products (from 2 400 events up; below that
    // the groups of four of head_fused_kernel spread over more SMs and are faster).  TE is the tile size whose
    // rounds of 148 blocks cost least: 4 000 events are 143 tiles of 28 -- one round on 143 SMs -- where tiles of 32
    // would leave 23 SMs idle for a longer round.
    const size_t ht32 = HeadTile<32>::smem_floats(d) * sizeof(float);
    if (d % 4 == 0 && d <= 256 && ht32 <= 225 * 1024 && n_q >= 32 * 74) {
      int te = 32, best = 1 << 30;
      for (int cand = 32; cand >= 20; cand -= 4) {
        const int tiles = (n_q + cand - 1) / cand, cost = ((tiles + 147) / 148) * cand;
        if (cost < best) { best = cost; te = cand; }
      }
      const int tiles = (n_q + te - 1) / te;
      const int grid = tiles < 148 ? tiles : 148;
      // W_1 transposed: written with the weight images at the start of the step; otherwise (fp32 mode, or the
      // backward step called on its own after the parameters changed) here
      if (!(ctx->images != nullptr && ctx->images_fresh)) RC(launch_prep_head(ctx, s));
      {
        KernelScope scope__(ctx, "head_fused", s);
#define TGNN_HEAD_TILE(TE_)                                                                                              \
  do {                                                                                                                   \
    static SmemLimit lim__;                                                                                              \
    const size_t bytes__ = HeadTile<TE_>::smem_floats(d) * sizeof(float);                                                \
    RC(raise_smem_limit(ctx, head_tile_kernel<TE_>, (int)bytes__, lim__));                                               \
    head_tile_kernel<TE_><<<grid, HeadTile<TE_>::THREADS, bytes__, s>>>(                                                 \
        ctx->e_h, w.head_wT, P + L.b1, P + L.w2, P + L.b2, loss_mask, n_q, d, w.cat1, w.hid1, w.hid_gate, w.dpre_o,      \
        G + L.w2, G + L.b2, w.st_scalars, relu_out);                                                                    \
  } while (0)
        if (te == 32) TGNN_HEAD_TILE(32);
        else if (te == 28) TGNN_HEAD_TILE(28);
        else if (te == 24) TGNN_HEAD_TILE(24);
        else TGNN_HEAD_TILE(20);
#undef TGNN_HEAD_TILE
      }
      TGNN_LAUNCH_OK(ctx, "head_fused");
      RC(fork_to(ctx, s, sa));
      RC(grad_w(ctx, w.hid1, d, w.cat1, 2 * d, 2 * n_q, nullptr, d, 2 * d, G + L.w1, G + L.b1, "dW_1", sa));
    } else if (hf_smem <= 200 * 1024) {
      static SmemLimit hf_limit;
      RC(raise_smem_limit(ctx, head_fused_kernel, (int)hf_smem, hf_limit));
      const int groups = (n_q + HF_EV - 1) / HF_EV;
      {
        KernelScope scope__(ctx, "head_fused", s);
        // two groups per block side by side; at most one block per SM
        head_fused_kernel<<<(groups + HF_TEAMS - 1) / HF_TEAMS < 148 ? (groups + HF_TEAMS - 1) / HF_TEAMS : 148, HF_THREADS, hf_smem, s>>>(
            ctx->e_h, P + L.w1, P + L.b1, P + L.w2, P + L.b2, loss_mask, n_q, d, w.cat1, w.hid1, w.hid_gate, w.dpre_o,
            G + L.w2, G + L.b2, w.st_scalars, relu_out);
      }
      TGNN_LAUNCH_OK(ctx, "head_fused");
      RC(fork_to(ctx, s, sa));
      RC(grad_w(ctx, w.hid1, d, w.cat1, 2 * d, 2 * n_q, nullptr, d, 2 * d, G + L.w1, G + L.b1, "dW_1", sa));
    } else {
      const int64_t tot = (int64_t)2 * n_q * 2 * d;
      {
        KernelScope scope__(ctx, "head_gather", s);
        head_gather_kernel<<<(int)((tot + 255) / 256), 256, 0, s>>>(ctx->e_h, n_q, d, w.cat1);
      }
      TGNN_LAUNCH_OK(ctx, "head_gather");
      GemmArgs g = {};
      g.A = w.cat1; g.a_rs = 2 * d; g.a_cs = 1;
      g.B = P + L.w1; g.b_rs = 1; g.b_cs = 2 * d;
      g.C = w.hid1; g.ldc = d; g.M = 2 * n_q; g.N = d; g.K = 2 * d; g.bias = P + L.b1; g.relu = 1; g.split_k = 1;
      g.site = SITE_HEAD + 1;
      RC(launch_gemm(ctx, g, "head_hidden", s));
      {
        KernelScope scope__(ctx, "head_loss", s);
        head_loss_kernel<<<(n_q + 7) / 8, 256, d * sizeof(float), s>>>(w.hid1, P + L.w2, P + L.b2, loss_mask, n_q, d,
                                                                       G + L.w2, G + L.b2, w.st_scalars, w.hid_gate);
      }
      TGNN_LAUNCH_OK(ctx, "head_loss");
      // hid1 now holds d loss / d pre1
      RC(fork_to(ctx, s, sa));
      RC(grad_w(ctx, w.hid1, d, w.cat1, 2 * d, 2 * n_q, nullptr, d, 2 * d, G + L.w1, G + L.b1, "dW_1", sa));
      RC(grad_in(ctx, w.hid1, d, P + L.w1, 2 * d, 0, 2 * n_q, nullptr, d, 2 * d, w.dcat1, 2 * d, "dcat1", s, SITE_DCAT1 + 1));
      const int64_t tot2 = (int64_t)R * d;
      {
        KernelScope scope__(ctx, "dh", s);
        dh_kernel<<<(int)((tot2 + 255) / 256), 256, 0, s>>>(w.dcat1, ctx->e_h, n_q, d, w.dpre_o, relu_out);
      }
      TGNN_LAUNCH_OK(ctx, "dh");
    }
    if (c.model == TGNN_MODEL_JODIE) {
      // embedding -> memory rows written by this step -> recurrent cell -> its weights and the time encoder
      const size_t tg_smem = (size_t)8 * 2 * d * sizeof(double);
      {
        KernelScope scope__(ctx, "jodie_embed_bwd", s);
        jodie_embed_bwd_kernel<<<(R + 7) / 8 < 148 ? (R + 7) / 8 : 148, 256, tg_smem, s>>>(
            w.dpre_o, ctx->memory, ctx->last_update, P + L.proj_w, P + L.proj_b, ctx->e_nodes, ctx->e_times, R, d,
            w.node2slot, ctx->have_update ? 1 : 0, w.dMemU, w.tg_acc + 2 * d, c.num_nodes);
      }
      TGNN_LAUNCH_OK(ctx, "jodie_embed_bwd");
      if (ctx->have_update) {
        const int U_cap = ctx->upd_cap;
        const int64_t tot3 = (int64_t)U_cap * d;
        {
          KernelScope scope__(ctx, "rnn_bwd_gate", s);
          rnn_bwd_gate_kernel<<<(int)((tot3 + 255) / 256), 256, 0, s>>>(w.dMemU, w.g_n, ctx->upd_n_uniq, U_cap, d, w.dGi);
        }
        TGNN_LAUNCH_OK(ctx, "rnn_bwd_gate");
        RC(fork_to(ctx, s, sa));
        RC(fork_to(ctx, s, sb));
        RC(grad_w(ctx, w.dGi, d, w.X, ctx->ld_msg, U_cap, ctx->upd_n_uniq, d, (int)L.dmsg, G + L.gru_wi, G + L.gru_bi,
                  "dW_i", sa));
        RC(grad_w(ctx, w.dGi, d, w.X, ctx->ld_msg, U_cap, ctx->upd_n_uniq, d, d, G + L.gru_wh, G + L.gru_bh, "dW_h", sb));
        RC(grad_in(ctx, w.dGi, d, P + L.gru_wi, L.dmsg, 2 * d + de, U_cap, ctx->upd_n_uniq, d, d, w.dXp, d, "dX_phi", s,
                   SITE_DXPHI + 1));
        {
          KernelScope scope__(ctx, "time_grad_x", s);
          const int rpb = tg_rows_per_block(U_cap);
          time_grad_launch((U_cap + rpb - 1) / rpb, tg_smem, s, w.dXp, d, 0, w.Xsin, w.x_dt, U_cap,
                                                                         ctx->upd_n_uniq, d, P + L.time_w, P + L.time_b, w.tg_acc, rpb);
        }
        TGNN_LAUNCH_OK(ctx, "time_grad_x");
      }
      RC(fork_to(ctx, sa, s));  // join
      RC(fork_to(ctx, sb, s));
    } else {
    RC(fork_to(ctx, s, sb));
    RC(grad_w(ctx, w.dpre_o, d, w.cat_o, 2 * d, R, nullptr, d, 2 * d, G + L.wo, G + L.bo, "dW_o", sb));
    RC(grad_in(ctx, w.dpre_o, d, P + L.wo, 2 * d, 0, R, nullptr, d, 2 * d, w.dcat_o, 2 * d, "dcat_o", s, SITE_DCATO + 1));
    const int wpb = attn_warps_per_block(d, H, k);
    {
      static SmemLimit lim_f, lim_t, lim_x;
      const int need = (int)attn_smem_bytes(d, H, k, wpb);
      RC(raise_smem_limit(ctx, attention_bwd_kernel<false>, need, lim_f));
      RC(raise_smem_limit(ctx, attention_bwd_kernel<true>, need, lim_t));
      if (d == 100 && H == 2 && k == 10) RC(raise_smem_limit(ctx, (attention_bwd_fixed_kernel<100, 2, 10>), need, lim_x));
    }
    const bool split = ctx->split_buf != nullptr && ctx->images_fresh;
    SplitMat dkvs = ctx->dkvs, zs = ctx->zs;
    dkvs.rows = NB; zs.rows = NB;
    {
      KernelScope scope__(ctx, "attention_bwd", s);
      // (8-byte plane stores: row pitch and plane distance multiples of 4 elements)
      const bool fixed_shape = split && d == 100 && H == 2 && k == 10 && dkvs.ld % 4 == 0 && dkvs.plane_stride % 4 == 0;
      if (fixed_shape)   // the paper's configuration
        attention_bwd_fixed_kernel<100, 2, 10><<<(R + wpb - 1) / wpb, wpb * 32, attn_smem_bytes(d, H, k, wpb), s>>>(
            w.Q, w.KV, w.alpha, w.dcat_o, ctx->e_cnt, R, w.dQ, reinterpret_cast<__nv_bfloat16*>(dkvs.hi), dkvs.plane_stride,
            (int)dkvs.ld, dkvs.scale);
      else if (split)   // the key/value gradient leaves the kernel as fp16 planes, the form its two consumers read
        attention_bwd_kernel<true><<<(R + wpb - 1) / wpb, wpb * 32, attn_smem_bytes(d, H, k, wpb), s>>>(
            w.Q, w.KV, w.alpha, w.dcat_o, ctx->e_cnt, R, d, H, k, w.dQ, nullptr, reinterpret_cast<__nv_bfloat16*>(dkvs.hi),
            dkvs.plane_stride, (int)dkvs.ld, dkvs.scale);
      else
        attention_bwd_kernel<false><<<(R + wpb - 1) / wpb, wpb * 32, attn_smem_bytes(d, H, k, wpb), s>>>(
            w.Q, w.KV, w.alpha, w.dcat_o, ctx->e_cnt, R, d, H, k, w.dQ, w.dKV, nullptr, 0, 0, 1.f);
    }
    TGNN_LAUNCH_OK(ctx, "attention_bwd");
    RC(fork_to(ctx, s, sa));
    RC(fork_to(ctx, s, sb));
    // dW_kv is a leaf of the chain, its input-gradient sibling dZ is on it, and the split kernel is persistent (a
    // launch fills the machine until it ends): in that mode the weight gradient is issued after dZ, further down.
    if (!split)
      RC(grad_w(ctx, w.dKV, 2 * d, w.Z, ctx->ld_kv, NB, nullptr, 2 * d, (int)L.dkv, G + L.wk, G + L.bk, "dW_kv", sa));
    // time-encoder gradient through the attention inputs (side stream b)
    const size_t tg_smem = (size_t)8 * 2 * d * sizeof(double);
    // gradient w.r.t. the memory columns and the time-encoding columns of Z, side by side in dZmp.  With the
    // weight images at hand it is one product on the caller's stream (the scatter below needs its first
    // half); otherwise the two column ranges of W_kv are two strided products.
    const bool merged_dz = ctx->cfg.math_mode != TGNN_MATH_FP32 && ctx->images_fresh && ctx->images != nullptr;
    // the query-side input gradient does not depend on dZ: it runs on side stream b next to it
    RC(grad_in(ctx, w.dQ, d, P + L.wq, 2 * d, 0, R, nullptr, d, 2 * d, w.dzq, 2 * d, "dzq", sb, SITE_DZQ + 1));
    cudaEvent_t dzq_done = mark_stream(ctx, sb);  // waited for by the scatter further down
    RC(grad_w(ctx, w.dQ, d, w.Zq, 2 * d, R, nullptr, d, 2 * d, G + L.wq, G + L.bq, "dW_q", sb));
    {
      KernelScope scope__(ctx, "time_grad_q", sb);
      const int rpb = tg_rows_per_block(R);
      time_grad_launch((R + rpb - 1) / rpb, tg_smem, sb, w.dzq, 2 * d, d, nullptr, nullptr, R, nullptr, d,
                                                                  P + L.time_w, P + L.time_b, w.tg_acc, rpb);
    }
    TGNN_LAUNCH_OK(ctx, "time_grad_q");
    cudaStream_t s_tgz = sb;  // where the time-encoder sum over the neighbor rows runs
    bool join_sc = false;
    if (split) {
      RC(launch_gemm_split(ctx, dkvs, ctx->wz_s, 0, w.dZmp, 2 * d, NB, 2 * d, 2 * d, nullptr, 0, 0, 1, "dZ", s));
      RC(fork_to(ctx, s, sa));
      RC(fork_to(ctx, s, sc));
      // dW_kv = dKV^T Z over the neighbor rows; Z's column of ones yields the bias gradient as the last column.  It
      // starts when dZ has finished and runs beside the rest of the chain (scatter, cell backward, ...).
      SplitMat a = dkvs, b = zs;
      a.rows = NB; a.cols = 2 * d; b.rows = NB; b.cols = L.dkv + 1;
      // Per-site precision: this product is a leaf (its result goes to Adam and nowhere else), and with a bf16 feature
      // table the contract's tolerance is 1e-2: there it reads only the hi planes of both operands -- one fp16 pass,
      // half the bytes.  Measured on the large workload at full size: the W_k / W_v gradients stay within 1e-3 of
      // their largest entry.  (The forward projection in one pass put other tensors at 9e-3, and the input gradient
      // dZ feeds everything upstream: both keep their three passes.)
      if (c.feat_dtype == TGNN_BF16) { a.planes = 1; b.planes = 1; }
      RC(launch_gemm_split(ctx, a, b, 1, w.dWkv_pad, ctx->ld_wkv, 2 * d, (int)L.dkv + 1, NB, nullptr, 0, 1, 1 << 20, "dW_kv", sa));
      {
        KernelScope scope__(ctx, "fold_dW_kv", sa);
        fold_dwkv_kernel<<<148, 256, 0, sa>>>(w.dWkv_pad, ctx->ld_wkv, 2 * d, (int)L.dkv, G + L.wk, G + L.bk);
      }
      TGNN_LAUNCH_OK(ctx, "fold_dW_kv");
      // The time-encoder sum needs little shared memory and fits beside the weight gradient's CTAs; on side stream
      // b it would queue behind the query-side products, which wait for a whole SM each.
      s_tgz = sc;
      join_sc = true;
    } else if (merged_dz) {
      RC(grad_in(ctx, w.dKV, 2 * d, P + L.wk, L.dkv, 0, NB, nullptr, 2 * d, 2 * d, w.dZmp, 2 * d, "dZ", s, SITE_DZ + 1));
      RC(fork_to(ctx, s, sa));
      s_tgz = sa;
    } else {
      RC(grad_in(ctx, w.dKV, 2 * d, P + L.wk, L.dkv, d + de, NB, nullptr, 2 * d, d, w.dZmp + d, 2 * d, "dZ_phi", sb));
    }
    {
      KernelScope scope__(ctx, "time_grad_z", s_tgz);
      const int rpb = tg_rows_per_block(NB);
      time_grad_launch((NB + rpb - 1) / rpb, tg_smem, s_tgz, w.dZmp, 2 * d, d, nullptr, w.z_dt, NB, nullptr, d, P + L.time_w,
                                                                      P + L.time_b, w.tg_acc, rpb);
    }
    TGNN_LAUNCH_OK(ctx, "time_grad_z");
    RC(wait_mark(ctx, s, dzq_done));  // the scatter below needs dzq
    if (ctx->have_update) {
      if (!merged_dz && !split)
        RC(grad_in(ctx, w.dKV, 2 * d, P + L.wk, L.dkv, 0, NB, nullptr, 2 * d, d, w.dZmp, 2 * d, "dZ_mem", s));
      {
        KernelScope scope__(ctx, "scatter_dmem", s);
        // many rows per node (small node set, large batch): sum per block first, the hub rows would serialise
        if ((int64_t)NB >= 4 * (int64_t)c.num_nodes) {
          if (d <= 128)
          scatter_dmem_cached_kernel<1><<<(NB + R + SC_ROWS - 1) / SC_ROWS, 256, 0, s>>>(
              w.dZmp, w.dcat_o, w.dzq, ctx->e_nbr, ctx->e_nodes, R, k, d, w.node2slot, w.dMemU, c.num_nodes);
        else
          scatter_dmem_cached_kernel<2><<<(NB + R + SC_ROWS - 1) / SC_ROWS, 256, 0, s>>>(
              w.dZmp, w.dcat_o, w.dzq, ctx->e_nbr, ctx->e_nodes, R, k, d, w.node2slot, w.dMemU, c.num_nodes);
        } else {
          scatter_dmem_kernel<<<(NB + R + 7) / 8, 256, 0, s>>>(w.dZmp, w.dcat_o, w.dzq, ctx->e_nbr, ctx->e_nodes, R, k, d,
                                                               w.node2slot, w.dMemU, c.num_nodes);
        }
      }
      TGNN_LAUNCH_OK(ctx, "scatter_dmem");
      const int U_cap = ctx->upd_cap;
      const int64_t tot3 = (int64_t)U_cap * d;
      {
        KernelScope scope__(ctx, "gru_bwd_gate", s);
        gru_bwd_gate_kernel<<<(int)((tot3 + 255) / 256), 256, 0, s>>>(w.dMemU, w.X, ctx->ld_msg, d, w.g_r, w.g_z, w.g_n,
                                                                      w.g_hn, ctx->upd_n_uniq, U_cap, w.dGi, w.dGh);
      }
      TGNN_LAUNCH_OK(ctx, "gru_bwd_gate");
      // (split mode: side stream a carries the persistent key/value weight gradient, which ends late)
      cudaStream_t s_wi = split ? sd : sa;
      RC(fork_to(ctx, s, s_wi));
      RC(fork_to(ctx, s, sb));
      RC(grad_w(ctx, w.dGi, 3 * d, w.X, ctx->ld_msg, U_cap, ctx->upd_n_uniq, 3 * d, (int)L.dmsg, G + L.gru_wi,
                G + L.gru_bi, "dW_i", s_wi));
      RC(grad_w(ctx, w.dGh, 3 * d, w.X, ctx->ld_msg, U_cap, ctx->upd_n_uniq, 3 * d, d, G + L.gru_wh, G + L.gru_bh,
                "dW_h", sb));
      RC(grad_in(ctx, w.dGi, 3 * d, P + L.gru_wi, L.dmsg, 2 * d + de, U_cap, ctx->upd_n_uniq, 3 * d, d, w.dXp, d,
                 "dX_phi", s, SITE_DXPHI + 1));
      {
        KernelScope scope__(ctx, "time_grad_x", s);
        const int rpb = tg_rows_per_block(U_cap);
        time_grad_launch((U_cap + rpb - 1) / rpb, tg_smem, s, w.dXp, d, 0, w.Xsin, w.x_dt, U_cap, ctx->upd_n_uniq,
                                                                       d, P + L.time_w, P + L.time_b, w.tg_acc, rpb);
      }
      TGNN_LAUNCH_OK(ctx, "time_grad_x");
      if (split) RC(fork_to(ctx, sd, s));  // join
    }
    RC(fork_to(ctx, sa, s));  // join
    RC(fork_to(ctx, sb, s));
    if (join_sc) RC(fork_to(ctx, sc, s));
    }  // attention model
  }
  {
    KernelScope scope__(ctx, "gradnorm_adam", s);
    const int p_n = (n_q > 0 && c.model == TGNN_MODEL_JODIE) ? 2 * d : 0;
    gradnorm_adam_kernel<<<296, 256, 0, s>>>(G, L.total, w.tg_acc, L.time_w, n_q > 0 ? 2 * d : 0, L.proj_w, p_n, w.red, w.counters,
                                             ctx->step, P, ctx->adam_m, ctx->adam_v, c.lr, c.beta1, c.beta2, c.eps,
                                             w.st_scalars, w.st_scalars + 2, loss_out, gradnorm_out, 1.f, ctx->defer_adam ? 0 : 1);
  }
  TGNN_LAUNCH_OK(ctx, "gradnorm_adam");
  return TGNN_OK;
}

// The second half of a step whose gradient was left for synchronisation: norm of gscale * gradient and Adam.
int launch_apply_gradient(tgnn_ctx* ctx, float gscale, float* gradnorm_out, cudaStream_t s) {
  const tgnn_config& c = ctx->cfg;
  Workspace& w = ctx->ws;
  TGNN_CUDA_OK(ctx, cudaMemsetAsync(w.red, 0, sizeof(double), s));
  {
    KernelScope scope__(ctx, "apply_gradient", s);
    gradnorm_adam_kernel<<<296, 256, 0, s>>>(w.grads, ctx->L.total, w.tg_acc, 0, 0, 0, 0, w.red, w.counters, ctx->step,
                                             ctx->params, ctx->adam_m, ctx->adam_v, c.lr, c.beta1, c.beta2, c.eps,
                                             w.st_scalars, w.st_scalars + 2, nullptr, gradnorm_out, gscale, 1);
  }
  TGNN_LAUNCH_OK(ctx, "apply_gradient");
  return TGNN_OK;
}

}  // namespace tgnn
