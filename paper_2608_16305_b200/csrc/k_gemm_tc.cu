// Dense projections on the 5th-generation tensor cores (TGNN_MATH_TF32).
//
// One CTA computes a 128 x BN tile of C = A B over a range of the contraction
// (split-K across blockIdx.z) with tcgen05.mma.kind::tf32: fp32 operands rounded to
// TF32 (round-to-nearest, by the producer warps, so there is no truncation bias),
// fp32 accumulation in tensor memory.  With `precise` set every operand is split into
// a TF32 head and a TF32 tail (x = hi + lo) and three MMAs (lo*hi, hi*lo, hi*hi) give
// close to fp32 accuracy; the gradient products, whose terms cancel, use it.
//
// Warp roles:
//   G producer groups of 4 warps.  Group g fills the stages of contraction blocks
//     i = g, g + G, ...: global -> registers (all 128-bit loads of a block issued before
//     the first use) -> round to TF32 -> shared memory in the swizzled canonical layout
//     the MMA descriptors expect.  Several blocks are therefore in flight at once.
//     Afterwards all groups run the epilogue (tcgen05.ld of the 32 TMEM lanes their warp
//     may touch, bias / ReLU / store or atomic accumulate), sharing the columns.
//   1 MMA warp: allocates tensor memory; one lane issues the MMAs and commits.
// A ring of (A tile, B tile) stages is handed over through mbarriers: full[s] (128
// producer arrivals) and empty[s] (tcgen05.commit).  Every wait is bounded; on expiry
// the kernel records TGNN_ETIMEOUT in the status word, stops waiting, frees its tensor
// memory and returns.
//
// Operands may be K-major (contraction index contiguous) or MN-major (row/column index
// contiguous), so the forward projections (activations [M,K] x weights [N,K]), the
// input gradients (dY [M,N'] x W [N',K]) and the weight gradients (dY^T x A, contraction
// over rows) all run here without a transposed copy.
#include <cuda.h>

#include <cstdlib>

#include "tgnn_internal.cuh"

namespace tgnn {
namespace {

constexpr int BM = 128;    // rows of C per CTA (UMMA M)
constexpr int BK = 32;     // contraction elements per stage: one 128-byte swizzle row of fp32
constexpr int UMMA_K = 8;  // tf32
constexpr int GROUP = 128; // threads per producer group
constexpr int EPI_PITCH = 36;  // floats between rows of an epilogue staging square (16-byte aligned, bank-staggered)
constexpr unsigned SPIN_LIMIT = 1u << 24;
constexpr unsigned FULL = 0xffffffffu;

enum { MAJOR_K = 0, MAJOR_MN = 1 };

struct TcArgs {
  const float* A; int64_t lda; int a_major;
  const float* B; int64_t ldb; int b_major;
  float* C; int64_t ldc;
  int M, N, K;
  const int32_t* dev_M;
  const int32_t* dev_K;
  const float* bias;
  float* rowsum_out;
  int relu, accumulate, split_k;
  int32_t* status;
  // B operand prepared as shared-memory images (see WeightSite): image of n-tile x, contraction block
  // kb at b_image + x * b_tile_stride + kb * (COPIES * B_BYTES); nullptr: B goes through registers
  const unsigned char* b_image;
  int64_t b_tile_stride;
  // Row-indirect leading columns of a K-major A: A(m, k) for k < a_tab_cols is a_tab[a_idx[m] * a_tab_cols + k]
  // (zero if a_idx[m] < 0) instead of A[m * lda + k]; nullptr: plain A.  Lets the key/value projection
  // read the neighbors' memory rows straight from the table.
  const int32_t* a_idx;
  const float* a_tab;
  int a_tab_cols;
  int64_t a_tab_rows;
  // K-major A as a tiled tensor map (box 32 x 128, 128-byte swizzle): the tensor-memory-access unit brings
  // whole activation tiles into shared memory; a_tma = 0: A goes through registers
  int a_tma;
  CUtensorMap a_map;
  // both operands MN-major (weight gradients): A and B as four-dimensional views of their row-major matrices
  // whose boxes land in the operand tiles' atom layout (see encode_mn_map); b_box_atoms = 32-column atoms per B box
  CUtensorMap b_map;
  int b_box_atoms;
};

template <int BN_T, bool PRECISE, int TMA = 0>
struct Cfg {
  static constexpr int STAGES = PRECISE ? (BN_T > 128 ? 2 : 3) : 4;
  // A group's consecutive blocks must not be more than one use of a stage apart (the waits tell phases apart
  // by parity only), so there are never more groups than stages.
  static constexpr int GROUPS = STAGES < 3 ? STAGES : 3;
  static_assert(GROUPS <= STAGES, "a producer group may not lap a stage");
  static constexpr int THREADS = GROUPS * GROUP + 32;
  static constexpr int A_BYTES = BM * 128, B_BYTES = BN_T * 128;
  static constexpr int COPIES = PRECISE ? 2 : 1;  // head (+ tail) copy of each operand tile
  static constexpr int STAGE_BYTES = COPIES * (A_BYTES + B_BYTES);
  static constexpr int SMEM = 1024 + STAGES * STAGE_BYTES;
  static constexpr uint32_t TMEM_COLS = BN_T <= 128 ? 128 : 256;
  static_assert(SMEM <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on a phase parity.  Returns false if the limit was reached.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (unsigned it = 0; it < SPIN_LIMIT; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

// Loads and stores are volatile asm so that the compiler keeps every load of a block ahead of
// the first store (it otherwise sinks each load next to its use and serialises the round trips).
__device__ __forceinline__ float4 ldg_v4(const float* p) {
  float4 v;
  asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ float ldg_f(const float* p) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// Round-to-nearest (ties away from zero) to the 10 mantissa bits of TF32: add half an ulp to the
// magnitude and clear the 13 low bits.  Same result as cvt.rna.tf32.f32 for finite inputs, but on
// the integer pipe at full rate (the conversion pipe would bound the producers).
__device__ __forceinline__ uint32_t to_tf32(float x) { return (__float_as_uint(x) + 0x1000u) & 0xffffe000u; }

// One 16-byte chunk of an operand tile.  Single pass: the values rounded to TF32.  Split: the values as they
// are in the head copy -- the tensor core reads sign, exponent and the upper 10 mantissa bits of a tf32
// operand and ignores the 13 bits below, so the head it sees is the value truncated -- and the exact
// remainder (the part it ignores) in the tail copy, of which it again sees the upper bits.  Head + tail then
// carry 21 mantissa bits; truncation's bias is in the tail's dropped bits only (2^-21 relative).
__device__ __forceinline__ uint32_t tf32_remainder(float x) {
  return __float_as_uint(x - __uint_as_float(__float_as_uint(x) & 0xffffe000u));
}
template <bool PRECISE>
__device__ __forceinline__ void store_chunk(uint32_t addr, uint32_t tail_offset, const float4& v) {
  if (PRECISE) {
    sts_v4(addr, __float_as_uint(v.x), __float_as_uint(v.y), __float_as_uint(v.z), __float_as_uint(v.w));
    sts_v4(addr + tail_offset, tf32_remainder(v.x), tf32_remainder(v.y), tf32_remainder(v.z), tf32_remainder(v.w));
  } else {
    sts_v4(addr, to_tf32(v.x), to_tf32(v.y), to_tf32(v.z), to_tf32(v.w));
  }
}

// A chunk that a TMA copy left in the head tile as plain fp32 stays there as the head; only its tail is written.
__device__ __forceinline__ void store_tail_of_raw(uint32_t tail_addr, const float4& v) {
  sts_v4(tail_addr, tf32_remainder(v.x), tf32_remainder(v.y), tf32_remainder(v.z), tf32_remainder(v.w));
}

// 64-bit shared-memory matrix descriptor.  layout: 2 = 128-byte swizzle on 16-byte chunks (K-major
// operands), 1 = 128-byte swizzle with a 32-byte base (the only layout for MN-major 32-bit operands).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version for this architecture
  d |= (uint64_t)layout << 61;
  return d;
}

// One producer group (128 threads, index t) fills one operand tile for contraction block [k0, k0+32).
//   K-major:  rows [r0, r0 + rows_t) x 32 k; row r lives at (r/8)*1024 + (r%8)*128, its 16-byte
//             chunk c at position c ^ (r%8).
//   MN-major: 32 k-rows x rows_t (MN) values in atoms of 4 k-rows x 32 values (512 B); k-row kk, MN
//             atom a, chunk c lives at (kk/4)*(atoms*512) + a*512 + (kk%4)*128 + ((c ^ 2*(kk%4))*16):
//             the swizzle exchanges 32-byte pairs of chunks (address bits 5-6 ^= bits 7-8).
// rows_t is a multiple of 32 (MN-major) or of 8 (K-major); chunks outside the valid range are zero.
// The tile is filled in two steps so that a producer can have the loads of its next block in flight
// while it waits for a free stage and stores the current one.
// FAST (every chunk is wholly inside or wholly outside the operand, pointers 16-byte aligned): the
// loads are unconditional -- an out-of-range chunk reads the operand's first chunk instead and is
// zeroed at store time from the returned mask -- so nothing between the loads depends on a loaded
// value and all of a block's round trips overlap.  Otherwise chunks are read element by element
// under their bounds checks.
template <int ROWS_MAX, bool FAST>
__device__ __forceinline__ uint32_t load_regs(float4 (&v)[ROWS_MAX * 8 / GROUP], const float* __restrict__ P, int64_t ld,
                                              int major, int r0, int R, int rows_t, int k0, int k1, bool vec, int t,
                                              const int32_t* tab_row = nullptr, const float* __restrict__ tab = nullptr,
                                              int tab_cols = 0) {
  constexpr int ITERS = ROWS_MAX * 8 / GROUP;
  uint32_t mask = 0;
  if (major == MAJOR_K) {
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const int idx = t + i * GROUP;
      const int r = idx >> 3, c = idx & 7;
      const int gr = r0 + r, gk = k0 + 4 * c;
      bool valid = r < rows_t && gr < R && gk < k1;
      const float* p = P + (int64_t)gr * ld + gk;
      if (tab_row != nullptr && gk < tab_cols) {  // tab_cols is a multiple of 4: the chunk is all table or all A
        valid = valid && tab_row[i] >= 0;
        p = tab + (int64_t)tab_row[i] * tab_cols + gk;
      }
      if (FAST) {
        v[i] = ldg_v4(valid ? p : P);
        mask |= (valid ? 1u : 0u) << i;
      } else {
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) {
          if (vec && gk + 3 < k1) {
            v[i] = ldg_v4(p);
          } else {
            v[i].x = ldg_f(p);
            if (gk + 1 < k1) v[i].y = ldg_f(p + 1);
            if (gk + 2 < k1) v[i].z = ldg_f(p + 2);
            if (gk + 3 < k1) v[i].w = ldg_f(p + 3);
          }
        }
      }
    }
  } else {
    const int cpr = rows_t >> 2;  // 16-byte chunks per k-row (multiple of 8)
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const int idx = t + i * GROUP;
      const int kk = idx / cpr, cm = idx - kk * cpr;
      const int gk = k0 + kk, gr = r0 + 4 * cm;
      const bool valid = kk < BK && gk < k1 && gr < R;
      const float* p = P + (int64_t)gk * ld + gr;
      if (FAST) {
        v[i] = ldg_v4(valid ? p : P);
        mask |= (valid ? 1u : 0u) << i;
      } else {
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) {
          if (vec && gr + 3 < R) {
            v[i] = ldg_v4(p);
          } else {
            v[i].x = ldg_f(p);
            if (gr + 1 < R) v[i].y = ldg_f(p + 1);
            if (gr + 2 < R) v[i].z = ldg_f(p + 2);
            if (gr + 3 < R) v[i].w = ldg_f(p + 3);
          }
        }
      }
    }
  }
  return FAST ? mask : 0xffffffffu;
}

template <int ROWS_MAX, bool PRECISE>
__device__ __forceinline__ void store_regs(const float4 (&v)[ROWS_MAX * 8 / GROUP], uint32_t mask, uint32_t tile,
                                           uint32_t tail_offset, int major, int rows_t, int t, float4* rowsum) {
  constexpr int ITERS = ROWS_MAX * 8 / GROUP;
  if (major == MAJOR_K) {
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const int idx = t + i * GROUP;
      const int r = idx >> 3, c = idx & 7;
      const float4 x = (mask >> i) & 1u ? v[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      if (r < rows_t) store_chunk<PRECISE>(tile + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4), tail_offset, x);
    }
  } else {
    const int cpr = rows_t >> 2;
    const int atoms = rows_t >> 5;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
      const int idx = t + i * GROUP;
      const int kk = idx / cpr, cm = idx - kk * cpr;
      if (kk < BK) {
        const int a = cm >> 3, c = cm & 7;
        const float4 x = (mask >> i) & 1u ? v[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        store_chunk<PRECISE>(tile + (kk >> 2) * (atoms * 512) + a * 512 + (kk & 3) * 128 + ((c ^ ((kk & 3) << 1)) << 4),
                             tail_offset, x);
        if (rowsum && rows_t == BM) {  // cm == t % 32 for every i: per-thread sums of 4 rows of C
          rowsum->x += x.x; rowsum->y += x.y; rowsum->z += x.z; rowsum->w += x.w;
        }
      }
    }
  }
}

template <int ROWS_MAX, bool PRECISE, bool FAST>
__device__ __forceinline__ void load_tile(uint32_t tile, uint32_t tail_offset, const float* __restrict__ P, int64_t ld,
                                          int major, int r0, int R, int rows_t, int k0, int k1, bool vec, int t,
                                          float4* rowsum) {
  float4 v[ROWS_MAX * 8 / GROUP];
  const uint32_t mask = load_regs<ROWS_MAX, FAST>(v, P, ld, major, r0, R, rows_t, k0, k1, vec, t);
  store_regs<ROWS_MAX, PRECISE>(v, mask, tile, tail_offset, major, rows_t, t, rowsum);
}

__device__ __forceinline__ void mma_tf32(uint32_t tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc)
      : "memory");
}

// grid: (n tiles, m tiles, split_k).  Dynamic shared memory: Cfg::SMEM bytes.
template <int BN_T, bool PRECISE, bool FAST, int TMA>
__global__ void __launch_bounds__(Cfg<BN_T, PRECISE, TMA>::THREADS, 1) gemm_tf32_kernel(const __grid_constant__ TcArgs g) {
  using C_ = Cfg<BN_T, PRECISE, TMA>;
  constexpr int STAGES = C_::STAGES, GROUPS = C_::GROUPS, THREADS = C_::THREADS;
  constexpr int MMA_WARP = GROUPS * 4;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_full[STAGES], s_empty[STAGES], s_accum, s_raw[STAGES];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ float s_rowsum[BM];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int M = g.dev_M ? min(*g.dev_M, g.M) : g.M;
  const int K = g.dev_K ? min(*g.dev_K, g.K) : g.K;
  const int m0 = blockIdx.y * BM;
  const int bn = min(BN_T, ((g.N + gridDim.x - 1) / gridDim.x + 31) / 32 * 32);  // columns per n-tile
  const int n0 = blockIdx.x * bn;
  if (m0 >= M || n0 >= g.N) return;
  const int n_valid = min(bn, g.N - n0);
  // MMA N: multiple of 16; MN-major B tiles are loaded in whole 32-column atoms
  const int n_mma = (n_valid + 15) / 16 * 16;
  const int b_rows = TMA == 2 ? g.b_box_atoms * 32  // the tile's layout is the box's, whatever part of it is valid
                              : (g.b_major == MAJOR_MN ? (n_valid + 31) / 32 * 32 : (n_mma + 7) / 8 * 8);
  const int nkb_total = (K + BK - 1) / BK;
  const int per = (nkb_total + g.split_k - 1) / g.split_k;
  const int kb0 = blockIdx.z * per, kb1 = min(nkb_total, kb0 + per);
  const int nkb = kb1 - kb0;

  if (nkb <= 0) {  // nothing to contract: store mode still owes bias (+ReLU)
    if (!g.accumulate && blockIdx.z == 0) {
      for (int e = tid; e < BM * n_valid; e += THREADS) {
        const int r = e / n_valid, c = e - r * n_valid;
        if (m0 + r < M) {
          float v = g.bias ? g.bias[n0 + c] : 0.f;
          if (g.relu) v = fmaxf(v, 0.f);
          g.C[(int64_t)(m0 + r) * g.ldc + n0 + c] = v;
        }
      }
    }
    return;
  }

  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t smem_base = smem_u32(smem);

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&s_full[s]), GROUP + (g.b_image ? 1 : 0));
      mbar_init(smem_u32(&s_empty[s]), 1);
    }
    mbar_init(smem_u32(&s_accum), 1);
    for (int r = 0; r < STAGES; ++r) mbar_init(smem_u32(&s_raw[r]), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < BM) s_rowsum[tid] = 0.f;
  if (warp == MMA_WARP) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                 "r"(C_::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;

  if (warp < MMA_WARP) {
    // ------------------------------------------------------------ producers
    const int grp = warp >> 2, t = tid & (GROUP - 1);
    const bool a_vec = (((uintptr_t)g.A & 15) == 0) && (g.lda % 4 == 0);
    const bool b_vec = (((uintptr_t)g.B & 15) == 0) && (g.ldb % 4 == 0);
    const bool want_rowsum = g.rowsum_out != nullptr && blockIdx.x == 0 && g.a_major == MAJOR_MN;
    float4 rs = make_float4(0.f, 0.f, 0.f, 0.f);
    const int k_end = min(K, kb1 * BK);
    bool ok = true;
    // The A registers of the group's next block are loaded before it waits for the current stage,
    // so that round trip overlaps the wait, the stores and the MMAs of the blocks in between.
    float4 va[BM * 8 / GROUP], vn[BM * 8 / GROUP];
    int32_t tab_row[BM * 8 / GROUP];  // table row of each of the thread's A rows (row-indirect mode)
    const int32_t* trp = nullptr;
    if (g.a_idx != nullptr && g.a_major == MAJOR_K) {
#pragma unroll
      for (int q = 0; q < BM * 8 / GROUP; ++q) {
        const int gr = m0 + ((t + q * GROUP) >> 3);
        const int ti = gr < M ? g.a_idx[gr] : -1;
        tab_row[q] = ti < g.a_tab_rows ? ti : -1;   // an index beyond the table reads as a zero row
      }
      trp = tab_row;
    }
    uint32_t ma = 0, mn = 0;
    // The B tile of block i into stage s: one bulk asynchronous copy of the prepared image (head and tail);
    // it signals full[s] itself.
    auto b_image_copy = [&](int i, int s, uint32_t b_tile) {
      constexpr uint32_t bytes = C_::COPIES * C_::B_BYTES;
      const unsigned char* src = g.b_image + blockIdx.x * g.b_tile_stride + (int64_t)(kb0 + i) * bytes;
      const uint32_t bar = smem_u32(&s_full[s]);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(b_tile), "l"(src), "r"(bytes), "r"(bar)
                   : "memory");
    };
    if constexpr (TMA == 2) {
      // Weight gradients: both operands are transposed views (contraction over rows).  One thread asks for the
      // block's two boxes -- 32 contraction rows x 128 (A) or 32 x b_rows (B) values, delivered as atoms of
      // 4 rows x 32 values with the 32-byte swizzle, i.e. in the operand tiles' own layout -- and when they have
      // landed every thread rounds / splits its own chunks in place.  Values beyond the matrix edge inside the
      // last atom are whatever follows in memory: they only reach rows / columns of C that are never stored.
      const int b_atoms = b_rows >> 5, b_cpr = b_rows >> 2;
      const uint32_t b_bytes = (uint32_t)b_rows * 128;
      for (int i = grp; i < nkb; i += GROUPS) {
        const int s = i % STAGES;
        if (i >= STAGES) {
          ok = mbar_wait(smem_u32(&s_empty[s]), ((i / STAGES) - 1) & 1);
          if (!ok) break;
        }
        const uint32_t a_tile = smem_base + s * C_::STAGE_BYTES;
        const uint32_t b_tile = a_tile + C_::COPIES * C_::A_BYTES;
        const uint32_t raw_bar = smem_u32(&s_raw[s]);
        if (t == 0) {
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(raw_bar), "r"((uint32_t)C_::A_BYTES + b_bytes)
                       : "memory");
          asm volatile(
              "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
              ::"r"(a_tile), "l"(&g.a_map), "r"(0), "r"(0), "r"(m0 >> 5), "r"((kb0 + i) * (BK / 4)), "r"(raw_bar)
              : "memory");
          asm volatile(
              "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
              ::"r"(b_tile), "l"(&g.b_map), "r"(0), "r"(0), "r"(n0 >> 5), "r"((kb0 + i) * (BK / 4)), "r"(raw_bar)
              : "memory");
        }
        ok = mbar_wait(raw_bar, (i / STAGES) & 1);
        if (!ok) break;
        // A: 32 rows x 128 values = 1024 chunks, 8 per thread; chunk (kk, cm) lives where store_regs would put it
#pragma unroll
        for (int q = 0; q < BM * 8 / GROUP; ++q) {
          const int idx = t + q * GROUP;
          const int kk = idx >> 5, cm = idx & 31;
          const uint32_t addr = a_tile + (kk >> 2) * ((BM / 32) * 512) + (cm >> 3) * 512 + (kk & 3) * 128 +
                                (((cm & 7) ^ ((kk & 3) << 1)) << 4);
          float4 x;
          asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(addr) : "memory");
          if (PRECISE) store_tail_of_raw(addr + C_::A_BYTES, x);
          else store_chunk<PRECISE>(addr, C_::A_BYTES, x);
          if (want_rowsum) { rs.x += x.x; rs.y += x.y; rs.z += x.z; rs.w += x.w; }  // cm == t % 32 for every q
        }
        // B: 32 rows x b_rows values
        for (int idx = t; idx < BK * b_cpr; idx += GROUP) {
          const int kk = idx / b_cpr, cm = idx - kk * b_cpr;
          const uint32_t addr = b_tile + (kk >> 2) * (b_atoms * 512) + (cm >> 3) * 512 + (kk & 3) * 128 +
                                (((cm & 7) ^ ((kk & 3) << 1)) << 4);
          float4 x;
          asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(addr) : "memory");
          if (PRECISE) store_tail_of_raw(addr + C_::B_BYTES, x);
          else store_chunk<PRECISE>(addr, C_::B_BYTES, x);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(smem_u32(&s_full[s]));
      }
    } else if constexpr (TMA == 1) {
      // A arrives as whole tiles: once the stage is free, one thread of the group asks the tensor-memory-access
      // unit for block i (box 32 x 128 at column k, row m0; rows and columns outside the matrix come back as
      // zeros) straight into the stage's head tile, already in its 128-byte-swizzled layout.  When the tile
      // has landed every thread rounds its own chunks in place and writes their tails -- shared memory to
      // shared memory, no thread touches another's chunk.  Blocks that overlap the row-indirect columns still
      // go through registers from global memory.
      auto by_tma = [&](int i) { return !(g.a_idx != nullptr && (kb0 + i) * BK < g.a_tab_cols); };
      for (int i = grp; i < nkb; i += GROUPS) {
        const int s = i % STAGES;
        const bool tile = by_tma(i);
        if (!tile)
          ma = load_regs<BM, FAST>(va, g.A, g.lda, g.a_major, m0, M, BM, (kb0 + i) * BK, k_end, a_vec, t, trp, g.a_tab,
                                   g.a_tab_cols);
        if (i >= STAGES) {
          ok = mbar_wait(smem_u32(&s_empty[s]), ((i / STAGES) - 1) & 1);
          if (!ok) break;
        }
        const uint32_t a_tile = smem_base + s * C_::STAGE_BYTES;
        const uint32_t b_tile = a_tile + C_::COPIES * C_::A_BYTES;
        const uint32_t raw_bar = smem_u32(&s_raw[s]);
        if (t == 0) {
          if (tile) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(raw_bar), "r"((uint32_t)C_::A_BYTES)
                         : "memory");
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                ::"r"(a_tile), "l"(&g.a_map), "r"((kb0 + i) * BK), "r"(m0), "r"(raw_bar)
                : "memory");
          }
          b_image_copy(i, s, b_tile);
        }
        if (tile) {
          int before = 0;  // tile blocks that used this stage (and its tile barrier) before block i: the phase
          for (int j = s; j < i; j += STAGES) before += by_tma(j) ? 1 : 0;
          ok = mbar_wait(raw_bar, before & 1);
          if (!ok) break;
#pragma unroll
          for (int q = 0; q < BM * 8 / GROUP; ++q) {
            const int idx = t + q * GROUP, r = idx >> 3, c = idx & 7;
            const uint32_t addr = a_tile + r * 128 + ((c ^ (r & 7)) << 4);
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                         : "=f"(va[q].x), "=f"(va[q].y), "=f"(va[q].z), "=f"(va[q].w) : "r"(addr) : "memory");
          }
          ma = 0xffffffffu;
        }
        if (tile && PRECISE) {  // the landed values stay in place as heads
#pragma unroll
          for (int q = 0; q < BM * 8 / GROUP; ++q) {
            const int idx = t + q * GROUP, r = idx >> 3, c = idx & 7;
            store_tail_of_raw(a_tile + C_::A_BYTES + r * 128 + ((c ^ (r & 7)) << 4), va[q]);
          }
        } else {
          store_regs<BM, PRECISE>(va, ma, a_tile, C_::A_BYTES, MAJOR_K, BM, t, nullptr);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(smem_u32(&s_full[s]));
      }
    } else {
    if (grp < nkb)
      ma = load_regs<BM, FAST>(va, g.A, g.lda, g.a_major, m0, M, BM, (kb0 + grp) * BK, k_end, a_vec, t, trp, g.a_tab,
                               g.a_tab_cols);
    for (int i = grp; i < nkb; i += GROUPS) {
      const int s = i % STAGES;
      if (i + GROUPS < nkb)
        mn = load_regs<BM, FAST>(vn, g.A, g.lda, g.a_major, m0, M, BM, (kb0 + i + GROUPS) * BK, k_end, a_vec, t, trp,
                                 g.a_tab, g.a_tab_cols);
      if (i >= STAGES) {
        ok = mbar_wait(smem_u32(&s_empty[s]), ((i / STAGES) - 1) & 1);
        if (!ok) break;
      }
      const uint32_t a_tile = smem_base + s * C_::STAGE_BYTES;
      const uint32_t b_tile = a_tile + C_::COPIES * C_::A_BYTES;
      const int k0 = (kb0 + i) * BK;
      if (g.b_image != nullptr && t == 0) b_image_copy(i, s, b_tile);
      store_regs<BM, PRECISE>(va, ma, a_tile, C_::A_BYTES, g.a_major, BM, t, want_rowsum ? &rs : nullptr);
      if (g.b_image == nullptr)
        load_tile<BN_T, PRECISE, FAST>(b_tile, C_::B_BYTES, g.B, g.ldb, g.b_major, n0, g.N, b_rows, k0, k_end, b_vec, t, nullptr);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&s_full[s]));
#pragma unroll
      for (int q = 0; q < BM * 8 / GROUP; ++q) va[q] = vn[q];
      ma = mn;
    }
    }
    if (!ok) { s_abort = 1; atomicCAS(g.status, 0, TGNN_ETIMEOUT); }
    if (want_rowsum) {  // the thread's chunks cover rows 4*(t%32) .. +3 of the tile
      const int r = 4 * (t & 31);
      atomicAdd(&s_rowsum[r], rs.x); atomicAdd(&s_rowsum[r + 1], rs.y);
      atomicAdd(&s_rowsum[r + 2], rs.z); atomicAdd(&s_rowsum[r + 3], rs.w);
    }
    // ------------------------------------------------------------ epilogue
    if (ok) ok = mbar_wait(smem_u32(&s_accum), 0);
    if (!ok) { s_abort = 1; atomicCAS(g.status, 0, TGNN_ETIMEOUT); }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("bar.sync 1, %0;" ::"n"(GROUPS * GROUP) : "memory");  // all producers: s_rowsum complete
    if (want_rowsum && tid < BM && m0 + tid < M && s_rowsum[tid] != 0.f) atomicAdd(&g.rowsum_out[m0 + tid], s_rowsum[tid]);
    if (__all_sync(FULL, ok && !s_abort)) {  // warp-uniform: the TMEM loads are warp-collective
      // Each warp moves 32 rows x 32 columns at a time: TMEM -> registers (one row per lane) -> its
      // own staging square in the now idle pipeline memory -> global, re-read so that 8 lanes cover
      // 128 contiguous bytes of one row of C (whole sectors per request; a lane-per-row store would
      // touch 32 rows with 16 bytes each).
      const int q4 = warp & 3;  // the TMEM lane quarter this warp may access
      const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16);
      float* stg = reinterpret_cast<float*>(smem) + warp * (32 * EPI_PITCH);
      const bool c_vec = (((uintptr_t)g.C & 15) == 0) && (g.ldc % 4 == 0);
      const int sub = lane >> 3, ch = lane & 7;
      for (int c0 = grp * 32; c0 < n_valid; c0 += GROUPS * 32) {
        uint32_t r[32];
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
            "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
              "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
              "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
            : "r"(taddr + (uint32_t)c0));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(stg + lane * EPI_PITCH + 4 * q) = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
        __syncwarp();
        const int col = c0 + 4 * ch;  // first of this lane's 4 columns, relative to the tile
        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (g.bias && blockIdx.z == 0 && col < n_valid) {
          const float* bp = g.bias + n0 + col;
          b4.x = bp[0];
          if (col + 1 < n_valid) b4.y = bp[1];
          if (col + 2 < n_valid) b4.z = bp[2];
          if (col + 3 < n_valid) b4.w = bp[3];
        }
        const bool full4 = col + 3 < n_valid;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int rr = j * 4 + sub;
          const int row = m0 + q4 * 32 + rr;
          float4 v = *reinterpret_cast<const float4*>(stg + rr * EPI_PITCH + 4 * ch);
          if (row < M && col < n_valid) {
            v.x += b4.x; v.y += b4.y; v.z += b4.z; v.w += b4.w;
            float* cp = g.C + (int64_t)row * g.ldc + n0 + col;
            if (g.accumulate) {
              if (full4 && c_vec) {
                atomicAdd(reinterpret_cast<float4*>(cp), v);
              } else {
                atomicAdd(cp, v.x);
                if (col + 1 < n_valid) atomicAdd(cp + 1, v.y);
                if (col + 2 < n_valid) atomicAdd(cp + 2, v.z);
                if (col + 3 < n_valid) atomicAdd(cp + 3, v.w);
              }
            } else {
              if (g.relu) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
              if (full4 && c_vec) {
                *reinterpret_cast<float4*>(cp) = v;
              } else {
                cp[0] = v.x;
                if (col + 1 < n_valid) cp[1] = v.y;
                if (col + 2 < n_valid) cp[2] = v.z;
                if (col + 3 < n_valid) cp[3] = v.w;
              }
            }
          }
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------ MMA issuer
    // instruction descriptor: D fp32, A/B tf32, majors, N >> 3, M >> 4
    const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)g.a_major << 15) | ((uint32_t)g.b_major << 16) |
                           ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    const int b_atoms = b_rows >> 5;
    bool ok = true;
    for (int i = 0; i < nkb && ok; ++i) {
      const int s = i % STAGES;
      ok = mbar_wait(smem_u32(&s_full[s]), (i / STAGES) & 1);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (lane == 0) {
        const uint32_t a_addr = smem_base + s * C_::STAGE_BYTES;
        const uint32_t b_addr = a_addr + C_::COPIES * C_::A_BYTES;
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          // K-major: 8-row x 128 B atoms 1024 B apart (SBO); one MMA advances 32 B inside the swizzle row.
          // MN-major: 4-k-row atoms of 512 B; MN atoms 512 B apart (LBO), k-groups atoms*512 B apart
          // (SBO); one MMA consumes two k-groups.
          const uint32_t a_off = g.a_major == MAJOR_K ? k * 32 : k * 2 * (BM / 32) * 512;
          const uint32_t b_off = g.b_major == MAJOR_K ? k * 32 : k * 2 * b_atoms * 512;
          const uint32_t a_lbo = g.a_major == MAJOR_K ? 16 : 512, a_sbo = g.a_major == MAJOR_K ? 1024 : (BM / 32) * 512;
          const uint32_t b_lbo = g.b_major == MAJOR_K ? 16 : 512, b_sbo = g.b_major == MAJOR_K ? 1024 : b_atoms * 512;
          const uint32_t a_lay = g.a_major == MAJOR_K ? 2 : 1, b_lay = g.b_major == MAJOR_K ? 2 : 1;
          const uint64_t da = make_desc(a_addr + a_off, a_lbo, a_sbo, a_lay);
          const uint64_t db = make_desc(b_addr + b_off, b_lbo, b_sbo, b_lay);
          const uint32_t first = (i > 0 || k > 0) ? 1u : 0u;
          if (PRECISE) {
            const uint64_t da_lo = make_desc(a_addr + C_::A_BYTES + a_off, a_lbo, a_sbo, a_lay);
            const uint64_t db_lo = make_desc(b_addr + C_::B_BYTES + b_off, b_lbo, b_sbo, b_lay);
            mma_tf32(tmem, da_lo, db, idesc, first);  // tail(A) * head(B)
            mma_tf32(tmem, da, db_lo, idesc, 1u);     // head(A) * tail(B)
            mma_tf32(tmem, da, db, idesc, 1u);        // head(A) * head(B)
          } else {
            mma_tf32(tmem, da, db, idesc, first);
          }
        }
        // frees the stage for the producers once the MMAs that read it have completed
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_empty[s]))
                     : "memory");
      }
      __syncwarp();
    }
    if (lane == 0) {
      if (ok)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_accum))
                     : "memory");
      else { s_abort = 1; atomicCAS(g.status, 0, TGNN_ETIMEOUT); }
    }
    __syncwarp();
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == MMA_WARP) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C_::TMEM_COLS) : "memory");
  }
}

// n-tiles of at most 256 columns, balanced, in whole 32-column atoms; narrower tiles (down to 64
// columns) when a store-mode product would otherwise occupy only a few SMs.
void tile_plan(int M, int N, bool split_accumulate, int* n_tiles, int* bn) {
  int nt = (N + 255) / 256;
  const int m_tiles = (M + BM - 1) / BM;
  // (only while the narrower tiles still make one wave of CTAs: a CTA takes a whole SM)
  if (!split_accumulate)
    while (m_tiles * (nt + 1) <= 148 && ((N + nt - 1) / nt + 31) / 32 * 32 > 64) ++nt;
  *n_tiles = nt;
  *bn = ((N + nt - 1) / nt + 31) / 32 * 32;
}

// Writes the B-operand images of every weight site from the current parameters.  One thread per
// 16-byte chunk: the same rounding / head-tail split and the same swizzled placement as load_tile.
__global__ void __launch_bounds__(256) prep_weights_kernel(const WeightSite* __restrict__ sites,
                                                           const float* __restrict__ params,
                                                           unsigned char* __restrict__ images) {
  const WeightSite st = sites[blockIdx.y];
  const int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (idx >= st.chunks) return;
  const int per_tile_kb = st.bn_t * 8;  // logical chunks per (tile, k-block)
  const int cidx = (int)(idx % per_tile_kb);
  const int64_t tk = idx / per_tile_kb;
  const int kb = (int)(tk % st.nkb), tile = (int)(tk / st.nkb);
  const int n0 = tile * st.bn;
  const int n_valid = min(st.bn, st.N - n0);
  const int n_mma = (n_valid + 15) / 16 * 16;
  const int copies = st.precise ? 2 : 1;
  const int b_bytes = st.bn_t * 128;
  unsigned char* img = images + st.image_off + ((int64_t)tile * st.nkb + kb) * copies * b_bytes;
  const float* W = params + st.w_off;
  float v[4] = {0.f, 0.f, 0.f, 0.f};
  uint32_t off;
  if (st.major == MAJOR_K) {
    const int r = cidx >> 3, c = cidx & 7;
    const int n = n0 + r, k = kb * BK + 4 * c;
    if (r < (n_mma + 7) / 8 * 8 && n < st.N)
      for (int e = 0; e < 4; ++e)
        if (k + e < st.K) v[e] = W[(int64_t)n * st.ld + k + e];
    off = (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4);
  } else {
    const int b_rows = (n_valid + 31) / 32 * 32;
    const int cpr = b_rows >> 2, atoms = b_rows >> 5;
    const int kk = cidx / cpr, cm = cidx - kk * cpr;
    if (kk >= BK) return;  // beyond the region this tile uses
    const int k = kb * BK + kk;
    for (int e = 0; e < 4; ++e) {
      const int n = n0 + 4 * cm + e;
      if (k < st.K && n < st.N) {
        const int col = n < st.n_split ? st.col0 + n : st.col1 + (n - st.n_split);
        v[e] = W[(int64_t)k * st.ld + col];
      }
    }
    const int a = cm >> 3, c = cm & 7;
    off = (kk >> 2) * (atoms * 512) + a * 512 + (kk & 3) * 128 + ((c ^ ((kk & 3) << 1)) << 4);
  }
  const uint32_t h0 = to_tf32(v[0]), h1 = to_tf32(v[1]), h2 = to_tf32(v[2]), h3 = to_tf32(v[3]);
  *reinterpret_cast<uint4*>(img + off) = make_uint4(h0, h1, h2, h3);
  if (st.precise)
    *reinterpret_cast<uint4*>(img + b_bytes + off) =
        make_uint4(to_tf32(v[0] - __uint_as_float(h0)), to_tf32(v[1] - __uint_as_float(h1)),
                   to_tf32(v[2] - __uint_as_float(h2)), to_tf32(v[3] - __uint_as_float(h3)));
}

template <int BN_T, bool PRECISE, bool FAST, int TMA>
int launch_tc(tgnn_ctx* ctx, const TcArgs& a, int n_tiles, const char* name, cudaStream_t s) {
  using C_ = Cfg<BN_T, PRECISE, TMA>;
  static SmemLimit smem_limit;   // one per template instance
  {
    const int rc = raise_smem_limit(ctx, gemm_tf32_kernel<BN_T, PRECISE, FAST, TMA>, C_::SMEM, smem_limit);
    if (rc) return rc;
  }
  dim3 grid(n_tiles, (a.M + BM - 1) / BM, a.split_k);
  {
    KernelScope scope__(ctx, name, s);
    gemm_tf32_kernel<BN_T, PRECISE, FAST, TMA><<<grid, C_::THREADS, C_::SMEM, s>>>(a);
  }
  TGNN_LAUNCH_OK(ctx, name);
  return TGNN_OK;
}

// The driver's tensor-map encoder, looked up once through the runtime (no link against the driver library);
// nullptr if it is unavailable.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn tensor_map_encoder() {
  static TensorMapEncodeFn enc = nullptr;
  static bool looked = false;
  if (!looked) {
    looked = true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      enc = reinterpret_cast<TensorMapEncodeFn>(fn);
    (void)cudaGetLastError();
  }
  return enc;
}

// Tiled tensor map of a row-major fp32 matrix [rows, cols] (row pitch ld floats): boxes of 32 columns x 128
// rows, 128-byte swizzle, zeros outside.  Returns false if the encoder is unavailable or refuses the shape.
bool encode_a_map(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, int64_t ld) {
  const TensorMapEncodeFn enc = tensor_map_encoder();
  if (!enc || rows <= 0 || cols <= 0) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  const cuuint32_t box[2] = {BK, BM};
  const cuuint32_t elem[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace {
// A row-major fp32 matrix [rows (contraction), cols] as the transposed operand of a product: a four-dimensional
// view (value within a 32-wide atom, row within a group of 4, atom, group) whose box of 32 x 4 x atoms x 8 lands
// in shared memory exactly as the MN-major operand tile is laid out: groups of 4 contraction rows, inside a group
// one 512-byte atom per 32 columns, 32-byte swizzle.  rows must be a multiple of 4; the last atom of a row may run
// past the row end (into the next row, or up to 124 bytes past the matrix).
bool encode_mn_map(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, int64_t ld, int box_atoms) {
  const TensorMapEncodeFn enc = tensor_map_encoder();
  if (!enc || rows <= 0 || cols <= 0 || rows % 4 != 0 || box_atoms < 1 || box_atoms > 8) return false;
  const cuuint64_t dims[4] = {32, 4, (cuuint64_t)((cols + 31) / 32), (cuuint64_t)(rows / 4)};
  const cuuint64_t strides[3] = {(cuuint64_t)ld * 4, 128, (cuuint64_t)ld * 16};
  const cuuint32_t box[4] = {32, 4, (cuuint32_t)box_atoms, BK / 4};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(base), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace

// Returns TGNN_OK after launching, or 1 if the product does not fit this kernel (caller falls back to the FMA tiles).
int launch_gemm_tf32(tgnn_ctx* ctx, const GemmArgs& g, const char* name, cudaStream_t s) {
  TcArgs a = {};
  if (g.a_cs == 1) { a.a_major = MAJOR_K; a.lda = g.a_rs; }
  else if (g.a_rs == 1) { a.a_major = MAJOR_MN; a.lda = g.a_cs; }
  else return 1;
  if (g.b_rs == 1) { a.b_major = MAJOR_K; a.ldb = g.b_cs; }
  else if (g.b_cs == 1) { a.b_major = MAJOR_MN; a.ldb = g.b_rs; }
  else return 1;
  if (g.rowsum_out && a.a_major != MAJOR_MN) return 1;
  a.A = g.A; a.B = g.B; a.C = g.C; a.ldc = g.ldc;
  a.M = g.M; a.N = g.N; a.K = g.K; a.dev_M = g.dev_M; a.dev_K = g.dev_K;
  a.bias = g.bias; a.rowsum_out = g.rowsum_out; a.relu = g.relu; a.accumulate = g.accumulate;
  a.status = ctx->ws.status;
  if (g.a_idx && a.a_major == MAJOR_K && g.a_tab_cols % 4 == 0 && (((uintptr_t)g.a_tab & 15) == 0)) {
    a.a_idx = g.a_idx; a.a_tab = g.a_tab; a.a_tab_cols = g.a_tab_cols;
    a.a_tab_rows = g.a_tab_rows > 0 ? g.a_tab_rows : ((int64_t)1 << 62);
  } else if (g.a_idx) {
    return 1;
  }
  int n_tiles, bn;
  bool precise = g.precise != 0;
  tile_plan(g.M, g.N, g.accumulate && g.split_k > 1, &n_tiles, &bn);
  if (g.site > 0 && ctx->images_fresh && ctx->images) {  // B is a weight matrix whose images are up to date
    const WeightSite& st = ctx->sites[g.site - 1];
    n_tiles = st.n_tiles; bn = st.bn; precise = st.precise != 0;
    a.b_image = ctx->images + st.image_off;
    a.b_tile_stride = (int64_t)st.nkb * (st.precise ? 2 : 1) * st.bn_t * 128;
    a.b_major = st.major;
  }
  a.split_k = 1;
  if (g.accumulate && g.split_k > 1) {
    // The caller allows split-K (weight gradients: leaves of the backward chain, run on a side stream).  The
    // CTAs fill about half the machine, with >= 4 stages of work each: the chain's own kernels keep the other
    // half, and fewer, longer CTAs pay the per-CTA set-up and the atomic epilogue less often.  Measured on
    // the wiki-shaped step: 148 CTAs 253.7 us, 74 CTAs 246.2 us; the batch-4000 workloads gain 1 - 3 %.
    const int tiles = n_tiles * ((g.M + BM - 1) / BM);
    const int max_s = (g.K + 4 * BK - 1) / (4 * BK);
    a.split_k = (74 + tiles - 1) / tiles;
    if (a.split_k > max_s) a.split_k = max_s;
    if (a.split_k < 1) a.split_k = 1;
  }
  // whole-chunk operands: 16-byte aligned rows, and the dimension the 16-byte chunks run along is a
  // multiple of 4 and known on the host
  // (An MN-major operand of a workspace buffer may end inside a chunk when its row pitch covers the chunk: the
  // values read past the end only reach rows or columns of C beyond M or N, which are not stored.)
  const bool slack = g.tail_slack != 0;
  const auto whole = [slack](const float* p, int64_t ld, int major, int k, const int* dev_k, int mn, const int* dev_mn) {
    if (((uintptr_t)p & 15) != 0 || ld % 4 != 0) return false;
    return major == MAJOR_K ? (k % 4 == 0 && dev_k == nullptr)
                            : ((mn % 4 == 0 || (slack && (mn + 3) / 4 * 4 <= ld)) && dev_mn == nullptr);
  };
  const bool fast = whole(a.A, a.lda, a.a_major, a.K, a.dev_K, a.M, a.dev_M) &&
                    (a.b_image != nullptr || whole(a.B, a.ldb, a.b_major, a.K, a.dev_K, a.N, nullptr));
  // activations as TMA tiles: K-major whole-chunk A beside a prepared weight image
  static const bool tma_off = getenv("TGNN_NO_TMA") != nullptr;  // debugging aid: activations through registers
  // (tiles need 16-byte aligned rows only: a ragged contraction length is the tensor map's edge, filled with zeros)
  const auto aligned = [](const float* p, int64_t ld) { return ((uintptr_t)p & 15) == 0 && ld % 4 == 0; };
  if (!tma_off && aligned(a.A, a.lda) && a.dev_K == nullptr && a.a_major == MAJOR_K && a.b_image != nullptr &&
      encode_a_map(&a.a_map, a.A, a.M, a.K, a.lda)) {
    a.a_tma = 1;
    if (precise) {
      if (bn <= 128) return launch_tc<128, true, true, 1>(ctx, a, n_tiles, name, s);
      return launch_tc<256, true, true, 1>(ctx, a, n_tiles, name, s);
    }
    if (bn <= 128) return launch_tc<128, false, true, 1>(ctx, a, n_tiles, name, s);
    return launch_tc<256, false, true, 1>(ctx, a, n_tiles, name, s);
  }
  // weight gradients: both operands transposed, contraction length static and a multiple of 4
  if (!tma_off && aligned(a.A, a.lda) && aligned(a.B, a.ldb) && precise && a.a_major == MAJOR_MN && a.b_major == MAJOR_MN &&
      a.b_image == nullptr &&
      a.dev_K == nullptr && a.K % 4 == 0 && bn % 32 == 0 &&
      (g.tail_slack || ((a.M + 31) / 32 * 32 <= a.lda && (a.N + 31) / 32 * 32 <= a.ldb)) &&  // no read past a caller's matrix
      encode_mn_map(&a.a_map, a.A, a.K, a.M, a.lda, BM / 32) && encode_mn_map(&a.b_map, a.B, a.K, a.N, a.ldb, bn / 32)) {
    a.a_tma = 2;
    a.b_box_atoms = bn / 32;
    if (bn <= 128) return launch_tc<128, true, true, 2>(ctx, a, n_tiles, name, s);
    return launch_tc<256, true, true, 2>(ctx, a, n_tiles, name, s);
  }
  const int sel = (precise ? 4 : 0) | (bn <= 128 ? 0 : 2) | (fast ? 1 : 0);
  switch (sel) {
    case 0: return launch_tc<128, false, false, 0>(ctx, a, n_tiles, name, s);
    case 1: return launch_tc<128, false, true, 0>(ctx, a, n_tiles, name, s);
    case 2: return launch_tc<256, false, false, 0>(ctx, a, n_tiles, name, s);
    case 3: return launch_tc<256, false, true, 0>(ctx, a, n_tiles, name, s);
    case 4: return launch_tc<128, true, false, 0>(ctx, a, n_tiles, name, s);
    case 5: return launch_tc<128, true, true, 0>(ctx, a, n_tiles, name, s);
    case 6: return launch_tc<256, true, false, 0>(ctx, a, n_tiles, name, s);
    default: return launch_tc<256, true, true, 0>(ctx, a, n_tiles, name, s);
  }
}

}  // namespace tgnn

namespace tgnn {

size_t plan_weight_sites(tgnn_ctx* ctx) {
  const ParamLayout& L = ctx->L;
  const int d = (int)L.d, de = (int)L.de;
  const bool all_precise = ctx->cfg.math_mode != TGNN_MATH_TF32_FAST;
  struct Def { int id; int64_t w_off, ld; int major, N, K, col0, n_split, col1, M_cap, split_acc, grad; };
  const int U = ctx->U_cap, R = ctx->R_cap, NB = ctx->NB_cap, Q2 = 2 * ctx->nq_cap;
  const int gd = (int)L.gates * d;              // rows of the update cell's matrices
  const int att = L.wo > L.wq ? 1 : 0;          // the attention block is empty for the time-projection model
  const Def defs[SITE_COUNT] = {
      {SITE_GI, L.gru_wi, L.dmsg, MAJOR_K, gd, (int)L.dmsg, 0, 0, 0, U, 1, 0},
      {SITE_GH, L.gru_wh, d, MAJOR_K, gd, d, 0, 0, 0, U, 0, 0},
      {SITE_KV, L.wk, L.dkv, MAJOR_K, att * 2 * d, (int)L.dkv, 0, 0, 0, NB, 0, 0},
      {SITE_Q, L.wq, 2 * d, MAJOR_K, att * d, 2 * d, 0, 0, 0, R, 0, 0},
      {SITE_OUT, L.wo, 2 * d, MAJOR_K, att * d, 2 * d, 0, 0, 0, R, 0, 0},
      {SITE_HEAD, L.w1, 2 * d, MAJOR_K, d, 2 * d, 0, 0, 0, Q2, 0, 0},
      {SITE_DCAT1, L.w1, 2 * d, MAJOR_MN, 2 * d, d, 0, 2 * d, 0, Q2, 0, 1},
      {SITE_DCATO, L.wo, 2 * d, MAJOR_MN, att * 2 * d, d, 0, 2 * d, 0, R, 0, 1},
      {SITE_DZQ, L.wq, 2 * d, MAJOR_MN, att * 2 * d, d, 0, 2 * d, 0, R, 0, 1},
      {SITE_DZ, L.wk, L.dkv, MAJOR_MN, att * 2 * d, 2 * d, 0, d, d + de, NB, 0, 1},
      {SITE_DXPHI, L.gru_wi, L.dmsg, MAJOR_MN, d, gd, 2 * d + de, d, 0, U, 0, 1},
  };
  size_t off = 0;
  for (const Def& f : defs) {
    WeightSite& st = ctx->sites[f.id];
    if (f.N == 0) {  // a projection this model does not have: an empty image
      st = WeightSite{};
      st.image_off = (int64_t)off;
      continue;
    }
    st.w_off = f.w_off; st.ld = f.ld; st.major = f.major; st.N = f.N; st.K = f.K;
    st.col0 = f.col0; st.n_split = f.n_split; st.col1 = f.col1;
    st.precise = (all_precise || f.grad) ? 1 : 0;
    tile_plan(f.M_cap, f.N, f.split_acc != 0, &st.n_tiles, &st.bn);
    st.bn_t = st.bn <= 128 ? 128 : 256;
    st.nkb = (f.K + BK - 1) / BK;
    st.image_off = (int64_t)off;
    st.chunks = (int64_t)st.n_tiles * st.nkb * st.bn_t * 8;
    off += (size_t)st.n_tiles * st.nkb * (st.precise ? 2 : 1) * st.bn_t * 128;
  }
  return off;
}

int launch_prep_weights(tgnn_ctx* ctx, cudaStream_t s) {
  if (!ctx->images || ctx->cfg.math_mode == TGNN_MATH_FP32) return TGNN_OK;
  int64_t mx = 0;
  for (int i = 0; i < SITE_COUNT; ++i) mx = ctx->sites[i].chunks > mx ? ctx->sites[i].chunks : mx;
  dim3 grid((unsigned)((mx + 255) / 256), SITE_COUNT);
  {
    KernelScope scope__(ctx, "prep_weights", s);
    prep_weights_kernel<<<grid, 256, 0, s>>>(ctx->sites_dev, ctx->params, ctx->images);
  }
  TGNN_LAUNCH_OK(ctx, "prep_weights");
  const int rch = launch_prep_head(ctx, s);    // W_1 transposed, for the tile form of the link-prediction head
  if (rch) return rch;
  return launch_prep_split_weights(ctx, s);   // the split planes of the key/value weights, when that mode is on
}

}  // namespace tgnn
