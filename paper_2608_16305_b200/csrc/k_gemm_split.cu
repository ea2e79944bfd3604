// The large projections on the 5th-generation tensor cores with split 16-bit operands (TGNN_MATH_F16X3).
//
// An fp32 value x is held as two 16-bit numbers, hi = r16(x) and lo = r16(x - hi).  With fp16 planes (what the
// library uses) they carry 22 mantissa bits for values inside fp16's range -- activations and weights as they are,
// gradients after multiplication by a power of two that the epilogue divides out again; with bf16 planes 16 bits
// at any range.  A product A B is then three tensor-core passes at the 16-bit rate,
//   lo(A) hi(B) + hi(A) lo(B) + hi(A) hi(B),
// with fp32 accumulation in tensor memory: the accuracy of the three-pass TF32 split at half its tensor time.  (One
// MMA cannot mix an fp16 operand with a bf16 one -- the hardware rejects it as an illegal instruction -- so both
// operands of a product use the same plane format.)  The operands are STORED split (two planes of the same shape,
// written by the kernel that produces the activation), so this kernel never touches operand data with a thread:
// tiles go from global memory to shared memory by the tensor-memory-access unit, already in the 128-byte-swizzled
// layout the MMA descriptors expect, and from there into the tensor cores.
//
// Roles (320 threads): warp 0 issues the tile copies (one per operand tile: the box spans both planes), warp 1 owns tensor memory and issues the MMAs,
// warps 2-9 are the epilogue (tensor memory -> registers -> a small staging square -> global memory in
// whole 64-byte row segments, with bias / ReLU or an atomic accumulate).
//
// A CTA is persistent: it takes a contiguous range of tile units (n-tile / contraction-split combination major,
// 128-row tile minor).  Activation x weight products walk it one row tile at a time with the accumulator
// alternating between the two halves of tensor memory, so the epilogue of one tile (a full store of C) runs
// while the MMAs of the next are issued.  Weight gradients (one long contraction range per CTA) take two row
// tiles at once, which share every B tile; their accumulators sit side by side.  A tiles and B tiles travel
// through two separate rings of shared-memory slots, each slot with a full (copy landed) and an empty (MMAs that
// read it retired, signalled by tcgen05.commit) mbarrier, so copies run several slots ahead of the MMAs and across
// item boundaries.  Every wait is bounded: on expiry the kernel records TGNN_ETIMEOUT, all roles leave their
// loops, tensor memory is freed and the kernel returns.
//
// Operand layouts.  K-major (the contraction index is contiguous in memory: activations [M, K] and weight
// planes [N, K]): a box of 64 elements x rows lands as rows of 128 bytes, 16-byte chunks XOR-swizzled
// by (row mod 8); one MMA step (16 elements) advances 32 bytes inside the row.  MN-major (the row / column
// index of C is contiguous: both operands of a weight gradient, whose contraction runs over matrix rows): a
// box of 64 columns x 32 contraction rows per 64-column chunk lands the same way with the roles swapped,
// which is the canonical MN-major layout of the 128-byte swizzle: chunks LBO apart, groups of 8 contraction
// rows SBO = 1024 bytes apart; one MMA step consumes two such groups.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "tgnn_internal.cuh"

namespace tgnn {
namespace {

constexpr int BM = 128;           // rows of C per tile (UMMA M)
constexpr int ACC_STRIDE = 256;   // tensor-memory columns between the two accumulators of a pair
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int MAX_SLOTS = 8;
constexpr int STG_PITCH = 20;     // floats between rows of a staged 32 x 16 square (16-byte aligned, bank-staggered)
constexpr int STG_WARP_BYTES = 4096;   // per epilogue warp: a 32 x 32 fp32 square for a bulk store (or the 32 x 16 square of the plain path)
constexpr int STG_BYTES = EPI_WARPS * STG_WARP_BYTES;
constexpr unsigned SPIN_LIMIT = 1u << 22;
constexpr int SMEM_LIMIT = 227 * 1024;

struct BfArgs {
  CUtensorMap a_map, b_map;   // three-dimensional: (contiguous index, row, plane)
  CUtensorMap c_map;          // C as (column, row) in boxes of 32 x 32 fp32 values, 128-byte swizzle (valid when c_bulk)
  int c_bulk;                 // C is 16-byte aligned with a pitch that is a multiple of 16 bytes: the epilogue stores (or
                              // reduces) whole 32 x 32 squares from shared memory with the tensor-memory-access unit
  float* C; int64_t ldc;
  int M, N, K;
  const float* bias;
  int relu, accumulate;
  int mn_major;               // 0: both operands K-major; 1: both MN-major
  int fp16;                   // both operands' planes hold fp16 numbers (bf16 otherwise; the two may not be mixed)
  int planes;                 // 2: hi and lo planes, three passes per product; 1: only the hi planes are read, one pass
  float out_scale;            // the product is multiplied by this (undoes the operands' power-of-two scales)
  int single;                 // work items are single row tiles whose accumulators alternate between the two halves of
                              // tensor memory, so that the epilogue of one overlaps the MMAs of the next (B tiles are
                              // then fetched once per row tile instead of once per pair)
  int m_tiles, n_tiles, bn, split_k;
  int kb_total;               // contraction blocks (64 elements K-major, 32 rows MN-major)
  int kb_begin, kb_end;       // the part of them this launch covers (a long weight gradient goes out as several launches)
  int ksteps_total;           // MMA steps of 16 over the whole contraction
  int a_slot_bytes, b_slot_bytes, n_a_slots, n_b_slots;
  int b_chunks;               // MN-major: 64-column chunks per B tile
  int stage_bytes, n_stages;  // CTA-pair kernel: one ring of stages, each an A tile (both planes) followed by this CTA's half of the B tile
  // accumulate mode: column `extra_col` of the product (if >= 0) is added to extra_out[row] instead of C --
  // a column of ones appended to B turns that column into the row sums of A, i.e. a bias gradient
  int extra_col;
  float* extra_out;
  int32_t* status;
  long long* trace;           // debug: clock stamps of CTA 0 (nullptr in normal use)
  int debug_withhold;         // test hook: the MMA warp skips this many slot releases (an empty-slot wait then expires)
  unsigned spin_limit;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity; gives up early when another role has already aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned limit, volatile int* abort_flag) {
  for (unsigned it = 0; it < limit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if ((it & 63) == 63 && *abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void tma_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void mma_f16(uint32_t tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void commit_to(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define TRACE(slot)                                                          \
  do {                                                                       \
    if (g.trace != nullptr && blockIdx.x == 0 && (slot) < 512) g.trace[slot] = clock64(); \
  } while (0)

struct Item {
  int mt0, tiles, n0, n_valid, kb0, kb1;
};
// A CTA's share of the work: a contiguous range of "tile units" (n-tile / contraction-split combination
// major, 128-row tile minor), walked in pairs of row tiles that share their B tiles; a pair never spans two
// combinations, and the last unit of a range may be a single tile.  All roles walk the same sequence.
struct Walk {
  int u, u_end;
};
__device__ __forceinline__ Walk cta_walk(const BfArgs& g) {
  const long long T = (long long)g.m_tiles * g.n_tiles * g.split_k;
  Walk w;
  w.u = (int)(T * blockIdx.x / gridDim.x);
  w.u_end = (int)(T * (blockIdx.x + 1) / gridDim.x);
  return w;
}
__device__ __forceinline__ bool next_item(const BfArgs& g, Walk& wk, Item& it) {
  while (wk.u < wk.u_end) {
    const int combo = wk.u / g.m_tiles, mt = wk.u - combo * g.m_tiles;
    it.mt0 = mt;
    it.tiles = g.single ? 1 : min(2, min(wk.u_end - wk.u, g.m_tiles - mt));
    wk.u += it.tiles;
    const int nt = combo % g.n_tiles, sp = combo / g.n_tiles;
    it.n0 = nt * g.bn;
    it.n_valid = nt == g.n_tiles - 1 ? g.N - it.n0 : g.bn;
    const int per = (g.kb_end - g.kb_begin + g.split_k - 1) / g.split_k;
    it.kb0 = g.kb_begin + sp * per;
    it.kb1 = min(g.kb_end, it.kb0 + per);
    if (it.kb0 < it.kb1) return true;   // an empty contraction range is skipped by every role alike
  }
  return false;
}
__device__ __forceinline__ void tma_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

// One epilogue warp's share of a finished 128-row accumulator: columns c_first, c_first + c_step, ... (groups of 32)
// of the lane quarter q4, from tensor memory through the warp's staging square to C (bias / ReLU / scale, or an
// atomic accumulate).
__device__ __forceinline__ void drain_tile(const BfArgs& g, const Item& it, int m0, uint32_t taddr, int c_first, int c_step,
                                           float* stg, int lane, int q4, bool c_vec) {
  const int sub = lane >> 2, ch = lane & 3;
  const bool with_bias = g.bias != nullptr && it.kb0 == 0;   // (the bias goes in with the first contraction block)
  const bool edge_tile = it.n0 + it.n_valid >= g.N;          // columns past n_valid lie outside C (and are clipped)
  for (int c0 = c_first; c0 < it.n_valid; c0 += c_step) {
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
    if (g.c_bulk && (edge_tile || c0 + 32 <= it.n_valid)) {
      // Bulk path: the lane holds 32 consecutive columns of its row; it finishes them (scale, bias, ReLU) and
      // writes them as one 128-byte row of a swizzled 32 x 32 square, which one bulk tensor store (or fp32
      // add-reduction) moves to C; rows past M and columns past N are clipped by the tensor map.
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the square is free again
      __syncwarp();
      float* row_p = stg + lane * 32;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 v = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]),
                               __uint_as_float(r[4 * q + 3]));
        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (with_bias) {
          const int col = c0 + 4 * q;
          const float* bp = g.bias + it.n0 + col;
          if (col < it.n_valid) b4.x = __ldg(bp);
          if (col + 1 < it.n_valid) b4.y = __ldg(bp + 1);
          if (col + 2 < it.n_valid) b4.z = __ldg(bp + 2);
          if (col + 3 < it.n_valid) b4.w = __ldg(bp + 3);
        }
        v.x = fmaf(v.x, g.out_scale, b4.x); v.y = fmaf(v.y, g.out_scale, b4.y);
        v.z = fmaf(v.z, g.out_scale, b4.z); v.w = fmaf(v.w, g.out_scale, b4.w);
        if (g.relu && !g.accumulate) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
        *reinterpret_cast<float4*>(row_p + 4 * (q ^ (lane & 7))) = v;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        const int x = it.n0 + c0, y = m0 + q4 * 32;
        if (g.accumulate)
          asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                       ::"l"(&g.c_map), "r"(x), "r"(y), "r"(smem_u32(stg)) : "memory");
        else
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                       ::"l"(&g.c_map), "r"(x), "r"(y), "r"(smem_u32(stg)) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
      continue;
    }
    if (g.c_bulk) {   // the plain path reuses the square: an earlier bulk store must have read it
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      __syncwarp();
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int cb0 = c0 + 16 * h;
      if (cb0 >= it.n_valid) break;   // warp-uniform
#pragma unroll
      for (int q = 0; q < 4; ++q)
        *reinterpret_cast<uint4*>(stg + lane * STG_PITCH + 4 * q) =
            make_uint4(r[16 * h + 4 * q], r[16 * h + 4 * q + 1], r[16 * h + 4 * q + 2], r[16 * h + 4 * q + 3]);
      __syncwarp();
      const int col = cb0 + 4 * ch;   // first of this lane's four columns, relative to the tile
      float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
      if (with_bias && col < it.n_valid) {
        const float* bp = g.bias + it.n0 + col;
        b4.x = bp[0];
        if (col + 1 < it.n_valid) b4.y = bp[1];
        if (col + 2 < it.n_valid) b4.z = bp[2];
        if (col + 3 < it.n_valid) b4.w = bp[3];
      }
      const int xc = g.extra_col - it.n0 - col;   // 0..3: one of this lane's columns is the extra column
      const bool full4 = col + 3 < it.n_valid && (xc < 0 || xc > 3);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int rr = j * 8 + sub;
        const int row = m0 + q4 * 32 + rr;
        float4 v = *reinterpret_cast<const float4*>(stg + rr * STG_PITCH + 4 * ch);
        if (row < g.M && col < it.n_valid) {
          v.x = fmaf(v.x, g.out_scale, b4.x); v.y = fmaf(v.y, g.out_scale, b4.y);
          v.z = fmaf(v.z, g.out_scale, b4.z); v.w = fmaf(v.w, g.out_scale, b4.w);
          float* cp = g.C + (int64_t)row * g.ldc + it.n0 + col;
          if (g.accumulate) {
            if (full4 && c_vec) {
              atomicAdd(reinterpret_cast<float4*>(cp), v);
            } else {
              const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int e2 = 0; e2 < 4; ++e2)
                if (col + e2 < it.n_valid) atomicAdd(e2 == xc ? g.extra_out + row : cp + e2, vv[e2]);
            }
          } else {
            if (g.relu) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
            if (full4 && c_vec) {
              *reinterpret_cast<float4*>(cp) = v;
            } else {
              cp[0] = v.x;
              if (col + 1 < it.n_valid) cp[1] = v.y;
              if (col + 2 < it.n_valid) cp[2] = v.z;
              if (col + 3 < it.n_valid) cp[3] = v.w;
            }
          }
        }
      }
      __syncwarp();
    }
  }
}

__global__ void __launch_bounds__(THREADS, 1) gemm_split_kernel(const __grid_constant__ BfArgs g) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_full_a[MAX_SLOTS], s_empty_a[MAX_SLOTS], s_full_b[MAX_SLOTS], s_empty_b[MAX_SLOTS];
  __shared__ __align__(8) uint64_t s_tmem_full[2], s_tmem_empty[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t a_ring = smem_u32(smem);
  const uint32_t b_ring = a_ring + (uint32_t)(g.n_a_slots * g.a_slot_bytes);
  float* stg_base = reinterpret_cast<float*>(smem + (size_t)g.n_a_slots * g.a_slot_bytes + (size_t)g.n_b_slots * g.b_slot_bytes);

  if (tid == 0) {
    for (int s = 0; s < MAX_SLOTS; ++s) {
      mbar_init(smem_u32(&s_full_a[s]), 1); mbar_init(smem_u32(&s_empty_a[s]), 1);
      mbar_init(smem_u32(&s_full_b[s]), 1); mbar_init(smem_u32(&s_empty_b[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&s_tmem_full[b]), 1);
      mbar_init(smem_u32(&s_tmem_empty[b]), EPI_WARPS);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  if (tid == 0) TRACE(0);
  volatile int* abort_flag = &s_abort;
  const unsigned limit = g.spin_limit;

  const int ks_per_kb = g.mn_major ? 2 : 4;

  if (warp == 0) {
    // ------------------------------------------------------------ tile copies
    if (lane == 0) {
      uint32_t ca = 0, cb = 0;
      bool ok = true;
      const uint32_t a_bytes = (uint32_t)g.a_slot_bytes, b_bytes = (uint32_t)g.b_slot_bytes;
      Walk wk = cta_walk(g);
      Item it;
      while (ok && next_item(g, wk, it)) {
        for (int kb = it.kb0; kb < it.kb1 && ok; ++kb) {
          {
            const uint32_t s = cb % (uint32_t)g.n_b_slots;
            ok = mbar_wait(smem_u32(&s_empty_b[s]), ((cb / (uint32_t)g.n_b_slots) & 1u) ^ 1u, limit, abort_flag);
            if (!ok) break;
            const uint32_t bar = smem_u32(&s_full_b[s]), dst = b_ring + s * b_bytes;
            mbar_expect_tx(bar, b_bytes);
            // one copy brings both planes of the tile (the box spans the plane dimension)
            if (!g.mn_major) tma_3d(dst, &g.b_map, kb * 64, it.n0, 0, bar);
            else tma_4d(dst, &g.b_map, 0, kb * 32, it.n0 >> 6, 0, bar);
            ++cb;
          }
          for (int t = 0; t < it.tiles && ok; ++t) {
            const uint32_t s = ca % (uint32_t)g.n_a_slots;
            ok = mbar_wait(smem_u32(&s_empty_a[s]), ((ca / (uint32_t)g.n_a_slots) & 1u) ^ 1u, limit, abort_flag);
            if (!ok) break;
            const uint32_t bar = smem_u32(&s_full_a[s]), dst = a_ring + s * a_bytes;
            const int m0 = (it.mt0 + t) * BM;
            mbar_expect_tx(bar, a_bytes);
            if (!g.mn_major) tma_3d(dst, &g.a_map, kb * 64, m0, 0, bar);
            else tma_4d(dst, &g.a_map, 0, kb * 32, m0 >> 6, 0, bar);
            TRACE(256 + (int)ca);
            ++ca;
          }
        }
      }
      if (!ok) { s_abort = 1; atomicCAS(g.status, 0, TGNN_ETIMEOUT); }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t ca = 0, cb = 0, n_item = 0;
      int withheld = 0;
      bool ok = true;
      const uint32_t a_bytes = (uint32_t)g.a_slot_bytes, b_bytes = (uint32_t)g.b_slot_bytes;
      const uint32_t a_plane = a_bytes / (uint32_t)g.planes, b_plane = b_bytes / (uint32_t)g.planes;
      const bool three = g.planes == 2;
      const uint32_t mn = g.mn_major ? 1u : 0u;
      // K-major: 8-row groups 1024 B apart (SBO), a step advances 32 B.  MN-major: 64-column chunks 4096 B apart
      // (LBO), 8-row contraction groups 1024 B apart (SBO), a step advances two groups.
      const uint32_t lbo = mn ? 4096u : 16u, sbo = 1024u, kstep_bytes = mn ? 2048u : 32u;
      Walk wk = cta_walk(g);
      Item it;
      while (ok && next_item(g, wk, it)) {
        const uint32_t buf = g.single ? (n_item & 1u) : 0u, use = g.single ? (n_item >> 1) : n_item;
        ok = mbar_wait(smem_u32(&s_tmem_empty[buf]), (use & 1u) ^ 1u, limit, abort_flag);   // accumulators drained
        if (!ok) break;
        ++n_item;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int n_mma = (it.n_valid + 15) / 16 * 16;
        // instruction descriptor: D fp32; A and B formats (the same for both: 1 = bf16, 0 = fp16 -- an MMA that
        // mixes the two is an illegal instruction); majors; N >> 3; M >> 4
        const uint32_t fmt = g.fp16 ? 0u : 1u;
        const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (mn << 15) | (mn << 16) |
                               ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        for (int kb = it.kb0; kb < it.kb1 && ok; ++kb) {
          const uint32_t sb = cb % (uint32_t)g.n_b_slots;
          ok = mbar_wait(smem_u32(&s_full_b[sb]), (cb / (uint32_t)g.n_b_slots) & 1u, limit, abort_flag);
          if (!ok) break;
          const uint32_t b_addr = b_ring + sb * b_bytes;
          const int ks_n = min(ks_per_kb, g.ksteps_total - kb * ks_per_kb);
          for (int t = 0; t < it.tiles && ok; ++t) {
            const uint32_t sa = ca % (uint32_t)g.n_a_slots;
            ok = mbar_wait(smem_u32(&s_full_a[sa]), (ca / (uint32_t)g.n_a_slots) & 1u, limit, abort_flag);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            TRACE(16 + 2 * (int)ca);
            const uint32_t a_addr = a_ring + sa * a_bytes;
            const uint32_t acc = tmem + (uint32_t)((g.single ? (int)buf : t) * ACC_STRIDE);
            for (int ks = 0; ks < ks_n; ++ks) {
              const uint64_t da_hi = make_desc(a_addr + ks * kstep_bytes, lbo, sbo);
              const uint64_t da_lo = make_desc(a_addr + a_plane + ks * kstep_bytes, lbo, sbo);
              const uint64_t db_hi = make_desc(b_addr + ks * kstep_bytes, lbo, sbo);
              const uint64_t db_lo = make_desc(b_addr + b_plane + ks * kstep_bytes, lbo, sbo);
              const uint32_t first = (kb > it.kb0 || ks > 0) ? 1u : 0u;
              if (three) {
                mma_f16(acc, da_lo, db_hi, idesc, first);
                mma_f16(acc, da_hi, db_lo, idesc, 1u);
              }
              mma_f16(acc, da_hi, db_hi, idesc, three ? 1u : first);
            }
            TRACE(17 + 2 * (int)ca);
            if (withheld < g.debug_withhold) ++withheld;   // test hook: this slot is never handed back
            else commit_to(smem_u32(&s_empty_a[sa]));
            ++ca;
          }
          if (ok) commit_to(smem_u32(&s_empty_b[sb]));
          ++cb;
        }
        if (ok) commit_to(smem_u32(&s_tmem_full[buf]));
      }
      if (!ok) { s_abort = 1; atomicCAS(g.status, 0, TGNN_ETIMEOUT); }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue
    const int e = warp - 2;
    const int t = e >> 2;          // which accumulator of the pair
    const int q4 = warp & 3;       // the tensor-memory lane quarter this warp may read
    float* stg = stg_base + e * (STG_WARP_BYTES / 4);
    const bool c_vec = (((uintptr_t)g.C & 15) == 0) && (g.ldc % 4 == 0);
    uint32_t n_item = 0;
    bool ok = true;
    Walk wk = cta_walk(g);
    Item it;
    while (ok && next_item(g, wk, it)) {
      const uint32_t buf = g.single ? (n_item & 1u) : 0u, use = g.single ? (n_item >> 1) : n_item;
      ok = mbar_wait(smem_u32(&s_tmem_full[buf]), use & 1u, limit, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) TRACE(2 + 2 * (int)n_item);
      ++n_item;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // pairs: warps 2-5 drain the first tile's accumulator, 6-9 the second's.  Single tiles: all eight warps
      // drain the one accumulator, the two warps of a lane quarter taking alternate 32-column groups.
      const int acc_i = g.single ? (int)buf : t;
      const int c_first = g.single ? 32 * t : 0, c_step = g.single ? 64 : 32;
      if (g.single || t < it.tiles) {
        const int m0 = (it.mt0 + (g.single ? 0 : t)) * BM;
        const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(acc_i * ACC_STRIDE);
        drain_tile(g, it, m0, taddr, c_first, c_step, stg, lane, q4, c_vec);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (e == 0 && lane == 0) TRACE(1 + 2 * (int)n_item);
      if (lane == 0) mbar_arrive(smem_u32(&s_tmem_empty[buf]));
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this warp's bulk stores have landed
    if (!ok && lane == 0) { s_abort = 1; atomicCAS(g.status, 0, TGNN_ETIMEOUT); }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (s_abort && warp == 0) {
    // copies this CTA asked for may still be on their way into its shared memory: give them a bounded while
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// ---- CTA pairs (a cluster of two CTAs on the two SMs of one processing cluster, one 256-row MMA across both) ----
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the shared::cluster address of the same shared-memory location in the CTA of rank `rank`
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// tile copy into this CTA's shared memory whose completion is counted on a barrier of the pair's leader
__device__ __forceinline__ void tma_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(cluster_bar)
      : "memory");
}
__device__ __forceinline__ void tma_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t cluster_bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(cluster_bar)
      : "memory");
}
__device__ __forceinline__ void mma_f16_pair(uint32_t tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc)
      : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far have retired
__device__ __forceinline__ void commit_to_pair(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(both) : "memory");
}

// The walk of a CTA pair: a contiguous range of units (n-tile major, 256-row tile minor), one unit per item.
__device__ __forceinline__ Walk pair_walk(const BfArgs& g) {
  const long long T = (long long)g.m_tiles * g.n_tiles;
  const unsigned c = blockIdx.x >> 1, nc = gridDim.x >> 1;
  Walk w;
  w.u = (int)(T * c / nc);
  w.u_end = (int)(T * (c + 1) / nc);
  return w;
}
__device__ __forceinline__ bool next_pair_item(const BfArgs& g, Walk& wk, Item& it) {
  if (wk.u >= wk.u_end) return false;
  const int nt = wk.u / g.m_tiles;
  it.mt0 = wk.u - nt * g.m_tiles;
  it.tiles = 1;
  ++wk.u;
  it.n0 = nt * g.bn;
  it.n_valid = nt == g.n_tiles - 1 ? g.N - it.n0 : g.bn;
  it.kb0 = 0;
  it.kb1 = g.kb_total;
  return true;
}

// K-major products with many row tiles, on pairs of CTAs.  A work item is a 256-row tile of C: each CTA of the
// pair loads its own 128 rows of A and HALF of the B tile (the leader the first n/2 rows of the [n, K] operand,
// its peer the second half), the leader issues one MMA of 256 rows for both, and each CTA finds its 128 rows of
// the accumulator in its own tensor memory and stores them.  Per flop a CTA pulls 58 KB instead of 84 KB through
// its shared memory for a 208-column tile, and the accumulators still alternate between two halves of tensor
// memory so that a tile's epilogue runs beside the next tile's MMAs.  Barriers: a stage's full barrier lives in the
// leader and counts the bytes of both CTAs' copies; its empty barrier and the accumulator-full barriers live in
// both CTAs and are signalled together by a multicast commit; the accumulator-empty barriers live in the leader
// and collect the epilogue warps of both CTAs.  Every wait is bounded as in the single-CTA kernel; a CTA that gives
// up also raises its peer's abort flag, and both meet at the cluster barrier before tensor memory is freed.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1) gemm_split_pair_kernel(const __grid_constant__ BfArgs g) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_full[MAX_SLOTS], s_empty[MAX_SLOTS];
  __shared__ __align__(8) uint64_t s_tmem_full[2], s_tmem_empty[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t ring = smem_u32(smem);
  float* stg_base = reinterpret_cast<float*>(smem + (size_t)g.n_stages * g.stage_bytes);

  if (tid == 0) {
    for (int s = 0; s < MAX_SLOTS; ++s) {
      mbar_init(smem_u32(&s_full[s]), 1);    // the leader's own arrive with the byte count of both CTAs' copies
      mbar_init(smem_u32(&s_empty[s]), 1);   // one multicast commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&s_tmem_full[b]), 1);
      mbar_init(smem_u32(&s_tmem_empty[b]), 2 * EPI_WARPS);   // (used in the leader: epilogue warps of both CTAs)
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // both CTAs of the pair take part in the pair-wide allocation
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();   // the peer's barriers are initialised before anything is counted on them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  if (tid == 0) TRACE(0);
  volatile int* abort_flag = &s_abort;
  const unsigned limit = g.spin_limit;
  const uint32_t stage_bytes = (uint32_t)g.stage_bytes, n_stages = (uint32_t)g.n_stages;
  const uint32_t planes = (uint32_t)g.planes;
  const uint32_t a_bytes = planes * BM * 128u;                  // the A tile (all its planes)
  const uint32_t b_plane = (stage_bytes - a_bytes) / planes;    // one plane of this CTA's half of the B tile
  const int b_rows = (int)(b_plane >> 7);                  // rows of the copied half (the widest n-tile's)

  if (warp == 0) {
    // ------------------------------------------------------------ tile copies (each CTA its own)
    if (lane == 0) {
      uint32_t c = 0;
      bool ok = true;
      Walk wk = pair_walk(g);
      Item it;
      (void)b_rows;
      while (ok && next_pair_item(g, wk, it)) {
        const int n_mma = (it.n_valid + 15) / 16 * 16;
        const int m0 = (2 * it.mt0 + (int)rank) * BM;
        const int nb0 = it.n0 + (int)rank * (n_mma >> 1);   // first B row of this CTA's half
        for (int kb = it.kb0; kb < it.kb1 && ok; ++kb) {
          const uint32_t s = c % n_stages;
          ok = mbar_wait(smem_u32(&s_empty[s]), ((c / n_stages) & 1u) ^ 1u, limit, abort_flag);
          if (!ok) break;
          const uint32_t dst = ring + s * stage_bytes;
          const uint32_t bar = peer_addr(smem_u32(&s_full[s]), 0);
          if (leader) mbar_expect_tx(smem_u32(&s_full[s]), 2u * stage_bytes);
          tma_3d_pair(dst, &g.a_map, kb * 64, m0, 0, bar);
          tma_3d_pair(dst + a_bytes, &g.b_map, kb * 64, nb0, 0, bar);
          TRACE(256 + (int)c);
          ++c;
        }
      }
      if (!ok) {
        s_abort = 1;
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(smem_u32(&s_abort), rank ^ 1u)), "r"(1) : "memory");
        atomicCAS(g.status, 0, TGNN_ETIMEOUT);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (the leader's, for both CTAs)
    if (lane == 0 && leader) {
      uint32_t c = 0, n_item = 0;
      int withheld = 0;
      bool ok = true;
      Walk wk = pair_walk(g);
      Item it;
      while (ok && next_pair_item(g, wk, it)) {
        const uint32_t buf = n_item & 1u, use = n_item >> 1;
        ok = mbar_wait(smem_u32(&s_tmem_empty[buf]), (use & 1u) ^ 1u, limit, abort_flag);   // drained in both CTAs
        if (!ok) break;
        ++n_item;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int n_mma = (it.n_valid + 15) / 16 * 16;
        const uint32_t fmt = g.fp16 ? 0u : 1u;
        const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(n_mma >> 3) << 17) |
                               ((uint32_t)((2 * BM) >> 4) << 24);
        const uint32_t acc = tmem + buf * (uint32_t)ACC_STRIDE;
        for (int kb = it.kb0; kb < it.kb1 && ok; ++kb) {
          const uint32_t s = c % n_stages;
          ok = mbar_wait(smem_u32(&s_full[s]), (c / n_stages) & 1u, limit, abort_flag);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          TRACE(16 + 2 * (int)c);
          const uint32_t a_addr = ring + s * stage_bytes, b_addr = a_addr + a_bytes;
          const int ks_n = min(4, g.ksteps_total - kb * 4);
          for (int ks = 0; ks < ks_n; ++ks) {
            const uint64_t da_hi = make_desc(a_addr + ks * 32u, 16u, 1024u);
            const uint64_t da_lo = make_desc(a_addr + BM * 128u + ks * 32u, 16u, 1024u);
            const uint64_t db_hi = make_desc(b_addr + ks * 32u, 16u, 1024u);
            const uint64_t db_lo = make_desc(b_addr + b_plane + ks * 32u, 16u, 1024u);
            const uint32_t first = (kb > it.kb0 || ks > 0) ? 1u : 0u;
            if (planes == 2u) {
              mma_f16_pair(acc, da_lo, db_hi, idesc, first);
              mma_f16_pair(acc, da_hi, db_lo, idesc, 1u);
            }
            mma_f16_pair(acc, da_hi, db_hi, idesc, planes == 2u ? 1u : first);
          }
          TRACE(17 + 2 * (int)c);
          if (withheld < g.debug_withhold) ++withheld;   // test hook: this stage is never handed back
          else commit_to_pair(smem_u32(&s_empty[s]));
          ++c;
        }
        if (ok) commit_to_pair(smem_u32(&s_tmem_full[buf]));
      }
      if (!ok) {
        s_abort = 1;
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(smem_u32(&s_abort), 1u)), "r"(1) : "memory");
        atomicCAS(g.status, 0, TGNN_ETIMEOUT);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue (each CTA its own 128 rows)
    const int e = warp - 2;
    const int t = e >> 2;
    const int q4 = warp & 3;
    float* stg = stg_base + e * (STG_WARP_BYTES / 4);
    const bool c_vec = (((uintptr_t)g.C & 15) == 0) && (g.ldc % 4 == 0);
    const uint32_t empty0 = peer_addr(smem_u32(&s_tmem_empty[0]), 0), empty1 = peer_addr(smem_u32(&s_tmem_empty[1]), 0);
    uint32_t n_item = 0;
    bool ok = true;
    Walk wk = pair_walk(g);
    Item it;
    while (ok && next_pair_item(g, wk, it)) {
      const uint32_t buf = n_item & 1u, use = n_item >> 1;
      ok = mbar_wait(smem_u32(&s_tmem_full[buf]), use & 1u, limit, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) TRACE(2 + 2 * (int)n_item);
      ++n_item;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int m0 = (2 * it.mt0 + (int)rank) * BM;
      const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + buf * (uint32_t)ACC_STRIDE;
      drain_tile(g, it, m0, taddr, 32 * t, 64, stg, lane, q4, c_vec);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (e == 0 && lane == 0) TRACE(1 + 2 * (int)n_item);
      if (lane == 0) mbar_arrive_cluster(buf ? empty1 : empty0);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this warp's bulk stores have landed
    if (!ok && lane == 0) {
      s_abort = 1;
      asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(smem_u32(&s_abort), rank ^ 1u)), "r"(1) : "memory");
      atomicCAS(g.status, 0, TGNN_ETIMEOUT);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (s_abort && warp == 0) {
    // copies this CTA asked for may still be on their way into its shared memory: give them a bounded while
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  __syncthreads();
  // neither CTA frees tensor memory or leaves while its peer's MMAs, commits or arrivals may still touch it
  cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// Weight gradients (both operands MN-major, C = A^T B accumulated over a long contraction) on pairs of CTAs.
// A pair owns a 256-row tile of C -- all of it, up to 512 columns, as two accumulators of 256 columns side by side
// in each CTA's tensor memory -- and a range of the contraction.  Per block of 32 contraction rows a CTA loads its
// own 128 columns of A (its rows of C) once, and from B only the 128 columns per accumulator that are its half of
// the MMA's B tile: every operand byte is fetched by exactly one CTA of the pair, where the single-CTA kernel
// fetches A once per n-tile.  Barriers and bounded waits as in gemm_split_pair_kernel.
// EPI epilogue warps (4 or 8): a unit's accumulators are drained once, at the end of a long contraction, so four warps
// (one per tensor-memory lane quarter) cost little -- and the CTA then holds 6 warps' registers instead of 10, which
// leaves room on every SM sub-partition for blocks of the kernels that run beside it.
template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(32 * (2 + EPI), 1) gemm_split_pair_mn_kernel(const __grid_constant__ BfArgs g) {
  static_assert(EPI == 4 || EPI == 8, "one or two warps per lane quarter");
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_full[MAX_SLOTS], s_empty[MAX_SLOTS];
  __shared__ __align__(8) uint64_t s_tmem_full, s_tmem_empty;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t ring = smem_u32(smem);
  float* stg_base = reinterpret_cast<float*>(smem + (size_t)g.n_stages * g.stage_bytes);

  if (tid == 0) {
    for (int s = 0; s < MAX_SLOTS; ++s) {
      mbar_init(smem_u32(&s_full[s]), 1);
      mbar_init(smem_u32(&s_empty[s]), 1);
    }
    mbar_init(smem_u32(&s_tmem_full), 1);
    mbar_init(smem_u32(&s_tmem_empty), 2 * EPI);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  if (tid == 0) TRACE(0);
  volatile int* abort_flag = &s_abort;
  const unsigned limit = g.spin_limit;
  const uint32_t stage_bytes = (uint32_t)g.stage_bytes, n_stages = (uint32_t)g.n_stages;
  const uint32_t PLANE = 2u * 4096u;                 // one plane of an operand tile: 128 columns x 32 contraction rows
  const uint32_t TILE = (uint32_t)g.planes * PLANE;  // (plane, chunk, row, 64 elements)
  const int n_sub = g.n_tiles;                  // accumulators (256 columns of C each): 1 or 2

  // the pair's units: (256-row tile of C, part of the contraction), contiguous per pair
  const int T = g.m_tiles * g.split_k;
  const int u_begin = (int)((long long)T * (blockIdx.x >> 1) / (gridDim.x >> 1));
  const int u_end = (int)((long long)T * ((blockIdx.x >> 1) + 1) / (gridDim.x >> 1));
  const int per = (g.kb_total + g.split_k - 1) / g.split_k;

  if (warp == 0) {
    // ------------------------------------------------------------ tile copies (each CTA its own)
    if (lane == 0) {
      uint32_t c = 0;
      bool ok = true;
      for (int u = u_begin; u < u_end && ok; ++u) {
        const int ms = u % g.m_tiles, sp = u / g.m_tiles;
        const int kb0 = sp * per, kb1 = min(g.kb_total, kb0 + per);
        const int a_chunk = ms * 4 + (int)rank * 2;
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
          const uint32_t s = c % n_stages;
          ok = mbar_wait(smem_u32(&s_empty[s]), ((c / n_stages) & 1u) ^ 1u, limit, abort_flag);
          if (!ok) break;
          const uint32_t dst = ring + s * stage_bytes;
          const uint32_t bar = peer_addr(smem_u32(&s_full[s]), 0);
          if (leader) mbar_expect_tx(smem_u32(&s_full[s]), 2u * stage_bytes);
          tma_4d_pair(dst, &g.a_map, 0, kb * 32, a_chunk, 0, bar);
          for (int j = 0; j < n_sub; ++j) tma_4d_pair(dst + TILE * (uint32_t)(1 + j), &g.b_map, 0, kb * 32, j * 4 + (int)rank * 2, 0, bar);
          TRACE(256 + (int)c);
          ++c;
        }
      }
      if (!ok) {
        s_abort = 1;
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(smem_u32(&s_abort), rank ^ 1u)), "r"(1) : "memory");
        atomicCAS(g.status, 0, TGNN_ETIMEOUT);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (the leader's, for both CTAs)
    if (lane == 0 && leader) {
      uint32_t c = 0, n_item = 0;
      int withheld = 0;
      bool ok = true;
      const uint32_t fmt = g.fp16 ? 0u : 1u;
      // D fp32; both operands MN-major; N = 256; M = 256 across the pair
      const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 15) | (1u << 16) | ((256u >> 3) << 17) |
                             ((uint32_t)((2 * BM) >> 4) << 24);
      for (int u = u_begin; u < u_end && ok; ++u) {
        const int sp = u / g.m_tiles;
        const int kb0 = sp * per, kb1 = min(g.kb_total, kb0 + per);
        if (kb0 >= kb1) continue;
        ok = mbar_wait(smem_u32(&s_tmem_empty), (n_item & 1u) ^ 1u, limit, abort_flag);   // drained in both CTAs
        if (!ok) break;
        ++n_item;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
          const uint32_t s = c % n_stages;
          ok = mbar_wait(smem_u32(&s_full[s]), (c / n_stages) & 1u, limit, abort_flag);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          TRACE(16 + 2 * (int)c);
          const uint32_t a_addr = ring + s * stage_bytes;
          const int ks_n = min(2, g.ksteps_total - kb * 2);
          for (int j = 0; j < n_sub; ++j) {
            const uint32_t b_addr = a_addr + TILE * (uint32_t)(1 + j);
            const uint32_t acc = tmem + (uint32_t)(j * ACC_STRIDE);
            for (int ks = 0; ks < ks_n; ++ks) {
              const uint64_t da_hi = make_desc(a_addr + ks * 2048u, 4096u, 1024u);
              const uint64_t da_lo = make_desc(a_addr + PLANE + ks * 2048u, 4096u, 1024u);
              const uint64_t db_hi = make_desc(b_addr + ks * 2048u, 4096u, 1024u);
              const uint64_t db_lo = make_desc(b_addr + PLANE + ks * 2048u, 4096u, 1024u);
              const uint32_t first = (kb > kb0 || ks > 0) ? 1u : 0u;
              if (g.planes == 2) {
                mma_f16_pair(acc, da_lo, db_hi, idesc, first);
                mma_f16_pair(acc, da_hi, db_lo, idesc, 1u);
              }
              mma_f16_pair(acc, da_hi, db_hi, idesc, g.planes == 2 ? 1u : first);
            }
          }
          TRACE(17 + 2 * (int)c);
          if (withheld < g.debug_withhold) ++withheld;   // test hook: this stage is never handed back
          else commit_to_pair(smem_u32(&s_empty[s]));
          ++c;
        }
        if (ok) commit_to_pair(smem_u32(&s_tmem_full));
      }
      if (!ok) {
        s_abort = 1;
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(smem_u32(&s_abort), 1u)), "r"(1) : "memory");
        atomicCAS(g.status, 0, TGNN_ETIMEOUT);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue (each CTA its own 128 rows)
    const int e = warp - 2;
    const int t = e >> 2;          // EPI = 8: warps 2-5 drain the first accumulator, 6-9 the second (all eight the only one)
    const int q4 = warp & 3;
    float* stg = stg_base + e * (STG_WARP_BYTES / 4);
    const bool c_vec = (((uintptr_t)g.C & 15) == 0) && (g.ldc % 4 == 0);
    const uint32_t empty_bar = peer_addr(smem_u32(&s_tmem_empty), 0);
    uint32_t n_item = 0;
    bool ok = true;
    for (int u = u_begin; u < u_end && ok; ++u) {
      const int ms = u % g.m_tiles, sp = u / g.m_tiles;
      const int kb0 = sp * per, kb1 = min(g.kb_total, kb0 + per);
      if (kb0 >= kb1) continue;
      ok = mbar_wait(smem_u32(&s_tmem_full), n_item & 1u, limit, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (e == 0 && lane == 0) TRACE(2 + 2 * (int)n_item);
      ++n_item;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int m0 = (2 * ms + (int)rank) * BM;
      for (int j = (EPI == 8 && n_sub == 2) ? t : 0; j < n_sub; ++j) {
        Item it;
        it.mt0 = ms; it.tiles = 1; it.kb0 = kb0; it.kb1 = kb1;
        it.n0 = j * 256;
        it.n_valid = min(256, g.N - it.n0);
        const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(j * ACC_STRIDE);
        if (EPI == 8) {
          drain_tile(g, it, m0, taddr, n_sub == 2 ? 0 : 32 * t, n_sub == 2 ? 32 : 64, stg, lane, q4, c_vec);
          break;
        }
        drain_tile(g, it, m0, taddr, 0, 32, stg, lane, q4, c_vec);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (e == 0 && lane == 0) TRACE(1 + 2 * (int)n_item);
      if (lane == 0) mbar_arrive_cluster(empty_bar);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this warp's bulk stores have landed
    if (!ok && lane == 0) {
      s_abort = 1;
      asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_addr(smem_u32(&s_abort), rank ^ 1u)), "r"(1) : "memory");
      atomicCAS(g.status, 0, TGNN_ETIMEOUT);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (s_abort && warp == 0) {
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // copies still on their way into this CTA's shared memory
  }
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// fp32 rows -> two 16-bit planes (hi, lo), fp16 or bf16, after multiplication by `scale`.  One thread per 4 consecutive columns; columns in [cols, ld_out) of the
// planes are written as zeros except column `ones_col` (if >= 0), which is 1 (the bias column of a weight gradient).
__global__ void __launch_bounds__(256) split_rows_kernel(const float* __restrict__ X, int64_t ld_in, int64_t rows, int cols,
                                                         const int32_t* __restrict__ dev_rows, __nv_bfloat16* __restrict__ hi,
                                                         __nv_bfloat16* __restrict__ lo, int64_t ld_out, int ones_col,
                                                         int fp16, float scale, int planes) {
  const int per_row = (int)(ld_out >> 2);
  const int64_t n_rows = dev_rows ? min((int64_t)*dev_rows, rows) : rows;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < rows * per_row; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / per_row;
    const int c = (int)(i - r * per_row) * 4;
    float v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int cc = c + e;
      v[e] = (r < n_rows && cc < cols) ? scale * X[r * ld_in + cc] : ((cc == ones_col && r < n_rows) ? 1.f : 0.f);
    }
    unsigned short h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (fp16) {
        const __half hh = __float2half_rn(v[e]);
        h[e] = __half_as_ushort(hh);
        l[e] = __half_as_ushort(__float2half_rn(v[e] - __half2float(hh)));
      } else {
        const __nv_bfloat16 hh = __float2bfloat16_rn(v[e]);
        h[e] = __bfloat16_as_ushort(hh);
        l[e] = __bfloat16_as_ushort(__float2bfloat16_rn(v[e] - __bfloat162float(hh)));
      }
    }
    *reinterpret_cast<uint2*>(hi + r * ld_out + c) = *reinterpret_cast<const uint2*>(h);
    if (planes == 2) *reinterpret_cast<uint2*>(lo + r * ld_out + c) = *reinterpret_cast<const uint2*>(l);
  }
}

// Split planes of the attention layer's key/value weights for this step's two big products:
//   wkv[n, k] = W_kv[n, k]                      (n < 2d, k < dkv: the forward projection's B operand)
//   wz[n, k]  = W_kv[k, col(n)]                 (n < 2d, k < 2d: the input gradient toward the memory columns,
//               col(n) = n for n < d, and the time-encoding columns, col(n) = d + de + (n - d) otherwise)
// Padding columns of the planes are zero.  Both planes hold fp16 numbers.
__global__ void __launch_bounds__(256) prep_split_weights_kernel(const float* __restrict__ Wkv, int d, int de,
                                                                 __nv_bfloat16* __restrict__ wkv_hi, int64_t wkv_plane, int ld_kv,
                                                                 __nv_bfloat16* __restrict__ wz_hi, int64_t wz_plane, int ld_z,
                                                                 int planes) {
  const int dkv = 2 * d + de, n_rows = 2 * d;
  const int64_t n_kv = (int64_t)n_rows * ld_kv, n_z = (int64_t)n_rows * ld_z;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_kv + n_z; i += (int64_t)gridDim.x * blockDim.x) {
    float v = 0.f;
    __nv_bfloat16 *hi, *lo;
    if (i < n_kv) {
      const int n = (int)(i / ld_kv), k = (int)(i - (int64_t)n * ld_kv);
      if (k < dkv) v = Wkv[(int64_t)n * dkv + k];
      hi = wkv_hi + i; lo = wkv_hi + wkv_plane + i;
    } else {
      const int64_t j = i - n_kv;
      const int n = (int)(j / ld_z), k = (int)(j - (int64_t)n * ld_z);
      if (k < n_rows) v = Wkv[(int64_t)k * dkv + (n < d ? n : d + de + (n - d))];
      hi = wz_hi + j; lo = wz_hi + wz_plane + j;
    }
    const __half h = __float2half_rn(v);   // weights: two fp16 numbers
    *reinterpret_cast<__half*>(hi) = h;
    if (planes == 2) *reinterpret_cast<__half*>(lo) = __float2half_rn(v - __half2float(h));
  }
}

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn encoder() {
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

// K-major operand: (contiguous index, row, plane) view of a split matrix; box = 64 elements x box_rows x both planes,
// 128-byte swizzle, zeros outside [0, cols) x [0, rows).
bool encode_k_map(CUtensorMap* map, const SplitMat& m, int box_rows) {
  const TensorMapEncodeFn enc = encoder();
  if (!enc || m.rows <= 0 || m.cols <= 0 || box_rows < 1 || box_rows > 256 || m.planes < 1 || m.planes > 2) return false;
  if (((uintptr_t)m.hi & 15) != 0 || m.ld % 8 != 0 || m.plane_stride % 8 != 0) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)m.cols, (cuuint64_t)m.rows, (cuuint64_t)m.planes};
  const cuuint64_t strides[2] = {(cuuint64_t)m.ld * 2, (cuuint64_t)m.plane_stride * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)m.planes};
  const cuuint32_t elem[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, m.hi, dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// MN-major operand: the matrix [rows = contraction, cols] seen as (element within a 64-column chunk, row, chunk,
// plane); one box of 64 x 32 rows x `chunks` x both planes lands chunk-major, i.e. as the operand tile's own
// layout (per chunk 32 rows of 128 bytes, swizzled).  The last chunk of a row may run past the row end into the
// next row (or, for the last row, up to 126 bytes past the plane): those values only reach rows / columns of C
// that are never stored, and the buffers end in slack.
bool encode_mn_map(CUtensorMap* map, const SplitMat& m, int chunks) {
  const TensorMapEncodeFn enc = encoder();
  if (!enc || m.rows <= 0 || m.cols <= 0 || chunks < 1 || chunks > 4 || m.planes < 1 || m.planes > 2) return false;
  if (((uintptr_t)m.hi & 15) != 0 || m.ld % 8 != 0 || m.plane_stride % 8 != 0) return false;
  const cuuint64_t dims[4] = {64, (cuuint64_t)m.rows, (cuuint64_t)((m.cols + 63) / 64), (cuuint64_t)m.planes};
  const cuuint64_t strides[3] = {(cuuint64_t)m.ld * 2, 128, (cuuint64_t)m.plane_stride * 2};
  const cuuint32_t box[4] = {64, 32, (cuuint32_t)chunks, (cuuint32_t)m.planes};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, m.hi, dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// C [M, N] fp32 with pitch ldc as (column, row); boxes of 32 x 32 values, 128-byte swizzle in shared memory.
bool encode_c_map(CUtensorMap* map, float* C, int64_t ldc, int M, int N) {
  const TensorMapEncodeFn enc = encoder();
  if (!enc || ((uintptr_t)C & 15) != 0 || ldc % 4 != 0) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)ldc * 4};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t elem[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int launch_prep_split_weights(tgnn_ctx* ctx, cudaStream_t s) {
  if (!ctx->split_buf) return TGNN_OK;
  const int d = ctx->cfg.d, de = ctx->cfg.d_e;
  {
    KernelScope scope__(ctx, "prep_split_weights", s);
    prep_split_weights_kernel<<<148, 256, 0, s>>>(ctx->params + ctx->L.wk, d, de, reinterpret_cast<__nv_bfloat16*>(ctx->wkv_s.hi),
                                                  ctx->wkv_s.plane_stride, (int)ctx->wkv_s.ld,
                                                  reinterpret_cast<__nv_bfloat16*>(ctx->wz_s.hi), ctx->wz_s.plane_stride,
                                                  (int)ctx->wz_s.ld, ctx->wkv_s.planes);
  }
  TGNN_LAUNCH_OK(ctx, "prep_split_weights");
  return TGNN_OK;
}

int launch_split_rows(tgnn_ctx* ctx, const float* X, int64_t ld_in, int64_t rows, int cols, const int32_t* dev_rows,
                      const SplitMat& out, int ones_col, const char* name, cudaStream_t s) {
  if (rows <= 0) return TGNN_OK;
  const int64_t work = rows * (out.ld >> 2);
  const int blocks = (int)((work + 255) / 256 < 148 * 16 ? (work + 255) / 256 : 148 * 16);
  {
    KernelScope scope__(ctx, name, s);
    split_rows_kernel<<<blocks, 256, 0, s>>>(X, ld_in, rows, cols, dev_rows, reinterpret_cast<__nv_bfloat16*>(out.hi),
                                             reinterpret_cast<__nv_bfloat16*>(out.hi) + out.plane_stride, out.ld, ones_col,
                                             out.fp16, out.scale, out.planes);
  }
  TGNN_LAUNCH_OK(ctx, name);
  return TGNN_OK;
}

// C[M,N] (+)= A B (+ bias) (ReLU) from split operands.
//   mn_major = 0: A is the matrix [M, K], B the matrix [N, K] (both with the contraction index contiguous);
//   mn_major = 1: A is the matrix [K, M], B the matrix [K, N] (contraction over rows: C = A^T B).
// split_k > 1 needs accumulate (C holds valid data; partial sums are added atomically).
int launch_gemm_split(tgnn_ctx* ctx, const SplitMat& A, const SplitMat& B, int mn_major, float* C, int64_t ldc, int M, int N,
                      int K, const float* bias, int relu, int accumulate, int split_k, const char* name, cudaStream_t s,
                      int debug_withhold, unsigned spin_limit, int extra_col, float* extra_out, long long* trace, int single,
                      int launches, int pair) {
  if (M <= 0 || N <= 0) return TGNN_OK;
  if (K <= 0) return set_error(ctx, TGNN_EINVAL, "gemm %s: empty contraction", name);
  if (split_k > 1 && !accumulate) return set_error(ctx, TGNN_EINVAL, "gemm %s: split_k needs accumulate", name);
  BfArgs a = {};
  a.C = C; a.ldc = ldc; a.M = M; a.N = N; a.K = K; a.bias = bias; a.relu = relu; a.accumulate = accumulate;
  a.mn_major = mn_major ? 1 : 0;
  if ((A.fp16 != 0) != (B.fp16 != 0))
    return set_error(ctx, TGNN_EINVAL, "gemm %s: one operand is held as fp16 planes and the other as bf16 planes", name);
  a.fp16 = A.fp16 ? 1 : 0;
  if (A.planes != B.planes) return set_error(ctx, TGNN_EINVAL, "gemm %s: the operands differ in their number of planes", name);
  a.planes = A.planes == 1 ? 1 : 2;
  const int planes = a.planes;
  a.out_scale = 1.f / (A.scale * B.scale);
  // single row tiles with alternating accumulators for the activation x weight products (their epilogue, a full
  // store of C, then overlaps the next tile's MMAs); pairs for the weight gradients (one item per CTA, B shared)
  a.single = single >= 0 ? (single ? 1 : 0) : (mn_major ? 0 : 1);
  a.status = ctx->ws.status;
  a.extra_col = (extra_out && accumulate) ? extra_col : -1;
  a.extra_out = extra_out;
  a.c_bulk = a.extra_col < 0 && encode_c_map(&a.c_map, C, ldc, M, N) ? 1 : 0;
  a.trace = trace;
  a.debug_withhold = debug_withhold;
  a.spin_limit = spin_limit ? spin_limit : SPIN_LIMIT;
  a.m_tiles = (M + BM - 1) / BM;
  // n-tiles: a common stride bn (a multiple of 16; of 64 for MN-major operands, whose tiles start on chunk
  // boundaries) and the remainder, at most 256 columns, in the last tile
  const int gran = mn_major ? 64 : 16;
  a.n_tiles = (N + 255) / 256;
  int n_last;
  for (;; ++a.n_tiles) {
    a.bn = a.n_tiles == 1 ? (N + gran - 1) / gran * gran : (N / a.n_tiles) / gran * gran;
    if (a.n_tiles > 1 && a.bn < gran) a.bn = gran;
    n_last = N - (a.n_tiles - 1) * a.bn;
    if (n_last <= 256) break;
  }
  if (n_last <= 0) return set_error(ctx, TGNN_ESHAPE, "gemm %s: n-tiling failed", name);
  const int n_widest = a.n_tiles == 1 ? N : (a.bn > n_last ? a.bn : n_last);
  const int b_rows = (n_widest + 15) / 16 * 16;     // K-major B box: rows of the widest n-tile
  const int bke = mn_major ? 32 : 64;
  a.kb_total = (K + bke - 1) / bke;
  a.ksteps_total = (K + 15) / 16;
  a.b_chunks = (n_widest + 63) / 64;
  a.a_slot_bytes = mn_major ? planes * 2 * 4096 : planes * BM * 128;
  a.b_slot_bytes = mn_major ? planes * a.b_chunks * 4096 : planes * b_rows * 128;
  const int budget = SMEM_LIMIT - 1024 - STG_BYTES - 1024;
  a.n_b_slots = a.b_slot_bytes > 40 * 1024 ? 2 : (a.b_slot_bytes > 20 * 1024 ? 3 : 4);
  a.n_a_slots = (budget - a.n_b_slots * a.b_slot_bytes) / a.a_slot_bytes;
  if (a.n_a_slots > MAX_SLOTS) a.n_a_slots = MAX_SLOTS;
  if (a.n_a_slots < 2) return set_error(ctx, TGNN_ESHAPE, "gemm %s: tile does not fit shared memory", name);
  const int m_pairs = (a.m_tiles + 1) / 2;
  a.split_k = 1;
  if (accumulate && split_k > 1) {
    const int base = m_pairs * a.n_tiles;
    int sp = (148 + base - 1) / base;
    const int max_s = (a.kb_total + 7) / 8;   // at least 8 contraction blocks per split
    if (sp > max_s) sp = max_s;
    if (sp > split_k) sp = split_k;
    a.split_k = sp < 1 ? 1 : sp;
  }
  const bool maps_ok = mn_major ? (encode_mn_map(&a.a_map, A, 2) && encode_mn_map(&a.b_map, B, a.b_chunks))
                                : (encode_k_map(&a.a_map, A, BM) && encode_k_map(&a.b_map, B, b_rows));
  if (!maps_ok) return set_error(ctx, TGNN_ECUDA, "gemm %s: tensor map encoding failed", name);
  // K-major products with more than a handful of row tiles: pairs of CTAs, each loading half of every B tile
  // (`pair` = 0 / 1 overrides the default).
  const bool can_pair = !mn_major && a.split_k == 1 && a.extra_col < 0 && M > BM;
  if (can_pair && (pair > 0 || (pair < 0 && a.m_tiles >= 32))) {
    const int n_mma = (n_widest + 15) / 16 * 16, bh = n_mma / 2;
    a.m_tiles = (M + 2 * BM - 1) / (2 * BM);
    a.stage_bytes = planes * (BM * 128 + bh * 128);
    a.n_stages = (SMEM_LIMIT - 1024 - STG_BYTES - 1024) / a.stage_bytes;
    if (a.n_stages > MAX_SLOTS) a.n_stages = MAX_SLOTS;
    if (a.n_stages >= 2 && encode_k_map(&a.b_map, B, bh)) {
      a.kb_begin = 0; a.kb_end = a.kb_total;
      const int units = a.m_tiles * a.n_tiles;
      const int clusters = units < 74 ? units : 74;
      const int smem = 1024 + a.n_stages * a.stage_bytes + STG_BYTES;
      static SmemLimit pair_limit;
      const int rc = raise_smem_limit(ctx, gemm_split_pair_kernel, SMEM_LIMIT - 1024, pair_limit);
      if (rc) return rc;
      {
        KernelScope scope__(ctx, name, s);
        gemm_split_pair_kernel<<<2 * clusters, THREADS, smem, s>>>(a);
      }
      TGNN_LAUNCH_OK(ctx, name);
      return TGNN_OK;
    }
    a.m_tiles = (M + BM - 1) / BM;   // (does not fit: the single-CTA kernel below)
    if (!encode_k_map(&a.b_map, B, b_rows)) return set_error(ctx, TGNN_ECUDA, "gemm %s: tensor map encoding failed", name);
  }
  // Weight gradients whose tile of C is more than 128 rows and at most 512 columns: pairs of CTAs, each operand
  // byte fetched once per pair.
  if (mn_major && accumulate && split_k > 1 && a.extra_col < 0 && M > BM && N <= 512 && (pair > 0 || pair < 0)) {
    BfArgs b = a;
    b.m_tiles = (M + 2 * BM - 1) / (2 * BM);
    b.n_tiles = (N + 255) / 256;
    b.bn = 256;
    b.stage_bytes = planes * 8192 * (1 + b.n_tiles);
    b.n_stages = (SMEM_LIMIT - 1024 - STG_BYTES - 1024) / b.stage_bytes;
    if (b.n_stages > MAX_SLOTS) b.n_stages = MAX_SLOTS;
    // three stages feed the MMAs as well as four do, and leave 48 KB of the SM's shared memory to blocks of the
    // kernels that run beside a weight gradient (gradient scatter, time-encoder sums): measured 11 us per step
    if (b.n_stages > 6 / planes) b.n_stages = 6 / planes;   // (144 KB of stages in either form)
    int sp = 74 / b.m_tiles;
    const int max_s = (b.kb_total + 7) / 8;
    if (sp > max_s) sp = max_s;
    if (sp > split_k) sp = split_k;
    b.split_k = sp < 1 ? 1 : sp;
    b.kb_begin = 0; b.kb_end = b.kb_total;
    if (b.n_stages >= 2 && encode_mn_map(&b.a_map, A, 2) && encode_mn_map(&b.b_map, B, 2)) {
      const int units = b.m_tiles * b.split_k;
      const int clusters = units < 74 ? units : 74;
      const int smem = 1024 + b.n_stages * b.stage_bytes + STG_BYTES;
      static SmemLimit pair_mn_limit;
      const int rc = raise_smem_limit(ctx, gemm_split_pair_mn_kernel<4>, SMEM_LIMIT - 1024, pair_mn_limit);
      if (rc) return rc;
      {
        KernelScope scope__(ctx, name, s);
        gemm_split_pair_mn_kernel<4><<<2 * clusters, 32 * (2 + 4), smem, s>>>(b);
      }
      TGNN_LAUNCH_OK(ctx, name);
      return TGNN_OK;
    }
  }
  const int units = a.m_tiles * a.n_tiles * a.split_k;
  const int items = a.single ? units : (units + 1) / 2;
  const int smem = 1024 + a.n_a_slots * a.a_slot_bytes + a.n_b_slots * a.b_slot_bytes + STG_BYTES;
  static SmemLimit smem_limit;
  {  // the largest dynamic size any shape asks for (the static barriers take a few hundred bytes of the 227 KB)
    const int rc = raise_smem_limit(ctx, gemm_split_kernel, SMEM_LIMIT - 1024, smem_limit);
    if (rc) return rc;
  }
  // A long accumulating product may go out as several launches over consecutive parts of the contraction: a
  // persistent launch holds every SM until it ends, and the boundaries between the parts are where kernels of
  // the step's critical chain (higher stream priority) get in.
  int parts = (accumulate && launches > 1) ? launches : 1;
  if (parts > a.kb_total / (4 * a.split_k)) parts = a.kb_total / (4 * a.split_k);
  if (parts < 1) parts = 1;
  for (int p = 0; p < parts; ++p) {
    a.kb_begin = (int)((long long)a.kb_total * p / parts);
    a.kb_end = (int)((long long)a.kb_total * (p + 1) / parts);
    {
      KernelScope scope__(ctx, name, s);
      gemm_split_kernel<<<items < 148 ? items : 148, THREADS, smem, s>>>(a);
    }
    TGNN_LAUNCH_OK(ctx, name);
  }
  return TGNN_OK;
}

}  // namespace tgnn
