// Small device helpers shared by the kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tgnn.h"

namespace tgnn {

// Index check of every gather and scatter: true if 0 <= v < n.  Otherwise TGNN_EBOUNDS is recorded in the status
// word (the first error stays) and the caller skips the access -- nothing traps, the kernel runs to its end.
__device__ __forceinline__ bool index_ok(long long v, long long n, int32_t* status) {
  if (v >= 0 && v < n) return true;
  if (status != nullptr) atomicCAS(status, 0, (int32_t)TGNN_EBOUNDS);
  return false;
}

// Phi(dt)_c = cos(fmaf(w_c, dt, b_c)) with the argument in fp32.
// The arguments span eight decades (w from 1 down to 1e-9, dt up to the stream's time range), so the cosine
// needs a full-range reduction; the library's cosf / sincosf spend well over a hundred instructions on
// theirs, which made the encoders the bulk of the gather kernels' time.  Here the fp32 argument is reduced
// to [-pi, pi] by a three-constant Cody-Waite step carried out with exact products (below), and the hardware
// approximations take it from there: absolute error below 2^-21 on that interval.
__device__ __forceinline__ float time_arg(float w, float b, float dtf) { return fmaf(w, dtf, b); }
__device__ __forceinline__ float reduce_two_pi(float x) {
  // x - k * 2 pi with 2 pi = C1 + C2 + C3 in fp32 pieces: k * C1 is formed exactly as a product and its
  // rounding residue (one fused multiply-add), x - k * C1 is then exact (the two are within a factor of 2),
  // and the two small corrections each round once: absolute error below 3e-7 up to |x| = 5e7 (checked
  // against exact arithmetic on 2 M random arguments).  k may be off by one for the largest arguments (the
  // product x / 2 pi is itself rounded); the remainder is then just outside [-pi, pi], which the hardware
  // routines accept.
  const float k = rintf(x * 0.15915494f);
  const float p = k * 6.2831855f;
  const float pl = fmaf(k, 6.2831855f, -p);
  float r = (x - p) - pl;
  r = fmaf(-k, -1.7484555e-7f, r);
  return fmaf(-k, -6.8604980e-15f, r);
}
__device__ __forceinline__ float time_encode(float w, float b, float dtf) { return __cosf(reduce_two_pi(time_arg(w, b, dtf))); }
// cos and sin of the same argument at once; the sine is kept for the backward pass (d Phi / d arg = -sin).
__device__ __forceinline__ void time_encode_sc(float w, float b, float dtf, float* cos_out, float* sin_out) {
  const float r = reduce_two_pi(time_arg(w, b, dtf));
  *sin_out = __sinf(r);
  *cos_out = __cosf(r);
}

// x as two bf16 numbers hi + lo (16 mantissa bits together); pairs of neighbours packed into 32-bit words.
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16* hi, __nv_bfloat16* lo) {
  *hi = __float2bfloat16_rn(x);
  *lo = __float2bfloat16_rn(x - __bfloat162float(*hi));
}
__device__ __forceinline__ void split_bf16_pair(float x0, float x1, uint32_t* hi, uint32_t* lo) {
  __nv_bfloat16 h0, l0, h1, l1;
  split_bf16(x0, &h0, &l0);
  split_bf16(x1, &h1, &l1);
  *hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  *lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}

// The same as two fp16 numbers: 22 mantissa bits together for values inside fp16's range (|x| < 65504; below
// 6e-5 the absolute error is 3e-8).  Used for operands of moderate size; gradients are scaled into range first.
// (Packed conversions: one instruction rounds both values and leaves them in place, and the way back is an fp16
// add unit operation; the scalar conversions would queue on the special-function pipe beside the cosines.)
__device__ __forceinline__ void split_f16_pair(float x0, float x1, uint32_t* hi, uint32_t* lo) {
  const __half2 h = __floats2half2_rn(x0, x1);             // .x = x0 in the low half
  const float2 hf = __half22float2(h);
  const __half2 l = __floats2half2_rn(x0 - hf.x, x1 - hf.y);
  *hi = *reinterpret_cast<const uint32_t*>(&h);
  *lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Two values as one fp16 number each, packed (the hi part alone).
__device__ __forceinline__ uint32_t pack_f16_pair(float x0, float x1) {
  const __half2 h = __floats2half2_rn(x0, x1);
  return *reinterpret_cast<const uint32_t*>(&h);
}

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + expf(-x)); }
__device__ __forceinline__ float softplusf_(float x) { return x > 0.f ? x + log1pf(expf(-x)) : log1pf(expf(x)); }

// Copy n floats with one warp: 128-bit accesses when both rows allow it.
__device__ __forceinline__ void warp_copy_f32(float* __restrict__ dst, const float* __restrict__ src, int n, int lane) {
  if ((((uintptr_t)dst | (uintptr_t)src) & 15) == 0 && (n & 3) == 0) {
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* d4 = reinterpret_cast<float4*>(dst);
    for (int q = lane; q < (n >> 2); q += 32) d4[q] = __ldg(s4 + q);
  } else {
    for (int q = lane; q < n; q += 32) dst[q] = __ldg(src + q);
  }
}

// One edge-feature row (fp32 or bf16 table) into fp32.
__device__ __forceinline__ void warp_copy_feat(float* __restrict__ dst, const void* __restrict__ efeat, int feat_bf16,
                                               int64_t eid, int de, int lane) {
  if (de == 0) return;
  if (!feat_bf16) {
    warp_copy_f32(dst, reinterpret_cast<const float*>(efeat) + eid * de, de, lane);
  } else {
    // rows are 2*de bytes, de even: 32-bit loads of bf16 pairs
    const uint32_t* s = reinterpret_cast<const uint32_t*>(reinterpret_cast<const __nv_bfloat16*>(efeat) + eid * de);
    for (int q = lane; q < (de >> 1); q += 32) {
      const uint32_t v = __ldg(s + q);
      dst[2 * q] = __uint_as_float(v << 16);
      dst[2 * q + 1] = __uint_as_float(v & 0xffff0000u);
    }
  }
}

// ---- attention kernels: per-warp shared-memory staging --------------------------------------------
// Floats one warp needs: K and V rows of the root's k slots, two d-vectors (query, upstream gradient)
// and three H*k scratch vectors, rounded to whole 16-byte chunks.
__host__ __device__ inline int attn_warp_floats(int d, int H, int k) { return 2 * k * d + 2 * d + ((3 * H * k + 3) & ~3); }
inline int attn_warps_per_block(int d, int H, int k) {
  const int per = attn_warp_floats(d, H, k) * 4;
  int w = (200 * 1024) / per;
  return w > 8 ? 8 : (w < 1 ? 1 : w);
}
inline size_t attn_smem_bytes(int d, int H, int k, int warps) { return (size_t)warps * attn_warp_floats(d, H, k) * 4; }

// Stage the root's valid K | V rows and its query in shared memory: asynchronous 16-byte copies, all
// issued before the single wait, so the whole 8 KB of a root costs one round trip instead of one per
// loop iteration.  Rows are 16-byte aligned (d is a multiple of 4).  Ends with the copies complete and
// visible to the warp (attn_stage_wait; other loads of the caller can be put between issue and wait).
__device__ __forceinline__ void cp_async16(float* smem_dst, const float* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void attn_stage_issue(float* Ks, float* Vs, float* Qs, const float* __restrict__ Q,
                                                 const float* __restrict__ KV, int i, int c, int d, int k, int lane) {
  const int d4 = d >> 2;
  const float* q = Q + (int64_t)i * d;
  for (int e = lane; e < d4; e += 32) cp_async16(Qs + 4 * e, q + 4 * e);
  const float* kv = KV + (int64_t)i * k * 2 * d;
  for (int e = lane; e < c * 2 * d4; e += 32) {
    const int s = e / (2 * d4), r = e - s * 2 * d4;
    cp_async16(r < d4 ? Ks + s * d + 4 * r : Vs + s * d + 4 * (r - d4), kv + 4 * e);
  }
}
__device__ __forceinline__ void attn_stage_wait() {
  cp_async_wait_all();
  __syncwarp();
}

}  // namespace tgnn
