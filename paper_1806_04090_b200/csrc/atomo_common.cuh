// Shared device/host helpers of the CUDA path (never included by the CPU oracle).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "atomo.h"

namespace atomo {

constexpr int kWarp = 32;

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  The Bernoulli draws of Eq. (2) only need independent
// uniforms; a counter-based generator makes them a pure function of (seed, step, layer, atom).
// ---------------------------------------------------------------------------------------------
struct PhiloxKey { uint32_t k0, k1; };

__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, PhiloxKey key) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)M0 * ctr.x, p1 = (uint64_t)M1 * ctr.z;     // one wide multiply each
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    ctr = make_uint4(hi1 ^ ctr.y ^ key.k0, lo1, hi0 ^ ctr.w ^ key.k1, lo0);
    key.k0 += W0;
    key.k1 += W1;
  }
  return ctr;
}

// Counter layout: (block low, block high, layer, (kind << 31) | (step & 0x7fffffff)); block = atom >> 2.
__device__ __forceinline__ uint4 atom_block_words(uint64_t block, uint32_t layer, uint32_t kind_step,
                                                  PhiloxKey key) {
  return philox4x32_10(make_uint4((uint32_t)block, (uint32_t)(block >> 32), layer, kind_step), key);
}

__host__ __device__ __forceinline__ uint32_t kind_step_word(uint32_t kind, uint64_t step) {
  return ((kind & 1u) << 31) | (uint32_t)(step & 0x7FFFFFFFull);
}

// t = 1 iff p >= 1 or word < floor(p * 2^32); p * 2^32 is exact in fp32, the floor is taken by
// the truncating conversion.  p = 0 (also NaN, negative) never keeps.
__device__ __forceinline__ bool bernoulli_keep(float p, uint32_t word) {
  if (p >= 1.0f) return true;
  if (!(p > 0.0f)) return false;
  const uint32_t thr = __float2uint_rz(p * 4294967296.0f);   // p < 1 -> fits 32 bits
  return word < thr;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ uint32_t warp_sum(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Packed pair of fp32 (sm_100: one instruction multiplies and adds two lanes' worth of a 64-bit register pair).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {      // a * b + c, both halves, round to nearest
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

__host__ __device__ __forceinline__ uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// raise a layer's status to `st` if it is still OK (first error wins)
__device__ __forceinline__ void raise_status(atomo_layer_header* h, uint32_t st) {
  atomicCAS(&h->status, (uint32_t)ATOMO_OK, st);
}

}  // namespace atomo
