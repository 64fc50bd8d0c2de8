// Device helpers shared by the libjackpot kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "jackpot.h"

namespace jp {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
#define JP_NEG_INF (__int_as_float(0xff800000))

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Order-preserving map float -> uint32 (larger float <=> larger integer), with
// -0 folded onto +0 so that numerically equal logits get equal keys.
__device__ __forceinline__ uint32_t f32_order_bits(float v) {
  uint32_t b = __float_as_uint(v);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_bits_f32(uint32_t o) {
  uint32_t b = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
  return __uint_as_float(b);
}
// 64-bit key of one vocabulary entry under the total order "higher logit first,
// equal logits by lower index": bigger key = better.  Key 0 is below every real
// entry and marks an empty slot.
__device__ __forceinline__ unsigned long long make_key(float v, uint32_t idx) {
  return ((unsigned long long)f32_order_bits(v) << 32) | (unsigned long long)(uint32_t)(~idx);
}
__device__ __forceinline__ uint32_t key_index(unsigned long long key) { return ~(uint32_t)key; }
__device__ __forceinline__ float key_value(unsigned long long key) {
  return order_bits_f32((uint32_t)(key >> 32));
}

// Philox4x32-10 (Salmon et al., SC'11) from the published round function; only
// the first output word is needed.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2,
                                                        uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0;
}
__device__ __forceinline__ float accept_uniform(uint64_t seed, uint64_t g) {
  uint32_t w = philox4x32_10_word0((uint32_t)g, (uint32_t)(g >> 32), 0u, 0u, (uint32_t)seed,
                                   (uint32_t)(seed >> 32));
  return (float)(w >> 8) * (1.0f / 16777216.0f);
}

// ---- 16-byte vectors of logits -------------------------------------------
// One uint4 holds 8 bf16 or 4 fp32 logits.  Lane e of a bf16 vector sits in the
// low (e even) or high (e odd) half of word e/2.
template <int DT> struct Vec;
template <> struct Vec<JP_BF16> {
  static constexpr int N = 8;
  static constexpr int ESIZE = 2;
  __device__ static __forceinline__ uint4 neg_inf() {
    return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
  }
  __device__ static __forceinline__ float get(const uint4& v, int e) {
    uint32_t w = (e >> 1) == 0 ? v.x : (e >> 1) == 1 ? v.y : (e >> 1) == 2 ? v.z : v.w;
    return __uint_as_float((e & 1) ? (w & 0xffff0000u) : (w << 16));
  }
  __device__ static __forceinline__ float vmax(const uint4& v) {
    __nv_bfloat162 a = __hmax2(*(const __nv_bfloat162*)&v.x, *(const __nv_bfloat162*)&v.y);
    __nv_bfloat162 b = __hmax2(*(const __nv_bfloat162*)&v.z, *(const __nv_bfloat162*)&v.w);
    a = __hmax2(a, b);
    uint32_t w = *(uint32_t*)&a;
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
  }
  // maximum over two vectors: one packed tree, unpacked once
  __device__ static __forceinline__ float vmax2(const uint4& u, const uint4& v) {
    __nv_bfloat162 a = __hmax2(*(const __nv_bfloat162*)&u.x, *(const __nv_bfloat162*)&u.y);
    __nv_bfloat162 b = __hmax2(*(const __nv_bfloat162*)&u.z, *(const __nv_bfloat162*)&u.w);
    __nv_bfloat162 c = __hmax2(*(const __nv_bfloat162*)&v.x, *(const __nv_bfloat162*)&v.y);
    __nv_bfloat162 d = __hmax2(*(const __nv_bfloat162*)&v.z, *(const __nv_bfloat162*)&v.w);
    a = __hmax2(__hmax2(a, b), __hmax2(c, d));
    uint32_t w = *(uint32_t*)&a;
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
  }
  __device__ static __forceinline__ float load_scalar(const void* row, int64_t i) {
    return __uint_as_float((uint32_t)((const uint16_t*)row)[i] << 16);
  }
  __device__ static __forceinline__ void set(uint4& v, int e, float f) {
    const uint32_t sh = (e & 1) ? 16u : 0u;
    const uint32_t keep = ~(0xffffu << sh);
    const uint32_t val = (__float_as_uint(f) >> 16) << sh;   // exact: f came from a bf16
    switch (e >> 1) {
      case 0: v.x = (v.x & keep) | val; break;
      case 1: v.y = (v.y & keep) | val; break;
      case 2: v.z = (v.z & keep) | val; break;
      default: v.w = (v.w & keep) | val; break;
    }
  }
};
template <> struct Vec<JP_F32> {
  static constexpr int N = 4;
  static constexpr int ESIZE = 4;
  __device__ static __forceinline__ uint4 neg_inf() {
    return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
  }
  __device__ static __forceinline__ float get(const uint4& v, int e) {
    return __uint_as_float(e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w);
  }
  __device__ static __forceinline__ float vmax(const uint4& v) {
    return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                 fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
  }
  __device__ static __forceinline__ float vmax2(const uint4& u, const uint4& v) { return fmaxf(vmax(u), vmax(v)); }
  __device__ static __forceinline__ float load_scalar(const void* row, int64_t i) {
    return ((const float*)row)[i];
  }
  __device__ static __forceinline__ void set(uint4& v, int e, float f) {
    uint32_t b = __float_as_uint(f);
    if (e == 0) v.x = b; else if (e == 1) v.y = b; else if (e == 2) v.z = b; else v.w = b;
  }
};

// Streaming 16-byte read that does not linger in L1.
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void stg_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

}  // namespace jp
