// Device-side pieces shared by the kernels of libhoccl: the arithmetic of one SUM (the paper has no reduction, Sec. 4
// "Limitations"; this is the per-step add of the textbook ring: one binary32 add, rounded to nearest even into the I/O
// dtype) and the flattened view of a batch of segments.  Everything here has internal linkage.
#pragma once
#include <cuda_bf16.h>

#include "kernels.cuh"

namespace hoccl {
namespace {

template <int DT>
struct Traits;
template <>
struct Traits<0> {  // fp32
  static constexpr int E = 4;
  static constexpr int VE = 4;
  __device__ static __forceinline__ uint4 add_vec(uint4 a, uint4 b) {
    uint4 r;
    r.x = __float_as_uint(__fadd_rn(__uint_as_float(a.x), __uint_as_float(b.x)));
    r.y = __float_as_uint(__fadd_rn(__uint_as_float(a.y), __uint_as_float(b.y)));
    r.z = __float_as_uint(__fadd_rn(__uint_as_float(a.z), __uint_as_float(b.z)));
    r.w = __float_as_uint(__fadd_rn(__uint_as_float(a.w), __uint_as_float(b.w)));
    return r;
  }
  __device__ static __forceinline__ void add_scalar(const void* a, const void* b, void* o, unsigned long long i) {
    static_cast<float*>(o)[i] = __fadd_rn(static_cast<const float*>(a)[i], static_cast<const float*>(b)[i]);
  }
};

// two bf16 in one 32-bit word: widen (exact), add in binary32, round to nearest even
__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
  float lo = __fadd_rn(__uint_as_float(a << 16), __uint_as_float(b << 16));
  float hi = __fadd_rn(__uint_as_float(a & 0xffff0000u), __uint_as_float(b & 0xffff0000u));
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
// The same add as one instruction.  add.rn.bf16x2 gives the bits of add_bf16x2 for ALL 2^32 operand pairs, NaN payloads
// included (checked exhaustively on the device: hoccl_selftest_bf16_add); a long chain of adds is issue bound without it.
__device__ __forceinline__ uint32_t add_bf16x2_native(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint4 add_vec_bf16_native(uint4 a, uint4 b) {
  uint4 r;
  r.x = add_bf16x2_native(a.x, b.x);
  r.y = add_bf16x2_native(a.y, b.y);
  r.z = add_bf16x2_native(a.z, b.z);
  r.w = add_bf16x2_native(a.w, b.w);
  return r;
}
template <>
struct Traits<1> {  // bf16
  static constexpr int E = 2;
  static constexpr int VE = 8;
  __device__ static __forceinline__ uint4 add_vec(uint4 a, uint4 b) {
    uint4 r;
    r.x = add_bf16x2(a.x, b.x);
    r.y = add_bf16x2(a.y, b.y);
    r.z = add_bf16x2(a.z, b.z);
    r.w = add_bf16x2(a.w, b.w);
    return r;
  }
  __device__ static __forceinline__ void add_scalar(const void* a, const void* b, void* o, unsigned long long i) {
    const unsigned short* pa = static_cast<const unsigned short*>(a);
    const unsigned short* pb = static_cast<const unsigned short*>(b);
    float s = __fadd_rn(__uint_as_float((uint32_t)pa[i] << 16), __uint_as_float((uint32_t)pb[i] << 16));
    __nv_bfloat16 h = __float2bfloat16_rn(s);
    static_cast<unsigned short*>(o)[i] = __bfloat16_as_ushort(h);
  }
};

__host__ __device__ __forceinline__ void split_segment(unsigned long long n, unsigned mis, bool congruent, int E, int VE,
                                              unsigned* head, unsigned long long* nvec, unsigned long long* nscalar) {
  if (congruent && (mis % E) == 0) {
    unsigned long long h = ((16u - mis) & 15u) / E;
    if (h > n) h = n;
    *head = (unsigned)h;
    *nvec = (n - h) / VE;
    *nscalar = n - *nvec * VE;
  } else {
    *head = 0;
    *nvec = 0;
    *nscalar = n;
  }
}

}  // namespace
}  // namespace hoccl
