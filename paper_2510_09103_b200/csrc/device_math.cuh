// Device helpers shared by the kernels: gradient element traits, 128-bit loads/stores and the
// parameter update of Algorithm 1 line 9.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "adapm_internal.h"

namespace adapm {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// bf16 gradients: 8 elements = one 16-byte load, kept packed in registers
struct GradBF16 {
  using elem = uint16_t;
  using raw8 = uint4;
  static __device__ __forceinline__ raw8 load8(const elem* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  static __device__ __forceinline__ raw8 load8_guarded(const elem* p, int n) {
    uint32_t h[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) h[i] = (i < n) ? (uint32_t)p[i] : 0u;
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
  }
  static __device__ __forceinline__ void unpack(const raw8& r, float* f) {
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
  }
  static __device__ __forceinline__ float load1(const elem* p) { return bf16_bits_to_float(*p); }
};

struct F32x8 { float4 a, b; };

struct GradF32 {
  using elem = float;
  using raw8 = F32x8;
  static __device__ __forceinline__ raw8 load8(const elem* p) {
    raw8 r;
    r.a = __ldg(reinterpret_cast<const float4*>(p));
    r.b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    return r;
  }
  static __device__ __forceinline__ raw8 load8_guarded(const elem* p, int n) {
    float h[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) h[i] = (i < n) ? p[i] : 0.f;
    raw8 r;
    r.a = make_float4(h[0], h[1], h[2], h[3]);
    r.b = make_float4(h[4], h[5], h[6], h[7]);
    return r;
  }
  static __device__ __forceinline__ void unpack(const raw8& r, float* f) {
    f[0] = r.a.x; f[1] = r.a.y; f[2] = r.a.z; f[3] = r.a.w;
    f[4] = r.b.x; f[5] = r.b.y; f[6] = r.b.z; f[7] = r.b.w;
  }
  static __device__ __forceinline__ float load1(const elem* p) { return *p; }
};

__device__ __forceinline__ void load8f(const float* p, float* f) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *(reinterpret_cast<const float4*>(p) + 1);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
  f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

__device__ __forceinline__ void store8f(float* p, const float* f) {
  *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  *(reinterpret_cast<float4*>(p) + 1) = make_float4(f[4], f[5], f[6], f[7]);
}

// two floats -> packed bf16 pair, round to nearest even (x0 in the low half)
__device__ __forceinline__ uint32_t pack_bf16x2(float x0, float x1) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(x1), "f"(x0));
  return d;
}

// Algorithm 1 line 9: W - lr s_b ( clamp(m^c / (sqrt(v) + eps)) + lambda_b W ).
// Comparisons (not fminf/fmaxf) so that a NaN ratio stays NaN.
__device__ __forceinline__ float adapm_param_update(float w, float mc, float v, const StepScalars& sc, float lr_s,
                                                    float wd) {
  const float den = sqrtf(v * sc.inv_bc2) + sc.eps;
  float ratio = (mc * sc.inv_bc1) / den;
  ratio = ratio > sc.clip ? sc.clip : (ratio < -sc.clip ? -sc.clip : ratio);
  return w - lr_s * (ratio + wd * w);
}

}  // namespace adapm
