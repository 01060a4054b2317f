// Shared device/host helpers for the TarFlow selective-Jacobi kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

// Device error word (one per model, in global memory).  A kernel that gives up on a bounded wait
// stores a non-zero code here and returns; the host reads it at the next synchronising call.
enum : int {
  TFERR_NONE = 0,
  TFERR_WAIT_FULL = 1,        // MMA warp: operand stage never arrived
  TFERR_WAIT_EMPTY = 2,       // TMA warp: stage never released
  TFERR_WAIT_TMEM_FULL = 3,   // epilogue: accumulator never committed
  TFERR_WAIT_TMEM_EMPTY = 4,  // MMA warp: accumulator never drained
  TFERR_WAIT_SELFTEST = 9,    // the bounded-wait self-test (a wait nothing satisfies) ran out, as it must
};

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(bf16 x) { return __bfloat162float(x); }
template <class T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float gelu_erf(float x) {
  return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f));
}

// GELU for results that are rounded to bf16 (or to a bf16 pair with 16 significant bits) anyway:
// erf(z), z >= 0, as 1 - 2^p(z) with a degree-7 polynomial p fitted to log2(erfc) on [0, 4]
// (coefficients and the error bound come from fit_gelu_poly.py beside this file; |erf error| <= 1.7e-7
// in fp32).  One exp2 and seven FMAs; the library erff costs about three times as much.
__device__ __forceinline__ float gelu_erf_fast(float x) {
  const float z = fminf(fabsf(x) * 0.70710678118654752440f, 4.0f);
  float p = fmaf(1.0021848e-4f, z, -4.6155503e-4f);
  p = fmaf(p, z, -2.302284e-3f);
  p = fmaf(p, z, 2.945257e-2f);
  p = fmaf(p, z, -1.489637e-1f);
  p = fmaf(p, z, -9.1832864e-1f);
  p = fmaf(p, z, -1.6279137f);
  const float erfc_abs = exp2f(p * z);            // erfc(|x| / sqrt 2)
  const float hx = 0.5f * x;
  return fmaf(fabsf(hx), 1.0f - erfc_abs, hx);   // 0.5 x (1 + erf(x / sqrt 2)) with erf odd
}

// Packed fp32 arithmetic (two lanes per instruction), three-input maximum and the bare exp2 unit.
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(d)
      : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)),
        "l"(*reinterpret_cast<unsigned long long*>(&c)));
  return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;"
      : "=l"(d)
      : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)));
  return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2_approx(float a) {
  float d;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(d) : "f"(a));
  return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;"
      : "=l"(d)
      : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)));
  return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 fabs2(float2 a) {
  unsigned long long d = *reinterpret_cast<unsigned long long*>(&a) & 0x7fffffff7fffffffull;
  return *reinterpret_cast<float2*>(&d);
}

// gelu_erf_fast on two values at once with the packed instructions: about half the issue slots per value.
__device__ __forceinline__ float2 gelu_erf_fast2(float2 x) {
  float2 z = fmul2(fabs2(x), make_float2(0.70710678118654752440f, 0.70710678118654752440f));
  z.x = fminf(z.x, 4.0f);
  z.y = fminf(z.y, 4.0f);
  float2 p = ffma2(make_float2(1.0021848e-4f, 1.0021848e-4f), z, make_float2(-4.6155503e-4f, -4.6155503e-4f));
  p = ffma2(p, z, make_float2(-2.302284e-3f, -2.302284e-3f));
  p = ffma2(p, z, make_float2(2.945257e-2f, 2.945257e-2f));
  p = ffma2(p, z, make_float2(-1.489637e-1f, -1.489637e-1f));
  p = ffma2(p, z, make_float2(-9.1832864e-1f, -9.1832864e-1f));
  p = ffma2(p, z, make_float2(-1.6279137f, -1.6279137f));
  const float2 t = fmul2(p, z);
  float2 e;  // erfc(|x| / sqrt 2)
  e.x = ex2_approx(t.x);
  e.y = ex2_approx(t.y);
  const float2 hx = fmul2(x, make_float2(0.5f, 0.5f));
  const float2 erf_abs = ffma2(e, make_float2(-1.0f, -1.0f), make_float2(1.0f, 1.0f));
  return ffma2(fabs2(hx), erf_abs, hx);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// max over non-negative floats (and NaN, whose bit pattern compares above +inf) through integer
// atomics: for x >= 0 the IEEE bit pattern is monotone in x, so the result is order independent.
__device__ __forceinline__ void atomic_max_nonneg(float* addr, float v) {
  atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
}

// Core position l of a block <-> raster token index (block permutation: reversal on odd blocks).
__device__ __forceinline__ int tok_index(int l, int L, int reversed) { return reversed ? (L - 1 - l) : l; }

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may be scheduled
// while its predecessor in the stream still runs; it must not touch anything the predecessor reads or writes
// before pdl_wait(), which returns once the predecessor has completed and its writes are visible.
// pdl_launch_dependents() lets the successor's CTAs be scheduled as soon as every CTA of this kernel has
// called it.  Both are no-ops in a kernel launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
