// Shared device helpers for the SRM kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace srm {

typedef __nv_bfloat16 bf16;
typedef __half fp16;                 // cache storage only: values are clamped to the finite fp16 range when stored

constexpr uint32_t kStatusTokenRange = 1u;
constexpr uint32_t kStatusWaitTimeout = 2u;
constexpr uint32_t kStatusNonFinite = 4u;

__device__ __forceinline__ void raise_status(uint32_t* status, uint32_t bit) {
  if (status != nullptr) atomicOr(status, bit);
}

// Programmatic dependent launch. Every kernel of this library is launched with the programmatic
// stream-serialization attribute: it may start while its predecessor in the stream is still draining,
// runs whatever does not touch global memory, and calls pdl_wait() before its first global access
// (the wait returns once the predecessor grid has completed and its writes are visible). pdl_trigger()
// lets the successor start launching; it only affects when that grid is scheduled, never its ordering.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Device-side step counters (words 1..3 of the state header; word 0 is the status word). When a decode
// step is replayed from a CUDA graph its kernel arguments are frozen, so the values that change from step
// to step are read from here instead, and a one-thread kernel advances them at the end of every step.
constexpr int kCtrPos = 1;     // absolute position of the token being consumed
constexpr int kCtrStep = 2;    // Philox step of the selection
constexpr int kCtrCol = 3;     // column of the token store the selection writes
constexpr int kCtrHandedBack = 4;   // rows the fused top-k selection handed back to the logits path, since the last reset

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- 4-wide loads/stores of the three storage types, always handled as float4 in registers ----
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 ld4(const bf16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
__device__ __forceinline__ float4 ld4(const fp16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  const float2 fa = __half22float2(*reinterpret_cast<__half2*>(&u.x)), fb = __half22float2(*reinterpret_cast<__half2*>(&u.y));
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ float clamp_fp16(float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); }
__device__ __forceinline__ void st4(fp16* p, float4 v) {
  __half2 a = __floats2half2_rn(clamp_fp16(v.x), clamp_fp16(v.y));
  __half2 b = __floats2half2_rn(clamp_fp16(v.z), clamp_fp16(v.w));
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
// read-only (parameter) variants
__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 ldg4(const bf16* p) {
  uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_float(fp16 v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ fp16 from_float<fp16>(float v) { return __float2half_rn(clamp_fp16(v)); }

// exact (erf) GELU in fp32
__device__ __forceinline__ float gelu_erf(float v) {
  return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f));
}

}  // namespace srm
