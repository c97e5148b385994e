// Small device helpers shared by the kernels: 16-byte vector access for fp32 / bf16 rows,
// warp and block reductions, activation functions (all arithmetic in fp32).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cmath>
#include <cstdlib>
#include <utility>

#include "kernels.h"

namespace fluid {

// Programmatic dependent launch: a kernel lets its successor start early (the successor's CTAs run
// their prologue on idle SMs) and every kernel waits for its predecessor's memory before it
// touches global memory. Cuts the launch gap between the many small steps of a plan.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

inline bool pdl_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("FLUID_PDL");
    return !(e && e[0] == '0');
  }();
  return on;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

template <typename T>
struct VecOf {
  static constexpr int N = 16 / sizeof(T);
};

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f(float v);
template <>
__device__ __forceinline__ float from_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16-byte load of VecOf<T>::N elements, widened to fp32
__device__ __forceinline__ void load16(const float* p, float (&v)[4]) {
  const float4 q = *reinterpret_cast<const float4*>(p);
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load16(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void store16(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void store16(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 q;
  q.x = pack_bf16x2(v[0], v[1]);
  q.y = pack_bf16x2(v[2], v[3]);
  q.z = pack_bf16x2(v[4], v[5]);
  q.w = pack_bf16x2(v[6], v[7]);
  *reinterpret_cast<uint4*>(p) = q;
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

// Sum across the block; `red` is 32 floats of shared memory. Every thread gets the total.
__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();  // protect `red` from the previous use
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = lane < nw ? red[lane] : 0.f;
  return warp_sum(t);
}

__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }
// GELU (erf form) on the fused-multiply-add pipe only: erf(z) = z * P(z^2) with a 9-term least-squares fit on
// |z| <= 2.9 (|error| < 1.3e-5; beyond, z is clamped and erf stays within 3e-5 of +-1), so the absolute error of
// the result is below 2.2e-5 for |x| <= 4.1 and below 1.7e-5 |x| after that: far under bf16 resolution of the
// outputs it is used for. No reciprocal and no exponential: a GEMM epilogue that applies this to every element
// of a 128 x 256 tile would otherwise spend 4000 cycles in the special-function unit alone.
__device__ __forceinline__ float gelu_erf_fast(float x) {
  const float z = fminf(fmaxf(x * 0.70710678118654752f, -2.9f), 2.9f);
  const float u = z * z;
  float q = fmaf(4.85526996385488e-08f, u, -2.210898173871101e-06f);
  q = fmaf(q, u, 4.476702451938763e-05f);
  q = fmaf(q, u, -0.0005382060771808028f);
  q = fmaf(q, u, 0.004347700159996748f);
  q = fmaf(q, u, -0.02536272630095482f);
  q = fmaf(q, u, 0.11139318346977234f);
  q = fmaf(q, u, -0.375481516122818f);
  q = fmaf(q, u, 1.128293514251709f);
  const float half_x = 0.5f * x;
  return fmaf(half_x, q * z, half_x);
}
// Two fp32 values in one 64-bit register: one issue slot for two fused multiply-adds or products (sm_100 packed fp32).
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// gelu_erf_fast on two values at once: the same operations in the same order, each a packed instruction, so the results
// are bit-identical to the scalar form at half the issue slots (a 128 x 256 GELU tile of a K = 768 GEMM otherwise takes
// its epilogue warps longer than the tensor cores take to produce the next tile).
__device__ __forceinline__ void gelu_erf_fast2(float& x0, float& x1) {
  const uint64_t x = f32x2_pack(x0, x1);
  float z0, z1;
  f32x2_unpack(f32x2_mul(x, f32x2_pack(0.70710678118654752f, 0.70710678118654752f)), z0, z1);
  z0 = fminf(fmaxf(z0, -2.9f), 2.9f);
  z1 = fminf(fmaxf(z1, -2.9f), 2.9f);
  const uint64_t z = f32x2_pack(z0, z1);
  const uint64_t u = f32x2_mul(z, z);
  auto k2 = [](float c) { return f32x2_pack(c, c); };
  uint64_t q = f32x2_fma(k2(4.85526996385488e-08f), u, k2(-2.210898173871101e-06f));
  q = f32x2_fma(q, u, k2(4.476702451938763e-05f));
  q = f32x2_fma(q, u, k2(-0.0005382060771808028f));
  q = f32x2_fma(q, u, k2(0.004347700159996748f));
  q = f32x2_fma(q, u, k2(-0.02536272630095482f));
  q = f32x2_fma(q, u, k2(0.11139318346977234f));
  q = f32x2_fma(q, u, k2(-0.375481516122818f));
  q = f32x2_fma(q, u, k2(1.128293514251709f));
  const uint64_t half_x = f32x2_mul(x, k2(0.5f));
  f32x2_unpack(f32x2_fma(half_x, f32x2_mul(q, z), half_x), x0, x1);
}
__device__ __forceinline__ float gelu_tanh(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return 0.5f * x * (1.f + tanhf(u));
}
// Rotary angle pos * f as (sin, cos), f = base^(-2i/D) = hi + lo. All in fp32 (double-precision arithmetic runs at a
// small fraction of the fp32 rate on this part: 64 angles per thread in a GEMM epilogue cost 20 us of a 140 us step
// when the product and the reduction were done in double). The product pos * hi is rounded once and its exact error
// (one fused multiply-add) goes back in together with pos * lo; the reduction to [-pi, pi] subtracts k * 2 pi in two
// fused steps (2 pi = 6.2831854820251465 - 1.7484555e-7). Absolute error of the reduced angle ~3e-7 rad at any
// position below 2^24, against ~2e-3 rad at position 2047 when everything is plain fp32; the hardware sine / cosine
// add about 2^-21.
__device__ __forceinline__ void rope_sincos(int pos, float f_hi, float f_lo, float& sn, float& cs) {
  const float pf = (float)pos;
  const float ang = pf * f_hi;
  float e = fmaf(pf, f_hi, -ang);
  e = fmaf(pf, f_lo, e);
  const float k = rintf(ang * 0.15915494309189535f);
  float r = fmaf(-k, 6.2831854820251465f, ang);
  r = fmaf(-k, -1.7484555e-7f, r);
  r += e;
  sn = __sinf(r);
  cs = __cosf(r);
}
// frequency i of a table (pairs beyond the table: computed here, in double, once per call site)
__device__ __forceinline__ void rope_freq(const RopeFreq& t, int i, int D, float& hi, float& lo) {
  if (i < 64) { hi = t.hi[i]; lo = t.lo[i]; return; }
  const double f = exp2(-2.0 * i / D * t.log2_base);
  hi = (float)f;
  lo = (float)(f - (double)hi);
}
__device__ __forceinline__ float silu(float x) { return x / (1.f + __expf(-x)); }

}  // namespace fluid
