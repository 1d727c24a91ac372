// kf_act.cuh -- epilogue arithmetic shared by the kernels: activations in fp32 registers,
// bf16 <-> fp32 conversion, and the enum values of the C ABI as plain ints.
#pragma once

#include <cuda_bf16.h>
#include <cstdint>
#include <type_traits>

namespace kf {

enum : int { ACT_NONE = 0, ACT_RELU = 1, ACT_GELU_TANH = 2, ACT_SIGMOID = 3, ACT_GELU_ERF = 4,
             ACT_SWISH = 5, ACT_TANH = 6, ACT_HARDTANH = 7, ACT_CHAIN95 = 8,
             // the codes below share ONE kernel instantiation (ACT_RUNTIME) and are told apart by
             // a switch on the run-time code inside the epilogue
             ACT_LEAKY_RELU = 9, ACT_ELU = 10, ACT_MISH = 11, ACT_HARDSWISH = 12, ACT_SOFTPLUS = 13,
             ACT_RELU6 = 14, ACT_HARDSIGMOID = 15, ACT_COUNT = 16, ACT_RUNTIME = 100 };
enum : int { RED_SOFTMAX = 0, RED_SUM = 1, RED_MAX = 2, RED_MEAN = 3, RED_LOGSUMEXP = 4, RED_COUNT = 5 };
enum : int { DT_F32 = 0, DT_BF16 = 1 };

__device__ __forceinline__ float tanh_approx(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// FAST = true: one MUFU op per transcendental (tanh.approx / ex2.approx); absolute error a few
// 1e-4 at most, meant for chains whose output is rounded to bf16.  FAST = false: libdevice
// single-precision routines (about 1 ulp), meant for fp32 chains.
template <bool FAST>
__device__ __forceinline__ float sigmoid_f(float z) {
  if constexpr (FAST) return fmaf(0.5f, tanh_approx(0.5f * z), 0.5f);
  else return 1.0f / (1.0f + expf(-z));
}
template <bool FAST>
__device__ __forceinline__ float tanh_f(float z) {
  if constexpr (FAST) return tanh_approx(z);
  else return tanhf(z);
}
template <bool FAST>
__device__ __forceinline__ float gelu_tanh_f(float z) {
  const float u = 0.7978845608028654f * fmaf(0.044715f * z * z, z, z);
  const float h = 0.5f * z;
  return fmaf(h, tanh_f<FAST>(u), h);
}
__device__ __forceinline__ float gelu_erf_f(float z) {
  return z * 0.5f * (1.0f + erff(z * 0.7071067811865475f));
}

// log(1 + e^z) without overflow
template <bool FAST>
__device__ __forceinline__ float softplus_f(float z) {
  if constexpr (FAST) return fmaxf(z, 0.0f) + __logf(1.0f + __expf(-fabsf(z)));
  else return fmaxf(z, 0.0f) + log1pf(expf(-fabsf(z)));
}
// The activations selected at run time (PyTorch's definitions and default parameters).
template <bool FAST>
__device__ __forceinline__ float act_rt(int code, float z) {
  switch (code) {
    case ACT_LEAKY_RELU: return z > 0.0f ? z : 0.01f * z;
    case ACT_ELU: return z > 0.0f ? z : (FAST ? __expf(z) - 1.0f : expm1f(z));
    case ACT_MISH: return z * tanh_f<FAST>(softplus_f<FAST>(z));
    case ACT_HARDSWISH: return z * fminf(fmaxf(z + 3.0f, 0.0f), 6.0f) * (1.0f / 6.0f);
    case ACT_SOFTPLUS: return softplus_f<FAST>(z);
    case ACT_RELU6: return fminf(fmaxf(z, 0.0f), 6.0f);
    case ACT_HARDSIGMOID: return fminf(fmaxf(fmaf(z, 1.0f / 6.0f, 0.5f), 0.0f), 1.0f);
    default: return z;
  }
}

// `code` is read only by the ACT_RUNTIME instantiation.
template <int ACT, bool FAST>
__device__ __forceinline__ float act_f(float z, int code = 0) {
  if constexpr (ACT == ACT_RUNTIME) return act_rt<FAST>(code, z);
  else if constexpr (ACT == ACT_NONE) return z;
  else if constexpr (ACT == ACT_RELU) return fmaxf(z, 0.0f);
  else if constexpr (ACT == ACT_GELU_TANH) return gelu_tanh_f<FAST>(z);
  else if constexpr (ACT == ACT_SIGMOID) return sigmoid_f<FAST>(z);
  else if constexpr (ACT == ACT_GELU_ERF) return gelu_erf_f(z);
  else if constexpr (ACT == ACT_SWISH) return z * sigmoid_f<FAST>(z);
  else if constexpr (ACT == ACT_TANH) return tanh_f<FAST>(z);
  else if constexpr (ACT == ACT_HARDTANH) return fminf(fmaxf(z, -1.0f), 1.0f);
  else {  // ACT_CHAIN95: swish -> tanh -> GELU(erf) -> hardtanh
    const float s = z * sigmoid_f<FAST>(z);
    const float t = tanh_f<FAST>(s);
    const float g = gelu_erf_f(t);
    return fminf(fmaxf(g, -1.0f), 1.0f);
  }
}

// Any activation by its run-time code (scalar kernels where the epilogue is not the hot part).
template <bool FAST>
__device__ __forceinline__ float act_any(int code, float z) {
  switch (code) {
    case ACT_NONE: return z;
    case ACT_RELU: return act_f<ACT_RELU, FAST>(z);
    case ACT_GELU_TANH: return act_f<ACT_GELU_TANH, FAST>(z);
    case ACT_SIGMOID: return act_f<ACT_SIGMOID, FAST>(z);
    case ACT_GELU_ERF: return act_f<ACT_GELU_ERF, FAST>(z);
    case ACT_SWISH: return act_f<ACT_SWISH, FAST>(z);
    case ACT_TANH: return act_f<ACT_TANH, FAST>(z);
    case ACT_HARDTANH: return act_f<ACT_HARDTANH, FAST>(z);
    case ACT_CHAIN95: return act_f<ACT_CHAIN95, FAST>(z);
    default: return act_rt<FAST>(code, z);
  }
}

// Runtime-to-compile-time dispatch over the activation code.
template <typename F>
__host__ inline bool dispatch_act(int act, F&& f) {
  switch (act) {
    case ACT_NONE: f(std::integral_constant<int, ACT_NONE>{}); return true;
    case ACT_RELU: f(std::integral_constant<int, ACT_RELU>{}); return true;
    case ACT_GELU_TANH: f(std::integral_constant<int, ACT_GELU_TANH>{}); return true;
    case ACT_SIGMOID: f(std::integral_constant<int, ACT_SIGMOID>{}); return true;
    case ACT_GELU_ERF: f(std::integral_constant<int, ACT_GELU_ERF>{}); return true;
    case ACT_SWISH: f(std::integral_constant<int, ACT_SWISH>{}); return true;
    case ACT_TANH: f(std::integral_constant<int, ACT_TANH>{}); return true;
    case ACT_HARDTANH: f(std::integral_constant<int, ACT_HARDTANH>{}); return true;
    case ACT_CHAIN95: f(std::integral_constant<int, ACT_CHAIN95>{}); return true;
    case ACT_LEAKY_RELU: case ACT_ELU: case ACT_MISH: case ACT_HARDSWISH: case ACT_SOFTPLUS:
    case ACT_RELU6: case ACT_HARDSIGMOID:
      f(std::integral_constant<int, ACT_RUNTIME>{}); return true;
  }
  return false;
}

// ---------------------------------------------------------------- storage conversion
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);  // .x = lo (low 16 bits), .y = hi
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

}  // namespace kf
