// Shared device helpers: storage-type conversion, 16-byte vector access, block reductions.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace et {

using bf16 = __nv_bfloat16;

// Activation codes mirror et_act in et.h.
constexpr int kActNone = 0, kActGelu = 1, kActRelu = 2;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// tanh-form GELU and its derivative, fp32.  tanh(u) = 1 - 2 / (exp(2u) + 1): exp overflow
// gives exactly 1, underflow exactly -1, and the absolute error stays near 1e-7.
__device__ __forceinline__ float tanh_f32(float u) {
  float e = __expf(2.0f * u);
  return 1.0f - __fdividef(2.0f, e + 1.0f);
}
__device__ __forceinline__ float gelu_tanh(float z) {
  const float c0 = 0.7978845608028654f, c1 = 0.044715f;
  float u = c0 * (z + c1 * z * z * z);
  return 0.5f * z * (1.0f + tanh_f32(u));
}
__device__ __forceinline__ float gelu_tanh_grad(float z) {
  const float c0 = 0.7978845608028654f, c1 = 0.044715f;
  float z2 = z * z;
  float u = c0 * (z + c1 * z * z2);
  float t = tanh_f32(u);
  float du = c0 * (1.0f + 3.0f * c1 * z2);
  return 0.5f * (1.0f + t) + 0.5f * z * (1.0f - t * t) * du;
}
__device__ __forceinline__ float act_apply(float z, int act) {
  if (act == kActGelu) return gelu_tanh(z);
  if (act == kActRelu) return z > 0.0f ? z : 0.0f;
  return z;
}
__device__ __forceinline__ float act_grad(float z, int act) {
  if (act == kActGelu) return gelu_tanh_grad(z);
  if (act == kActRelu) return z > 0.0f ? 1.0f : 0.0f;
  return 1.0f;
}

// bf16-storage variants: tanh from the MUFU unit (tanh.approx.f32, relative error about 2^-11,
// below the 2^-9 rounding of the bf16 value the result is stored as).
__device__ __forceinline__ float tanh_fast(float u) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return t;
}
__device__ __forceinline__ float act_apply_fast(float z, int act) {
  if (act == kActGelu) {
    const float c0 = 0.7978845608028654f, c1 = 0.044715f;
    return 0.5f * z * (1.0f + tanh_fast(c0 * (z + c1 * z * z * z)));
  }
  if (act == kActRelu) return z > 0.0f ? z : 0.0f;
  return z;
}
__device__ __forceinline__ float act_grad_fast(float z, int act) {
  if (act == kActGelu) {
    const float c0 = 0.7978845608028654f, c1 = 0.044715f;
    const float z2 = z * z;
    const float t = tanh_fast(c0 * (z + c1 * z * z2));
    const float du = c0 * (1.0f + 3.0f * c1 * z2);
    return 0.5f * (1.0f + t) + 0.5f * z * (1.0f - t * t) * du;
  }
  if (act == kActRelu) return z > 0.0f ? 1.0f : 0.0f;
  return 1.0f;
}

// tanh-GELU derivative for two values at a time in packed fp16 arithmetic (half the instructions
// of the fp32 form; fp16's 2^-11 rounding per operation stays below the 2^-9 rounding of the bf16
// value the product is stored as).  z is clamped to +-16, where the derivative has long saturated,
// so z^3 cannot overflow.
__device__ __forceinline__ float2 gelu_tanh_grad_x2(float z0, float z1) {
  const __half2 c0 = __float2half2_rn(0.7978845608028654f);
  const __half2 c1 = __float2half2_rn(0.044715f);
  const __half2 c3 = __float2half2_rn(3.0f * 0.044715f * 0.7978845608028654f);
  const __half2 half = __float2half2_rn(0.5f), one = __float2half2_rn(1.0f);
  const __half2 lim = __float2half2_rn(16.0f);
  __half2 z = __floats2half2_rn(z0, z1);
  z = __hmax2(__hmin2(z, lim), __hneg2(lim));
  const __half2 z2 = __hmul2(z, z);
  const __half2 u = __hmul2(c0, __hfma2(__hmul2(c1, z2), z, z));
  uint32_t ur = *reinterpret_cast<const uint32_t*>(&u), tr;
  asm("tanh.approx.f16x2 %0, %1;" : "=r"(tr) : "r"(ur));
  const __half2 t = *reinterpret_cast<const __half2*>(&tr);
  const __half2 du = __hfma2(c3, z2, c0);
  const __half2 a = __hfma2(half, t, half);
  const __half2 omt2 = __hfma2(__hneg2(t), t, one);
  const __half2 b = __hmul2(__hmul2(half, z), omt2);
  return __half22float2(__hfma2(b, du, a));
}

// ---- row segments: NV consecutive elements of one row, vectorised when aligned ----------
// `n` = how many of the NV elements exist (ragged right edge); the rest read as 0.
template <int NV>
__device__ __forceinline__ void load_seg(const float* p, int n, float (&v)[NV]) {
  if constexpr (NV % 4 == 0) {
    if (n >= NV && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < NV; i += 4) {
        float4 q = *reinterpret_cast<const float4*>(p + i);
        v[i] = q.x; v[i + 1] = q.y; v[i + 2] = q.z; v[i + 3] = q.w;
      }
      return;
    }
  }
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = i < n ? p[i] : 0.0f;
}
template <int NV>
__device__ __forceinline__ void load_seg(const bf16* p, int n, float (&v)[NV]) {
  if constexpr (NV % 8 == 0) {
    if (n >= NV && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < NV; i += 8) {
        uint4 q = *reinterpret_cast<const uint4*>(p + i);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[i + 2 * j] = __uint_as_float(w[j] << 16);
          v[i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
      }
      return;
    }
  }
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = i < n ? __bfloat162float(p[i]) : 0.0f;
}
template <int NV>
__device__ __forceinline__ void store_seg(float* p, int n, const float (&v)[NV]) {
  if constexpr (NV % 4 == 0) {
    if (n >= NV && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < NV; i += 4)
        *reinterpret_cast<float4*>(p + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
      return;
    }
  }
#pragma unroll
  for (int i = 0; i < NV; ++i)
    if (i < n) p[i] = v[i];
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
template <int NV>
__device__ __forceinline__ void store_seg(bf16* p, int n, const float (&v)[NV]) {
  if constexpr (NV % 8 == 0) {
    if (n >= NV && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < NV; i += 8) {
        uint4 q;
        q.x = pack_bf16x2(v[i], v[i + 1]);
        q.y = pack_bf16x2(v[i + 2], v[i + 3]);
        q.z = pack_bf16x2(v[i + 4], v[i + 5]);
        q.w = pack_bf16x2(v[i + 6], v[i + 7]);
        *reinterpret_cast<uint4*>(p + i) = q;
      }
      return;
    }
  }
#pragma unroll
  for (int i = 0; i < NV; ++i)
    if (i < n) p[i] = __float2bfloat16_rn(v[i]);
}

// ---- deterministic block reduction (fixed shuffle tree, fixed warp order) ----------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// All threads of a 1-D block must call; result valid in thread 0.  blockDim.x a multiple
// of 32, at most 1024.
__device__ __forceinline__ float block_sum(float v) {
  __shared__ float warp_part[32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();               // protects warp_part across back-to-back calls
  if (lane == 0) warp_part[wid] = v;
  __syncthreads();
  float r = 0.0f;
  if (wid == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    r = lane < nw ? warp_part[lane] : 0.0f;
    r = warp_sum(r);
  }
  return r;
}

}  // namespace et
