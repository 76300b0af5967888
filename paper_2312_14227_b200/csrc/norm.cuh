// Layer normalisation as a member of the stack (Section 5.2: a normalisation layer carries two
// trainable tensors, Gamma and Beta).  Memory-bound row kernels: one warp owns a row at a time and
// keeps it in registers, so every activation byte crosses HBM once per pass.
//
//   forward   xhat = (x - mean) * rstd,  y = xhat * gamma + beta;  (mean, rstd) kept per row
//   backward  gy = g * gamma
//             dx = rstd * (gy - mean_row(gy) - xhat * mean_row(gy * xhat))   (+ skip gradient)
//             d gamma = column sums of g * xhat   (per-block partials, finished by bias_finish_kernel)
//             d beta  = column sums of g          (the bias-gradient path of the stack)
#pragma once

#include "common.cuh"

namespace et {

constexpr int kNormThreads = 256;
constexpr int kNormWarps = kNormThreads / 32;
constexpr int kNormMaxWidth = 2048;             // 8 register chunks of 8 elements per lane

// Lane `lane` holds, for chunk c = 0 .. VPL-1, the 8 consecutive columns starting at
// (c * 32 + lane) * 8; chunks past the row's end read as zeros.  d is a multiple of 8.
template <typename T, int VPL>
__device__ __forceinline__ void norm_load_row(const T* __restrict__ row, int d, int lane, float (&v)[VPL * 8]) {
#pragma unroll
  for (int c = 0; c < VPL; ++c) {
    const int col = (c * 32 + lane) * 8;
    float t[8];
    if (col < d) {
      load_seg<8>(row + col, 8, t);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) t[e] = 0.0f;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) v[c * 8 + e] = t[e];
  }
}
template <typename T, int VPL>
__device__ __forceinline__ void norm_store_row(T* __restrict__ row, int d, int lane, const float (&v)[VPL * 8]) {
#pragma unroll
  for (int c = 0; c < VPL; ++c) {
    const int col = (c * 32 + lane) * 8;
    if (col < d) {
      float t[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) t[e] = v[c * 8 + e];
      store_seg<8>(row + col, 8, t);
    }
  }
}

template <typename T, int VPL>
__global__ void __launch_bounds__(kNormThreads)
norm_forward_kernel(const T* __restrict__ x, const T* __restrict__ gamma, const T* __restrict__ beta,
                    T* __restrict__ y, float2* __restrict__ stats, int M, int d, float eps) {
  const int lane = threadIdx.x & 31;
  const int warp = blockIdx.x * kNormWarps + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * kNormWarps;
  float g[VPL * 8], b[VPL * 8];
  norm_load_row<T, VPL>(gamma, d, lane, g);
  norm_load_row<T, VPL>(beta, d, lane, b);
  const float inv_d = 1.0f / (float)d;
  for (int r = warp; r < M; r += nwarps) {
    float v[VPL * 8];
    norm_load_row<T, VPL>(x + (size_t)r * d, d, lane, v);
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL * 8; ++i) s += v[i];
    const float mean = warp_sum(s) * inv_d;
    float q = 0.0f;
#pragma unroll
    for (int c = 0; c < VPL; ++c) {
      const bool in = (c * 32 + lane) * 8 < d;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float t = v[c * 8 + e] - mean;
        q += in ? t * t : 0.0f;
      }
    }
    const float rstd = rsqrtf(warp_sum(q) * inv_d + eps);
#pragma unroll
    for (int i = 0; i < VPL * 8; ++i) v[i] = (v[i] - mean) * rstd * g[i] + b[i];
    norm_store_row<T, VPL>(y + (size_t)r * d, d, lane, v);
    if (lane == 0) stats[r] = make_float2(mean, rstd);
  }
}

// WANT_DX: the error gradient G_l (optionally + skip), and dZ_{l-1} = G_l * act'(Z_{l-1}) when the
// layer below has an activation.  WANT_DG: per-block partial column sums of g * xhat into
// gpart[blockIdx.x][d] (every block writes its row, zeros included).
template <typename T, int VPL, bool WANT_DX, bool WANT_DG>
__global__ void __launch_bounds__(kNormThreads)
norm_backward_kernel(const T* __restrict__ g_out, const T* __restrict__ x, const float2* __restrict__ stats,
                     const T* __restrict__ gamma, const T* __restrict__ skip, T* __restrict__ G_in,
                     const T* __restrict__ z_prev, T* __restrict__ dz_prev, int act_prev,
                     float* __restrict__ gpart, int M, int d) {
  __shared__ float red[WANT_DG ? VPL * 8 * 32 : 1];
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  const int warp = blockIdx.x * kNormWarps + wib;
  const int nwarps = gridDim.x * kNormWarps;
  float gam[VPL * 8], acc[VPL * 8];
  if constexpr (WANT_DX) norm_load_row<T, VPL>(gamma, d, lane, gam);
#pragma unroll
  for (int i = 0; i < VPL * 8; ++i) acc[i] = 0.0f;
  const float inv_d = 1.0f / (float)d;
  for (int r = warp; r < M; r += nwarps) {
    float g[VPL * 8], xh[VPL * 8];
    norm_load_row<T, VPL>(g_out + (size_t)r * d, d, lane, g);
    norm_load_row<T, VPL>(x + (size_t)r * d, d, lane, xh);
    const float2 st = stats[r];
#pragma unroll
    for (int i = 0; i < VPL * 8; ++i) xh[i] = (xh[i] - st.x) * st.y;
    if constexpr (WANT_DG) {
#pragma unroll
      for (int i = 0; i < VPL * 8; ++i) acc[i] = fmaf(g[i], xh[i], acc[i]);   // g is 0 past the row's end
    }
    if constexpr (WANT_DX) {
      float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
      for (int i = 0; i < VPL * 8; ++i) {
        g[i] *= gam[i];                                                      // gy
        s1 += g[i];
        s2 = fmaf(g[i], xh[i], s2);
      }
      const float c1 = warp_sum(s1) * inv_d, c2 = warp_sum(s2) * inv_d;
#pragma unroll
      for (int i = 0; i < VPL * 8; ++i) g[i] = st.y * (g[i] - c1 - xh[i] * c2);
      if (skip != nullptr) {
        norm_load_row<T, VPL>(skip + (size_t)r * d, d, lane, xh);
#pragma unroll
        for (int i = 0; i < VPL * 8; ++i) g[i] += xh[i];
      }
      if (G_in != nullptr) norm_store_row<T, VPL>(G_in + (size_t)r * d, d, lane, g);
      if (dz_prev != nullptr) {
        norm_load_row<T, VPL>(z_prev + (size_t)r * d, d, lane, xh);
#pragma unroll
        for (int i = 0; i < VPL * 8; ++i) g[i] *= act_grad(xh[i], act_prev);
        norm_store_row<T, VPL>(dz_prev + (size_t)r * d, d, lane, g);
      }
    }
  }
  if constexpr (WANT_DG) {
    // the block's warps add their sums one after the other: fixed order, no atomics
    for (int w = 0; w < kNormWarps; ++w) {
      if (wib == w) {
#pragma unroll
        for (int i = 0; i < VPL * 8; ++i) {
          const int at = i * 32 + lane;
          red[at] = (w == 0 ? 0.0f : red[at]) + acc[i];
        }
      }
      __syncthreads();
    }
    for (int at = threadIdx.x; at < VPL * 8 * 32; at += kNormThreads) {
      const int i = at >> 5, ln = at & 31;
      const int col = ((i >> 3) * 32 + ln) * 8 + (i & 7);
      if (col < d) gpart[(size_t)blockIdx.x * d + col] = red[at];
    }
  }
}

}  // namespace et
