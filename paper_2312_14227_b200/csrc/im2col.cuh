// Patch gather of a k x k convolution (stride 1, zero padding k / 2) on NHWC rows, and its
// backward.  Together with the dense layer that follows it in the stack this is the convolutional
// layer of Section 5.1: the dense layer's kernel is the convolution kernel in (kh, kw, c_in) x c_out
// layout, so the three backward operations of the convolution (error gradient, kernel update, bias
// update) are the dense layer's dgrad / wgrad / bias kernels on the gathered rows.
//
//   forward   col[(n,h,w), (kh*k + kw)*C + c] = x[(n, h + kh - p, w + kw - p), c]     0 outside the image
//   backward  dx[(n,h,w), c] = sum over taps of dcol[(n, h - kh + p, w - kw + p), (kh*k + kw)*C + c]
//             (+ skip gradient), and dZ of the layer below = dx * act'(Z) when that layer has an activation
//
// HBM-bound gathers: one thread moves 8 channels (16 bytes of bf16) at a time; the gathered matrix is
// k*k times the activation, which is what an explicit gather costs; fetching the patches inside the
// GEMM's own operand loads instead is the next step.
#pragma once

#include "common.cuh"

namespace et {

constexpr int kGatherThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kGatherThreads)
im2col_kernel(const T* __restrict__ x, T* __restrict__ col, long long M, int H, int W, int C, int k) {
  const int chunks = C / 8;                        // C is a multiple of 8
  const long long total = M * k * k * chunks;
  const long long i = (long long)blockIdx.x * kGatherThreads + threadIdx.x;
  if (i >= total) return;
  const int ch = (int)(i % chunks);
  const int tap = (int)((i / chunks) % (k * k));
  const long long m = i / ((long long)chunks * k * k);
  const int w = (int)(m % W), h = (int)((m / W) % H);
  const int hs = h + tap / k - k / 2, ws = w + tap % k - k / 2;
  float v[8];
  if (hs >= 0 && hs < H && ws >= 0 && ws < W) {
    load_seg<8>(x + (m + (long long)(hs - h) * W + (ws - w)) * C + ch * 8, 8, v);
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = 0.0f;
  }
  store_seg<8>(col + (m * k * k + tap) * C + ch * 8, 8, v);
}

// G_in / dz_prev may be null (not needed); skip may be null.
template <typename T>
__global__ void __launch_bounds__(kGatherThreads)
col2im_kernel(const T* __restrict__ dcol, const T* __restrict__ skip, T* __restrict__ G_in,
              const T* __restrict__ z_prev, T* __restrict__ dz_prev, int act_prev, long long M, int H, int W, int C,
              int k) {
  const int chunks = C / 8;
  const long long i = (long long)blockIdx.x * kGatherThreads + threadIdx.x;
  if (i >= M * chunks) return;
  const int ch = (int)(i % chunks);
  const long long m = i / chunks;
  const int w = (int)(m % W), h = (int)((m / W) % H);
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
  for (int kh = 0; kh < k; ++kh) {
    const int ho = h - kh + k / 2;                 // the output pixel whose patch holds (h, w) in tap (kh, kw)
    if (ho < 0 || ho >= H) continue;
    for (int kw = 0; kw < k; ++kw) {
      const int wo = w - kw + k / 2;
      if (wo < 0 || wo >= W) continue;
      float v[8];
      load_seg<8>(dcol + ((m + (long long)(ho - h) * W + (wo - w)) * k * k + kh * k + kw) * C + ch * 8, 8, v);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += v[e];
    }
  }
  const size_t at = (size_t)m * C + ch * 8;
  if (skip != nullptr) {
    float v[8];
    load_seg<8>(skip + at, 8, v);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] += v[e];
  }
  if (G_in != nullptr) store_seg<8>(G_in + at, 8, acc);
  if (dz_prev != nullptr) {
    float z[8];
    load_seg<8>(z_prev + at, 8, z);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] *= act_grad(z[e], act_prev);
    store_seg<8>(dz_prev + at, 8, acc);
  }
}

}  // namespace et
