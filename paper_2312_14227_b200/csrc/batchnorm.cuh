// Batch normalisation (training mode: statistics of each feature over all rows) as a member of the
// stack, the layer Section 5.2 is written about; Gamma and Beta are selectable tensors.
//
//   forward   mean_c, var_c over the rows;  xhat = (x - mean_c) * rstd_c;  z = xhat * gamma + beta;  a = act(z)
//   backward  dz = g * act'(z) (formed by the layer above, like any layer with an activation)
//             s1_c = sum_rows dz,  s2_c = sum_rows dz * xhat          (d beta = s1, d gamma = s2)
//             dx = gamma_c * rstd_c * (dz - s1_c / M - xhat * s2_c / M)   (+ skip gradient)
//
// HBM-bound.  Column statistics are two-stage: per 128-row chunk partial sums (every chunk a block,
// fixed order inside), then one small kernel sums the chunks per column in a fixed order (no atomics).
// The variance is taken around the mean in a second pass over x, not as E[x^2] - mean^2.
#pragma once

#include "common.cuh"

namespace et {

constexpr int kBnRows = 128;      // rows per chunk of the column reductions

enum BnMode : int { kBnSum = 0, kBnCentredSquares = 1, kBnBackward = 2 };

// grid (ceil(C / 256), ceil(M / kBnRows)); block (32, 8): x -> 8 columns, y -> row phase.
//   kBnSum:            part0[chunk][c] = sum x
//   kBnCentredSquares: part0[chunk][c] = sum (x - mean_c)^2                      (stats.x = mean)
//   kBnBackward:       part0 = sum dz, part1 = sum dz * (x - mean_c) * rstd_c    (a = dz, b = x)
template <typename T, int MODE>
__global__ void __launch_bounds__(256)
bn_colstats_kernel(const T* __restrict__ a, const T* __restrict__ b, const float2* __restrict__ stats, int M, int C,
                   float* __restrict__ part0, float* __restrict__ part1) {
  __shared__ float sm[2][8][256 + 8];
  const int col0 = blockIdx.x * 256 + threadIdx.x * 8;
  const int r0 = blockIdx.y * kBnRows, r1 = min(M, r0 + kBnRows);
  float acc0[8], acc1[8], mean[8], rstd[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { acc0[i] = acc1[i] = 0.0f; mean[i] = 0.0f; rstd[i] = 1.0f; }
  const bool live = col0 < C;                      // C is a multiple of 8
  if (live && MODE != kBnSum) {
#pragma unroll
    for (int i = 0; i < 8; ++i) { const float2 s = stats[col0 + i]; mean[i] = s.x; rstd[i] = s.y; }
  }
  if (live) {
    for (int r = r0 + threadIdx.y; r < r1; r += 8) {
      float v[8];
      load_seg<8>(a + (size_t)r * C + col0, 8, v);
      if constexpr (MODE == kBnSum) {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc0[i] += v[i];
      } else if constexpr (MODE == kBnCentredSquares) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { const float t = v[i] - mean[i]; acc0[i] = fmaf(t, t, acc0[i]); }
      } else {
        float x[8];
        load_seg<8>(b + (size_t)r * C + col0, 8, x);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          acc0[i] += v[i];
          acc1[i] = fmaf(v[i], (x[i] - mean[i]) * rstd[i], acc1[i]);
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    sm[0][threadIdx.y][threadIdx.x * 8 + i] = acc0[i];
    if constexpr (MODE == kBnBackward) sm[1][threadIdx.y][threadIdx.x * 8 + i] = acc1[i];
  }
  __syncthreads();
  const int t = threadIdx.y * 32 + threadIdx.x;    // 256 threads: one column each, row phases in a fixed order
  const int col = blockIdx.x * 256 + t;
  if (col < C) {
    float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
    for (int y = 0; y < 8; ++y) {
      s0 += sm[0][y][t];
      if constexpr (MODE == kBnBackward) s1 += sm[1][y][t];
    }
    part0[(size_t)blockIdx.y * C + col] = s0;
    if constexpr (MODE == kBnBackward) part1[(size_t)blockIdx.y * C + col] = s1;
  }
}

// Sums the chunks of up to two partial arrays per column (block (32, 32): 32 columns, 32 chunk lanes, fixed
// order) and turns the sums into what the next pass needs:
//   what 0: stats[c].x = s0 / M                    (mean)
//   what 1: stats[c].y = rsqrt(s0 / M + eps)       (1 / standard deviation)
//   what 2: means[c] = (s0 / M, s1 / M)            (the two column means of the backward formula)
static __global__ void __launch_bounds__(1024)
bn_finalize_kernel(const float* __restrict__ part0, const float* __restrict__ part1, int chunks, int C, float inv_m,
                   float eps, int what, float2* __restrict__ stats, float2* __restrict__ means) {
  __shared__ float sm[2][32][33];
  const int c = blockIdx.x * 32 + threadIdx.x;
  float s0 = 0.0f, s1 = 0.0f;
  if (c < C) {
    for (int k = threadIdx.y; k < chunks; k += 32) {
      s0 += part0[(size_t)k * C + c];
      if (what == 2) s1 += part1[(size_t)k * C + c];
    }
  }
  sm[0][threadIdx.y][threadIdx.x] = s0;
  sm[1][threadIdx.y][threadIdx.x] = s1;
  __syncthreads();
  if (threadIdx.y == 0 && c < C) {
    s0 = s1 = 0.0f;
#pragma unroll
    for (int y = 0; y < 32; ++y) { s0 += sm[0][y][threadIdx.x]; s1 += sm[1][y][threadIdx.x]; }
    if (what == 0) stats[c].x = s0 * inv_m;
    else if (what == 1) stats[c].y = rsqrtf(s0 * inv_m + eps);
    else means[c] = make_float2(s0 * inv_m, s1 * inv_m);
  }
}

constexpr int kBnEltThreads = 256;

// one thread per 8 consecutive columns of one row
template <typename T>
__global__ void __launch_bounds__(kBnEltThreads)
bn_forward_kernel(const T* __restrict__ x, const T* __restrict__ gamma, const T* __restrict__ beta,
                  const float2* __restrict__ stats, T* __restrict__ Z, T* __restrict__ out, int act, long long M, int C) {
  const int chunks = C / 8;
  const long long i = (long long)blockIdx.x * kBnEltThreads + threadIdx.x;
  if (i >= M * chunks) return;
  const int col0 = (int)(i % chunks) * 8;
  const size_t at = (size_t)(i / chunks) * C + col0;
  float v[8], g[8], b[8];
  load_seg<8>(x + at, 8, v);
  load_seg<8>(gamma + col0, 8, g);
  load_seg<8>(beta + col0, 8, b);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float2 s = stats[col0 + e];
    v[e] = fmaf((v[e] - s.x) * s.y, g[e], b[e]);
  }
  if (Z != nullptr) store_seg<8>(Z + at, 8, v);
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = act_apply(v[e], act);
  store_seg<8>(out + at, 8, v);
}

template <typename T>
__global__ void __launch_bounds__(kBnEltThreads)
bn_backward_kernel(const T* __restrict__ dz, const T* __restrict__ x, const float2* __restrict__ stats,
                   const float2* __restrict__ means, const T* __restrict__ gamma, const T* __restrict__ skip,
                   T* __restrict__ G_in, const T* __restrict__ z_prev, T* __restrict__ dz_prev, int act_prev,
                   long long M, int C) {
  const int chunks = C / 8;
  const long long i = (long long)blockIdx.x * kBnEltThreads + threadIdx.x;
  if (i >= M * chunks) return;
  const int col0 = (int)(i % chunks) * 8;
  const size_t at = (size_t)(i / chunks) * C + col0;
  float g[8], v[8], gam[8];
  load_seg<8>(dz + at, 8, g);
  load_seg<8>(x + at, 8, v);
  load_seg<8>(gamma + col0, 8, gam);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float2 s = stats[col0 + e], m = means[col0 + e];
    const float xh = (v[e] - s.x) * s.y;
    g[e] = gam[e] * s.y * (g[e] - m.x - xh * m.y);
  }
  if (skip != nullptr) {
    load_seg<8>(skip + at, 8, v);
#pragma unroll
    for (int e = 0; e < 8; ++e) g[e] += v[e];
  }
  if (G_in != nullptr) store_seg<8>(G_in + at, 8, g);
  if (dz_prev != nullptr) {
    load_seg<8>(z_prev + at, 8, v);
#pragma unroll
    for (int e = 0; e < 8; ++e) g[e] *= act_grad(v[e], act_prev);
    store_seg<8>(dz_prev + at, 8, g);
  }
}

}  // namespace et
