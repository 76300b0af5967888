// fp32 GEMM on the ordinary FMA pipes, used by fp32 stacks (tensor cores would need TF32,
// whose 10-bit mantissa cannot hold a 1e-4 bound).  One kernel covers forward, dgrad and
// wgrad through element strides:
//   C[i, j] = sum_seg sum_kk  A[i*sa_i + kk*sa_k] * B[kk*sb_k + seg*sb_seg + (j mod b_wrap)*sb_j]
#pragma once

#include "common.cuh"
#include "epilogue.cuh"

namespace et {
namespace simt {

constexpr int TM = 64, TN = 64, TK = 16, THREADS = 256;

struct Params {
  int rows, cols;       // output extent
  int kc;               // contraction length per segment
  int segs;             // fold segments
  long long sa_i, sa_k;
  long long sb_k, sb_seg, sb_j;
  int b_wrap;           // 0 = off
};

template <typename T, class Epi>
__global__ void __launch_bounds__(THREADS)
gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ B, const Params p, const Epi epi) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;   // 16 x 16 threads, 4 x 4 outputs each
  const int i0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;

  for (int seg = 0; seg < p.segs; ++seg) {
    for (int k0 = 0; k0 < p.kc; k0 += TK) {
      // each thread loads 4 elements of each operand tile
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int idx = threadIdx.x + e * THREADS;   // 0 .. 1023
        {
          const int kk = idx & (TK - 1), ii = idx >> 4;
          const int gi = i0 + ii, gk = k0 + kk;
          float v = 0.0f;
          if (gi < p.rows && gk < p.kc) v = to_f32(A[gi * p.sa_i + gk * p.sa_k]);
          As[kk][ii] = v;
        }
        {
          const int jj = idx & (TN - 1), kk = idx >> 6;
          const int gj = j0 + jj, gk = k0 + kk;
          float v = 0.0f;
          if (gj < p.cols && gk < p.kc) {
            const int jw = p.b_wrap > 0 ? gj % p.b_wrap : gj;
            v = to_f32(B[gk * p.sb_k + seg * p.sb_seg + jw * p.sb_j]);
          }
          Bs[kk][jj] = v;
        }
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < TK; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { a[q] = As[kk][ty * 4 + q]; b[q] = Bs[kk][tx * 4 + q]; }
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int r = 0; r < 4; ++r) acc[q][r] = fmaf(a[q], b[r], acc[q][r]);
      }
      __syncthreads();
    }
  }
  const int col0 = j0 + tx * 4;
  const int n = p.cols - col0;
  if (n <= 0) return;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int row = i0 + ty * 4 + q;
    if (row < p.rows) epi.template operator()<4>(row, col0, n, acc[q]);
  }
}

}  // namespace simt
}  // namespace et
