// Layer normalisation as a member of the stack (Section 5.2: a normalisation layer carries two
// trainable tensors, Gamma and Beta).  Memory-bound row kernels: one warp owns a row at a time and
// keeps it in registers, so every activation byte crosses HBM once per pass.
//
//   forward   xhat = (x - mean) * rstd,  y = xhat * gamma + beta;  (mean, rstd) kept per row
//   backward  gy = g * gamma
//             dx = rstd * (gy - mean_row(gy) - xhat * mean_row(gy * xhat))   (+ skip gradient)
//             d gamma = column sums of g * xhat   (per-block partials, finished by bias_finish_kernel)
//             d beta  = column sums of g          (the bias-gradient path of the stack)
//
// A warp's work per row is two reductions and a few hundred dependent instructions, so the row
// loop is software-pipelined: the loads of the warp's next row (kept packed, 16 bytes per 8 bf16)
// are issued before the current row is worked on.  Measured alternatives on 12608 x 768 bf16 rows:
// no prefetch 24 us per backward pass; rows staged through shared memory by cp.async.bulk with an
// mbarrier ring, per warp 21 us, per block (8 rows per copy, producer warp) 30 us.
#pragma once

#include "common.cuh"

namespace et {

constexpr int kNormThreads = 128;
constexpr int kNormWarps = kNormThreads / 32;
constexpr int kNormMaxWidth = 2048;             // 8 register chunks of 8 elements per lane

// Lane `lane` holds, for chunk c = 0 .. VPL-1, the 8 consecutive columns starting at
// (c * 32 + lane) * 8; chunks past the row's end read as zeros.  d is a multiple of 8, rows are
// 16-byte aligned.  Chunks stay packed as loaded until they are needed.
template <typename T> struct RawChunk { uint4 q[sizeof(T) * 8 / 16]; };
template <typename T, int VPL>
__device__ __forceinline__ void norm_load_raw(const T* __restrict__ row, int d, int lane, RawChunk<T> (&v)[VPL]) {
#pragma unroll
  for (int c = 0; c < VPL; ++c) {
    const int col = (c * 32 + lane) * 8;
#pragma unroll
    for (int j = 0; j < (int)(sizeof(T) * 8 / 16); ++j)
      v[c].q[j] = col < d ? reinterpret_cast<const uint4*>(row + col)[j] : make_uint4(0u, 0u, 0u, 0u);
  }
}
__device__ __forceinline__ void raw_unpack(const RawChunk<bf16>& r, float (&t)[8]) {
  const uint32_t w[4] = {r.q[0].x, r.q[0].y, r.q[0].z, r.q[0].w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    t[2 * j] = __uint_as_float(w[j] << 16);
    t[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
  }
}
__device__ __forceinline__ void raw_unpack(const RawChunk<float>& r, float (&t)[8]) {
  t[0] = __uint_as_float(r.q[0].x); t[1] = __uint_as_float(r.q[0].y);
  t[2] = __uint_as_float(r.q[0].z); t[3] = __uint_as_float(r.q[0].w);
  t[4] = __uint_as_float(r.q[1].x); t[5] = __uint_as_float(r.q[1].y);
  t[6] = __uint_as_float(r.q[1].z); t[7] = __uint_as_float(r.q[1].w);
}
// 8 floats -> one stored chunk
__device__ __forceinline__ void store_chunk(bf16* p, const float (&t)[8]) {
  uint4 q;
  q.x = pack_bf16x2(t[0], t[1]); q.y = pack_bf16x2(t[2], t[3]);
  q.z = pack_bf16x2(t[4], t[5]); q.w = pack_bf16x2(t[6], t[7]);
  *reinterpret_cast<uint4*>(p) = q;
}
__device__ __forceinline__ void store_chunk(float* p, const float (&t)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(t[0], t[1], t[2], t[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(t[4], t[5], t[6], t[7]);
}
// gamma (or beta) as floats in shared memory, padded with zeros to VPL * 256 entries
template <typename T, int VPL>
__device__ __forceinline__ void stage_vector(const T* __restrict__ v, int d, float* dst) {
  for (int i = threadIdx.x; i < VPL * 256; i += kNormThreads) dst[i] = i < d ? to_f32(v[i]) : 0.0f;
}
__device__ __forceinline__ void lds8(const float* p, float (&t)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  t[0] = a.x; t[1] = a.y; t[2] = a.z; t[3] = a.w; t[4] = b.x; t[5] = b.y; t[6] = b.z; t[7] = b.w;
}
// Prefetching the next row doubles the packed registers; beyond 1024 bf16 / 512 fp32 features that
// would spill, and such rows are long enough to keep the memory system busy on their own.
template <typename T, int VPL> struct NormPrefetch { static constexpr bool value = VPL * (int)sizeof(T) <= 8; };

// Rows a warp loads at once in the forward kernel.  With one resident wave a warp owns only two or three
// rows: taking their loads one after the other would make the kernel a chain of that many memory
// latencies, so they are all requested up front (12 packed registers per 768-wide bf16 row).
template <typename T, int VPL> struct NormBatch { static constexpr int value = VPL * (int)sizeof(T) <= 6 ? 3 : 1; };

template <typename T, int VPL>
__global__ void __launch_bounds__(kNormThreads, VPL <= 3 ? 6 : 1)
norm_forward_kernel(const T* __restrict__ x, const T* __restrict__ gamma, const T* __restrict__ beta,
                    T* __restrict__ y, float2* __restrict__ stats, int M, int d, float eps) {
  __shared__ __align__(16) float s_gamma[VPL * 256], s_beta[VPL * 256];
  constexpr int R = NormBatch<T, VPL>::value;
  const int lane = threadIdx.x & 31;
  const int warp = blockIdx.x * kNormWarps + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * kNormWarps;
  const float inv_d = 1.0f / (float)d;
  RawChunk<T> raw[R][VPL];
  auto fetch = [&](int r0) {
#pragma unroll
    for (int j = 0; j < R; ++j) {
      const int r = r0 + j * nwarps;
      if (r < M) norm_load_raw<T, VPL>(x + (size_t)r * d, d, lane, raw[j]);
    }
  };
  fetch(warp);                                     // the first batch is on its way before anything else
  stage_vector<T, VPL>(gamma, d, s_gamma);
  stage_vector<T, VPL>(beta, d, s_beta);
  __syncthreads();
  for (int r0 = warp; r0 < M; r0 += R * nwarps) {
    if (r0 != warp) fetch(r0);
#pragma unroll
    for (int j = 0; j < R; ++j) {
      const int r = r0 + j * nwarps;
      if (r >= M) break;
      float v[VPL * 8];
      float s = 0.0f;
#pragma unroll
      for (int c = 0; c < VPL; ++c) {
        float t[8];
        raw_unpack(raw[j][c], t);
#pragma unroll
        for (int e = 0; e < 8; ++e) { v[c * 8 + e] = t[e]; s += t[e]; }
      }
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
      const float shift = -mean * rstd;
      T* yp = y + (size_t)r * d;
#pragma unroll
      for (int c = 0; c < VPL; ++c) {
        const int col = (c * 32 + lane) * 8;
        if (col < d) {
          float g[8], b[8], o[8];
          lds8(s_gamma + col, g);
          lds8(s_beta + col, b);
#pragma unroll
          for (int e = 0; e < 8; ++e) o[e] = fmaf(fmaf(v[c * 8 + e], rstd, shift), g[e], b[e]);
          store_chunk(yp + col, o);
        }
      }
      if (lane == 0) stats[r] = make_float2(mean, rstd);
    }
  }
}

// WANT_DX: the error gradient G_l (optionally + skip), and dZ_{l-1} = G_l * act'(Z_{l-1}) when the
// layer below has an activation.  WANT_DG: per-block partial column sums of g * xhat into
// gpart[blockIdx.x][d] (every block writes its row, zeros included).
template <typename T, int VPL>
struct NormRowIn {
  RawChunk<T> g[VPL], x[VPL], sk[VPL];
  float2 st;
};
template <typename T, int VPL, bool WANT_DX, bool WANT_DG>
__global__ void __launch_bounds__(kNormThreads)
norm_backward_kernel(const T* __restrict__ g_out, const T* __restrict__ x, const float2* __restrict__ stats,
                     const T* __restrict__ gamma, const T* __restrict__ skip, T* __restrict__ G_in,
                     const T* __restrict__ z_prev, T* __restrict__ dz_prev, int act_prev,
                     float* __restrict__ gpart, int M, int d) {
  // gamma during the rows; afterwards reused for the block's d gamma sums
  __shared__ __align__(16) float s_vec[VPL * 256];
  constexpr bool PRE = NormPrefetch<T, VPL>::value;
  const int lane = threadIdx.x & 31;
  const int wib = threadIdx.x >> 5;
  const int warp = blockIdx.x * kNormWarps + wib;
  const int nwarps = gridDim.x * kNormWarps;
  if constexpr (WANT_DX) {
    stage_vector<T, VPL>(gamma, d, s_vec);
    __syncthreads();
  }
  const bool has_skip = WANT_DX && skip != nullptr;
  const bool has_z = WANT_DX && dz_prev != nullptr;
  float acc[VPL * 8];
#pragma unroll
  for (int i = 0; i < VPL * 8; ++i) acc[i] = 0.0f;
  const float inv_d = 1.0f / (float)d;
  const size_t step = (size_t)nwarps * d;
  size_t off = (size_t)warp * d;
  auto fetch = [&](size_t at, int r, NormRowIn<T, VPL>& in) {
    norm_load_raw<T, VPL>(g_out + at, d, lane, in.g);
    norm_load_raw<T, VPL>(x + at, d, lane, in.x);
    if (has_skip) norm_load_raw<T, VPL>(skip + at, d, lane, in.sk);
    in.st = stats[r];
  };
  NormRowIn<T, VPL> nxt;
  if (PRE && warp < M) fetch(off, warp, nxt);
  for (int r = warp; r < M; r += nwarps, off += step) {
    NormRowIn<T, VPL> cur;
    if constexpr (PRE) {
      cur = nxt;
      if (r + nwarps < M) fetch(off + step, r + nwarps, nxt);
    } else {
      fetch(off, r, cur);
    }
    const float scale = cur.st.y, shift = -cur.st.x * cur.st.y;
    float g[VPL * 8], xh[VPL * 8];
    float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
    for (int c = 0; c < VPL; ++c) {
      float tg[8], tx[8], gam[8];
      raw_unpack(cur.g[c], tg);
      raw_unpack(cur.x[c], tx);
      if constexpr (WANT_DX) lds8(s_vec + (c * 32 + lane) * 8, gam);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float h = fmaf(tx[e], scale, shift);                   // xhat (meaningless past the row's end,
        if constexpr (WANT_DG) acc[c * 8 + e] = fmaf(tg[e], h, acc[c * 8 + e]);   //  where g = 0 cancels it)
        if constexpr (WANT_DX) {
          const float gy = tg[e] * gam[e];
          s1 += gy;
          s2 = fmaf(gy, h, s2);
          g[c * 8 + e] = gy;
          xh[c * 8 + e] = h;
        }
      }
    }
    if constexpr (WANT_DX) {
      // dx = rstd * (gy - c1 - xhat * c2)
      const float c1 = warp_sum(s1) * inv_d, c2 = warp_sum(s2) * inv_d;
      const float k0 = -c1 * cur.st.y, k2 = -c2 * cur.st.y;
#pragma unroll
      for (int c = 0; c < VPL; ++c) {
        const int col = (c * 32 + lane) * 8;
        if (col >= d) continue;
        float o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = fmaf(xh[c * 8 + e], k2, fmaf(g[c * 8 + e], cur.st.y, k0));
        if (has_skip) {
          float t[8];
          raw_unpack(cur.sk[c], t);
#pragma unroll
          for (int e = 0; e < 8; ++e) o[e] += t[e];
        }
        if (G_in != nullptr) store_chunk(G_in + off + col, o);
        if (has_z) {
          RawChunk<T> zc[1];
          float t[8];
          zc[0].q[0] = reinterpret_cast<const uint4*>(z_prev + off + col)[0];
          if constexpr (sizeof(T) == 4) zc[0].q[sizeof(T) * 8 / 16 - 1] = reinterpret_cast<const uint4*>(z_prev + off + col)[1];
          raw_unpack(zc[0], t);
#pragma unroll
          for (int e = 0; e < 8; ++e) o[e] *= act_grad(t[e], act_prev);
          store_chunk(dz_prev + off + col, o);
        }
      }
    }
  }
  if constexpr (WANT_DG) {
    // the block's warps add their sums one after the other: fixed order, no atomics
    __syncthreads();                               // gamma is no longer needed
    for (int w = 0; w < kNormWarps; ++w) {
      if (wib == w) {
#pragma unroll
        for (int i = 0; i < VPL * 8; ++i) {
          const int at = ((i >> 3) * 32 + lane) * 8 + (i & 7);      // = the column
          s_vec[at] = (w == 0 ? 0.0f : s_vec[at]) + acc[i];
        }
      }
      __syncthreads();
    }
    for (int col = threadIdx.x; col < d; col += kNormThreads) gpart[(size_t)blockIdx.x * d + col] = s_vec[col];
  }
}

}  // namespace et
