// Softmax attention core as a member of the stack: a layer without trainable tensors (the paper
// counts attention operations among the non-trainable layers, Sections 5.3 and 5.4).  Input rows
// are [q | k | v] (3 * heads * 64 columns), grouped in sequences of S consecutive rows; output
// rows are the heads' P v side by side.
//
//   forward   P = softmax_j( q_i . k_j / 8 ),  o_i = sum_j P_ij v_j ;  keeps logsumexp per (head, row)
//   backward  dV = P^T dO ;  dP = dO V^T ;  D_i = dO_i . o_i ;  dS = P * (dP - D_i) / 8 ;
//             dQ = dS K ;  dK = dS^T Q          (P is recomputed from q, k and the saved logsumexp)
//
// One CTA per (sequence, head); K and V of the head stay in shared memory, queries go through in
// blocks of 64 rows.  The five small GEMMs per block (64 x S x 64 and S x 64 x 64) run on the tensor
// cores through the warp-level matrix fragments (16 x 16 x 16, bf16 in, fp32 accumulate); with S
// around 200 and a head width of 64 the tiles are too small for a TMEM accumulator pipeline to pay.
// Limits: head width 64, S <= 208, bf16 storage.
#pragma once

#include <mma.h>

#include "common.cuh"

namespace et {
namespace attn {

constexpr int DH = 64;           // head width
constexpr int S_MAX = 208;       // longest sequence (padded to a multiple of 16)
constexpr int RB = 64;           // query rows per pass, backward
constexpr int RB_FWD = 32;       // query rows per pass, forward: two CTAs fit on an SM
constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int LDK = DH + 8;      // row stride (elements) of the 64-wide bf16 tiles: breaks bank conflicts
constexpr int THREADS_BWD = 512; // backward: 16 warps, each with a quarter of the registers' worth of dK / dV tiles
constexpr int WARPS_BWD = THREADS_BWD / 32;
constexpr int MAX_OWN = 4;       // (S_MAX / 16) * (DH / 16) = 52 output tiles of dK (or dV) over 16 warps
constexpr float SCALE = 0.125f;  // 1 / sqrt(DH)

__host__ __device__ inline int pad16(int s) { return (s + 15) & ~15; }
// row stride (floats) of the fp32 score buffer; it also stages 64-column results, so never below 68
__host__ __device__ inline int score_ld(int SP) { return SP + 4 > DH + 4 ? SP + 4 : DH + 4; }
inline size_t forward_smem_bytes(int S) {
  const int SP = pad16(S);
  return (size_t)(2 * SP + RB_FWD) * LDK * 2 + (size_t)RB_FWD * score_ld(SP) * 4 + (size_t)RB_FWD * (SP + 8) * 2;
}
inline size_t backward_smem_bytes(int S) {
  const int SP = pad16(S);
  return (size_t)(2 * SP + 2 * RB) * LDK * 2 + (size_t)RB * score_ld(SP) * 4 + (size_t)2 * RB * (SP + 8) * 2;
}

using FragA = nvcuda::wmma::fragment<nvcuda::wmma::matrix_a, 16, 16, 16, bf16, nvcuda::wmma::row_major>;
using FragAT = nvcuda::wmma::fragment<nvcuda::wmma::matrix_a, 16, 16, 16, bf16, nvcuda::wmma::col_major>;
using FragB = nvcuda::wmma::fragment<nvcuda::wmma::matrix_b, 16, 16, 16, bf16, nvcuda::wmma::row_major>;
using FragBT = nvcuda::wmma::fragment<nvcuda::wmma::matrix_b, 16, 16, 16, bf16, nvcuda::wmma::col_major>;
using FragC = nvcuda::wmma::fragment<nvcuda::wmma::accumulator, 16, 16, 16, float>;

// rows [row0, row0 + nrows) of one head's 64 columns -> tile[r][LDK]; rows at or past S read as zeros
template <int NT = THREADS>
__device__ __forceinline__ void load_tile(bf16* tile, const bf16* src, size_t ld, int row0, int nrows, int S) {
  for (int i = threadIdx.x; i < nrows * 8; i += NT) {
    const int r = i >> 3, ch = i & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + r < S) v = *reinterpret_cast<const uint4*>(src + (size_t)(row0 + r) * ld + ch * 8);
    *reinterpret_cast<uint4*>(tile + r * LDK + ch * 8) = v;
  }
}
// 16 consecutive floats of a staged fp32 tile -> 16 bf16 in global memory
__device__ __forceinline__ void store16(bf16* dst, const float* src) {
  uint4 a, b;
  a.x = pack_bf16x2(src[0], src[1]);   a.y = pack_bf16x2(src[2], src[3]);
  a.z = pack_bf16x2(src[4], src[5]);   a.w = pack_bf16x2(src[6], src[7]);
  b.x = pack_bf16x2(src[8], src[9]);   b.y = pack_bf16x2(src[10], src[11]);
  b.z = pack_bf16x2(src[12], src[13]); b.w = pack_bf16x2(src[14], src[15]);
  reinterpret_cast<uint4*>(dst)[0] = a;
  reinterpret_cast<uint4*>(dst)[1] = b;
}

// Sf[RBT][ldsf] = A[RBT][64] * Bt[SP][64]^T (fp32).  A warp keeps its row tile's four A fragments and
// walks over column tiles two at a time (two independent accumulator chains).
template <int RBT, int NW = WARPS>
__device__ __forceinline__ void abt_tiles(const bf16* A, const bf16* Bt, float* Sf, int ntn, int ldsf, int warp) {
  constexpr int MT = RBT / 16, G = NW / MT;
  const int mi = warp % MT, g = warp / MT;
  FragA a[DH / 16];
#pragma unroll
  for (int kk = 0; kk < DH / 16; ++kk) nvcuda::wmma::load_matrix_sync(a[kk], A + mi * 16 * LDK + kk * 16, LDK);
  for (int nj = g; nj < ntn; nj += 2 * G) {
    const int nj2 = nj + G;
    const bool two = nj2 < ntn;                    // the same for the whole warp
    FragC acc0, acc1;
    nvcuda::wmma::fill_fragment(acc0, 0.0f);
    nvcuda::wmma::fill_fragment(acc1, 0.0f);
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
      FragBT b0, b1;
      nvcuda::wmma::load_matrix_sync(b0, Bt + nj * 16 * LDK + kk * 16, LDK);       // B[k][n] = Bt[n][k]
      if (two) nvcuda::wmma::load_matrix_sync(b1, Bt + nj2 * 16 * LDK + kk * 16, LDK);
      nvcuda::wmma::mma_sync(acc0, a[kk], b0, acc0);
      if (two) nvcuda::wmma::mma_sync(acc1, a[kk], b1, acc1);
    }
    nvcuda::wmma::store_matrix_sync(Sf + mi * 16 * ldsf + nj * 16, acc0, ldsf, nvcuda::wmma::mem_row_major);
    if (two) nvcuda::wmma::store_matrix_sync(Sf + mi * 16 * ldsf + nj2 * 16, acc1, ldsf, nvcuda::wmma::mem_row_major);
  }
}
// Of[RBT][ldsf] (columns 0..63) = A[RBT][SP] * Bm[SP][64], A bf16 with stride lda.  64 rows: two column
// tiles per warp sharing the A fragment; 32 rows: one tile per warp, even and odd k steps in two chains.
template <int RBT, int NW = WARPS>
__device__ __forceinline__ void rows_times_head(const bf16* A, int lda, const bf16* Bm, float* Of, int ntn, int ldsf,
                                                int warp) {
  FragC acc0, acc1;
  nvcuda::wmma::fill_fragment(acc0, 0.0f);
  nvcuda::wmma::fill_fragment(acc1, 0.0f);
  constexpr int MT = RBT / 16;
  if constexpr (MT * 4 == 2 * NW) {
    const int mi = warp & 3, nj = (warp >> 2) * 2;
    for (int kk = 0; kk < ntn; ++kk) {
      FragA a;
      FragB b0, b1;
      nvcuda::wmma::load_matrix_sync(a, A + mi * 16 * lda + kk * 16, lda);
      nvcuda::wmma::load_matrix_sync(b0, Bm + kk * 16 * LDK + nj * 16, LDK);
      nvcuda::wmma::load_matrix_sync(b1, Bm + kk * 16 * LDK + nj * 16 + 16, LDK);
      nvcuda::wmma::mma_sync(acc0, a, b0, acc0);
      nvcuda::wmma::mma_sync(acc1, a, b1, acc1);
    }
    nvcuda::wmma::store_matrix_sync(Of + mi * 16 * ldsf + nj * 16, acc0, ldsf, nvcuda::wmma::mem_row_major);
    nvcuda::wmma::store_matrix_sync(Of + mi * 16 * ldsf + nj * 16 + 16, acc1, ldsf, nvcuda::wmma::mem_row_major);
  } else {
    static_assert(MT * 4 == NW, "one output tile per warp");
    const int mi = warp % MT, nj = warp / MT;
    for (int kk = 0; kk < ntn; kk += 2) {
      FragA a0, a1;
      FragB b0, b1;
      nvcuda::wmma::load_matrix_sync(a0, A + mi * 16 * lda + kk * 16, lda);
      nvcuda::wmma::load_matrix_sync(b0, Bm + kk * 16 * LDK + nj * 16, LDK);
      nvcuda::wmma::mma_sync(acc0, a0, b0, acc0);
      if (kk + 1 < ntn) {
        nvcuda::wmma::load_matrix_sync(a1, A + mi * 16 * lda + (kk + 1) * 16, lda);
        nvcuda::wmma::load_matrix_sync(b1, Bm + (kk + 1) * 16 * LDK + nj * 16, LDK);
        nvcuda::wmma::mma_sync(acc1, a1, b1, acc1);
      }
    }
#pragma unroll
    for (int i = 0; i < acc0.num_elements; ++i) acc0.x[i] += acc1.x[i];
    nvcuda::wmma::store_matrix_sync(Of + mi * 16 * ldsf + nj * 16, acc0, ldsf, nvcuda::wmma::mem_row_major);
  }
}
// 8 consecutive floats of a staged fp32 tile -> 8 bf16 in global memory
__device__ __forceinline__ void store8(bf16* dst, const float* src) {
  uint4 a;
  a.x = pack_bf16x2(src[0], src[1]); a.y = pack_bf16x2(src[2], src[3]);
  a.z = pack_bf16x2(src[4], src[5]); a.w = pack_bf16x2(src[6], src[7]);
  *reinterpret_cast<uint4*>(dst) = a;
}

// grid = sequences * heads.  qkv: [M][3d]; out: [M][d]; lse: [sequences * heads][S].
static __global__ void __launch_bounds__(THREADS, 2)
attn_forward_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ out, float* __restrict__ lse, int S, int H, int d) {
  extern __shared__ __align__(128) uint8_t smem[];
  constexpr int RBT = RB_FWD;
  constexpr int TPR = THREADS / RBT;               // threads per row in the row-wise parts: 8
  const int SP = pad16(S), ntn = SP / 16, ldsf = score_ld(SP), ldp = SP + 8;
  bf16* Ks = reinterpret_cast<bf16*>(smem);
  bf16* Vs = Ks + SP * LDK;
  bf16* Qs = Vs + SP * LDK;
  float* Sf = reinterpret_cast<float*>(Qs + RBT * LDK);
  bf16* Pb = reinterpret_cast<bf16*>(Sf + RBT * ldsf);
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int warp = threadIdx.x >> 5;
  const size_t ld = (size_t)3 * d;
  const bf16* base = qkv + (size_t)b * S * ld + h * DH;
  load_tile(Ks, base + d, ld, 0, SP, S);
  load_tile(Vs, base + 2 * d, ld, 0, SP, S);
  for (int rb0 = 0; rb0 < S; rb0 += RBT) {
    load_tile(Qs, base, ld, rb0, RBT, S);
    __syncthreads();
    abt_tiles<RBT>(Qs, Ks, Sf, ntn, ldsf, warp);
    __syncthreads();
    {   // softmax of row r by TPR neighbouring lanes
      const int r = threadIdx.x / TPR, sub = threadIdx.x % TPR;
      const bool valid = rb0 + r < S;
      float* row = Sf + r * ldsf;
      float m = -INFINITY;
      for (int c = sub; c < S; c += TPR) m = fmaxf(m, row[c]);
#pragma unroll
      for (int o = 1; o < TPR; o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      float sum = 0.0f;
      for (int c = sub; c < S; c += TPR) {
        const float e = __expf((row[c] - m) * SCALE);
        row[c] = e;
        sum += e;
      }
#pragma unroll
      for (int o = 1; o < TPR; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float inv = 1.0f / sum;
      for (int c = sub; c < SP; c += TPR) Pb[r * ldp + c] = __float2bfloat16_rn((valid && c < S) ? row[c] * inv : 0.0f);
      if (valid && sub == 0) lse[(size_t)blockIdx.x * S + rb0 + r] = m * SCALE + __logf(sum);
    }
    __syncthreads();
    rows_times_head<RBT>(Pb, ldp, Vs, Sf, ntn, ldsf, warp);
    __syncthreads();
    {
      const int r = threadIdx.x / TPR, c0 = (threadIdx.x % TPR) * (DH / TPR);
      if (rb0 + r < S) store8(out + ((size_t)b * S + rb0 + r) * d + h * DH + c0, Sf + r * ldsf + c0);
    }
    __syncthreads();
  }
}

// dqkv: [M][3d] gradient of the layer's input; every element of this head's columns is written.
// 16 warps: the row-wise passes use 8 lanes per row, every GEMM helper runs with 16 warps.
static __global__ void __launch_bounds__(THREADS_BWD, 1)
attn_backward_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ out, const bf16* __restrict__ dout,
                     const float* __restrict__ lse, bf16* __restrict__ dqkv, int S, int H, int d) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ float Dsm[RB];
  constexpr int NT = THREADS_BWD, NW = WARPS_BWD;
  constexpr int TPR = NT / RB;                      // lanes per row in the row-wise passes: 8
  const int SP = pad16(S), ntn = SP / 16, ldsf = score_ld(SP), ldp = SP + 8;
  bf16* Ks = reinterpret_cast<bf16*>(smem);
  bf16* Vs = Ks + SP * LDK;
  bf16* Qs = Vs + SP * LDK;
  bf16* dOs = Qs + RB * LDK;
  float* Sf = reinterpret_cast<float*>(dOs + RB * LDK);
  bf16* Pb = reinterpret_cast<bf16*>(Sf + RB * ldsf);
  bf16* dSb = Pb + RB * ldp;
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int warp = threadIdx.x >> 5;
  const int r = threadIdx.x / TPR, sub = threadIdx.x % TPR;       // row and lane-in-row of the row-wise passes
  const size_t ld = (size_t)3 * d;
  const bf16* base = qkv + (size_t)b * S * ld + h * DH;
  bf16* gbase = dqkv + (size_t)b * S * ld + h * DH;
  const bf16* obase = out + (size_t)b * S * d + h * DH;
  const bf16* dobase = dout + (size_t)b * S * d + h * DH;
  load_tile<NT>(Ks, base + d, ld, 0, SP, S);
  load_tile<NT>(Vs, base + 2 * d, ld, 0, SP, S);
  FragC accK[MAX_OWN], accV[MAX_OWN];
#pragma unroll
  for (int i = 0; i < MAX_OWN; ++i) {
    nvcuda::wmma::fill_fragment(accK[i], 0.0f);
    nvcuda::wmma::fill_fragment(accV[i], 0.0f);
  }
  for (int rb0 = 0; rb0 < S; rb0 += RB) {
    const bool valid = rb0 + r < S;
    load_tile<NT>(Qs, base, ld, rb0, RB, S);
    load_tile<NT>(dOs, dobase, (size_t)d, rb0, RB, S);
    __syncthreads();
    abt_tiles<RB, NW>(Qs, Ks, Sf, ntn, ldsf, warp);
    {   // D_r = dO_r . o_r, 8 columns per lane
      float s = 0.0f;
      if (valid) {
        float ov[8], gv[8];
        load_seg<8>(obase + (size_t)(rb0 + r) * d + sub * 8, 8, ov);
        load_seg<8>(dOs + r * LDK + sub * 8, 8, gv);
#pragma unroll
        for (int c = 0; c < 8; ++c) s = fmaf(gv[c], ov[c], s);
      }
#pragma unroll
      for (int o = 1; o < TPR; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (sub == 0) Dsm[r] = s;
    }
    __syncthreads();
    {   // P = exp(s / 8 - logsumexp), zero outside the sequence
      const float l = valid ? lse[(size_t)blockIdx.x * S + rb0 + r] : 0.0f;
      const float* row = Sf + r * ldsf;
      for (int c = 2 * sub; c < SP; c += 2 * TPR) {  // two columns at a time
        const float2 x = *reinterpret_cast<const float2*>(row + c);
        const float p0 = (valid && c < S) ? __expf(x.x * SCALE - l) : 0.0f;
        const float p1 = (valid && c + 1 < S) ? __expf(x.y * SCALE - l) : 0.0f;
        *reinterpret_cast<uint32_t*>(Pb + r * ldp + c) = pack_bf16x2(p0, p1);
      }
    }
    __syncthreads();
    // dP = dO V^T -> Sf
    abt_tiles<RB, NW>(dOs, Vs, Sf, ntn, ldsf, warp);
    __syncthreads();
    {   // dS = P * (dP - D) / 8
      const float Dr = Dsm[r];
      const float* row = Sf + r * ldsf;
      for (int c = 2 * sub; c < SP; c += 2 * TPR) {
        const float2 x = *reinterpret_cast<const float2*>(row + c);
        const uint32_t pp = *reinterpret_cast<const uint32_t*>(Pb + r * ldp + c);
        const float p0 = __uint_as_float(pp << 16), p1 = __uint_as_float(pp & 0xffff0000u);
        *reinterpret_cast<uint32_t*>(dSb + r * ldp + c) = pack_bf16x2(p0 * (x.x - Dr) * SCALE, p1 * (x.y - Dr) * SCALE);
      }
    }
    __syncthreads();
    // dQ_blk = dS K -> Sf (columns 0..63)
    rows_times_head<RB, NW>(dSb, ldp, Ks, Sf, ntn, ldsf, warp);
    // dV^T += dO^T P ; dK^T += Q^T dS   (contraction over the 64 rows of this block).  Transposed so that
    // the operand that has to be read column-wise is the small one: a warp's output tiles (64-row head
    // tile mi = warp & 3, key tiles nj = warp / 4 + 4 i) share mi, so its four dO^T / Q^T fragments per
    // block are loaded once, and P / dS are read row-wise.
    {
      const int mi = warp & 3;
      FragAT ot[RB / 16], qt[RB / 16];
#pragma unroll
      for (int kk = 0; kk < RB / 16; ++kk) {
        nvcuda::wmma::load_matrix_sync(ot[kk], dOs + kk * 16 * LDK + mi * 16, LDK);   // A[m][k] = dO[k][m]
        nvcuda::wmma::load_matrix_sync(qt[kk], Qs + kk * 16 * LDK + mi * 16, LDK);
      }
#pragma unroll
      for (int i = 0; i < MAX_OWN; ++i) {
        const int nj = (warp >> 2) + (NW / 4) * i;
        if (nj < ntn) {
#pragma unroll
          for (int kk = 0; kk < RB / 16; ++kk) {
            FragB pb, sb;
            nvcuda::wmma::load_matrix_sync(pb, Pb + kk * 16 * ldp + nj * 16, ldp);
            nvcuda::wmma::load_matrix_sync(sb, dSb + kk * 16 * ldp + nj * 16, ldp);
            nvcuda::wmma::mma_sync(accV[i], ot[kk], pb, accV[i]);
            nvcuda::wmma::mma_sync(accK[i], qt[kk], sb, accK[i]);
          }
        }
      }
    }
    __syncthreads();
    if (valid) store8(gbase + (size_t)(rb0 + r) * ld + sub * 8, Sf + r * ldsf + sub * 8);
    __syncthreads();
  }
  // dK, then dV: accumulators (transposed tiles) -> fp32 staging [SP][64] (it fits the score buffer) -> bf16 rows
  float* stage = Sf;
  for (int which = 0; which < 2; ++which) {
#pragma unroll
    for (int i = 0; i < MAX_OWN; ++i) {
      const int nj = (warp >> 2) + (NW / 4) * i;
      if (nj < ntn)
        nvcuda::wmma::store_matrix_sync(stage + nj * 16 * DH + (warp & 3) * 16, which == 0 ? accK[i] : accV[i], DH,
                                        nvcuda::wmma::mem_col_major);       // element (dh, key) -> stage[key][dh]
    }
    __syncthreads();
    for (int i = threadIdx.x; i < S * 8; i += NT) {
      const int row = i >> 3, c0 = (i & 7) * 8;
      store8(gbase + (size_t)row * ld + (which + 1) * d + c0, stage + row * DH + c0);
    }
    __syncthreads();
  }
}

}  // namespace attn
}  // namespace et
