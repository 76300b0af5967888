// Softmax attention core as a member of the stack: a layer without trainable tensors (the paper
// counts attention operations among the non-trainable layers, Sections 5.3 and 5.4).  Input rows
// are [q | k | v] (3 * heads * 64 columns), grouped in sequences of S consecutive rows; output
// rows are the heads' P v side by side.
//
//   forward   P = softmax_j( q_i . k_j / 8 ),  o_i = sum_j P_ij v_j ;  keeps logsumexp per (head, row)
//   backward  dV = P^T dO ;  dP = dO V^T ;  D_i = dO_i . o_i ;  dS = P * (dP - D_i) / 8 ;
//             dQ = dS K ;  dK = dS^T Q          (P is recomputed from q, k and the saved logsumexp)
//
// One CTA per (sequence, head).  All five products run on the tcgen05 tensor cores with their
// accumulators in tensor memory; q, k, v and dO tiles (64 columns x 128 rows, 128-byte swizzle) come in by
// TMA.  The row-wise work (softmax; P and dS) is done by threads that own one accumulator row each: they
// read scores from tensor memory, and write P / dS as bf16 into swizzled shared memory in exactly the layout
// the next product reads as its operand -- K-major for P v and dS k, MN-major (the same bytes, other
// descriptor) for P^T dO and dS^T q.  Nothing but q, k, v, dO, o and the log-sum-exp touches global memory.
//
// Tensor memory (512 columns of fp32):
//   forward   scores of query rows 0..127 in columns 0..255, of rows 128..255 in 256..511; each half's
//             output accumulator (64 columns) reuses the start of its score block once P has been taken.
//   backward  one 128 x 128 block of (query rows rh, keys kh) at a time: S 0..127, dP 128..255,
//             dQ of the two row halves 256..383 (accumulated over kh), dK and dV of the current key half
//             384..511 (accumulated over rh, written out before the next key half).
// Limits: head width 64, S <= 256, bf16 storage.  Rows of a tile beyond the sequence belong to the next
// sequence (or are zero-filled past the end of the tensor): their probabilities are forced to zero and
// nothing is stored for them.
#pragma once

#include "gemm_tc.cuh"

namespace et {
namespace attn {

using namespace et::tc;

constexpr int DH = 64;           // head width
constexpr int S_MAX = 256;       // longest sequence
constexpr float SCALE = 0.125f;  // 1 / sqrt(DH)
constexpr float SCALE_LOG2E = 0.125f * 1.4426950408889634f;   // exp(x / 8) = 2^(x * SCALE_LOG2E)
constexpr float LOG2E = 1.4426950408889634f;
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
constexpr uint32_t TILE_BYTES = 128 * DH * 2;          // one 128-row x 64-column bf16 tile: 16 KB
constexpr int THREADS = 320;     // warp 0: TMA, warp 1: MMA issue + TMEM, warps 2-9: row threads
constexpr uint32_t FWD_SMEM = 6 * TILE_BYTES + 8 * TILE_BYTES + 1024 + 256;   // q, k, v (2 tiles each), P (2 x 4 tiles)
constexpr uint32_t BWD_SMEM = 8 * TILE_BYTES + 4 * TILE_BYTES + 1024 + 256;   // q, k, v, dO; P block, dS block (2 tiles each)

enum AttnStatus : uint32_t { kTimeoutAttn = 7 };

__host__ __device__ inline int pad16(int s) { return (s + 15) & ~15; }

// instruction descriptor, cta_group::1, M = 128: bf16 operands, fp32 accumulate
__device__ __forceinline__ uint32_t idesc128(int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// K-major operand (rows of 64 contraction elements): 16 contraction elements further = 32 bytes along the
// swizzled row; the next 64 contraction elements are the next 16-KB tile.
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t tile0, int kstep) {
  return make_desc(tile0 + (uint32_t)(kstep >> 2) * TILE_BYTES + (uint32_t)(kstep & 3) * 32u, 16, 1024);
}
// MN-major operand (rows of 64 mn elements, one row per contraction index): 16 contraction rows = 2048
// bytes; the next 64 mn elements are `chunk_bytes` further.
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t tile0, int kstep, uint32_t chunk_bytes) {
  return make_desc(tile0 + (uint32_t)kstep * 2048u, chunk_bytes, 1024);
}
__device__ __forceinline__ void store32_bf16(bf16* dst, const float (&v)[32], float scale) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint4 q;
    q.x = pack_bf16x2(v[j * 8 + 0] * scale, v[j * 8 + 1] * scale);
    q.y = pack_bf16x2(v[j * 8 + 2] * scale, v[j * 8 + 3] * scale);
    q.z = pack_bf16x2(v[j * 8 + 4] * scale, v[j * 8 + 5] * scale);
    q.w = pack_bf16x2(v[j * 8 + 6] * scale, v[j * 8 + 7] * scale);
    reinterpret_cast<uint4*>(dst)[j] = q;
  }
}

// grid = sequences * heads.  map_qkv: [M][3d] with 64-column x 128-row boxes; out: [M][d];
// lse: [sequences * heads][S].
static __global__ void __launch_bounds__(THREADS, 1)
attn_forward_kernel(const __grid_constant__ CUtensorMap map_qkv, bf16* __restrict__ out, float* __restrict__ lse,
                    const int S, const int H, const int d, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t sQ = base, sK = base + 2 * TILE_BYTES, sV = base + 4 * TILE_BYTES, sP = base + 6 * TILE_BYTES;
  const uint32_t bars = base + 14 * TILE_BYTES;
  const uint32_t bar_qk = bars, bar_v = bars + 8;
  auto bar_s = [&](int h) { return bars + 16u + 8u * h; };       // scores of half h complete
  auto bar_p = [&](int h) { return bars + 32u + 8u * h; };       // P of half h is in shared memory
  auto bar_o = [&](int h) { return bars + 48u + 8u * h; };       // output accumulator of half h complete
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 14 * TILE_BYTES + 64);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int SP = pad16(S);
  const int halves = S > 128 ? 2 : 1;
  const int row0 = b * S;

  if (threadIdx.x == 0) {
    prefetch_tmap(&map_qkv);
    mbar_init(bar_qk, 1); mbar_init(bar_v, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(bar_s(i), 1); mbar_init(bar_p(i), 128); mbar_init(bar_o(i), 1); }
    *abort_flag = 0;
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bar_qk, (uint32_t)(2 * halves) * TILE_BYTES);
      for (int t = 0; t < halves; ++t) {
        tma_load_2d(sQ + t * TILE_BYTES, &map_qkv, bar_qk, h * DH, row0 + t * 128);
        tma_load_2d(sK + t * TILE_BYTES, &map_qkv, bar_qk, d + h * DH, row0 + t * 128);
      }
      mbar_expect_tx(bar_v, (uint32_t)halves * TILE_BYTES);
      for (int t = 0; t < halves; ++t) tma_load_2d(sV + t * TILE_BYTES, &map_qkv, bar_v, 2 * d + h * DH, row0 + t * 128);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = mbar_wait(bar_qk, 0, abort_flag, status, kTimeoutAttn);
      if (ok) {
        tc_fence_after();
        const uint32_t id_s = idesc128(SP, false, false);
        for (int hh = 0; hh < halves; ++hh) {                    // S_hh = q_hh k^T
          for (int ks = 0; ks < DH / UK; ++ks)
            tc_mma(tmem_base + hh * 256, kmajor_desc(sQ + hh * TILE_BYTES, ks), kmajor_desc(sK, ks), id_s, ks > 0 ? 1u : 0u);
          tc_commit(bar_s(hh));
        }
        ok = mbar_wait(bar_v, 0, abort_flag, status, kTimeoutAttn);
        const uint32_t id_o = idesc128(DH, false, true);
        for (int hh = 0; hh < halves && ok; ++hh) {              // O_hh = P_hh v, into the start of S_hh's columns
          ok = mbar_wait(bar_p(hh), 0, abort_flag, status, kTimeoutAttn);
          if (!ok) break;
          tc_fence_after();
          for (int ks = 0; ks < SP / UK; ++ks)
            tc_mma(tmem_base + hh * 256, kmajor_desc(sP + hh * 4 * TILE_BYTES, ks), mnmajor_desc(sV, ks, TILE_BYTES), id_o,
                   ks > 0 ? 1u : 0u);
          tc_commit(bar_o(hh));
        }
      }
    }
  } else {
    const int hh = (warp - 2) >> 2;                              // which half of the query rows
    const int quad = warp & 3;
    const int trow = quad * 32 + lane;
    const int row = hh * 128 + trow;                             // row inside the sequence
    if (hh < halves) {
      bool ok = mbar_wait(bar_s(hh), 0, abort_flag, status, kTimeoutAttn);
      if (ok) {
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(hh * 256);
        const int nchunk = (SP + 31) / 32;
        // chunks of 32 keys; only the last one can reach past the sequence and needs the per-key test
        const int nfull = S / 32;
        float m = -INFINITY;
        for (int c = 0; c < nchunk; ++c) {
          float v[32];
          tmem_ld32(taddr + c * 32, v);
          if (c < nfull) {
#pragma unroll
            for (int i = 0; i < 32; ++i) m = fmaxf(m, v[i]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) m = fmaxf(m, (c * 32 + i < S) ? v[i] : -INFINITY);
          }
        }
        float sum = 0.0f;
        uint8_t* Pt = gen + 6 * TILE_BYTES + hh * 4 * TILE_BYTES;
        const bool valid = row < S;
        const float mk = valid ? m * SCALE_LOG2E : INFINITY;     // rows past the sequence: 2^(-inf) = 0 everywhere
        for (int c = 0; c < nchunk; ++c) {
          float v[32];
          tmem_ld32(taddr + c * 32, v);
          if (c < nfull) {
#pragma unroll
            for (int i = 0; i < 32; ++i) { v[i] = ex2(fmaf(v[i], SCALE_LOG2E, -mk)); sum += v[i]; }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              v[i] = (c * 32 + i < S) ? ex2(fmaf(v[i], SCALE_LOG2E, -mk)) : 0.0f;
              sum += v[i];
            }
          }
          sts_row32(Pt + (c >> 1) * TILE_BYTES, trow, c & 1, v);
        }
        tc_fence_before();
        fence_async_smem();
        mbar_arrive(bar_p(hh));
        ok = mbar_wait(bar_o(hh), 0, abort_flag, status, kTimeoutAttn);
        if (ok) {
          tc_fence_after();
          float o0[32], o1[32];
          tmem_ld32_issue(taddr, o0);
          tmem_ld32_issue(taddr + 32, o1);
          tmem_ld_wait(o0, o1);
          if (valid) {
            const float inv = 1.0f / sum;
            bf16* dst = out + (size_t)(row0 + row) * d + h * DH;
            store32_bf16(dst, o0, inv);
            store32_bf16(dst + 32, o1, inv);
            lse[(size_t)blockIdx.x * S + row] = m * SCALE + __logf(sum);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// dqkv: [M][3d] gradient of the layer's input; every element of this head's columns in rows of the sequence
// is written.  map_qkv as above; map_do: [M][d] with 64 x 128 boxes.
static __global__ void __launch_bounds__(THREADS, 1)
attn_backward_kernel(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_do,
                     const bf16* __restrict__ out, const bf16* __restrict__ dout, const float* __restrict__ lse,
                     bf16* __restrict__ dqkv, const int S, const int H, const int d, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t sQ = base, sK = base + 2 * TILE_BYTES, sV = base + 4 * TILE_BYTES, sG = base + 6 * TILE_BYTES;
  const uint32_t sP = base + 8 * TILE_BYTES, sD = base + 10 * TILE_BYTES;     // P block, dS block: 2 tiles each
  const uint32_t bars = base + 12 * TILE_BYTES;
  const uint32_t bar_load = bars, bar_sdp = bars + 8, bar_sfree = bars + 16, bar_pds = bars + 24, bar_used = bars + 32,
                 bar_kv_done = bars + 40, bar_kv_free = bars + 48, bar_q_done = bars + 56;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 12 * TILE_BYTES + 64);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  constexpr uint32_t C_S = 0, C_DP = 128, C_DQ = 256, C_DK = 384, C_DV = 448;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int halves = S > 128 ? 2 : 1;
  const int row0 = b * S;
  const int steps = halves * halves;

  if (threadIdx.x == 0) {
    prefetch_tmap(&map_qkv);
    prefetch_tmap(&map_do);
    mbar_init(bar_load, 1); mbar_init(bar_sdp, 1); mbar_init(bar_sfree, 256); mbar_init(bar_pds, 256);
    mbar_init(bar_used, 1); mbar_init(bar_kv_done, 1); mbar_init(bar_kv_free, 256); mbar_init(bar_q_done, 1);
    *abort_flag = 0;
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bar_load, (uint32_t)(4 * halves) * TILE_BYTES);
      for (int t = 0; t < halves; ++t) {
        tma_load_2d(sQ + t * TILE_BYTES, &map_qkv, bar_load, h * DH, row0 + t * 128);
        tma_load_2d(sK + t * TILE_BYTES, &map_qkv, bar_load, d + h * DH, row0 + t * 128);
        tma_load_2d(sV + t * TILE_BYTES, &map_qkv, bar_load, 2 * d + h * DH, row0 + t * 128);
        tma_load_2d(sG + t * TILE_BYTES, &map_do, bar_load, h * DH, row0 + t * 128);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = mbar_wait(bar_load, 0, abort_flag, status, kTimeoutAttn);
      const uint32_t id_sdp = idesc128(128, false, false);     // q k^T and dO v^T: both operands K-major
      const uint32_t id_dq = idesc128(DH, false, true);        // dS (K-major) times k (MN-major)
      const uint32_t id_kv = idesc128(DH, true, true);         // P^T dO and dS^T q: both operands MN-major
      auto issue_sdp = [&](int i) {
        const int kh = i / halves, rh = i - kh * halves;
        for (int ks = 0; ks < DH / UK; ++ks)
          tc_mma(tmem_base + C_S, kmajor_desc(sQ + rh * TILE_BYTES, ks), kmajor_desc(sK + kh * TILE_BYTES, ks), id_sdp,
                 ks > 0 ? 1u : 0u);
        for (int ks = 0; ks < DH / UK; ++ks)
          tc_mma(tmem_base + C_DP, kmajor_desc(sG + rh * TILE_BYTES, ks), kmajor_desc(sV + kh * TILE_BYTES, ks), id_sdp,
                 ks > 0 ? 1u : 0u);
        tc_commit(bar_sdp);
      };
      if (ok) {
        tc_fence_after();
        issue_sdp(0);
      }
      for (int i = 0; i < steps && ok; ++i) {
        const int kh = i / halves, rh = i - kh * halves;
        ok = mbar_wait(bar_pds, (uint32_t)i & 1u, abort_flag, status, kTimeoutAttn);       // P and dS of step i are in place
        if (!ok) break;
        if (rh == 0 && kh > 0) {                                  // dK / dV of the previous key half have been read out
          ok = mbar_wait(bar_kv_free, (uint32_t)(kh - 1) & 1u, abort_flag, status, kTimeoutAttn);
          if (!ok) break;
        }
        tc_fence_after();
        for (int ks = 0; ks < 128 / UK; ++ks) {
          // dQ_rh += dS k_kh   (contraction over the 128 keys of the block)
          tc_mma(tmem_base + C_DQ + rh * 64, kmajor_desc(sD, ks), mnmajor_desc(sK + kh * TILE_BYTES, ks, TILE_BYTES), id_dq,
                 (kh > 0 || ks > 0) ? 1u : 0u);
          // dV_kh += P^T dO_rh ; dK_kh += dS^T q_rh   (contraction over the 128 query rows of the block)
          tc_mma(tmem_base + C_DV, mnmajor_desc(sP, ks, TILE_BYTES), mnmajor_desc(sG + rh * TILE_BYTES, ks, TILE_BYTES), id_kv,
                 (rh > 0 || ks > 0) ? 1u : 0u);
          tc_mma(tmem_base + C_DK, mnmajor_desc(sD, ks, TILE_BYTES), mnmajor_desc(sQ + rh * TILE_BYTES, ks, TILE_BYTES), id_kv,
                 (rh > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(bar_used);
        if (rh == halves - 1) tc_commit(bar_kv_done);
        if (i + 1 < steps) {
          ok = mbar_wait(bar_sfree, (uint32_t)i & 1u, abort_flag, status, kTimeoutAttn);   // S, dP of step i have been read
          if (!ok) break;
          tc_fence_after();
          issue_sdp(i + 1);
        }
      }
      if (ok) tc_commit(bar_q_done);
    }
  } else {
    const int cg = (warp - 2) >> 2;                               // which 64 of the block's 128 keys this thread handles
    const int quad = warp & 3;
    const int trow = quad * 32 + lane;
    const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16);
    float Dr[2] = {0.0f, 0.0f}, lr[2] = {0.0f, 0.0f};
    for (int rh = 0; rh < halves; ++rh) {                          // D_r = dO_r . o_r and the row's log-sum-exp
      const int row = rh * 128 + trow;
      if (row < S) {
        const bf16* o = out + (size_t)(row0 + row) * d + h * DH;
        const bf16* g = dout + (size_t)(row0 + row) * d + h * DH;
        float s = 0.0f;
#pragma unroll
        for (int c = 0; c < DH; c += 8) {
          float ov[8], gv[8];
          load_seg<8>(o + c, 8, ov);
          load_seg<8>(g + c, 8, gv);
#pragma unroll
          for (int i = 0; i < 8; ++i) s = fmaf(gv[i], ov[i], s);
        }
        Dr[rh] = s;
        lr[rh] = lse[(size_t)blockIdx.x * S + row];
      }
    }
    bool ok = true;
    for (int i = 0; i < steps && ok; ++i) {
      const int kh = i / halves, rh = i - kh * halves;
      const int row = rh * 128 + trow;
      const bool rvalid = row < S;
      // P = 2^(s log2e / 8 - lse log2e), all zero in rows past the sequence; dS = P (dP - D) / 8
      const float DS = (rh == 0 ? Dr[0] : Dr[1]) * SCALE;
      const float l2 = rvalid ? (rh == 0 ? lr[0] : lr[1]) * LOG2E : INFINITY;
      ok = mbar_wait(bar_sdp, (uint32_t)i & 1u, abort_flag, status, kTimeoutAttn);
      if (!ok) break;
      if (i > 0) {                                                // the previous block's P / dS have been consumed
        ok = mbar_wait(bar_used, (uint32_t)(i - 1) & 1u, abort_flag, status, kTimeoutAttn);
        if (!ok) break;
      }
      tc_fence_after();
      uint8_t* Pt = gen + 8 * TILE_BYTES + cg * TILE_BYTES;
      uint8_t* Dt = gen + 10 * TILE_BYTES + cg * TILE_BYTES;
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {                               // 32 keys at a time
        float sv[32], pv[32];
        tmem_ld32_issue(tlane + C_S + cg * 64 + c * 32, sv);
        tmem_ld32_issue(tlane + C_DP + cg * 64 + c * 32, pv);
        tmem_ld_wait(sv, pv);
        if (c == 1) {                                             // last read of this block's S and dP by this thread
          tc_fence_before();
          mbar_arrive(bar_sfree);
        }
        const int key0 = kh * 128 + cg * 64 + c * 32;
        if (key0 + 32 <= S) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float p = ex2(fmaf(sv[j], SCALE_LOG2E, -l2));
            sv[j] = p;
            pv[j] = p * fmaf(pv[j], SCALE, -DS);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float p = key0 + j < S ? ex2(fmaf(sv[j], SCALE_LOG2E, -l2)) : 0.0f;
            sv[j] = p;
            pv[j] = p * fmaf(pv[j], SCALE, -DS);
          }
        }
        sts_row32(Pt, trow, c, sv);
        sts_row32(Dt, trow, c, pv);
      }
      fence_async_smem();
      mbar_arrive(bar_pds);
      if (rh == halves - 1) {
        // dK and dV of key half kh are complete: lane = key, 32 of the 64 head columns per thread
        ok = mbar_wait(bar_kv_done, (uint32_t)kh & 1u, abort_flag, status, kTimeoutAttn);
        if (!ok) break;
        tc_fence_after();
        float kv[32], vv[32];
        tmem_ld32_issue(tlane + C_DK + cg * 32, kv);
        tmem_ld32_issue(tlane + C_DV + cg * 32, vv);
        tmem_ld_wait(kv, vv);
        tc_fence_before();
        mbar_arrive(bar_kv_free);
        const int key = kh * 128 + trow;
        if (key < S) {
          bf16* g = dqkv + (size_t)(row0 + key) * 3 * d + h * DH + cg * 32;
          store32_bf16(g + d, kv, 1.0f);
          store32_bf16(g + 2 * d, vv, 1.0f);
        }
      }
    }
    if (ok) ok = mbar_wait(bar_q_done, 0, abort_flag, status, kTimeoutAttn);
    if (ok) {
      tc_fence_after();
      float q0[32], q1[32];                                       // dQ of row halves 0 and 1 (the second unused when S <= 128)
      tmem_ld32_issue(tlane + C_DQ + cg * 32, q0);
      tmem_ld32_issue(tlane + C_DQ + 64 + cg * 32, q1);
      tmem_ld_wait(q0, q1);
      if (trow < S) store32_bf16(dqkv + (size_t)(row0 + trow) * 3 * d + h * DH + cg * 32, q0, 1.0f);
      if (halves == 2 && 128 + trow < S)
        store32_bf16(dqkv + (size_t)(row0 + 128 + trow) * 3 * d + h * DH + cg * 32, q1, 1.0f);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace attn
}  // namespace et
