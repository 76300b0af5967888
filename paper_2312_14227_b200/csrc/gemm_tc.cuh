// bf16 x bf16 -> fp32 GEMM on the sm_100a tensor cores: TMA-fed shared-memory ring,
// tcgen05.mma issued by one thread, accumulators in tensor memory (double-buffered so the
// epilogue of one tile overlaps the main loop of the next), persistent over work units.
//
// One kernel serves the three GEMMs of a dense layer; they differ in which operand
// dimension is contiguous in memory ("major"):
//   forward  Z  = a  * W      A = a   K-major,   B = W   MN-major
//   dgrad    dX = dZ * W^T    A = dZ  K-major,   B = W   K-major
//   wgrad    dW = a^T * dZ    A = a   MN-major,  B = dZ  MN-major   (contraction over tokens)
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "epilogue.cuh"

namespace et {
namespace tc {

constexpr int BM = 128;          // output rows per tile  (UMMA M)
constexpr int BN = 256;          // output cols per tile  (UMMA N)
constexpr int BK = 64;           // contraction elements per stage = one 128-byte swizzle row
constexpr int UK = 16;           // contraction elements per tcgen05.mma (bf16)
constexpr int STAGES = 4;
constexpr int ACC_STAGES = 2;    // 2 x 256 fp32 columns = all 512 TMEM columns
constexpr int THREADS = 192;     // warp 0: TMA, warp 1: MMA + TMEM alloc, warps 2-5: epilogue
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;
constexpr uint32_t B_STAGE_BYTES = BN * BK * 2;
constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr uint32_t CHUNK_BYTES = 64 * BK * 2;   // one TMA box: 64 rows of 128 B
constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr uint32_t TMEM_COLS = 512;

// Bounded waits: a wait that has not succeeded after this many polls gives up, records
// where, and the CTA winds down.  Each poll may block inside try_wait for a while, so the
// limit corresponds to seconds, far beyond any legitimate wait.
constexpr uint32_t WAIT_LIMIT = 1u << 24;

enum StatusCode : uint32_t {
  kStatusOk = 0,
  kTimeoutProducer = 1,
  kTimeoutMma = 2,
  kTimeoutEpilogue = 3,
  kTimeoutDrain = 4,
};

struct Params {
  int rows, cols;            // extent of the output
  int tiles_m, tiles_n;      // ceil(rows/BM), ceil(cols/BN)
  int split;                 // number of contraction splits (1 unless wgrad)
  int kb_total;              // BK-blocks in the whole contraction (all fold segments)
  int kb_per_seg;            // BK-blocks per fold segment; A's k coordinate restarts each segment
  int kb_per_split;          // ceil(kb_total / split); every split is non-empty
  int b_k_seg_stride;        // added to B's k coordinate per segment   (dgrad through a fold)
  int b_mn_seg_stride;       // added to B's mn coordinate per segment  (forward through a fold)
  int b_mn_wrap;             // B's mn coordinate taken modulo this, 0 = off (wgrad through a fold)
  uint32_t* status;          // device word, 0 = ok; first failure wins
};

// --------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Returns false if the wait gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t code) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag != 0) return false;
  }
  *abort_flag = 1;
  atomicCAS(status, 0u, code);
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout code 2), descriptor version 1.
// Every operand stage is a sequence of 8-KB chunks, one TMA box each: 64 rows of 128 B.
//   K-major  : a row holds 64 contraction elements of one mn index; 8-row groups are 1024 B
//              apart (stride offset); the leading offset is unused with swizzling (set 1).
//   MN-major : a row holds 64 mn elements of one k; 8 k-rows form a 1024-B group (stride
//              offset = distance between k groups); the next 64 mn elements are one chunk
//              further (leading offset = CHUNK_BYTES).
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lead_bytes, uint32_t stride_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lead_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((stride_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulate (bits 4-5 = 1), bf16 A and B
// (bits 7-9, 10-12 = 1), operand major-ness (bits 15, 16), N/8 (bits 17-22), M/16 (bits 24-28).
template <bool A_MN, bool B_MN>
__host__ __device__ constexpr uint32_t make_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
         ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

template <class Epi>
__device__ __forceinline__ void epi_set_split(Epi&, int) {}
__device__ __forceinline__ void epi_set_split(PartialEpi& e, int s) { e.split = s; }

// --------------------------------------------------------------------------- the kernel
template <bool A_MN, bool B_MN, class Epi>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const Params p, const Epi epi_in) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzle atoms need 1024-B alignment
  uint8_t* gen_base = smem_raw + (base - raw);
  const uint32_t bars = base + STAGES * STAGE_BYTES;
  // barrier slots (8 B each): full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int s) { return bars + 8u * (2 * STAGES + s); };
  auto acc_empty_bar = [&](int s) { return bars + 8u * (2 * STAGES + ACC_STAGES + s); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * STAGE_BYTES + 128);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < ACC_STAGES; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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

  const int tiles = p.tiles_m * p.tiles_n;
  const int units = tiles * p.split;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t fills[STAGES];
#pragma unroll
      for (int s = 0; s < STAGES; ++s) fills[s] = 0;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int sp = u / tiles, t = u - sp * tiles;
        const int m0 = (t / p.tiles_n) * BM, n0 = (t % p.tiles_n) * BN;
        const int kb0 = sp * p.kb_per_split;
        const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, kTimeoutProducer);
          if (!ok) break;
          const int seg = kb / p.kb_per_seg, kk = (kb - seg * p.kb_per_seg) * BK;
          const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
          const uint32_t bar = full_bar(stage);
          mbar_expect_tx(bar, STAGE_BYTES);
          // every tensor map has a 64 x 64 box: one box = one 8-KB chunk of 64 rows of 128 B
#pragma unroll
          for (int c = 0; c < BM / 64; ++c) {
            if (A_MN) tma_load_2d(sa + c * CHUNK_BYTES, &map_a, bar, m0 + c * 64, kk);
            else      tma_load_2d(sa + c * CHUNK_BYTES, &map_a, bar, kk, m0 + c * 64);
          }
          const int bk = kk + seg * p.b_k_seg_stride;
          int bn = p.b_mn_wrap > 0 ? n0 % p.b_mn_wrap : n0;
          bn += seg * p.b_mn_seg_stride;
#pragma unroll
          for (int c = 0; c < BN / 64; ++c) {
            if (B_MN) tma_load_2d(sb + c * CHUNK_BYTES, &map_b, bar, bn + c * 64, bk);
            else      tma_load_2d(sb + c * CHUNK_BYTES, &map_b, bar, bk, bn + c * 64);
          }
          ++fills[stage];
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // wind-down: let every copy this thread issued land before the CTA's shared memory goes away
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
          if (fills[s] == 0) continue;
          const uint32_t par = (fills[s] - 1u) & 1u;
          bool landed = false;
          for (uint32_t it = 0; it < (1u << 20) && !landed; ++it) landed = mbar_try_wait(full_bar(s), par);
          if (!landed) atomicCAS(p.status, 0u, (uint32_t)kTimeoutDrain);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc<A_MN, B_MN>();
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int sp = u / tiles;
        const int kb0 = sp * p.kb_per_split;
        const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        ok = mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, kTimeoutMma);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, kTimeoutMma);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
            // K-major: 16 elements = 32 B further along the swizzled row.
            // MN-major: 16 k-rows = two 1024-B groups further.
            const uint64_t da = A_MN ? make_desc(sa + k * 2048, CHUNK_BYTES, 1024) : make_desc(sa + k * 32, 16, 1024);
            const uint64_t db = B_MN ? make_desc(sb + k * 2048, CHUNK_BYTES, 1024) : make_desc(sb + k * 32, 16, 1024);
            tc_mma(d_tmem, da, db, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));              // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(acc_full_bar(acc));               // accumulator complete
        if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps)
    Epi epi = epi_in;
    const int quad = warp & 3;                      // TMEM lanes this warp may read: 32*quad ...
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
      const int sp = u / tiles, t = u - sp * tiles;
      const int m0 = (t / p.tiles_n) * BM, n0 = (t % p.tiles_n) * BN;
      epi_set_split(epi, sp);
      ok = mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, p.status, kTimeoutEpilogue);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + quad * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        float v[32];
        tmem_ld32(taddr + c * 32, v);               // warp-collective: every lane takes part
        const int col0 = n0 + c * 32;
        const int n = p.cols - col0;
        if (row < p.rows && n > 0) epi.template operator()<32>(row, col0, n, v);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty_bar(acc));
      if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tc
}  // namespace et
