// bf16 x bf16 -> fp32 GEMM on the sm_100a tensor cores: TMA-fed shared-memory ring,
// tcgen05.mma issued by one thread, accumulators in tensor memory (double-buffered so the
// epilogue of one tile overlaps the main loop of the next), persistent over work units.
//
// One kernel serves the three GEMMs of a dense layer; they differ in which operand
// dimension is contiguous in memory ("major"):
//   forward  Z  = a  * W      A = a   K-major,   B = W   MN-major
//   dgrad    dX = dZ * W^T    A = dZ  K-major,   B = W   K-major
//   wgrad    dW = a^T * dZ    A = a   MN-major,  B = dZ  MN-major   (contraction over tokens)
//
// PAIR = true runs two CTAs of a cluster as one unit (tcgen05 cta_group::2): a 256-row tile whose
// B operand is split between the two CTAs' shared memories, so each CTA fetches half as many B
// bytes from L2 per flop.  CTA 0 of the pair issues the MMAs; every load of either CTA reports
// to CTA 0's "full" barrier; MMA completion is signalled to both CTAs' "empty" / "accumulator
// full" barriers; both CTAs' epilogue warps report to CTA 0's "accumulator empty" barrier.
//
// Epilogues that read or write bf16 tensors (forward, dgrad) move them with TMA through
// 128-byte-swizzled shared-memory chunks of 128 rows x 64 columns.  Two groups of four epilogue
// warps each take every other chunk of a tile; per group one extra thread does all the TMA work:
// it prefetches the operand chunks (skip gradient, pre-activation, residual) while the main
// loop of the tile is still running, and stores a chunk once the group's 128 threads have
// combined it with the accumulator in place.  The epilogue warps therefore never wait for a
// copy they issued themselves, and global traffic is fully coalesced although each epilogue
// thread owns one accumulator row.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "epilogue.cuh"

namespace et {
namespace tc {

constexpr int BM = 128;          // output rows per tile  (UMMA M)
constexpr int BK = 64;           // contraction elements per stage = one 128-byte swizzle row
constexpr int UK = 16;           // contraction elements per tcgen05.mma (bf16)
constexpr int ACC_STAGES = 2;    // accumulator stages at TMEM columns 0 and 256
constexpr int ACC_STRIDE = 256;
constexpr int THREADS = 384;     // warp 0: TMA producer, warp 1: MMA + TMEM alloc, warps 2-9: two epilogue groups,
                                 // warps 10-11: one TMA thread per epilogue group
constexpr int EPI_GROUPS = 2;
constexpr uint32_t CHUNK_BYTES = 64 * BK * 2;       // one TMA box: 64 rows of 128 B
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;
constexpr uint32_t EPI_CHUNK_BYTES = BM * 64 * 2;   // 128 rows x 64 bf16 columns
constexpr int EPI_SETS = 2;      // staged-epilogue buffer sets per group: one being combined, one in flight
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t SMEM_LIMIT = 227 * 1024;
constexpr uint32_t SMEM_SLACK = 1024 /*alignment*/ + 256 /*barriers*/;

template <int BN, int SLOTS, bool PAIR>
struct Cfg {
  static constexpr int BNH = PAIR ? BN / 2 : BN;                 // B columns this CTA loads
  static constexpr uint32_t B_STAGE_BYTES = BNH * BK * 2;
  static constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
  static constexpr uint32_t EPI_BYTES = (uint32_t)EPI_GROUPS * EPI_SETS * SLOTS * EPI_CHUNK_BYTES;
  static constexpr int STAGES_FIT = (int)((SMEM_LIMIT - SMEM_SLACK - EPI_BYTES) / STAGE_BYTES);
  static constexpr int STAGES = STAGES_FIT > 6 ? 6 : STAGES_FIT;
  static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + SMEM_SLACK;
  static_assert(STAGES >= 3, "too few pipeline stages");
  static_assert(BN % 64 == 0 && BN >= 64 && BN <= 256, "tile width");
  static_assert(BNH % 32 == 0, "half tile width");
};

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
  kTimeoutEpiTma = 5,
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
  int a_3d, b_3d;            // MN-major operand fetched by one 3-D copy (all 64-wide chunks at once)
                             // instead of one 2-D copy per chunk; needs its width to be a multiple of 64
  // Convolution without a gathered matrix (single-CTA tiles only): A's tiles are fetched by TMA in im2col
  // mode from the NHWC tensor.  1: rows of A are pixels (forward, dgrad: K-major, one tap per fold segment,
  // map with 128 pixels per column); 2: the contraction runs over pixels (wgrad: MN-major, rows of A are
  // (tap, channel), map with 64 pixels per column).
  int a_im2col;
  int img_w, img_h, ksize;   // image extent in pixels, taps per side (zero padding ksize / 2, stride 1)
  int chan;                  // wgrad: channels per tap (a multiple of 128)
  int a_tap_flip;            // dgrad: segment s reads tap ksize^2 - 1 - s (the kernel turned by 180 degrees)
  uint32_t* status;          // device word, 0 = ok; first failure wins
};

// Tensor maps of the staged epilogue: per slot one optional input and one optional output,
// all [rows x cols] bf16 row-major with the output's shape, boxes of 64 columns x 128 rows.
struct EpiMaps {
  CUtensorMap in[2];
  CUtensorMap out[2];
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
// Pair variant: the copy lands in this CTA's shared memory, its bytes are reported to the barrier
// at the same offset in CTA 0 of the pair (cluster shared addresses carry the CTA rank in bit 24).
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar & kPeerBitMask), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar & kPeerBitMask), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// im2col mode: `pixels per column` consecutive base pixels of the tensor map's bounding box, walked w first,
// then h, then image, starting at base pixel (w, h, n); each read at offset (ow, oh) from its base pixel,
// channels [c, c + 64); zeros outside the image.
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w, int h, int n,
                                                int ow, int oh) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"((uint16_t)ow), "h"((uint16_t)oh)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `cta` of the cluster
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t cta) {
  asm volatile(
      "{\n\t.reg .b32 rem;\n\t"
      "mapa.shared::cluster.u32 rem, %0, %1;\n\t"
      "mbarrier.arrive.shared::cluster.b64 _, [rem];\n\t}"
      ::"r"(bar), "r"(cta)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {     // arrives in both CTAs of the pair
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
// The TMA unit reads a descriptor from memory the first time an instruction names it (about a
// microsecond); asking for it at kernel entry hides that behind the barrier and TMEM set-up.
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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

// Two 32-column reads in flight, one wait.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, float (&v)[32]) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
// The "+r" constraints tie the wait to the registers the loads write: the compiler may not read
// them earlier or move the wait past their first use.
__device__ __forceinline__ void tmem_ld_wait(float (&a)[32], float (&b)[32]) {
  uint32_t* x = reinterpret_cast<uint32_t*>(a);
  uint32_t* y = reinterpret_cast<uint32_t*>(b);
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(x[0]), "+r"(x[1]), "+r"(x[2]), "+r"(x[3]), "+r"(x[4]), "+r"(x[5]), "+r"(x[6]), "+r"(x[7]),
                 "+r"(x[8]), "+r"(x[9]), "+r"(x[10]), "+r"(x[11]), "+r"(x[12]), "+r"(x[13]), "+r"(x[14]), "+r"(x[15]),
                 "+r"(x[16]), "+r"(x[17]), "+r"(x[18]), "+r"(x[19]), "+r"(x[20]), "+r"(x[21]), "+r"(x[22]), "+r"(x[23]),
                 "+r"(x[24]), "+r"(x[25]), "+r"(x[26]), "+r"(x[27]), "+r"(x[28]), "+r"(x[29]), "+r"(x[30]), "+r"(x[31])
               :: "memory");
  asm volatile(""
               : "+r"(y[0]), "+r"(y[1]), "+r"(y[2]), "+r"(y[3]), "+r"(y[4]), "+r"(y[5]), "+r"(y[6]), "+r"(y[7]),
                 "+r"(y[8]), "+r"(y[9]), "+r"(y[10]), "+r"(y[11]), "+r"(y[12]), "+r"(y[13]), "+r"(y[14]), "+r"(y[15]),
                 "+r"(y[16]), "+r"(y[17]), "+r"(y[18]), "+r"(y[19]), "+r"(y[20]), "+r"(y[21]), "+r"(y[22]), "+r"(y[23]),
                 "+r"(y[24]), "+r"(y[25]), "+r"(y[26]), "+r"(y[27]), "+r"(y[28]), "+r"(y[29]), "+r"(y[30]), "+r"(y[31])
               :: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout code 2), descriptor version 1.
// Every operand stage is a sequence of 8-KB chunks of 64 rows of 128 B.
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
template <int MM, int BN, bool A_MN, bool B_MN>
__host__ __device__ constexpr uint32_t make_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
         ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(MM >> 4) << 24);
}

template <class Epi>
__device__ __forceinline__ void epi_set_split(Epi&, int) {}
__device__ __forceinline__ void epi_set_split(PartialEpi& e, int s) { e.split = s; }

// 16-byte piece `piece` (0..7) of row `row` (0..127) inside a staged 128 x 64 bf16 chunk.
__device__ __forceinline__ uint32_t epi_chunk_off(int row, int piece) {
  return (uint32_t)((row >> 6) * CHUNK_BYTES + (row & 63) * 128 + ((piece ^ (row & 7)) << 4));
}
__device__ __forceinline__ void lds_row32(const uint8_t* chunk, int row, int half, float (&v)[32]) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint4 q = *reinterpret_cast<const uint4*>(chunk + epi_chunk_off(row, half * 4 + j));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[j * 8 + 2 * i] = __uint_as_float(w[i] << 16);
      v[j * 8 + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
}
__device__ __forceinline__ void sts_row32(uint8_t* chunk, int row, int half, const float (&v)[32]) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint4 q;
    q.x = pack_bf16x2(v[j * 8 + 0], v[j * 8 + 1]);
    q.y = pack_bf16x2(v[j * 8 + 2], v[j * 8 + 3]);
    q.z = pack_bf16x2(v[j * 8 + 4], v[j * 8 + 5]);
    q.w = pack_bf16x2(v[j * 8 + 6], v[j * 8 + 7]);
    *reinterpret_cast<uint4*>(chunk + epi_chunk_off(row, half * 4 + j)) = q;
  }
}

// --------------------------------------------------------------------------- the kernel
// Epi::kSlots == 0: direct epilogue, Epi::operator()<32>(row, col0, n, acc) stores by itself.
// Epi::kSlots  > 0: staged epilogue, Epi::combine(col0, acc, s0, s1) turns the accumulator and
//                   the slots' input values into the slots' output values, in place; the flags
//                   Epi::has_in[s] / has_out[s] say which slots carry an input / an output.
template <int BN, bool A_MN, bool B_MN, class Epi, bool PAIR>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ EpiMaps emaps, const Params p, const Epi epi_in) {
  constexpr int SLOTS = Epi::kSlots;
  using C = Cfg<BN, SLOTS, PAIR>;
  constexpr int BNH = C::BNH;
  static_assert(BNH % 64 == 0 || !B_MN, "an MN-major B needs whole 64-element chunks per CTA");
  constexpr int TILE_M = PAIR ? 2 * BM : BM;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const bool leader_cta = rank == 0;
  const int unit0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int unit_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr int STAGES = C::STAGES;
  constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES;
  constexpr int NCHUNK = BN / 64;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzle atoms need 1024-B alignment
  uint8_t* gen_base = smem_raw + (base - raw);
  const uint32_t epi_base = base + STAGES * STAGE_BYTES;        // [group][buffer set][slot][EPI_CHUNK_BYTES]
  const uint32_t bars = epi_base + C::EPI_BYTES;
  // barrier slots (8 B each)
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int s) { return bars + 8u * (2 * STAGES + s); };
  auto acc_empty_bar = [&](int s) { return bars + 8u * (2 * STAGES + 2 + s); };
  // per epilogue group g and buffer set b: "operands have landed" and "result is in place"
  auto in_full_bar = [&](int g, int b) { return bars + 8u * (2 * STAGES + 4 + g * EPI_SETS + b); };
  auto out_ready_bar = [&](int g, int b) { return bars + 8u * (2 * STAGES + 4 + (EPI_GROUPS + g) * EPI_SETS + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      gen_base + STAGES * STAGE_BYTES + C::EPI_BYTES + 8 * (2 * STAGES + 4 + 2 * EPI_GROUPS * EPI_SETS));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (warp == 0 && lane == 0) { prefetch_tmap(&map_a); prefetch_tmap(&map_b); }
  if constexpr (SLOTS > 0) {
    if (warp >= 2 + 4 * EPI_GROUPS && lane == 0) {
#pragma unroll
      for (int s = 0; s < SLOTS; ++s) {
        if (epi_in.has_in[s]) prefetch_tmap(&emaps.in[s]);
        if (epi_in.has_out[s]) prefetch_tmap(&emaps.out[s]);
      }
    }
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), PAIR ? 16 : 8); }
    for (int g = 0; g < EPI_GROUPS; ++g)
      for (int b = 0; b < EPI_SETS; ++b) { mbar_init(in_full_bar(g, b), 1); mbar_init(out_ready_bar(g, b), 128); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();          // the peer's barriers exist before anything targets them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: everything above touched only this CTA's own shared and tensor
  // memory, so it may run while the previous kernel of the stream drains.  From here on global memory
  // is read and written: wait until that kernel has completed and its writes are visible (returns at
  // once in an ordinary launch), then let the next kernel's CTAs take each SM as this grid leaves it.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
      auto load = [&](uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1) {
        if constexpr (PAIR) tma_load_2d_pair(dst, m, bar, c0, c1);
        else tma_load_2d(dst, m, bar, c0, c1);
      };
      auto load3 = [&](uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2) {
        if constexpr (PAIR) tma_load_3d_pair(dst, m, bar, c0, c1, c2);
        else tma_load_3d(dst, m, bar, c0, c1, c2);
      };
      for (int u = unit0; u < units && ok; u += unit_step) {
        const int sp = u / tiles, t = u - sp * tiles;
        const int m0 = (t / p.tiles_n) * TILE_M + (int)rank * BM, n0 = (t % p.tiles_n) * BN;
        const int kb0 = sp * p.kb_per_split;
        const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        int seg = kb0 / p.kb_per_seg, kk = (kb0 - seg * p.kb_per_seg) * BK;   // fold segment, k offset inside it
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, kTimeoutProducer);
          if (!ok) break;
          const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
          const uint32_t bar = full_bar(stage);
          // in a pair, CTA 0 announces the bytes of both CTAs' copies
          if (leader_cta) mbar_expect_tx(bar, (PAIR ? 2u : 1u) * STAGE_BYTES);
          // Few, large copies: issuing a TMA copy costs the producer thread far more than
          // the copy's size does.  K-major operands come as one box of 64 k x (tile rows);
          // MN-major operands as one 3-D box (64 mn, 64 k, chunks) when their width allows.
          if (!PAIR && p.a_im2col != 0) {
            const int pad = p.ksize >> 1, hw = p.img_h * p.img_w;
            if constexpr (!A_MN) {
              // 128 pixels from m0 on; this segment's tap
              const int tap = p.a_tap_flip ? p.ksize * p.ksize - 1 - seg : seg;
              const int n_img = m0 / hw, r = m0 - n_img * hw, ph = r / p.img_w, pw = r - ph * p.img_w;
              tma_load_im2col(sa, &map_a, bar, kk, pw - pad, ph - pad, n_img, tap % p.ksize, tap / p.ksize);
            } else {
              // rows m0.. of A are (tap, channel); this k-block is 64 pixels from pixel kk on
              const int tap = m0 / p.chan, c0 = m0 - tap * p.chan;
              const int n_img = kk / hw, r = kk - n_img * hw, ph = r / p.img_w, pw = r - ph * p.img_w;
#pragma unroll
              for (int c = 0; c < BM / 64; ++c)
                tma_load_im2col(sa + c * CHUNK_BYTES, &map_a, bar, c0 + c * 64, pw - pad, ph - pad, n_img, tap % p.ksize,
                                tap / p.ksize);
            }
          } else if constexpr (!A_MN) {
            load(sa, &map_a, bar, kk, m0);
          } else if (p.a_3d) {
            load3(sa, &map_a, bar, 0, kk, m0 >> 6);
          } else {
#pragma unroll
            for (int c = 0; c < BM / 64; ++c) load(sa + c * CHUNK_BYTES, &map_a, bar, m0 + c * 64, kk);
          }
          const int bk = kk + seg * p.b_k_seg_stride;
          int bn = p.b_mn_wrap > 0 ? n0 % p.b_mn_wrap : n0;
          bn += seg * p.b_mn_seg_stride + (int)rank * BNH;
          if constexpr (!B_MN) {
            load(sb, &map_b, bar, bk, bn);
          } else if (p.b_3d) {
            load3(sb, &map_b, bar, 0, bk, bn >> 6);
          } else {
#pragma unroll
            for (int c = 0; c < BNH / 64; ++c) load(sb + c * CHUNK_BYTES, &map_b, bar, bn + c * 64, bk);
          }
          ++fills[stage];
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          kk += BK;
          if (kk == p.kb_per_seg * BK) { kk = 0; ++seg; }
        }
      }
      if (!ok) {
        // wind-down: let every copy this thread issued land before the CTA's shared memory goes away
        if (leader_cta) {
#pragma unroll
          for (int s = 0; s < STAGES; ++s) {
            if (fills[s] == 0) continue;
            const uint32_t par = (fills[s] - 1u) & 1u;
            bool landed = false;
            for (uint32_t it = 0; it < (1u << 20) && !landed; ++it) landed = mbar_try_wait(full_bar(s), par);
            if (!landed) atomicCAS(p.status, 0u, (uint32_t)kTimeoutDrain);
          }
        } else {
          for (int it = 0; it < 2000; ++it) __nanosleep(1000);   // CTA 1 has no barrier of its own to watch
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && leader_cta) {
      constexpr uint32_t idesc = make_idesc<TILE_M, BN, A_MN, B_MN>();
      const uint64_t desc_a0 = A_MN ? make_desc(base, CHUNK_BYTES, 1024) : make_desc(base, 16, 1024);
      const uint64_t desc_b0 = B_MN ? make_desc(base + A_STAGE_BYTES, CHUNK_BYTES, 1024)
                                    : make_desc(base + A_STAGE_BYTES, 16, 1024);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = unit0; u < units && ok; u += unit_step) {
        const int sp = u / tiles;
        const int kb0 = sp * p.kb_per_split;
        const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        ok = mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, kTimeoutMma);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_STRIDE);
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, kTimeoutMma);
          if (!ok) break;
          tc_fence_after();
          // descriptors of this stage: the address field (16-byte units) is the only part that
          // moves.  K-major: 16 elements = 32 B further along the swizzled row per MMA;
          // MN-major: 16 k-rows = two 1024-B groups further.
          const uint64_t da = desc_a0 + (uint64_t)((uint32_t)stage * (STAGE_BYTES >> 4));
          const uint64_t db = desc_b0 + (uint64_t)((uint32_t)stage * (STAGE_BYTES >> 4));
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
            constexpr uint32_t step_a = (A_MN ? 2048u : 32u) >> 4, step_b = (B_MN ? 2048u : 32u) >> 4;
            const uint32_t accumulate = (kb > kb0 || k > 0) ? 1u : 0u;
            if constexpr (PAIR) tc_mma_pair(d_tmem, da + k * step_a, db + k * step_b, idesc, accumulate);
            else tc_mma(d_tmem, da + k * step_a, db + k * step_b, idesc, accumulate);
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if constexpr (PAIR) tc_commit_pair(empty_bar(stage)); else tc_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if constexpr (PAIR) tc_commit_pair(acc_full_bar(acc)); else tc_commit(acc_full_bar(acc));   // accumulator complete
        if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 2 + 4 * EPI_GROUPS) {
    // ------------------------------------------------------------------ epilogue TMA thread of group g
    if constexpr (SLOTS > 0) {
      const int g = warp - (2 + 4 * EPI_GROUPS);
      if (lane == 0 && g < EPI_GROUPS) {
        uint32_t tx = 0;
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) tx += epi_in.has_in[s] ? EPI_CHUNK_BYTES : 0u;
        // The group's chunks, in order, are numbered j = 0, 1, ...; chunk j uses buffer set j % 2.
        // fetch(j) may start once the store of chunk j - 2 has finished reading that set.
        // Two cursors walk the same chunk sequence: one for fetches (two chunks ahead), one for stores.
        struct Cursor {
          int u, c, m0, n0;
          bool fresh;
        };
        auto advance = [&](Cursor& k, int* m0, int* col0) -> bool {      // next chunk of this group, if any
          while (k.u < units) {
            if (k.fresh) {
              const int t = k.u % tiles;
              k.m0 = (t / p.tiles_n) * TILE_M + (int)rank * BM;
              k.n0 = (t % p.tiles_n) * BN;
              k.c = g;
              k.fresh = false;
            }
            if (k.c < NCHUNK && k.n0 + k.c * 64 < p.cols) {
              *m0 = k.m0;
              *col0 = k.n0 + k.c * 64;
              k.c += EPI_GROUPS;
              return true;
            }
            k.u += unit_step;
            k.fresh = true;
          }
          return false;
        };
        Cursor fc{unit0, 0, 0, 0, true}, sc{unit0, 0, 0, 0, true};
        int fetched = 0;                                                 // chunks requested so far
        auto fetch = [&]() {
          int m0, col0;
          if (!advance(fc, &m0, &col0)) return;
          const int b = fetched & 1;
          ++fetched;
          const uint32_t bar = in_full_bar(g, b);
          if (tx > 0) {
            mbar_expect_tx(bar, tx);
#pragma unroll
            for (int s = 0; s < SLOTS; ++s) {
              if (!epi_in.has_in[s]) continue;
              const uint32_t dst = epi_base + (uint32_t)(((g * EPI_SETS + b) * SLOTS + s) * EPI_CHUNK_BYTES);
              tma_load_2d(dst, &emaps.in[s], bar, col0, m0);       // one box of 64 columns x 128 rows
            }
          } else {
            mbar_arrive(bar);                                      // nothing to fetch: hand the set over
          }
        };
        fetch();
        fetch();
        bool ok = true;
        int j = 0;
        for (;; ++j) {
          int m0, col0;
          if (!advance(sc, &m0, &col0)) break;
          const int b = j & 1;
          ok = mbar_wait(out_ready_bar(g, b), (uint32_t)(j >> 1) & 1u, abort_flag, p.status, kTimeoutEpiTma);
          if (!ok) break;
          if (m0 < p.rows) {
#pragma unroll
            for (int s = 0; s < SLOTS; ++s) {
              if (!epi_in.has_out[s]) continue;
              const uint32_t src = epi_base + (uint32_t)(((g * EPI_SETS + b) * SLOTS + s) * EPI_CHUNK_BYTES);
              tma_store_2d(&emaps.out[s], src, col0, m0);
            }
          }
          tma_store_commit();
          tma_store_wait_read<0>();                   // the set may be overwritten from here on
          fetch();
        }
        tma_store_wait_all();                         // shared memory must outlive the last store
        if (!ok && tx > 0) {
          // wind-down: copies already requested must land before the CTA's shared memory goes away
          for (int f = max(j, fetched - 2); f < fetched; ++f) {
            bool landed = false;
            for (uint32_t it = 0; it < (1u << 20) && !landed; ++it)
              landed = mbar_try_wait(in_full_bar(g, f & 1), (uint32_t)(f >> 1) & 1u);
            if (!landed) atomicCAS(p.status, 0u, (uint32_t)kTimeoutDrain);
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 2..9
    Epi epi = epi_in;
    const int g = (warp - 2) >> 2;                  // epilogue group: takes the tile's chunks c with c % 2 == g
    const int quad = warp & 3;                      // TMEM lanes this warp may read: 32*quad ...
    const int trow = quad * 32 + lane;              // row inside the tile
    int acc = 0;
    uint32_t acc_phase = 0;
    int j = 0;                                      // staged path: running chunk number of this group
    bool ok = true;
    auto release_acc = [&](int a) {
      if constexpr (PAIR) mbar_arrive_remote(acc_empty_bar(a), 0u);
      else mbar_arrive(acc_empty_bar(a));
    };
    for (int u = unit0; u < units && ok; u += unit_step) {
      const int sp = u / tiles, t = u - sp * tiles;
      const int m0 = (t / p.tiles_n) * TILE_M + (int)rank * BM, n0 = (t % p.tiles_n) * BN;
      epi_set_split(epi, sp);
      ok = mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, p.status, kTimeoutEpilogue);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * ACC_STRIDE);
      if constexpr (SLOTS == 0) {
        const int row = m0 + trow;
#pragma unroll 1
        for (int c = g; c < NCHUNK; c += EPI_GROUPS) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float v[32];
            tmem_ld32(taddr + c * 64 + h * 32, v);  // warp-collective: every lane takes part
            const int col0 = n0 + c * 64 + h * 32;
            const int nv = p.cols - col0;
            if (row < p.rows && nv > 0) epi.template operator()<32>(row, col0, nv, v);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) release_acc(acc);
      } else {
        int nch = 0;                                // this group's chunks in this tile
#pragma unroll
        for (int c = 0; c < NCHUNK; ++c) nch += ((c & 1) == g && n0 + c * 64 < p.cols) ? 1 : 0;
        if (nch == 0) {                             // nothing to read, but the accumulator still has to be handed back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) release_acc(acc);
        }
#pragma unroll 1
        for (int i = 0; i < nch; ++i, ++j) {
          const int c = g + 2 * i;
          const int col0 = n0 + c * 64;
          const int b = j & 1;
          float v0[32], v1[32];
          tmem_ld32_issue(taddr + c * 64, v0);
          tmem_ld32_issue(taddr + c * 64 + 32, v1);
          tmem_ld_wait(v0, v1);
          if (i == nch - 1) {                       // last read of this accumulator by this warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) release_acc(acc);
          }
          ok = mbar_wait(in_full_bar(g, b), (uint32_t)(j >> 1) & 1u, abort_flag, p.status, kTimeoutEpilogue);
          if (!ok) break;
          uint8_t* buf0 = gen_base + STAGES * STAGE_BYTES + ((g * EPI_SETS + b) * SLOTS + 0) * EPI_CHUNK_BYTES;
          uint8_t* buf1 = gen_base + STAGES * STAGE_BYTES + ((g * EPI_SETS + b) * SLOTS + (SLOTS - 1)) * EPI_CHUNK_BYTES;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float (&v)[32] = h == 0 ? v0 : v1;
            float s0[32], s1[32];
            if (epi.has_in[0]) lds_row32(buf0, trow, h, s0);
            if (SLOTS > 1 && epi.has_in[SLOTS - 1]) lds_row32(buf1, trow, h, s1);
            epi.combine(col0 + h * 32, p.cols - (col0 + h * 32), v, s0, s1);
            if (epi.has_out[0]) sts_row32(buf0, trow, h, s0);
            if (SLOTS > 1 && epi.has_out[SLOTS - 1]) sts_row32(buf1, trow, h, s1);
            epi.column_sums((m0 >> 5) + quad, col0 + h * 32, p.cols - (col0 + h * 32), s0, s1, lane);
          }
          fence_async_smem();                       // generic-proxy writes -> visible to the TMA engine
          mbar_arrive(out_ready_bar(g, b));         // 128 arrivals: the group's TMA thread may store the chunk
        }
      }
      if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();          // neither CTA leaves while the other may still touch it
  if (warp == 1) {
    tc_fence_after();
    if constexpr (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tc
}  // namespace et
