// One persistent launch for all the GEMMs of an elastic backward pass.
//
// The error-gradient GEMMs dX_l = dZ_l W_l^T of consecutive layers form a chain, but only row tile
// by row tile: rows [r, r + 256) of dX_l need rows [r, r + 256) of dZ_l and nothing else of it.
// Launching one kernel per layer therefore waits far more than the data does -- every launch ends
// in a partly filled last wave, a drain and the next kernel's prologue.  Here the work units of
// every selected GEMM of the pass (error gradients above the deepest selected layer, Section 2.2;
// weight gradients of the selected kernels, Section 5.1) form one list in device memory that the
// CTA pairs of a single cooperative launch walk round-robin.  A unit waits on a counter in global
// memory until the units that produce its operand rows have stored them; counters are bumped after
// the producing stores have completed.  Units only ever depend on units earlier in the list and
// every CTA takes its units in list order, so with all CTAs resident (cooperative launch) some
// unit can always proceed.  Every wait is bounded and ends in the status word, as in gemm_tc.cuh.
//
// Tile: 256 x 256 per CTA pair (tcgen05 cta_group::2), the shape and the warp roles of
// gemm_tc_kernel<256, ., ., ., true>; operand major-ness and the epilogue are per task:
//   kDgrad  A = dZ_l K-major, B = W_l K-major, staged epilogue DgradEpiS<1> (skip gradient or
//           act'(Z) of the layer below, optional fused bias column sums)
//   kWgrad  A = a_l MN-major, B = dZ_l MN-major, fp32 partial sums of one contraction split
//   kFwd    the forward pass as the same kind of list (rows [r, r + 256) of a_{l+1} need rows [r, r + 256) of
//           a_l): A = a_l K-major, B = W_l MN-major, staged epilogue FwdEpiS (bias, activation, residual);
//           a layer with an activation stores two chunks per 64 columns, Z_l and a_{l+1}
#pragma once

#include "gemm_tc.cuh"

namespace et {
namespace tl {

using namespace et::tc;

constexpr int LBN = 256;                                 // tile width
constexpr int LBNH = 128;                                // B columns per CTA of the pair
constexpr int LSTAGES = 5;
constexpr uint32_t LB_STAGE_BYTES = LBNH * BK * 2;
constexpr uint32_t LSTAGE_BYTES = A_STAGE_BYTES + LB_STAGE_BYTES;
constexpr uint32_t LEPI_BYTES = (uint32_t)EPI_GROUPS * EPI_SETS * EPI_CHUNK_BYTES;
constexpr uint32_t LSMEM_BYTES = LSTAGES * LSTAGE_BYTES + LEPI_BYTES + SMEM_SLACK;
static_assert(LSMEM_BYTES <= SMEM_LIMIT, "shared memory");
constexpr int LNCHUNK = LBN / 64;
constexpr uint32_t DEP_POLL_LIMIT = 1u << 24;           // polls of a dependency counter before giving up

enum TaskKind : int { kDgrad = 0, kWgrad = 1, kFwd = 2 };
enum ListStatus : uint32_t { kTimeoutDependency = 6 };

struct alignas(128) Task {
  CUtensorMap map_a, map_b;      // operands
  CUtensorMap map_in, map_out;   // staged epilogue: input chunk (skip gradient, Z, or residual), output chunk
  CUtensorMap map_out2;          // kFwd with an activation: Z_l (stored before a_{l+1})
  int kind;
  int rows, cols;                // extent of the output
  int tiles_m, tiles_n, split;
  int kb_total, kb_per_seg, kb_per_split;
  int b_k_seg_stride, b_mn_wrap, b_mn_seg_stride;
  int unit_begin, units;         // this task's slice of the list
  // dependency: counters[wait_base + (wait_per_row ? row tile : 0)] >= wait_target before the A operand
  // (and the epilogue input) of a unit may be fetched; wait2_* likewise for the epilogue input alone
  int wait_base, wait_per_row;
  unsigned wait_target;
  int wait2_base;
  unsigned wait2_target;
  // completion: counters[signal_base + row tile] and counters[signal_base + tiles_m] get one increment per
  // epilogue group and CTA (4 per unit) once the unit's stores have completed; -1 = nobody waits
  int signal_base;
  // kDgrad epilogue
  int has_in, mul_act, act_prev, ld;
  float* colsum;
  // kFwd epilogue (has_in = a residual is added; ld = out_features / fold)
  int entries;                   // chunks stored per 64 columns: 2 with an activation (Z, then the output), else 1
  int act, fold;
  const bf16* bias;
  // kWgrad epilogue
  float* partial;
  unsigned long long split_stride;
  int ld_out;
};

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ const Task* find_task(const Task* tasks, int& ti, int u) {
  while (u >= tasks[ti].unit_begin + tasks[ti].units) ++ti;
  return tasks + ti;
}
__device__ __forceinline__ bool dep_ready(const unsigned* counters, int base, int row_tile, unsigned target) {
  return base < 0 || ld_acquire(counters + base + row_tile) >= target;
}
// Blocking form for a thread that has nothing else to do meanwhile.  False = gave up (or someone else did).
__device__ __forceinline__ bool dep_wait(const unsigned* counters, int base, int row_tile, unsigned target,
                                         volatile uint32_t* abort_flag, uint32_t* status) {
  if (base < 0) return true;
  const unsigned* c = counters + base + row_tile;
  for (uint32_t it = 0; it < DEP_POLL_LIMIT; ++it) {
    if (ld_acquire(c) >= target) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag != 0 || *reinterpret_cast<volatile uint32_t*>(status) != 0) return false;
      __nanosleep(64);
    }
  }
  *abort_flag = 1;
  atomicCAS(status, 0u, (uint32_t)kTimeoutDependency);
  return false;
}

struct UnitPos { int sp, tm, tn; };
__device__ __forceinline__ UnitPos unit_pos(const Task* T, int u) {
  const int lu = u - T->unit_begin, tiles = T->tiles_m * T->tiles_n;
  UnitPos q;
  q.sp = lu / tiles;
  const int t = lu - q.sp * tiles;
  q.tm = t / T->tiles_n;
  q.tn = t - q.tm * T->tiles_n;
  return q;
}

__global__ void __launch_bounds__(THREADS, 1)
gemm_list_kernel(const Task* __restrict__ tasks, const int total_units, unsigned* counters, uint32_t* status) {
  constexpr int TILE_M = 2 * BM;
  const uint32_t rank = cluster_ctarank();
  const bool leader_cta = rank == 0;
  const int unit0 = (int)(blockIdx.x >> 1);
  const int unit_step = (int)(gridDim.x >> 1);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - raw);
  const uint32_t epi_base = base + LSTAGES * LSTAGE_BYTES;      // [group][buffer set][EPI_CHUNK_BYTES]
  const uint32_t bars = epi_base + LEPI_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (LSTAGES + s); };
  auto acc_full_bar = [&](int s) { return bars + 8u * (2 * LSTAGES + s); };
  auto acc_empty_bar = [&](int s) { return bars + 8u * (2 * LSTAGES + 2 + s); };
  auto in_full_bar = [&](int g, int b) { return bars + 8u * (2 * LSTAGES + 4 + g * EPI_SETS + b); };
  auto out_ready_bar = [&](int g, int b) { return bars + 8u * (2 * LSTAGES + 4 + (EPI_GROUPS + g) * EPI_SETS + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(
      gen_base + LSTAGES * LSTAGE_BYTES + LEPI_BYTES + 8 * (2 * LSTAGES + 4 + 2 * EPI_GROUPS * EPI_SETS));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < LSTAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 16); }
    for (int g = 0; g < EPI_GROUPS; ++g)
      for (int b = 0; b < EPI_SETS; ++b) { mbar_init(in_full_bar(g, b), 1); mbar_init(out_ready_bar(g, b), 128); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t fills[LSTAGES];
#pragma unroll
      for (int s = 0; s < LSTAGES; ++s) fills[s] = 0;
      int stage = 0, ti = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = unit0; u < total_units && ok; u += unit_step) {
        const Task* T = find_task(tasks, ti, u);
        const UnitPos q = unit_pos(T, u);
        const int m0 = q.tm * TILE_M + (int)rank * BM, n0 = q.tn * LBN;
        const int kb0 = q.sp * T->kb_per_split;
        const int kb1 = min(T->kb_total, kb0 + T->kb_per_split);
        const int kb_per_seg = T->kb_per_seg, b_k_seg_stride = T->b_k_seg_stride;
        const bool a_mn = T->kind == kWgrad, b_mn = T->kind != kDgrad;
        const int b_mn_seg_stride = T->b_mn_seg_stride;
        int seg = kb0 / kb_per_seg, kk = (kb0 - seg * kb_per_seg) * BK;
        int bn = T->b_mn_wrap > 0 ? n0 % T->b_mn_wrap : n0;
        bn += (int)rank * LBNH;
        // the operand rows must have been stored (and be visible to the TMA unit) before they are fetched
        ok = dep_wait(counters, T->wait_base, T->wait_per_row ? q.tm : 0, T->wait_target, abort_flag, status);
        if (!ok) break;
        fence_proxy_async_all();
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, status, kTimeoutProducer);
          if (!ok) break;
          const uint32_t sa = base + stage * LSTAGE_BYTES, sb = sa + A_STAGE_BYTES;
          const uint32_t bar = full_bar(stage);
          if (leader_cta) mbar_expect_tx(bar, 2u * LSTAGE_BYTES);
          const int bk = kk + seg * b_k_seg_stride;
          const int bnk = bn + seg * b_mn_seg_stride;
          if (!a_mn) tma_load_2d_pair(sa, &T->map_a, bar, kk, m0);
          else tma_load_3d_pair(sa, &T->map_a, bar, 0, kk, m0 >> 6);
          if (!b_mn) tma_load_2d_pair(sb, &T->map_b, bar, bk, bnk);
          else tma_load_3d_pair(sb, &T->map_b, bar, 0, bk, bnk >> 6);
          ++fills[stage];
          if (++stage == LSTAGES) { stage = 0; phase ^= 1u; }
          kk += BK;
          if (kk == kb_per_seg * BK) { kk = 0; ++seg; }
        }
      }
      if (!ok) {
        if (leader_cta) {
#pragma unroll
          for (int s = 0; s < LSTAGES; ++s) {
            if (fills[s] == 0) continue;
            const uint32_t par = (fills[s] - 1u) & 1u;
            bool landed = false;
            for (uint32_t it = 0; it < (1u << 20) && !landed; ++it) landed = mbar_try_wait(full_bar(s), par);
            if (!landed) atomicCAS(status, 0u, (uint32_t)kTimeoutDrain);
          }
        } else {
          for (int it = 0; it < 2000; ++it) __nanosleep(1000);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && leader_cta) {
      int stage = 0, ti = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = unit0; u < total_units && ok; u += unit_step) {
        const Task* T = find_task(tasks, ti, u);
        const UnitPos q = unit_pos(T, u);
        const int kb0 = q.sp * T->kb_per_split;
        const int kb1 = min(T->kb_total, kb0 + T->kb_per_split);
        const bool a_mn = T->kind == kWgrad, b_mn = T->kind != kDgrad;
        const uint32_t idesc = make_idesc<TILE_M, LBN, false, false>() | (a_mn ? (1u << 15) : 0u) | (b_mn ? (1u << 16) : 0u);
        const uint64_t desc_a0 = a_mn ? make_desc(base, CHUNK_BYTES, 1024) : make_desc(base, 16, 1024);
        const uint64_t desc_b0 = b_mn ? make_desc(base + A_STAGE_BYTES, CHUNK_BYTES, 1024)
                                      : make_desc(base + A_STAGE_BYTES, 16, 1024);
        const uint32_t step_a = (a_mn ? 2048u : 32u) >> 4, step_b = (b_mn ? 2048u : 32u) >> 4;
        ok = mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, status, kTimeoutMma);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_STRIDE);
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, abort_flag, status, kTimeoutMma);
          if (!ok) break;
          tc_fence_after();
          const uint64_t da = desc_a0 + (uint64_t)((uint32_t)stage * (LSTAGE_BYTES >> 4));
          const uint64_t db = desc_b0 + (uint64_t)((uint32_t)stage * (LSTAGE_BYTES >> 4));
#pragma unroll
          for (int k = 0; k < BK / UK; ++k)
            tc_mma_pair(d_tmem, da + k * step_a, db + k * step_b, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          tc_commit_pair(empty_bar(stage));
          if (++stage == LSTAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(acc_full_bar(acc));
        if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 2 + 4 * EPI_GROUPS) {
    // ------------------------------------------------------------------ epilogue TMA thread of group g
    const int g = warp - (2 + 4 * EPI_GROUPS);
    if (lane == 0 && g < EPI_GROUPS) {
      // Walks the units with a staged epilogue (kDgrad, kFwd) of this CTA in list order, twice: once ahead,
      // requesting the input chunks, once behind, storing finished chunks and signalling finished units.  Neither
      // walk ever blocks the other: a request whose dependency is not met yet is simply retried on the next
      // round.  What moves through a buffer set is an "entry": one per 64-column chunk, or two (Z, then the
      // output) for a forward layer with an activation.
      struct Walk {
        int u, ti;
        bool valid;
        const Task* T;
        int tm, m0, n0, nch, k, ent;  // row tile, first row / column, entries of this group in the unit, entries done, entries per chunk
      };
      auto enter = [&](Walk& w) {      // position w on the staged-epilogue unit at or after w.u
        w.valid = false;
        while (w.u < total_units) {
          const Task* T = find_task(tasks, w.ti, w.u);
          if (T->kind != kWgrad) {
            const UnitPos q = unit_pos(T, w.u);
            w.T = T; w.tm = q.tm;
            w.m0 = q.tm * TILE_M + (int)rank * BM; w.n0 = q.tn * LBN;
            w.ent = T->kind == kFwd ? T->entries : 1;
            w.nch = 0;
            for (int c = g; c < LNCHUNK; c += EPI_GROUPS) w.nch += (w.n0 + c * 64 < T->cols) ? w.ent : 0;
            w.k = 0; w.valid = true;
            return;
          }
          w.u += unit_step;
        }
      };
      Walk fw{unit0, 0, false, nullptr, 0, 0, 0, 0, 0, 1}, sw = fw;
      enter(fw);
      enter(sw);
      int fetched = 0, stored = 0;
      uint32_t idle = 0;
      bool ok = true;
      while (true) {
        // units whose chunks have all been stored (or that have none for this group): signal, move on
        while (sw.valid && sw.k == sw.nch) {
          if (sw.T->signal_base >= 0) {
            tma_store_wait_all();            // this thread's stores so far are complete
            fence_proxy_async_all();
            __threadfence();
            atomicAdd(counters + sw.T->signal_base + sw.tm, 1u);
            atomicAdd(counters + sw.T->signal_base + sw.T->tiles_m, 1u);
          }
          sw.u += unit_step;
          enter(sw);
        }
        if (!sw.valid) break;
        bool progress = false;
        while (fetched < stored + EPI_SETS) {
          while (fw.valid && fw.k == fw.nch) { fw.u += unit_step; enter(fw); }
          if (!fw.valid) break;
          const Task* T = fw.T;
          const int b = fetched & 1;
          const uint32_t bar = in_full_bar(g, b);
          if (T->has_in) {
            if (!dep_ready(counters, T->wait_base, T->wait_per_row ? fw.tm : 0, T->wait_target) ||
                !dep_ready(counters, T->wait2_base, fw.tm, T->wait2_target))
              break;
            fence_proxy_async_all();
            mbar_expect_tx(bar, EPI_CHUNK_BYTES);
            const uint32_t dst = epi_base + (uint32_t)((g * EPI_SETS + b) * EPI_CHUNK_BYTES);
            tma_load_2d(dst, &T->map_in, bar, fw.n0 + (g + EPI_GROUPS * (fw.k / fw.ent)) * 64, fw.m0);
          } else {
            mbar_arrive(bar);
          }
          ++fw.k; ++fetched;
          progress = true;
        }
        if (mbar_try_wait(out_ready_bar(g, stored & 1), (uint32_t)(stored >> 1) & 1u)) {
          if (sw.m0 < sw.T->rows) {
            const uint32_t src = epi_base + (uint32_t)((g * EPI_SETS + (stored & 1)) * EPI_CHUNK_BYTES);
            const CUtensorMap* om = (sw.ent == 2 && (sw.k & 1) == 0) ? &sw.T->map_out2 : &sw.T->map_out;
            tma_store_2d(om, src, sw.n0 + (g + EPI_GROUPS * (sw.k / sw.ent)) * 64, sw.m0);
          }
          tma_store_commit();
          tma_store_wait_read<0>();
          ++sw.k; ++stored;
          progress = true;
        }
        if (progress) { idle = 0; continue; }
        if ((++idle & 1023u) == 0u) {
          if (*abort_flag != 0 || *reinterpret_cast<volatile uint32_t*>(status) != 0) { ok = false; break; }
          if (idle >= (1u << 24)) {
            *abort_flag = 1;
            atomicCAS(status, 0u, (uint32_t)kTimeoutEpiTma);
            ok = false;
            break;
          }
        }
      }
      tma_store_wait_all();
      if (!ok) {
        for (int f = max(stored, fetched - EPI_SETS); f < fetched; ++f) {
          bool landed = false;
          for (uint32_t it = 0; it < (1u << 20) && !landed; ++it)
            landed = mbar_try_wait(in_full_bar(g, f & 1), (uint32_t)(f >> 1) & 1u);
          if (!landed) atomicCAS(status, 0u, (uint32_t)kTimeoutDrain);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 2..9
    const int g = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int trow = quad * 32 + lane;
    int acc = 0, ti = 0;
    uint32_t acc_phase = 0;
    int j = 0;
    bool ok = true;
    for (int u = unit0; u < total_units && ok; u += unit_step) {
      const Task* T = find_task(tasks, ti, u);
      const UnitPos q = unit_pos(T, u);
      const int m0 = q.tm * TILE_M + (int)rank * BM, n0 = q.tn * LBN;
      const int rows = T->rows, cols = T->cols;
      ok = mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, status, kTimeoutEpilogue);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * ACC_STRIDE);
      if (T->kind == kWgrad) {
        PartialEpi epi;
        epi.base = T->partial; epi.split_stride = (size_t)T->split_stride; epi.ld = T->ld_out; epi.split = q.sp;
        const int row = m0 + trow;
#pragma unroll 1
        for (int c = g; c < LNCHUNK; c += EPI_GROUPS) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float v[32];
            tmem_ld32(taddr + c * 64 + h * 32, v);
            const int col0 = n0 + c * 64 + h * 32;
            const int nv = cols - col0;
            if (row < rows && nv > 0) epi.template operator()<32>(row, col0, nv, v);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(acc_empty_bar(acc), 0u);
      } else if (T->kind == kFwd) {
        // Z = acc + bias; with an activation two entries per chunk: Z into buffer set j, a_{l+1} into set j + 1
        FwdEpiS<2> epi;
        epi.has_in[0] = T->has_in != 0; epi.has_in[1] = false; epi.has_out[0] = true; epi.has_out[1] = T->entries == 2;
        epi.bias = T->bias; epi.fold = T->fold; epi.ld = T->ld; epi.act = T->act;
        const int ent = T->entries;
        int nch = 0;
#pragma unroll
        for (int c = 0; c < LNCHUNK; ++c) nch += ((c & 1) == g && n0 + c * 64 < cols) ? 1 : 0;
        if (nch == 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(acc_empty_bar(acc), 0u);
        }
#pragma unroll 1
        for (int i = 0; i < nch; ++i, j += ent) {
          const int c = g + 2 * i;
          const int col0 = n0 + c * 64;
          const int bz = j & 1, bo = (j + ent - 1) & 1;          // buffer sets of Z (if stored) and of the output
          ok = mbar_wait(in_full_bar(g, bz), (uint32_t)(j >> 1) & 1u, abort_flag, status, kTimeoutEpilogue);
          if (ok && ent == 2)
            ok = mbar_wait(in_full_bar(g, bo), (uint32_t)((j + 1) >> 1) & 1u, abort_flag, status, kTimeoutEpilogue);
          if (!ok) break;
          uint8_t* bufz = gen_base + LSTAGES * LSTAGE_BYTES + (g * EPI_SETS + bz) * EPI_CHUNK_BYTES;
          uint8_t* bufo = gen_base + LSTAGES * LSTAGE_BYTES + (g * EPI_SETS + bo) * EPI_CHUNK_BYTES;
#pragma unroll 1
          for (int h = 0; h < 2; ++h) {                          // 32 columns at a time keeps the register count down
            float v[32], s0[32], s1[32];
            tmem_ld32(taddr + c * 64 + h * 32, v);
            if (i == nch - 1 && h == 1) {                        // last read of this accumulator by this warp
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive_remote(acc_empty_bar(acc), 0u);
            }
            if (epi.has_in[0]) lds_row32(bufo, trow, h, s0);
            epi.combine(col0 + h * 32, cols - (col0 + h * 32), v, s0, s1);
            if (ent == 2) sts_row32(bufz, trow, h, s1);
            sts_row32(bufo, trow, h, s0);
          }
          fence_async_smem();
          mbar_arrive(out_ready_bar(g, bz));
          if (ent == 2) mbar_arrive(out_ready_bar(g, bo));
        }
      } else {
        DgradEpiS<1> epi;
        epi.has_in[0] = T->has_in != 0; epi.has_in[1] = false; epi.has_out[0] = true; epi.has_out[1] = false;
        epi.mul_act = T->mul_act != 0; epi.act_prev = T->act_prev; epi.colsum = T->colsum; epi.ld = T->ld;
        int nch = 0;
#pragma unroll
        for (int c = 0; c < LNCHUNK; ++c) nch += ((c & 1) == g && n0 + c * 64 < cols) ? 1 : 0;
        if (nch == 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(acc_empty_bar(acc), 0u);
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
          if (i == nch - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(acc_empty_bar(acc), 0u);
          }
          ok = mbar_wait(in_full_bar(g, b), (uint32_t)(j >> 1) & 1u, abort_flag, status, kTimeoutEpilogue);
          if (!ok) break;
          uint8_t* buf = gen_base + LSTAGES * LSTAGE_BYTES + (g * EPI_SETS + b) * EPI_CHUNK_BYTES;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float (&v)[32] = h == 0 ? v0 : v1;
            float s0[32], s1[32];
            if (epi.has_in[0]) lds_row32(buf, trow, h, s0);
            epi.combine(col0 + h * 32, cols - (col0 + h * 32), v, s0, s1);
            sts_row32(buf, trow, h, s0);
            epi.column_sums((m0 >> 5) + quad, col0 + h * 32, cols - (col0 + h * 32), s0, s1, lane);
          }
          fence_async_smem();
          mbar_arrive(out_ready_bar(g, b));
        }
      }
      if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tl
}  // namespace et
