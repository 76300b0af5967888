// Host side of the C ABI declared in et.h: stack object, workspace layout, execution plan
// from the selection mask, kernel launches.  No device memory is allocated here.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "et.h"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_list.cuh"
#include "kernels.cuh"
#include "norm.cuh"
#include "attn.cuh"
#include "im2col.cuh"
#include "batchnorm.cuh"

namespace {

thread_local int g_last_cuda = 0;
std::atomic<long long> g_launches{0};
std::atomic<int> g_guard_regions{0};      // et_debug_guard_regions: stacks created from now on get guard words
constexpr size_t kGuardBytes = 256;
constexpr unsigned char kGuardByte = 0xA5;

#define CU_TRY(expr)                                   \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) {                          \
      g_last_cuda = (int)e__;                          \
      return ET_ERR_CUDA;                              \
    }                                                  \
  } while (0)
#define ET_TRY(expr)                                   \
  do {                                                 \
    et_status s__ = (expr);                            \
    if (s__ != ET_OK) return s__;                      \
  } while (0)

inline et_status after_launch() {
  CU_TRY(cudaGetLastError());
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return ET_OK;
}
inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }
inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// ---- TMA descriptors ---------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn lookup_encode_fn() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return (EncodeTiledFn)p;
  (void)cudaGetLastError();
  return nullptr;
}
EncodeTiledFn get_encode_fn() {
  static const EncodeTiledFn fn = lookup_encode_fn();     // initialised once, thread-safe
  return fn;
}
// Guards the per-device caches of kernel attributes and occupancy answers below: stacks may be driven
// from several host threads.
std::mutex g_cache_mutex;
// Row-major bf16 matrix [outer x inner]: box of 64 columns x box_rows rows, 128-byte swizzle,
// zero fill outside.
et_status make_map(CUtensorMap* m, const void* ptr, int inner, long long outer, int box_rows = 64) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return ET_ERR_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda = (int)cudaErrorInvalidValue;
    return ET_ERR_CUDA;
  }
  return ET_OK;
}
// The same matrix seen as [inner/64 chunks][outer][64]: one box = `depth` chunks of 64 columns x
// 64 rows, which is how an MN-major operand tile lies in shared memory.  inner % 64 == 0.
et_status make_map3(CUtensorMap* m, const void* ptr, int inner, long long outer, int depth) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return ET_ERR_CUDA;
  cuuint64_t dims[3] = {64, (cuuint64_t)outer, (cuuint64_t)(inner / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)inner * 2, 128};
  cuuint32_t box[3] = {64, 64, (cuuint32_t)depth};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda = (int)cudaErrorInvalidValue;
    return ET_ERR_CUDA;
  }
  return ET_OK;
}
// NHWC bf16 tensor [images x height x width x channels] for TMA's im2col mode: a load fetches `pixels`
// consecutive base pixels (w fastest, then h, then image) x 64 channels, each pixel read at a tap offset in
// [0, ksize) from its base; base pixels range over [-pad, extent - pad) (stride 1, zero padding ksize / 2), and
// whatever falls outside the image reads as zero.
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeIm2colFn lookup_im2col_fn() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return (EncodeIm2colFn)p;
  (void)cudaGetLastError();
  return nullptr;
}
et_status make_im2col_map(CUtensorMap* m, const void* ptr, int channels, int width, int height, long long images, int ksize,
                          int pixels) {
  static const EncodeIm2colFn fn = lookup_im2col_fn();
  if (fn == nullptr) return ET_ERR_CUDA;
  const int pad = ksize / 2;
  cuuint64_t dims[4] = {(cuuint64_t)channels, (cuuint64_t)width, (cuuint64_t)height, (cuuint64_t)images};
  cuuint64_t strides[3] = {(cuuint64_t)channels * 2, (cuuint64_t)channels * 2 * width, (cuuint64_t)channels * 2 * width * height};
  int lower[2] = {-pad, -pad};
  int upper[2] = {pad - (ksize - 1), pad - (ksize - 1)};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, lower, upper, 64,
                  (cuuint32_t)pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda = (int)cudaErrorInvalidValue;
    return ET_ERR_CUDA;
  }
  return ET_OK;
}
// All the views of one bf16 activation / gradient / weight matrix that the GEMMs use.
struct TMaps {
  CUtensorMap b64;     // 64 x 64 boxes: MN-major operand fetched chunk by chunk
  CUtensorMap b128;    // 64 columns x 128 rows: K-major A tile, epilogue chunks
  CUtensorMap c3[2];   // 3-D, depth 2 and 4: MN-major operand tile in one copy (width % 64 == 0)
  bool has3 = false;
};
et_status make_tmaps(TMaps* t, const void* ptr, int inner, long long outer) {
  ET_TRY(make_map(&t->b64, ptr, inner, outer, 64));
  ET_TRY(make_map(&t->b128, ptr, inner, outer, 128));
  t->has3 = inner % 64 == 0;
  if (t->has3) {
    ET_TRY(make_map3(&t->c3[0], ptr, inner, outer, 2));
    ET_TRY(make_map3(&t->c3[1], ptr, inner, outer, 4));
  }
  return ET_OK;
}
// MN-major operand of `chunks` 64-wide chunks: the 3-D view if there is one, else the 64 x 64 view.
const CUtensorMap& mn_map(const TMaps& t, int chunks, int* use3d) {
  if (t.has3 && (chunks == 2 || chunks == 4)) { *use3d = 1; return t.c3[chunks == 2 ? 0 : 1]; }
  *use3d = 0;
  return t.b64;
}

struct LayerRT {
  int K = 0, N = 0, Nw = 0, fold = 1, act = 0, residual_src = -1;
  int kind = ET_LAYER_DENSE;     // ET_LAYER_NORM: K = N = Nw = features, W = gamma, b = beta
  float eps = 0.f;
  size_t off_stats = 0;     // norm: (mean, rstd) per row
  size_t off_gpart = 0;     // norm: per-block partial column sums of g * xhat
  int norm_blocks = 0;      // norm: blocks of the backward kernel = rows of off_gpart
  int heads = 0, seq = 0;   // attention: K = 3N, N = 64 * heads, rows in sequences of `seq`
  size_t off_lse = 0;       // attention: log-sum-exp per (sequence, head, row)
  int consumer = -1;        // layer whose residual reads a_l (its output gradient joins G_l), or -1
  void* W = nullptr;
  void* b = nullptr;
  float* W32 = nullptr;     // optional fp32 master copies (et_stack_bind_master)
  float* b32 = nullptr;
  float* st1[2] = {nullptr, nullptr};   // optimiser state of kernel / bias: first moment (momentum)
  float* st2[2] = {nullptr, nullptr};   // second moment (Adam)
  size_t off_a_out = 0;     // a_{l+1}           (unused for the last layer: that is the caller's y)
  size_t off_Z = 0;         // Z_l               (act != none)
  size_t off_G_out = 0;     // G_{l+1}           (unused for the last layer: that is the caller's dY)
  size_t off_dZ = 0;        // dZ_l              (act != none)
  size_t off_biaspart = 0;  // column partials of dZ_l for the bias gradient (own buffer per layer, so
                            // that finishing a bias never has to be ordered against later GEMMs)
  int split = 1;            // wgrad contraction splits
  int split_shared = 1;     // the same while the error-gradient chain runs beside the weight gradients (dense masks)
  int bn_fwd = 256, bn_dgrad = 256, bn_wgrad = 256;   // tile widths chosen per GEMM
  bool pair_fwd = false, pair_dgrad = false, pair_wgrad = false;   // CTA-pair (cta_group::2) tiles
  int bn_dgrad_sh = 256; bool pair_dgrad_sh = false;   // dgrad tiles while the two streams share the GPU
  bool big_gemm = false;    // its GEMMs run for tens of microseconds (10 GFLOP and more)
  int imp_count_w = 0, imp_count_b = 0;
  int img_h = 0, img_w = 0, ksize = 0;   // patch gather: K = channels, N = ksize^2 * K
  bool trainable() const { return kind == ET_LAYER_DENSE || kind == ET_LAYER_NORM || kind == ET_LAYER_BATCHNORM; }
  bool vector_params() const { return kind == ET_LAYER_NORM || kind == ET_LAYER_BATCHNORM; }   // gamma, beta: [N]
  size_t off_means = 0;     // batch norm: the two column means of the backward formula
  size_t w_count() const { return !trainable() ? 0 : vector_params() ? (size_t)N : (size_t)K * N; }   // elements of tensor 2l
  // bf16 stacks: one TMA descriptor per tensor (the caller's x, y and dY get theirs per call)
  TMaps map_W, map_aout, map_Gout, map_Z, map_dZ;
  CUtensorMap map_Wd;       // W as the K-major B of the dgrad GEMM: one box = the CTA's whole B tile
  CUtensorMap map_Wd_sh;    // the same for the shared-GPU tile shape
  CUtensorMap map_Wd_list;  // the same for the 256-wide pair tiles of the one-launch backward (128-row boxes)
  int split_list = 1;       // wgrad contraction splits in the one-launch backward
  size_t off_partial_list = 0;   // this layer's own split partials there (kept until the grouped reducer runs)
  bool list_ok = false;     // shapes the one-launch backward takes (bf16 dense layer, widths multiples of 64)
  // Patch gather whose gathered matrix is never formed: the three GEMMs of the dense layer above fetch the
  // patches themselves (TMA im2col mode).  Set on the gather layer.
  bool implicit = false;
  CUtensorMap im_fwd, im_wg, im_dg;          // im2col views: input (128 / 64 pixels per load), dZ of the layer above
  const void* im_in_ptr = nullptr;           // what im_fwd / im_wg were made for
  const void* im_dg_ptr = nullptr;           // what im_dg was made for
  CUtensorMap map_Wd_conv;                   // on the dense layer above: W as K-major B in 128-row boxes
  int split_now = 1;        // per task list: splits of this layer's weight-gradient task
};

}  // namespace

struct et_stack {
  int L = 0;
  long long M = 0;
  et_dtype dtype = ET_F32;
  size_t elt = 4;
  int sms = 148;
  std::vector<LayerRT> ly;
  std::vector<int> imp_offs, imp_counts;
  size_t ws_bytes = 0;
  std::vector<size_t> guards;          // offsets of the guard words that follow each workspace region (debug aid)
  size_t off_status = 0, off_partial = 0, off_imp_parts = 0, off_imp_offs = 0,
         off_imp_counts = 0, off_loss_parts = 0, off_dy_stage = 0, off_imp_stage = 0;
  int imp_total = 0;
  char* ws = nullptr;
  bool bound = false, forwarded = false;
  const void* x = nullptr;
  TMaps map_x, map_y, map_dy;
  const void* map_dy_ptr = nullptr;
  const void* map_y_ptr = nullptr;
  et_optimizer_config opt_cfg = {ET_OPT_SGD, 0.f, 0.f, 0.f, 0.f, 0.f};
  int opt_step = 1;                    // Adam's t (1-based)
  float opt_wd_now = 0.f;              // this step's (scheduled) decoupled weight decay
  bool delta_is_snapshot = false;      // per call: the delta tensors hold a weight snapshot
  bool wgrad_one_unit = false;         // per call: weight-gradient CTAs take one unit each and leave
  bool overlap_launch = true;          // forward / dgrad kernels start their prologue under the previous kernel's tail
  bool chain_shares_gpu = false;       // per call: weight gradients run beside the error-gradient chain
  bool shared_plan = false;            // per call: the GEMMs use the tile plan made for that case
  bool opt_two_streams = true;         // et_stack_set_option
  int opt_tile_plan = ET_TILE_PLAN_AUTO;
  bool opt_gemm_list = true;
  bool opt_list_cooperative = true;
  // one-launch backward: task list, dependency counters and the grouped reducers' tables (device, in the
  // workspace) with the host copies they were last filled from
  size_t off_tasks = 0, off_counters = 0, off_rtab = 0, off_btab = 0;
  int max_counters = 0;
  std::vector<et::tl::Task> tasks_host;
  std::vector<uint8_t> tasks_key;      // mask and pointers the device task list was built for
  int tasks_units = 0, tasks_counters = 0;
  size_t off_ftasks = 0;               // the forward pass's task list
  std::vector<et::tl::Task> ftasks_host;
  std::vector<uint8_t> ftasks_key;
  int ftasks_units = 0, ftasks_counters = 0;
  std::vector<et::ReduceEntry> rtab_host;
  std::vector<et::BiasEntry> btab_host;
  int list_state = 0;                  // 0 = untried, 1 = works, -1 = the cooperative launch was refused: per-layer path
  unsigned bind_serial = 0;
  // second stream: the error-gradient chain runs here while weight gradients run on the caller's
  cudaStream_t chain_stream = nullptr;
  std::vector<cudaEvent_t> chain_ev;   // [l] = dgrad(l) finished; [L] = top-layer dZ ready; [L+1] = join
  cudaEvent_t fork_ev = nullptr;
  int two_streams = -1;                // -1 = not set up yet, 0 = off, 1 = on
  // optional per-kernel timing
  bool timing = false;
  struct Timed { int cls; cudaEvent_t e0, e1; };
  std::vector<Timed> timed;            // recorded this period
  std::vector<cudaEvent_t> event_pool; // spare events

  char* at(size_t off) const { return ws + off; }
  int width_in(int l) const { return ly[l].K; }
  int out_width() const { return ly[L - 1].Nw; }
};

namespace {

using et::bf16;

// Tile shape and contraction split of one GEMM.  Model: an SM spends, per 64-deep k-block of
// its tile, the larger of the tensor-pipe time and the time to pull the operands from L2
// (about 10.5 TB/s over all SMs, measured with this kernel); a unit costs (k-blocks + a fixed
// prologue/epilogue allowance) of those; the GEMM takes as many unit times as the busiest SM
// gets units.  A CTA pair (cta_group::2) loads half of B per CTA and so moves fewer L2 bytes per
// flop; a 192-wide pair tile needs 32-row B boxes and therefore a K-major B (dgrad only).
struct TilePlan { int bn; int split; bool pair; };
// fractional: the GEMM shares the GPU with another stream's work, which fills the SMs a partly filled
// last wave leaves idle, so the cost is the work itself (fractional waves), not whole waves.
TilePlan choose_tiles(int rows, int cols, int kb_total, int sms, bool allow_split, bool b_k_major, int n_multiple,
                      bool fractional = false) {
  TilePlan best{256, 1, false};
  double best_cost = -1.0;
  const double sm_flops = 10.5e12, sm_l2_bytes = 10.5e12 / 148.0;
  for (int pair = 0; pair < 2; ++pair) {
    for (int bn : {256, 192, 128}) {
      if (pair && bn == 192 && !b_k_major) continue;
      if (n_multiple > 0 && n_multiple % bn != 0) continue;          // a folded wgrad tile must not straddle slices
      const int tile_m = pair ? 256 : 128;
      const long long tiles = (long long)ceil_div(rows, tile_m) * ceil_div(cols, bn);
      const int workers = pair ? sms / 2 : sms;
      const double flops = 2.0 * 128 * bn * 64;                      // per CTA per k-block
      const double bytes = 128.0 * 128 + (pair ? bn / 2 : bn) * 128.0;
      const double kb_time = std::max(flops / sm_flops, bytes / sm_l2_bytes);
      const int smax = allow_split ? std::min(16, kb_total) : 1;
      for (int sp = 1; sp <= smax; ++sp) {
        const int kbs = ceil_div(kb_total, sp);
        if ((long long)(sp - 1) * kbs >= kb_total) continue;         // an empty split
        const double waves = fractional ? std::max(1.0, (double)(tiles * sp) / workers) : (double)ceil_div(tiles * sp, workers);
        const double cost = waves * (kbs + 6) * kb_time;
        if (best_cost < 0 || cost < best_cost * 0.999) { best_cost = cost; best = {bn, sp, pair != 0}; }
      }
    }
  }
  return best;
}

// ---- per-kernel timing: an event pair around one launch ---------------------------------------
cudaEvent_t take_event(et_stack* s) {
  cudaEvent_t e = nullptr;
  if (!s->event_pool.empty()) { e = s->event_pool.back(); s->event_pool.pop_back(); return e; }
  if (cudaEventCreate(&e) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
  return e;
}
struct TimedLaunch {
  et_stack* s; cudaStream_t st; cudaEvent_t e0 = nullptr, e1 = nullptr; int cls;
  TimedLaunch(et_stack* s_, int cls_, cudaStream_t st_) : s(s_), st(st_), cls(cls_) {
    if (!s->timing) return;
    e0 = take_event(s); e1 = take_event(s);
    if (e0 != nullptr) cudaEventRecord(e0, st);
  }
  ~TimedLaunch() {
    if (e0 == nullptr || e1 == nullptr) return;
    cudaEventRecord(e1, st);
    s->timed.push_back({cls, e0, e1});
  }
};

template <typename T> struct is_bf16 : std::false_type {};
template <> struct is_bf16<bf16> : std::true_type {};

// ---- pointer helpers -----------------------------------------------------------------------
template <typename T> const T* act_in(const et_stack* s, int l) {       // a_l
  return l == 0 ? (const T*)s->x : (const T*)s->at(s->ly[l - 1].off_a_out);
}
template <typename T> T* grad_act(const et_stack* s, int i, const void* dY) {   // G_i = dL/da_i, i >= 1
  return i == s->L ? (T*)const_cast<void*>(dY) : (T*)s->at(s->ly[i - 1].off_G_out);
}
template <typename T> const T* dz_src(const et_stack* s, int l, const void* dY) {   // dZ_l (width Nw)
  const LayerRT& y = s->ly[l];
  return y.act != ET_ACT_NONE ? (const T*)s->at(y.off_dZ) : grad_act<T>(s, l + 1, dY);
}
const TMaps& a_map(const et_stack* s, int l) { return l == 0 ? s->map_x : s->ly[l - 1].map_aout; }   // a_l
const TMaps& g_map(const et_stack* s, int i) { return i == s->L ? s->map_dy : s->ly[i - 1].map_Gout; }  // G_i
const TMaps& dz_map(const et_stack* s, int l) {                                                         // dZ_l
  return s->ly[l].act != ET_ACT_NONE ? s->ly[l].map_dZ : g_map(s, l + 1);
}

// ---- GEMM launches ---------------------------------------------------------------------------
template <int BN, bool A_MN, bool B_MN, bool PAIR, class Epi>
et_status launch_tc_bn(const CUtensorMap& ma, const CUtensorMap& mb, const et::tc::EpiMaps& em, et::tc::Params p,
                       const Epi& epi, int sms, cudaStream_t st, bool one_unit, bool overlap_prev) {
  auto kern = et::tc::gemm_tc_kernel<BN, A_MN, B_MN, Epi, PAIR>;
  using C = et::tc::Cfg<BN, Epi::kSlots, PAIR>;
  // function attributes and occupancy are per device
  static bool attr_done_dev[64] = {};
  static int max_clusters_dev[64] = {};
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return ET_ERR_UNSUPPORTED;
  std::unique_lock<std::mutex> cache_lock(g_cache_mutex);
  bool& attr_done = attr_done_dev[dev];
  int& max_clusters_ref = max_clusters_dev[dev];
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(et::tc::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cfg.attrs = attr;
  if (PAIR) {
    attr[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
    attr[cfg.numAttrs].val.clusterDim.x = 2; attr[cfg.numAttrs].val.clusterDim.y = 1;
    attr[cfg.numAttrs].val.clusterDim.z = 1;
    ++cfg.numAttrs;
  }
  const unsigned n_plain_attrs = cfg.numAttrs;
  if (overlap_prev) {
    // the kernel's prologue may start while the stream's previous kernel drains; the kernel itself
    // waits (griddepcontrol.wait) before it touches global memory
    attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    ++cfg.numAttrs;
  }
  if (!attr_done) {
    CU_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES));
    if (PAIR) {
      cfg.gridDim = dim3(sms & ~1);
      cudaLaunchConfig_t occ = cfg;
      occ.numAttrs = n_plain_attrs;
      if (cudaOccupancyMaxActiveClusters(&max_clusters_ref, kern, &occ) != cudaSuccess || max_clusters_ref < 1) {
        (void)cudaGetLastError();
        max_clusters_ref = sms / 2;
      }
    }
    attr_done = true;
  }
  const int max_clusters = max_clusters_ref;
  cache_lock.unlock();
  p.tiles_m = ceil_div(p.rows, PAIR ? 2 * et::tc::BM : et::tc::BM);
  p.tiles_n = ceil_div(p.cols, BN);
  const int units = p.tiles_m * p.tiles_n * p.split;
  // Persistent by default; one_unit: one work unit per CTA (pair), so that its SMs go back to
  // the scheduler after every unit instead of after a whole persistent loop.
  const int workers = one_unit ? units : std::min(units, PAIR ? max_clusters : sms);
  cfg.gridDim = PAIR ? dim3(2 * workers) : dim3(workers);
  CU_TRY(cudaLaunchKernelEx(&cfg, kern, ma, mb, em, p, epi));
  return after_launch();
}
template <bool A_MN, bool B_MN, class Epi>
et_status launch_tc(int bn, bool pair, const CUtensorMap& ma, const CUtensorMap& mb, const et::tc::EpiMaps& em,
                    const et::tc::Params& p, const Epi& epi, int sms, cudaStream_t st, bool one_unit = false,
                    bool overlap_prev = false) {
  if (pair) {
    if (bn == 128) return launch_tc_bn<128, A_MN, B_MN, true>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
    if constexpr (!B_MN) {
      if (bn == 192) return launch_tc_bn<192, A_MN, B_MN, true>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
    }
    return launch_tc_bn<256, A_MN, B_MN, true>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
  }
  // staged epilogues take 64 KB of shared memory per slot: a single CTA keeps a deep enough
  // operand ring only with narrower tiles
  if constexpr (Epi::kSlots == 2) {
    return launch_tc_bn<128, A_MN, B_MN, false>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
  } else if constexpr (Epi::kSlots == 1) {
    if (bn == 128) return launch_tc_bn<128, A_MN, B_MN, false>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
    return launch_tc_bn<192, A_MN, B_MN, false>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
  } else {
    if (bn == 128) return launch_tc_bn<128, A_MN, B_MN, false>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
    if (bn == 192) return launch_tc_bn<192, A_MN, B_MN, false>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
    return launch_tc_bn<256, A_MN, B_MN, false>(ma, mb, em, p, epi, sms, st, one_unit, overlap_prev);
  }
}
template <typename T, class Epi>
et_status launch_simt(const T* A, const T* B, const et::simt::Params& p, const Epi& epi, cudaStream_t st) {
  dim3 grid(ceil_div(p.cols, et::simt::TN), ceil_div(p.rows, et::simt::TM));
  et::simt::gemm_simt_kernel<T, Epi><<<grid, et::simt::THREADS, 0, st>>>(A, B, p, epi);
  return after_launch();
}

et::tc::Params tc_params(const et_stack* s, int rows, int cols, int contraction, int fold, int split) {
  et::tc::Params p;
  p.rows = rows; p.cols = cols;
  p.tiles_m = 0; p.tiles_n = 0;        // set at launch from the tile shape
  p.split = split;
  p.kb_per_seg = ceil_div(contraction, et::tc::BK);
  p.kb_total = p.kb_per_seg * fold;
  p.kb_per_split = ceil_div(p.kb_total, split);
  p.b_k_seg_stride = 0; p.b_mn_seg_stride = 0; p.b_mn_wrap = 0;
  p.a_3d = 0; p.b_3d = 0;
  p.a_im2col = 0; p.img_w = 0; p.img_h = 0; p.ksize = 0; p.chan = 0; p.a_tap_flip = 0;
  p.status = (uint32_t*)s->at(s->off_status);
  return p;
}

// Z_l = a_l W_l + b_l, activation, fold, residual -> a_{l+1}
// The im2col views of gather layer g's input (made again when the input pointer has changed: layer 0 reads
// the caller's x).
et_status conv_input_maps(et_stack* s, int g) {
  LayerRT& G = s->ly[g];
  const void* in = g == 0 ? s->x : (const void*)s->at(s->ly[g - 1].off_a_out);
  if (G.im_in_ptr == in) return ET_OK;
  const long long images = s->M / ((long long)G.img_h * G.img_w);
  ET_TRY(make_im2col_map(&G.im_fwd, in, G.K, G.img_w, G.img_h, images, G.ksize, 128));
  ET_TRY(make_im2col_map(&G.im_wg, in, G.K, G.img_w, G.img_h, images, G.ksize, 64));
  G.im_in_ptr = in;
  return ET_OK;
}
void conv_params(et::tc::Params* p, const LayerRT& G, int mode) {
  p->a_im2col = mode; p->img_w = G.img_w; p->img_h = G.img_h; p->ksize = G.ksize; p->chan = G.K;
}

template <typename T>
et_status run_forward_layer(et_stack* s, int l, void* y, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_FORWARD, st);
  const LayerRT& L = s->ly[l];
  if constexpr (is_bf16<T>::value) {
    const bool conv = l >= 1 && s->ly[l - 1].implicit;      // A = patches of the gather layer's input, one tap per segment
    et::tc::Params p = conv ? tc_params(s, (int)s->M, L.Nw, s->ly[l - 1].K, s->ly[l - 1].ksize * s->ly[l - 1].ksize, 1)
                            : tc_params(s, (int)s->M, L.Nw, L.K, L.fold, 1);
    p.b_mn_seg_stride = L.Nw;
    if (conv) {
      ET_TRY(conv_input_maps(s, l - 1));
      conv_params(&p, s->ly[l - 1], 1);
      p.b_mn_seg_stride = 0;
      p.b_k_seg_stride = s->ly[l - 1].K;                   // W's rows are (tap, channel)
    }
    et::tc::EpiMaps em;
    const CUtensorMap& out = (l == s->L - 1 ? s->map_y : L.map_aout).b128;
    em.in[0] = L.residual_src >= 0 ? a_map(s, L.residual_src).b128 : out;
    em.out[0] = out;
    em.in[1] = out;
    em.out[1] = L.act != ET_ACT_NONE ? L.map_Z.b128 : out;
    const int bn_f = conv ? 128 : L.bn_fwd;
    const bool pair_f = conv ? false : L.pair_fwd;
    const int bnh = pair_f ? bn_f / 2 : bn_f;
    const CUtensorMap& wmap = mn_map(L.map_W, bnh / 64, &p.b_3d);
    const CUtensorMap& amap = conv ? s->ly[l - 1].im_fwd : a_map(s, l).b128;
    auto fill = [&](auto& epi) {
      epi.has_in[0] = L.residual_src >= 0; epi.has_in[1] = false;
      epi.has_out[0] = true; epi.has_out[1] = L.act != ET_ACT_NONE;
      epi.bias = (const bf16*)L.b; epi.fold = L.fold; epi.ld = L.Nw; epi.act = L.act;
    };
    if (L.act != ET_ACT_NONE) {
      et::FwdEpiS<2> epi; fill(epi);
      return launch_tc<false, true>(bn_f, pair_f, amap, wmap, em, p, epi, s->sms, st, false, s->overlap_launch);
    }
    et::FwdEpiS<1> epi; fill(epi);
    return launch_tc<false, true>(bn_f, pair_f, amap, wmap, em, p, epi, s->sms, st, false, s->overlap_launch);
  } else {
    et::FwdEpi<T> epi;
    epi.bias = (const T*)L.b;
    epi.fold = L.fold;
    epi.Z = L.act != ET_ACT_NONE ? (T*)s->at(L.off_Z) : nullptr;
    epi.act = L.act;
    epi.resid = L.residual_src >= 0 ? act_in<T>(s, L.residual_src) : nullptr;
    epi.out = l == s->L - 1 ? (T*)y : (T*)s->at(L.off_a_out);
    epi.ld = L.Nw;
    et::simt::Params p;
    p.rows = (int)s->M; p.cols = L.Nw; p.kc = L.K; p.segs = L.fold;
    p.sa_i = L.K; p.sa_k = 1;
    p.sb_k = L.N; p.sb_seg = L.Nw; p.sb_j = 1; p.b_wrap = 0;
    return launch_simt<T>(act_in<T>(s, l), (const T*)L.W, p, epi, st);
  }
}

// G_l = dZ_l W_l^T (+ skip gradient), dZ_{l-1} = G_l * act'(Z_{l-1});  l >= 1
// Row blocks of 32 that the dgrad GEMM of layer l writes fused column sums for.
int dgrad_row_blocks(const et_stack* s, int l) {
  const bool pair = s->shared_plan ? s->ly[l].pair_dgrad_sh : s->ly[l].pair_dgrad;
  const int tile_m = pair ? 2 * et::tc::BM : et::tc::BM;
  return ceil_div(s->M, tile_m) * (tile_m / 32);
}

// want_colsum: also leave the column sums of dZ_{l-1} (layer l-1's bias gradient) in the bias
// partial buffer (tensor-core path only).
template <typename T>
et_status run_dgrad_layer(et_stack* s, int l, const void* dY, cudaStream_t st, bool want_colsum = false) {
  TimedLaunch tl(s, ET_K_DGRAD, st);
  const LayerRT& L = s->ly[l];
  // Above a patch gather that is never materialised this GEMM is the convolution's error gradient: it goes
  // straight to the gather's input (layer l - 1's), reading dZ_l's patches with the kernel turned by 180 degrees.
  const bool conv = is_bf16<T>::value && s->ly[l - 1].implicit;
  const int lo = conv ? l - 1 : l;                          // G_lo is what this GEMM produces
  const LayerRT& Lc = s->ly[lo];
  const LayerRT& P = s->ly[lo - 1];
  const bool need_skip = Lc.consumer >= 0;
  const bool need_act = P.act != ET_ACT_NONE;
  const bool need_G = !need_act || P.residual_src >= 0;     // G_lo itself is read later
  if constexpr (is_bf16<T>::value) {
    et::tc::Params p = conv ? tc_params(s, (int)s->M, Lc.K, L.Nw, Lc.ksize * Lc.ksize, 1)
                            : tc_params(s, (int)s->M, L.K, L.Nw, L.fold, 1);
    p.b_k_seg_stride = L.Nw;
    if (conv) {
      LayerRT& G = s->ly[lo];
      const void* dz = dz_src<T>(s, l, dY);
      if (G.im_dg_ptr != dz) {
        ET_TRY(make_im2col_map(&G.im_dg, dz, L.Nw, G.img_w, G.img_h, s->M / ((long long)G.img_h * G.img_w), G.ksize, 128));
        G.im_dg_ptr = dz;
      }
      conv_params(&p, G, 1);
      p.a_tap_flip = 1;
      p.b_k_seg_stride = 0;
      p.b_mn_seg_stride = G.K;                              // W's rows are (tap, channel): one tap per segment
      want_colsum = false;                                  // the bias below a gather takes the column-sum kernel
    }
    et::tc::EpiMaps em;
    const CUtensorMap& gout = P.map_Gout.b128;                // G_l lives in layer l-1's buffer
    // Two tile plans: alone on the GPU whole waves count (768-wide outputs on 12608 rows: 192-wide pair
    // tiles, 200 units in 3 waves at 90 %); beside the weight-gradient stream the idle SMs of a last wave are
    // not lost, and the wider tile with less operand traffic per flop wins (256-wide: 150 units; measured on
    // the ViT-B step 2.45 -> 2.33 ms).
    const bool sh = s->shared_plan;
    const int bn_d = conv ? 128 : sh ? L.bn_dgrad_sh : L.bn_dgrad;
    const bool pair_d = conv ? false : sh ? L.pair_dgrad_sh : L.pair_dgrad;
    const CUtensorMap& wmap = conv ? L.map_Wd_conv : sh ? L.map_Wd_sh : L.map_Wd;
    const CUtensorMap& amap = conv ? s->ly[lo].im_dg : dz_map(s, l).b128;
    const int ld_out = Lc.K;
    const CUtensorMap& skip = need_skip ? g_map(s, Lc.consumer + 1).b128 : gout;
    const CUtensorMap& zmap = P.map_Z.b128;
    const CUtensorMap& dzout = P.map_dZ.b128;
    if (!need_act) {                                          // G_l = acc (+ skip)
      et::DgradEpiS<1> epi;
      epi.has_in[0] = need_skip; epi.has_in[1] = false; epi.has_out[0] = true; epi.has_out[1] = false;
      epi.mul_act = false; epi.act_prev = P.act;
      epi.colsum = want_colsum ? (float*)s->at(P.off_biaspart) : nullptr; epi.ld = ld_out;
      em.in[0] = skip; em.out[0] = gout; em.in[1] = gout; em.out[1] = gout;
      return launch_tc<false, false>(bn_d, pair_d, amap, wmap, em, p, epi, s->sms, st, false, s->overlap_launch && !s->chain_shares_gpu);
    }
    if (!need_skip && !need_G) {                              // dZ_{l-1} = acc * act'(Z_{l-1})
      et::DgradEpiS<1> epi;
      epi.has_in[0] = true; epi.has_in[1] = false; epi.has_out[0] = true; epi.has_out[1] = false;
      epi.mul_act = true; epi.act_prev = P.act;
      epi.colsum = want_colsum ? (float*)s->at(P.off_biaspart) : nullptr; epi.ld = ld_out;
      em.in[0] = zmap; em.out[0] = dzout; em.in[1] = zmap; em.out[1] = dzout;
      return launch_tc<false, false>(bn_d, pair_d, amap, wmap, em, p, epi, s->sms, st, false, s->overlap_launch && !s->chain_shares_gpu);
    }
    et::DgradEpiS<2> epi;                                     // both G_l and dZ_{l-1}
    epi.has_in[0] = need_skip; epi.has_in[1] = true; epi.has_out[0] = need_G; epi.has_out[1] = true;
    epi.mul_act = false; epi.act_prev = P.act;
    epi.colsum = want_colsum ? (float*)s->at(P.off_biaspart) : nullptr; epi.ld = ld_out;
    em.in[0] = skip; em.out[0] = gout; em.in[1] = zmap; em.out[1] = dzout;
    return launch_tc<false, false>(bn_d, pair_d, amap, wmap, em, p, epi, s->sms, st, false, s->overlap_launch && !s->chain_shares_gpu);
  } else {
    et::DgradEpi<T> epi;
    epi.skip = need_skip ? grad_act<T>(s, L.consumer + 1, dY) : nullptr;
    epi.act_prev = P.act;
    epi.ld = L.K;
    if (!need_act) {
      epi.Zprev = nullptr;
      epi.outG = (T*)s->at(P.off_G_out);
      epi.outdZ = nullptr;
    } else {
      epi.Zprev = (const T*)s->at(P.off_Z);
      epi.outdZ = (T*)s->at(P.off_dZ);
      epi.outG = need_G ? (T*)s->at(P.off_G_out) : nullptr;
    }
    et::simt::Params p;
    p.rows = (int)s->M; p.cols = L.K; p.kc = L.Nw; p.segs = L.fold;
    p.sa_i = L.Nw; p.sa_k = 1;
    p.sb_k = 1; p.sb_seg = L.Nw; p.sb_j = L.N; p.b_wrap = 0;
    return launch_simt<T>(dz_src<T>(s, l, dY), (const T*)L.W, p, epi, st);
  }
}

// Optimiser parameters of this step.  plain = true forces plain SGD (et_sgd_masked).
et::OptParams opt_params(const et_stack* s, float lr, bool plain = false) {
  et::OptParams o{};
  o.kind = plain ? et::kOptSgd : s->opt_cfg.kind;
  o.lr = lr;
  if (o.kind == et::kOptSgdw) { o.a = s->opt_cfg.momentum; o.b = s->opt_wd_now; }
  if (o.kind == et::kOptAdam) {
    o.a = s->opt_cfg.beta1; o.b = s->opt_cfg.beta2; o.eps = s->opt_cfg.eps;
    o.c1 = (float)(1.0 / (1.0 - std::pow((double)o.a, (double)s->opt_step)));
    o.c2 = (float)(1.0 / (1.0 - std::pow((double)o.b, (double)s->opt_step)));
  }
  return o;
}

// ---- normalisation layers ------------------------------------------------------------------
// Register chunks per lane for a row of `d` features: 1..4, 6 or 8 (d <= 2048).
template <typename F>
et_status norm_dispatch(int d, F&& f) {
  const int need = ceil_div(d, 256);
  if (need <= 1) return f(std::integral_constant<int, 1>());
  if (need == 2) return f(std::integral_constant<int, 2>());
  if (need == 3) return f(std::integral_constant<int, 3>());
  if (need == 4) return f(std::integral_constant<int, 4>());
  if (need <= 6) return f(std::integral_constant<int, 6>());
  if (need <= 8) return f(std::integral_constant<int, 8>());
  return ET_ERR_UNSUPPORTED;
}

// Blocks of a row kernel that fit on one SM at a time (by registers and shared memory): grids are sized
// to exactly one resident wave, so that no block starts late into a half-empty GPU.  The kernels differ
// only in template arguments (one pointer type for all), so the answer is remembered per function address.
template <class K>
int norm_blocks_per_sm(K kern) {
  struct Seen { const void* fn; int dev, per_sm; };
  static std::vector<Seen> seen;
  std::lock_guard<std::mutex> cache_lock(g_cache_mutex);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 1; }
  for (const auto& e : seen)
    if (e.fn == (const void*)kern && e.dev == dev) return e.per_sm;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, et::kNormThreads, 0) != cudaSuccess || per_sm < 1) {
    (void)cudaGetLastError();
    per_sm = 1;
  }
  seen.push_back({(const void*)kern, dev, per_sm});
  return per_sm;
}

template <typename T>
et_status run_norm_forward(et_stack* s, int l, void* y, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_NORM, st);
  const LayerRT& L = s->ly[l];
  T* out = l == s->L - 1 ? (T*)y : (T*)s->at(L.off_a_out);
  return norm_dispatch(L.N, [&](auto vpl) -> et_status {
    auto kern = et::norm_forward_kernel<T, decltype(vpl)::value>;
    const int grid = std::min(ceil_div(s->M, et::kNormWarps), s->sms * norm_blocks_per_sm(kern));
    kern<<<grid, et::kNormThreads, 0, st>>>(
        act_in<T>(s, l), (const T*)L.W, (const T*)L.b, out, (float2*)s->at(L.off_stats), (int)s->M, L.N, L.eps);
    return after_launch();
  });
}

// Backward of normalisation layer l.  want_dx: G_l (with the skip gradient) and dZ_{l-1} for the layer
// below (l >= 1); want_dgamma: the partial column sums of g * xhat, finished into the gradient of
// gamma with importance and update like a bias.
template <typename T>
et_status run_norm_backward(et_stack* s, int l, const void* dY, bool want_dx, bool want_dgamma, float* grad,
                            const T* delta, bool sgd, float lr, int* launches, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_NORM, st);
  const LayerRT& L = s->ly[l];
  if (!want_dx && !want_dgamma) return ET_OK;
  const T* skip = nullptr;
  T* G_in = nullptr;
  const T* z_prev = nullptr;
  T* dz_prev = nullptr;
  int act_prev = ET_ACT_NONE;
  if (want_dx) {
    const LayerRT& P = s->ly[l - 1];
    const bool need_act = P.act != ET_ACT_NONE;
    const bool need_G = !need_act || P.residual_src >= 0;
    if (L.consumer >= 0) skip = grad_act<T>(s, L.consumer + 1, dY);
    if (need_G) G_in = (T*)s->at(P.off_G_out);
    if (need_act) { z_prev = (const T*)s->at(P.off_Z); dz_prev = (T*)s->at(P.off_dZ); act_prev = P.act; }
  }
  float* gpart = (float*)s->at(L.off_gpart);
  int grid = 0;                       // blocks launched = rows of gpart written (at most L.norm_blocks)
  ET_TRY(norm_dispatch(L.N, [&](auto vpl) -> et_status {
    constexpr int V = decltype(vpl)::value;
    auto go = [&](auto kern) -> et_status {
      grid = std::min(L.norm_blocks, s->sms * norm_blocks_per_sm(kern));
      kern<<<grid, et::kNormThreads, 0, st>>>(dz_src<T>(s, l, dY), act_in<T>(s, l), (const float2*)s->at(L.off_stats),
                                              (const T*)L.W, skip, G_in, z_prev, dz_prev, act_prev, gpart, (int)s->M, L.N);
      return after_launch();
    };
    if (want_dx && want_dgamma) return go(et::norm_backward_kernel<T, V, true, true>);
    if (want_dx) return go(et::norm_backward_kernel<T, V, true, false>);
    return go(et::norm_backward_kernel<T, V, false, true>);
  }));
  ++*launches;
  if (!want_dgamma || (grad == nullptr && delta == nullptr && !sgd)) return ET_OK;
  float* imp = (float*)s->at(s->off_imp_parts) + s->imp_offs[2 * l];
  et::bias_finish_kernel<T><<<L.imp_count_w, dim3(et::kBiasCols, et::kBiasLanes), 0, st>>>(
      gpart, grid, L.N, L.N, grad, delta, imp, (T*)L.W, opt_params(s, lr), sgd ? 1 : 0,
      s->delta_is_snapshot ? 1 : 0, L.W32, L.st1[0], L.st2[0]);
  ++*launches;
  return after_launch();
}

// ---- batch normalisation -------------------------------------------------------------------
template <typename T>
et_status run_bn_forward(et_stack* s, int l, void* y, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_NORM, st);
  const LayerRT& L = s->ly[l];
  const int M = (int)s->M, C = L.N, chunks = L.norm_blocks;
  const T* x = act_in<T>(s, l);
  float* part = (float*)s->at(L.off_gpart);
  float2* stats = (float2*)s->at(L.off_stats);
  const dim3 grid(ceil_div(C, 256), chunks), block(32, 8);
  const float inv_m = (float)(1.0 / (double)M);
  et::bn_colstats_kernel<T, et::kBnSum><<<grid, block, 0, st>>>(x, nullptr, nullptr, M, C, part, nullptr);
  ET_TRY(after_launch());
  et::bn_finalize_kernel<<<ceil_div(C, 32), dim3(32, 32), 0, st>>>(part, nullptr, chunks, C, inv_m, L.eps, 0, stats, nullptr);
  ET_TRY(after_launch());
  et::bn_colstats_kernel<T, et::kBnCentredSquares><<<grid, block, 0, st>>>(x, nullptr, stats, M, C, part, nullptr);
  ET_TRY(after_launch());
  et::bn_finalize_kernel<<<ceil_div(C, 32), dim3(32, 32), 0, st>>>(part, nullptr, chunks, C, inv_m, L.eps, 1, stats, nullptr);
  ET_TRY(after_launch());
  T* out = l == s->L - 1 ? (T*)y : (T*)s->at(L.off_a_out);
  const long long total = (long long)M * (C / 8);
  et::bn_forward_kernel<T><<<ceil_div(total, et::kBnEltThreads), et::kBnEltThreads, 0, st>>>(
      x, (const T*)L.W, (const T*)L.b, stats, L.act != ET_ACT_NONE ? (T*)s->at(L.off_Z) : nullptr, out, L.act, s->M, C);
  return after_launch();
}
// Same contract as run_norm_backward.
template <typename T>
et_status run_bn_backward(et_stack* s, int l, const void* dY, bool want_dx, bool want_dgamma, float* grad,
                          const T* delta, bool sgd, float lr, int* launches, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_NORM, st);
  const LayerRT& L = s->ly[l];
  if (!want_dx && !want_dgamma) return ET_OK;
  const int M = (int)s->M, C = L.N, chunks = L.norm_blocks;
  const T* x = act_in<T>(s, l);
  const T* dz = dz_src<T>(s, l, dY);
  float* part0 = (float*)s->at(L.off_gpart);
  float* part1 = part0 + (size_t)chunks * C;
  const float2* stats = (const float2*)s->at(L.off_stats);
  float2* means = (float2*)s->at(L.off_means);
  et::bn_colstats_kernel<T, et::kBnBackward><<<dim3(ceil_div(C, 256), chunks), dim3(32, 8), 0, st>>>(dz, x, stats, M, C,
                                                                                                 part0, part1);
  ET_TRY(after_launch());
  ++*launches;
  if (want_dx) {
    const LayerRT& P = s->ly[l - 1];
    const bool need_act = P.act != ET_ACT_NONE;
    const bool need_G = !need_act || P.residual_src >= 0;
    et::bn_finalize_kernel<<<ceil_div(C, 32), dim3(32, 32), 0, st>>>(part0, part1, chunks, C, (float)(1.0 / (double)M),
                                                                   L.eps, 2, nullptr, means);
    ET_TRY(after_launch());
    const long long total = (long long)M * (C / 8);
    et::bn_backward_kernel<T><<<ceil_div(total, et::kBnEltThreads), et::kBnEltThreads, 0, st>>>(
        dz, x, stats, means, (const T*)L.W, L.consumer >= 0 ? grad_act<T>(s, L.consumer + 1, dY) : nullptr,
        need_G ? (T*)s->at(P.off_G_out) : nullptr, need_act ? (const T*)s->at(P.off_Z) : nullptr,
        need_act ? (T*)s->at(P.off_dZ) : nullptr, P.act, s->M, C);
    ET_TRY(after_launch());
    *launches += 2;
  }
  if (!want_dgamma || (grad == nullptr && delta == nullptr && !sgd)) return ET_OK;
  float* imp = (float*)s->at(s->off_imp_parts) + s->imp_offs[2 * l];
  et::bias_finish_kernel<T><<<L.imp_count_w, dim3(et::kBiasCols, et::kBiasLanes), 0, st>>>(
      part1, chunks, C, C, grad, delta, imp, (T*)L.W, opt_params(s, lr), sgd ? 1 : 0, s->delta_is_snapshot ? 1 : 0, L.W32,
      L.st1[0], L.st2[0]);
  ++*launches;
  return after_launch();
}

// ---- attention core --------------------------------------------------------------------------
// Dynamic shared memory above 48 KB has to be allowed per kernel and device.
et_status attn_allow_smem() {
  static bool done[64] = {};
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return ET_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> cache_lock(g_cache_mutex);
  if (!done[dev]) {
    CU_TRY(cudaFuncSetAttribute(et::attn::attn_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)et::attn::FWD_SMEM));
    CU_TRY(cudaFuncSetAttribute(et::attn::attn_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)et::attn::BWD_SMEM));
    done[dev] = true;
  }
  return ET_OK;
}

et_status run_attn_forward(et_stack* s, int l, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_ATTENTION, st);
  const LayerRT& L = s->ly[l];
  ET_TRY(attn_allow_smem());
  const int grid = (int)(s->M / L.seq) * L.heads;
  et::attn::attn_forward_kernel<<<grid, et::attn::THREADS, et::attn::FWD_SMEM, st>>>(
      a_map(s, l).b128, (bf16*)s->at(L.off_a_out), (float*)s->at(L.off_lse), L.seq, L.heads, L.N,
      (uint32_t*)s->at(s->off_status));
  return after_launch();
}
// G_l (gradient of [q | k | v]) from G_{l+1}; l >= 1 and the layer below has no activation, so G_l is its dZ.
et_status run_attn_backward(et_stack* s, int l, const void* dY, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_ATTENTION, st);
  const LayerRT& L = s->ly[l];
  ET_TRY(attn_allow_smem());
  const int grid = (int)(s->M / L.seq) * L.heads;
  et::attn::attn_backward_kernel<<<grid, et::attn::THREADS, et::attn::BWD_SMEM, st>>>(
      a_map(s, l).b128, g_map(s, l + 1).b128, (const bf16*)s->at(L.off_a_out), grad_act<bf16>(s, l + 1, dY),
      (const float*)s->at(L.off_lse), (bf16*)s->at(s->ly[l - 1].off_G_out), L.seq, L.heads, L.N,
      (uint32_t*)s->at(s->off_status));
  return after_launch();
}

// ---- patch gather of a convolution --------------------------------------------------------------
template <typename T>
et_status run_im2col_forward(et_stack* s, int l, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_ATTENTION, st);
  const LayerRT& L = s->ly[l];
  const long long total = (long long)s->M * L.ksize * L.ksize * (L.K / 8);
  et::im2col_kernel<T><<<ceil_div(total, et::kGatherThreads), et::kGatherThreads, 0, st>>>(
      act_in<T>(s, l), (T*)s->at(L.off_a_out), s->M, L.img_h, L.img_w, L.K, L.ksize);
  return after_launch();
}
// G_l (with the skip gradient) and dZ_{l-1} from the gradient of the gathered rows; l >= 1.
template <typename T>
et_status run_im2col_backward(et_stack* s, int l, const void* dY, cudaStream_t st) {
  TimedLaunch tl(s, ET_K_ATTENTION, st);
  const LayerRT& L = s->ly[l];
  const LayerRT& P = s->ly[l - 1];
  const bool need_act = P.act != ET_ACT_NONE;
  const bool need_G = !need_act || P.residual_src >= 0;
  const T* skip = L.consumer >= 0 ? grad_act<T>(s, L.consumer + 1, dY) : nullptr;
  const long long total = (long long)s->M * (L.K / 8);
  et::col2im_kernel<T><<<ceil_div(total, et::kGatherThreads), et::kGatherThreads, 0, st>>>(
      grad_act<T>(s, l + 1, dY), skip, need_G ? (T*)s->at(P.off_G_out) : nullptr,
      need_act ? (const T*)s->at(P.off_Z) : nullptr, need_act ? (T*)s->at(P.off_dZ) : nullptr, P.act, s->M, L.img_h,
      L.img_w, L.K, L.ksize);
  return after_launch();
}

// dW_l = a_l^T dZ_l as split partials, then the reducer with grad / importance / SGD.
template <typename T>
et_status run_wgrad_layer(et_stack* s, int l, const void* dY, float* grad, const T* delta, bool sgd, float lr,
                          int* launches, cudaStream_t st, cudaEvent_t before_reduce = nullptr) {
  const LayerRT& L = s->ly[l];
  float* partial = (float*)s->at(s->off_partial);
  const size_t count = (size_t)L.K * L.N;
  et::PartialEpi epi;
  epi.base = partial; epi.split_stride = count; epi.ld = L.N; epi.split = 0;
  int split = 1;
  {
    TimedLaunch tl(s, ET_K_WGRAD, st);
    if constexpr (is_bf16<T>::value) {
      split = (s->shared_plan && !s->wgrad_one_unit) ? L.split_shared : L.split;
      et::tc::Params p = tc_params(s, L.K, L.N, (int)s->M, 1, split);
      p.b_mn_wrap = L.fold > 1 ? L.Nw : 0;
      et::tc::EpiMaps em;
      em.in[0] = em.in[1] = em.out[0] = em.out[1] = L.map_W.b64;      // unused by the direct epilogue
      if (l >= 1 && s->ly[l - 1].implicit) {
        // kernel gradient of a convolution: the rows of A^T are (tap, channel), gathered 64 pixels at a time
        ET_TRY(conv_input_maps(s, l - 1));
        conv_params(&p, s->ly[l - 1], 2);
        const CUtensorMap& bmap = mn_map(dz_map(s, l), 2, &p.b_3d);
        ET_TRY((launch_tc<true, true>(128, false, s->ly[l - 1].im_wg, bmap, em, p, epi, s->sms, st, s->wgrad_one_unit)));
      } else {
      const int bnh = L.pair_wgrad ? L.bn_wgrad / 2 : L.bn_wgrad;
      const CUtensorMap& amap = mn_map(a_map(s, l), 2, &p.a_3d);
      const CUtensorMap& bmap = mn_map(dz_map(s, l), bnh / 64, &p.b_3d);
      ET_TRY((launch_tc<true, true>(L.bn_wgrad, L.pair_wgrad, amap, bmap, em, p, epi, s->sms, st, s->wgrad_one_unit)));
      }
    } else {
      et::simt::Params p;
      p.rows = L.K; p.cols = L.N; p.kc = (int)s->M; p.segs = 1;
      p.sa_i = 1; p.sa_k = L.K;
      p.sb_k = L.Nw; p.sb_seg = 0; p.sb_j = 1; p.b_wrap = L.fold > 1 ? L.Nw : 0;
      ET_TRY(launch_simt<T>(act_in<T>(s, l), dz_src<T>(s, l, dY), p, epi, st));
    }
  }
  ++*launches;
  if (grad == nullptr && delta == nullptr && !sgd) return ET_OK;     // nothing consumes g
  if (before_reduce != nullptr) CU_TRY(cudaStreamWaitEvent(st, before_reduce, 0));
  TimedLaunch tl(s, ET_K_WGRAD_REDUCE, st);
  float* imp = (float*)s->at(s->off_imp_parts) + s->imp_offs[2 * l];
  et::wgrad_reduce_kernel<T><<<L.imp_count_w, et::kEltThreads, 0, st>>>(partial, split, count, count, grad, delta, imp,
                                                                        (T*)L.W, opt_params(s, lr), sgd ? 1 : 0,
                                                                        s->delta_is_snapshot ? 1 : 0, L.W32, L.st1[0],
                                                                        L.st2[0]);
  ++*launches;
  return after_launch();
}

// fused_chunks > 0: the column partials (that many row blocks) were already written by the dgrad
// GEMM of the layer above; only the finishing kernel runs.
template <typename T>
et_status run_bgrad_layer(et_stack* s, int l, const void* dY, float* grad, const T* delta, bool sgd, float lr,
                          int* launches, cudaStream_t st, int fused_chunks = 0) {
  TimedLaunch tl(s, ET_K_BGRAD, st);
  const LayerRT& L = s->ly[l];
  float* part = (float*)s->at(L.off_biaspart);
  int chunks = fused_chunks;
  if (fused_chunks == 0) {
    chunks = ceil_div(s->M, et::kColsumRows);
    dim3 grid(ceil_div(L.Nw, 256), chunks), block(32, 8);
    et::colsum_partial_kernel<T><<<grid, block, 0, st>>>(dz_src<T>(s, l, dY), (int)s->M, L.Nw, part);
    ET_TRY(after_launch());
    ++*launches;
  }
  float* imp = (float*)s->at(s->off_imp_parts) + s->imp_offs[2 * l + 1];
  et::bias_finish_kernel<T><<<L.imp_count_b, dim3(et::kBiasCols, et::kBiasLanes), 0, st>>>(part, chunks, L.Nw, L.N, grad, delta, imp,
                                                                       (T*)L.b, opt_params(s, lr), sgd ? 1 : 0, s->delta_is_snapshot ? 1 : 0, L.b32,
                                                                       L.st1[1], L.st2[1]);
  ++*launches;
  return after_launch();
}

et::MaskBits mask_bits(const uint8_t* mask, int n) {
  et::MaskBits b;
  std::memset(&b, 0, sizeof(b));
  for (int t = 0; t < n; ++t)
    if (mask[t]) b.w[t >> 5] |= 1u << (t & 31);
  return b;
}

et_status check_ready(const et_stack* s, const uint8_t* mask, int n_tensors) {
  if (s == nullptr || mask == nullptr) return ET_ERR_INVALID_ARG;
  if (n_tensors != 2 * s->L) return ET_ERR_INVALID_ARG;
  for (int t = 0; t < n_tensors; ++t)
    if (mask[t] && !s->ly[t / 2].trainable()) return ET_ERR_INVALID_ARG;   // nothing there to select
  if (!s->bound) return ET_ERR_STATE;
  return ET_OK;
}

// The dgrad chain dZ_{L-1} -> dZ_{L-2} -> ... is the critical path of the backward pass; weight
// gradients only hang off it.  Running the chain on its own high-priority stream lets weight-gradient
// CTAs fill the SMs a chain kernel leaves idle in its last wave and during its prologue and drain.
// Streams and events are host objects (no device memory).  et_stack_set_option(ET_OPTION_TWO_STREAMS, 0)
// turns this off.
bool setup_two_streams(et_stack* s) {
  if (s->two_streams >= 0) return s->two_streams == 1;
  s->two_streams = 0;
  int least = 0, greatest = 0;
  if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess) { (void)cudaGetLastError(); return false; }
  if (cudaStreamCreateWithPriority(&s->chain_stream, cudaStreamNonBlocking, greatest) != cudaSuccess) {
    (void)cudaGetLastError();
    s->chain_stream = nullptr;
    return false;
  }
  s->chain_ev.assign(s->L + 2, nullptr);
  bool ok = cudaEventCreateWithFlags(&s->fork_ev, cudaEventDisableTiming) == cudaSuccess;
  for (auto& e : s->chain_ev) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) { (void)cudaGetLastError(); return false; }
  s->two_streams = 1;
  return true;
}
void destroy_two_streams(et_stack* s) {
  for (auto e : s->chain_ev) if (e != nullptr) cudaEventDestroy(e);
  s->chain_ev.clear();
  if (s->fork_ev != nullptr) cudaEventDestroy(s->fork_ev);
  if (s->chain_stream != nullptr) cudaStreamDestroy(s->chain_stream);
  s->fork_ev = nullptr; s->chain_stream = nullptr; s->two_streams = -1;
}

// ---- one-launch backward -----------------------------------------------------------------------
// CTA pairs of gemm_list_kernel that fit on the current device at once (0 if that cannot be found out).
int list_max_clusters(int sms) {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 0; }
  std::lock_guard<std::mutex> cache_lock(g_cache_mutex);
  if (cached[dev] == 0) {
    cached[dev] = -1;
    auto kern = et::tl::gemm_list_kernel;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)et::tl::LSMEM_BYTES) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cudaLaunchAttribute attr[1];
      cfg.gridDim = dim3(sms & ~1); cfg.blockDim = dim3(et::tc::THREADS); cfg.dynamicSmemBytes = et::tl::LSMEM_BYTES;
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n >= 1) cached[dev] = n;
    }
    (void)cudaGetLastError();
  }
  return cached[dev] > 0 ? cached[dev] : 0;
}

// The epilogue dgrad(l) needs, as the list kernel has it: one input chunk (skip gradient, or Z of the layer
// below) and one output (G_l, or dZ_{l-1}).  False when both G_l and dZ_{l-1} must be stored.
bool list_dgrad_form(const et_stack* s, int l, bool* has_in, bool* mul_act) {
  const LayerRT& Y = s->ly[l];
  const LayerRT& P = s->ly[l - 1];
  const bool need_skip = Y.consumer >= 0;
  const bool need_act = P.act != ET_ACT_NONE;
  const bool need_G = !need_act || P.residual_src >= 0;
  if (!need_act) { *has_in = need_skip; *mul_act = false; return true; }
  if (!need_skip && !need_G) { *has_in = true; *mul_act = true; return true; }
  return false;
}
bool list_eligible(const et_stack* s, int d) {
  if (s->dtype != ET_BF16 || !s->opt_gemm_list || s->list_state < 0) return false;
  for (int l = d; l < s->L; ++l)
    if (!s->ly[l].list_ok) return false;
  for (int l = d + 1; l < s->L; ++l) {
    bool a, b;
    if (!list_dgrad_form(s, l, &a, &b)) return false;
  }
  return list_max_clusters(s->sms) > 0;
}

et_status launch_list(et_stack* s, const et::tl::Task* tasks_dev, int units, int counters, cudaStream_t st, bool* refused);

// Every GEMM of the pass as one task list and one cooperative launch of gemm_list_kernel, then one grouped
// launch each for the split reductions and the bias finishers.  *refused: the device would not take the
// cooperative launch; nothing of the pass has been changed, the caller runs the per-layer path instead.
et_status backward_list(et_stack* s, const void* dY, const uint8_t* mask, float* const* grads,
                        const void* const* delta, bool sgd, float lr, int d, int* launches_out, double* flops_out,
                        cudaStream_t st, bool* refused) {
  namespace tl = et::tl;
  const int L = s->L;
  const long long M = s->M;
  int launches = 0;
  *refused = false;
  const LayerRT& top = s->ly[L - 1];
  if (top.act != ET_ACT_NONE) {
    TimedLaunch tlch(s, ET_K_OTHER, st);
    const size_t count = (size_t)M * top.N;
    et::act_backward_kernel<bf16><<<ceil_div(count, et::kEltThreads * et::kVec), et::kEltThreads, 0, st>>>(
        (const bf16*)dY, (const bf16*)s->at(top.off_Z), (bf16*)s->at(top.off_dZ), count, top.act);
    ET_TRY(after_launch());
    ++launches;
  }
  const int top_chunks = ceil_div(M, et::kColsumRows);
  if (mask[2 * (L - 1) + 1]) {
    TimedLaunch tlch(s, ET_K_BGRAD, st);
    dim3 grid(ceil_div(top.Nw, 256), top_chunks), block(32, 8);
    et::colsum_partial_kernel<bf16><<<grid, block, 0, st>>>(dz_src<bf16>(s, L - 1, dY), (int)M, top.Nw,
                                                            (float*)s->at(top.off_biaspart));
    ET_TRY(after_launch());
    ++launches;
  }

  // ---- the task list (rebuilt only when the mask, dY or the binding changed)
  std::vector<uint8_t> key(mask, mask + 2 * L);
  {
    const void* p = dY;
    const unsigned serial = s->bind_serial;
    key.insert(key.end(), (const uint8_t*)&p, (const uint8_t*)&p + sizeof(p));
    key.insert(key.end(), (const uint8_t*)&serial, (const uint8_t*)&serial + sizeof(serial));
    for (int l = d; l < L; ++l) {                 // the reduce tasks hold these pointers
      if (!mask[2 * l]) continue;
      const void* q[2] = {grads ? (const void*)grads[2 * l] : nullptr, delta ? delta[2 * l] : nullptr};
      key.insert(key.end(), (const uint8_t*)q, (const uint8_t*)q + sizeof(q));
    }
    key.push_back(sgd ? 1 : 0);
  }
  const int tiles_m_tok = ceil_div(M, 2 * et::tc::BM);
  if (key != s->tasks_key) {
    std::vector<tl::Task>& tk = s->tasks_host;
    tk.clear();
    std::vector<int> sig_base(L + 1, -1), tiles_n_of(L + 1, 0);
    int counters = 0, units = 0;
    auto add_dgrad = [&](int l) {
      const LayerRT& Y = s->ly[l];
      const LayerRT& P = s->ly[l - 1];
      tl::Task t;
      std::memset(&t, 0, sizeof(t));
      bool has_in = false, mul_act = false;
      list_dgrad_form(s, l, &has_in, &mul_act);
      t.kind = tl::kDgrad;
      t.rows = (int)M; t.cols = Y.K;
      t.tiles_m = tiles_m_tok; t.tiles_n = ceil_div(Y.K, tl::LBN); t.split = 1;
      t.kb_per_seg = ceil_div(Y.Nw, et::tc::BK); t.kb_total = t.kb_per_seg * Y.fold; t.kb_per_split = t.kb_total;
      t.b_k_seg_stride = Y.Nw; t.b_mn_wrap = 0;
      t.map_a = dz_map(s, l).b128;
      t.map_b = Y.map_Wd_list;
      if (mul_act) { t.map_in = P.map_Z.b128; t.map_out = P.map_dZ.b128; }
      else { t.map_in = has_in ? g_map(s, Y.consumer + 1).b128 : P.map_Gout.b128; t.map_out = P.map_Gout.b128; }
      t.has_in = has_in ? 1 : 0; t.mul_act = mul_act ? 1 : 0; t.act_prev = P.act; t.ld = Y.K;
      t.colsum = mask[2 * (l - 1) + 1] ? (float*)s->at(P.off_biaspart) : nullptr;
      t.unit_begin = units; t.units = t.tiles_m * t.tiles_n; units += t.units;
      t.wait_base = l + 1 <= L - 1 ? sig_base[l + 1] : -1; t.wait_per_row = 1;
      t.wait_target = 4u * (unsigned)tiles_n_of[l + 1];
      t.wait2_base = -1; t.wait2_target = 0;
      if (!mul_act && has_in && Y.consumer + 1 <= L - 1) {
        t.wait2_base = sig_base[Y.consumer + 1];
        t.wait2_target = 4u * (unsigned)tiles_n_of[Y.consumer + 1];
      }
      t.signal_base = counters; sig_base[l] = counters; tiles_n_of[l] = t.tiles_n;
      counters += t.tiles_m + 1;
      tk.push_back(t);
    };
    auto add_wgrad = [&](int l) {
      const LayerRT& Y = s->ly[l];
      tl::Task t;
      std::memset(&t, 0, sizeof(t));
      t.kind = tl::kWgrad;
      t.rows = Y.K; t.cols = Y.N;
      t.tiles_m = ceil_div(Y.K, 2 * et::tc::BM); t.tiles_n = ceil_div(Y.N, tl::LBN); t.split = s->ly[l].split_now;
      t.kb_per_seg = ceil_div(M, et::tc::BK); t.kb_total = t.kb_per_seg; t.kb_per_split = ceil_div(t.kb_total, t.split);
      t.b_k_seg_stride = 0; t.b_mn_wrap = Y.fold > 1 ? Y.Nw : 0;
      t.map_a = a_map(s, l).c3[0];
      t.map_b = dz_map(s, l).c3[0];
      t.map_in = t.map_a; t.map_out = t.map_a;                 // unused by this kind
      t.partial = (float*)s->at(Y.off_partial_list); t.split_stride = (unsigned long long)Y.K * Y.N; t.ld_out = Y.N;
      t.unit_begin = units; t.units = t.tiles_m * t.tiles_n * t.split; units += t.units;
      t.wait_base = -1; t.wait_per_row = 0; t.wait_target = 0;
      if (l + 1 <= L - 1) {                                    // dZ_l is complete once every unit of dgrad(l+1) is
        t.wait_base = sig_base[l + 1] + tiles_m_tok;
        t.wait_target = 4u * (unsigned)tiles_m_tok * (unsigned)tiles_n_of[l + 1];
      }
      t.wait2_base = -1; t.signal_base = -1;
      tk.push_back(t);
    };
    // Order: the whole error-gradient chain first, then the weight gradients.  (Interleaved, a CTA busy with a
    // long weight-gradient unit holds up the chain units queued behind it and every row tile below them;
    // measured on the ViT-B- and ViT-L-shaped stacks the chain-first list is 2 to 10 % faster, on the narrow 1x1
    // convolution stack the two orders tie.)
    // Contraction splits: with the chain out of the way a weight gradient runs unsplit, so that its partial sum
    // is the gradient and nothing is written and read twice; the last two of the list are cut into shorter
    // units so that the launch does not end on a few CTAs working through 200-k-block units while the rest idle.
    std::vector<int> sel;                                      // selected kernels, top first
    for (int l = L - 1; l >= d; --l)
      if (mask[2 * l]) sel.push_back(l);
    for (size_t i = 0; i < sel.size(); ++i)
      s->ly[sel[i]].split_now = i + 2 < sel.size() ? 1 : s->ly[sel[i]].split_list;
    for (int l = L - 1; l > d; --l) add_dgrad(l);
    for (int l : sel) add_wgrad(l);
    s->tasks_units = units;
    s->tasks_counters = counters;
    if (counters > s->max_counters || tk.size() > (size_t)2 * L) return ET_ERR_WORKSPACE;
    if (!tk.empty())
      CU_TRY(cudaMemcpyAsync(s->at(s->off_tasks), tk.data(), tk.size() * sizeof(tl::Task), cudaMemcpyHostToDevice, st));
    s->tasks_key = key;
  }
  double flops = 0.0;
  for (int l = d; l < L; ++l) {
    const double gemm = 2.0 * (double)M * s->ly[l].K * s->ly[l].N;
    if (l > d) flops += gemm;
    if (mask[2 * l]) flops += gemm;
  }

  const et::OptParams opt = opt_params(s, lr);
  const int snap = s->delta_is_snapshot ? 1 : 0;
  if (s->tasks_units > 0) {
    ET_TRY(launch_list(s, (const tl::Task*)s->at(s->off_tasks), s->tasks_units, s->tasks_counters, st, refused));
    if (*refused) return ET_OK;
    ++launches;
  }

  // ---- grouped split reduction (gradient export, Eq. 2, update) and grouped bias finishers
  float* imp_parts = (float*)s->at(s->off_imp_parts);
  {
    std::vector<et::ReduceEntry> tab;
    std::vector<int> chunk_blocks;                  // blocks of each launch of at most kGroupMax tensors
    int blocks = 0;
    for (int l = d; l < L; ++l) {
      if (!mask[2 * l]) continue;
      const LayerRT& Y = s->ly[l];
      float* g = grads ? grads[2 * l] : nullptr;
      const void* dl = delta ? delta[2 * l] : nullptr;
      if (g == nullptr && dl == nullptr && !sgd) continue;       // nothing consumes the gradient
      et::ReduceEntry e;
      std::memset(&e, 0, sizeof(e));
      e.partial = (const float*)s->at(Y.off_partial_list); e.grad = g; e.delta = dl;
      e.imp_part = imp_parts + s->imp_offs[2 * l]; e.W = Y.W; e.master = Y.W32; e.m_state = Y.st1[0]; e.v_state = Y.st2[0];
      e.count = (unsigned long long)Y.K * Y.N; e.splits = Y.split_now;
      if (tab.size() % et::kGroupMax == 0) { chunk_blocks.push_back(0); blocks = 0; }   // a new launch starts here
      e.block_begin = blocks;
      blocks += Y.imp_count_w;
      chunk_blocks.back() = blocks;
      tab.push_back(e);
    }
    if (!tab.empty()) {
      if (tab.size() != s->rtab_host.size() ||
          std::memcmp(tab.data(), s->rtab_host.data(), tab.size() * sizeof(et::ReduceEntry)) != 0) {
        CU_TRY(cudaMemcpyAsync(s->at(s->off_rtab), tab.data(), tab.size() * sizeof(et::ReduceEntry),
                               cudaMemcpyHostToDevice, st));
        s->rtab_host = tab;
      }
      for (size_t i0 = 0; i0 < tab.size(); i0 += et::kGroupMax) {
        const int n = (int)std::min(tab.size() - i0, (size_t)et::kGroupMax);
        const int nb = chunk_blocks[i0 / et::kGroupMax];
        TimedLaunch tlch(s, ET_K_WGRAD_REDUCE, st);
        et::wgrad_reduce_group_kernel<bf16><<<std::min(nb, s->sms * et::kGroupBlocksPerSm), et::kEltThreads, 0, st>>>(
            (const et::ReduceEntry*)s->at(s->off_rtab) + i0, n, nb, opt, sgd ? 1 : 0, snap);
        ET_TRY(after_launch());
        ++launches;
      }
    }
  }
  {
    std::vector<et::BiasEntry> tab;
    std::vector<int> chunk_blocks;
    int blocks = 0;
    for (int l = d; l < L; ++l) {
      if (!mask[2 * l + 1]) continue;
      const LayerRT& Y = s->ly[l];
      et::BiasEntry e;
      std::memset(&e, 0, sizeof(e));
      e.part = (const float*)s->at(Y.off_biaspart);
      e.grad = grads ? grads[2 * l + 1] : nullptr; e.delta = delta ? delta[2 * l + 1] : nullptr;
      e.imp_part = imp_parts + s->imp_offs[2 * l + 1]; e.b = Y.b; e.master = Y.b32; e.m_state = Y.st1[1]; e.v_state = Y.st2[1];
      // row blocks the partials come in: 32-row blocks of the dgrad epilogue above, 128-row chunks for the top layer
      e.chunks = l == L - 1 ? top_chunks : tiles_m_tok * (2 * et::tc::BM / 32);
      e.width = Y.Nw; e.count = Y.N;
      if (tab.size() % et::kGroupMax == 0) { chunk_blocks.push_back(0); blocks = 0; }
      e.block_begin = blocks;
      blocks += Y.imp_count_b;
      chunk_blocks.back() = blocks;
      tab.push_back(e);
    }
    if (!tab.empty()) {
      if (tab.size() != s->btab_host.size() ||
          std::memcmp(tab.data(), s->btab_host.data(), tab.size() * sizeof(et::BiasEntry)) != 0) {
        CU_TRY(cudaMemcpyAsync(s->at(s->off_btab), tab.data(), tab.size() * sizeof(et::BiasEntry),
                               cudaMemcpyHostToDevice, st));
        s->btab_host = tab;
      }
      for (size_t i0 = 0; i0 < tab.size(); i0 += et::kGroupMax) {
        const int n = (int)std::min(tab.size() - i0, (size_t)et::kGroupMax);
        const int nb = chunk_blocks[i0 / et::kGroupMax];
        TimedLaunch tlch(s, ET_K_BGRAD, st);
        et::bias_finish_group_kernel<bf16><<<std::min(nb, s->sms * 2), dim3(et::kBiasCols, et::kBiasLanes), 0, st>>>(
            (const et::BiasEntry*)s->at(s->off_btab) + i0, n, nb, opt, sgd ? 1 : 0, snap);
        ET_TRY(after_launch());
        ++launches;
      }
    }
  }
  *launches_out += launches;
  *flops_out += flops;
  return ET_OK;
}

template <typename T>
et_status backward_impl(et_stack* s, const void* dY, const uint8_t* mask, float* const* grads,
                        const void* const* delta, float* importance_dev, uint32_t flags, float lr,
                        et_exec_report* report, cudaStream_t st) {
  const int L = s->L;
  int d = L;
  for (int l = 0; l < L; ++l)
    if (mask[2 * l] || mask[2 * l + 1]) { d = l; break; }
  const bool sgd = (flags & ET_FLAG_FUSE_SGD) != 0;
  s->delta_is_snapshot = delta != nullptr && (flags & ET_FLAG_DELTA_IS_SNAPSHOT) != 0;
  int launches = 0;
  double flops = 0.0;

  if (report != nullptr) {
    for (int l = 0; l < L; ++l) {
      if (report->dgrad) report->dgrad[l] = l > d;
      if (report->wgrad) report->wgrad[l] = mask[2 * l] != 0;
      if (report->bgrad) report->bgrad[l] = mask[2 * l + 1] != 0;
      if (report->updated) {
        report->updated[2 * l] = sgd && mask[2 * l];
        report->updated[2 * l + 1] = sgd && mask[2 * l + 1];
      }
    }
    report->deepest = d;
  }

  if (d == L) {
    if (delta != nullptr) CU_TRY(cudaMemsetAsync(importance_dev, 0, sizeof(float) * 2 * L, st));
  } else {
    if constexpr (is_bf16<T>::value) {
      if (s->map_dy_ptr != dY) {
        ET_TRY(make_tmaps(&s->map_dy, dY, s->out_width(), s->M));
        s->map_dy_ptr = dY;
      }
    }
    // Stacks of plain dense layers take the one-launch path: all GEMMs of the pass in one cooperative kernel,
    // one grouped reducer, one grouped bias finisher.
    bool done_by_list = false;
    if constexpr (is_bf16<T>::value) {
      if (list_eligible(s, d)) {
        bool refused = false;
        ET_TRY(backward_list(s, dY, mask, grads, delta, sgd, lr, d, &launches, &flops, st, &refused));
        done_by_list = !refused;
      }
    }
    if (!done_by_list) {
    const bool two = !s->timing && s->opt_two_streams && setup_two_streams(s);   // per-kernel timing wants kernels one at a time
    // Sharing the GPU with the higher-priority error-gradient chain: when few kernels are selected
    // the weight gradients are filler work and should hand their SMs back after every unit; when
    // they are as much work as the chain itself, persistent CTAs (epilogue overlap) pay more (ViT-B step:
    // 2.33 ms with one-unit CTAs against 2.46 ms persistent; full backprop 4.0 ms persistent against 4.5 ms).
    int n_w = 0;
    for (int l = d; l < L; ++l) n_w += mask[2 * l] ? 1 : 0;
    // Tile plan: the one made for a shared GPU whenever the two streams run (or on request, so that
    // per-kernel timing on one stream can time the very kernels the two-stream step launches).
    s->shared_plan = s->opt_tile_plan == ET_TILE_PLAN_SHARED || (s->opt_tile_plan == ET_TILE_PLAN_AUTO && two);
    s->wgrad_one_unit = s->shared_plan && 2 * n_w <= L - d;
    // With a second stream the weight-gradient CTAs get their SMs in the gaps between the chain's
    // kernels; a chain kernel that took over each SM the moment its predecessor left would starve
    // them until the chain ends (measured: 2.45 -> 2.62 ms per ViT-B step), so no launch overlap then.
    s->chain_shares_gpu = two;
    cudaStream_t cs = two ? s->chain_stream : st;          // stream of the error-gradient chain
    if (two) {
      CU_TRY(cudaEventRecord(s->fork_ev, st));
      CU_TRY(cudaStreamWaitEvent(cs, s->fork_ev, 0));
    }
    const LayerRT& top = s->ly[L - 1];
    if (top.act != ET_ACT_NONE) {
      TimedLaunch tl(s, ET_K_OTHER, cs);
      const size_t count = (size_t)s->M * top.N;
      et::act_backward_kernel<T><<<ceil_div(count, et::kEltThreads * et::kVec), et::kEltThreads, 0, cs>>>(
          (const T*)dY, (const T*)s->at(top.off_Z), (T*)s->at(top.off_dZ), count, top.act);
      ET_TRY(after_launch());
      ++launches;
    }
    if (two) CU_TRY(cudaEventRecord(s->chain_ev[L], cs));  // dZ_{L-1} is ready
    for (int l = L - 1; l >= d; --l) {
      const LayerRT& Y = s->ly[l];
      const bool norm = Y.vector_params();
      const double gemm = Y.kind != ET_LAYER_DENSE ? 0.0 : 2.0 * (double)s->M * Y.K * Y.N;
      if (mask[2 * l + 1]) {
        // On the tensor-core path the column partials of dZ_l were left by dgrad(l+1) in this
        // layer's own buffer; finishing them need not sit on the chain's critical path.
        // (A normalisation layer above leaves none: the column-sum kernel runs instead.)
        const int fused = (is_bf16<T>::value && l < L - 1 && s->ly[l + 1].kind == ET_LAYER_DENSE)
                              ? dgrad_row_blocks(s, l + 1) : 0;
        // Which stream: with few selected kernels the caller's stream is nearly idle and takes
        // the finishers off the chain; with many it is the busier one and the chain keeps them.
        cudaStream_t bs = s->wgrad_one_unit ? st : cs;
        if (two && bs == st) CU_TRY(cudaStreamWaitEvent(st, s->chain_ev[l + 1], 0));
        ET_TRY(run_bgrad_layer<T>(s, l, dY, grads ? grads[2 * l + 1] : nullptr,
                                  delta ? (const T*)delta[2 * l + 1] : nullptr, sgd, lr, &launches, bs, fused));
      }
      if (!Y.trainable()) {
        // a non-trainable layer: only passes the error gradient on, above the deepest selected layer
        if (Y.implicit) continue;                            // done by the error-gradient GEMM of the layer above
        if (l > d) {
          if (Y.kind == ET_LAYER_ATTENTION) ET_TRY(run_attn_backward(s, l, dY, cs));
          else ET_TRY(run_im2col_backward<T>(s, l, dY, cs));
          ++launches;
          if (two) CU_TRY(cudaEventRecord(s->chain_ev[l], cs));
        }
        continue;
      }
      if (norm) {
        // one kernel passes the error gradient on (above the deepest selected layer) and leaves the
        // partials of d gamma (if selected); it reads gamma, so the finisher that may update gamma
        // follows it on the same stream
        if (l > d || mask[2 * l]) {
          if (Y.kind == ET_LAYER_NORM)
            ET_TRY(run_norm_backward<T>(s, l, dY, l > d, mask[2 * l] != 0, grads ? grads[2 * l] : nullptr,
                                        delta ? (const T*)delta[2 * l] : nullptr, sgd, lr, &launches, cs));
          else
            ET_TRY(run_bn_backward<T>(s, l, dY, l > d, mask[2 * l] != 0, grads ? grads[2 * l] : nullptr,
                                      delta ? (const T*)delta[2 * l] : nullptr, sgd, lr, &launches, cs));
        }
        if (two && l > d) CU_TRY(cudaEventRecord(s->chain_ev[l], cs));
        continue;
      }
      if (l > d) {
        ET_TRY(run_dgrad_layer<T>(s, l, dY, cs, mask[2 * (l - 1) + 1] != 0));
        if (two) CU_TRY(cudaEventRecord(s->chain_ev[l], cs));   // dZ_{l-1} ready, W_l no longer needed
        if (two && s->ly[l - 1].implicit) CU_TRY(cudaEventRecord(s->chain_ev[l - 1], cs));   // and the gather's backward with it
        ++launches;
        flops += gemm;
      }
      if (mask[2 * l]) {
        // needs dZ_l (left by dgrad(l+1)); its update of W_l has to wait until dgrad(l) has read W_l
        if (two) CU_TRY(cudaStreamWaitEvent(st, s->chain_ev[l + 1], 0));
        ET_TRY(run_wgrad_layer<T>(s, l, dY, grads ? grads[2 * l] : nullptr,
                                  delta ? (const T*)delta[2 * l] : nullptr, sgd, lr, &launches, st,
                                  (two && l > d) ? s->chain_ev[l] : nullptr));
        flops += gemm;
      }
    }
    if (two) {
      CU_TRY(cudaEventRecord(s->chain_ev[L + 1], cs));
      CU_TRY(cudaStreamWaitEvent(st, s->chain_ev[L + 1], 0));
    }
    }   // per-layer path
    if (delta != nullptr) {
      TimedLaunch tl(s, ET_K_OTHER, st);
      et::importance_finalize_kernel<<<2 * L, 128, 0, st>>>((const float*)s->at(s->off_imp_parts),
                                                            (const int*)s->at(s->off_imp_offs),
                                                            (const int*)s->at(s->off_imp_counts), mask_bits(mask, 2 * L),
                                                            importance_dev);
      ET_TRY(after_launch());
      ++launches;
    }
  }
  if (report != nullptr) {
    report->launches = launches;
    report->flops_executed = flops;
  }
  return ET_OK;
}

et_status validate_backward_args(const et_stack* s, const void* dY, const uint8_t* mask, int32_t n_tensors,
                                 const void* const* delta, const void* importance) {
  ET_TRY(check_ready(s, mask, n_tensors));
  if (dY == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->forwarded) return ET_ERR_STATE;
  if (delta != nullptr) {
    if (importance == nullptr) return ET_ERR_INVALID_ARG;
    for (int t = 0; t < n_tensors; ++t)
      if (mask[t] && delta[t] == nullptr) return ET_ERR_INVALID_ARG;
  }
  return ET_OK;
}

// The forward pass of a stack of plain dense layers as one task list (the same kernel as the one-launch
// backward): layer l + 1's row tile r waits for layer l's row tile r.  *refused as in backward_list.
et_status launch_list(et_stack* s, const et::tl::Task* tasks_dev, int units, int counters, cudaStream_t st, bool* refused) {
  namespace tl = et::tl;
  *refused = false;
  if (counters > 0) CU_TRY(cudaMemsetAsync(s->at(s->off_counters), 0, sizeof(unsigned) * (size_t)counters, st));
  TimedLaunch tlch(s, ET_K_LIST, st);
  const int workers = std::min(units, list_max_clusters(s->sms));
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.gridDim = dim3(2 * workers); cfg.blockDim = dim3(et::tc::THREADS); cfg.dynamicSmemBytes = tl::LSMEM_BYTES;
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;           // every CTA resident: units may wait on one another
  attr[1].val.cooperative = 1;
  cfg.attrs = attr; cfg.numAttrs = s->opt_list_cooperative ? 2 : 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, tl::gemm_list_kernel, tasks_dev, units, (unsigned*)s->at(s->off_counters),
                                           (uint32_t*)s->at(s->off_status));
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    if (s->list_state == 0) { s->list_state = -1; *refused = true; return ET_OK; }
    g_last_cuda = (int)e;
    return ET_ERR_CUDA;
  }
  s->list_state = 1;
  return after_launch();
}

bool forward_list_eligible(const et_stack* s) {
  if (s->dtype != ET_BF16 || !s->opt_gemm_list || s->list_state < 0) return false;
  for (int l = 0; l < s->L; ++l) {
    const LayerRT& y = s->ly[l];
    if (!y.list_ok) return false;
    if (y.act != ET_ACT_NONE && y.residual_src >= 0) return false;   // Z, the output and a residual: three chunks
  }
  return list_max_clusters(s->sms) > 0;
}

et_status forward_list(et_stack* s, const void* x, void* y, cudaStream_t st, bool* refused) {
  namespace tl = et::tl;
  const int L = s->L;
  const long long M = s->M;
  const int tiles_m = ceil_div(M, 2 * et::tc::BM);
  std::vector<uint8_t> key;
  {
    const void* q[2] = {x, y};
    const unsigned serial = s->bind_serial;
    key.insert(key.end(), (const uint8_t*)q, (const uint8_t*)q + sizeof(q));
    key.insert(key.end(), (const uint8_t*)&serial, (const uint8_t*)&serial + sizeof(serial));
  }
  if (key != s->ftasks_key) {
    std::vector<tl::Task>& tk = s->ftasks_host;
    tk.clear();
    std::vector<int> sig_base(L, -1), tiles_n_of(L, 0);
    int counters = 0, units = 0;
    for (int l = 0; l < L; ++l) {
      const LayerRT& Y = s->ly[l];
      tl::Task t;
      std::memset(&t, 0, sizeof(t));
      t.kind = tl::kFwd;
      t.rows = (int)M; t.cols = Y.Nw;
      t.tiles_m = tiles_m; t.tiles_n = ceil_div(Y.Nw, tl::LBN); t.split = 1;
      t.kb_per_seg = ceil_div(Y.K, et::tc::BK); t.kb_total = t.kb_per_seg * Y.fold; t.kb_per_split = t.kb_total;
      t.b_k_seg_stride = 0; t.b_mn_wrap = 0; t.b_mn_seg_stride = Y.Nw;
      t.map_a = a_map(s, l).b128;
      t.map_b = Y.map_W.c3[0];
      const CUtensorMap& out = (l == L - 1 ? s->map_y : Y.map_aout).b128;
      t.map_in = Y.residual_src >= 0 ? a_map(s, Y.residual_src).b128 : out;
      t.map_out = out;
      t.map_out2 = Y.act != ET_ACT_NONE ? Y.map_Z.b128 : out;
      t.has_in = Y.residual_src >= 0 ? 1 : 0;
      t.entries = Y.act != ET_ACT_NONE ? 2 : 1;
      t.act = Y.act; t.fold = Y.fold; t.ld = Y.Nw; t.bias = (const bf16*)Y.b;
      t.unit_begin = units; t.units = t.tiles_m * t.tiles_n; units += t.units;
      t.wait_base = l >= 1 ? sig_base[l - 1] : -1; t.wait_per_row = 1;
      t.wait_target = l >= 1 ? 4u * (unsigned)tiles_n_of[l - 1] : 0u;
      t.wait2_base = -1; t.wait2_target = 0;
      if (Y.residual_src >= 1) {                              // a_j is the output of layer j - 1
        t.wait2_base = sig_base[Y.residual_src - 1];
        t.wait2_target = 4u * (unsigned)tiles_n_of[Y.residual_src - 1];
      }
      t.signal_base = counters; sig_base[l] = counters; tiles_n_of[l] = t.tiles_n;
      counters += t.tiles_m + 1;
      tk.push_back(t);
    }
    if (counters > s->max_counters) return ET_ERR_WORKSPACE;
    s->ftasks_units = units; s->ftasks_counters = counters;
    CU_TRY(cudaMemcpyAsync(s->at(s->off_ftasks), tk.data(), tk.size() * sizeof(tl::Task), cudaMemcpyHostToDevice, st));
    s->ftasks_key = key;
  }
  return launch_list(s, (const tl::Task*)s->at(s->off_ftasks), s->ftasks_units, s->ftasks_counters, st, refused);
}

template <typename T>
et_status forward_impl(et_stack* s, const void* x, void* y, cudaStream_t st) {
  if constexpr (is_bf16<T>::value) {
    if (s->x != x || !s->forwarded) ET_TRY(make_tmaps(&s->map_x, x, s->ly[0].K, s->M));
    if (s->map_y_ptr != y) {
      ET_TRY(make_tmaps(&s->map_y, y, s->out_width(), s->M));
      s->map_y_ptr = y;
    }
  }
  s->x = x;
  if constexpr (is_bf16<T>::value) {
    if (forward_list_eligible(s)) {
      bool refused = false;
      ET_TRY(forward_list(s, x, y, st, &refused));
      if (!refused) { s->forwarded = true; return ET_OK; }
    }
  }
  for (int l = 0; l < s->L; ++l) {
    if (s->ly[l].kind == ET_LAYER_NORM) ET_TRY(run_norm_forward<T>(s, l, y, st));
    else if (s->ly[l].kind == ET_LAYER_BATCHNORM) ET_TRY(run_bn_forward<T>(s, l, y, st));
    else if (s->ly[l].kind == ET_LAYER_ATTENTION) ET_TRY(run_attn_forward(s, l, st));
    else if (s->ly[l].kind == ET_LAYER_IM2COL) { if (!s->ly[l].implicit) ET_TRY(run_im2col_forward<T>(s, l, st)); }
    else ET_TRY(run_forward_layer<T>(s, l, y, st));
  }
  s->forwarded = true;
  return ET_OK;
}

double median(std::vector<float>& v) {
  std::sort(v.begin(), v.end());
  return v.empty() ? 0.0 : (double)v[v.size() / 2];
}

}  // namespace

// =============================================================================================
extern "C" {

et_status et_stack_create(const et_layer_desc* layers, int32_t L, int64_t M, et_dtype dtype, et_stack** out) {
  if (layers == nullptr || out == nullptr || L < 1 || L > 1024 || M < 1 || M > (1ll << 30)) return ET_ERR_INVALID_ARG;
  // the column-sum kernels run one grid row per 128 rows of the activations: at most 65535 of them
  if ((M + et::kColsumRows - 1) / et::kColsumRows > 65535) return ET_ERR_UNSUPPORTED;
  if (dtype != ET_F32 && dtype != ET_BF16) return ET_ERR_DTYPE;
  et_stack* s = new (std::nothrow) et_stack();
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  s->L = L; s->M = M; s->dtype = dtype; s->elt = dtype == ET_BF16 ? 2 : 4;
  s->ly.resize(L);
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      s->sms = sms;
    else
      (void)cudaGetLastError();
  }
  et_status err = ET_OK;
  std::vector<int> width(L + 1);
  width[0] = layers[0].in_features;
  for (int l = 0; l < L && err == ET_OK; ++l) {
    const et_layer_desc& d = layers[l];
    LayerRT& y = s->ly[l];
    if (d.in_features < 1 || d.out_features < 1 || d.fold < 1 || d.act < 0 || d.act > 2) { err = ET_ERR_INVALID_ARG; break; }
    if (d.out_features % d.fold != 0) { err = ET_ERR_SHAPE; break; }
    if (d.fold > 1 && d.act != ET_ACT_NONE) { err = ET_ERR_UNSUPPORTED; break; }
    y.K = d.in_features; y.N = d.out_features; y.fold = d.fold; y.Nw = d.out_features / d.fold;
    y.act = d.act; y.residual_src = d.residual_src;
    if (d.kind < ET_LAYER_DENSE || d.kind > ET_LAYER_BATCHNORM) { err = ET_ERR_INVALID_ARG; break; }
    y.kind = d.kind; y.eps = d.eps;
    if (y.kind == ET_LAYER_BATCHNORM) {
      if (y.K != y.N || y.fold != 1 || y.residual_src != -1 || !(y.eps >= 0.f)) { err = ET_ERR_INVALID_ARG; break; }
      if (y.N % 8) { err = ET_ERR_UNSUPPORTED; break; }
    }
    if (y.kind == ET_LAYER_IM2COL) {
      y.img_h = d.height; y.img_w = d.width; y.ksize = d.ksize;
      if (y.fold != 1 || y.act != ET_ACT_NONE || y.residual_src != -1 || y.img_h < 1 || y.img_w < 1 || y.ksize < 1 ||
          y.ksize % 2 == 0 || (long long)y.N != (long long)y.ksize * y.ksize * y.K) {
        err = ET_ERR_INVALID_ARG; break;
      }
      if (M % ((long long)y.img_h * y.img_w) != 0) { err = ET_ERR_SHAPE; break; }
      if (y.K % 8 || y.ksize > 7 || l == L - 1) { err = ET_ERR_UNSUPPORTED; break; }
    }
    if (y.kind == ET_LAYER_ATTENTION) {
      y.heads = d.heads; y.seq = d.seq_len;
      if (y.fold != 1 || y.act != ET_ACT_NONE || y.residual_src != -1 || y.heads < 1 || y.seq < 1 || y.K != 3 * y.N) {
        err = ET_ERR_INVALID_ARG; break;
      }
      if (M % y.seq != 0) { err = ET_ERR_SHAPE; break; }
      if (dtype != ET_BF16 || y.N != et::attn::DH * y.heads || y.seq > et::attn::S_MAX || l == 0 || l == L - 1 ||
          s->ly[l - 1].act != ET_ACT_NONE) {
        err = ET_ERR_UNSUPPORTED; break;
      }
    }
    if (y.kind == ET_LAYER_NORM) {
      if (y.K != y.N || y.fold != 1 || y.act != ET_ACT_NONE || y.residual_src != -1 || !(y.eps >= 0.f)) {
        err = ET_ERR_INVALID_ARG; break;
      }
      if (y.N % 8 || y.N > et::kNormMaxWidth) { err = ET_ERR_UNSUPPORTED; break; }
    }
    if (y.K != width[l]) { err = ET_ERR_SHAPE; break; }
    width[l + 1] = y.Nw;
    if (d.residual_src < -1 || d.residual_src > l) { err = ET_ERR_INVALID_ARG; break; }
    if (d.residual_src >= 0) {
      if (width[d.residual_src] != y.Nw) { err = ET_ERR_SHAPE; break; }
      if (d.residual_src >= 1) {          // a_0's gradient is never formed, no bookkeeping needed
        LayerRT& src = s->ly[d.residual_src];
        if (src.consumer >= 0) { err = ET_ERR_UNSUPPORTED; break; }   // one skip consumer per activation
        src.consumer = l;
      }
    }
    if (dtype == ET_BF16) {
      if (y.K % 8 || y.N % 8 || y.Nw % 8) { err = ET_ERR_UNSUPPORTED; break; }
      if (y.fold > 1 && y.Nw % 256) { err = ET_ERR_UNSUPPORTED; break; }
    }
  }
  for (int l = 0; l < L && err == ET_OK; ++l)
    if (s->ly[l].kind == ET_LAYER_ATTENTION && s->ly[l].consumer >= 0) err = ET_ERR_UNSUPPORTED;   // [q|k|v] feeds nothing else
  // A patch gather followed directly by a dense layer is folded into that layer's GEMMs (the gathered matrix is
  // never formed) when the shapes allow TMA's im2col loads: bf16, channels a multiple of 128 (a 128-row tile of
  // the kernel gradient then lies within one tap), not the first layer (its input would need no gradient).
  for (int l = 1; l + 1 < L && err == ET_OK; ++l) {
    LayerRT& y = s->ly[l];
    const LayerRT& up = s->ly[l + 1];
    y.implicit = dtype == ET_BF16 && y.kind == ET_LAYER_IM2COL && y.K % 128 == 0 && up.kind == ET_LAYER_DENSE &&
                 up.fold == 1 && up.N % 64 == 0;
  }
  if (err != ET_OK) { delete s; return err; }

  // ---- workspace layout
  size_t off = 0;
  const bool guarded = g_guard_regions.load() != 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off += align256(bytes);
    if (guarded) { s->guards.push_back(off); off += kGuardBytes; }   // a region's overrun lands here first
    return o;
  };
  s->off_status = take(256);
  size_t max_partial = 0;
  const int chunks = ceil_div(M, et::kColsumRows);
  s->imp_offs.resize(2 * L); s->imp_counts.resize(2 * L);
  int imp_total = 0;
  for (int l = 0; l < L; ++l) {
    LayerRT& y = s->ly[l];
    const size_t act_bytes = (size_t)M * y.Nw * s->elt;
    if (l < L - 1 && !y.implicit) { y.off_a_out = take(act_bytes); y.off_G_out = take(act_bytes); }
    if (y.act != ET_ACT_NONE) { y.off_Z = take(act_bytes); y.off_dZ = take(act_bytes); }
    if (y.kind == ET_LAYER_ATTENTION) {
      y.off_lse = take((size_t)M * y.heads * sizeof(float));
    } else if (y.kind == ET_LAYER_BATCHNORM) {
      y.off_stats = take((size_t)y.N * sizeof(float2));
      y.off_means = take((size_t)y.N * sizeof(float2));
      y.norm_blocks = ceil_div(M, et::kBnRows);                           // chunks of the column reductions
      y.off_gpart = take((size_t)2 * y.norm_blocks * y.N * sizeof(float));
    } else if (y.kind == ET_LAYER_NORM) {
      y.off_stats = take((size_t)M * sizeof(float2));
      y.norm_blocks = std::min(ceil_div(M, et::kNormWarps), s->sms * 8);
      y.off_gpart = take((size_t)y.norm_blocks * y.N * sizeof(float));
    } else if (dtype == ET_BF16) {
      const int kb_n = ceil_div(y.Nw, et::tc::BK) * y.fold;
      const TilePlan f = choose_tiles((int)M, y.Nw, ceil_div(y.K, et::tc::BK) * y.fold, s->sms, false, false, 0);
      const TilePlan d = choose_tiles((int)M, y.K, kb_n, s->sms, false, true, 0);
      const TilePlan w = choose_tiles(y.K, y.N, ceil_div(M, et::tc::BK), s->sms, true, false, y.fold > 1 ? y.Nw : 0);
      y.bn_fwd = f.bn; y.pair_fwd = f.pair;
      y.bn_dgrad = d.bn; y.pair_dgrad = d.pair;
      // The shared-GPU variants assume kernels long enough to keep the GPU busy; GEMMs of a few microseconds
      // (the 1x1 convolutions of a ResNet block: 3.3 GFLOP) are launch-bound, the other stream finds the GPU
      // mostly idle and is better off with the stand-alone plan (its full backprop went 0.34 -> 0.41 ms otherwise).
      y.big_gemm = 2.0 * (double)M * y.K * y.N >= 10e9;
      const TilePlan dsh = y.big_gemm ? choose_tiles((int)M, y.K, kb_n, s->sms, false, true, 0, true) : d;
      y.bn_dgrad_sh = dsh.bn; y.pair_dgrad_sh = dsh.pair;
      y.bn_wgrad = w.bn; y.pair_wgrad = w.pair; y.split = w.split;
      // One-launch backward: units of all GEMMs share the CTAs, so a weight gradient need not fill the GPU by
      // itself.  Splits of about 32 k-blocks for small tensors (units of a size with the error-gradient tiles),
      // fewer for large ones: every split writes and re-reads 4 bytes per parameter (at most 24 MB per tensor).
      y.list_ok = y.kind == ET_LAYER_DENSE && y.K % 64 == 0 && y.Nw % 64 == 0;
      if (y.list_ok) {
        const int kb = ceil_div(M, et::tc::BK);
        int sp = std::max(1, std::min(8, kb / 32));
        while (sp > 1 && (double)sp * y.K * y.N * 4.0 > 24e6) --sp;
        while (sp > 1 && (long long)(sp - 1) * ceil_div(kb, sp) >= kb) --sp;
        y.split_list = sp;
      }
#ifdef ET_DEBUG_HOOKS
      if (const char* force = getenv("ET_DEBUG_TILES")) {          // debug builds only: "<bn>,<pair>[,<split>]" for every GEMM
        int fb = 0, fp = 0, fs = 0;
        if (sscanf(force, "%d,%d,%d", &fb, &fp, &fs) >= 2 && (fb == 128 || fb == 192 || fb == 256)) {
          y.bn_dgrad = fb; y.pair_dgrad = fp != 0;
          y.bn_dgrad_sh = fb; y.pair_dgrad_sh = fp != 0;
          const int fbm = (fb == 192) ? 256 : fb;                   // MN-major B has no 192-wide pair tile
          y.bn_fwd = fp ? fbm : fb; y.pair_fwd = fp != 0;
          if (y.fold == 1 || y.Nw % (fp ? fbm : fb) == 0) { y.bn_wgrad = fp ? fbm : fb; y.pair_wgrad = fp != 0; }
          if (fs > 0) y.split = std::min(fs, ceil_div(M, et::tc::BK));
        }
      }
#endif
    }
    if (!y.trainable()) {                                  // no tensors: no partials, no importance slots
      y.imp_count_w = y.imp_count_b = 0;
      s->imp_offs[2 * l] = s->imp_offs[2 * l + 1] = imp_total;
      s->imp_counts[2 * l] = s->imp_counts[2 * l + 1] = 0;
      continue;
    }
    // Weight gradients that run persistently beside the error-gradient chain (dense masks) need not fill the
    // GPU by themselves: at most two splits keep the partial-sum traffic and the reducers small, the chain
    // takes the SMs they leave free (ViT-B full backprop 4.33 -> 4.02 ms; "as many splits as give every SM
    // pair a unit" gave 4.23 ms, a single split 4.59 ms).
    y.split_shared = y.split;
    bool forced_tiles = false;
#ifdef ET_DEBUG_HOOKS
    forced_tiles = getenv("ET_DEBUG_TILES") != nullptr;
#endif
    if (y.kind == ET_LAYER_DENSE && dtype == ET_BF16 && y.big_gemm && !forced_tiles) {
      const int kb = ceil_div(M, et::tc::BK);
      int sp = std::min(y.split, 2);
      while (sp > 1 && (long long)(sp - 1) * ceil_div(kb, sp) >= kb) --sp;
      y.split_shared = sp;
    }
    max_partial = std::max(max_partial, y.vector_params() ? (size_t)y.N * sizeof(float)
                                                          : (size_t)std::max(y.split, y.split_shared) * y.K * y.N * sizeof(float));
    y.off_biaspart = take((size_t)std::max(chunks, ceil_div(M, 256) * 8 + 8) * y.Nw * sizeof(float));
    if (y.list_ok) y.off_partial_list = take((size_t)y.split_list * y.K * y.N * sizeof(float));
    y.imp_count_w = y.vector_params() ? ceil_div(y.N, et::kBiasCols)
                                            : ceil_div((long long)y.K * y.N, et::kEltThreads * et::kVec);
    y.imp_count_b = ceil_div(y.N, et::kBiasCols);
    s->imp_offs[2 * l] = imp_total; s->imp_counts[2 * l] = y.imp_count_w; imp_total += y.imp_count_w;
    s->imp_offs[2 * l + 1] = imp_total; s->imp_counts[2 * l + 1] = y.imp_count_b; imp_total += y.imp_count_b;
  }
  s->imp_total = imp_total;
  s->off_partial = take(max_partial);
  s->off_imp_parts = take((size_t)imp_total * sizeof(float));
  s->off_imp_offs = take((size_t)2 * L * sizeof(int));
  s->off_imp_counts = take((size_t)2 * L * sizeof(int));
  const size_t out_count = (size_t)M * s->out_width();
  s->off_loss_parts = take((size_t)ceil_div(out_count, et::kEltThreads * et::kVec) * sizeof(float));
  s->off_dy_stage = take(out_count * s->elt);
  s->off_imp_stage = take((size_t)2 * L * sizeof(float));
  if (dtype == ET_BF16) {
    s->off_tasks = take((size_t)2 * L * sizeof(et::tl::Task));
    s->off_ftasks = take((size_t)L * sizeof(et::tl::Task));
    s->max_counters = L * (ceil_div(M, 2 * et::tc::BM) + 1);
    s->off_counters = take((size_t)s->max_counters * sizeof(unsigned));
    s->off_rtab = take((size_t)L * sizeof(et::ReduceEntry));
    s->off_btab = take((size_t)L * sizeof(et::BiasEntry));
  }
  s->ws_bytes = off;
  *out = s;
  return ET_OK;
}

et_status et_stack_destroy(et_stack* s) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  et_timing_enable(s, 0);
  destroy_two_streams(s);
  delete s;
  return ET_OK;
}

et_status et_stack_set_option(et_stack* s, int32_t option, int32_t value) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  switch (option) {
    case ET_OPTION_TWO_STREAMS:
      if (value != 0 && value != 1) return ET_ERR_INVALID_ARG;
      s->opt_two_streams = value != 0;
      return ET_OK;
    case ET_OPTION_LAUNCH_OVERLAP:
      if (value != 0 && value != 1) return ET_ERR_INVALID_ARG;
      s->overlap_launch = value != 0;
      return ET_OK;
    case ET_OPTION_TILE_PLAN:
      if (value != ET_TILE_PLAN_AUTO && value != ET_TILE_PLAN_ALONE && value != ET_TILE_PLAN_SHARED) return ET_ERR_INVALID_ARG;
      s->opt_tile_plan = value;
      return ET_OK;
    case ET_OPTION_GEMM_LIST:
      if (value != 0 && value != 1) return ET_ERR_INVALID_ARG;
      s->opt_gemm_list = value != 0;
      return ET_OK;
    case ET_OPTION_LIST_COOPERATIVE:
      if (value != 0 && value != 1) return ET_ERR_INVALID_ARG;
      s->opt_list_cooperative = value != 0;
      return ET_OK;
    default:
      return ET_ERR_INVALID_ARG;
  }
}

et_status et_stack_workspace_bytes(const et_stack* s, size_t* bytes) {
  if (s == nullptr || bytes == nullptr) return ET_ERR_INVALID_ARG;
  *bytes = s->ws_bytes;
  return ET_OK;
}

et_status et_stack_bind(et_stack* s, void* const* W, void* const* b, void* workspace, size_t workspace_bytes,
                        void* stream) {
  if (s == nullptr || W == nullptr || b == nullptr || workspace == nullptr) return ET_ERR_INVALID_ARG;
  if (workspace_bytes < s->ws_bytes || ((uintptr_t)workspace & 255) != 0) return ET_ERR_WORKSPACE;
  for (int l = 0; l < s->L; ++l) {
    if (!s->ly[l].trainable()) continue;                  // no tensors: its pointers are ignored
    if (W[l] == nullptr || b[l] == nullptr || ((uintptr_t)W[l] & 15) || ((uintptr_t)b[l] & 15)) return ET_ERR_INVALID_ARG;
  }
  cudaStream_t st = (cudaStream_t)stream;
  s->bound = false;
  s->ws = (char*)workspace;
  for (int l = 0; l < s->L; ++l) { s->ly[l].W = W[l]; s->ly[l].b = b[l]; s->ly[l].W32 = nullptr; s->ly[l].b32 = nullptr;
    for (int k = 0; k < 2; ++k) { s->ly[l].st1[k] = nullptr; s->ly[l].st2[k] = nullptr; } }
  s->opt_cfg = {ET_OPT_SGD, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (s->dtype == ET_BF16) {
    for (int l = 0; l < s->L; ++l) {
      LayerRT& y = s->ly[l];
      if (y.kind == ET_LAYER_DENSE) {
        ET_TRY(make_tmaps(&y.map_W, y.W, y.N, y.K));
        ET_TRY(make_map(&y.map_Wd, y.W, y.N, y.K, y.pair_dgrad ? y.bn_dgrad / 2 : y.bn_dgrad));
        ET_TRY(make_map(&y.map_Wd_sh, y.W, y.N, y.K, y.pair_dgrad_sh ? y.bn_dgrad_sh / 2 : y.bn_dgrad_sh));
        if (y.list_ok) ET_TRY(make_map(&y.map_Wd_list, y.W, y.N, y.K, et::tl::LBNH));
      }
      if (l < s->L - 1 && !y.implicit) {
        ET_TRY(make_tmaps(&y.map_aout, s->at(y.off_a_out), y.Nw, s->M));
        ET_TRY(make_tmaps(&y.map_Gout, s->at(y.off_G_out), y.Nw, s->M));
      }
      y.im_in_ptr = nullptr; y.im_dg_ptr = nullptr;
      if (y.kind == ET_LAYER_DENSE && l >= 1 && s->ly[l - 1].implicit) ET_TRY(make_map(&y.map_Wd_conv, y.W, y.N, y.K, 128));
      if (y.act != ET_ACT_NONE) {
        ET_TRY(make_tmaps(&y.map_Z, s->at(y.off_Z), y.Nw, s->M));
        ET_TRY(make_tmaps(&y.map_dZ, s->at(y.off_dZ), y.Nw, s->M));
      }
    }
  }
  CU_TRY(cudaMemsetAsync(s->at(s->off_status), 0, 256, st));
  for (size_t g : s->guards) CU_TRY(cudaMemsetAsync(s->at(g), kGuardByte, kGuardBytes, st));
  CU_TRY(cudaMemcpyAsync(s->at(s->off_imp_offs), s->imp_offs.data(), sizeof(int) * 2 * s->L, cudaMemcpyHostToDevice, st));
  CU_TRY(cudaMemcpyAsync(s->at(s->off_imp_counts), s->imp_counts.data(), sizeof(int) * 2 * s->L, cudaMemcpyHostToDevice, st));
  CU_TRY(cudaStreamSynchronize(st));     // the host vectors may be freed / changed afterwards
  ++s->bind_serial;                      // device tables of the one-launch backward are rebuilt on next use
  s->tasks_key.clear();
  s->ftasks_key.clear();
  s->rtab_host.clear();
  s->btab_host.clear();
  s->bound = true;
  s->forwarded = false;
  s->map_dy_ptr = nullptr;
  s->map_y_ptr = nullptr;
  s->x = nullptr;
  return ET_OK;
}

et_status et_stack_bind_master(et_stack* s, float* const* W32, float* const* b32) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  if (s->dtype != ET_BF16) return ET_ERR_DTYPE;
  if ((W32 == nullptr) != (b32 == nullptr)) return ET_ERR_INVALID_ARG;
  if (W32 != nullptr)
    for (int l = 0; l < s->L; ++l)
      if (s->ly[l].trainable() &&
          (W32[l] == nullptr || b32[l] == nullptr || ((uintptr_t)W32[l] & 15) || ((uintptr_t)b32[l] & 15)))
        return ET_ERR_INVALID_ARG;
  for (int l = 0; l < s->L; ++l) {
    s->ly[l].W32 = W32 ? W32[l] : nullptr;
    s->ly[l].b32 = b32 ? b32[l] : nullptr;
  }
  ++s->bind_serial;                      // task lists hold these pointers
  return ET_OK;
}

et_status et_forward_stack(et_stack* s, const void* x, void* y, void* stream) {
  if (s == nullptr || x == nullptr || y == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  if (((uintptr_t)x & 15) || ((uintptr_t)y & 15)) return ET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  return s->dtype == ET_BF16 ? forward_impl<bf16>(s, x, y, st) : forward_impl<float>(s, x, y, st);
}

et_status et_loss_mse_grad(et_stack* s, const void* y, const void* target, void* dY, float* loss_dev, void* stream) {
  if (s == nullptr || y == nullptr || target == nullptr || dY == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t count = (size_t)s->M * s->out_width();
  const int blocks = ceil_div(count, et::kEltThreads * et::kVec);
  float* parts = (float*)s->at(s->off_loss_parts);
  const float scale = (float)(2.0 / (double)count);
  if (s->dtype == ET_BF16)
    et::mse_grad_kernel<bf16><<<blocks, et::kEltThreads, 0, st>>>((const bf16*)y, (const bf16*)target, (bf16*)dY, count, scale, parts);
  else
    et::mse_grad_kernel<float><<<blocks, et::kEltThreads, 0, st>>>((const float*)y, (const float*)target, (float*)dY, count, scale, parts);
  ET_TRY(after_launch());
  if (loss_dev != nullptr) {
    et::loss_finalize_kernel<<<1, 256, 0, st>>>(parts, blocks, (float)(1.0 / (double)count), loss_dev);
    ET_TRY(after_launch());
  }
  return ET_OK;
}

et_status et_backward_elastic(et_stack* s, const void* dY, const uint8_t* mask, int32_t n_tensors,
                              float* const* grads, const void* const* delta, float* importance_dev,
                              uint32_t flags, float lr, et_exec_report* report, void* stream) {
  ET_TRY(validate_backward_args(s, dY, mask, n_tensors, delta, importance_dev));
  if ((uintptr_t)dY & 15) return ET_ERR_INVALID_ARG;
  if (flags & ~(uint32_t)(ET_FLAG_FUSE_SGD | ET_FLAG_DELTA_IS_SNAPSHOT)) return ET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  return s->dtype == ET_BF16
             ? backward_impl<bf16>(s, dY, mask, grads, delta, importance_dev, flags, lr, report, st)
             : backward_impl<float>(s, dY, mask, grads, delta, importance_dev, flags, lr, report, st);
}

et_status et_backward_elastic_host(et_stack* s, const void* dY_host, const uint8_t* mask, int32_t n_tensors,
                                   float* const* grads, const void* const* delta, float* importance_host,
                                   uint32_t flags, float lr, et_exec_report* report, void* stream) {
  ET_TRY(validate_backward_args(s, dY_host, mask, n_tensors, delta, importance_host));
  if (flags & ~(uint32_t)(ET_FLAG_FUSE_SGD | ET_FLAG_DELTA_IS_SNAPSHOT)) return ET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  void* dY = s->at(s->off_dy_stage);
  float* imp = (float*)s->at(s->off_imp_stage);
  CU_TRY(cudaMemcpyAsync(dY, dY_host, (size_t)s->M * s->out_width() * s->elt, cudaMemcpyHostToDevice, st));
  et_status r = s->dtype == ET_BF16
                    ? backward_impl<bf16>(s, dY, mask, grads, delta, imp, flags, lr, report, st)
                    : backward_impl<float>(s, dY, mask, grads, delta, imp, flags, lr, report, st);
  if (r != ET_OK) return r;
  if (delta != nullptr)
    CU_TRY(cudaMemcpyAsync(importance_host, imp, sizeof(float) * 2 * s->L, cudaMemcpyDeviceToHost, st));
  CU_TRY(cudaStreamSynchronize(st));
  return ET_OK;
}

et_status et_importance(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads,
                        const void* const* delta, float* importance_dev, void* stream) {
  ET_TRY(check_ready(s, mask, n_tensors));
  if (grads == nullptr || delta == nullptr || importance_dev == nullptr) return ET_ERR_INVALID_ARG;
  for (int t = 0; t < n_tensors; ++t)
    if (mask[t] && (grads[t] == nullptr || delta[t] == nullptr)) return ET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  float* parts = (float*)s->at(s->off_imp_parts);
  for (int t = 0; t < n_tensors; ++t) {
    if (!mask[t]) continue;
    const LayerRT& y = s->ly[t / 2];
    const bool is_w = (t & 1) == 0;
    const size_t count = is_w ? y.w_count() : (size_t)y.N;
    const int blocks = s->imp_counts[t];
    float* out = parts + s->imp_offs[t];
    const bool wide = is_w && !y.vector_params();           // 8 elements per thread; gamma goes like a bias
    if (s->dtype == ET_BF16) {
      if (wide) et::importance_kernel<bf16, 8><<<blocks, et::kEltThreads, 0, st>>>(grads[t], (const bf16*)delta[t], count, out);
      else      et::importance_kernel<bf16, 1><<<blocks, et::kEltThreads, 0, st>>>(grads[t], (const bf16*)delta[t], count, out);
    } else {
      if (wide) et::importance_kernel<float, 8><<<blocks, et::kEltThreads, 0, st>>>(grads[t], (const float*)delta[t], count, out);
      else      et::importance_kernel<float, 1><<<blocks, et::kEltThreads, 0, st>>>(grads[t], (const float*)delta[t], count, out);
    }
    ET_TRY(after_launch());
  }
  et::importance_finalize_kernel<<<n_tensors, 128, 0, st>>>(parts, (const int*)s->at(s->off_imp_offs),
                                                            (const int*)s->at(s->off_imp_counts),
                                                            mask_bits(mask, n_tensors), importance_dev);
  return after_launch();
}

et_status et_tensor_metric(et_stack* s, const uint8_t* mask, int32_t n_tensors, int32_t kind, float* const* grads,
                           float* metric_dev, void* stream) {
  ET_TRY(check_ready(s, mask, n_tensors));
  if (metric_dev == nullptr) return ET_ERR_INVALID_ARG;
  if (kind != ET_METRIC_WEIGHT_MAGNITUDE && kind != ET_METRIC_GRADIENT_MAGNITUDE) return ET_ERR_INVALID_ARG;
  if (kind == ET_METRIC_GRADIENT_MAGNITUDE) {
    if (grads == nullptr) return ET_ERR_INVALID_ARG;
    for (int t = 0; t < n_tensors; ++t)
      if (mask[t] && grads[t] == nullptr) return ET_ERR_INVALID_ARG;
  }
  cudaStream_t st = (cudaStream_t)stream;
  float* parts = (float*)s->at(s->off_imp_parts);
  for (int t = 0; t < n_tensors; ++t) {
    if (!mask[t]) continue;
    const LayerRT& y = s->ly[t / 2];
    const bool is_w = (t & 1) == 0;
    const size_t count = is_w ? y.w_count() : (size_t)y.N;
    const int blocks = s->imp_counts[t];
    float* out = parts + s->imp_offs[t];
    const bool wide = is_w && !y.vector_params();
    const float* f32 = kind == ET_METRIC_GRADIENT_MAGNITUDE ? grads[t] : (is_w ? y.W32 : y.b32);   // masters if attached
    const void* stored = is_w ? y.W : y.b;
    if (f32 != nullptr || s->dtype == ET_F32) {
      const float* p = f32 != nullptr ? f32 : (const float*)stored;
      if (wide) et::abs_sum_kernel<float, 8><<<blocks, et::kEltThreads, 0, st>>>(p, count, out);
      else      et::abs_sum_kernel<float, 1><<<blocks, et::kEltThreads, 0, st>>>(p, count, out);
    } else {
      if (wide) et::abs_sum_kernel<bf16, 8><<<blocks, et::kEltThreads, 0, st>>>((const bf16*)stored, count, out);
      else      et::abs_sum_kernel<bf16, 1><<<blocks, et::kEltThreads, 0, st>>>((const bf16*)stored, count, out);
    }
    ET_TRY(after_launch());
  }
  et::importance_finalize_kernel<<<n_tensors, 128, 0, st>>>(parts, (const int*)s->at(s->off_imp_offs),
                                                            (const int*)s->at(s->off_imp_counts),
                                                            mask_bits(mask, n_tensors), metric_dev);
  return after_launch();
}

namespace {
et_status update_masked_impl(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads, float lr,
                             void* stream, bool plain) {
  ET_TRY(check_ready(s, mask, n_tensors));
  if (grads == nullptr) return ET_ERR_INVALID_ARG;
  for (int t = 0; t < n_tensors; ++t)
    if (mask[t] && grads[t] == nullptr) return ET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const et::OptParams o = opt_params(s, lr, plain);
  for (int t = 0; t < n_tensors; ++t) {
    if (!mask[t]) continue;
    const LayerRT& y = s->ly[t / 2];
    const bool is_w = (t & 1) == 0;
    const size_t count = is_w ? y.w_count() : (size_t)y.N;
    void* w = is_w ? y.W : y.b;
    float* m = is_w ? y.W32 : y.b32;
    float* s1 = y.st1[t & 1];
    float* s2 = y.st2[t & 1];
    const int blocks = ceil_div(count, et::kEltThreads * et::kVec);
    if (s->dtype == ET_BF16) et::sgd_kernel<bf16><<<blocks, et::kEltThreads, 0, st>>>((bf16*)w, grads[t], count, o, m, s1, s2);
    else                     et::sgd_kernel<float><<<blocks, et::kEltThreads, 0, st>>>((float*)w, grads[t], count, o, m, s1, s2);
    ET_TRY(after_launch());
  }
  return ET_OK;
}
}  // namespace

et_status et_sgd_masked(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads, float lr,
                        void* stream) {
  return update_masked_impl(s, mask, n_tensors, grads, lr, stream, true);
}

et_status et_update_masked(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads, float lr,
                           void* stream) {
  return update_masked_impl(s, mask, n_tensors, grads, lr, stream, false);
}

et_status et_stack_set_optimizer(et_stack* s, const et_optimizer_config* cfg, float* const* state1,
                                 float* const* state2) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  et_optimizer_config c = {ET_OPT_SGD, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (cfg != nullptr) c = *cfg;
  if (c.kind != ET_OPT_SGD && c.kind != ET_OPT_SGDW && c.kind != ET_OPT_ADAM) return ET_ERR_INVALID_ARG;
  if (c.kind != ET_OPT_SGD && state1 == nullptr) return ET_ERR_INVALID_ARG;
  if (c.kind == ET_OPT_ADAM && state2 == nullptr) return ET_ERR_INVALID_ARG;
  if (c.kind == ET_OPT_ADAM && !(c.beta1 >= 0.f && c.beta1 < 1.f && c.beta2 >= 0.f && c.beta2 < 1.f && c.eps > 0.f))
    return ET_ERR_INVALID_ARG;
  const int n = 2 * s->L;
  for (int t = 0; t < n; ++t) {
    if (!s->ly[t / 2].trainable()) continue;
    if (c.kind != ET_OPT_SGD && (state1[t] == nullptr || ((uintptr_t)state1[t] & 15))) return ET_ERR_INVALID_ARG;
    if (c.kind == ET_OPT_ADAM && (state2[t] == nullptr || ((uintptr_t)state2[t] & 15))) return ET_ERR_INVALID_ARG;
  }
  for (int t = 0; t < n; ++t) {
    s->ly[t / 2].st1[t & 1] = c.kind != ET_OPT_SGD ? state1[t] : nullptr;
    s->ly[t / 2].st2[t & 1] = c.kind == ET_OPT_ADAM ? state2[t] : nullptr;
  }
  s->opt_cfg = c;
  s->opt_step = 1;
  s->opt_wd_now = c.weight_decay;
  ++s->bind_serial;                      // task lists hold the state pointers
  return ET_OK;
}

et_status et_stack_set_optimizer_step(et_stack* s, int32_t step, float weight_decay) {
  if (s == nullptr || step < 1 || !(weight_decay >= 0.f)) return ET_ERR_INVALID_ARG;
  s->opt_step = step;
  s->opt_wd_now = weight_decay;
  return ET_OK;
}

et_status et_profile_costs(et_stack* s, const void* x, void* y, const void* dY, int32_t iters, double* t_dw,
                           double* t_dy, double* t_fwd, void* stream) {
  if (s == nullptr || x == nullptr || y == nullptr || dY == nullptr || t_dw == nullptr || t_dy == nullptr ||
      iters < 1 || iters > 10000)
    return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const int L = s->L;
  cudaEvent_t e0, e1;
  CU_TRY(cudaEventCreate(&e0));
  CU_TRY(cudaEventCreate(&e1));
  et_status rc = ET_OK;
  std::vector<float> ts;
  auto timed = [&](auto&& fn, double* out) -> et_status {
    ts.clear();
    for (int it = 0; it < iters + 1; ++it) {          // first run is a warm-up
      CU_TRY(cudaEventRecord(e0, st));
      ET_TRY(fn());
      CU_TRY(cudaEventRecord(e1, st));
      CU_TRY(cudaEventSynchronize(e1));
      float ms = 0.f;
      CU_TRY(cudaEventElapsedTime(&ms, e0, e1));
      if (it > 0) ts.push_back(ms);
    }
    *out = median(ts);
    return ET_OK;
  };
  auto body = [&]() -> et_status {
    double fwd = 0.0;
    ET_TRY(timed([&]() { return et_forward_stack(s, x, y, stream); }, &fwd));
    if (t_fwd != nullptr) *t_fwd = fwd;
    std::vector<uint8_t> ones(2 * L, 1);
    for (int l = 0; l < L; ++l)
      if (!s->ly[l].trainable()) ones[2 * l] = ones[2 * l + 1] = 0;
    ET_TRY(et_backward_elastic(s, dY, ones.data(), 2 * L, nullptr, nullptr, nullptr, 0, 0.f, nullptr, stream));
    s->chain_shares_gpu = false;                              // the launches below run one at a time
    s->shared_plan = false;
    s->wgrad_one_unit = false;
    float* scratch_grad = (float*)s->at(s->off_partial);      // in-place: each element is read before it is written
    double pending_nontrainable = 0.0;
    for (int l = L - 1; l >= 0; --l) {
      int dummy = 0;
      t_dy[2 * l] = 0.0; t_dy[2 * l + 1] = 0.0;
      if (!s->ly[l].trainable()) {
        // Section 5.3: a non-trainable layer's backward time joins t_dy of the closest tensor of the
        // trainable layer below it (that layer's bias)
        t_dw[2 * l] = 0.0; t_dw[2 * l + 1] = 0.0;
        double t_attn = 0.0;
        if (l >= 1) {
          if (s->ly[l].kind == ET_LAYER_ATTENTION) ET_TRY(timed([&]() { return run_attn_backward(s, l, dY, st); }, &t_attn));
          else if (s->ly[l].implicit) t_attn = 0.0;       // part of the error-gradient GEMM of the layer above
          else if (s->dtype == ET_BF16) ET_TRY(timed([&]() { return run_im2col_backward<bf16>(s, l, dY, st); }, &t_attn));
          else ET_TRY(timed([&]() { return run_im2col_backward<float>(s, l, dY, st); }, &t_attn));
        }
        pending_nontrainable += t_attn;
        continue;
      }
      const double carried = pending_nontrainable;
      pending_nontrainable = 0.0;
      struct AddCarried {
        double* slot; double v;
        ~AddCarried() { *slot += v; }
      } add_carried{&t_dy[2 * l + 1], carried};
      if (s->ly[l].kind == ET_LAYER_BATCHNORM) {
        // Section 5.2, its own subject: one black box, all of its backward time in t_dy of beta
        t_dw[2 * l] = 0.0; t_dw[2 * l + 1] = 0.0;
        double t_box = 0.0, t_beta = 0.0;
        if (s->dtype == ET_BF16) {
          ET_TRY(timed([&]() { return run_bn_backward<bf16>(s, l, dY, l >= 1, true, scratch_grad, nullptr, false, 0.f, &dummy, st); }, &t_box));
          ET_TRY(timed([&]() { return run_bgrad_layer<bf16>(s, l, dY, nullptr, nullptr, false, 0.f, &dummy, st); }, &t_beta));
        } else {
          ET_TRY(timed([&]() { return run_bn_backward<float>(s, l, dY, l >= 1, true, scratch_grad, nullptr, false, 0.f, &dummy, st); }, &t_box));
          ET_TRY(timed([&]() { return run_bgrad_layer<float>(s, l, dY, nullptr, nullptr, false, 0.f, &dummy, st); }, &t_beta));
        }
        t_dy[2 * l + 1] = t_box + t_beta;
        continue;
      }
      if (s->ly[l].kind == ET_LAYER_NORM) {
        // Section 5.2: the layer is one black box whose whole backward time belongs to t_dy of beta
        t_dw[2 * l] = 0.0; t_dw[2 * l + 1] = 0.0;
        double t_box = 0.0, t_beta = 0.0;
        if (s->dtype == ET_BF16) {
          ET_TRY(timed([&]() { return run_norm_backward<bf16>(s, l, dY, l >= 1, true, scratch_grad, nullptr, false, 0.f, &dummy, st); }, &t_box));
          ET_TRY(timed([&]() { return run_bgrad_layer<bf16>(s, l, dY, nullptr, nullptr, false, 0.f, &dummy, st); }, &t_beta));
        } else {
          ET_TRY(timed([&]() { return run_norm_backward<float>(s, l, dY, l >= 1, true, scratch_grad, nullptr, false, 0.f, &dummy, st); }, &t_box));
          ET_TRY(timed([&]() { return run_bgrad_layer<float>(s, l, dY, nullptr, nullptr, false, 0.f, &dummy, st); }, &t_beta));
        }
        t_dy[2 * l + 1] = t_box + t_beta;
        continue;
      }
      if (s->dtype == ET_BF16) {
        if (l >= 1) ET_TRY(timed([&]() { return run_dgrad_layer<bf16>(s, l, dY, st); }, &t_dy[2 * l]));
        ET_TRY(timed([&]() { return run_wgrad_layer<bf16>(s, l, dY, scratch_grad, nullptr, false, 0.f, &dummy, st); }, &t_dw[2 * l]));
        ET_TRY(timed([&]() { return run_bgrad_layer<bf16>(s, l, dY, nullptr, nullptr, false, 0.f, &dummy, st); }, &t_dw[2 * l + 1]));
      } else {
        if (l >= 1) ET_TRY(timed([&]() { return run_dgrad_layer<float>(s, l, dY, st); }, &t_dy[2 * l]));
        ET_TRY(timed([&]() { return run_wgrad_layer<float>(s, l, dY, scratch_grad, nullptr, false, 0.f, &dummy, st); }, &t_dw[2 * l]));
        ET_TRY(timed([&]() { return run_bgrad_layer<float>(s, l, dY, nullptr, nullptr, false, 0.f, &dummy, st); }, &t_dw[2 * l + 1]));
      }
    }
    return ET_OK;
  };
  rc = body();
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  return rc;
}

et_status et_timing_enable(et_stack* s, int32_t on) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  s->timing = on != 0;
  if (!s->timing) {
    for (auto& t : s->timed) { cudaEventDestroy(t.e0); cudaEventDestroy(t.e1); }
    for (auto e : s->event_pool) cudaEventDestroy(e);
    s->timed.clear();
    s->event_pool.clear();
  }
  return ET_OK;
}

et_status et_timing_read(et_stack* s, double* ms, int64_t* launches) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  for (int c = 0; c < ET_K_CLASSES; ++c) {
    if (ms) ms[c] = 0.0;
    if (launches) launches[c] = 0;
  }
  et_status rc = ET_OK;
  for (auto& t : s->timed) {
    float v = 0.f;
    if (cudaEventSynchronize(t.e1) != cudaSuccess || cudaEventElapsedTime(&v, t.e0, t.e1) != cudaSuccess) {
      g_last_cuda = (int)cudaGetLastError();
      rc = ET_ERR_CUDA;
    } else {
      if (ms) ms[t.cls] += v;
      if (launches) launches[t.cls] += 1;
    }
    s->event_pool.push_back(t.e0);
    s->event_pool.push_back(t.e1);
  }
  s->timed.clear();
  return rc;
}

et_status et_debug_guard_regions(int32_t on) {
  g_guard_regions.store(on != 0 ? 1 : 0);
  return ET_OK;
}

et_status et_debug_check_guards(et_stack* s, void* stream, int32_t* first_bad_region) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  if (first_bad_region != nullptr) *first_bad_region = -1;
  if (s->guards.empty()) return ET_OK;
  cudaStream_t st = (cudaStream_t)stream;
  std::vector<unsigned char> host(s->guards.size() * kGuardBytes);
  for (size_t i = 0; i < s->guards.size(); ++i)
    CU_TRY(cudaMemcpyAsync(host.data() + i * kGuardBytes, s->at(s->guards[i]), kGuardBytes, cudaMemcpyDeviceToHost, st));
  CU_TRY(cudaStreamSynchronize(st));
  for (size_t i = 0; i < host.size(); ++i)
    if (host[i] != kGuardByte) {
      if (first_bad_region != nullptr) *first_bad_region = (int32_t)(i / kGuardBytes);
      return ET_ERR_GUARD;
    }
  return ET_OK;
}

et_status et_device_status(et_stack* s, void* stream) {
  if (s == nullptr) return ET_ERR_INVALID_ARG;
  if (!s->bound) return ET_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t word = 0;
  CU_TRY(cudaMemcpyAsync(&word, s->at(s->off_status), sizeof(word), cudaMemcpyDeviceToHost, st));
  CU_TRY(cudaStreamSynchronize(st));
  return word == 0 ? ET_OK : ET_ERR_TIMEOUT;
}

const char* et_status_string(et_status st) {
  switch (st) {
    case ET_OK: return "ok";
    case ET_ERR_INVALID_ARG: return "invalid argument";
    case ET_ERR_SHAPE: return "layer shapes do not chain";
    case ET_ERR_DTYPE: return "unknown dtype";
    case ET_ERR_STATE: return "call out of order (bind / forward first)";
    case ET_ERR_WORKSPACE: return "workspace too small or misaligned";
    case ET_ERR_UNSUPPORTED: return "shape not supported by the kernels";
    case ET_ERR_CUDA: return "CUDA call failed";
    case ET_ERR_TIMEOUT: return "device-side wait timed out";
    case ET_ERR_TOO_LARGE: return "problem exceeds the built-in scratch capacity of the no-allocation call";
    case ET_ERR_GUARD: return "a guard word after a workspace region was overwritten";
  }
  return "unknown status";
}

int32_t et_last_cuda_error(void) { return g_last_cuda; }
int64_t et_launch_count(void) { return (int64_t)g_launches.load(); }

}  // extern "C"
