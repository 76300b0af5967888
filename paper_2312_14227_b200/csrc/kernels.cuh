// Memory-bound kernels: split-K reduction with the fused importance / SGD epilogue, bias
// gradient (column sums), stand-alone importance and SGD, activation backward for the top
// layer, MSE loss gradient.  16-byte accesses, fixed-order reductions (results do not
// depend on scheduling).
#pragma once

#include "common.cuh"

namespace et {

constexpr int kEltThreads = 256;
constexpr int kVec = 8;                         // elements per thread per step
constexpr int kColsumRows = 128;                // rows per column-sum chunk

// Optimiser of the masked update (Section 8 of the paper: SGDW for the convolutional models,
// Adam for ViT; plain SGD otherwise).  Schedules live with the caller: lr and wd are this
// step's values.
//   SGD : w <- w - lr g
//   SGDW: m <- momentum m + lr g ;  w <- w - m - wd w            (decoupled weight decay)
//   Adam: m <- b1 m + (1-b1) g ;  v <- b2 v + (1-b2) g^2 ;  w <- w - lr (m c1) / (sqrt(v c2) + eps),
//         c1 = 1 / (1 - b1^t), c2 = 1 / (1 - b2^t)
constexpr int kOptSgd = 0, kOptSgdw = 1, kOptAdam = 2;
struct OptParams {
  int kind;
  float lr;
  float a;       // SGDW: momentum      Adam: beta1
  float b;       // SGDW: weight decay  Adam: beta2
  float eps;     // Adam
  float c1, c2;  // Adam bias corrections
};
__device__ __forceinline__ float opt_update(float w, float g, const OptParams& o, float& m, float& v) {
  if (o.kind == kOptSgdw) {
    m = fmaf(o.a, m, o.lr * g);
    return w - m - o.b * w;
  }
  if (o.kind == kOptAdam) {
    m = fmaf(o.a, m, (1.0f - o.a) * g);
    v = fmaf(o.b, v, (1.0f - o.b) * g * g);
    return w - o.lr * (m * o.c1) / (sqrtf(v * o.c2) + o.eps);
  }
  return fmaf(-o.lr, g, w);
}
// Update of kVec consecutive weights with their state (state pointers may be null for SGD).
__device__ __forceinline__ void opt_update_seg(float (&w)[8], const float (&g)[8], const OptParams& o,
                                               float* m_state, float* v_state, size_t i0, int n) {
  float m[8], v[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { m[i] = 0.0f; v[i] = 0.0f; }
  if (o.kind != kOptSgd) load_seg<8>(m_state + i0, n, m);
  if (o.kind == kOptAdam) load_seg<8>(v_state + i0, n, v);
#pragma unroll
  for (int i = 0; i < 8; ++i) w[i] = opt_update(w[i], g[i], o, m[i], v[i]);
  if (o.kind != kOptSgd) store_seg<8>(m_state + i0, n, m);
  if (o.kind == kOptAdam) store_seg<8>(v_state + i0, n, v);
}

// ---- weight gradient: sum the K-split partials, then everything that consumes g ----------
//   g = sum_s partial[s]                       (fixed order s = 0, 1, ...)
//   grad        <- g                           if grad != nullptr
//   imp_part[b] <- sum over this block of g * dw        if delta != nullptr   (Eq. 2);
//                  dw = delta, or W - delta when delta holds a snapshot of W
//   W           <- optimiser update of W with g if do_sgd   (fp32 arithmetic, one rounding)
//   master != nullptr: the weight lives in fp32 there (W is its rounded copy): the update and
//                  the snapshot difference use it, and a snapshot `delta` is fp32 as well
template <typename T>
__device__ __forceinline__ float wgrad_reduce_elems(size_t i0, const float* partial, int splits, size_t split_stride,
                                                    size_t count, float* grad, const T* __restrict__ delta,
                                                    T* __restrict__ W, const OptParams& opt, int do_sgd,
                                                    int delta_is_snapshot, float* __restrict__ master,
                                                    float* __restrict__ m_state, float* __restrict__ v_state);
template <typename T>
__device__ __forceinline__ void wgrad_reduce_block(int block, const float* partial, int splits, size_t split_stride,
                                                   size_t count, float* grad, const T* __restrict__ delta,
                                                   float* __restrict__ imp_part, T* __restrict__ W, const OptParams& opt,
                                                   int do_sgd, int delta_is_snapshot, float* __restrict__ master,
                                                   float* __restrict__ m_state, float* __restrict__ v_state) {
  const size_t i0 = ((size_t)block * kEltThreads + threadIdx.x) * kVec;
  float dot = 0.0f;
  if (i0 < count)
    dot = wgrad_reduce_elems<T>(i0, partial, splits, split_stride, count, grad, delta, W, opt, do_sgd, delta_is_snapshot,
                                master, m_state, v_state);
  if (delta != nullptr) {
    dot = block_sum(dot);
    if (threadIdx.x == 0) imp_part[block] = dot;
  }
}
// The work on kVec consecutive elements starting at i0 < count; returns their share of sum(g * dw).
template <typename T>
__device__ __forceinline__ float wgrad_reduce_elems(size_t i0, const float* partial, int splits, size_t split_stride,
                                                    size_t count, float* grad, const T* __restrict__ delta,
                                                    T* __restrict__ W, const OptParams& opt, int do_sgd,
                                                    int delta_is_snapshot, float* __restrict__ master,
                                                    float* __restrict__ m_state, float* __restrict__ v_state) {
  float dot = 0.0f;
  {
    const int n = (int)min((size_t)kVec, count - i0);
    float g[kVec], t[kVec], w[kVec];
    load_seg<kVec>(partial + i0, n, g);
    for (int s = 1; s < splits; ++s) {
      load_seg<kVec>(partial + (size_t)s * split_stride + i0, n, t);
#pragma unroll
      for (int i = 0; i < kVec; ++i) g[i] += t[i];
    }
    if (grad != nullptr) store_seg<kVec>(grad + i0, n, g);
    if (do_sgd || (delta != nullptr && delta_is_snapshot)) {      // the current weight is needed
      if (master != nullptr) load_seg<kVec>(master + i0, n, w);
      else load_seg<kVec>(W + i0, n, w);
    }
    if (delta != nullptr) {
      if (delta_is_snapshot) {                        // dw = current weight - weight at the window start
        if (master != nullptr) load_seg<kVec>(reinterpret_cast<const float*>(delta) + i0, n, t);
        else load_seg<kVec>(delta + i0, n, t);
#pragma unroll
        for (int i = 0; i < kVec; ++i) t[i] = w[i] - t[i];
      } else {
        load_seg<kVec>(delta + i0, n, t);
      }
#pragma unroll
      for (int i = 0; i < kVec; ++i) dot = fmaf(g[i], t[i], dot);
    }
    if (do_sgd) {
      opt_update_seg(w, g, opt, m_state, v_state, i0, n);
      if (master != nullptr) store_seg<kVec>(master + i0, n, w);
      store_seg<kVec>(W + i0, n, w);
    }
  }
  return dot;
}
template <typename T>
__global__ void __launch_bounds__(kEltThreads)
wgrad_reduce_kernel(const float* partial, int splits, size_t split_stride, size_t count,
                    float* grad /* may alias partial: each thread reads its elements before writing them */, const T* __restrict__ delta, float* __restrict__ imp_part,
                    T* __restrict__ W, OptParams opt, int do_sgd, int delta_is_snapshot, float* __restrict__ master,
                    float* __restrict__ m_state, float* __restrict__ v_state) {
  wgrad_reduce_block<T>((int)blockIdx.x, partial, splits, split_stride, count, grad, delta, imp_part, W, opt, do_sgd,
                        delta_is_snapshot, master, m_state, v_state);
}

// One launch for every selected kernel tensor of a step: a table in device memory names each tensor's
// partial sums, outputs and first block; a block finds its tensor by binary search and does exactly what
// a wgrad_reduce_kernel block of that tensor does (same elements, same order: results are identical).
struct ReduceEntry {
  const float* partial;
  float* grad;
  const void* delta;
  float* imp_part;
  void* W;
  float* master;
  float* m_state;
  float* v_state;
  unsigned long long count;
  int splits;
  int block_begin;         // first block of this tensor in the grouped grid
};
// The grid is a few blocks per SM; each walks the concatenated block range with the table held in shared
// memory, so that finding a block's tensor costs no chain of global loads.
constexpr int kGroupMax = 128;                          // table entries per launch
constexpr int kGroupBlocksPerSm = 4;                    // resident blocks the grouped reducer is compiled for
template <typename T>
__global__ void __launch_bounds__(kEltThreads, kGroupBlocksPerSm)
wgrad_reduce_group_kernel(const ReduceEntry* __restrict__ tab, int n, int total_blocks, OptParams opt, int do_sgd,
                          int delta_is_snapshot) {
  __shared__ ReduceEntry sh[kGroupMax];
  for (int i = threadIdx.x; i < n * (int)(sizeof(ReduceEntry) / 8); i += blockDim.x)
    reinterpret_cast<unsigned long long*>(sh)[i] = reinterpret_cast<const unsigned long long*>(tab)[i];
  __syncthreads();
  for (int vb = blockIdx.x; vb < total_blocks; vb += gridDim.x) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {                                 // last entry with block_begin <= vb
      const int mid = (lo + hi + 1) >> 1;
      if (sh[mid].block_begin <= vb) lo = mid; else hi = mid - 1;
    }
    const ReduceEntry& e = sh[lo];
    wgrad_reduce_block<T>(vb - e.block_begin, e.partial, e.splits, (size_t)e.count, (size_t)e.count, e.grad,
                          (const T*)e.delta, e.imp_part, (T*)e.W, opt, do_sgd, delta_is_snapshot, e.master, e.m_state,
                          e.v_state);
  }
}

// ---- bias gradient, stage 1: column sums of one chunk of rows ------------------------------
// grid (ceil(width / 256), ceil(M / kColsumRows)); block (32, 8): x -> 8 columns, y -> row phase.
// Each thread keeps four independent 16-byte loads in flight.
template <typename T>
__global__ void __launch_bounds__(256)
colsum_partial_kernel(const T* __restrict__ dZ, int M, int width, float* __restrict__ part) {
  __shared__ float sm[8][256 + 8];
  const int col0 = blockIdx.x * 256 + threadIdx.x * kVec;
  const int r0 = blockIdx.y * kColsumRows;
  const int r1 = min(M, r0 + kColsumRows);
  float acc[kVec];
#pragma unroll
  for (int i = 0; i < kVec; ++i) acc[i] = 0.0f;
  const int n = width - col0;
  if (n > 0) {
    const T* base = dZ + col0;
    int r = r0 + threadIdx.y;
    for (; r + 24 < r1; r += 32) {
      float v[4][kVec];
#pragma unroll
      for (int q = 0; q < 4; ++q) load_seg<kVec>(base + (size_t)(r + 8 * q) * width, n, v[q]);
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int i = 0; i < kVec; ++i) acc[i] += v[q][i];
    }
    for (; r < r1; r += 8) {
      float v[kVec];
      load_seg<kVec>(base + (size_t)r * width, n, v);
#pragma unroll
      for (int i = 0; i < kVec; ++i) acc[i] += v[i];
    }
  }
#pragma unroll
  for (int i = 0; i < kVec; ++i) sm[threadIdx.y][threadIdx.x * kVec + i] = acc[i];
  __syncthreads();
  const int tid = threadIdx.y * 32 + threadIdx.x;      // 256 threads, one column each
  const int col = blockIdx.x * 256 + tid;
  if (col < width) {
    float s = 0.0f;
#pragma unroll
    for (int y = 0; y < 8; ++y) s += sm[y][tid];
    part[(size_t)blockIdx.y * width + col] = s;
  }
}

// ---- bias gradient, stage 2: sum the chunks, then grad / importance / SGD -----------------
// Block (32, 32) handles kBiasCols bias elements j in [0, fold*width): x -> element, y -> which
// chunks (y, y+32, ...) this thread adds (a few independent loads each: the kernel is latency-
// bound); a fixed-order shared-memory sum joins the 32.
// column = j mod width (a folded layer's dZ is the same gradient repeated for each slice).
constexpr int kBiasCols = 32;
constexpr int kBiasLanes = 32;
template <typename T>
__device__ __forceinline__ void bias_finish_block(int block, const float* __restrict__ part, int chunks, int width,
                                                  int count, float* __restrict__ grad, const T* __restrict__ delta,
                                                  float* __restrict__ imp_part, T* __restrict__ b, const OptParams& opt,
                                                  int do_sgd, int delta_is_snapshot, float* __restrict__ master,
                                                  float* __restrict__ m_state, float* __restrict__ v_state) {
  __shared__ float sm[kBiasLanes][kBiasCols + 1];
  const int j = block * kBiasCols + threadIdx.x;
  float g = 0.0f;
  if (j < count) {
    const int col = j % width;
    // four independent chains of loads: the kernel is latency-bound
    float g1 = 0.0f, g2 = 0.0f, g3 = 0.0f;
    int c = threadIdx.y;
    for (; c + 3 * kBiasLanes < chunks; c += 4 * kBiasLanes) {
      g += part[(size_t)c * width + col];
      g1 += part[(size_t)(c + kBiasLanes) * width + col];
      g2 += part[(size_t)(c + 2 * kBiasLanes) * width + col];
      g3 += part[(size_t)(c + 3 * kBiasLanes) * width + col];
    }
    for (; c < chunks; c += kBiasLanes) g += part[(size_t)c * width + col];
    g = (g + g1) + (g2 + g3);
  }
  sm[threadIdx.y][threadIdx.x] = g;
  __syncthreads();
  float dot = 0.0f;
  if (threadIdx.y == 0) {
    if (j < count) {
      g = 0.0f;
#pragma unroll
      for (int y = 0; y < kBiasLanes; ++y) g += sm[y][threadIdx.x];
      if (grad != nullptr) grad[j] = g;
      float w = 0.0f;
      if (do_sgd || (delta != nullptr && delta_is_snapshot)) w = master != nullptr ? master[j] : to_f32(b[j]);
      if (delta != nullptr) {
        float dw;
        if (delta_is_snapshot)
          dw = w - (master != nullptr ? reinterpret_cast<const float*>(delta)[j] : to_f32(delta[j]));
        else
          dw = to_f32(delta[j]);
        dot = g * dw;
      }
      if (do_sgd) {
        float m = opt.kind != kOptSgd ? m_state[j] : 0.0f;
        float v = opt.kind == kOptAdam ? v_state[j] : 0.0f;
        w = opt_update(w, g, opt, m, v);
        if (opt.kind != kOptSgd) m_state[j] = m;
        if (opt.kind == kOptAdam) v_state[j] = v;
        if (master != nullptr) master[j] = w;
        b[j] = from_f32<T>(w);
      }
    }
    if (delta != nullptr) {                           // one warp: fixed shuffle tree
      dot = warp_sum(dot);
      if (threadIdx.x == 0) imp_part[block] = dot;
    }
  }
}
template <typename T>
__global__ void __launch_bounds__(kBiasCols * kBiasLanes)
bias_finish_kernel(const float* __restrict__ part, int chunks, int width, int count,
                   float* __restrict__ grad, const T* __restrict__ delta, float* __restrict__ imp_part,
                   T* __restrict__ b, OptParams opt, int do_sgd, int delta_is_snapshot, float* __restrict__ master,
                   float* __restrict__ m_state, float* __restrict__ v_state) {
  bias_finish_block<T>((int)blockIdx.x, part, chunks, width, count, grad, delta, imp_part, b, opt, do_sgd,
                       delta_is_snapshot, master, m_state, v_state);
}
// One launch for every selected bias of a step: a table in device memory names each bias's partial sums,
// outputs and first block; a block finds its entry by binary search and does exactly what a
// bias_finish_kernel block of that bias does.
struct BiasEntry {
  const float* part;
  float* grad;
  const void* delta;
  float* imp_part;
  void* b;
  float* master;
  float* m_state;
  float* v_state;
  int chunks, width, count;
  int block_begin;
};
template <typename T>
__global__ void __launch_bounds__(kBiasCols * kBiasLanes)
bias_finish_group_kernel(const BiasEntry* __restrict__ tab, int n, int total_blocks, OptParams opt, int do_sgd,
                         int delta_is_snapshot) {
  __shared__ BiasEntry sh[kGroupMax];
  const int tid = threadIdx.y * blockDim.x + threadIdx.x;
  for (int i = tid; i < n * (int)(sizeof(BiasEntry) / 8); i += blockDim.x * blockDim.y)
    reinterpret_cast<unsigned long long*>(sh)[i] = reinterpret_cast<const unsigned long long*>(tab)[i];
  __syncthreads();
  for (int vb = blockIdx.x; vb < total_blocks; vb += gridDim.x) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sh[mid].block_begin <= vb) lo = mid; else hi = mid - 1;
    }
    const BiasEntry& e = sh[lo];
    bias_finish_block<T>(vb - e.block_begin, e.part, e.chunks, e.width, e.count, e.grad, (const T*)e.delta,
                         e.imp_part, (T*)e.b, opt, do_sgd, delta_is_snapshot, e.master, e.m_state, e.v_state);
    __syncthreads();                                  // the block's shared partials are reused by the next one
  }
}

// ---- importance, last stage: per tensor, sum its block partials in a fixed order ----------
struct MaskBits { uint32_t w[64]; };            // up to 2048 tensors
static __global__ void __launch_bounds__(128)
importance_finalize_kernel(const float* __restrict__ parts, const int* __restrict__ offs,
                           const int* __restrict__ counts, const MaskBits active, float* __restrict__ out) {
  const int t = blockIdx.x;
  float s = 0.0f;
  if ((active.w[t >> 5] >> (t & 31)) & 1u) {
    const int o = offs[t], c = counts[t];
    for (int i = threadIdx.x; i < c; i += blockDim.x) s += parts[o + i];
  }
  s = block_sum(s);
  if (threadIdx.x == 0) out[t] = s;
}

// ---- stand-alone Eq. 2 on a materialised gradient (V elements per thread) ------------------
template <typename T, int V>
__global__ void __launch_bounds__(kEltThreads)
importance_kernel(const float* __restrict__ grad, const T* __restrict__ delta, size_t count,
                  float* __restrict__ imp_part) {
  const size_t i0 = ((size_t)blockIdx.x * kEltThreads + threadIdx.x) * V;
  float dot = 0.0f;
  if (i0 < count) {
    const int n = (int)min((size_t)V, count - i0);
    float g[V], t[V];
    load_seg<V>(grad + i0, n, g);
    load_seg<V>(delta + i0, n, t);
#pragma unroll
    for (int i = 0; i < V; ++i) dot = fmaf(g[i], t[i], dot);
  }
  dot = block_sum(dot);
  if (threadIdx.x == 0) imp_part[blockIdx.x] = dot;
}

// ---- magnitude of one tensor: block partials of sum |x| (V elements per thread) -------------
template <typename T, int V>
__global__ void __launch_bounds__(kEltThreads)
abs_sum_kernel(const T* __restrict__ x, size_t count, float* __restrict__ part) {
  const size_t i0 = ((size_t)blockIdx.x * kEltThreads + threadIdx.x) * V;
  float acc = 0.0f;
  if (i0 < count) {
    const int n = (int)min((size_t)V, count - i0);
    float t[V];
    load_seg<V>(x + i0, n, t);
#pragma unroll
    for (int i = 0; i < V; ++i) acc += fabsf(t[i]);
  }
  acc = block_sum(acc);
  if (threadIdx.x == 0) part[blockIdx.x] = acc;
}

// ---- stand-alone masked SGD on one selected tensor -----------------------------------------
template <typename T>
__global__ void __launch_bounds__(kEltThreads)
sgd_kernel(T* __restrict__ w, const float* __restrict__ grad, size_t count, OptParams opt, float* __restrict__ master,
           float* __restrict__ m_state, float* __restrict__ v_state) {
  const size_t i0 = ((size_t)blockIdx.x * kEltThreads + threadIdx.x) * kVec;
  if (i0 >= count) return;
  const int n = (int)min((size_t)kVec, count - i0);
  float g[kVec], t[kVec];
  load_seg<kVec>(grad + i0, n, g);
  if (master != nullptr) load_seg<kVec>(master + i0, n, t);
  else load_seg<kVec>(w + i0, n, t);
  opt_update_seg(t, g, opt, m_state, v_state, i0, n);
  if (master != nullptr) store_seg<kVec>(master + i0, n, t);
  store_seg<kVec>(w + i0, n, t);
}

// ---- dZ = dY * act'(Z) for a top layer that has an activation -------------------------------
template <typename T>
__global__ void __launch_bounds__(kEltThreads)
act_backward_kernel(const T* __restrict__ dY, const T* __restrict__ Z, T* __restrict__ dZ, size_t count, int act) {
  const size_t i0 = ((size_t)blockIdx.x * kEltThreads + threadIdx.x) * kVec;
  if (i0 >= count) return;
  const int n = (int)min((size_t)kVec, count - i0);
  float g[kVec], z[kVec];
  load_seg<kVec>(dY + i0, n, g);
  load_seg<kVec>(Z + i0, n, z);
#pragma unroll
  for (int i = 0; i < kVec; ++i) g[i] *= act_grad(z[i], act);
  store_seg<kVec>(dZ + i0, n, g);
}

// ---- MSE: dY = 2 (y - t) / count, block partials of (y - t)^2 ---------------------------------
template <typename T>
__global__ void __launch_bounds__(kEltThreads)
mse_grad_kernel(const T* __restrict__ y, const T* __restrict__ target, T* __restrict__ dY, size_t count,
                float scale, float* __restrict__ loss_part) {
  const size_t i0 = ((size_t)blockIdx.x * kEltThreads + threadIdx.x) * kVec;
  float sq = 0.0f;
  if (i0 < count) {
    const int n = (int)min((size_t)kVec, count - i0);
    float a[kVec], t[kVec];
    load_seg<kVec>(y + i0, n, a);
    load_seg<kVec>(target + i0, n, t);
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
      const float d = a[i] - t[i];
      sq = fmaf(d, d, sq);
      a[i] = d * scale;
    }
    store_seg<kVec>(dY + i0, n, a);
  }
  sq = block_sum(sq);
  if (threadIdx.x == 0) loss_part[blockIdx.x] = sq;
}
static __global__ void __launch_bounds__(256)
loss_finalize_kernel(const float* __restrict__ parts, int n, float inv_count, float* __restrict__ loss) {
  float s = 0.0f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) s += parts[i];
  s = block_sum(s);
  if (threadIdx.x == 0) *loss = s * inv_count;
}

}  // namespace et
