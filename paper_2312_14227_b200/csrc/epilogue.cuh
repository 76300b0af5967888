// Epilogue functors shared by the tensor-core and the SIMT GEMM kernels.
// Each is called with NV consecutive accumulator values of one output row:
//   op(row, col0, n_valid, v)   -- n_valid < NV only at the ragged right edge.
#pragma once

#include "common.cuh"

namespace et {

// Forward: Z = acc + b (bias summed over the fold slices), optional save of Z,
// H = act(Z), optional residual add, store a_{l+1}.
template <typename T>
struct FwdEpi {
  const T* bias;     // [fold * ld]
  int fold;
  T* Z;              // [M x ld] or nullptr (only layers with an activation keep Z)
  int act;
  const T* resid;    // a_j [M x ld] or nullptr
  T* out;            // a_{l+1} [M x ld]
  int ld;            // out_features / fold

  template <int NV>
  __device__ __forceinline__ void operator()(int row, int col0, int n, float (&v)[NV]) const {
    float t[NV];
    for (int s = 0; s < fold; ++s) {
      load_seg<NV>(bias + (size_t)s * ld + col0, n, t);
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] += t[i];
    }
    const size_t off = (size_t)row * ld + col0;
    if (Z != nullptr) store_seg<NV>(Z + off, n, v);
    if (act != kActNone) {
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] = act_apply(v[i], act);
    }
    if (resid != nullptr) {
      load_seg<NV>(resid + off, n, t);
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] += t[i];
    }
    store_seg<NV>(out + off, n, v);
  }
};

// Error-gradient pass of layer l: G_l = acc + (gradient arriving over the skip connection),
// then through the non-trainable work below it: dZ_{l-1} = G_l * act'(Z_{l-1}).
template <typename T>
struct DgradEpi {
  const T* skip;     // [M x ld] or nullptr
  const T* Zprev;    // [M x ld] or nullptr (layer l-1 has no activation)
  int act_prev;
  T* outG;           // G_l, or nullptr when only dZ_{l-1} is needed
  T* outdZ;          // dZ_{l-1}, or nullptr when it is the same tensor as G_l
  int ld;            // in_features of layer l

  template <int NV>
  __device__ __forceinline__ void operator()(int row, int col0, int n, float (&v)[NV]) const {
    const size_t off = (size_t)row * ld + col0;
    float t[NV];
    if (skip != nullptr) {
      load_seg<NV>(skip + off, n, t);
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] += t[i];
    }
    if (outG != nullptr) store_seg<NV>(outG + off, n, v);
    if (outdZ != nullptr) {
      load_seg<NV>(Zprev + off, n, t);
#pragma unroll
      for (int i = 0; i < NV; ++i) v[i] *= act_grad(t[i], act_prev);
      store_seg<NV>(outdZ + off, n, v);
    }
  }
};

// Weight-gradient partial of one K split: plain fp32 store.
struct PartialEpi {
  float* base;           // [split][rows x ld]
  size_t split_stride;   // rows * ld
  int ld;
  int split;             // set per work unit by the kernel

  template <int NV>
  __device__ __forceinline__ void operator()(int row, int col0, int n, float (&v)[NV]) const {
    store_seg<NV>(base + (size_t)split * split_stride + (size_t)row * ld + col0, n, v);
  }
};

}  // namespace et
