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

// ---- staged variants for the tensor-core kernel ---------------------------------------------
// The kernel moves bf16 operand / result chunks through shared memory; combine() sees 32
// consecutive columns of one row: the accumulator, and per slot the input values (on entry)
// which it replaces by the output values (on exit).  has_in / has_out tell the kernel which
// slots to load and store.

// Column sums over a warp's 32 rows: on entry lane r holds 32 consecutive columns of row r; on exit
// lane i's v[0] is the sum over the 32 rows of column i.  31 shuffles (halving exchange).
__device__ __forceinline__ void warp_column_sums(float (&v)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < off; ++k) {
      const float send = upper ? v[k] : v[k + off];
      const float keep = upper ? v[k + off] : v[k];
      v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
}

// Forward.  slot 0: in = residual a_j (optional), out = a_{l+1}.  slot 1 (SLOTS == 2): out = Z.
template <int SLOTS>
struct FwdEpiS {
  static constexpr int kSlots = SLOTS;
  bool has_in[2], has_out[2];
  const bf16* bias;  // [fold * ld]
  int fold, ld, act;

  __device__ __forceinline__ void combine(int col0, int nv, float (&v)[32], float (&s0)[32], float (&s1)[32]) const {
    float t[32];
    for (int s = 0; s < fold; ++s) {
      load_seg<32>(bias + (size_t)s * ld + col0, nv, t);
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] += t[i];
    }
    if constexpr (SLOTS == 2) {
#pragma unroll
      for (int i = 0; i < 32; ++i) s1[i] = v[i];
    }
    const bool res = has_in[0];
#pragma unroll
    for (int i = 0; i < 32; ++i) s0[i] = act_apply_fast(v[i], act) + (res ? s0[i] : 0.0f);
  }
  __device__ __forceinline__ void column_sums(int, int, int, float (&)[32], float (&)[32], int) const {}
};

// Error-gradient pass.  SLOTS == 2: slot 0: in = skip gradient (optional), out = G_l (optional);
// slot 1: in = Z_{l-1}, out = dZ_{l-1} = G_l * act'(Z_{l-1}).
// SLOTS == 1, mul_act == false: in = skip (optional), out = G_l = acc + skip.
// SLOTS == 1, mul_act == true : in = Z_{l-1}, out = dZ_{l-1} = acc * act'(Z_{l-1}).
// colsum != nullptr: the column sums of dZ_{l-1} over each warp's 32 rows are written to
// colsum[row_block][column] as well -- the bias gradient of layer l-1 without re-reading dZ_{l-1}.
template <int SLOTS>
struct DgradEpiS {
  static constexpr int kSlots = SLOTS;
  bool has_in[2], has_out[2];
  bool mul_act;
  int act_prev;
  float* colsum;     // [row blocks of 32][ld] or nullptr
  int ld;

  // s0 / s1 as combine() left them; destroys them.  row_block = (first row of the warp) / 32.
  __device__ __forceinline__ void column_sums(int row_block, int col0, int nv, float (&s0)[32], float (&s1)[32],
                                              int lane) const {
    if (colsum == nullptr) return;
    float (&dz)[32] = SLOTS == 1 ? s0 : s1;
    warp_column_sums(dz, lane);
    if (lane < nv) colsum[(size_t)row_block * ld + col0 + lane] = dz[0];
  }

  __device__ __forceinline__ void combine(int, int, float (&v)[32], float (&s0)[32], float (&s1)[32]) const {
    if constexpr (SLOTS == 1) {
      if (mul_act) {
        if (act_prev == kActGelu) {
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float2 d = gelu_tanh_grad_x2(s0[i], s0[i + 1]);
            s0[i] = v[i] * d.x;
            s0[i + 1] = v[i + 1] * d.y;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) s0[i] = v[i] * act_grad_fast(s0[i], act_prev);
        }
      } else {
        const bool skip = has_in[0];
#pragma unroll
        for (int i = 0; i < 32; ++i) s0[i] = v[i] + (skip ? s0[i] : 0.0f);
      }
    } else {
      const bool skip = has_in[0];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float g = v[i] + (skip ? s0[i] : 0.0f);
        s0[i] = g;
        s1[i] = g * act_grad_fast(s1[i], act_prev);
      }
    }
  }
};

// Weight-gradient partial of one K split: plain fp32 store.
struct PartialEpi {
  static constexpr int kSlots = 0;
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
