// et_bias_grad_noalloc: the bias gradient (column sums of an error-gradient matrix) for callers
// that cannot allocate device memory.  The scratch that the two-stage reduction needs lives in a
// fixed array inside the library image instead of in a caller-provided workspace.
#include <cuda_runtime.h>

#include "et.h"
#include "kernels.cuh"

namespace {

// Stage-1 partial sums: ceil(M / 128) rows of `width` floats.  4 MiB per GPU that loads the
// library, held until the process exits.
static __device__ __align__(256) float g_noalloc_scratch[ET_NOALLOC_SCRATCH_FLOATS];

// In host code `g_noalloc_scratch` is only a handle for the symbol; the address a kernel can use
// has to be asked for with the device current.  It is asked for on every call and never cached:
// once the module is loaded the lookup is a host-side table read, while a remembered address
// would go stale if the embedding application reset the device or made another context current
// (a kernel given a stale address faults instead of returning a status).
et_status scratch_for_current_device(float** out) {
  float* p = nullptr;
  if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
    (void)cudaGetLastError();
    return ET_ERR_CUDA;
  }
  *out = p;
  return ET_OK;
}

template <typename T>
et_status run(const void* dZ, int64_t M, int32_t width, float* db, float* scratch, cudaStream_t st) {
  const int chunks = (int)((M + et::kColsumRows - 1) / et::kColsumRows);
  dim3 grid((width + 255) / 256, chunks), block(32, 8);
  // stage 1 writes every partial that stage 2 reads, so nothing left over from an earlier
  // call is ever consumed and nothing has to be cleared first
  et::colsum_partial_kernel<T><<<grid, block, 0, st>>>((const T*)dZ, (int)M, width, scratch);
  if (cudaGetLastError() != cudaSuccess) return ET_ERR_CUDA;
  et::bias_finish_kernel<T><<<(width + et::kBiasCols - 1) / et::kBiasCols, dim3(et::kBiasCols, et::kBiasLanes), 0, st>>>(
      scratch, chunks, width, width, db, (const T*)nullptr, nullptr, (T*)nullptr, et::OptParams{}, 0, 0, nullptr, nullptr, nullptr);
  if (cudaGetLastError() != cudaSuccess) return ET_ERR_CUDA;
  return ET_OK;
}

}  // namespace

extern "C" et_status et_bias_grad_noalloc(const void* dZ, int64_t M, int32_t width, et_dtype dtype, float* db,
                                          void* stream) {
  if (dZ == nullptr || db == nullptr || M < 1 || width < 1 || M > (1ll << 30)) return ET_ERR_INVALID_ARG;
  if (dtype != ET_F32 && dtype != ET_BF16) return ET_ERR_DTYPE;
  const int64_t chunks = (M + et::kColsumRows - 1) / et::kColsumRows;
  if (chunks * (int64_t)width > (int64_t)ET_NOALLOC_SCRATCH_FLOATS) return ET_ERR_TOO_LARGE;
  if (chunks > 65535) return ET_ERR_TOO_LARGE;     // one grid row per chunk (narrow matrices with millions of rows)
  float* scratch = nullptr;
  et_status st = scratch_for_current_device(&scratch);
  if (st != ET_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  return dtype == ET_BF16 ? run<et::bf16>(dZ, M, width, db, scratch, s) : run<float>(dZ, M, width, db, scratch, s);
}
