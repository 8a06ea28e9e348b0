// Host side of TMA: tensor-map encoding through the driver entry point (the library does not link libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>
#include <string>

namespace dnnf {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tma_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// rank <= 4; dims / box innermost first; strides_bytes[i] is the byte stride of dim i+1 (a multiple of 16);
// base 16-byte aligned; box[0] * element size a multiple of 16 bytes.  Out-of-range elements read as zero.
inline bool tma_encode(CUtensorMap* tm, CUtensorMapDataType type, int rank, void* base, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                       const cuuint32_t* box, CUtensorMapSwizzle swizzle, std::string& err) {
  if ((uintptr_t)base & 15) { err = "TMA operand is not 16-byte aligned"; return false; }
  EncodeTiledFn fn = tma_encode_fn();
  if (!fn) { err = "cuTensorMapEncodeTiled is not available"; return false; }
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult rc = fn(tm, type, (cuuint32_t)rank, base, dims, strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) { err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)rc); return false; }
  return true;
}

}  // namespace dnnf
