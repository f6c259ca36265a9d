// Host side of the TMA tile loads: building CUtensorMap descriptors for tensors in THIS GPU's memory.
// The driver's encoder is looked up through the runtime (no link against libcuda).  Every map made
// here is used with plain tile loads (cp.async.bulk.tensor ... tile, one destination CTA): no cluster
// multicast anywhere.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pisa {
namespace tma {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encoder() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// rank <= 5.  dims[i] elements, strides_bytes[i] = byte stride of dimension i (strides_bytes[0] is the
// element size and is implied), box[i] elements per tile.  elem_bytes: 2 (bf16) or 4 (fp32).
// swizzle128: rows of 128 bytes land in the 128-byte-swizzled layout the UMMA descriptors expect;
// otherwise the tile is stored densely.  Out-of-range elements read as zero.
inline bool make_map(CUtensorMap* out, int elem_bytes, int rank, const void* base, const uint64_t* dims,
                     const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128) {
  EncodeTiledFn enc = encoder();
  if (enc == nullptr || rank < 1 || rank > 5) return false;
  cuuint64_t gdim[5], gstride[5];
  cuuint32_t bdim[5], estr[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bdim[i] = box[i];
    estr[i] = 1;
    if (i > 0) gstride[i - 1] = strides_bytes[i];
  }
  const CUtensorMapDataType dt = (elem_bytes == 2) ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  const CUresult r = enc(out, dt, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride, bdim, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace tma
}  // namespace pisa
