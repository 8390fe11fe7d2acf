// Host-side construction of TMA tensor maps.  The driver entry point is looked up at run time so
// the library does not link against the driver library.
#include <mutex>

#include <cudaTypedefs.h>

#include "common.cuh"
#include "ptx.cuh"

namespace gvote {

namespace {
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
std::once_flag g_once;

void resolve() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
}

bool encode(CUtensorMap* out, const void* base, CUtensorMapDataType type, int elem_bytes, CUtensorMapSwizzle swizzle,
            CUtensorMapL2promotion promotion, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box) {
  std::call_once(g_once, resolve);
  if (!g_encode || rank < 1 || rank > 5) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return false;
  cuuint64_t gdims[5];
  cuuint64_t gstrides[4];
  cuuint32_t gbox[5], estr[5];
  for (int i = 0; i < rank; ++i) {
    if (dims[i] == 0 || dims[i] > 0xFFFFFFFFull || box[i] == 0 || box[i] > 256) return false;
    gdims[i] = dims[i];
    gbox[i] = box[i];
    estr[i] = 1;
  }
  if (((uint64_t)box[0] * elem_bytes) % 16 != 0) return false;
  for (int i = 0; i + 1 < rank; ++i) {
    if (strides_bytes[i] % 16 != 0 || strides_bytes[i] == 0 || strides_bytes[i] >= (1ull << 40)) return false;
    gstrides[i] = strides_bytes[i];
  }
  const CUresult res = g_encode(out, type, (cuuint32_t)rank, const_cast<void*>(base), gdims, gstrides, gbox, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promotion,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return res == CUDA_SUCCESS;
}
}  // namespace

bool encode_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box) {
  return encode(out, base, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, rank, dims, strides_bytes, box);
}

bool encode_tensor_map_plain(CUtensorMap* out, const void* base, int elem_bytes, int rank, const uint64_t* dims,
                             const uint64_t* strides_bytes, const uint32_t* box) {
  if (elem_bytes != 2 && elem_bytes != 4) return false;
  return encode(out, base, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                elem_bytes, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, rank, dims, strides_bytes, box);
}

}  // namespace gvote
