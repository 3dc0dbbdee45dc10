// TMA tensor maps over the K / V page pools, shared by the decode and prefill kernels.
//
// A pool [num_pages][n_kv_heads][page_size][head_dim] bf16 is described to the TMA unit as a 2-D tensor
// [num_pages * n_kv_heads * page_size rows][head_dim]; one box is 64 dims x 16 rows (one 16-token group of one
// head, one 64-dim half), written to shared memory with the 128-byte swizzle that both ldmatrix and the tcgen05
// matrix descriptors read without bank conflicts.  x coordinates are 0 or 64 elements, i.e. multiples of 16 bytes.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include "mepic.h"
#include "mepic_internal.h"

namespace {

// The driver's encoder, looked up through the runtime so that the library links no driver stub and still loads
// on a machine without a driver.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static std::mutex mu;
  static EncodeTiledFn fn = nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) == cudaSuccess &&
        res == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

}  // namespace

int32_t mepic_make_pool_map(const mepic_config_t* cfg, const void* pool, void* out_map) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map is 128 bytes");
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) { mepic_set_error("cuTensorMapEncodeTiled is not available from the driver"); return MEPIC_E_CUDA; }
  const cuuint64_t rows = static_cast<cuuint64_t>(cfg->num_pages) * cfg->n_kv_heads * cfg->page_size;
  if (rows > 0x7fffffffull) { mepic_set_error("pool has too many rows for 32-bit tensor coordinates"); return MEPIC_E_INVAL; }
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cfg->head_dim), rows};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cfg->head_dim) * 2};
  const cuuint32_t box[2] = {64, 16};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(static_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(pool), dims, strides,
                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { mepic_set_error("cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r)); return MEPIC_E_CUDA; }
  return MEPIC_OK;
}

// The same for a pool of 8-bit elements (fp8 pages, head_dim = 128): rows of 128 bytes, one box = a whole
// 16-token group (16 rows x 128 bytes).
int32_t mepic_make_pool_map_u8(const mepic_config_t* cfg, const void* pool, void* out_map) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) { mepic_set_error("cuTensorMapEncodeTiled is not available from the driver"); return MEPIC_E_CUDA; }
  if (cfg->head_dim != 128) { mepic_set_error("8-bit pools need head_dim 128"); return MEPIC_E_INVAL; }
  const cuuint64_t rows = static_cast<cuuint64_t>(cfg->num_pages) * cfg->n_kv_heads * cfg->page_size;
  if (rows > 0x7fffffffull) { mepic_set_error("pool has too many rows for 32-bit tensor coordinates"); return MEPIC_E_INVAL; }
  const cuuint64_t dims[2] = {128, rows};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {128, 16};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(static_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(pool), dims, strides,
                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { mepic_set_error("cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r)); return MEPIC_E_CUDA; }
  return MEPIC_OK;
}
