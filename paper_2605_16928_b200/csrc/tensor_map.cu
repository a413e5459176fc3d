// Host side of the TMA descriptors: cuTensorMapEncodeTiled through the runtime's driver entry point.
#include <mutex>

#include "tc_common.cuh"

namespace rtp {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The entry point is a property of the driver, not of a device: looked up once per process, under a lock.
EncodeTiledFn encode_fn(cudaError_t* err) {
  static std::mutex mu;
  static EncodeTiledFn fn = nullptr;
  std::lock_guard<std::mutex> lock(mu);
  *err = cudaSuccess;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
    if (e != cudaSuccess) { *err = e; return nullptr; }
    if (qres != cudaDriverEntryPointSuccess || !p) { *err = cudaErrorNotSupported; return nullptr; }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}
}  // namespace

// A descriptor depends only on (base, rows, row length, box, swizzle): the last few are kept, so a cache that does
// not move is encoded once instead of once per launch.  (The descriptor holds a global address, which is the same
// number on every device of the process only by accident: the device ordinal is part of the key.)
namespace {
struct MapKey {
  const void* base;
  int64_t rows;
  int row_elems, box_cols, box_rows, swizzle, device;
  bool operator==(const MapKey& o) const {
    return base == o.base && rows == o.rows && row_elems == o.row_elems && box_cols == o.box_cols &&
           box_rows == o.box_rows && swizzle == o.swizzle && device == o.device;
  }
};
constexpr int kMapSlots = 16;
std::mutex g_map_mu;
MapKey g_map_key[kMapSlots] = {};
CUtensorMap g_map_val[kMapSlots];
bool g_map_used[kMapSlots] = {};
int g_map_next = 0;
}  // namespace

cudaError_t make_rows_map(CUtensorMap* map, const void* base, int64_t rows, int row_elems, int box_cols, int box_rows,
                          int swizzle) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const MapKey key = {base, rows, row_elems, box_cols, box_rows, swizzle, dev};
  {
    std::lock_guard<std::mutex> lock(g_map_mu);
    for (int i = 0; i < kMapSlots; ++i)
      if (g_map_used[i] && g_map_key[i] == key) {
        *map = g_map_val[i];
        return cudaSuccess;
      }
  }
  EncodeTiledFn encode = encode_fn(&e);
  if (!encode) return e;
  const cuuint64_t dims[2] = {(cuuint64_t)row_elems, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_elems * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, (CUtensorMapSwizzle)swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  std::lock_guard<std::mutex> lock(g_map_mu);
  g_map_key[g_map_next] = key;
  g_map_val[g_map_next] = *map;
  g_map_used[g_map_next] = true;
  g_map_next = (g_map_next + 1) % kMapSlots;
  return cudaSuccess;
}

}  // namespace rtp
