// Registry storage.  Kernel instantiations register themselves from static initialisers
// of the program translation units when the library is loaded.
#include "registry.h"

#include <map>

namespace acc {

static std::map<std::string, KernelEntry>& table() {
  static std::map<std::string, KernelEntry> t;
  return t;
}

void register_kernel(const KernelEntry& e) {
  table().emplace(e.sig, e);   // the first instantiation of a sub-DAG wins; later ones are identical code
}

const KernelEntry* find_kernel(const std::string& sig) {
  auto it = table().find(sig);
  return it == table().end() ? nullptr : &it->second;
}

int registry_size() { return (int)table().size(); }

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaDeviceProp p;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&p, dev) == cudaSuccess) n = p.multiProcessorCount;
    else n = 148;
    cudaGetLastError();
  }
  return n;
}

bool cooperative_launch_ok() {
  int dev = 0, ok = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&ok, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return ok != 0;
}

}  // namespace acc

// ---- tensor maps for cp.async.bulk.tensor copies -------------------------------------------
#include <cuda.h>

#include <cstring>
#include <mutex>
#include <tuple>

namespace acc {

using EncodeTiled = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Describes a row-major rows x cols array of 4-byte elements for copies of box_rows x box_cols
// boxes (out-of-range parts of a box read as zero).  `out` points to a CUtensorMap.
// The driver entry point is looked up through the runtime, so libcuda is not linked.
bool make_tensor_map_2d(void* out, const void* base, int rows, int cols, int box_rows, int box_cols) {
  static EncodeTiled encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return false;
    }
    encode = reinterpret_cast<EncodeTiled>(fn);
  }
  if (rows < 1 || cols < 1 || cols % 4 || (reinterpret_cast<uintptr_t>(base) & 15)) return false;
  // the descriptor depends on nothing but these five values: programs that run again and again
  // over the same buffers get it from a small table instead of the driver
  using Key = std::tuple<const void*, int, int, int, int>;
  static std::map<Key, CUtensorMap> known;
  static std::mutex guard;
  const Key key{base, rows, cols, box_rows, box_cols};
  {
    std::lock_guard<std::mutex> lock(guard);
    auto it = known.find(key);
    if (it != known.end()) {
      memcpy(out, &it->second, sizeof(CUtensorMap));
      return true;
    }
  }
  CUtensorMap made;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};                 // bytes between rows: a multiple of 16
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t step[2] = {1, 1};
  if (encode(&made, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(base), dims, strides, box, step, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  memcpy(out, &made, sizeof(CUtensorMap));
  std::lock_guard<std::mutex> lock(guard);
  if (known.size() >= 4096) known.clear();
  known.emplace(key, made);
  return true;
}

}  // namespace acc
