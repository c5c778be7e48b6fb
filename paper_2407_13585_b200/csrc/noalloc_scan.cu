// acc_scanl_add_i32_static: the single-pass inclusive prefix sum of the library, usable by
// callers that cannot hand the library a workspace.
//
// The regular path takes its tile states and its ticket counter from the caller's workspace,
// which the caller obtains with cudaMalloc or a framework allocator.  Some callers cannot do
// that at the point of the call: code running where device allocation is forbidden (a callback
// or plug-in that was given raw pointers and no allocator, a process whose device memory was
// handed out completely up front).  The call itself still blocks the host until the scan has
// finished, so it must never run on a capturing stream.  For such callers the scratch lives in a
// file-scope device array of fixed size that every GPU loading this library holds until the
// process exits; the caller passes only the input and the output.
//
// The host never uses the array's name as an address: in host code that name stands for a
// host-side shadow, and a kernel given it would fault or read the wrong memory.  The device
// address is looked up once per device with cudaGetSymbolAddress and cached.
#include <cuda_runtime.h>

#include <mutex>

#include "acc.h"
#include "device/skeletons.cuh"
#include "graph.h"
#include "registry.h"

namespace acc {
namespace {

constexpr int64_t kMaxElements = ACC_STATIC_SCAN_MAX_ELEMENTS;
constexpr int kSmallestTile = 256 * 16;                   // the static array holds a state per tile of the smallest tile shape
constexpr int64_t kMaxTiles = (kMaxElements + kSmallestTile - 1) / kSmallestTile;
constexpr size_t kHeaderBytes = 256;                      // status word, padded
constexpr size_t kScratchBytes = kHeaderBytes + 16 + (size_t)kMaxTiles * 8;

// [0, 256): status word.  [256, ...): the scan's own layout (ticket, then one state per tile).
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr CProgram scan_program() {
  CProgram p{2, 1ull << 1, {}};
  p.nodes[0] = pnode(ACC_INPUT, ACC_I32, 1, 0, 0, 0);
  p.nodes[1] = pnode(ACC_SCANL, ACC_I32, 1, ACC_FN_ADD, 0, 1, 0);
  return p;
}
inline constexpr CProgram kScanProgram = scan_program();
struct ScanCluster { static constexpr CCluster c = extract(kScanProgram, 0x2); };

constexpr int kMaxDevices = 64;
std::mutex g_lock;
unsigned char* g_device_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up on first use.
int scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return set_error(ACC_ERR_UNSUPPORTED, "device ordinal %d beyond %d", dev, kMaxDevices);
  std::lock_guard<std::mutex> guard(g_lock);
  if (!g_device_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p)
      return set_error(ACC_ERR_CUDA, "cudaGetSymbolAddress for the static scratch failed: %s", cudaGetErrorString(e));
    g_device_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_device_ptr[dev];
  return ACC_OK;
}

}  // namespace
}  // namespace acc

extern "C" int acc_scanl_add_i32_static(const int32_t* in, int32_t* out, int64_t n, void* cuda_stream) {
  using namespace acc;
  clear_error();
  if (n < 0) return set_error(ACC_ERR_ARG, "negative length");
  if (n > kMaxElements)
    return set_error(ACC_ERR_TOO_LARGE, "%lld elements: the static scratch of acc_scanl_add_i32_static covers at most %lld",
                     (long long)n, (long long)kMaxElements);
  if (n == 0) return ACC_OK;
  if (!in || !out) return set_error(ACC_ERR_ARG, "null array");
  unsigned char* base = nullptr;
  int rc = scratch_for_current_device(&base);
  if (rc != ACC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  constexpr int kScanBlock = dev::scan_block<ScanCluster>();
  constexpr int kTile = kScanBlock * dev::scan_rows<ScanCluster>() * 4;
  static_assert(kTile >= kSmallestTile, "the static tile states are sized for tiles of at least 4096 elements");
  const int tiles = (int)((n + kTile - 1) / kTile);
  // the array keeps whatever the previous call left: status, ticket and the states in use start at zero
  cudaError_t e = cudaMemsetAsync(base, 0, kHeaderBytes + 16 + (size_t)tiles * 8, stream);
  if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "clearing the static scratch failed: %s", cudaGetErrorString(e));

  dev::Args<ScanCluster::c.n> a{};
  a.n[0].ptr = in;
  a.n[0].R = 1;
  a.n[0].C = (int32_t)n;
  a.n[1].ptr = out;
  a.n[1].R = 1;
  a.n[1].C = (int32_t)n;
  a.R = 1;
  a.C = (int32_t)n;
  a.scratch = reinterpret_cast<uint32_t*>(base + kHeaderBytes);
  a.status = reinterpret_cast<uint32_t*>(base);
  a.spin_limit = 1u << 22;
  a.grid = 0;
  const bool vec = n % 4 == 0 && ((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15) == 0;
  const int resident = sm_count() * (1536 / kScanBlock);
  const int grid = tiles < resident ? tiles : resident;
  if (vec) dev::k_scan<ScanCluster, true><<<grid, kScanBlock, 0, stream>>>(a, tiles, tiles);
  else dev::k_scan<ScanCluster, false><<<grid, kScanBlock, 0, stream>>>(a, tiles, tiles);
  e = cudaGetLastError();
  if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  uint32_t status = 0;
  e = cudaMemcpyAsync(&status, base, 4, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "waiting for the scan failed: %s", cudaGetErrorString(e));
  if (status & dev::kStatusTimeout) return set_error(ACC_ERR_DEVICE_TIMEOUT, "a device-side wait ran out of iterations");
  return ACC_OK;
}
