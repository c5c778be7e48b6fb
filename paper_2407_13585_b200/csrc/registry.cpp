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

}  // namespace acc
