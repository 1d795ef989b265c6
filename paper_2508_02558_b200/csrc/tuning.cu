// Host-side state shared by the launchers (see tuning.cuh). Everything here is guarded by one mutex.
#include "tuning.cuh"

#include <string.h>

#include <mutex>

namespace sdllm {
namespace {

std::mutex g_mutex;
Tuning g_tuning;
int g_sm_count[kMaxDevices] = {};

}  // namespace

Tuning tuning() {
  std::lock_guard<std::mutex> lock(g_mutex);
  return g_tuning;
}

void tuning_reset() {
  std::lock_guard<std::mutex> lock(g_mutex);
  g_tuning = Tuning{};
}

bool tuning_set(const char* name, long long value) {
  if (name == nullptr) return false;
  std::lock_guard<std::mutex> lock(g_mutex);
  struct Field { const char* name; int Tuning::*field; };
  static const Field fields[] = {
      {"splits", &Tuning::splits}, {"kernel", &Tuning::kernel}, {"pdl", &Tuning::pdl}, {"early_loads", &Tuning::early_loads},
      {"cluster", &Tuning::cluster}, {"fused_tail", &Tuning::fused_tail}, {"dual", &Tuning::dual}, {"key_tile", &Tuning::key_tile},
      {"lpt", &Tuning::lpt}, {"select", &Tuning::select}, {"stages", &Tuning::stages}, {"debug", &Tuning::debug}, {"trigger", &Tuning::trigger},
      {"persist", &Tuning::persist},
  };
  for (const Field& f : fields)
    if (strcmp(name, f.name) == 0) {
      g_tuning.*(f.field) = (int)value;
      return true;
    }
  if (strcmp(name, "wait_cycles") == 0) {
    g_tuning.wait_cycles = value < 0 ? 0 : value;
    return true;
  }
  return false;
}

cudaError_t configure_smem(const void* func, size_t bytes, SmemConfig& cfg, bool max_carveout) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (bytes <= cfg.bytes[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  if (max_carveout) (void)cudaFuncSetAttribute(func, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  cfg.bytes[dev] = bytes;
  return cudaSuccess;
}

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_sm_count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    g_sm_count[dev] = n;
  }
  return g_sm_count[dev];
}

}  // namespace sdllm
