// Host-side state shared by the launchers: the tuning overrides (set only through sdllm_tuning_set, never read from the
// environment), the per-device kernel attributes and the per-device SM count.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace sdllm {

constexpr int kMaxDevices = 64;

// Overrides of the launch planner. Every field has a neutral value meaning "the planner decides"; the planner is a
// pure function of the description and of this struct, so the workspace query and the launch agree as long as no
// override changes between them.
struct Tuning {
  int splits = 0;            // > 0: key splits per (sequence, KV head)
  int kernel = 0;            // 0: automatic; 1: cp.async kernels; 2: tcgen05 kernel with the queries on the accumulator
                             // rows; 3: tcgen05 kernel with the keys on the accumulator rows
  int pdl = 1;               // 0: no programmatic dependent launch
  int early_loads = 1;       // 0: no loads ahead of the grid dependency
  int cluster = 1;           // query-row kernel: 2 merges few key splits through a cluster where the shape allows (off otherwise)
  int fused_tail = -1;       // query-row kernel: 0 / 1 forces the tail into the second launch / into the last CTA
  int dual = -1;             // query-row kernel: 0 / 1 forces the two-CTAs-per-SM variant off / on
  int key_tile = 0;          // query-row kernel: 64 or 128
  int lpt = -1;              // 0 / 1 forces the longest-first order of ragged batches off / on
  int select = 0;            // top-k: 1 one CTA per head, 2 a cluster per head
  int stages = 0;            // key-row kernel: ring slots (1..3)
  int trigger = 1;           // key-row kernel: 1 releases the next kernel in the stream at its start, 0 after its own dependency
  int persist = -1;          // key-row kernel: 0 / 1 forces the streaming variant (resident CTAs walk the units) off / on;
                             // n >= 2: on, with at most n CTAs (small test shapes then walk several units per CTA)
  int debug = 0;             // 1: print the CUDA error behind an SDLLM_ERR_CUDA to stderr
  long long wait_cycles = 400000000LL;   // limit of an abortable device-side wait, ~0.2 s
};

Tuning tuning();                                     // a snapshot
bool tuning_set(const char* name, long long value);  // false: unknown name
void tuning_reset();

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device attribute: remember, per kernel and device, what was set.
struct SmemConfig {
  size_t bytes[kMaxDevices] = {};
};
cudaError_t configure_smem(const void* func, size_t bytes, SmemConfig& cfg, bool max_carveout);

// Streaming multiprocessors of the current device (148 on a B200), looked up once per device.
int sm_count();

}  // namespace sdllm
