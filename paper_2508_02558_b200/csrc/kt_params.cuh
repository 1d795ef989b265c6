// Launch parameters of the kernels that put the keys on the accumulator rows (attn_kt.cu, attn_kt_stream.cu).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace sdllm {

struct KtMaps {
  CUtensorMap q, k1, v1, k2, v2;   // boxes of 32 rows (source 2: min(32, n2))
  CUtensorMap k1t, v1t;            // source 1 again, boxes of 128 rows: a whole tile per copy
};

struct KtParams {
  AttnParams a;
  int N;             // query columns of a KV head (b * G)
  int S;             // key splits of a unit = CTAs of its cluster (1..8)
  int NS;            // ring slots (one 128-key K tile + V tile each)
  int PB;            // P^T buffers (1 or 2)
  int DL;            // head dimensions a CTA owns in the merge: ceil(D / S)
  int cpt;           // merge: columns per thread, a multiple of 4
  int gr2;           // rows of a source-2 box: min(32, n2)
  int early_src1;    // 1: source 1 and its count are older than every kernel that may still run (reuse step)
  int early_trigger; // 1: release the next kernel in the stream as soon as this CTA is set up
  int lpt;           // 1: grid z counts the sequences from the longest to the shortest (several waves of ragged work)
  long long wait_cycles;   // limit of every abortable mbarrier wait
};

// The streaming variant (attn_kt_stream.cu): one CTA per SM walks the (sequence, KV head) units of a large batch.
size_t kt_stream_smem_bytes(int D);
cudaError_t launch_kt_stream(const KtMaps& tm, const KtParams& kp, int D, size_t smem_bytes, bool pdl, cudaStream_t st);

}  // namespace sdllm
