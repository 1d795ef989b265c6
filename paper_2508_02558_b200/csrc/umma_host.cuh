// Host-side helpers shared by the tcgen05 attention kernels.
#pragma once
#include <cuda.h>
#include <stdint.h>

namespace sdllm {

// Tiled tensor map (128-byte swizzle, zero fill outside the tensor) of a bf16 [batch, heads, rows, D] tensor whose
// rows are D contiguous elements; strides (batch, head, row) in elements; the box is 64 columns x box_rows x box_heads.
// False when the driver does not export the encoder or refuses the shape.
bool umma_make_map(CUtensorMap* m, const void* base, int D, int rows, int heads, int batch, const int64_t* stride_bhr, int box_rows,
                   int box_heads);

}  // namespace sdllm
