// Decode-path (batch 1..16) kernel launchers.
#pragma once
#include "common.cuh"

namespace vptq {

// codebooks in shared memory, ldmatrix gathers + mma.sync
bool smem_mma_supported(const LayerView &L, int B);
cudaError_t launch_decode_smem_mma(const LayerView &L, const void *x, int B, void *out, cudaStream_t st);

}  // namespace vptq
