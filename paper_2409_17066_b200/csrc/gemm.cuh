// Batched (B > 16) tensor-core path launchers.
#pragma once
#include "common.cuh"

namespace vptq {

bool gemm_tcgen05_supported(const LayerView &L, int B);
long long gemm_tcgen05_workspace_bytes(const LayerView &L, int B);
int gemm_tcgen05_launches(const LayerView &L, int B);
// true when split tiles meet by flag order (a CTA waits for a flag another CTA of the grid raises)
bool gemm_tcgen05_waits_between_ctas(const LayerView &L, int B);
// Workspace layout: int32 status word at byte 0 (0 = ok, VPTQ_E_TIMEOUT = a bounded wait gave up),
// then the per-token bias terms, then the scaled FP16 activations.
cudaError_t launch_gemm_tcgen05(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st);

}  // namespace vptq
