// Decode-path (batch 1..16) kernel launchers.
#pragma once
#include "common.cuh"

namespace vptq {

// codebooks in shared memory, LDS gathers + FP32 FMAs, up to 8 tokens per launch, no scratch
bool smem_fma_supported(const LayerView &L, int B);
int smem_fma_launches(const LayerView &L, int B);
cudaError_t launch_decode_smem_fma(const LayerView &L, const void *x, int B, void *out, cudaStream_t st);
bool smem_fma_fused_supported(const LayerView *Ls, int n, int B);
cudaError_t launch_decode_smem_fma_fused(const LayerView *Ls, int n, const void *x, int B, void *const *outs, cudaStream_t st);

// codebooks in shared memory, ldmatrix gathers + mma.sync (per-output-row scale, all-outlier layers)
bool smem_mma_supported(const LayerView &L, int B);
long long smem_mma_workspace_bytes(const LayerView &L, int B);
cudaError_t launch_decode_smem_mma(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st);

// the same family for the common kind of layer (main columns, per-column scale): persistent row-owner grid,
// activations staged in shared memory in mma A-fragment order, 32 warps (decode_smem_tc.cu)
bool smem_tc_supported(const LayerView &L, int B);
long long smem_tc_workspace_bytes(const LayerView &L, int B);
cudaError_t launch_decode_smem_tc(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st);

// main codebook in global memory (L2), residual codebook in shared memory, FP32 FMAs
bool l2_fma_supported(const LayerView &L, int B);
long long l2_fma_workspace_bytes(const LayerView &L, int B);
int l2_fma_launches(const LayerView &L, int B);
// row-owner mode with its ordered partial sums fits shared memory for this layer (deterministic mode)
bool l2_fma_deterministic_ok(const LayerView &L, int B);
cudaError_t launch_decode_l2_fma(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st);
// ... several layers that read the same activations in one launch per token group (no scratch)
bool l2_fma_fused_supported(const LayerView *Ls, int n, int B);
int l2_fma_fused_launches(int B);
cudaError_t launch_decode_l2_fma_fused(const LayerView *Ls, int n, const void *x, int B, void *const *outs, cudaStream_t st);

// codebooks in global memory, any even v <= 16, group-wise codebooks, FP32 FMAs, no scratch
bool gl_fma_supported(const LayerView &L, int B);
int gl_fma_launches(const LayerView &L, int B);
cudaError_t launch_decode_gl_fma(const LayerView &L, const void *x, int B, void *out, cudaStream_t st);
bool gl_fma_fused_supported(const LayerView *Ls, int n, int B);
cudaError_t launch_decode_gl_fma_fused(const LayerView *Ls, int n, const void *x, int B, void *const *outs, cudaStream_t st);

}  // namespace vptq
