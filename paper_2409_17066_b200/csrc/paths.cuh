// Kernel-family selection for vptq_linear.
#pragma once
#include "common.cuh"

namespace vptq {

enum LinearPath { PATH_GENERIC = 0, PATH_DECODE_SMEM_FMA, PATH_DECODE_SMEM_MMA, PATH_DECODE_L2_FMA, PATH_DECODE_GL_FMA, PATH_GEMM_TCGEN05, PATH_DECODE_BUCKET_FMA };

LinearPath choose_path(const LayerView &L, int B, int flags);
const char *linear_path_name(const LayerView &L, int B, int flags);
long long linear_workspace_bytes(const LayerView &L, int B, int flags);
int linear_launches(const LayerView &L, int B, int flags);
// returns VPTQ_OK / VPTQ_E_*; *cuda_err is set when the result is VPTQ_E_CUDA
int linear_dispatch(const LayerView &L, int flags, const void *x, int B, void *out, void *ws,
                    cudaStream_t st, cudaError_t *cuda_err);

// n layers over the same activations: one fused launch per token group when all of them take the same decode
// kernel family (main codebook in L2, in shared memory, or per group in global memory; for the latter two the
// layers must share their format apart from M) and whole vector rows spread evenly over the SMs, else one
// layer after the other
LinearPath fused_path(const LayerView *Ls, const int *flags, int n, int B);
const char *linear_fused_path_name(const LayerView *Ls, const int *flags, int n, int B);
long long linear_fused_workspace_bytes(const LayerView *Ls, const int *flags, int n, int B);
int linear_fused_launches(const LayerView *Ls, const int *flags, int n, int B);
int linear_fused_dispatch(const LayerView *Ls, const int *flags, int n, const void *x, int B, void *const *outs,
                          void *ws, cudaStream_t st, cudaError_t *cuda_err);

}  // namespace vptq
