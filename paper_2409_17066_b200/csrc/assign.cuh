// Assignment step of the quantizer (Eq. 2): launchers shared between the two kernel files.
#pragma once
#include "common.cuh"

namespace vptq {

// the FP32 definition for the vectors list[0 .. *count) only (both on the device): one warp per vector
cudaError_t launch_assign_listed(const __half *W, int M, int N, int v, const __half *C, int k, int *idx,
                                 const int *list, const int *count, int sm_count, cudaStream_t st);

// tensor-core filter + FP32 decision: same indices as the plain kernel
bool assign_tcgen05_supported(int M, int N, int v, int k);
long long assign_tcgen05_workspace_bytes(int M, int N, int v, int k);
cudaError_t launch_assign_tcgen05(const __half *W, int M, int N, int v, const __half *C, int k, int *idx, void *ws,
                                  cudaStream_t st);

}  // namespace vptq
