// Which kernel family runs a given (layer, batch), and the scratch it needs.
#include "paths.cuh"
#include "decode.cuh"

namespace vptq {

LinearPath choose_path(const LayerView &L, int B, int flags)
{
    if (flags & VPTQ_FLAG_FORCE_GENERIC) return PATH_GENERIC;
    if (B <= 16 && smem_mma_supported(L, B)) return PATH_DECODE_SMEM_MMA;
    return PATH_GENERIC;
}

const char *linear_path_name(const LayerView &L, int B, int flags)
{
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_MMA: return "decode_smem_mma";
    case PATH_DECODE_L2_FMA: return "decode_l2_fma";
    case PATH_GEMM_TCGEN05: return "gemm_tcgen05";
    default: return "generic";
    }
}

long long linear_workspace_bytes(const LayerView &L, int B, int flags)
{
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_MMA: return 0;
    default: return generic_workspace_bytes(L, B);
    }
}

int linear_launches(const LayerView &L, int B, int flags)
{
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_MMA: return 1;
    default: return generic_launches(L, B);
    }
}

int linear_dispatch(const LayerView &L, int flags, const void *x, int B, void *out, void *ws,
                    cudaStream_t st, cudaError_t *cuda_err)
{
    cudaError_t e;
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_MMA: e = launch_decode_smem_mma(L, x, B, out, st); break;
    default: e = launch_linear_generic(L, x, B, out, ws, st); break;
    }
    *cuda_err = e;
    return e == cudaSuccess ? VPTQ_OK : VPTQ_E_CUDA;
}

}  // namespace vptq
