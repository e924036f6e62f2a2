// Which kernel family runs a given (layer, batch), and the scratch it needs.
#include "paths.cuh"
#include "decode.cuh"
#include "gemm.cuh"
#include "prepared.cuh"
#include "fused_split.cuh"

namespace vptq {

namespace {
constexpr int DECODE_MAX_B = 16;
int decode_group(int B) { return B < DECODE_MAX_B ? B : DECODE_MAX_B; }
}

LinearPath choose_path(const LayerView &L, int B, int flags)
{
    if (flags & VPTQ_FLAG_FORCE_GENERIC) return PATH_GENERIC;
    if (L.deterministic) {
        // fixed summation order: the batched path with whole tiles, the L2 decode kernel in row-owner mode with
        // ordered warp partial sums, else the plain kernel (one warp per output row)
        if (B > DECODE_MAX_B && gemm_tcgen05_supported(L, B)) return PATH_GEMM_TCGEN05;
        if (l2_fma_supported(L, decode_group(B)) && l2_fma_deterministic_ok(L, decode_group(B))) return PATH_DECODE_L2_FMA;
        return PATH_GENERIC;
    }
    if (L.prep_parts > 0 && bucket_fma_supported(L, B) && L.prep_parts <= device_sm_count() &&
        ceil_div(L.R, L.prep_parts / prepared_split(L.R, ceil_div(L.k1, PREP_BUCKET), L.prep_parts)) <= PREP_MAX_ROWS)
        return PATH_DECODE_BUCKET_FMA;
    if (B > DECODE_MAX_B && gemm_tcgen05_supported(L, B)) return PATH_GEMM_TCGEN05;
    const int Bg = decode_group(B);
    if (smem_fma_supported(L, Bg)) return PATH_DECODE_SMEM_FMA;
    if (smem_mma_supported(L, Bg)) return PATH_DECODE_SMEM_MMA;
    if (l2_fma_supported(L, Bg)) return PATH_DECODE_L2_FMA;
    if (gl_fma_supported(L, Bg)) return PATH_DECODE_GL_FMA;
    return PATH_GENERIC;
}

const char *linear_path_name(const LayerView &L, int B, int flags)
{
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_FMA: return "decode_smem_fma";
    case PATH_DECODE_SMEM_MMA: return "decode_smem_mma";
    case PATH_DECODE_L2_FMA: return "decode_l2_fma";
    case PATH_DECODE_GL_FMA: return "decode_gl_fma";
    case PATH_GEMM_TCGEN05: return "gemm_tcgen05";
    case PATH_DECODE_BUCKET_FMA: return "decode_bucket_fma";
    default: return "generic";
    }
}

long long linear_workspace_bytes(const LayerView &L, int B, int flags)
{
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_FMA: return 0;
    case PATH_DECODE_SMEM_MMA: return smem_mma_workspace_bytes(L, decode_group(B));
    case PATH_DECODE_L2_FMA: return l2_fma_workspace_bytes(L, decode_group(B));
    case PATH_DECODE_GL_FMA: return 0;
    case PATH_GEMM_TCGEN05: return gemm_tcgen05_workspace_bytes(L, B);
    case PATH_DECODE_BUCKET_FMA: return (long long)bucket_fma_workspace_bytes(&L, &L.prep_parts, 1);
    default: return generic_workspace_bytes(L, B);
    }
}

int linear_launches(const LayerView &L, int B, int flags)
{
    const int groups = (B + DECODE_MAX_B - 1) / DECODE_MAX_B;
    const int last = B - (groups - 1) * DECODE_MAX_B;
    switch (choose_path(L, B, flags)) {
    case PATH_DECODE_SMEM_FMA:
        return (groups - 1) * smem_fma_launches(L, DECODE_MAX_B) + smem_fma_launches(L, last);
    case PATH_DECODE_SMEM_MMA: return groups * (smem_tc_supported(L, decode_group(B)) ? 2 : 1);      // pre-pass + main kernel
    case PATH_GEMM_TCGEN05: return gemm_tcgen05_launches(L, B);
    case PATH_DECODE_BUCKET_FMA: return 1;
    case PATH_DECODE_L2_FMA:
        return (groups - 1) * l2_fma_launches(L, DECODE_MAX_B) + l2_fma_launches(L, last);
    case PATH_DECODE_GL_FMA:
        return (groups - 1) * gl_fma_launches(L, DECODE_MAX_B) + gl_fma_launches(L, last);
    default: return generic_launches(L, B);
    }
}

int linear_dispatch(const LayerView &L, int flags, const void *x, int B, void *out, void *ws,
                    cudaStream_t st, cudaError_t *cuda_err)
{
    cudaError_t e = cudaSuccess;
    const LinearPath path = choose_path(L, B, flags);
    if (path == PATH_GENERIC) {
        e = launch_linear_generic(L, x, B, out, ws, st);
    } else if (path == PATH_GEMM_TCGEN05) {
        e = launch_gemm_tcgen05(L, x, B, out, ws, st);
    } else if (path == PATH_DECODE_BUCKET_FMA) {
        const void *img = L.prepared;
        void *o = out;
        e = launch_decode_bucket_fma(&L, &img, &L.prep_parts, 1, x, &o, ws, debug_wait_limit(), st);
    } else {
        // decode kernels take up to 16 tokens per launch
        const size_t oe = (L.out_dtype == VPTQ_DTYPE_FP32) ? 4 : 2;
        for (int t0 = 0; t0 < B && e == cudaSuccess; t0 += DECODE_MAX_B) {
            const int Bg = (B - t0 < DECODE_MAX_B) ? (B - t0) : DECODE_MAX_B;
            const void *xg = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * L.N * 2;
            void *og = reinterpret_cast<uint8_t *>(out) + (size_t)t0 * L.M * oe;
            if (path == PATH_DECODE_SMEM_FMA) e = launch_decode_smem_fma(L, xg, Bg, og, st);
            else if (path == PATH_DECODE_SMEM_MMA) e = launch_decode_smem_mma(L, xg, Bg, og, ws, st);
            else if (path == PATH_DECODE_GL_FMA) e = launch_decode_gl_fma(L, xg, Bg, og, st);
            else e = launch_decode_l2_fma(L, xg, Bg, og, ws, st);
        }
    }
    *cuda_err = e;
    return e == cudaSuccess ? VPTQ_OK : VPTQ_E_CUDA;
}

// ---- several layers that read the same activations ---------------------------------------------------

// The kernel family that serves all n layers with one launch per token group, or PATH_GENERIC when there is none.
LinearPath fused_path(const LayerView *Ls, const int *flags, int n, int B)
{
    if (n < 2 || B > DECODE_MAX_B) return PATH_GENERIC;
    for (int l = 0; l < n; l++)
        if (Ls[l].deterministic) return PATH_GENERIC;          // one layer after the other
    const LinearPath path = choose_path(Ls[0], B, flags[0]);
    for (int l = 1; l < n; l++)
        if (choose_path(Ls[l], B, flags[l]) != path) return PATH_GENERIC;
    if (path == PATH_DECODE_BUCKET_FMA) {
        // prepared layers share a launch when their partitions fit the SMs side by side
        int ctas = 0;
        for (int l = 0; l < n; l++) {
            if (Ls[l].N != Ls[0].N || Ls[l].x_bf16 != Ls[0].x_bf16 || (Ls[l].k2 > 0) != (Ls[0].k2 > 0)) return PATH_GENERIC;
            ctas += Ls[l].prep_parts;
        }
        return (n <= MAX_FUSED && ctas <= device_sm_count()) ? path : PATH_GENERIC;
    }
    if (path == PATH_DECODE_L2_FMA && l2_fma_fused_supported(Ls, n, B)) return path;
    if (path == PATH_DECODE_SMEM_FMA && smem_fma_fused_supported(Ls, n, B)) return path;
    if (path == PATH_DECODE_GL_FMA && gl_fma_fused_supported(Ls, n, B)) return path;
    return PATH_GENERIC;
}

const char *linear_fused_path_name(const LayerView *Ls, const int *flags, int n, int B)
{
    switch (fused_path(Ls, flags, n, B)) {
    case PATH_DECODE_L2_FMA: return "fused_decode_l2_fma";
    case PATH_DECODE_SMEM_FMA: return "fused_decode_smem_fma";
    case PATH_DECODE_GL_FMA: return "fused_decode_gl_fma";
    case PATH_DECODE_BUCKET_FMA: return "fused_decode_bucket_fma";
    default: return "one_by_one";
    }
}

long long linear_fused_workspace_bytes(const LayerView *Ls, const int *flags, int n, int B)
{
    const LinearPath fp = fused_path(Ls, flags, n, B);
    if (fp == PATH_DECODE_BUCKET_FMA) {
        int parts[MAX_FUSED];
        for (int l = 0; l < n; l++) parts[l] = Ls[l].prep_parts;
        return (long long)bucket_fma_workspace_bytes(Ls, parts, n);
    }
    if (fp != PATH_GENERIC) return 0;
    long long need = 0;       // one layer after the other on the stream: they share the scratch
    for (int l = 0; l < n; l++) {
        const long long w = linear_workspace_bytes(Ls[l], B, flags[l]);
        if (w > need) need = w;
    }
    return need;
}

int linear_fused_launches(const LayerView *Ls, const int *flags, int n, int B)
{
    const LinearPath path = fused_path(Ls, flags, n, B);
    if (path == PATH_DECODE_L2_FMA) return l2_fma_fused_launches(B);
    if (path == PATH_DECODE_SMEM_FMA) return smem_fma_launches(Ls[0], B);      // one launch per token group
    if (path == PATH_DECODE_GL_FMA) return gl_fma_launches(Ls[0], B);
    if (path == PATH_DECODE_BUCKET_FMA) return 1;
    int total = 0;
    for (int l = 0; l < n; l++) total += linear_launches(Ls[l], B, flags[l]);
    return total;
}

int linear_fused_dispatch(const LayerView *Ls, const int *flags, int n, const void *x, int B, void *const *outs,
                          void *ws, cudaStream_t st, cudaError_t *cuda_err)
{
    const LinearPath path = fused_path(Ls, flags, n, B);
    if (path != PATH_GENERIC) {
        if (path == PATH_DECODE_L2_FMA) *cuda_err = launch_decode_l2_fma_fused(Ls, n, x, B, outs, st);
        else if (path == PATH_DECODE_BUCKET_FMA) {
            const void *imgs[MAX_FUSED];
            int parts[MAX_FUSED];
            for (int l = 0; l < n; l++) { imgs[l] = Ls[l].prepared; parts[l] = Ls[l].prep_parts; }
            *cuda_err = launch_decode_bucket_fma(Ls, imgs, parts, n, x, outs, ws, debug_wait_limit(), st);
        }
        else if (path == PATH_DECODE_SMEM_FMA) *cuda_err = launch_decode_smem_fma_fused(Ls, n, x, B, outs, st);
        else *cuda_err = launch_decode_gl_fma_fused(Ls, n, x, B, outs, st);
        return *cuda_err == cudaSuccess ? VPTQ_OK : VPTQ_E_CUDA;
    }
    for (int l = 0; l < n; l++) {
        const int rc = linear_dispatch(Ls[l], flags[l], x, B, outs[l], ws, st, cuda_err);
        if (rc != VPTQ_OK) return rc;
    }
    return VPTQ_OK;
}

}  // namespace vptq
