// C ABI of libvptq: argument validation, dispatch, error reporting.  No kernel code here.
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "decode.cuh"
#include "paths.cuh"
#include "assign.cuh"
#include "prepared.cuh"
#include "gemm.cuh"

#include <vector>

using namespace vptq;

namespace {

thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e)
{
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return VPTQ_E_CUDA;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_desc(const vptq_layer_desc *d)
{
    if (d == nullptr) return VPTQ_E_NULL;
    if (d->M <= 0 || d->N <= 0) return VPTQ_E_SHAPE;
    if (d->v <= 0 || d->v > 32 || d->k1 <= 0 || d->k1 > 65536) return VPTQ_E_SHAPE;
    if (d->k2 < 0 || d->k2 > 65536) return VPTQ_E_SHAPE;
    if (d->n_outlier < 0 || d->n_outlier > d->N) return VPTQ_E_SHAPE;
    if (d->n_groups < 0 || (d->n_groups > 1 && d->n_groups > d->N - d->n_outlier)) return VPTQ_E_SHAPE;
    if (d->n_outlier > 0 && (d->v0 <= 0 || d->v0 > 32 || d->k0 <= 0 || d->k0 > 65536)) return VPTQ_E_SHAPE;
    if (d->x_dtype != VPTQ_DTYPE_FP16 && d->x_dtype != VPTQ_DTYPE_BF16) return VPTQ_E_UNSUPPORTED;
    if (d->out_dtype != VPTQ_DTYPE_FP16 && d->out_dtype != VPTQ_DTYPE_BF16 &&
        d->out_dtype != VPTQ_DTYPE_FP32) return VPTQ_E_UNSUPPORTED;
    if (d->flags & ~(VPTQ_FLAG_SCALE_BIAS | VPTQ_FLAG_SCALE_ROWS | VPTQ_FLAG_FORCE_GENERIC | VPTQ_FLAG_COL_PERM | VPTQ_FLAG_PREPARED | VPTQ_FLAG_CONCURRENT | VPTQ_FLAG_DETERMINISTIC)) return VPTQ_E_UNSUPPORTED;
    if ((d->flags & VPTQ_FLAG_PREPARED) && d->prepared_parts < 1) return VPTQ_E_SHAPE;
    if ((d->flags & VPTQ_FLAG_SCALE_ROWS) && !(d->flags & VPTQ_FLAG_SCALE_BIAS)) return VPTQ_E_UNSUPPORTED;
    return VPTQ_OK;
}

int check_ptrs(const vptq_layer_desc *d, const vptq_layer_ptrs *p)
{
    if (p == nullptr) return VPTQ_E_NULL;
    const bool has_main = d->n_outlier < d->N;
    if (has_main && (p->packed_idx == nullptr || p->codebook == nullptr)) return VPTQ_E_NULL;
    if (has_main && d->k2 > 0 && (p->res_idx == nullptr || p->res_codebook == nullptr)) return VPTQ_E_NULL;
    if (d->n_outlier > 0 && (p->outlier_idx == nullptr || p->outlier_codebook == nullptr)) return VPTQ_E_NULL;
    if ((d->flags & VPTQ_FLAG_SCALE_BIAS) && (p->scale == nullptr || p->bias == nullptr)) return VPTQ_E_NULL;
    if (d->flags & VPTQ_FLAG_COL_PERM) {
        if (p->col_perm == nullptr) return VPTQ_E_NULL;
        if (!aligned16(p->col_perm)) return VPTQ_E_ALIGN;
    }
    if (d->flags & VPTQ_FLAG_PREPARED) {
        if (p->prepared == nullptr) return VPTQ_E_NULL;
        if ((reinterpret_cast<uintptr_t>(p->prepared) & 255u) != 0) return VPTQ_E_ALIGN;
    }
    const void *all[8] = {has_main ? p->packed_idx : nullptr, has_main ? p->codebook : nullptr,
                          (has_main && d->k2 > 0) ? p->res_idx : nullptr,
                          (has_main && d->k2 > 0) ? p->res_codebook : nullptr,
                          d->n_outlier > 0 ? p->outlier_idx : nullptr,
                          d->n_outlier > 0 ? p->outlier_codebook : nullptr,
                          (d->flags & VPTQ_FLAG_SCALE_BIAS) ? p->scale : nullptr,
                          (d->flags & VPTQ_FLAG_SCALE_BIAS) ? p->bias : nullptr};
    for (int i = 0; i < 8; i++)
        if (all[i] != nullptr && !aligned16(all[i])) return VPTQ_E_ALIGN;
    return VPTQ_OK;
}

LayerView make_view(const vptq_layer_desc *d, const vptq_layer_ptrs *p)
{
    LayerView L;
    memset(&L, 0, sizeof(L));
    L.M = d->M; L.N = d->N; L.v = d->v; L.k1 = d->k1;
    L.n_out = d->n_outlier;
    L.v0 = L.n_out ? d->v0 : 1;
    L.k0 = L.n_out ? d->k0 : 1;
    L.Nc = L.N - L.n_out;
    L.k2 = L.Nc > 0 ? d->k2 : 0;
    L.G = (d->n_groups > 1 && L.Nc > 0) ? d->n_groups : 1;
    L.cpg = L.Nc > 0 ? ceil_div(L.Nc, L.G) : 1;
    L.R = ceil_div(L.M, L.v);
    L.R0 = L.n_out ? ceil_div(L.M, L.v0) : 0;
    L.has_scale = (d->flags & VPTQ_FLAG_SCALE_BIAS) ? 1 : 0;
    L.scale_rows = (d->flags & VPTQ_FLAG_SCALE_ROWS) ? 1 : 0;
    L.x_bf16 = d->x_dtype == VPTQ_DTYPE_BF16;
    L.out_dtype = d->out_dtype;
    // stream geometry is part of the view even without pointers (path selection reads it)
    L.s1 = make_stream(p ? p->packed_idx : nullptr, L.Nc, L.k1);
    L.s2 = make_stream((p && L.k2) ? p->res_idx : nullptr, L.Nc, L.k2 ? L.k2 : 1);
    L.s0 = make_stream((p && L.n_out) ? p->outlier_idx : nullptr, L.n_out, L.k0);
    if (p != nullptr) {
        L.c1 = reinterpret_cast<const __half *>(p->codebook);
        L.c2 = L.k2 ? reinterpret_cast<const __half *>(p->res_codebook) : nullptr;
        L.c0 = L.n_out ? reinterpret_cast<const __half *>(p->outlier_codebook) : nullptr;
        L.scale = L.has_scale ? reinterpret_cast<const __half *>(p->scale) : nullptr;
        L.bias = L.has_scale ? reinterpret_cast<const __half *>(p->bias) : nullptr;
        L.perm = (d->flags & VPTQ_FLAG_COL_PERM) ? reinterpret_cast<const int *>(p->col_perm) : nullptr;
        L.prepared = (d->flags & VPTQ_FLAG_PREPARED) ? p->prepared : nullptr;
    }
    L.prep_parts = (d->flags & VPTQ_FLAG_PREPARED) ? d->prepared_parts : 0;
    L.concurrent = (d->flags & VPTQ_FLAG_CONCURRENT) ? 1 : 0;
    L.deterministic = (d->flags & VPTQ_FLAG_DETERMINISTIC) ? 1 : 0;
    return L;
}

}  // namespace

extern "C" {

int vptq_index_bits(int32_t k)
{
    if (k < 1 || k > 65536) return VPTQ_E_SHAPE;
    return index_bits(k);
}

int64_t vptq_packed_row_bytes(int32_t n_cols, int32_t k)
{
    if (n_cols < 0 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    return row_bytes(n_cols, k);
}

int64_t vptq_packed_bytes(int32_t n_rows, int32_t n_cols, int32_t k)
{
    if (n_rows < 0 || n_cols < 0 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    return (int64_t)n_rows * row_bytes(n_cols, k);
}

int64_t vptq_layer_weight_bytes(const vptq_layer_desc *d)
{
    int rc = check_desc(d);
    if (rc != VPTQ_OK) return rc;
    LayerView L = make_view(d, nullptr);
    int64_t bytes = 0;
    if (L.Nc > 0) {
        bytes += (int64_t)L.R * row_bytes(L.Nc, L.k1) + 2LL * L.G * L.k1 * L.v;
        if (L.k2) bytes += (int64_t)L.R * row_bytes(L.Nc, L.k2) + 2LL * L.G * L.k2 * L.v;
    }
    if (L.n_out) bytes += (int64_t)L.R0 * row_bytes(L.n_out, L.k0) + 2LL * L.k0 * L.v0;
    if (L.has_scale) bytes += 4LL * (L.scale_rows ? L.M : L.N);
    if (d->flags & VPTQ_FLAG_COL_PERM) bytes += 4LL * L.N;
    return bytes;
}

int vptq_pack(const int32_t *idx, int32_t n_rows, int32_t n_cols, int32_t k,
              uint8_t *packed, int32_t *bad_count, void *stream)
{
    if (n_rows < 0 || n_cols < 0 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (n_rows == 0 || n_cols == 0) return VPTQ_OK;
    if (idx == nullptr || packed == nullptr) return VPTQ_E_NULL;
    if (!aligned16(packed)) return VPTQ_E_ALIGN;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (bad_count != nullptr) {
        e = cudaMemsetAsync(bad_count, 0, sizeof(int32_t), st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    e = launch_pack(idx, n_rows, n_cols, k, packed, bad_count, st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (bad_count != nullptr) {
        int32_t host_bad = 0;
        e = cudaMemcpyAsync(&host_bad, bad_count, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(e);
        if (host_bad != 0) return VPTQ_E_INDEX_RANGE;
    }
    return VPTQ_OK;
}

int vptq_unpack(const uint8_t *packed, int32_t n_rows, int32_t n_cols, int32_t k,
                int32_t *idx, void *stream)
{
    if (n_rows < 0 || n_cols < 0 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (n_rows == 0 || n_cols == 0) return VPTQ_OK;
    if (idx == nullptr || packed == nullptr) return VPTQ_E_NULL;
    if (!aligned16(packed)) return VPTQ_E_ALIGN;
    cudaError_t e = launch_unpack(packed, n_rows, n_cols, k, idx, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? VPTQ_OK : cuda_fail(e);
}

int vptq_pack_host(const int32_t *idx, int32_t n_rows, int32_t n_cols, int32_t k, uint8_t *packed)
{
    if (n_rows < 0 || n_cols < 0 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (n_rows == 0 || n_cols == 0) return VPTQ_OK;
    if (idx == nullptr || packed == nullptr) return VPTQ_E_NULL;
    return pack_host(idx, n_rows, n_cols, k, packed) == 0 ? VPTQ_OK : VPTQ_E_INDEX_RANGE;
}

int vptq_unpack_host(const uint8_t *packed, int32_t n_rows, int32_t n_cols, int32_t k, int32_t *idx)
{
    if (n_rows < 0 || n_cols < 0 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (n_rows == 0 || n_cols == 0) return VPTQ_OK;
    if (idx == nullptr || packed == nullptr) return VPTQ_E_NULL;
    unpack_host(packed, n_rows, n_cols, k, idx);
    return VPTQ_OK;
}

// descriptor -> geometry of the prepared image, or an error code
static int prepared_geometry_of(const vptq_layer_desc *desc, int32_t n_parts, PreparedGeometry *g)
{
    int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    if (n_parts < 0) return VPTQ_E_SHAPE;
    const LayerView L = make_view(desc, nullptr);
    if (!prepared_eligible(L) || (desc->flags & VPTQ_FLAG_SCALE_ROWS)) return VPTQ_E_UNSUPPORTED;
    return prepared_geometry(L, n_parts, g) ? VPTQ_OK : VPTQ_E_UNSUPPORTED;
}

int64_t vptq_prepare_bytes(const vptq_layer_desc *desc, int32_t n_parts)
{
    PreparedGeometry g;
    const int rc = prepared_geometry_of(desc, n_parts, &g);
    if (rc != VPTQ_OK) return rc;
    return (int64_t)prepared_capacity(g);
}

int vptq_prepare_host(const vptq_layer_desc *desc, const uint8_t *packed_idx, const uint8_t *res_idx,
                      int32_t n_parts, void *image, size_t image_bytes, size_t *used_bytes)
{
    PreparedGeometry g;
    const int rc = prepared_geometry_of(desc, n_parts, &g);
    if (rc != VPTQ_OK) return rc;
    if (packed_idx == nullptr || image == nullptr || (g.k2 > 0 && res_idx == nullptr)) return VPTQ_E_NULL;
    if (image_bytes < 256) return VPTQ_E_WORKSPACE;
    return prepare_host(g, packed_idx, res_idx, image, image_bytes, used_bytes);
}

int vptq_prepare(const vptq_layer_desc *desc, const vptq_layer_ptrs *p, int32_t n_parts,
                 void *image, size_t image_bytes, size_t *used_bytes, void *stream)
{
    PreparedGeometry g;
    int rc = prepared_geometry_of(desc, n_parts, &g);
    if (rc != VPTQ_OK) return rc;
    if (p == nullptr || p->packed_idx == nullptr || image == nullptr || (g.k2 > 0 && p->res_idx == nullptr)) return VPTQ_E_NULL;
    if ((reinterpret_cast<uintptr_t>(image) & 255u) != 0) return VPTQ_E_ALIGN;
    if (image_bytes < 256) return VPTQ_E_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t b1 = (size_t)g.R * (size_t)row_bytes(g.Nc, g.k1), b2 = g.k2 ? (size_t)g.R * (size_t)row_bytes(g.Nc, g.k2) : 0;
    std::vector<uint8_t> h1, h2, himg;
    try {
        h1.resize(b1); h2.resize(b2 ? b2 : 1); himg.resize(image_bytes);
    } catch (...) {
        return VPTQ_E_WORKSPACE;
    }
    cudaError_t e = cudaMemcpyAsync(h1.data(), p->packed_idx, b1, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && b2) e = cudaMemcpyAsync(h2.data(), p->res_idx, b2, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    size_t used = 0;
    rc = prepare_host(g, h1.data(), b2 ? h2.data() : nullptr, himg.data(), image_bytes, &used);
    if (used_bytes) *used_bytes = used;
    if (rc != VPTQ_OK) return rc;
    e = cudaMemcpyAsync(image, himg.data(), used, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? VPTQ_OK : cuda_fail(e);
}

int vptq_dequant(const vptq_layer_desc *desc, const vptq_layer_ptrs *p, void *W_out, void *stream)
{
    int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    rc = check_ptrs(desc, p);
    if (rc != VPTQ_OK) return rc;
    if (W_out == nullptr) return VPTQ_E_NULL;
    if (!aligned16(W_out)) return VPTQ_E_ALIGN;
    LayerView L = make_view(desc, p);
    cudaError_t e = launch_dequant(L, reinterpret_cast<__half *>(W_out), reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? VPTQ_OK : cuda_fail(e);
}

static bool assign_uses_tensor_cores(int32_t M, int32_t N, int32_t v, int32_t k, int32_t flags)
{
    return !(flags & VPTQ_FLAG_FORCE_GENERIC) && assign_tcgen05_supported(M, N, v, k);
}

const char *vptq_assign_path(int32_t M, int32_t N, int32_t v, int32_t k, int32_t flags)
{
    if (M < 0 || N < 0 || v < 1 || k < 1 || k > 65536 || !assign_supported(v, k)) return "invalid";
    return assign_uses_tensor_cores(M, N, v, k, flags) ? "assign_tcgen05" : "assign_fp32";
}

int64_t vptq_assign_workspace_bytes(int32_t M, int32_t N, int32_t v, int32_t k, int32_t flags)
{
    if (M < 0 || N < 0 || v < 1 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (!assign_supported(v, k)) return VPTQ_E_UNSUPPORTED;
    return assign_uses_tensor_cores(M, N, v, k, flags) ? assign_tcgen05_workspace_bytes(M, N, v, k) : 0;
}

int vptq_assign(const void *W, int32_t M, int32_t N, int32_t v, const void *codebook, int32_t k,
                int32_t *idx, int32_t flags, void *workspace, size_t workspace_bytes, void *stream)
{
    if (M < 0 || N < 0 || v < 1 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (!assign_supported(v, k)) return VPTQ_E_UNSUPPORTED;
    if (flags & ~VPTQ_FLAG_FORCE_GENERIC) return VPTQ_E_UNSUPPORTED;
    if (M == 0 || N == 0) return VPTQ_OK;
    if (W == nullptr || codebook == nullptr || idx == nullptr) return VPTQ_E_NULL;
    if ((reinterpret_cast<uintptr_t>(W) & 1u) || (reinterpret_cast<uintptr_t>(codebook) & 1u) ||
        (reinterpret_cast<uintptr_t>(idx) & 3u)) return VPTQ_E_ALIGN;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (assign_uses_tensor_cores(M, N, v, k, flags)) {
        if (workspace == nullptr || (long long)workspace_bytes < assign_tcgen05_workspace_bytes(M, N, v, k))
            return VPTQ_E_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return VPTQ_E_ALIGN;
        e = launch_assign_tcgen05(reinterpret_cast<const __half *>(W), M, N, v,
                                  reinterpret_cast<const __half *>(codebook), k, idx, workspace, st);
    } else {
        e = launch_assign(reinterpret_cast<const __half *>(W), M, N, v,
                          reinterpret_cast<const __half *>(codebook), k, idx, st);
    }
    return e == cudaSuccess ? VPTQ_OK : cuda_fail(e);
}

int64_t vptq_kmeans_update_workspace_bytes(int32_t v, int32_t k)
{
    if (v < 1 || v > 32 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    return kmeans_update_workspace_bytes(v, k);
}

int vptq_kmeans_update(const void *W, int32_t M, int32_t N, int32_t v, const int32_t *idx,
                       const float *col_weight, int32_t k, void *codebook,
                       void *workspace, size_t workspace_bytes, void *stream)
{
    if (M < 0 || N < 0 || v < 1 || v > 32 || k < 1 || k > 65536) return VPTQ_E_SHAPE;
    if (codebook == nullptr) return VPTQ_E_NULL;
    if (M > 0 && N > 0 && (W == nullptr || idx == nullptr)) return VPTQ_E_NULL;
    if (workspace == nullptr || (long long)workspace_bytes < kmeans_update_workspace_bytes(v, k)) return VPTQ_E_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(W) & 1u) || (reinterpret_cast<uintptr_t>(codebook) & 1u) ||
        (reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(col_weight) & 3u) ||
        (reinterpret_cast<uintptr_t>(workspace) & 3u)) return VPTQ_E_ALIGN;
    cudaError_t e = launch_kmeans_update(reinterpret_cast<const __half *>(W), M, N, v, idx, col_weight, k,
                                         reinterpret_cast<__half *>(codebook), workspace,
                                         reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? VPTQ_OK : cuda_fail(e);
}

int64_t vptq_linear_workspace_bytes(const vptq_layer_desc *desc, int32_t B)
{
    int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    if (B <= 0) return VPTQ_E_SHAPE;
    LayerView L = make_view(desc, nullptr);
    return linear_workspace_bytes(L, B, desc->flags);
}

int vptq_linear(const vptq_layer_desc *desc, const void *x, int32_t B,
                const vptq_layer_ptrs *p, void *out,
                void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    if (B <= 0) return VPTQ_E_SHAPE;
    rc = check_ptrs(desc, p);
    if (rc != VPTQ_OK) return rc;
    if (x == nullptr || out == nullptr) return VPTQ_E_NULL;
    if (!aligned16(x) || !aligned16(out)) return VPTQ_E_ALIGN;
    LayerView L = make_view(desc, p);
    long long need = linear_workspace_bytes(L, B, desc->flags);
    if (need > 0) {
        if (workspace == nullptr || (long long)workspace_bytes < need) return VPTQ_E_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return VPTQ_E_ALIGN;
    }
    cudaError_t e = cudaSuccess;
    rc = linear_dispatch(L, desc->flags, x, B, out, workspace, reinterpret_cast<cudaStream_t>(stream), &e);
    if (rc == VPTQ_E_CUDA) return cuda_fail(e);
    return rc;
}

// descriptors (and pointers) of a fused call -> views; VPTQ_OK or the first error
static int fused_views(const vptq_layer_desc *descs, const vptq_layer_ptrs *ptrs, int32_t n_layers, int32_t B,
                       LayerView *Ls, int *flags)
{
    if (descs == nullptr) return VPTQ_E_NULL;
    if (n_layers < 1 || n_layers > VPTQ_MAX_FUSED_LAYERS || B <= 0) return VPTQ_E_SHAPE;
    for (int l = 0; l < n_layers; l++) {
        int rc = check_desc(&descs[l]);
        if (rc != VPTQ_OK) return rc;
        if (descs[l].N != descs[0].N || descs[l].x_dtype != descs[0].x_dtype) return VPTQ_E_SHAPE;
        if (ptrs != nullptr) {
            rc = check_ptrs(&descs[l], &ptrs[l]);
            if (rc != VPTQ_OK) return rc;
        }
        Ls[l] = make_view(&descs[l], ptrs != nullptr ? &ptrs[l] : nullptr);
        flags[l] = descs[l].flags;
    }
    return VPTQ_OK;
}

int64_t vptq_linear_fused_workspace_bytes(const vptq_layer_desc *descs, int32_t n_layers, int32_t B)
{
    LayerView Ls[VPTQ_MAX_FUSED_LAYERS];
    int flags[VPTQ_MAX_FUSED_LAYERS];
    const int rc = fused_views(descs, nullptr, n_layers, B, Ls, flags);
    if (rc != VPTQ_OK) return rc;
    return linear_fused_workspace_bytes(Ls, flags, n_layers, B);
}

int vptq_linear_fused(const vptq_layer_desc *descs, const vptq_layer_ptrs *ptrs, int32_t n_layers,
                      const void *x, int32_t B, void *const *outs,
                      void *workspace, size_t workspace_bytes, void *stream)
{
    LayerView Ls[VPTQ_MAX_FUSED_LAYERS];
    int flags[VPTQ_MAX_FUSED_LAYERS];
    if (ptrs == nullptr || outs == nullptr || x == nullptr) return VPTQ_E_NULL;
    const int rc = fused_views(descs, ptrs, n_layers, B, Ls, flags);
    if (rc != VPTQ_OK) return rc;
    if (!aligned16(x)) return VPTQ_E_ALIGN;
    for (int l = 0; l < n_layers; l++) {
        if (outs[l] == nullptr) return VPTQ_E_NULL;
        if (!aligned16(outs[l])) return VPTQ_E_ALIGN;
    }
    const long long need = linear_fused_workspace_bytes(Ls, flags, n_layers, B);
    if (need > 0) {
        if (workspace == nullptr || (long long)workspace_bytes < need) return VPTQ_E_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return VPTQ_E_ALIGN;
    }
    cudaError_t e = cudaSuccess;
    const int rc2 = linear_fused_dispatch(Ls, flags, n_layers, x, B, outs, workspace,
                                          reinterpret_cast<cudaStream_t>(stream), &e);
    if (rc2 == VPTQ_E_CUDA) return cuda_fail(e);
    return rc2;
}

int vptq_linear_fused_launches(const vptq_layer_desc *descs, int32_t n_layers, int32_t B)
{
    LayerView Ls[VPTQ_MAX_FUSED_LAYERS];
    int flags[VPTQ_MAX_FUSED_LAYERS];
    const int rc = fused_views(descs, nullptr, n_layers, B, Ls, flags);
    if (rc != VPTQ_OK) return rc;
    return linear_fused_launches(Ls, flags, n_layers, B);
}

const char *vptq_linear_fused_path(const vptq_layer_desc *descs, int32_t n_layers, int32_t B)
{
    LayerView Ls[VPTQ_MAX_FUSED_LAYERS];
    int flags[VPTQ_MAX_FUSED_LAYERS];
    if (fused_views(descs, nullptr, n_layers, B, Ls, flags) != VPTQ_OK) return "invalid";
    return linear_fused_path_name(Ls, flags, n_layers, B);
}

// The device's address of a pinned (page-locked, mapped) host buffer, or nullptr for any other memory.  A kernel
// that stores every output element exactly once with plain stores can write such a buffer itself, which saves
// the copy that would otherwise follow it on the stream.
static void *device_alias_of_pinned_host(void *host)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
}

// Small activations from pinned host memory: a kernel that reads them over the bus and writes the device buffer
// starts sooner on a stream than a copy does (no copy engine to wake), and the decode kernel behind it may begin
// its prologue while it runs.  16-byte words; `n16` of them.
constexpr size_t FETCH_MAX_BYTES = 256 * 1024;
__global__ void __launch_bounds__(256) fetch_host_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int n16)
{
    pdl_launch_dependents();
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i < n16) dst[i] = src[i];
}

// x_host -> x_dev on the stream: by that kernel when x_host is pinned, both ends are 16-byte aligned and the size
// is a small multiple of 16 bytes, else by cudaMemcpyAsync.
static cudaError_t activations_to_device(void *x_dev, const void *x_host, size_t bytes, cudaStream_t st)
{
    if (bytes <= FETCH_MAX_BYTES && bytes % 16 == 0 && (reinterpret_cast<uintptr_t>(x_dev) & 15u) == 0) {
        void *alias = device_alias_of_pinned_host(const_cast<void *>(x_host));
        if (alias != nullptr && (reinterpret_cast<uintptr_t>(alias) & 15u) == 0) {
            const int n16 = (int)(bytes / 16);
            fetch_host_kernel<<<(n16 + 255) / 256, 256, 0, st>>>(reinterpret_cast<const uint4 *>(alias), reinterpret_cast<uint4 *>(x_dev), n16);
            return cudaGetLastError();
        }
    }
    return cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, st);
}

int vptq_linear_host_io(const vptq_layer_desc *desc, const void *x_host, int32_t B,
                        const vptq_layer_ptrs *p, void *out_host,
                        void *x_dev, void *out_dev,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    if (B <= 0) return VPTQ_E_SHAPE;
    if (x_host == nullptr || out_host == nullptr || x_dev == nullptr || out_dev == nullptr) return VPTQ_E_NULL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    size_t xb = (size_t)B * desc->N * 2;
    size_t ob = (size_t)B * desc->M * (desc->out_dtype == VPTQ_DTYPE_FP32 ? 4 : 2);
    cudaError_t e = activations_to_device(x_dev, x_host, xb, st);
    if (e != cudaSuccess) return cuda_fail(e);
    // the prepared-image kernel stores each output once: into the pinned host buffer directly when it can
    if (strcmp(vptq_linear_path(desc, B), "decode_bucket_fma") == 0) {
        void *alias = device_alias_of_pinned_host(out_host);
        if (alias != nullptr) return vptq_linear(desc, x_dev, B, p, alias, workspace, workspace_bytes, stream);
    }
    rc = vptq_linear(desc, x_dev, B, p, out_dev, workspace, workspace_bytes, stream);
    if (rc != VPTQ_OK) return rc;
    e = cudaMemcpyAsync(out_host, out_dev, ob, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e);
    return VPTQ_OK;
}

int vptq_linear_fused_host_io(const vptq_layer_desc *descs, const vptq_layer_ptrs *ptrs, int32_t n_layers,
                              const void *x_host, int32_t B, void *const *outs_host,
                              void *x_dev, void *const *outs_dev,
                              void *workspace, size_t workspace_bytes, void *stream)
{
    if (descs == nullptr || x_host == nullptr || outs_host == nullptr || x_dev == nullptr || outs_dev == nullptr)
        return VPTQ_E_NULL;
    if (n_layers < 1 || n_layers > VPTQ_MAX_FUSED_LAYERS || B <= 0) return VPTQ_E_SHAPE;
    for (int l = 0; l < n_layers; l++) {
        const int rc = check_desc(&descs[l]);
        if (rc != VPTQ_OK) return rc;
        if (outs_host[l] == nullptr || outs_dev[l] == nullptr) return VPTQ_E_NULL;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = activations_to_device(x_dev, x_host, (size_t)B * descs[0].N * 2, st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (strcmp(vptq_linear_fused_path(descs, n_layers, B), "fused_decode_bucket_fma") == 0) {
        void *alias[VPTQ_MAX_FUSED_LAYERS];
        bool all = true;
        for (int l = 0; l < n_layers; l++) all = (alias[l] = device_alias_of_pinned_host(outs_host[l])) != nullptr && all;
        if (all) return vptq_linear_fused(descs, ptrs, n_layers, x_dev, B, alias, workspace, workspace_bytes, stream);
    }
    const int rc = vptq_linear_fused(descs, ptrs, n_layers, x_dev, B, outs_dev, workspace, workspace_bytes, stream);
    if (rc != VPTQ_OK) return rc;
    for (int l = 0; l < n_layers; l++) {
        const size_t ob = (size_t)B * descs[l].M * (descs[l].out_dtype == VPTQ_DTYPE_FP32 ? 4 : 2);
        e = cudaMemcpyAsync(outs_host[l], outs_dev[l], ob, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return VPTQ_OK;
}

const char *vptq_status_string(int code)
{
    switch (code) {
    case VPTQ_OK: return "ok";
    case VPTQ_E_NULL: return "a required pointer is null";
    case VPTQ_E_SHAPE: return "bad shape or size argument";
    case VPTQ_E_ALIGN: return "a data pointer is not sufficiently aligned";
    case VPTQ_E_UNSUPPORTED: return "unsupported dtype or flag combination";
    case VPTQ_E_WORKSPACE: return "workspace missing or too small";
    case VPTQ_E_INDEX_RANGE: return "an index lies outside [0,k)";
    case VPTQ_E_CUDA: return "a CUDA runtime call failed";
    case VPTQ_E_TIMEOUT: return "a bounded device-side wait gave up";
    case VPTQ_E_SCRATCH_LIMIT: return "the layer needs more scratch than the built-in array of vptq_linear_noalloc holds";
    default: return "unknown status code";
    }
}

const char *vptq_last_cuda_error(void) { return g_cuda_err; }

void vptq_debug_set_wait_limit(uint64_t cycles) { set_debug_wait_limit(cycles); }

int vptq_workspace_status(const void *workspace, void *stream)
{
    if (workspace == nullptr) return VPTQ_OK;
    int32_t word = 0;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    return (word == VPTQ_E_TIMEOUT || word == VPTQ_E_UNSUPPORTED) ? word : VPTQ_OK;
}

const char *vptq_linear_path(const vptq_layer_desc *desc, int32_t B)
{
    if (check_desc(desc) != VPTQ_OK || B <= 0) return "invalid";
    LayerView L = make_view(desc, nullptr);
    return linear_path_name(L, B, desc->flags);
}

int vptq_linear_waits_between_ctas(const vptq_layer_desc *desc, int32_t B)
{
    const int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    if (B <= 0) return VPTQ_E_SHAPE;
    LayerView L = make_view(desc, nullptr);
    return choose_path(L, B, desc->flags) == PATH_GEMM_TCGEN05 && gemm_tcgen05_waits_between_ctas(L, B) ? 1 : 0;
}

int vptq_linear_launches(const vptq_layer_desc *desc, int32_t B)
{
    if (check_desc(desc) != VPTQ_OK || B <= 0) return VPTQ_E_SHAPE;
    LayerView L = make_view(desc, nullptr);
    return linear_launches(L, B, desc->flags);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// vptq_linear_noalloc: the split-K decode kernel with its scratch in a built-in device array.
// ---------------------------------------------------------------------------------------------
// The array lives in this library's device image: every GPU that loads the library holds
// VPTQ_NOALLOC_SCRATCH_BYTES of it until the process exits.  In host code the name below is
// only a handle for the runtime, not a device address, so the address is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernel receives.
static __device__ __align__(256) unsigned char g_noalloc_scratch[VPTQ_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void *g_noalloc_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on the CURRENT device (looked up on first use).
int noalloc_scratch(void **ptr)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return VPTQ_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_ptr[dev] == nullptr) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        if (p == nullptr) return VPTQ_E_CUDA;
        g_noalloc_ptr[dev] = p;
    }
    *ptr = g_noalloc_ptr[dev];
    return VPTQ_OK;
}

}  // namespace

extern "C" int vptq_linear_noalloc(const vptq_layer_desc *desc, const void *x, int32_t B,
                                   const vptq_layer_ptrs *p, void *out, void *stream)
{
    int rc = check_desc(desc);
    if (rc != VPTQ_OK) return rc;
    if (B <= 0 || B > 16) return VPTQ_E_SHAPE;
    rc = check_ptrs(desc, p);
    if (rc != VPTQ_OK) return rc;
    if (x == nullptr || out == nullptr) return VPTQ_E_NULL;
    if (!aligned16(x) || !aligned16(out)) return VPTQ_E_ALIGN;
    if (desc->flags & VPTQ_FLAG_FORCE_GENERIC) return VPTQ_E_UNSUPPORTED;
    LayerView L = make_view(desc, p);
    if (!l2_fma_supported(L, B)) return VPTQ_E_UNSUPPORTED;
    if (l2_fma_workspace_bytes(L, B) > (long long)VPTQ_NOALLOC_SCRATCH_BYTES) return VPTQ_E_SCRATCH_LIMIT;
    void *scratch = nullptr;
    rc = noalloc_scratch(&scratch);
    if (rc != VPTQ_OK) return rc;
    // the launcher clears the part of the scratch that has to start at zero, on `stream`
    cudaError_t e = launch_decode_l2_fma(L, x, B, out, scratch, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? VPTQ_OK : cuda_fail(e);
}

