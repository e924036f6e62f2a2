// Bit-exact restoration of the FP16 weight matrix from indices and codebooks
// (Sec. 2.2 lookup; Sec. 3.2.2 residual sum; Sec. 3.2.3 outlier columns; App. D.2 "restore
// to FP16").  One thread per (vector row, input column): it reads its index (or two),
// gathers the centroid(s) and writes v weights down the column.  Adjacent threads own
// adjacent columns, so every row of stores is contiguous.
#include "common.cuh"

namespace vptq {

__device__ __forceinline__ __half finish_weight(float t, int has_scale, float s, float b)
{
    if (has_scale) {
        float p = __fmul_rn(t, s);     // separately rounded multiply and add: never contracted to an FMA
        t = __fadd_rn(p, b);
    }
    return __float2half_rn(t);
}

__global__ void __launch_bounds__(256)
dequant_kernel(LayerView L, __half *__restrict__ W)
{
    // blockIdx.y selects the region: 0 = main columns, 1 = outlier columns
    const bool outlier = (blockIdx.y == 1);
    const int cols = outlier ? L.n_out : L.Nc;
    const int vrows = outlier ? L.R0 : L.R;
    const int vlen = outlier ? L.v0 : L.v;
    long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (long long)vrows * cols) return;
    const int r = (int)(gid / cols);
    const int c = (int)(gid % cols);
    const int n = outlier ? c : c + L.n_out;

    const __half *e1, *e2 = nullptr;
    if (outlier) {
        int i0 = clamp_index(load_index(L.s0.ptr + (long long)r * L.s0.stride, c, L.s0.bits), L.k0);
        e1 = L.c0 + (long long)i0 * vlen;
    } else {
        int i1 = clamp_index(load_index(L.s1.ptr + (long long)r * L.s1.stride, c, L.s1.bits), L.k1);
        const int g = c / L.cpg;                       // Sec. 3.1: this column's group has its own tables
        e1 = L.c1 + ((long long)g * L.k1 + i1) * vlen;
        if (L.k2 > 0) {
            int i2 = clamp_index(load_index(L.s2.ptr + (long long)r * L.s2.stride, c, L.s2.bits), L.k2);
            e2 = L.c2 + ((long long)g * L.k2 + i2) * vlen;
        }
    }
    float s = 1.f, b = 0.f;
    if (L.has_scale && !L.scale_rows) {
        s = __half2float(__ldg(L.scale + n));
        b = __half2float(__ldg(L.bias + n));
    }
    const int m0 = r * vlen;
    for (int j = 0; j < vlen; j++) {
        int m = m0 + j;
        if (m >= L.M) break;              // last vector row may be partial: extra components are dropped
        float t = __half2float(__ldg(e1 + j));
        if (e2 != nullptr) t = __fadd_rn(t, __half2float(__ldg(e2 + j)));
        if (L.has_scale && L.scale_rows) {
            s = __half2float(__ldg(L.scale + m));
            b = __half2float(__ldg(L.bias + m));
        }
        W[(long long)m * L.N + in_col(L, n)] = finish_weight(t, L.has_scale, s, b);
    }
}

cudaError_t launch_dequant(const LayerView &L, __half *W, cudaStream_t st)
{
    long long main_items = (long long)L.R * L.Nc;
    long long out_items = (long long)L.R0 * L.n_out;
    long long most = main_items > out_items ? main_items : out_items;
    if (most == 0) return cudaSuccess;
    dim3 grid((unsigned)((most + 255) / 256), L.n_out > 0 ? 2 : 1);
    dequant_kernel<<<grid, 256, 0, st>>>(L, W);
    return cudaGetLastError();
}

}  // namespace vptq
