// Plain fallback for the fused linear layer: any vector length, any index width, any
// batch.  One warp per output row m; lanes stride over the input columns, restore each
// weight from its index (Sec. 2.2 lookup, Sec. 3.2.2 residual sum, Sec. 3.2.3 outliers) and
// accumulate in FP32.  It re-reads every index v times, so it is only used for geometries
// the specialised kernels do not cover (and by the tests, to check those kernels against a
// second CUDA formulation).
#include "common.cuh"

namespace vptq {

constexpr int GEN_TB = 4;   // tokens per pass

__global__ void __launch_bounds__(256)
linear_generic_kernel(LayerView L, const void *__restrict__ x, int B, void *__restrict__ out)
{
    const int warp = (int)((blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (warp >= L.M) return;
    const int m = warp;
    const int r = m / L.v, j = m % L.v;
    const int r0 = L.n_out ? m / L.v0 : 0, j0 = L.n_out ? m % L.v0 : 0;
    const uint8_t *row1 = L.s1.ptr + (long long)r * L.s1.stride;
    const uint8_t *row2 = L.k2 ? L.s2.ptr + (long long)r * L.s2.stride : nullptr;
    const uint8_t *row0 = L.n_out ? L.s0.ptr + (long long)r0 * L.s0.stride : nullptr;
    float sm = 1.f, bm = 0.f;
    if (L.has_scale && L.scale_rows) {
        sm = __half2float(L.scale[m]);
        bm = __half2float(L.bias[m]);
    }
    for (int t0 = 0; t0 < B; t0 += GEN_TB) {
        float acc[GEN_TB];
#pragma unroll
        for (int t = 0; t < GEN_TB; t++) acc[t] = 0.f;
        for (int n = lane; n < L.N; n += 32) {
            float w;
            if (n < L.n_out) {
                int i0 = clamp_index(load_index(row0, n, L.s0.bits), L.k0);
                w = __half2float(__ldg(L.c0 + (long long)i0 * L.v0 + j0));
            } else {
                int c = n - L.n_out;
                int i1 = clamp_index(load_index(row1, c, L.s1.bits), L.k1);
                const int g = c / L.cpg;          // Sec. 3.1: this column's group has its own tables
                w = __half2float(__ldg(L.c1 + ((long long)g * L.k1 + i1) * L.v + j));
                if (L.k2) {
                    int i2 = clamp_index(load_index(row2, c, L.s2.bits), L.k2);
                    w += __half2float(__ldg(L.c2 + ((long long)g * L.k2 + i2) * L.v + j));
                }
            }
            if (L.has_scale) {
                float s = L.scale_rows ? sm : __half2float(__ldg(L.scale + n));
                float b = L.scale_rows ? bm : __half2float(__ldg(L.bias + n));
                w = w * s + b;
            }
#pragma unroll
            for (int t = 0; t < GEN_TB; t++)
                if (t0 + t < B) acc[t] += load_act(x, (long long)(t0 + t) * L.N + in_col(L, n), L.x_bf16) * w;
        }
#pragma unroll
        for (int t = 0; t < GEN_TB; t++) {
            float a = acc[t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0 && t0 + t < B) store_out(out, (long long)(t0 + t) * L.M + m, a, L.out_dtype);
        }
    }
}

long long generic_workspace_bytes(const LayerView &, int) { return 0; }
int generic_launches(const LayerView &, int) { return 1; }

cudaError_t launch_linear_generic(const LayerView &L, const void *x, int B, void *out,
                                  void *, cudaStream_t st)
{
    long long threads = (long long)L.M * 32;
    int grid = (int)((threads + 255) / 256);
    linear_generic_kernel<<<grid, 256, 0, st>>>(L, x, B, out);
    return cudaGetLastError();
}

}  // namespace vptq
