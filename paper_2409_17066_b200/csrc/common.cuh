// Shared device/host helpers of libvptq (CUDA side only; the CPU oracle has its own).
#pragma once

#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/vptq.h"

namespace vptq {

// ---- host-side format arithmetic -----------------------------------------------------
__host__ __device__ inline int index_bits(int k)
{
    int b = 0;
    while ((1 << b) < k) b++;
    return b < 1 ? 1 : b;
}

__host__ __device__ inline long long row_bytes(int cols, int k)
{
    long long bytes = ((long long)cols * index_bits(k) + 7) / 8;
    return (bytes + 15) / 16 * 16;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// One packed index stream as the kernels see it.
struct Stream {
    const uint8_t *ptr;    // packed rows
    long long stride;      // bytes per row (multiple of 16)
    int bits;              // bits per index
    int k;                 // codebook size (indices are clamped to k-1)
};

inline Stream make_stream(const uint8_t *p, int cols, int k)
{
    Stream s;
    s.ptr = p;
    s.stride = row_bytes(cols, k);
    s.bits = index_bits(k);
    s.k = k;
    return s;
}

// Kernel-side view of a layer.
struct LayerView {
    int M, N, v, k1, k2, n_out, v0, k0;
    int R, R0, Nc;
    int G, cpg;            // column groups with codebooks of their own, columns per group (Sec. 3.1)
    int has_scale, scale_rows;
    int x_bf16, out_dtype;
    Stream s1, s2, s0;
    const __half *c1, *c2, *c0;
    const __half *scale, *bias;
    const int *perm;       // nullptr, or [N]: stored column n is input feature perm[n] (Sec. 3.2.3)
    const void *prepared;  // nullptr, or the prepared image of the layer
    int prep_parts;        // partitions of the prepared image
    int concurrent;        // the call may share the GPU: no waits between CTAs of a grid
    int deterministic;     // every sum in a fixed order
};

#ifdef __CUDACC__
// ---- device helpers --------------------------------------------------------------------

// Index c of a packed row, any bit width 1..16.  Reads one or two aligned 32-bit words;
// the second word is touched only when the index crosses a word boundary, in which case it
// lies inside the row.
__device__ __forceinline__ int load_index(const uint8_t *row, int c, int bits)
{
    unsigned bit = (unsigned)c * (unsigned)bits;
    const uint32_t *w = reinterpret_cast<const uint32_t *>(row) + (bit >> 5);
    unsigned sh = bit & 31u;
    uint32_t lo = __ldg(w);
    uint32_t hi = (sh + bits > 32u) ? __ldg(w + 1) : 0u;
    uint32_t val = __funnelshift_r(lo, hi, sh);
    return (int)(val & ((1u << bits) - 1u));
}

__device__ __forceinline__ int clamp_index(int i, int k) { return i < k ? i : k - 1; }

// a0 += x * lo(w), a1 += x * hi(w) with x and the two halves of w in FP16: the mixed-precision fma of sm_100
// (f16 factors, f32 addend and result; the product of two f16 values is exact in f32, so this is the same
// arithmetic as converting both factors and using an f32 fma, in a third of the instructions).
// `hi_x` selects the upper half of xw as x.
__device__ __forceinline__ void fma_f16x2(float &a0, float &a1, uint32_t xw, bool hi_x, uint32_t w)
{
    if (hi_x)
        asm("{\n\t.reg .b16 xl, xh, lo, hi;\n\tmov.b32 {xl, xh}, %2;\n\tmov.b32 {lo, hi}, %3;\n\t"
            "fma.rn.f32.f16 %0, xh, lo, %0;\n\tfma.rn.f32.f16 %1, xh, hi, %1;\n\t}" : "+f"(a0), "+f"(a1) : "r"(xw), "r"(w));
    else
        asm("{\n\t.reg .b16 xl, xh, lo, hi;\n\tmov.b32 {xl, xh}, %2;\n\tmov.b32 {lo, hi}, %3;\n\t"
            "fma.rn.f32.f16 %0, xl, lo, %0;\n\tfma.rn.f32.f16 %1, xl, hi, %1;\n\t}" : "+f"(a0), "+f"(a1) : "r"(xw), "r"(w));
}

// Programmatic dependent launch (the decode kernels of consecutive calls on a stream): a kernel lets the next
// one start as soon as SMs free up, and waits for the previous one only where it first touches data that the
// previous one may have written (the activations).  What comes before the wait must read weights only and
// write nothing outside the CTA.  Both are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Input feature of stored column n.  A list entry outside [0, N) is clamped, as indices are.
__device__ __forceinline__ int in_col(const LayerView &L, int n)
{
    if (L.perm == nullptr) return n;
    const unsigned f = (unsigned)__ldg(L.perm + n);
    return (int)(f < (unsigned)L.N ? f : (unsigned)(L.N - 1));
}

__device__ __forceinline__ float load_act(const void *x, long long i, int is_bf16)
{
    if (is_bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(x)[i]);
    return __half2float(reinterpret_cast<const __half *>(x)[i]);
}

__device__ __forceinline__ void store_out(void *out, long long i, float val, int dtype)
{
    if (dtype == VPTQ_DTYPE_FP16) reinterpret_cast<__half *>(out)[i] = __float2half_rn(val);
    else if (dtype == VPTQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16 *>(out)[i] = __float2bfloat16_rn(val);
    else reinterpret_cast<float *>(out)[i] = val;
}
#endif

// streaming multiprocessors of the current device, cached per device ordinal (device_info.cu)
int device_sm_count();

// limit, in clock cycles, of the bounded device-side waits: 0 = each kernel's default (about two seconds);
// set by vptq_debug_set_wait_limit, for tests that let a wait run out (device_info.cu)
unsigned long long debug_wait_limit();
void set_debug_wait_limit(unsigned long long cycles);

// true unless the environment variable VPTQ_NO_PDL names this kernel family (or "all"): then the kernel is
// launched the ordinary way, after the stream's previous kernel has finished (device_info.cu)
bool pdl_enabled(const char *family);

#ifdef __CUDACC__
// Launch `kernel` as a programmatic dependent of the stream's previous kernel (see pdl_wait above).
template <typename Params>
inline cudaError_t launch_dependent(const char *family, void (*kernel)(Params), int grid, int block, size_t smem,
                                    cudaStream_t st, const Params &P)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled(family) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, P);
}
#endif

// ---- launchers implemented in the kernel files -------------------------------------------
cudaError_t launch_pack(const int32_t *idx, int rows, int cols, int k, uint8_t *packed,
                        int32_t *bad_count, cudaStream_t st);
cudaError_t launch_unpack(const uint8_t *packed, int rows, int cols, int k, int32_t *idx,
                          cudaStream_t st);
// the same two steps on host memory (pack_host.cu); pack_host returns the number of indices outside [0,k)
long long pack_host(const int32_t *idx, int rows, int cols, int k, uint8_t *packed);
void unpack_host(const uint8_t *packed, int rows, int cols, int k, int32_t *idx);
cudaError_t launch_dequant(const LayerView &L, __half *W, cudaStream_t st);
// assignment step of the quantizer (Eq. 2): idx [ceil(M/v)][N]
bool assign_supported(int v, int k);
// (weighted) k-means centroid update (Sec. 3.2.1); workspace = 2*k*v floats
long long kmeans_update_workspace_bytes(int v, int k);
cudaError_t launch_kmeans_update(const __half *W, int M, int N, int v, const int *idx, const float *h, int k,
                                 __half *C, void *ws, cudaStream_t st);
cudaError_t launch_assign(const __half *W, int M, int N, int v, const __half *C, int k, int *idx, cudaStream_t st);

// generic fallback linear (any geometry, any B): workspace = B*M floats
long long generic_workspace_bytes(const LayerView &L, int B);
cudaError_t launch_linear_generic(const LayerView &L, const void *x, int B, void *out,
                                  void *ws, cudaStream_t st);
int generic_launches(const LayerView &L, int B);

}  // namespace vptq
