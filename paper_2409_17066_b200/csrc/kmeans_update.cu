// Centroid update of (weighted) k-means (Sec. 2.2: k-means builds the codebook; Sec. 3.2.1: with the
// Hessian diagonal of a vector's column as its weight): with the assignment fixed, every centroid
// becomes the weighted mean of the vectors assigned to it,
//   C_i[j] = sum h_n x_j / sum h_n   over vectors (r, n) with idx[r][n] = i that have component j,
// and a component that received no weight keeps its old value.
//
// accumulate: one thread per vector adds h*x and h into FP32 sums per (centroid, component): in a
//             shared-memory copy per block when the table is small (k*v <= 4096: few centroids mean many
//             vectors per address), straight into the workspace otherwise;
// finish:     one thread per (centroid, component): C = fp16(sum / weight) where weight > 0.
// FP32 atomic sums: the order of the additions is not fixed, so the result agrees with a FP64 mean
// to FP32 summation error, not bit for bit.
#include "common.cuh"

namespace vptq {

namespace {

constexpr int KM_THREADS = 256;
constexpr int KM_SMEM_ENTRIES = 4096;      // (centroid, component) pairs that fit the per-block copy: 32 KB

template <bool PRIVATE>
__global__ void __launch_bounds__(KM_THREADS)
kmeans_accumulate_kernel(const __half *__restrict__ W, int M, int N, int v, const int *__restrict__ idx,
                         const float *__restrict__ h, int k, float *__restrict__ sums, float *__restrict__ wsums,
                         long long n_vectors)
{
    __shared__ float s_sum[PRIVATE ? KM_SMEM_ENTRIES : 1];
    __shared__ float s_w[PRIVATE ? KM_SMEM_ENTRIES : 1];
    const int entries = k * v;
    if (PRIVATE) {
        for (int e = threadIdx.x; e < entries; e += KM_THREADS) { s_sum[e] = 0.f; s_w[e] = 0.f; }
        __syncthreads();
    }
    for (long long g = (long long)blockIdx.x * KM_THREADS + threadIdx.x; g < n_vectors;
         g += (long long)gridDim.x * KM_THREADS) {
        const int r = (int)(g / N), n = (int)(g % N);
        const int i = __ldg(idx + g);
        if (i < 0 || i >= k) continue;                 // an index outside the table takes no part
        const float w = h != nullptr ? __ldg(h + n) : 1.f;
        const int vlen = min(v, M - r * v);
        for (int j = 0; j < vlen; j++) {
            const float x = __half2float(__ldg(W + (long long)(r * v + j) * N + n));
            if (PRIVATE) {
                atomicAdd(&s_sum[i * v + j], w * x);
                atomicAdd(&s_w[i * v + j], w);
            } else {
                atomicAdd(sums + (long long)i * v + j, w * x);
                atomicAdd(wsums + (long long)i * v + j, w);
            }
        }
    }
    if (PRIVATE) {
        __syncthreads();
        for (int e = threadIdx.x; e < entries; e += KM_THREADS)
            if (s_w[e] != 0.f) { atomicAdd(sums + e, s_sum[e]); atomicAdd(wsums + e, s_w[e]); }
    }
}

__global__ void __launch_bounds__(KM_THREADS)
kmeans_finish_kernel(const float *__restrict__ sums, const float *__restrict__ wsums, long long entries,
                     __half *__restrict__ C)
{
    const long long e = (long long)blockIdx.x * KM_THREADS + threadIdx.x;
    if (e >= entries) return;
    const float w = wsums[e];
    if (w > 0.f) C[e] = __float2half_rn(__fdiv_rn(sums[e], w));
}

}  // namespace

long long kmeans_update_workspace_bytes(int v, int k) { return 2LL * k * v * (long long)sizeof(float); }

cudaError_t launch_kmeans_update(const __half *W, int M, int N, int v, const int *idx, const float *h, int k,
                                 __half *C, void *ws, cudaStream_t st)
{
    const long long entries = (long long)k * v;
    const long long n_vectors = (long long)ceil_div(M, v) * N;
    float *sums = reinterpret_cast<float *>(ws);
    float *wsums = sums + entries;
    cudaError_t e = cudaMemsetAsync(ws, 0, (size_t)kmeans_update_workspace_bytes(v, k), st);
    if (e != cudaSuccess) return e;
    if (n_vectors == 0) return cudaSuccess;
    if (entries <= KM_SMEM_ENTRIES) {
        // a block flushes its copy once: give every block many vectors
        long long blocks = (n_vectors + 16LL * KM_THREADS - 1) / (16LL * KM_THREADS);
        if (blocks > 4096) blocks = 4096;
        kmeans_accumulate_kernel<true><<<(unsigned)blocks, KM_THREADS, 0, st>>>(W, M, N, v, idx, h, k, sums, wsums, n_vectors);
    } else {
        long long blocks = (n_vectors + KM_THREADS - 1) / KM_THREADS;
        if (blocks > 65535LL * 16) blocks = 65535LL * 16;
        kmeans_accumulate_kernel<false><<<(unsigned)blocks, KM_THREADS, 0, st>>>(W, M, N, v, idx, h, k, sums, wsums, n_vectors);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    kmeans_finish_kernel<<<(unsigned)((entries + KM_THREADS - 1) / KM_THREADS), KM_THREADS, 0, st>>>(sums, wsums, entries, C);
    return cudaGetLastError();
}

}  // namespace vptq
