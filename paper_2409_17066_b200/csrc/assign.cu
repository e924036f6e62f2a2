// Assignment step of the quantizer (Eq. 2): every length-v vector of the weight matrix (v consecutive
// rows of one column: Sec. 3.1, Algorithm 1) takes the index of the centroid at the smallest squared
// Euclidean distance.
//
// Floating point decides an integer here, so the arithmetic is part of the definition: FP32, components
// in ascending order, d = fma(t, t, d) with t = x_j - c_j; of equal distances the lowest index wins; a
// NaN distance never wins.  Components that do not exist (the last vector row when v does not divide M)
// are left out.
//
// One thread per vector (its components in registers), 256 vectors per block, consecutive threads on
// consecutive columns (coalesced loads of W).  The codebook passes through shared memory in chunks of
// 4096 / VMAX centroids converted to FP32 and zero-padded to VMAX components; all threads of a warp read the
// same centroid (broadcast).  The work is n_vectors * k * v subtract + fma pairs: bound by the FP32
// pipes, not by memory (the codebook is re-read from L2 once per block).
#include "common.cuh"
#include "assign.cuh"

namespace vptq {

namespace {

constexpr int ASSIGN_THREADS = 256;
constexpr int CHUNK_FLOATS = 4096;        // 16 KB of shared memory: CHUNK_FLOATS / VMAX centroids per chunk

template <int VMAX>
__global__ void __launch_bounds__(ASSIGN_THREADS)
assign_kernel(const __half *__restrict__ W, int M, int N, int v, const __half *__restrict__ C, int k,
              int *__restrict__ idx, long long n_vectors)
{
    constexpr int CHUNK = CHUNK_FLOATS / VMAX;
    __shared__ __align__(16) float cb[CHUNK_FLOATS];
    const long long g = (long long)blockIdx.x * ASSIGN_THREADS + threadIdx.x;
    const bool valid = g < n_vectors;
    const int r = valid ? (int)(g / N) : 0, n = valid ? (int)(g % N) : 0;
    const int vlen = min(v, M - r * v);              // components of this vector that exist
    float x[VMAX];
#pragma unroll
    for (int j = 0; j < VMAX; j++)
        x[j] = (valid && j < vlen) ? __half2float(__ldg(W + (long long)(r * v + j) * N + n)) : 0.f;

    float best_d = __int_as_float(0x7f800000);        // +inf
    int best = 0;
    for (int c0 = 0; c0 < k; c0 += CHUNK) {
        const int cn = min(CHUNK, k - c0);
        __syncthreads();                               // the previous chunk has been read
        for (int e = threadIdx.x; e < cn * VMAX; e += ASSIGN_THREADS) {
            const int i = e / VMAX, j = e % VMAX;
            cb[e] = j < v ? __half2float(__ldg(C + (long long)(c0 + i) * v + j)) : 0.f;
        }
        __syncthreads();
        if (!valid) continue;
        if (vlen == v) {
            // components j >= v are zero in the vector and in the table: they add fma(0, 0, d) = d
#pragma unroll 4
            for (int i = 0; i < cn; i++) {
                float d = 0.f;
#pragma unroll
                for (int j = 0; j < VMAX; j++) {
                    const float t = __fsub_rn(x[j], cb[i * VMAX + j]);
                    d = __fmaf_rn(t, t, d);
                }
                if (d < best_d) { best_d = d; best = c0 + i; }
            }
        } else {
            for (int i = 0; i < cn; i++) {
                float d = 0.f;
#pragma unroll
                for (int j = 0; j < VMAX; j++) {
                    const float t = j < vlen ? __fsub_rn(x[j], cb[i * VMAX + j]) : 0.f;
                    d = __fmaf_rn(t, t, d);
                }
                if (d < best_d) { best_d = d; best = c0 + i; }
            }
        }
    }
    if (valid) idx[g] = best;
}

// ---- the same decision for a short list of vectors: a warp takes VPW vectors at a time and its lanes share out
//      the centroids (component-major in shared memory: consecutive lanes, consecutive banks); every table
//      value read serves VPW distances ----
constexpr int LISTED_WARPS = 8;

template <int VMAX, int VPW>
__global__ void __launch_bounds__(LISTED_WARPS * 32)
assign_listed_kernel(const __half *__restrict__ W, int M, int N, int v, const __half *__restrict__ C, int k,
                     int *__restrict__ idx, const int *__restrict__ list, const int *__restrict__ count)
{
    constexpr int CHUNK = CHUNK_FLOATS / VMAX;
    constexpr int PER_BLOCK = LISTED_WARPS * VPW;
    __shared__ __align__(16) float cb[CHUNK_FLOATS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cnt = __ldg(count);
    for (long long first = (long long)blockIdx.x * PER_BLOCK; first < cnt; first += (long long)gridDim.x * PER_BLOCK) {
        long long g[VPW];
        int vlen[VPW];
        bool valid[VPW];
        float x[VPW][VMAX];
#pragma unroll
        for (int u = 0; u < VPW; u++) {
            const long long slot = first + warp * VPW + u;
            valid[u] = slot < cnt;
            g[u] = valid[u] ? __ldg(list + slot) : 0;
            const int r = (int)(g[u] / N), n = (int)(g[u] % N);
            vlen[u] = min(v, M - r * v);
#pragma unroll
            for (int j = 0; j < VMAX; j++)
                x[u][j] = (valid[u] && j < vlen[u]) ? __half2float(__ldg(W + (long long)(r * v + j) * N + n)) : 0.f;
        }
        float best_d[VPW];
        int best[VPW];
#pragma unroll
        for (int u = 0; u < VPW; u++) { best_d[u] = __int_as_float(0x7f800000); best[u] = 0x7fffffff; }   // nothing finite yet
        for (int c0 = 0; c0 < k; c0 += CHUNK) {
            const int cn = min(CHUNK, k - c0);
            __syncthreads();
            for (int e = threadIdx.x; e < cn * VMAX; e += LISTED_WARPS * 32) {
                const int i = e / VMAX, j = e % VMAX;
                cb[j * CHUNK + i] = j < v ? __half2float(__ldg(C + (long long)(c0 + i) * v + j)) : 0.f;
            }
            __syncthreads();
            if (!valid[0]) continue;
            // (ascending within a lane: the first of equal distances stays)
            for (int i = lane; i < cn; i += 32) {
                float c[VMAX];
#pragma unroll
                for (int j = 0; j < VMAX; j++) c[j] = cb[j * CHUNK + i];
#pragma unroll
                for (int u = 0; u < VPW; u++) {
                    float d = 0.f;
#pragma unroll
                    for (int j = 0; j < VMAX; j++) {
                        const float t = j < vlen[u] ? __fsub_rn(x[u][j], c[j]) : 0.f;
                        d = __fmaf_rn(t, t, d);
                    }
                    if (d < best_d[u]) { best_d[u] = d; best[u] = c0 + i; }
                }
            }
        }
        // across the lanes: the smallest distance, and of equal distances the lowest index
#pragma unroll
        for (int u = 0; u < VPW; u++) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float od = __shfl_xor_sync(0xffffffffu, best_d[u], o);
                const int oi = __shfl_xor_sync(0xffffffffu, best[u], o);
                if (od < best_d[u] || (od == best_d[u] && oi < best[u])) { best_d[u] = od; best[u] = oi; }
            }
            if (valid[u] && lane == 0) idx[g[u]] = best[u] == 0x7fffffff ? 0 : best[u];
        }
    }
}

}  // namespace

bool assign_supported(int v, int k) { return v >= 1 && v <= 32 && k >= 1 && k <= 65536; }

cudaError_t launch_assign(const __half *W, int M, int N, int v, const __half *C, int k, int *idx, cudaStream_t st)
{
    const long long n_vectors = (long long)ceil_div(M, v) * N;
    if (n_vectors == 0) return cudaSuccess;
    const long long blocks = (n_vectors + ASSIGN_THREADS - 1) / ASSIGN_THREADS;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)blocks);
    if (v <= 4) assign_kernel<4><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors);
    else if (v <= 8) assign_kernel<8><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors);
    else if (v <= 16) assign_kernel<16><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors);
    else assign_kernel<32><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors);
    return cudaGetLastError();
}

cudaError_t launch_assign_listed(const __half *W, int M, int N, int v, const __half *C, int k, int *idx,
                                 const int *list, const int *count, int sm_count, cudaStream_t st)
{
    // a fixed grid (the count is on the device): every block takes up to 32 listed vectors at a time
    const dim3 grid((unsigned)(8 * sm_count));
    if (v <= 4) assign_listed_kernel<4, 4><<<grid, LISTED_WARPS * 32, 0, st>>>(W, M, N, v, C, k, idx, list, count);
    else if (v <= 8) assign_listed_kernel<8, 4><<<grid, LISTED_WARPS * 32, 0, st>>>(W, M, N, v, C, k, idx, list, count);
    else if (v <= 16) assign_listed_kernel<16, 2><<<grid, LISTED_WARPS * 32, 0, st>>>(W, M, N, v, C, k, idx, list, count);
    else assign_listed_kernel<32, 1><<<grid, LISTED_WARPS * 32, 0, st>>>(W, M, N, v, C, k, idx, list, count);
    return cudaGetLastError();
}

}  // namespace vptq
