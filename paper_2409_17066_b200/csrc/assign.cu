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
              int *__restrict__ idx, long long n_vectors, const int *__restrict__ list, const int *__restrict__ count)
{
    constexpr int CHUNK = CHUNK_FLOATS / VMAX;
    __shared__ __align__(16) float cb[CHUNK_FLOATS];
    // all vectors, or (list != nullptr) the vectors list[0 .. *count) only
    const long long slot = (long long)blockIdx.x * ASSIGN_THREADS + threadIdx.x;
    long long g = slot;
    bool valid = slot < n_vectors;
    if (list != nullptr) {
        const int cnt = __ldg(count);
        if ((long long)blockIdx.x * ASSIGN_THREADS >= cnt) return;       // the whole block has nothing to do
        valid = slot < cnt;
        g = valid ? __ldg(list + slot) : 0;
    }
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

}  // namespace

bool assign_supported(int v, int k) { return v >= 1 && v <= 32 && k >= 1 && k <= 65536; }

cudaError_t launch_assign_listed(const __half *W, int M, int N, int v, const __half *C, int k, int *idx,
                                 const int *list, const int *count, long long n_vectors, cudaStream_t st)
{
    if (n_vectors == 0) return cudaSuccess;
    // (with a list the grid is sized for the worst case, every vector listed; blocks beyond the count return at once)
    const long long blocks = (n_vectors + ASSIGN_THREADS - 1) / ASSIGN_THREADS;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)blocks);
    if (v <= 4) assign_kernel<4><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors, list, count);
    else if (v <= 8) assign_kernel<8><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors, list, count);
    else if (v <= 16) assign_kernel<16><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors, list, count);
    else assign_kernel<32><<<grid, ASSIGN_THREADS, 0, st>>>(W, M, N, v, C, k, idx, n_vectors, list, count);
    return cudaGetLastError();
}

cudaError_t launch_assign(const __half *W, int M, int N, int v, const __half *C, int k, int *idx, cudaStream_t st)
{
    return launch_assign_listed(W, M, N, v, C, k, idx, nullptr, nullptr, (long long)ceil_div(M, v) * N, st);
}

}  // namespace vptq
