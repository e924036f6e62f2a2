// Assignment step of the quantizer (Eq. 2) on the tensor cores, with the result of the FP32 definition.
//
// The squared distance is ||c||^2 - 2 x.c + ||x||^2, and the first two terms are a contraction over the
// vector's components: D[vector][centroid] = A * B^T with
//   A row (a vector):   x_0 .. x_{v-1}, 0 .., 1, 2^-11            (16 FP16 values, K = 16)
//   B row (a centroid): -2c_0 .. -2c_{v-1}, 0 .., hi, 2^11 lo     hi + lo = ||c||^2 split into two FP16 values
// with x and c first multiplied by a power of two 2^s that brings max ||c||^2 to about 2^8: FP16 keeps its
// 11 bits only for normal numbers, and small weights (1e-4) and their squared norms are far below them.
// The scaling is exact for values that stay in range and leaves the order of the distances unchanged.
// One tcgen05.mma (M = 128 vectors, N = 128 centroids, K = 16) gives 16 K approximate distances.  They
// only FILTER: per vector the kernel keeps the smallest and the second smallest minimum over groups of
// 32 centroids and the group of the smallest.  Then the 32 centroids of that group are evaluated with
// the arithmetic that defines the result (FP32 fma chain, lowest index wins: the same code as the plain
// kernel), and a vector whose two group minima are closer than a bound on the filter's error is put on
// a list; a second kernel scans all centroids for the vectors on the list (one warp per vector).  The indices are therefore
// those of the FP32 definition, bit for bit, whatever the tensor core's summation order.
//   bound: |filter - (definition - ||x||^2)| <= 2^-18 (||x||^2 + max ||c||^2) (FP16 split of the norm,
//   FP32 accumulation of 10 products, rounding of the fma chain); the margin tested is 2^-15 of that sum,
//   four times what two such errors can add up to.
//
// Persistent grid, one CTA per SM, 256 vectors (two A tiles) per step.  Warp 0 streams the prepared
// centroid tiles (4 KB, shared-memory image with the 32-byte swizzle applied by the preparation kernel)
// with linear bulk copies into a ring; warp 1 issues the MMAs (two per centroid tile, fresh accumulators
// in one of two TMEM buffers); warps 2-9 write the A tiles of a step, then drain the accumulators: a lane
// owns one vector, reads 32 distances per tcgen05.ld and keeps its two running minima (about 40 instructions
// per 32 distances, nearly all of them min/compare/select on the ALU pipe: that pipe, not the tensor core,
// bounds the kernel; the three-input min.f32 was tried and changes nothing).
// Every mbarrier wait is bounded; a wait that gives up sets the status word of the workspace.
#include "common.cuh"
#include "assign.cuh"
#include "tcgen05_ptx.cuh"

namespace vptq {

namespace {

using namespace tc;

constexpr int KT = 128;                       // centroids per tile (N of the MMA)
constexpr int ROW_BYTES = 32;                 // K = 16 FP16 values
constexpr int TILE_BYTES = KT * ROW_BYTES;    // 4 KB: an A tile (128 vectors) or a B tile (128 centroids)
constexpr int B_STAGES = 8;
constexpr int EPI_WARPS = 8;
constexpr int SCAN_THREADS = 32 * (2 + EPI_WARPS);
constexpr int STEP_VECTORS = 256;             // two A tiles
constexpr int GROUP = 32;                     // centroids per candidate group (one tcgen05.ld)
constexpr float PAD_NORM = 60000.f;           // norm of the padding rows of the last centroid tile: never the minimum
constexpr float MARGIN = 1.0f / 32768.0f;     // 2^-15

struct ScanParams {
    const __half *W;
    int M, N, v, k;
    const __half *C;          // [k][v]
    const uint8_t *Bimg;      // [k_tiles][TILE_BYTES]
    const float *cmax;        // max ||c||^2
    int *idx;                 // [n_vectors]
    int *list;                // vectors that need the full scan
    int *count;               // entries of the list
    int *status;
    long long n_vectors;
    int k_tiles;
};

// K-major operand with 32-byte rows and the 32-byte swizzle: 8-row groups of 256 bytes
__device__ __forceinline__ uint64_t operand_desc(uint32_t saddr) { return make_smem_desc(saddr, 16, 8 * ROW_BYTES, LAYOUT_SW32); }
// kind::f16: FP16 x FP16 -> FP32, both operands K-major, M = 128, N = 128
constexpr uint32_t SCAN_IDESC = (1u << 4) | ((uint32_t)(KT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
__device__ __forceinline__ void umma_fresh(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(SCAN_IDESC) : "memory");
}
// 32 consecutive accumulator columns of this lane's row: the load is only issued here ...
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
// ... and its registers may be read after this wait (they are operands of the wait so that no use moves above it)
__device__ __forceinline__ void tmem_ld32_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :: "memory");
}
// smallest of 32 values
__device__ __forceinline__ float min32(const uint32_t (&d)[32])
{
    float m[16];
#pragma unroll
    for (int j = 0; j < 16; j++) m[j] = fminf(__uint_as_float(d[j]), __uint_as_float(d[j + 16]));
#pragma unroll
    for (int w = 8; w > 0; w >>= 1)
#pragma unroll
        for (int j = 0; j < w; j++) m[j] = fminf(m[j], m[j + w]);
    return m[0];
}

// byte offset of 16-byte chunk c (0 or 1) of row r in a tile image (32-byte swizzle: bit 4 ^= bit 7)
__device__ __forceinline__ int image_offset(int r, int c) { return r * ROW_BYTES + ((c ^ ((r >> 2) & 1)) << 4); }

// The power of two that brings max ||c||^2 to [2^8, 2^10): 2^s multiplies vectors and centroids.
__device__ __forceinline__ int scale_exponent(float cmax)
{
    if (!(cmax > 0.f) || !(cmax < 3.0e38f)) return 0;
    int s = (8 - ilogbf(cmax) + 1) / 2;                 // ilogbf: floor(log2)
    return s < -12 ? -12 : (s > 24 ? 24 : s);
}

// ---- preparation, first pass: max ||c||^2; clears the list count and the status word -------------------------
__global__ void __launch_bounds__(256)
assign_norms_kernel(const __half *__restrict__ C, int k, int v, float *cmax, int *count, int *status)
{
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i == 0) { *count = 0; *status = 0; }
    if (i >= k) return;
    float norm = 0.f;
    for (int j = 0; j < v; j++) {
        const float c = __half2float(__ldg(C + (long long)i * v + j));
        norm = __fmaf_rn(c, c, norm);
    }
    // norm >= 0: integer order = float order; a NaN norm has the largest bit pattern and so becomes the maximum
    atomicMax(reinterpret_cast<int *>(cmax), __float_as_int(norm));
}

// ---- preparation, second pass: the scaled centroid tiles as shared-memory images -----------------------------
__global__ void __launch_bounds__(256)
assign_prepare_kernel(const __half *__restrict__ C, int k, int v, uint8_t *__restrict__ Bimg, const float *cmax, int k_tiles)
{
    const int i = blockIdx.x * 256 + threadIdx.x;          // centroid (or padding row of the last tile)
    if (i >= k_tiles * KT) return;
    const float scale = exp2f((float)scale_exponent(*cmax));
    __half row[16];
#pragma unroll
    for (int j = 0; j < 16; j++) row[j] = __float2half_rn(0.f);
    float norm = PAD_NORM;
    if (i < k) {
        norm = 0.f;
        for (int j = 0; j < v; j++) {
            const float c = __half2float(__ldg(C + (long long)i * v + j)) * scale;
            norm = __fmaf_rn(c, c, norm);
            row[j] = __float2half_rn(-2.f * c);             // exact while in range
        }
    }
    const __half hi = __float2half_rn(norm);
    row[14] = hi;
    row[15] = __float2half_rn((norm - __half2float(hi)) * 2048.f);     // the A row multiplies it by 2^-11
    uint8_t *tile = Bimg + (long long)(i / KT) * TILE_BYTES;
    const uint4 *src = reinterpret_cast<const uint4 *>(row);
    *reinterpret_cast<uint4 *>(tile + image_offset(i % KT, 0)) = src[0];
    *reinterpret_cast<uint4 *>(tile + image_offset(i % KT, 1)) = src[1];
}

// ---- the scan ---------------------------------------------------------------------------------------------
template <int VMAX>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
assign_scan_kernel(ScanParams P)
{
    __shared__ __align__(1024) uint8_t sA[2 * TILE_BYTES];
    __shared__ __align__(1024) uint8_t sB[B_STAGES * TILE_BYTES];
    __shared__ __align__(8) uint64_t bars[2 * B_STAGES + 5];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;

    const uint32_t bar0 = smem_addr(bars);
    auto bar_fullB = [&](int s) { return bar0 + 8u * s; };
    auto bar_emptyB = [&](int s) { return bar0 + 8u * (B_STAGES + s); };
    auto bar_accFull = [&](int b) { return bar0 + 8u * (2 * B_STAGES + b); };
    auto bar_accEmpty = [&](int b) { return bar0 + 8u * (2 * B_STAGES + 2 + b); };
    const uint32_t bar_aFull = bar0 + 8u * (2 * B_STAGES + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < B_STAGES; s++) { mbar_init(bar_fullB(s), 1); mbar_init(bar_emptyB(s), 1); }
        for (int b = 0; b < 2; b++) { mbar_init(bar_accFull(b), 1); mbar_init(bar_accEmpty(b), EPI_WARPS); }
        mbar_init(bar_aFull, EPI_WARPS);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    const long long n_steps = (P.n_vectors + STEP_VECTORS - 1) / STEP_VECTORS;
    bool ok = true;

    if (warp == 0) {
        // ================= centroid tiles: linear bulk copies into the ring =================
        if (lane == 0) {
            long long it = 0;
            for (long long step = blockIdx.x; step < n_steps && ok; step += gridDim.x)
                for (int kt = 0; kt < P.k_tiles; kt++, it++) {
                    const int s = (int)(it % B_STAGES);
                    if (!(ok = mbar_wait(bar_emptyB(s), (uint32_t)((it / B_STAGES) & 1) ^ 1u, abort_flag, P.status))) break;
                    mbar_expect_tx(bar_fullB(s), TILE_BYTES);
                    bulk_load(smem_addr(sB) + s * TILE_BYTES, P.Bimg + (long long)kt * TILE_BYTES, TILE_BYTES, bar_fullB(s));
                }
            if (!ok) {
                // abandoned: give copies still in flight a bounded time to land before the CTA exits
                const long long first = it > B_STAGES ? it - B_STAGES : 0;
                for (long long j = first; j < it; j++) {
                    const long long t0c = clock64();
                    while (!mbar_try(bar_fullB((int)(j % B_STAGES)), (uint32_t)((j / B_STAGES) & 1)) &&
                           clock64() - t0c < 20000000ll) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issue =================
        if (lane == 0) {
            const uint64_t adesc0 = operand_desc(smem_addr(sA));
            const uint64_t bdesc0 = operand_desc(smem_addr(sB));
            long long it = 0, step_no = 0;
            for (long long step = blockIdx.x; step < n_steps && ok; step += gridDim.x, step_no++) {
                if (!(ok = mbar_wait(bar_aFull, (uint32_t)(step_no & 1), abort_flag, P.status))) break;
                for (int kt = 0; kt < P.k_tiles; kt++, it++) {
                    const int s = (int)(it % B_STAGES), b = (int)(it & 1);
                    if (!(ok = mbar_wait(bar_fullB(s), (uint32_t)((it / B_STAGES) & 1), abort_flag, P.status))) break;
                    if (!(ok = mbar_wait(bar_accEmpty(b), (uint32_t)((it >> 1) & 1) ^ 1u, abort_flag, P.status))) break;
                    tc_fence_after();
                    const uint64_t bd = bdesc0 + (uint64_t)((s * TILE_BYTES) >> 4);
                    umma_fresh(tmem_base + (uint32_t)((b * 2 + 0) * KT), adesc0, bd);
                    umma_fresh(tmem_base + (uint32_t)((b * 2 + 1) * KT), adesc0 + (uint64_t)(TILE_BYTES >> 4), bd);
                    umma_commit(bar_emptyB(s));
                    umma_commit(bar_accFull(b));
                }
            }
        }
    } else {
        // ================= A tiles, then the running minima; a lane owns one vector of the step =================
        const int ew = warp - 2;
        const int q = warp & 3;                      // TMEM lane quarter this warp may read
        const int a = ew >> 2;                       // A tile
        const int row = 32 * q + lane;               // row of the A tile = TMEM lane
        const float scale = exp2f((float)scale_exponent(__ldg(P.cmax)));
        const float cmax = __ldg(P.cmax) * scale * scale;      // in the filter's units
        long long it = 0;
        for (long long step = blockIdx.x; step < n_steps && ok; step += gridDim.x) {
            const long long g = step * STEP_VECTORS + a * 128 + row;
            const bool valid = g < P.n_vectors;
            const int r = valid ? (int)(g / P.N) : 0, n = valid ? (int)(g % P.N) : 0;
            float x[VMAX];
            float xn = 0.f;
#pragma unroll
            for (int j = 0; j < VMAX; j++) {
                x[j] = (valid && j < P.v) ? __half2float(__ldg(P.W + (long long)(r * P.v + j) * P.N + n)) : 0.f;
                xn = __fmaf_rn(x[j] * scale, x[j] * scale, xn);
            }
            // the A tile of this step may be overwritten: its MMAs completed before the last accFull of the previous step
            {
                __half rowv[16];
#pragma unroll
                for (int j = 0; j < 14; j++) rowv[j] = __float2half_rn(j < VMAX ? x[j < VMAX ? j : 0] * scale : 0.f);   // exact while in range
                rowv[14] = __float2half_rn(1.f);         // times hi
                rowv[15] = __float2half_rn(1.f / 2048.f);    // times 2^11 lo
                const uint4 *src = reinterpret_cast<const uint4 *>(rowv);
                uint8_t *tile = sA + a * TILE_BYTES;
                *reinterpret_cast<uint4 *>(tile + image_offset(row, 0)) = src[0];
                *reinterpret_cast<uint4 *>(tile + image_offset(row, 1)) = src[1];
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_aFull);
            }
            float b1 = __int_as_float(0x7f800000), b2 = b1;
            int g1 = 0;
            for (int kt = 0; kt < P.k_tiles; kt++, it++) {
                const int b = (int)(it & 1);
                ok = __all_sync(0xffffffffu, mbar_wait(bar_accFull(b), (uint32_t)((it >> 1) & 1), abort_flag, P.status));
                if (!ok) break;
                tc_fence_after();
                // the load of the next group of 32 distances is in flight while this one is reduced
                const uint32_t t_row = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)((b * 2 + a) * KT);
                uint32_t d0[32], d1[32];
                tmem_ld32_issue(t_row, d0);
#pragma unroll
                for (int grp = 0; grp < KT / GROUP; grp += 2) {
                    tmem_ld32_wait(d0);
                    tmem_ld32_issue(t_row + (uint32_t)((grp + 1) * GROUP), d1);
                    float gm = min32(d0);
                    if (gm < b1) { b2 = b1; b1 = gm; g1 = kt * (KT / GROUP) + grp; }
                    else if (gm < b2) b2 = gm;
                    tmem_ld32_wait(d1);
                    if (grp + 2 < KT / GROUP) tmem_ld32_issue(t_row + (uint32_t)((grp + 2) * GROUP), d0);
                    gm = min32(d1);
                    if (gm < b1) { b2 = b1; b1 = gm; g1 = kt * (KT / GROUP) + grp + 1; }
                    else if (gm < b2) b2 = gm;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_accEmpty(b));
            }
            if (!ok) break;
            if (valid) {
                // the group of the smallest filter value, with the arithmetic that defines the result
                int best = 0;
                float best_d = __int_as_float(0x7f800000);
                const int i0 = g1 * GROUP, i1 = min(P.k, i0 + GROUP);
                for (int i = i0; i < i1; i++) {
                    float dd = 0.f;
#pragma unroll
                    for (int j = 0; j < VMAX; j++) {
                        const float c = j < P.v ? __half2float(__ldg(P.C + (long long)i * P.v + j)) : 0.f;
                        const float t = __fsub_rn(x[j], c);
                        dd = __fmaf_rn(t, t, dd);
                    }
                    if (dd < best_d) { best_d = dd; best = i; }
                }
                P.idx[g] = best;
                // not clearly the only candidate group: the full scan decides
                const float eps = MARGIN * (xn + cmax);
                // (a vector or a table that leaves the FP16 range even after scaling makes the filter meaningless:
                //  such vectors, or then all of them, are listed)
                if (!(b2 - b1 > eps) || !(fabsf(b1) < 3.0e38f) || !(xn < 3.0e9f) || !(cmax < PAD_NORM))
                    P.list[atomicAdd(P.count, 1)] = (int)g;
            }
        }
    }

    tc_fence_before();
    __syncwarp();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

struct ScanLayout {
    long long off_cmax, off_count, off_bimg, off_list, bytes;
    int k_tiles;
};

ScanLayout scan_layout(long long n_vectors, int k)
{
    ScanLayout l;
    l.k_tiles = ceil_div(k, KT);
    l.off_cmax = 16;                    // status word at byte 0
    l.off_count = 32;
    l.off_bimg = 256;
    l.off_list = l.off_bimg + (long long)l.k_tiles * TILE_BYTES;
    l.bytes = l.off_list + (n_vectors * 4 + 255) / 256 * 256;
    return l;
}

}  // namespace

// vectors of at most 14 components (two of the 16 K columns carry the norm), whole vector rows, enough
// centroids for the filter to pay, vector numbers that fit an int
bool assign_tcgen05_supported(int M, int N, int v, int k)
{
    if (v < 1 || v > 14 || k < 1024 || k > 65536 || M % v != 0) return false;
    return (long long)(M / v) * N < 0x7fffffffLL && (long long)(M / v) * N >= 4096;
}

long long assign_tcgen05_workspace_bytes(int M, int N, int v, int k)
{
    return scan_layout((long long)ceil_div(M, v) * N, k).bytes;
}

cudaError_t launch_assign_tcgen05(const __half *W, int M, int N, int v, const __half *C, int k, int *idx, void *ws,
                                  cudaStream_t st)
{
    const long long n_vectors = (long long)(M / v) * N;
    const ScanLayout l = scan_layout(n_vectors, k);
    uint8_t *w8 = reinterpret_cast<uint8_t *>(ws);
    ScanParams P;
    P.W = W; P.M = M; P.N = N; P.v = v; P.k = k; P.C = C;
    P.Bimg = w8 + l.off_bimg;
    P.cmax = reinterpret_cast<const float *>(w8 + l.off_cmax);
    P.idx = idx;
    P.list = reinterpret_cast<int *>(w8 + l.off_list);
    P.count = reinterpret_cast<int *>(w8 + l.off_count);
    P.status = reinterpret_cast<int *>(w8);
    P.n_vectors = n_vectors;
    P.k_tiles = l.k_tiles;
    cudaError_t e = cudaMemsetAsync(w8 + l.off_cmax, 0, 4, st);
    if (e != cudaSuccess) return e;
    assign_norms_kernel<<<ceil_div(k, 256), 256, 0, st>>>(C, k, v, reinterpret_cast<float *>(w8 + l.off_cmax),
                                                          P.count, P.status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    assign_prepare_kernel<<<ceil_div(l.k_tiles * KT, 256), 256, 0, st>>>(C, k, v, w8 + l.off_bimg, P.cmax, l.k_tiles);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long n_steps = (n_vectors + STEP_VECTORS - 1) / STEP_VECTORS;
    const int grid = (int)(n_steps < device_sm_count() ? n_steps : device_sm_count());
    if (v <= 8) assign_scan_kernel<8><<<grid, SCAN_THREADS, 0, st>>>(P);
    else assign_scan_kernel<14><<<grid, SCAN_THREADS, 0, st>>>(P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // the vectors whose candidate group was not clearly the only one: all centroids, FP32
    return launch_assign_listed(W, M, N, v, C, k, idx, P.list, P.count, device_sm_count(), st);
}

}  // namespace vptq
