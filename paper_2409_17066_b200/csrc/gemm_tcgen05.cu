// Batched / prefill path: out[B][M] = x[B][N] * W_hat^T as a tensor-core GEMM whose weight
// operand is dequantised on the fly into shared memory (the FP16 weight matrix never exists in
// global memory; App. D.2 describes the paper's two-phase scheme that this replaces).
//
//   D[m][t] (TMEM, FP32, 128 lanes x 512 columns) += A[m][k] * B[t][k]
//   A = W tile, 128 output rows x 32 input columns, written by producer warps: one 16-byte
//       centroid (8 consecutive output rows of one input column) = C1[i1] + C2[i2] per store,
//       in the MN-major 128-byte-swizzled layout tcgen05.mma reads;
//   B = x*s tile (FP16, scale folded into the activations by a pre-pass), 512 tokens x 32
//       columns, K-major with the 64-byte swizzle.  The pre-pass writes the activations as the
//       shared-memory image of these tiles ([256-token half][k block] -> 16 KB, swizzle applied),
//       so a tile half arrives by one linear bulk copy of whole 128-byte lines (a tiled TMA load of
//       64-byte rows asks L2 for twice as many pieces);
//   tcgen05.mma.cta_group::1.kind::f16, M = 128, N = 256 (two per token tile), K = 16.
//
// Warp roles (640 threads): warp 0 bulk loads of B; warp 1 TMEM allocation + MMA issue (one
// thread); warps 2-11 dequant producers (a pair per k block: a1 unpack with the next visit's
// indices already in flight, a3 main lookup from the L2-resident codebook, a4 residual lookup
// from shared memory, add, store); warps 12-19 epilogue (tcgen05.ld -> + bias term -> shared
// memory -> TMA store or reduce-add), two per TMEM lane quarter.  Twenty warps are five per
// scheduler: the register budget per thread is the same from 17 to 20 warps.
// A and B have rings of their own: A has a stage per producer pair and one to spare (the
// producers' gathers need a few microseconds), B holds 32 KB per stage and is shallow.
// What bounds the k loop is the SM's request path to L2 (about one request per clock): per k block
// 512 centroid reads and 256 lines of activations.  Two ways of sharing the activation tiles in a
// CTA pair were measured and dropped: tcgen05 cta_group::2 (each CTA loads half of the tokens; the
// pair advances at the pace of its slower half: 103 us against 88 us on the 14336 x 4096 layer at
// 512 tokens) and forwarding the own half into the partner's shared memory (the forwarded bytes
// load the same outgoing path: 117 us).
// Persistent grid, one CTA per SM.  The work is the list of (tile, k block) units, tile =
// (token tile, 128-row tile); with an FP32 output every CTA takes an equal, contiguous share of
// the units, whatever tile they fall in, so all SMs stay busy; other output types are dealt out in
// whole tiles.  When a share is long (FLAG_ORDER_MIN_SHARE k blocks or more) the pieces of a split
// tile meet in the output without a zero-fill: the piece that holds the tile's last k blocks is the
// first thing its CTA works on, so it finishes early; it stores and then raises the tile's flag in
// the workspace; the other pieces (the last thing their CTAs work on) wait for the flag (a bounded
// wait that is normally over before it starts) and reduce-add.  With short shares all pieces end
// together, so there the pre-pass clears the output and every piece reduce-adds.
//
// Every mbarrier wait is bounded: after about two seconds a waiter records VPTQ_E_TIMEOUT in
// the status word of the workspace, raises a CTA-wide abort flag and every role leaves its
// loop; TMEM is freed on all paths.
#include <cuda.h>

#include "common.cuh"
#include "gemm.cuh"
#include "tcgen05_ptx.cuh"

namespace vptq {

namespace {

using namespace tc;

constexpr int TILE_M = 128;
constexpr int TILE_K = 32;
constexpr int TILE_N = 512;
constexpr int MMA_N = 256;
constexpr int A_STAGES = 6;                              // ring of dequantised weight tiles
constexpr int A_STAGE_BYTES = TILE_M * TILE_K * 2;       // 8 KB
constexpr int B_STAGES = 3;                              // ring of activation tiles
constexpr int B_HALF_BYTES = MMA_N * TILE_K * 2;         // 256 tokens x 32 columns: 16 KB, one bulk copy
constexpr int B_STAGE_BYTES = 2 * B_HALF_BYTES;          // 32 KB
constexpr int PAIRS = 5;                                 // producer warp pairs; pair p fills k blocks p, p+PAIRS, ...
constexpr int PRODUCER_WARPS = 2 * PAIRS;
constexpr int EPI_WARPS = 8;
constexpr int EPI_BUF_BYTES = 16 * 32 * 4;                // one staged piece of the output: 16 tokens x 32 rows, FP32
constexpr int EPI_STAGE_BYTES = EPI_WARPS * 2 * EPI_BUF_BYTES;   // two buffers per epilogue warp: 32 KB
constexpr int CB2_REPLICAS = 4;                          // copies of a small residual table (16-byte skew)
static_assert(A_STAGES >= PAIRS, "a producer pair needs a stage of its own");
constexpr int GEMM_THREADS = 32 * (2 + PRODUCER_WARPS + EPI_WARPS);   // 640
constexpr int A_SBO = 2048;   // bytes between consecutive 8-column groups of the A stage
constexpr int A_LBO = 1024;   // bytes between the two 64-row blocks of the A stage
constexpr int B_SBO = 512;    // bytes between consecutive 8-token groups of the B stage (8 x 64 B)

constexpr int WS_STATUS_BYTES = 256;
constexpr int FLAG_ORDER_MIN_SHARE = 24;

struct GemmParams {
    LayerView L;
    void *out;
    int B;
    int tiles_m, tiles_t, kb_total;
    int unit_gran;       // a CTA's share of the units is a multiple of this (1, or kb_total = whole tiles)
    long long units;     // tiles_m * tiles_t * kb_total
    int cb2_replicated;
    int cb2_bytes;
    int flag_order;      // split tiles: 1 = last piece stores and raises a flag, the others wait and add; 0 = all add
    int tma_out;         // FP32 output written by TMA store / reduce from shared memory (needs M % 4 == 0)
    int *status;         // workspace status word
    const float *bterm;  // [B]
    int *tile_flags;     // [tiles]: epilogue warps that have stored the piece with the tile's last k blocks
    const uint8_t *xs;   // activation tile images, [ceil(B / 256)][kb_total][16 KB]
};

// ---- PTX wrappers ----------------------------------------------------------------------------
// Bounded wait until *flag >= target (set by another CTA of this grid; all CTAs of the grid are resident).
__device__ __forceinline__ bool flag_wait(const int *flag, int target, volatile int *abort_flag, int *status)
{
    const long long t0 = clock64();
    unsigned spins = 0;
    while (true) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v >= target) return true;
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            if ((unsigned long long)(clock64() - t0) > WAIT_LIMIT_CYCLES) {
                *abort_flag = 1;
                grid_dependency_wait();                  // the pre-pass clears the status word
                atomicExch(status, VPTQ_E_TIMEOUT);
                return false;
            }
        }
        __nanosleep(64);
    }
}

// kind::f16, FP16 x FP16 -> FP32, A MN-major, B K-major, M = 128, N = 256
constexpr uint32_t IDESC = (1u << 4) | (0u << 7) | (0u << 10) | (1u << 15) | (0u << 16) |
                           ((uint32_t)(MMA_N >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(IDESC), "r"(accumulate) : "memory");
}
// The MMAs of one 32-column k block: two k16 steps x one or two 256-token halves, issued back to back.
// `ad`/`bd` describe the k16 = 0 slice of the stage; the second slice lies 2 * A_SBO (A) and 32 bytes (B)
// further, the second token half B_HALF_BYTES further (descriptor address units are 16 bytes).
__device__ __forceinline__ void umma_kblock(uint32_t d_tmem, uint64_t ad, uint64_t bd, uint32_t accumulate, bool two_halves)
{
    const uint64_t ad1 = ad + (uint64_t)((2 * A_SBO) >> 4);
    const uint64_t bd1 = bd + 2u;
    const uint64_t bh = (uint64_t)(B_HALF_BYTES >> 4);
    umma_f16(d_tmem, ad, bd, accumulate);
    if (two_halves) umma_f16(d_tmem + MMA_N, ad, bd + bh, accumulate);
    umma_f16(d_tmem, ad1, bd1, 1u);
    if (two_halves) umma_f16(d_tmem + MMA_N, ad1, bd1 + bh, 1u);
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// TMA store / reduce-add of a [16 tokens][32 rows] FP32 box from shared memory into the output
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y, bool add)
{
    if (add)
        asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.bulk_group [%0, {%2, %3}], [%1];"
                     ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                     ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// ---- pre-pass: xs = fp16(x * s) written as tile images, bterm[t] = sum_n x[t][n] * b[n], status = 0, tile
//      flags = 0; clears row t of an FP32 output in which all pieces of split tiles reduce-add (zero_out != nullptr).
// Image of the tile half (256 tokens) x (k block of 32 columns): token r, 16-byte chunk q (8 columns) at
//      (r / 8) * 512 + (r % 8) * 64 + ((q ^ ((r % 8) / 2)) * 16: the K-major 64-byte-swizzled operand layout.
// One block per token of the padded range; tokens >= B and columns >= N are written as zeros. ---------------
constexpr int PRE_THREADS = 128;

__global__ void __launch_bounds__(PRE_THREADS)
gemm_prepass_kernel(LayerView L, const void *__restrict__ x, int B, uint8_t *__restrict__ xs,
                    float *__restrict__ bterm, int *status, int *__restrict__ tile_flags, int n_tiles,
                    float *__restrict__ zero_out)
{
    // the GEMM is launched as a programmatic dependent: its CTAs may become resident and run their set-up and
    // first centroid reads as soon as every block of this grid has started; whatever reads this kernel's
    // output waits for the whole grid (griddepcontrol.wait) first
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int t = blockIdx.x;
    for (int i = t * PRE_THREADS + threadIdx.x; i < n_tiles; i += gridDim.x * PRE_THREADS) tile_flags[i] = 0;
    const int kb_total = (L.N + TILE_K - 1) / TILE_K;
    // where token t's 64 bytes of k block 0 start; the other k blocks follow at B_HALF_BYTES each
    uint8_t *img_row = xs + (long long)(t / MMA_N) * kb_total * B_HALF_BYTES + ((t % MMA_N) >> 3) * B_SBO + (t & 7) * 64;
    const int sw = (t & 7) >> 1;
    if (t >= B) {
        for (int q = threadIdx.x; q < 4 * kb_total; q += PRE_THREADS)
            *reinterpret_cast<uint4 *>(img_row + (long long)(q >> 2) * B_HALF_BYTES + (((q & 3) ^ sw) << 4)) = make_uint4(0, 0, 0, 0);
        return;
    }
    if (t == 0 && threadIdx.x == 0) *status = 0;
    if (zero_out != nullptr) {
        float *row = zero_out + (long long)t * L.M;
        if ((L.M & 3) == 0) {
            float4 *r4 = reinterpret_cast<float4 *>(row);          // rows of M floats start 16-byte aligned
            for (int i = threadIdx.x; i < (L.M >> 2); i += PRE_THREADS) r4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
            for (int i = threadIdx.x; i < L.M; i += PRE_THREADS) row[i] = 0.f;
        }
    }
    float acc = 0.f;
    if ((L.N & 7) == 0 && L.perm == nullptr) {
        // 8 columns = one chunk per thread and step, 128-bit loads and stores; the loads of four steps are
        // issued together (a thread with one load in flight at a time leaves the memory system idle)
        constexpr int UNROLL = 4;
        const uint4 one = make_uint4(0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u), zero = make_uint4(0, 0, 0, 0);
        for (int n0 = 8 * threadIdx.x; n0 < kb_total * TILE_K; n0 += UNROLL * 8 * PRE_THREADS) {
            uint4 xq[UNROLL], sq[UNROLL], bq[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; u++) {
                const int n = n0 + u * 8 * PRE_THREADS;
                xq[u] = zero; sq[u] = one; bq[u] = zero;
                if (n < L.N) {
                    xq[u] = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(x) + (long long)t * L.N + n));
                    if (L.has_scale) {
                        sq[u] = __ldg(reinterpret_cast<const uint4 *>(L.scale + n));
                        bq[u] = __ldg(reinterpret_cast<const uint4 *>(L.bias + n));
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; u++) {
                const int n = n0 + u * 8 * PRE_THREADS;
                if (n >= kb_total * TILE_K) break;
                const uint32_t xw[4] = {xq[u].x, xq[u].y, xq[u].z, xq[u].w}, sc[4] = {sq[u].x, sq[u].y, sq[u].z, sq[u].w},
                               bw[4] = {bq[u].x, bq[u].y, bq[u].z, bq[u].w};
                uint32_t ow[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {       // columns >= N were loaded as zeros: they store zeros and add nothing
                    float2 xv;
                    if (L.x_bf16) xv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&xw[i]));
                    else xv = __half22float2(*reinterpret_cast<const __half2 *>(&xw[i]));
                    const float2 sv = __half22float2(*reinterpret_cast<const __half2 *>(&sc[i]));
                    const float2 bv = __half22float2(*reinterpret_cast<const __half2 *>(&bw[i]));
                    const __half2 o = __floats2half2_rn(xv.x * sv.x, xv.y * sv.y);
                    ow[i] = *reinterpret_cast<const uint32_t *>(&o);
                    acc += xv.x * bv.x + xv.y * bv.y;
                }
                const int q = n >> 3;
                *reinterpret_cast<uint4 *>(img_row + (long long)(q >> 2) * B_HALF_BYTES + (((q & 3) ^ sw) << 4)) =
                    make_uint4(ow[0], ow[1], ow[2], ow[3]);
            }
        }
    } else {
        for (int n = threadIdx.x; n < kb_total * TILE_K; n += PRE_THREADS) {
            float xv = 0.f, sc = 1.f, bi = 0.f;
            if (n < L.N) {
                xv = load_act(x, (long long)t * L.N + in_col(L, n), L.x_bf16);
                if (L.has_scale) {
                    sc = __half2float(__ldg(L.scale + n));
                    bi = __half2float(__ldg(L.bias + n));
                }
            }
            const int q = n >> 3;
            *reinterpret_cast<__half *>(img_row + (long long)(q >> 2) * B_HALF_BYTES + (((q & 3) ^ sw) << 4) + (n & 7) * 2) =
                __float2half_rn(xv * sc);
            acc += xv * bi;
        }
    }
    __shared__ float red[PRE_THREADS / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = 0.f;
        for (int w = 0; w < PRE_THREADS / 32; w++) a += red[w];
        bterm[t] = a;
    }
}

// ---- the GEMM ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_out, GemmParams P)
{
    extern __shared__ uint8_t smem_raw[];
    const LayerView &L = P.L;
    // carve shared memory; swizzled operand stages need 1024-byte alignment
    const uint32_t raw = smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const uint32_t sA = base;                                   // A_STAGES x 8 KB
    const uint32_t sB = sA + A_STAGES * A_STAGE_BYTES;          // B_STAGES x 32 KB
    uint8_t *cb2_ptr = sm + A_STAGES * A_STAGE_BYTES + B_STAGES * B_STAGE_BYTES;
    const uint32_t sEpi = smem_addr(cb2_ptr + P.cb2_bytes);     // EPI_WARPS x 2 x 2 KB output staging
    uint8_t *misc = cb2_ptr + P.cb2_bytes + EPI_STAGE_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(misc);   // fullA[] emptyA[] fullB[] emptyB[] accum_full accum_empty
    const uint32_t bar0 = smem_addr(bars);
    auto bar_fullA = [&](int s) { return bar0 + 8u * s; };
    auto bar_emptyA = [&](int s) { return bar0 + 8u * (A_STAGES + s); };
    auto bar_fullB = [&](int s) { return bar0 + 8u * (2 * A_STAGES + s); };
    auto bar_emptyB = [&](int s) { return bar0 + 8u * (2 * A_STAGES + B_STAGES + s); };
    constexpr int N_RING_BARS = 2 * A_STAGES + 2 * B_STAGES;
    const uint32_t bar_accum_full = bar0 + 8u * N_RING_BARS;
    const uint32_t bar_accum_empty = bar0 + 8u * (N_RING_BARS + 1);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(misc + 8 * (N_RING_BARS + 2));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < A_STAGES; s++) {
            mbar_init(bar_fullA(s), 2);       // one arrival per producer warp of a pair
            mbar_init(bar_emptyA(s), 1);      // tcgen05.commit
        }
        for (int s = 0; s < B_STAGES; s++) {
            mbar_init(bar_fullB(s), 1);       // the expect_tx arrival
            mbar_init(bar_emptyB(s), 1);      // tcgen05.commit
        }
        mbar_init(bar_accum_full, 1);
        mbar_init(bar_accum_empty, EPI_WARPS);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // residual codebook -> shared memory (all threads)
    if (L.k2) {
        const uint4 *src = reinterpret_cast<const uint4 *>(L.c2);
        uint4 *dst = reinterpret_cast<uint4 *>(cb2_ptr);
        // (loads of 4 entries are issued before the first store: one L2 round trip per 4 entries)
        const int n2 = P.cb2_replicated ? L.k2 * CB2_REPLICAS : L.k2, sh = P.cb2_replicated ? 2 : 0;
        for (int i0 = threadIdx.x; i0 < n2; i0 += 4 * GEMM_THREADS) {
            uint4 row[4];
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (i0 + u * GEMM_THREADS < n2) row[u] = __ldg(src + ((i0 + u * GEMM_THREADS) >> sh));
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (i0 + u * GEMM_THREADS < n2) dst[i0 + u * GEMM_THREADS] = row[u];
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // this CTA's share of the (tile, k block) units: [u_begin, u_end), boundaries multiples of unit_gran
    const long long n_workers = gridDim.x, worker = blockIdx.x;
    const long long groups = P.units / P.unit_gran;
    const long long u_begin = groups * worker / n_workers * P.unit_gran;
    const long long u_end = groups * (worker + 1) / n_workers * P.unit_gran;
    // A segment is the part of one tile inside the share: k blocks [kb0, kb1) of tile `tile`.
#define FOR_EACH_SEGMENT                                                                          \
    for (long long u = u_begin; u < u_end && ok; u += kb1 - kb0)                                    \
        if (tile = (int)(u / P.kb_total), kb0 = (int)(u % P.kb_total),                              \
            kb1 = (int)min((long long)P.kb_total, kb0 + (u_end - u)), true)
    int tile = 0, kb0 = 0, kb1 = 0;
    bool ok = true;

    if (warp == 0) {
        // ================= bulk copies: B tiles =================
        if (lane == 0) {
            grid_dependency_wait();                              // the tile images are the pre-pass's output
            int it = 0;
            uint32_t s = 0, ps = 1;                              // ring position, parity to wait for
            FOR_EACH_SEGMENT {
                const int tt = tile / P.tiles_m;
                const int t0 = tt * TILE_N;
                const int halves = (P.B - t0 > MMA_N) ? 2 : 1;
                for (int kb = kb0; kb < kb1; kb++, it++, s = (s + 1 == B_STAGES ? 0 : s + 1), ps ^= (s == 0 ? 1u : 0u)) {
                    if (!(ok = mbar_wait(bar_emptyB(s), ps, abort_flag, P.status))) break;
                    mbar_expect_tx(bar_fullB(s), halves * B_HALF_BYTES);
                    for (int h = 0; h < halves; h++)
                        bulk_load(sB + s * B_STAGE_BYTES + h * B_HALF_BYTES,
                                  P.xs + ((long long)(2 * tt + h) * P.kb_total + kb) * B_HALF_BYTES, B_HALF_BYTES, bar_fullB(s));
                }
            }
            if (!ok) {
                // abandoned: give copies still in flight a bounded time to land before the CTA exits
                const int first = it > B_STAGES ? it - B_STAGES : 0;
                for (int j = first; j < it; j++) {
                    const long long t0c = clock64();
                    while (!mbar_try(bar_fullB(j % B_STAGES), (j / B_STAGES) & 1) && clock64() - t0c < 20000000ll) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issue =================
        if (lane == 0) {
            // One thread runs this loop as a serial instruction chain, so it is kept short: descriptors
            // are a constant plus a stage offset, stage numbers and parities are running counters, and the
            // MMAs of a k block go out in one asm block.
            const uint64_t adesc0 = make_smem_desc(sA, A_LBO, A_SBO, LAYOUT_SW128);
            const uint64_t bdesc0 = make_smem_desc(sB, 16, B_SBO, LAYOUT_SW64);
            uint32_t sa = 0, pa = 0, sb = 0, pb = 0;          // ring positions and their phase parities
            int seg_no = 0;
            FOR_EACH_SEGMENT {
                const int tt = tile / P.tiles_m;
                const bool two_halves = P.B - tt * TILE_N > MMA_N;
                // the accumulators must have been drained by the epilogues of the previous segment
                if (!(ok = mbar_wait(bar_accum_empty, (seg_no & 1) ^ 1, abort_flag, P.status))) break;
                tc_fence_after();
                for (int kb = kb0; kb < kb1; kb++) {
                    if (!(ok = mbar_wait(bar_fullA(sa), pa, abort_flag, P.status))) break;
                    if (!(ok = mbar_wait(bar_fullB(sb), pb, abort_flag, P.status))) break;
                    // (stage offsets only touch the 14-bit address field of the descriptors: no carry)
                    const uint64_t ad = adesc0 + (uint64_t)((sa * A_STAGE_BYTES) >> 4);
                    const uint64_t bd = bdesc0 + (uint64_t)((sb * B_STAGE_BYTES) >> 4);
                    umma_kblock(tmem_base, ad, bd, kb > kb0 ? 1u : 0u, two_halves);
                    umma_commit(bar_emptyA(sa));      // the stages may be refilled once these MMAs have read them
                    umma_commit(bar_emptyB(sb));
                    if (++sa == A_STAGES) { sa = 0; pa ^= 1u; }
                    if (++sb == B_STAGES) { sb = 0; pb ^= 1u; }
                }
                if (ok) umma_commit(bar_accum_full);  // accumulators complete
                seg_no++;
            }
        }
    } else if (warp < 2 + PRODUCER_WARPS) {
        // ================= dequant producers: A tiles =================
        const int pw = warp - 2, pair = pw >> 1, half = pw & 1;
        const int c = lane & 7, grp = lane >> 3;             // row chunk within the 64-row block, 8-column group
        const uint4 *cb1 = reinterpret_cast<const uint4 *>(L.c1);
        const uint4 *cb2 = reinterpret_cast<const uint4 *>(cb2_ptr);
        const int rep = P.cb2_replicated ? (lane & (CB2_REPLICAS - 1)) : 0, rshift = P.cb2_replicated ? 2 : 0;
        const uint32_t kmax1 = (uint32_t)(L.k1 - 1), kmax2 = L.k2 ? (uint32_t)(L.k2 - 1) : 0u;
        int it0 = 0;                                         // k blocks of earlier segments
        FOR_EACH_SEGMENT {
            const int mt = tile % P.tiles_m;
            const int vrow = mt * (TILE_M / 8) + 8 * half + c;
            const bool row_ok = vrow < L.R;
            const uint8_t *row1 = L.s1.ptr + (long long)vrow * L.s1.stride;
            const uint8_t *row2 = L.k2 ? L.s2.ptr + (long long)vrow * L.s2.stride : nullptr;
            // this pair's k blocks of the segment: those whose running number is = pair (mod PAIRS)
            int kb = kb0 + ((pair - it0 % PAIRS) + PAIRS) % PAIRS;
            // a1: packed indices of 8 columns; the next visit's are loaded one visit ahead
            uint4 raw1 = make_uint4(0, 0, 0, 0);
            uint2 raw2 = make_uint2(0, 0);
            if (kb < kb1 && row_ok && kb * TILE_K + 8 * grp < L.N) {
                raw1 = __ldg(reinterpret_cast<const uint4 *>(row1 + 2LL * (kb * TILE_K + 8 * grp)));
                if (L.k2) raw2 = __ldg(reinterpret_cast<const uint2 *>(row2 + (kb * TILE_K + 8 * grp)));
            }
            for (; kb < kb1; kb += PAIRS) {
                const int it = it0 + (kb - kb0);
                const int s = it % A_STAGES;
                const int col0 = kb * TILE_K + 8 * grp;
                const bool live = row_ok && col0 < L.N;
                const uint32_t w1[4] = {raw1.x, raw1.y, raw1.z, raw1.w};
                const uint2 cur2 = raw2;
                {
                    const int ncol = col0 + PAIRS * TILE_K;
                    if (kb + PAIRS < kb1 && row_ok && ncol < L.N) {
                        raw1 = __ldg(reinterpret_cast<const uint4 *>(row1 + 2LL * ncol));
                        if (L.k2) raw2 = __ldg(reinterpret_cast<const uint2 *>(row2 + ncol));
                    }
                }
                // a3: main centroids, 8 reads in flight (issued before the wait: they do not touch the stage)
                uint4 cw[8];
#pragma unroll
                for (int j = 0; j < 8; j++) {
                    uint32_t id = (w1[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
                    id = min(id, kmax1);
                    // (no L1 allocation: the tensor core's operand reads share the L1 data path)
                    if (live) asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                                           : "=r"(cw[j].x), "=r"(cw[j].y), "=r"(cw[j].z), "=r"(cw[j].w) : "l"(cb1 + id));
                    else cw[j] = make_uint4(0, 0, 0, 0);
                }
                // a4: residual centroids from shared memory, all 8 before the wait as well: one shared-memory
                // round trip per visit instead of one per store
                uint4 rv[8];
#pragma unroll
                for (int j = 0; j < 8; j++) {
                    rv[j] = make_uint4(0, 0, 0, 0);
                    if (L.k2 && live) {
                        uint32_t id2 = ((j < 4 ? cur2.x : cur2.y) >> (8 * (j & 3))) & 0xFFu;
                        id2 = min(id2, kmax2);
                        rv[j] = cb2[(id2 << rshift) + rep];
                    }
                }
                // the whole warp takes the same decision: the stores below end in a warp-wide barrier
                ok = __all_sync(0xffffffffu, mbar_wait(bar_emptyA(s), ((it / A_STAGES) & 1) ^ 1, abort_flag, P.status));
                if (!ok) break;
                const uint32_t dst0 = sA + s * A_STAGE_BYTES + grp * A_SBO + half * A_LBO;
#pragma unroll
                for (int j = 0; j < 8; j++) {
                    uint4 w = cw[j];
                    {   // sum in FP16 (adding zero when there is no residual stage changes nothing)
                        __half2 a0 = __hadd2(*reinterpret_cast<__half2 *>(&w.x), *reinterpret_cast<const __half2 *>(&rv[j].x));
                        __half2 a1 = __hadd2(*reinterpret_cast<__half2 *>(&w.y), *reinterpret_cast<const __half2 *>(&rv[j].y));
                        __half2 a2 = __hadd2(*reinterpret_cast<__half2 *>(&w.z), *reinterpret_cast<const __half2 *>(&rv[j].z));
                        __half2 a3 = __hadd2(*reinterpret_cast<__half2 *>(&w.w), *reinterpret_cast<const __half2 *>(&rv[j].w));
                        w.x = *reinterpret_cast<uint32_t *>(&a0); w.y = *reinterpret_cast<uint32_t *>(&a1);
                        w.z = *reinterpret_cast<uint32_t *>(&a2); w.w = *reinterpret_cast<uint32_t *>(&a3);
                    }
                    if (col0 + j >= L.N) w = make_uint4(0, 0, 0, 0);
                    const uint32_t dst = dst0 + j * 128 + ((c ^ j) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the MMA
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_fullA(s));
            }
            it0 += kb1 - kb0;
        }
    } else {
        // ================= epilogue: two warps per TMEM lane quarter, one per 256-token half =================
        const int q = warp & 3;                                  // TMEM lane quarter this warp may read
        const int h = (warp - (2 + PRODUCER_WARPS)) >> 2;        // token half of the tile
        const bool fp32_out = L.out_dtype == VPTQ_DTYPE_FP32;
        const unsigned Mu = (unsigned)L.M;
        int seg_no = 0;
        unsigned epi_piece = 0;                                  // staged pieces so far (buffer parity)
        grid_dependency_wait();                                  // bias terms, tile flags and a cleared output come from the pre-pass
        FOR_EACH_SEGMENT {
            const int mt = tile % P.tiles_m, tt = tile / P.tiles_m;
            const int t0 = tt * TILE_N;
            const int m = mt * TILE_M + 32 * q + lane;
            const int t_cnt = min(TILE_N, P.B - t0);
            // a split tile: the piece with the last k blocks stores and announces it, the others add afterwards
            const bool split = kb0 != 0 || kb1 != P.kb_total;
            const bool add = P.flag_order ? kb1 != P.kb_total : split;
            const bool announce = P.flag_order && kb0 != 0 && kb1 == P.kb_total;
            // bias terms of this warp's 256 tokens, loaded before the wait (a load inside the drain would
            // cost an L2 round trip under load): lane l holds token 32*i + l of chunk i
            float bt_chunk[MMA_N / 32];
#pragma unroll
            for (int i = 0; i < MMA_N / 32; i++) {
                const int t = t0 + h * MMA_N + 32 * i + lane;
                bt_chunk[i] = (kb0 == 0 && t < P.B) ? __ldg(P.bterm + t) : 0.f;
            }
            ok = __all_sync(0xffffffffu, mbar_wait(bar_accum_full, seg_no & 1, abort_flag, P.status));
            if (!ok) break;
            tc_fence_after();
            if (add && P.flag_order) {
                ok = __all_sync(0xffffffffu, lane != 0 || flag_wait(P.tile_flags + tile, EPI_WARPS, abort_flag, P.status));
                if (!ok) break;
                asm volatile("fence.proxy.async;" ::: "memory");     // the reduce-adds below go through the async proxy
            }
            if (P.tma_out) {
                // FP32 output through shared memory: per 16 tokens a warp stages its [16][32] piece (lane =
                // output row: conflict free) and one lane hands it to TMA (store, or reduce-add for a partial
                // tile); two staging buffers per warp, so the copy of one piece overlaps the next.
                const uint32_t ebuf = sEpi + (uint32_t)(warp - (2 + PRODUCER_WARPS)) * (2 * EPI_BUF_BYTES);
                const int m0 = mt * TILE_M + 32 * q;
#pragma unroll
                for (int ci = 0; ci < MMA_N / 32; ci++) {    // unrolled: bt_chunk[] stays in registers
                    const int c0 = h * MMA_N + 32 * ci;
                    if (c0 >= t_cnt) break;
                    const float bt_lane = bt_chunk[ci];
#pragma unroll
                    for (int hh = 0; hh < 2; hh++) {
                        const int c1 = c0 + 16 * hh;
                        if (c1 >= t_cnt) break;
                        uint32_t r[16];
                        tmem_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c1, r);
                        if (kb0 == 0) {
#pragma unroll
                            for (int j = 0; j < 16; j++)
                                r[j] = __float_as_uint(__uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bt_lane, 16 * hh + j));
                        }
                        // the buffer written two pieces ago must have been read by its copy
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        __syncwarp();
                        const uint32_t buf = ebuf + (uint32_t)(epi_piece & 1) * EPI_BUF_BYTES;
#pragma unroll
                        for (int j = 0; j < 16; j++)
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(buf + j * 128u + lane * 4u), "r"(r[j]) : "memory");
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0 && m0 < L.M) tma_store_2d(&tmap_out, buf, m0, t0 + c1, add);
                        epi_piece++;
                    }
                }
            } else
#pragma unroll
            for (int ci = 0; ci < MMA_N / 32; ci++) {        // unrolled: bt_chunk[] stays in registers
                const int c0 = h * MMA_N + 32 * ci;
                if (c0 >= t_cnt) break;
                const float bt_lane = bt_chunk[ci];
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c0, r);
                if (kb0 == 0) {
#pragma unroll
                    for (int j = 0; j < 32; j++)
                        r[j] = __float_as_uint(__uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bt_lane, j));
                }
                if (m < L.M) {
                    const int nt = min(32, P.B - (t0 + c0));           // tokens of this chunk that exist
                    if (fp32_out) {
                        // one element per token row; independent addresses, no serial pointer chain
                        float *p = reinterpret_cast<float *>(P.out) + (long long)(t0 + c0) * L.M + m;
                        if (nt == 32 && !add) {
#pragma unroll
                            for (int j = 0; j < 32; j++) p[(unsigned)j * Mu] = __uint_as_float(r[j]);
                        } else if (nt == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j++) atomicAdd(p + (unsigned)j * Mu, __uint_as_float(r[j]));
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; j++) {
                                if (j < nt) {
                                    if (!add) p[(unsigned)j * Mu] = __uint_as_float(r[j]);
                                    else atomicAdd(p + (unsigned)j * Mu, __uint_as_float(r[j]));
                                }
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j++)
                            if (j < nt) store_out(P.out, (long long)(t0 + c0 + j) * L.M + m, __uint_as_float(r[j]), L.out_dtype);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_accum_empty);
            if (announce) {
                // this warp's part of the tile is in memory before the flag counts it
                if (lane == 0) {
                    if (P.tma_out) {
                        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                        asm volatile("fence.proxy.async;" ::: "memory");
                    }
                    __threadfence();
                    atomicAdd(P.tile_flags + tile, 1);
                }
            }
            seg_no++;
        }
        // the staging buffers must outlive the copies that read them, the copies must land before the end
        if (P.tma_out && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
#undef FOR_EACH_SEGMENT

    // ---- teardown: everybody meets, then the allocating warp frees TMEM ---------------
    tc_fence_before();
    __syncwarp();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

// ---- host side ----------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

struct GemmPlan {
    int tiles_m, tiles_t, kb_total, unit_gran, grid, any_split, flag_order, cb2_rep, cb2_bytes;
    long long units;
    size_t smem;
    long long ws_bytes, off_flags, off_bterm, off_xs;
};

size_t gemm_smem_bytes(int cb2_bytes)
{
    return 1024 + (size_t)A_STAGES * A_STAGE_BYTES + (size_t)B_STAGES * B_STAGE_BYTES + cb2_bytes +
           EPI_STAGE_BYTES + 8 * (2 * A_STAGES + 2 * B_STAGES + 2) + 16;
}

GemmPlan plan_gemm(const LayerView &L, int B)
{
    GemmPlan p;
    int workers = device_sm_count();
    p.cb2_rep = (L.k2 > 0 && L.k2 <= 256) ? 1 : 0;
    p.cb2_bytes = L.k2 ? L.k2 * 16 * (p.cb2_rep ? CB2_REPLICAS : 1) : 0;
    p.tiles_m = ceil_div(L.M, TILE_M);
    p.tiles_t = ceil_div(B, TILE_N);
    p.kb_total = ceil_div(L.N, TILE_K);
    p.units = (long long)p.tiles_m * p.tiles_t * p.kb_total;
    // the pieces of a split tile meet in an FP32 output by red.add; other output types get whole tiles
    // (and so does a deterministic call: reduce-adds of several pieces arrive in no fixed order)
    p.unit_gran = (L.out_dtype == VPTQ_DTYPE_FP32 && !L.deterministic) ? 1 : p.kb_total;
    const long long groups = p.units / p.unit_gran;
    if (groups < workers) workers = (int)groups;
    p.grid = workers;
    p.any_split = 0;
    for (int c = 1; c < workers; c++)
        if ((groups * c / workers * p.unit_gran) % p.kb_total != 0) p.any_split = 1;
    // flag order makes CTAs wait for one another: only for a call that has the GPU to itself
    p.flag_order = (p.any_split && p.units / workers >= FLAG_ORDER_MIN_SHARE && !L.concurrent) ? 1 : 0;
    p.smem = gemm_smem_bytes(p.cb2_bytes);
    p.off_flags = WS_STATUS_BYTES;
    p.off_bterm = p.off_flags + ((long long)p.tiles_m * p.tiles_t * 4 + 255) / 256 * 256;
    p.off_xs = p.off_bterm + ((long long)B * 4 + 255) / 256 * 256;
    // activation tile images: whole 256-token halves and whole k blocks
    p.ws_bytes = p.off_xs + (long long)ceil_div(B, MMA_N) * p.kb_total * B_HALF_BYTES;
    return p;
}

}  // namespace

bool gemm_tcgen05_supported(const LayerView &L, int B)
{
    if (L.G > 1) return false;          // one codebook pair per layer here
    if (B <= 16) return false;
    if (L.v != 8 || L.n_out != 0 || L.scale_rows) return false;
    if (L.s1.bits != 16) return false;
    if (L.k2 && (L.s2.bits != 8 || L.k2 > 2048)) return false;
    return true;
}

// (the scratch layout does not depend on the device, so this query makes no CUDA call)
long long gemm_tcgen05_workspace_bytes(const LayerView &L, int B) { return plan_gemm(L, B).ws_bytes; }

int gemm_tcgen05_launches(const LayerView &, int) { return 2; }   // pre-pass + GEMM

bool gemm_tcgen05_waits_between_ctas(const LayerView &L, int B) { return plan_gemm(L, B).flag_order != 0; }

cudaError_t launch_gemm_tcgen05(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st)
{
    const GemmPlan pl = plan_gemm(L, B);
    uint8_t *w8 = reinterpret_cast<uint8_t *>(ws);
    int *status = reinterpret_cast<int *>(w8);
    int *tile_flags = reinterpret_cast<int *>(w8 + pl.off_flags);
    float *bterm = reinterpret_cast<float *>(w8 + pl.off_bterm);
    uint8_t *xs = w8 + pl.off_xs;

    // FP32 output with 16-byte aligned rows: the epilogue goes through shared memory and TMA
    const int tma_out = (L.out_dtype == VPTQ_DTYPE_FP32 && (L.M & 3) == 0) ? 1 : 0;
    CUtensorMap tmap_out;
    memset(&tmap_out, 0, sizeof(tmap_out));      // not read by the kernel when tma_out == 0
    if (tma_out) {
        EncodeTiledFn encode = get_encode_fn();
        if (encode == nullptr) return cudaErrorNotSupported;
        const cuuint64_t odim[2] = {(cuuint64_t)L.M, (cuuint64_t)B};
        const cuuint64_t ostride[1] = {(cuuint64_t)L.M * 4};
        const cuuint32_t obox[2] = {32, 16};
        const cuuint32_t estr[2] = {1, 1};
        const CUresult r = encode(&tmap_out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, out, odim, ostride, obox, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }

    cudaError_t e;
    gemm_prepass_kernel<<<ceil_div(B, MMA_N) * MMA_N, PRE_THREADS, 0, st>>>(
        L, x, B, xs, bterm, status, tile_flags, pl.tiles_m * pl.tiles_t,
        (pl.any_split && !pl.flag_order) ? reinterpret_cast<float *>(out) : nullptr);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    GemmParams P;
    P.L = L; P.out = out; P.B = B;
    P.tiles_m = pl.tiles_m; P.tiles_t = pl.tiles_t; P.kb_total = pl.kb_total;
    P.unit_gran = pl.unit_gran; P.units = pl.units;
    P.cb2_replicated = pl.cb2_rep; P.cb2_bytes = pl.cb2_bytes;
    P.status = status; P.bterm = bterm; P.xs = xs; P.tile_flags = tile_flags; P.flag_order = pl.flag_order; P.tma_out = tma_out;
    e = cudaFuncSetAttribute(gemm_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    // programmatic dependent launch: set-up and the producers' first reads overlap the pre-pass
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(pl.grid, 1, 1);
    cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel, tmap_out, P);
}

}  // namespace vptq
