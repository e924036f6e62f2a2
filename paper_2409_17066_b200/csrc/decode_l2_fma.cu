// Decode path for a main codebook too large for shared memory (k1 = 65536, v = 8: 1 MiB),
// batch 1..4 per launch.
//
// The codebook stays in global memory and is served by L2 (and whatever part of it the
// per-SM L1 holds); every index costs one 16-byte random read (a3).  The kernel is therefore
// organised around keeping many of those reads in flight: a lane takes 8 consecutive indices
// with one 128-bit load (a1), issues the 8 centroid loads back to back, and only then
// consumes them.  The residual codebook (a4) sits in shared memory, replicated 8 times with a
// 16-byte skew so that the 8 lanes of a quarter warp always hit different banks.
//
// Work split: grid = (row blocks, K slabs).  A CTA stages the scaled activations of its slab
// (x*s, FP32) in shared memory once and its warps walk vector rows; per (row, slab) a warp
// reduces its 8*B partial sums with a halving butterfly.  With one slab the result is stored
// directly; with several, partial sums meet in an FP32 scratch array through atomic adds and
// the last CTA of a row block (a counter tells) converts and stores (a7).
#include "common.cuh"
#include "decode.cuh"

namespace vptq {

namespace {

constexpr int L2_WARPS = 8;
constexpr int L2_THREADS = L2_WARPS * 32;

struct L2FmaParams {
    LayerView L;
    const void *x;
    void *out;
    int B;                 // tokens in this launch (<= TB)
    int slab_cols;         // columns per K slab (multiple of 256)
    int n_slabs;
    int rows_per_warp;
    int cb2_replicated;    // 1: [k2][8 replicas][16 B], 0: [k2][16 B]
    float *yacc;           // [B][M] scratch (n_slabs > 1)
    unsigned *counters;    // [row blocks] scratch (n_slabs > 1)
};

__device__ __forceinline__ float2 h2f(uint32_t w)
{
    return __half22float2(*reinterpret_cast<__half2 *>(&w));
}

template <int TB>
__global__ void __launch_bounds__(L2_THREADS)
decode_l2_fma_kernel(L2FmaParams P)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const LayerView &L = P.L;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slab = blockIdx.y;
    const int c_begin = slab * P.slab_cols;
    const int c_end = min(L.N, c_begin + P.slab_cols);
    const int n_iter = (c_end - c_begin + 255) / 256;

    float *xs = reinterpret_cast<float *>(smem);                       // [n_iter][TB][2][32][4]
    const int xs_floats = (P.slab_cols / 256) * TB * 256;
    float *bterm = xs + xs_floats;                                     // [TB]
    float *red = bterm + 4;                                            // [L2_WARPS][TB]
    uint4 *cb2 = reinterpret_cast<uint4 *>(red + L2_WARPS * 4);
    __shared__ unsigned s_last;

    // ---- stage scaled activations of the slab, and the slab's share of the bias term -----------
    {
        float bacc[TB];
#pragma unroll
        for (int t = 0; t < TB; t++) bacc[t] = 0.f;
        for (int cl = threadIdx.x; cl < n_iter * 256; cl += L2_THREADS) {
            const int n = c_begin + cl;
            const int i = cl >> 8, ln = (cl >> 3) & 31, s = cl & 7;
            float sc = 1.f, bi = 0.f;
            if (n < c_end && L.has_scale) {
                sc = __half2float(__ldg(L.scale + n));
                bi = __half2float(__ldg(L.bias + n));
            }
#pragma unroll
            for (int t = 0; t < TB; t++) {
                float xv = (n < c_end && t < P.B) ? load_act(P.x, (long long)t * L.N + n, L.x_bf16) : 0.f;
                xs[((i * TB + t) * 2 + (s >> 2)) * 128 + ln * 4 + (s & 3)] = xv * sc;
                bacc[t] += xv * bi;
            }
        }
#pragma unroll
        for (int t = 0; t < TB; t++) {
            float a = bacc[t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0) red[warp * 4 + t] = a;
        }
    }
    // ---- residual codebook -> shared memory ---------------------------------------------------------
    if (L.k2) {
        const uint4 *src = reinterpret_cast<const uint4 *>(L.c2);
        if (P.cb2_replicated) {
            for (int i = threadIdx.x; i < L.k2 * 8; i += L2_THREADS) cb2[i] = __ldg(src + (i >> 3));
        } else {
            for (int i = threadIdx.x; i < L.k2; i += L2_THREADS) cb2[i] = __ldg(src + i);
        }
    }
    __syncthreads();
    if (threadIdx.x < TB) {
        float a = 0.f;
        for (int w = 0; w < L2_WARPS; w++) a += red[w * 4 + threadIdx.x];
        bterm[threadIdx.x] = a;
    }
    __syncthreads();

    const uint4 *cb1 = reinterpret_cast<const uint4 *>(L.c1);
    const int rows_per_cta = L2_WARPS * P.rows_per_warp;
    const int r0 = blockIdx.x * rows_per_cta;
    const int rep = P.cb2_replicated ? (lane & 7) : 0;
    const int rshift = P.cb2_replicated ? 3 : 0;

    for (int rw = 0; rw < P.rows_per_warp; rw++) {
        const int r = r0 + rw * L2_WARPS + warp;
        if (r >= L.R) break;
        const uint8_t *row1 = L.s1.ptr + (long long)r * L.s1.stride;
        const uint8_t *row2 = L.k2 ? L.s2.ptr + (long long)r * L.s2.stride : nullptr;
        float acc[TB][8];
#pragma unroll
        for (int t = 0; t < TB; t++)
#pragma unroll
            for (int j = 0; j < 8; j++) acc[t][j] = 0.f;

        // packed indices of iteration 0 (a lane's 8 columns: c_begin + 256*i + 8*lane + s)
        int grp = (c_begin >> 3) + lane;
        uint4 raw1 = make_uint4(0, 0, 0, 0);
        uint2 raw2 = make_uint2(0, 0);
        bool live = 8 * grp < L.N;
        if (live) {
            raw1 = __ldg(reinterpret_cast<const uint4 *>(row1) + grp);
            if (L.k2) raw2 = __ldg(reinterpret_cast<const uint2 *>(row2) + grp);
        }
        for (int i = 0; i < n_iter; i++) {
            const uint32_t w1[4] = {raw1.x, raw1.y, raw1.z, raw1.w};
            const uint2 cur2 = raw2;
            const bool cur_live = live;
            // prefetch the next iteration's indices
            grp += 32;
            live = (i + 1 < n_iter) && (8 * grp < c_end);
            if (live) {
                raw1 = __ldg(reinterpret_cast<const uint4 *>(row1) + grp);
                if (L.k2) raw2 = __ldg(reinterpret_cast<const uint2 *>(row2) + grp);
            }
            if (!cur_live) continue;       // this lane's 8 columns lie beyond the row: xs there is 0 anyway
            // a3: 8 centroid reads in flight
            uint4 cw[8];
#pragma unroll
            for (int s = 0; s < 8; s++) {
                uint32_t id = (w1[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                id = min(id, (uint32_t)(L.k1 - 1));
                cw[s] = __ldg(cb1 + id);
            }
            const float *xp = xs + (size_t)i * TB * 256 + lane * 4;
#pragma unroll
            for (int s = 0; s < 8; s++) {
                float2 c01 = h2f(cw[s].x), c23 = h2f(cw[s].y), c45 = h2f(cw[s].z), c67 = h2f(cw[s].w);
                if (L.k2) {
                    uint32_t id2 = ((s < 4 ? cur2.x : cur2.y) >> (8 * (s & 3))) & 0xFFu;
                    id2 = min(id2, (uint32_t)(L.k2 - 1));
                    const uint4 rv = cb2[(id2 << rshift) + rep];
                    float2 r01 = h2f(rv.x), r23 = h2f(rv.y), r45 = h2f(rv.z), r67 = h2f(rv.w);
                    c01.x += r01.x; c01.y += r01.y; c23.x += r23.x; c23.y += r23.y;
                    c45.x += r45.x; c45.y += r45.y; c67.x += r67.x; c67.y += r67.y;
                }
#pragma unroll
                for (int t = 0; t < TB; t++) {
                    const float xv = xp[(t * 2 + (s >> 2)) * 128 + (s & 3)];
                    acc[t][0] += xv * c01.x; acc[t][1] += xv * c01.y;
                    acc[t][2] += xv * c23.x; acc[t][3] += xv * c23.y;
                    acc[t][4] += xv * c45.x; acc[t][5] += xv * c45.y;
                    acc[t][6] += xv * c67.x; acc[t][7] += xv * c67.y;
                }
            }
        }

        // ---- halving butterfly: 8*TB partial sums per lane -> one (or a few equal) totals per lane ----
        constexpr int NV = 8 * TB;
        float v[NV];
#pragma unroll
        for (int t = 0; t < TB; t++)
#pragma unroll
            for (int j = 0; j < 8; j++) v[t * 8 + j] = acc[t][j];
        int vi = 0;            // index of the value this lane ends up holding
        {
            int n = NV, o = 16;
#pragma unroll
            for (int step = 0; step < 5; step++) {
                if (n > 1) {
                    const bool up = (lane & o) != 0;
                    const int h = n / 2;
#pragma unroll
                    for (int k = 0; k < NV / 2; k++) {
                        if (k < h) {
                            float send = up ? v[k] : v[k + h];
                            float keep = up ? v[k + h] : v[k];
                            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                        }
                    }
                    vi += up ? h : 0;
                    n = h;
                } else {
                    v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
                }
                o >>= 1;
            }
        }
        // lanes that hold a distinct value: for NV = 8 those with (lane & 3) == 0, NV = 16: (lane & 1) == 0
        const int dup = 32 / NV;
        if ((lane & (dup - 1)) == 0) {
            const int t = vi >> 3, j = vi & 7;
            const int m = r * 8 + j;
            if (t < P.B && m < L.M) {
                float y = v[0] + bterm[t];
                if (P.n_slabs == 1) store_out(P.out, (long long)t * L.M + m, y, L.out_dtype);
                else atomicAdd(P.yacc + (long long)t * L.M + m, y);
            }
        }
    }

    // ---- several slabs: the last CTA of this row block converts and stores -----------------------------
    if (P.n_slabs > 1) {
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_last = (atomicAdd(P.counters + blockIdx.x, 1u) == (unsigned)(P.n_slabs - 1));
        __syncthreads();
        if (s_last) {
            __threadfence();
            const int m_lo = r0 * 8;
            const int m_hi = min(L.M, (r0 + rows_per_cta) * 8);
            const int n_m = m_hi - m_lo;
            for (int i = threadIdx.x; i < n_m * P.B; i += L2_THREADS) {
                const int t = i / n_m, m = m_lo + i % n_m;
                float y = __ldcg(P.yacc + (long long)t * L.M + m);
                store_out(P.out, (long long)t * L.M + m, y, L.out_dtype);
            }
        }
    }
}

struct L2Plan {
    int slab_cols, n_slabs, rows_per_warp, row_blocks, cb2_rep;
    size_t smem;
    long long ws_bytes;
};

L2Plan plan_l2(const LayerView &L, int TB)
{
    L2Plan p;
    const long long chunks = (L.N + 255) / 256;
    long long units = (long long)L.R * chunks;
    long long iters = (units + 3500) / 7000;
    if (iters < 1) iters = 1;
    if (iters > 8) iters = 8;
    if (iters > chunks) iters = chunks;
    p.n_slabs = (int)((chunks + iters - 1) / iters);
    iters = (chunks + p.n_slabs - 1) / p.n_slabs;      // balance the slabs
    p.slab_cols = (int)iters * 256;
    p.n_slabs = (int)((chunks + iters - 1) / iters);
    long long wu = (long long)L.R * p.n_slabs;
    long long rpw = wu / (L2_WARPS * 888);
    if (rpw < 1) rpw = 1;
    if (rpw > 8) rpw = 8;
    p.rows_per_warp = (int)rpw;
    p.row_blocks = ceil_div(L.R, L2_WARPS * p.rows_per_warp);
    p.cb2_rep = (L.k2 > 0 && L.k2 <= 256) ? 1 : 0;
    p.smem = (size_t)(p.slab_cols / 256) * TB * 256 * 4 + 4 * 4 + L2_WARPS * 4 * 4 +
             (size_t)L.k2 * 16 * (p.cb2_rep ? 8 : 1);
    p.ws_bytes = 0;
    if (p.n_slabs > 1) {
        long long y = ((long long)TB * L.M * 4 + 255) / 256 * 256;
        long long c = ((long long)p.row_blocks * 4 + 255) / 256 * 256;
        p.ws_bytes = y + c;
    }
    return p;
}

int token_group(int B) { return B >= 4 ? 4 : (B >= 2 ? 2 : 1); }

}  // namespace

bool l2_fma_supported(const LayerView &L, int B)
{
    if (B < 1 || B > 16) return false;
    if (L.v != 8 || L.n_out != 0 || L.scale_rows) return false;
    if (L.s1.bits != 16) return false;
    if (L.k2 && (L.s2.bits != 8 || L.k2 > 2048)) return false;
    return true;
}

long long l2_fma_workspace_bytes(const LayerView &L, int B)
{
    return plan_l2(L, token_group(B)).ws_bytes;
}

int l2_fma_launches(const LayerView &L, int B)
{
    const int TB = token_group(B);
    const int groups = (B + TB - 1) / TB;
    (void)L;
    return groups;     // one kernel per token group (the scratch memset is not a kernel)
}

template <int TB>
static cudaError_t launch_group(const LayerView &L, const L2Plan &pl, const void *x, int Bg, void *out,
                                void *ws, cudaStream_t st)
{
    L2FmaParams P;
    P.L = L; P.x = x; P.out = out; P.B = Bg;
    P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs; P.rows_per_warp = pl.rows_per_warp;
    P.cb2_replicated = pl.cb2_rep;
    P.yacc = nullptr; P.counters = nullptr;
    cudaError_t e;
    if (pl.n_slabs > 1) {
        long long y = ((long long)TB * L.M * 4 + 255) / 256 * 256;
        P.yacc = reinterpret_cast<float *>(ws);
        P.counters = reinterpret_cast<unsigned *>(reinterpret_cast<uint8_t *>(ws) + y);
        e = cudaMemsetAsync(ws, 0, (size_t)pl.ws_bytes, st);
        if (e != cudaSuccess) return e;
    }
    e = cudaFuncSetAttribute(decode_l2_fma_kernel<TB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    dim3 grid(pl.row_blocks, pl.n_slabs);
    decode_l2_fma_kernel<TB><<<grid, L2_THREADS, pl.smem, st>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_decode_l2_fma(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st)
{
    const int TB = token_group(B);
    const L2Plan pl = plan_l2(L, TB);
    const size_t xe = 2, oe = (L.out_dtype == VPTQ_DTYPE_FP32) ? 4 : 2;
    for (int t0 = 0; t0 < B; t0 += TB) {
        const int Bg = (B - t0 < TB) ? (B - t0) : TB;
        const void *xg = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * L.N * xe;
        void *og = reinterpret_cast<uint8_t *>(out) + (size_t)t0 * L.M * oe;
        cudaError_t e;
        if (TB == 4) e = launch_group<4>(L, pl, xg, Bg, og, ws, st);
        else if (TB == 2) e = launch_group<2>(L, pl, xg, Bg, og, ws, st);
        else e = launch_group<1>(L, pl, xg, Bg, og, ws, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace vptq
