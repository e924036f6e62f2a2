// Decode path for layers the shared-memory and L2 kernels do not take: group-wise codebooks
// (Sec. 3.1), vector lengths up to 16 (the published 2-bit models use v = 12 with two 4096-entry
// codebooks per group, App. B table), any index width; batch 1..4 per launch, FP32 FMAs.
//
// Codebooks stay in global memory (a group's pair is 2 x k x 2v bytes; all groups together are a
// few hundred KB, L2-resident and partly L1-resident) and every index costs one random read of a
// 2v-byte row (a3, a4).  Organisation as in the other decode kernels: persistent grid, one CTA per
// SM owning whole vector rows; (vector row, 256-column chunk) tasks dealt out evenly over the warps;
// per task a lane unpacks 8 consecutive indices of each stream (a1; the next task's packed words are
// already in flight) and handles them four at a time: main and residual rows of its column's group
// are read, added in FP16 and accumulated into v sums per token.  x*s is staged per CTA as FP16,
// main and outlier columns apart; outlier columns (a5) are a small pass of their own; warp partial
// sums meet in shared memory; the epilogue adds the bias term and converts (a7).  No scratch.
#include "common.cuh"
#include "decode.cuh"
#include "index_words.cuh"
#include "fused_split.cuh"

namespace vptq {

namespace {

constexpr int XS_BUDGET = 96 * 1024;        // bytes of staged main-column activations per CTA
constexpr int PART_BUDGET = 32 * 1024;      // bytes of per-row partial sums per CTA
constexpr int GL_WARPS = 16;

struct GlFmaParams {
    LayerView L[MAX_FUSED];        // a fused launch: layer l is the work of CTAs [cta_begin[l], cta_begin[l + 1])
    void *out[MAX_FUSED];
    int cta_begin[MAX_FUSED + 1];
    int n_layers;
    const void *x;
    int B;                 // tokens in this launch (<= TB)
    int slab_cols;         // main columns per slab (multiple of 256)
    int n_slabs;
    int n_out_pad;         // outlier columns rounded up to 8
    int part_floats;
};

__device__ __forceinline__ float2 h2f(uint32_t w)
{
    return __half22float2(*reinterpret_cast<__half2 *>(&w));
}

// One centroid of an even vector length v <= 2*VW as VW half2 words (zero beyond v).
template <int VW>
__device__ __forceinline__ void load_row_words(const __half *__restrict__ tab, long long e, int vw, uint32_t (&w)[VW])
{
    if ((vw & 1) == 0) {
        // v a multiple of 4: rows are 8-byte aligned, half as many load instructions
        const uint2 *p = reinterpret_cast<const uint2 *>(tab) + e * (vw >> 1);
#pragma unroll
        for (int i = 0; i < VW / 2; i++) {
            uint2 t = make_uint2(0u, 0u);
            if (2 * i < vw) t = __ldg(p + i);
            w[2 * i] = t.x; w[2 * i + 1] = t.y;
        }
        if (VW & 1) w[VW - 1] = 0u;
    } else {
        const uint32_t *p = reinterpret_cast<const uint32_t *>(tab) + e * vw;     // rows are 2v bytes: 4-byte aligned
#pragma unroll
        for (int i = 0; i < VW; i++) w[i] = i < vw ? __ldg(p + i) : 0u;
    }
}

template <int TB, int VV, bool RES, bool FUSED>
__global__ void __launch_bounds__(GL_WARPS * 32, 1)
decode_gl_fma_kernel(const __grid_constant__ GlFmaParams P)
{
    constexpr int WARPS = GL_WARPS, THREADS = WARPS * 32, VW = VV / 2;
    extern __shared__ __align__(16) uint8_t smem[];
    // the layer this CTA works on, and its place among that layer's CTAs
    int li = 0;
    if (FUSED)
        while (li + 1 < P.n_layers && (int)blockIdx.x >= P.cta_begin[li + 1]) li++;
    const LayerView &L = P.L[FUSED ? li : 0];
    void *const out = P.out[FUSED ? li : 0];
    const int bid = FUSED ? (int)blockIdx.x - P.cta_begin[li] : (int)blockIdx.x;
    const int gdim = FUSED ? P.cta_begin[li + 1] - P.cta_begin[li] : (int)gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    __half *xs_out = reinterpret_cast<__half *>(smem);                                       // [TB][n_out_pad]
    __half *xs = xs_out + (size_t)TB * P.n_out_pad;                                          // [TB][slab_cols]
    float *part = reinterpret_cast<float *>(xs + (size_t)TB * P.slab_cols);                  // [rows][TB][16]
    float *bterm = part + P.part_floats;                                                     // [8]
    float *red = bterm + 8;                                                                  // [WARPS][8]

    // vector rows of this CTA, and the output rows they cover
    const int r0 = (int)((long long)L.R * bid / gdim);
    const int r1 = (int)((long long)L.R * (bid + 1) / gdim);
    const int m_lo = r0 * L.v;
    const int m_hi = min(L.M, r1 * L.v);
    const int vw = L.v >> 1;

    for (int i = threadIdx.x; i < P.part_floats; i += THREADS) part[i] = 0.f;
    if (threadIdx.x < 8) bterm[threadIdx.x] = 0.f;

    for (int slab = 0; slab < P.n_slabs; slab++) {
        const int c_begin = slab * P.slab_cols;                 // main-region columns of the slab
        const int c_end = min(L.Nc, c_begin + P.slab_cols);
        const int chunks = (c_end - c_begin + 255) >> 8;

        // ---- this warp's task range: (row, chunk of the slab), chunk fastest; first task's packed words --
        const int n_tasks = (r1 - r0) * chunks;
        int q = (int)((long long)n_tasks * warp / WARPS);
        const int q_end = (int)((long long)n_tasks * (warp + 1) / WARPS);
        int r = r0 + (chunks ? q / chunks : 0), ch = chunks ? q % chunks : 0;
        uint4 raw1 = make_uint4(0, 0, 0, 0), raw2 = make_uint4(0, 0, 0, 0);
        if (q < q_end) {
            const int grp = (c_begin >> 3) + ch * 32 + lane;
            raw1 = load_raw8(L.s1.ptr + (long long)r * L.s1.stride, L.s1.stride, grp, c_end, L.s1.bits);
            if (RES) raw2 = load_raw8(L.s2.ptr + (long long)r * L.s2.stride, L.s2.stride, grp, c_end, L.s2.bits);
        }

        // ---- stage x*s (FP16): outlier columns once, the slab's main columns; bias term in slab 0 -----
        {
            float bacc[TB];
#pragma unroll
            for (int t = 0; t < TB; t++) bacc[t] = 0.f;
            // columns to visit: all of them in slab 0 (bias term, outlier columns), else the slab's own
            const int n_first = slab == 0 ? 0 : L.n_out + c_begin;
            const int n_last = slab == 0 ? L.N : L.n_out + c_end;
#pragma unroll 4
            for (int n = n_first + threadIdx.x; n < n_last; n += THREADS) {
                float sc = 1.f, bi = 0.f;
                if (L.has_scale) {
                    sc = __half2float(__ldg(L.scale + n));
                    bi = __half2float(__ldg(L.bias + n));
                }
                const int c = n - L.n_out;
                const bool mine = c >= c_begin && c < c_end;
#pragma unroll
                for (int t = 0; t < TB; t++) {
                    const float xv = t < P.B ? load_act(P.x, (long long)t * L.N + in_col(L, n), L.x_bf16) : 0.f;
                    const __half hv = __float2half_rn(xv * sc);
                    if (c < 0) xs_out[t * P.n_out_pad + n] = hv;
                    else if (mine) xs[t * P.slab_cols + (c - c_begin)] = hv;
                    if (slab == 0) bacc[t] += xv * bi;
                }
            }
            // zero the ragged end of the slab (columns >= Nc inside the last chunk)
            for (int cl = (c_end - c_begin) + threadIdx.x; cl < chunks * 256; cl += THREADS)
#pragma unroll
                for (int t = 0; t < TB; t++) xs[t * P.slab_cols + cl] = __float2half_rn(0.f);
            if (slab == 0) {
#pragma unroll
                for (int t = 0; t < TB; t++) {
                    float a = bacc[t];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                    if (lane == 0) red[warp * 8 + t] = a;
                }
            }
        }
        __syncthreads();
        if (slab == 0 && threadIdx.x < TB) {
            float a = 0.f;
            for (int w = 0; w < WARPS; w++) a += red[w * 8 + threadIdx.x];
            bterm[threadIdx.x] = a;
        }

        // ---- a5: outlier columns (slab 0 only): FP32, centroids gathered from global memory ------------
        if (slab == 0 && L.n_out > 0) {
            const int q_lo = m_lo / L.v0, q_hi = (m_hi + L.v0 - 1) / L.v0;
            for (int qq = q_lo + warp; qq < q_hi; qq += WARPS) {
                const uint8_t *row0 = L.s0.ptr + (long long)qq * L.s0.stride;
#pragma unroll 1
                for (int t0 = 0; t0 < P.B; t0 += 4) {
                    float oacc[8][4];
#pragma unroll
                    for (int j = 0; j < 8; j++)
#pragma unroll
                        for (int t = 0; t < 4; t++) oacc[j][t] = 0.f;
                    for (int n = lane; n < L.n_out; n += 32) {
                        const int i0 = clamp_index(load_index(row0, n, L.s0.bits), L.k0);
                        const uint4 cw = load_centroid_row(L.c0, i0, L.v0);
                        const float2 c01 = h2f(cw.x), c23 = h2f(cw.y), c45 = h2f(cw.z), c67 = h2f(cw.w);
                        const float cj[8] = {c01.x, c01.y, c23.x, c23.y, c45.x, c45.y, c67.x, c67.y};
#pragma unroll
                        for (int t = 0; t < 4; t++) {
                            const float xv = (t0 + t < TB) ? __half2float(xs_out[min(t0 + t, TB - 1) * P.n_out_pad + n]) : 0.f;
#pragma unroll
                            for (int j = 0; j < 8; j++) oacc[j][t] += xv * cj[j];
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; j++) {
#pragma unroll
                        for (int t = 0; t < 4; t++) {
                            float a = oacc[j][t];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                            const int m = qq * L.v0 + j;
                            if (lane == 0 && j < L.v0 && m >= m_lo && m < m_hi && t0 + t < P.B) {
                                const int rr = m / L.v, jj = m - rr * L.v;
                                atomicAdd(part + ((rr - r0) * TB + t0 + t) * 16 + jj, a);
                            }
                        }
                    }
                }
            }
        }

        // ---- main tasks -----------------------------------------------------------------------------
        float acc[TB][VV];
#pragma unroll
        for (int t = 0; t < TB; t++)
#pragma unroll
            for (int j = 0; j < VV; j++) acc[t][j] = 0.f;

        while (q < q_end) {
            uint32_t w1[4], w2[4] = {0, 0, 0, 0};
            decode8(raw1, L.s1.bits, L.k1, w1);
            if (RES) decode8(raw2, L.s2.bits, L.k2, w2);
            const int cur_r = r, cur_ch = ch;
            const int col0 = c_begin + cur_ch * 256 + lane * 8;      // this lane's first main column
            const bool cur_live = col0 < c_end;
            // next task, and its packed words
            q++;
            if (++ch == chunks) { ch = 0; r++; }
            if (q < q_end) {
                const int grp = (c_begin >> 3) + ch * 32 + lane;
                raw1 = load_raw8(L.s1.ptr + (long long)r * L.s1.stride, L.s1.stride, grp, c_end, L.s1.bits);
                if (RES) raw2 = load_raw8(L.s2.ptr + (long long)r * L.s2.stride, L.s2.stride, grp, c_end, L.s2.bits);
            }
            if (cur_live) {
                // this lane's 8 scaled activations per token
                uint4 xv4[TB];
#pragma unroll
                for (int t = 0; t < TB; t++)
                    xv4[t] = *reinterpret_cast<const uint4 *>(xs + t * P.slab_cols + cur_ch * 256 + lane * 8);
                // Sec. 3.1: a column's tables are those of its group (pad columns of the last chunk stay in
                // the last group: their indices are 0 and their activations 0)
                int g = col0 / L.cpg;
                int g_next = (g + 1) * L.cpg;                       // first column of the next group
#pragma unroll
                for (int s0 = 0; s0 < 8; s0 += 4) {
                    // a3/a4: main and residual rows of 4 columns in flight
                    uint32_t cw[4][VW], rw[4][VW];
#pragma unroll
                    for (int u = 0; u < 4; u++) {
                        const int s = s0 + u;
                        if (col0 + s >= g_next && g + 1 < L.G) { g++; g_next += L.cpg; }
                        const uint32_t id1 = (w1[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                        load_row_words<VW>(L.c1, (long long)g * L.k1 + id1, vw, cw[u]);
                        if (RES) {
                            const uint32_t id2 = (w2[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                            load_row_words<VW>(L.c2, (long long)g * L.k2 + id2, vw, rw[u]);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; u++) {
                        const int s = s0 + u;
                        float cj[VV];
#pragma unroll
                        for (int i = 0; i < VW; i++) {
                            uint32_t w = cw[u][i];
                            if (RES) {      // summed in FP16 (one rounding of 2^-11)
                                const __half2 a = __hadd2(*reinterpret_cast<__half2 *>(&w), *reinterpret_cast<const __half2 *>(&rw[u][i]));
                                w = *reinterpret_cast<const uint32_t *>(&a);
                            }
                            const float2 p = h2f(w);
                            cj[2 * i] = p.x; cj[2 * i + 1] = p.y;
                        }
#pragma unroll
                        for (int t = 0; t < TB; t++) {
                            const uint32_t xw = (s >> 1) == 0 ? xv4[t].x : (s >> 1) == 1 ? xv4[t].y : (s >> 1) == 2 ? xv4[t].z : xv4[t].w;
                            const float2 xp = h2f(xw);
                            const float xv = (s & 1) ? xp.y : xp.x;
#pragma unroll
                            for (int j = 0; j < VV; j++) acc[t][j] += xv * cj[j];
                        }
                    }
                }
            }
            if (q < q_end && r == cur_r) continue;

            // ---- row change (or end of range): halving butterfly over 16*TB values per lane ---------------
            constexpr int NV = 16 * TB;
            float v[NV];
#pragma unroll
            for (int t = 0; t < TB; t++)
#pragma unroll
                for (int j = 0; j < 16; j++) {
                    v[t * 16 + j] = j < VV ? acc[t][j < VV ? j : 0] : 0.f;
                    if (j < VV) acc[t][j] = 0.f;
                }
            const int vi = halving_butterfly<NV>(v, lane);     // index of the first value this lane ends up holding
            // NV >= 32: every lane holds NV/32 distinct values; NV = 16: lanes with the low bit clear
            constexpr int KEEP = NV >= 32 ? NV / 32 : 1;
            constexpr int dup = NV >= 32 ? 1 : 32 / NV;
            if ((lane & (dup - 1)) == 0) {
#pragma unroll
                for (int k = 0; k < KEEP; k++) {
                    const int idx = vi + k, t = idx >> 4, j = idx & 15;
                    if (j < VV) atomicAdd(part + ((cur_r - r0) * TB + t) * 16 + j, v[k]);
                }
            }
        }
        __syncthreads();      // the slab's xs is dead; part[] complete after the last slab
    }

    // ---- bias term, conversion, store ----------------------------------------------------------------
    const int n_m = m_hi - m_lo;
    for (int i = threadIdx.x; i < n_m * P.B; i += THREADS) {
        const int t = i / n_m, ml = i % n_m;       // consecutive threads -> consecutive m
        const int m = m_lo + ml;
        const int rr = m / L.v, jj = m - rr * L.v;
        const float y = part[((rr - r0) * TB + t) * 16 + jj] + bterm[t];
        store_out(out, (long long)t * L.M + m, y, L.out_dtype);
    }
}

struct GlFmaPlan {
    int slab_cols, n_slabs, grid, part_floats, n_out_pad;
    size_t smem;
    bool ok;
    int cta_begin[MAX_FUSED + 1];   // fused launches only
};

int gl_token_group(int B) { return B >= 4 ? 4 : (B >= 2 ? 2 : 1); }

GlFmaPlan plan_gl_fma(const LayerView &L, int TB)
{
    GlFmaPlan p;
    const int G = device_sm_count();
    p.grid = L.R < G ? L.R : G;
    const int rows_cta = ceil_div(L.R, p.grid);
    p.part_floats = rows_cta * TB * 16;
    p.n_out_pad = (L.n_out + 7) / 8 * 8;
    const int nc_pad = (L.Nc + 255) / 256 * 256;
    int slab = XS_BUDGET / (2 * TB) / 256 * 256;
    if (slab > nc_pad) slab = nc_pad;
    p.slab_cols = slab;
    p.n_slabs = slab > 0 ? (nc_pad + slab - 1) / slab : 0;
    p.smem = (size_t)TB * p.n_out_pad * 2 + (size_t)TB * slab * 2 + (size_t)p.part_floats * 4 + 8 * 4 +
             (size_t)GL_WARPS * 8 * 4;
    p.ok = (long long)p.part_floats * 4 <= PART_BUDGET && p.smem <= 200 * 1024 && p.n_slabs > 0;
    return p;
}

template <int TB, int VV, bool RES, bool FUSED>
cudaError_t launch_kernel(const GlFmaParams &P, const GlFmaPlan &pl, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(decode_gl_fma_kernel<TB, VV, RES, FUSED>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    decode_gl_fma_kernel<TB, VV, RES, FUSED><<<pl.grid, GL_WARPS * 32, pl.smem, st>>>(P);
    return cudaGetLastError();
}

template <int TB, int VV>
cudaError_t launch_one(const GlFmaParams &P, const GlFmaPlan &pl, bool res, cudaStream_t st)
{
    const bool fused = P.n_layers > 1;
    if (res) return fused ? launch_kernel<TB, VV, true, true>(P, pl, st) : launch_kernel<TB, VV, true, false>(P, pl, st);
    return fused ? launch_kernel<TB, VV, false, true>(P, pl, st) : launch_kernel<TB, VV, false, false>(P, pl, st);
}

template <int TB>
cudaError_t launch_vv(const GlFmaParams &P, const GlFmaPlan &pl, int v, bool res, cudaStream_t st)
{
    if (v <= 8) return launch_one<TB, 8>(P, pl, res, st);
    if (v <= 12) return launch_one<TB, 12>(P, pl, res, st);
    return launch_one<TB, 16>(P, pl, res, st);
}

// several layers of the same format (apart from M) in one grid
bool plan_gl_fma_fused(const LayerView *Ls, int n, int TB, GlFmaPlan *out)
{
    if (n < 2 || n > MAX_FUSED) return false;
    for (int l = 1; l < n; l++)
        if (!same_geometry(Ls[0], Ls[l])) return false;
    GlFmaPlan p = plan_gl_fma(Ls[0], TB);
    if (!p.ok) return false;
    int R[MAX_FUSED], rows_cta = 0;
    for (int l = 0; l < n; l++) R[l] = Ls[l].R;
    if (!split_ctas(R, n, device_sm_count(), p.cta_begin, &rows_cta)) return false;
    p.grid = device_sm_count();
    p.smem -= (size_t)p.part_floats * 4;
    p.part_floats = rows_cta * TB * 16;
    p.smem += (size_t)p.part_floats * 4;
    if ((long long)p.part_floats * 4 > PART_BUDGET || p.smem > 200 * 1024) return false;
    *out = p;
    return true;
}

}  // namespace

bool gl_fma_supported(const LayerView &L, int B)
{
    if (B < 1 || B > 16) return false;
    if (L.Nc <= 0 || L.scale_rows) return false;
    if (L.v > 16 || (L.v & 1) || (L.n_out > 0 && L.v0 > 8)) return false;
    if (L.n_out > 2048) return false;
    return plan_gl_fma(L, gl_token_group(B)).ok;
}

int gl_fma_launches(const LayerView &L, int B)
{
    (void)L;
    const int TB = gl_token_group(B);
    return (B + TB - 1) / TB;
}

cudaError_t launch_decode_gl_fma(const LayerView &L, const void *x, int B, void *out, cudaStream_t st)
{
    const int TB = gl_token_group(B);
    const GlFmaPlan pl = plan_gl_fma(L, TB);
    const size_t xe = 2, oe = (L.out_dtype == VPTQ_DTYPE_FP32) ? 4 : 2;
    const bool res = L.k2 > 0;
    for (int t0 = 0; t0 < B; t0 += TB) {
        GlFmaParams P;
        memset(&P, 0, sizeof(P));
        P.L[0] = L; P.n_layers = 1; P.cta_begin[1] = pl.grid;
        P.B = (B - t0 < TB) ? (B - t0) : TB;
        P.x = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * L.N * xe;
        P.out[0] = reinterpret_cast<uint8_t *>(out) + (size_t)t0 * L.M * oe;
        P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs;
        P.n_out_pad = pl.n_out_pad; P.part_floats = pl.part_floats;
        cudaError_t e;
        if (TB == 4) e = launch_vv<4>(P, pl, L.v, res, st);
        else if (TB == 2) e = launch_vv<2>(P, pl, L.v, res, st);
        else e = launch_vv<1>(P, pl, L.v, res, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

bool gl_fma_fused_supported(const LayerView *Ls, int n, int B)
{
    for (int l = 0; l < n; l++)
        if (!gl_fma_supported(Ls[l], B)) return false;
    GlFmaPlan pl;
    return plan_gl_fma_fused(Ls, n, gl_token_group(B), &pl);
}

cudaError_t launch_decode_gl_fma_fused(const LayerView *Ls, int n, const void *x, int B, void *const *outs, cudaStream_t st)
{
    const int TB = gl_token_group(B);
    GlFmaPlan pl;
    if (!plan_gl_fma_fused(Ls, n, TB, &pl)) return cudaErrorInvalidValue;
    const bool res = Ls[0].k2 > 0;
    for (int t0 = 0; t0 < B; t0 += TB) {
        GlFmaParams P;
        memset(&P, 0, sizeof(P));
        for (int l = 0; l < n; l++) {
            P.L[l] = Ls[l];
            P.out[l] = reinterpret_cast<uint8_t *>(outs[l]) + (size_t)t0 * Ls[l].M * (Ls[l].out_dtype == VPTQ_DTYPE_FP32 ? 4 : 2);
        }
        for (int l = 0; l <= n; l++) P.cta_begin[l] = pl.cta_begin[l];
        P.n_layers = n;
        P.B = (B - t0 < TB) ? (B - t0) : TB;
        P.x = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * Ls[0].N * 2;
        P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs;
        P.n_out_pad = pl.n_out_pad; P.part_floats = pl.part_floats;
        cudaError_t e;
        if (TB == 4) e = launch_vv<4>(P, pl, Ls[0].v, res, st);
        else if (TB == 2) e = launch_vv<2>(P, pl, Ls[0].v, res, st);
        else e = launch_vv<1>(P, pl, Ls[0].v, res, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace vptq
