// Decode path for codebooks that fit shared memory (k1*16 B <= 128 KB, v <= 8), batch 1..8 per
// launch, FP32 FMAs.
//
// y[t][m] = sum_n x[t][n] * W_hat[m][n]   (App. D.2: lookup fused with the product; the FP16
// weight matrix is never formed).  With W_hat = s[n]*(C1[i1]+C2[i2]) + b[n] the scale folds
// into the activations and the bias into one scalar per token:
//     y[t][m] = sum_n (x[t][n]*s[n]) * (C1[i1][j] + C2[i2][j])  +  sum_n x[t][n]*b[n].
//
// Every index costs one 16-byte random read of shared memory (a3, a4); their rate (bank
// conflicts included) bounds the kernel, so it is organised like the L2-codebook kernel:
// persistent grid, one CTA per SM owning whole vector rows; the work is cut into (vector row,
// 256-column chunk) tasks and every warp owns an equal, contiguous range of them; per task a
// lane unpacks 8 consecutive indices of each stream (a1; the next task's packed words are
// already in flight), reads its 8 main centroids (rows padded to 16 bytes) and 8 residual
// centroids (table replicated 8 times with a 16-byte skew: conflict free), adds them in FP16
// and accumulates 8 x tokens products per output component.  The scaled activations x*s are
// staged per CTA as FP16, main columns and outlier columns apart.  Outlier columns (a5, Sec.
// 3.2.3) are a small pass of their own (centroids from global memory through L1).  Warp partial
// sums meet in shared memory; the epilogue adds the bias term and converts (a7).  No scratch.
#include "common.cuh"
#include "decode.cuh"
#include "index_words.cuh"
#include "fused_split.cuh"

namespace vptq {

namespace {

constexpr int XS_BUDGET = 96 * 1024;        // bytes of staged main-column activations per CTA
constexpr int PART_BUDGET = 16 * 1024;      // bytes of per-row partial sums per CTA
constexpr int SMEM_FMA_MAX_B = 4;

struct SmemFmaParams {
    LayerView L[MAX_FUSED];        // a fused launch: layer l is the work of CTAs [cta_begin[l], cta_begin[l + 1])
    void *out[MAX_FUSED];
    int cta_begin[MAX_FUSED + 1];
    int n_layers;
    const void *x;
    int B;                 // tokens in this launch (<= TB)
    int slab_cols;         // main columns per slab (multiple of 256)
    int n_slabs;
    int cb2_replicated;    // 1: [k2][8 replicas][16 B], 0: [k2][16 B]
    int n_out_pad;         // outlier columns rounded up to 8
    int part_floats;
};

__device__ __forceinline__ float2 h2f(uint32_t w)
{
    return __half22float2(*reinterpret_cast<__half2 *>(&w));
}

template <int TB, int VV, bool RES, int WARPS, bool FUSED>
__global__ void __launch_bounds__(WARPS * 32, 1)
decode_smem_fma_kernel(const __grid_constant__ SmemFmaParams P)
{
    constexpr int THREADS = WARPS * 32;
    extern __shared__ __align__(16) uint8_t smem[];
    pdl_launch_dependents();
    // the layer this CTA works on, and its place among that layer's CTAs
    int li = 0;
    if (FUSED)
        while (li + 1 < P.n_layers && (int)blockIdx.x >= P.cta_begin[li + 1]) li++;
    const LayerView &L = P.L[FUSED ? li : 0];
    void *const out = P.out[FUSED ? li : 0];
    const int bid = FUSED ? (int)blockIdx.x - P.cta_begin[li] : (int)blockIdx.x;
    const int gdim = FUSED ? P.cta_begin[li + 1] - P.cta_begin[li] : (int)gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint4 *cb1 = reinterpret_cast<uint4 *>(smem);                                            // [k1]
    uint4 *cb2 = cb1 + L.k1;                                                                 // [k2][rep]
    __half *xs_out = reinterpret_cast<__half *>(cb2 + (RES ? (size_t)L.k2 * (P.cb2_replicated ? 8 : 1) : 0));   // [TB][n_out_pad]
    __half *xs = xs_out + (size_t)TB * P.n_out_pad;                                          // [TB][slab_cols]
    float *part = reinterpret_cast<float *>(xs + (size_t)TB * P.slab_cols);                  // [rows][TB][8]
    float *bterm = part + P.part_floats;                                                     // [8]
    float *red = bterm + 8;                                                                  // [WARPS][8]

    // vector rows of this CTA, and the output rows they cover
    const int r0 = (int)((long long)L.R * bid / gdim);
    const int r1 = (int)((long long)L.R * (bid + 1) / gdim);
    const int m_lo = r0 * L.v;
    const int m_hi = min(L.M, r1 * L.v);

    // ---- a2: codebooks -> shared memory as 16-byte rows; clear the partial sums -------------------
    // (loads of 4 entries are issued before the first store: one L2 round trip per 4 entries, not per entry)
    for (int e0 = threadIdx.x; e0 < L.k1; e0 += 4 * THREADS) {
        uint4 row[4];
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (e0 + u * THREADS < L.k1) row[u] = load_centroid_row(L.c1, e0 + u * THREADS, L.v);
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (e0 + u * THREADS < L.k1) cb1[e0 + u * THREADS] = row[u];
    }
    if (RES) {
        const int n2 = P.cb2_replicated ? L.k2 * 8 : L.k2, sh = P.cb2_replicated ? 3 : 0;
        for (int i0 = threadIdx.x; i0 < n2; i0 += 4 * THREADS) {
            uint4 row[4];
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (i0 + u * THREADS < n2) row[u] = load_centroid_row(L.c2, (i0 + u * THREADS) >> sh, L.v);
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (i0 + u * THREADS < n2) cb2[i0 + u * THREADS] = row[u];
        }
    }
    for (int i = threadIdx.x; i < P.part_floats; i += THREADS) part[i] = 0.f;
    if (threadIdx.x < 8) bterm[threadIdx.x] = 0.f;

    const int rep = P.cb2_replicated ? (lane & 7) : 0;
    const int rshift = P.cb2_replicated ? 3 : 0;

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
        // (the activations may be the previous kernel's output: everything above read weights only)
        pdl_wait();
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
                                atomicAdd(part + ((rr - r0) * TB + t0 + t) * 8 + jj, a);
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
            const bool cur_live = 8 * ((c_begin >> 3) + cur_ch * 32 + lane) < c_end;
            // next task, and its packed words
            q++;
            if (++ch == chunks) { ch = 0; r++; }
            if (q < q_end) {
                const int grp = (c_begin >> 3) + ch * 32 + lane;
                raw1 = load_raw8(L.s1.ptr + (long long)r * L.s1.stride, L.s1.stride, grp, c_end, L.s1.bits);
                if (RES) raw2 = load_raw8(L.s2.ptr + (long long)r * L.s2.stride, L.s2.stride, grp, c_end, L.s2.bits);
            }
            if (cur_live) {
                // a3: 8 main centroids
                uint4 cw[8];
#pragma unroll
                for (int s = 0; s < 8; s++) cw[s] = cb1[(w1[s >> 1] >> (16 * (s & 1))) & 0xFFFFu];
                // this lane's 8 scaled activations per token
                uint4 xv4[TB];
#pragma unroll
                for (int t = 0; t < TB; t++)
                    xv4[t] = *reinterpret_cast<const uint4 *>(xs + t * P.slab_cols + cur_ch * 256 + lane * 8);
#pragma unroll
                for (int s = 0; s < 8; s++) {
                    uint4 w = cw[s];
                    if (RES) {
                        // a4: residual centroid, summed in FP16 (one rounding of 2^-11)
                        const uint32_t id2 = (w2[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                        const uint4 rv = cb2[(id2 << rshift) + rep];
                        __half2 a0 = __hadd2(*reinterpret_cast<__half2 *>(&w.x), *reinterpret_cast<const __half2 *>(&rv.x));
                        __half2 a1 = __hadd2(*reinterpret_cast<__half2 *>(&w.y), *reinterpret_cast<const __half2 *>(&rv.y));
                        w.x = *reinterpret_cast<uint32_t *>(&a0); w.y = *reinterpret_cast<uint32_t *>(&a1);
                        if (VV > 4) {
                            __half2 a2 = __hadd2(*reinterpret_cast<__half2 *>(&w.z), *reinterpret_cast<const __half2 *>(&rv.z));
                            w.z = *reinterpret_cast<uint32_t *>(&a2);
                        }
                        if (VV > 6) {
                            __half2 a3 = __hadd2(*reinterpret_cast<__half2 *>(&w.w), *reinterpret_cast<const __half2 *>(&rv.w));
                            w.w = *reinterpret_cast<uint32_t *>(&a3);
                        }
                    }
#pragma unroll
                    for (int t = 0; t < TB; t++) {
                        const uint32_t xw = (s >> 1) == 0 ? xv4[t].x : (s >> 1) == 1 ? xv4[t].y : (s >> 1) == 2 ? xv4[t].z : xv4[t].w;
                        fma_f16x2(acc[t][0], acc[t][1], xw, (s & 1) != 0, w.x);
                        fma_f16x2(acc[t][2], acc[t][3], xw, (s & 1) != 0, w.y);
                        if (VV > 4) fma_f16x2(acc[t][4], acc[t][VV > 4 ? 5 : 0], xw, (s & 1) != 0, w.z);
                        if (VV > 6) fma_f16x2(acc[t][VV > 6 ? 6 : 0], acc[t][VV > 6 ? 7 : 0], xw, (s & 1) != 0, w.w);
                    }
                }
            }
            if (q < q_end && r == cur_r) continue;

            // ---- row change (or end of range): halving butterfly over 8*TB values per lane ---------------
            constexpr int NV = 8 * TB;
            float v[NV];
#pragma unroll
            for (int t = 0; t < TB; t++)
#pragma unroll
                for (int j = 0; j < 8; j++) {
                    v[t * 8 + j] = j < VV ? acc[t][j < VV ? j : 0] : 0.f;
                    if (j < VV) acc[t][j] = 0.f;
                }
            const int vi = halving_butterfly<NV>(v, lane);     // index of the first value this lane ends up holding
            // NV >= 32: every lane holds NV/32 distinct values; NV < 32: lanes with the low bits clear
            constexpr int KEEP = NV >= 32 ? NV / 32 : 1;
            constexpr int dup = NV >= 32 ? 1 : 32 / NV;
            if ((lane & (dup - 1)) == 0) {
#pragma unroll
                for (int k = 0; k < KEEP; k++) {
                    const int idx = vi + k, t = idx >> 3, j = idx & 7;
                    if (j < VV) atomicAdd(part + ((cur_r - r0) * TB + t) * 8 + j, v[k]);
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
        const float y = part[((rr - r0) * TB + t) * 8 + jj] + bterm[t];
        store_out(out, (long long)t * L.M + m, y, L.out_dtype);
    }
}

struct SmemFmaPlan {
    int slab_cols, n_slabs, cb2_rep, grid, part_floats, n_out_pad, warps;
    size_t smem;
    bool ok;
    int cta_begin[MAX_FUSED + 1];   // fused launches only
};

int fma_token_group(int B) { return B >= 8 ? 8 : (B >= 4 ? 4 : (B >= 2 ? 2 : 1)); }

SmemFmaPlan plan_smem_fma(const LayerView &L, int TB)
{
    SmemFmaPlan p;
    p.warps = TB >= 4 ? 16 : 32;
    const int G = device_sm_count();
    p.grid = L.R < G ? L.R : G;
    const int rows_cta = ceil_div(L.R, p.grid);
    p.part_floats = rows_cta * TB * 8;
    p.n_out_pad = (L.n_out + 7) / 8 * 8;
    const int nc_pad = (L.Nc + 255) / 256 * 256;
    int slab = XS_BUDGET / (2 * TB) / 256 * 256;
    if (slab > nc_pad) slab = nc_pad;
    p.slab_cols = slab;
    p.n_slabs = slab > 0 ? (nc_pad + slab - 1) / slab : 0;
    p.cb2_rep = (L.k2 > 0 && L.k2 <= 256) ? 1 : 0;
    p.smem = (size_t)L.k1 * 16 + (size_t)L.k2 * 16 * (p.cb2_rep ? 8 : 1) + (size_t)TB * p.n_out_pad * 2 +
             (size_t)TB * slab * 2 + (size_t)p.part_floats * 4 + 8 * 4 + (size_t)p.warps * 8 * 4;
    p.ok = (long long)p.part_floats * 4 <= PART_BUDGET && p.smem <= 224 * 1024 && p.n_slabs > 0;
    return p;
}

template <int TB, int VV, bool RES, int WARPS, bool FUSED>
cudaError_t launch_kernel(const SmemFmaParams &P, const SmemFmaPlan &pl, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(decode_smem_fma_kernel<TB, VV, RES, WARPS, FUSED>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    return launch_dependent("smem_fma", decode_smem_fma_kernel<TB, VV, RES, WARPS, FUSED>, pl.grid, WARPS * 32, pl.smem, st, P);
}

template <int TB, int VV, int WARPS>
cudaError_t launch_one(const SmemFmaParams &P, const SmemFmaPlan &pl, bool res, cudaStream_t st)
{
    const bool fused = P.n_layers > 1;
    if (res) return fused ? launch_kernel<TB, VV, true, WARPS, true>(P, pl, st) : launch_kernel<TB, VV, true, WARPS, false>(P, pl, st);
    return fused ? launch_kernel<TB, VV, false, WARPS, true>(P, pl, st) : launch_kernel<TB, VV, false, WARPS, false>(P, pl, st);
}

// several layers of the same format (apart from M) in one grid
bool plan_smem_fma_fused(const LayerView *Ls, int n, int TB, SmemFmaPlan *out)
{
    if (n < 2 || n > MAX_FUSED) return false;
    for (int l = 1; l < n; l++)
        if (!same_geometry(Ls[0], Ls[l])) return false;
    SmemFmaPlan p = plan_smem_fma(Ls[0], TB);
    if (!p.ok) return false;
    int R[MAX_FUSED], rows_cta = 0;
    for (int l = 0; l < n; l++) R[l] = Ls[l].R;
    if (!split_ctas(R, n, device_sm_count(), p.cta_begin, &rows_cta)) return false;
    p.grid = device_sm_count();
    p.smem -= (size_t)p.part_floats * 4;
    p.part_floats = rows_cta * TB * 8;
    p.smem += (size_t)p.part_floats * 4;
    if ((long long)p.part_floats * 4 > PART_BUDGET || p.smem > 224 * 1024) return false;
    *out = p;
    return true;
}

template <int TB, int WARPS>
cudaError_t launch_vv(const SmemFmaParams &P, const SmemFmaPlan &pl, int v, bool res, cudaStream_t st)
{
    if (v <= 4) return launch_one<TB, 4, WARPS>(P, pl, res, st);
    if (v <= 6) return launch_one<TB, 6, WARPS>(P, pl, res, st);
    return launch_one<TB, 8, WARPS>(P, pl, res, st);
}

}  // namespace

bool smem_fma_supported(const LayerView &L, int B)
{
    if (L.G > 1) return false;          // one codebook pair per layer here
    if (B < 1 || B > SMEM_FMA_MAX_B) return false;     // beyond that the mma.sync kernel is faster
    if (L.Nc <= 0 || L.scale_rows) return false;
    if (L.v > 8 || (L.n_out > 0 && L.v0 > 8)) return false;
    if ((long long)L.k1 * 16 > 128 * 1024) return false;
    if (L.k2 && (long long)L.k2 * 16 > 32 * 1024) return false;
    if (L.n_out > 2048) return false;
    return plan_smem_fma(L, fma_token_group(B)).ok;
}

int smem_fma_launches(const LayerView &L, int B)
{
    (void)L;
    const int TB = fma_token_group(B);
    return (B + TB - 1) / TB;
}

cudaError_t launch_decode_smem_fma(const LayerView &L, const void *x, int B, void *out, cudaStream_t st)
{
    const int TB = fma_token_group(B);
    const SmemFmaPlan pl = plan_smem_fma(L, TB);
    const size_t xe = 2, oe = (L.out_dtype == VPTQ_DTYPE_FP32) ? 4 : 2;
    const bool res = L.k2 > 0;
    for (int t0 = 0; t0 < B; t0 += TB) {
        SmemFmaParams P;
        memset(&P, 0, sizeof(P));
        P.L[0] = L; P.n_layers = 1; P.cta_begin[1] = pl.grid;
        P.B = (B - t0 < TB) ? (B - t0) : TB;
        P.x = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * L.N * xe;
        P.out[0] = reinterpret_cast<uint8_t *>(out) + (size_t)t0 * L.M * oe;
        P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs; P.cb2_replicated = pl.cb2_rep;
        P.n_out_pad = pl.n_out_pad; P.part_floats = pl.part_floats;
        cudaError_t e;
        if (TB == 8) e = launch_vv<8, 16>(P, pl, L.v, res, st);
        else if (TB == 4) e = launch_vv<4, 16>(P, pl, L.v, res, st);
        else if (TB == 2) e = launch_vv<2, 32>(P, pl, L.v, res, st);
        else e = launch_vv<1, 32>(P, pl, L.v, res, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

bool smem_fma_fused_supported(const LayerView *Ls, int n, int B)
{
    for (int l = 0; l < n; l++)
        if (!smem_fma_supported(Ls[l], B)) return false;
    SmemFmaPlan pl;
    return plan_smem_fma_fused(Ls, n, fma_token_group(B), &pl);
}

cudaError_t launch_decode_smem_fma_fused(const LayerView *Ls, int n, const void *x, int B, void *const *outs, cudaStream_t st)
{
    const int TB = fma_token_group(B);
    SmemFmaPlan pl;
    if (!plan_smem_fma_fused(Ls, n, TB, &pl)) return cudaErrorInvalidValue;
    const bool res = Ls[0].k2 > 0;
    for (int t0 = 0; t0 < B; t0 += TB) {
        SmemFmaParams P;
        memset(&P, 0, sizeof(P));
        for (int l = 0; l < n; l++) {
            P.L[l] = Ls[l];
            P.out[l] = reinterpret_cast<uint8_t *>(outs[l]) + (size_t)t0 * Ls[l].M * (Ls[l].out_dtype == VPTQ_DTYPE_FP32 ? 4 : 2);
        }
        for (int l = 0; l <= n; l++) P.cta_begin[l] = pl.cta_begin[l];
        P.n_layers = n;
        P.B = (B - t0 < TB) ? (B - t0) : TB;
        P.x = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * Ls[0].N * 2;
        P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs; P.cb2_replicated = pl.cb2_rep;
        P.n_out_pad = pl.n_out_pad; P.part_floats = pl.part_floats;
        cudaError_t e;
        if (TB == 8) e = launch_vv<8, 16>(P, pl, Ls[0].v, res, st);
        else if (TB == 4) e = launch_vv<4, 16>(P, pl, Ls[0].v, res, st);
        else if (TB == 2) e = launch_vv<2, 32>(P, pl, Ls[0].v, res, st);
        else e = launch_vv<1, 32>(P, pl, Ls[0].v, res, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace vptq
