// Decode path for codebooks that fit shared memory (k1*16 B <= ~128 KB, v <= 8), batch 1..16.
//
// y[t][m] = sum_n x[t][n] * W_hat[m][n]   (App. D.2: lookup fused with the product; the FP16
// weight matrix is never formed).  With W_hat = s[n]*(C1[i1]+C2[i2]) + b[n] the scale folds
// into the activations and the bias into one scalar per token:
//     y[t][m] = sum_n (x[t][n]*s[n]) * (C1[i1][j] + C2[i2][j])  +  sum_n x[t][n]*b[n].
//
// One CTA per SM owns a contiguous range of vector rows and the whole input dimension.
// The codebooks sit in shared memory as 16-byte rows (shorter vectors are zero padded).
// A warp owns 256-column chunks.  For one chunk it keeps the (scaled) activations of up
// to 16 tokens in registers as mma A fragments, and for every vector row it
//   - reads 8 packed indices per lane with one vector load (a1: index unpack),
//   - lets every lane name one centroid row per step; ldmatrix.x4.trans gathers the 32
//     rows and hands them out directly in mma B-fragment order (a3/a4: lookups),
//   - issues mma.m16n8k16 (tokens x 8 outputs x 16 columns), main and residual codebook
//     into the same FP32 accumulator (the residual sum of Sec. 3.2.2 by linearity).
// The k order inside an mma is a fixed permutation of the columns (lane l, step s holds
// column 8*l+s), and the A fragments are built with the same permutation.
// Warp partial sums meet in shared memory; outlier columns (Sec. 3.2.3) are added by a small
// FP32 pass that gathers their centroids from global memory; the epilogue adds the bias
// term and converts.
#include "common.cuh"
#include "decode.cuh"
#include "index_words.cuh"

namespace vptq {

namespace {

constexpr int WARPS = 16;
constexpr int THREADS = WARPS * 32;
constexpr int CHUNK = 256;        // columns per warp chunk: 32 lanes x 8 indices

struct SmemMmaParams {
    LayerView L;
    const void *x;
    void *out;
    int B;
    int rows_per_cta;    // vector rows per CTA
    int rows_per_pass;   // vector rows whose partial sums fit the slot area
    int cb1_bytes, cb2_bytes;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Stage a codebook [k][v] fp16 (dense) into shared memory as [k][8] fp16, zero padded.  The loads of
// 4 entries are issued before the first store: one L2 round trip per 4 entries, not per entry.
__device__ void stage_codebook(const __half *__restrict__ src, int k, int v, __half *dst)
{
    uint4 *d4 = reinterpret_cast<uint4 *>(dst);
    for (int e0 = threadIdx.x; e0 < k; e0 += 4 * THREADS) {
        uint4 row[4];
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (e0 + u * THREADS < k) row[u] = load_centroid_row(src, e0 + u * THREADS, v);
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (e0 + u * THREADS < k) d4[e0 + u * THREADS] = row[u];
    }
}

// 16 consecutive 16-bit elements starting at element E of a buffer of `total` elements whose
// base is 16-byte aligned; elements at or beyond `total` read as zero.  Returns 8 words.
__device__ __forceinline__ void load16_elems(const uint16_t *__restrict__ base, long long E, long long total,
                                             uint32_t (&out)[8])
{
    const long long A0 = E & ~7LL;
    const int mis = (int)(E - A0);            // 0..7 elements
    uint32_t W[12];
#pragma unroll
    for (int i = 0; i < 3; i++) {
        long long off = A0 + 8 * i;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (off + 8 <= total) {
            q = __ldg(reinterpret_cast<const uint4 *>(base + off));
        } else if (off < total) {
            uint32_t tmp[4] = {0, 0, 0, 0};
            for (int e = 0; e < 8 && off + e < total; e++)
                tmp[e >> 1] |= (uint32_t)__ldg(base + off + e) << (16 * (e & 1));
            q = make_uint4(tmp[0], tmp[1], tmp[2], tmp[3]);
        }
        W[4 * i] = q.x; W[4 * i + 1] = q.y; W[4 * i + 2] = q.z; W[4 * i + 3] = q.w;
    }
    // shift left by `mis` elements: two word-granular conditional moves, then one half-word funnel
    if (mis & 4) {
#pragma unroll
        for (int i = 0; i < 10; i++) W[i] = W[i + 2];
    }
    if (mis & 2) {
#pragma unroll
        for (int i = 0; i < 9; i++) W[i] = W[i + 1];
    }
    if (mis & 1) {
#pragma unroll
        for (int i = 0; i < 8; i++) out[i] = __funnelshift_r(W[i], W[i + 1], 16);
    } else {
#pragma unroll
        for (int i = 0; i < 8; i++) out[i] = W[i];
    }
}

// 16 scaled activations (x*s, FP16) for token t, absolute columns [n0, n0+16); columns at or
// beyond n_end read as zero.
// (PERM: the layer has a stored column order; a template parameter so that the plain case keeps its
// loads free of branches and the compiler can issue them together)
template <bool PERM>
__device__ __forceinline__ void load_xs16(const SmemMmaParams &P, int t, int n0, int n_end, uint32_t (&hw)[8])
{
    const LayerView &L = P.L;
    uint32_t xw[8];
    if (PERM) {
        // a stored column order: the 16 activations are gathered one by one
        const uint16_t *xr = reinterpret_cast<const uint16_t *>(P.x) + (long long)t * L.N;
#pragma unroll
        for (int i = 0; i < 8; i++) {
            const uint32_t lo = n0 + 2 * i < n_end ? __ldg(xr + in_col(L, n0 + 2 * i)) : 0u;
            const uint32_t hi = n0 + 2 * i + 1 < n_end ? __ldg(xr + in_col(L, n0 + 2 * i + 1)) : 0u;
            xw[i] = lo | (hi << 16);
        }
    } else
    load16_elems(reinterpret_cast<const uint16_t *>(P.x), (long long)t * L.N + n0,
                 (long long)t * L.N + n_end, xw);
    const bool scaled = L.has_scale && !L.scale_rows;
    uint32_t sw[8];
    if (scaled) load16_elems(reinterpret_cast<const uint16_t *>(L.scale), n0, n_end, sw);
#pragma unroll
    for (int i = 0; i < 8; i++) {
        __half2 xv;
        if (L.x_bf16) {
            __nv_bfloat162 bv = *reinterpret_cast<__nv_bfloat162 *>(&xw[i]);
            xv = __float22half2_rn(__bfloat1622float2(bv));
        } else {
            xv = *reinterpret_cast<__half2 *>(&xw[i]);
        }
        if (scaled) {
            float2 xf = __half22float2(xv);
            float2 sf = __half22float2(*reinterpret_cast<__half2 *>(&sw[i]));
            xv = __floats2half2_rn(xf.x * sf.x, xf.y * sf.y);
        }
        hw[i] = *reinterpret_cast<uint32_t *>(&xv);
    }
}

template <int NT, bool PERM>   // NT = 1: up to 8 tokens, NT = 2: up to 16 tokens
__global__ void __launch_bounds__(THREADS, 1)
decode_smem_mma_kernel(SmemMmaParams P)
{
    extern __shared__ __align__(16) uint8_t smem[];
    const LayerView &L = P.L;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    constexpr int TP = 8 * NT;                 // token slots
    __half *cb1 = reinterpret_cast<__half *>(smem);
    __half *cb2 = reinterpret_cast<__half *>(smem + P.cb1_bytes);
    float *slots = reinterpret_cast<float *>(smem + P.cb1_bytes + P.cb2_bytes);     // [WARPS][rows_per_pass][TP][8]
    float *fin = slots + (size_t)WARPS * P.rows_per_pass * TP * 8;                  // [rows_per_pass*8][TP]
    float *tok = fin + (size_t)P.rows_per_pass * 8 * TP;                            // [TP] bias term / x sum
    float *red = tok + TP;                                                          // [WARPS][TP]

    const int r_begin = blockIdx.x * P.rows_per_cta;
    const int r_end = min(L.R, r_begin + P.rows_per_cta);
    if (r_begin >= r_end) return;

    // ---- a2: codebook staging ---------------------------------------------------------------
    if (L.Nc > 0) {
        stage_codebook(L.c1, L.k1, L.v, cb1);
        if (L.k2) stage_codebook(L.c2, L.k2, L.v, cb2);
    }

    // ---- per-token scalar: sum_n x*bias (or sum_n x for per-row scale) -------------------------
    {
        float acc[TP];
#pragma unroll
        for (int t = 0; t < TP; t++) acc[t] = 0.f;
        if (L.has_scale) {
#pragma unroll 4
            for (int n = threadIdx.x; n < L.N; n += THREADS) {
                float bn = L.scale_rows ? 1.f : __half2float(__ldg(L.bias + n));
#pragma unroll
                for (int t = 0; t < TP; t++)
                    if (t < P.B) acc[t] += load_act(P.x, (long long)t * L.N + (PERM ? in_col(L, n) : n), L.x_bf16) * bn;
            }
        }
#pragma unroll
        for (int t = 0; t < TP; t++) {
            float a = acc[t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0) red[warp * TP + t] = a;
        }
    }
    __syncthreads();
    if (threadIdx.x < TP) {
        float a = 0.f;
        for (int w = 0; w < WARPS; w++) a += red[w * TP + threadIdx.x];
        tok[threadIdx.x] = a;
    }

    const uint32_t cb1_addr = smem_u32(cb1), cb2_addr = smem_u32(cb2);
    const int n_chunks = (L.Nc + CHUNK - 1) / CHUNK;
    const int n_end = L.N;

    for (int p0 = r_begin; p0 < r_end; p0 += P.rows_per_pass) {
        const int p1 = min(r_end, p0 + P.rows_per_pass);
        const int nrows = p1 - p0;
        // zero this warp's slots (a warp with no chunk still contributes zeros)
        {
            float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            float4 *s4 = reinterpret_cast<float4 *>(slots + (size_t)warp * P.rows_per_pass * TP * 8);
            for (int i = lane; i < nrows * TP * 2; i += 32) s4[i] = z;
        }
        __syncwarp();

        for (int chunk = warp; chunk < n_chunks; chunk += WARPS) {
            const int cb = chunk * CHUNK;
            // ---- A fragments: scaled activations of this chunk, in the gather's column order ----
            uint32_t A[2][8][2 * NT];
#pragma unroll
            for (int f = 0; f < 2; f++) {
#pragma unroll
                for (int kb = 0; kb < 2; kb++) {
                    const int n0 = L.n_out + cb + 8 * (16 * f + 2 * q + 8 * kb);
#pragma unroll
                    for (int th = 0; th < NT; th++) {
                        const int t = g + 8 * th;
                        uint32_t hw[8];
                        if (t < P.B && n0 < n_end) {
                            load_xs16<PERM>(P, t, n0, n_end, hw);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; i++) hw[i] = 0u;
                        }
#pragma unroll
                        for (int s = 0; s < 8; s++)
                            A[f][s][NT * kb + th] = __byte_perm(hw[s >> 1], hw[4 + (s >> 1)], (s & 1) ? 0x7632 : 0x5410);
                    }
                }
            }
            // ---- rows ----------------------------------------------------------------------------
            const int grp = cb / 8 + lane;         // this lane's index group within a packed row
            const uint8_t *row1 = L.s1.ptr + (long long)p0 * L.s1.stride;
            const uint8_t *row2 = L.k2 ? L.s2.ptr + (long long)p0 * L.s2.stride : nullptr;
            // packed indices of the next PF rows are kept in flight: one row of compute is far shorter than
            // a DRAM round trip
            constexpr int PF = NT == 1 ? 4 : 1;          // 16 tokens leave no registers for more
            uint4 pre1[PF], pre2[PF];
#pragma unroll
            for (int i = 0; i < PF; i++) {
                pre1[i] = make_uint4(0, 0, 0, 0);
                pre2[i] = make_uint4(0, 0, 0, 0);
                if (i < nrows) {
                    pre1[i] = load_raw8(row1 + (long long)i * L.s1.stride, L.s1.stride, grp, L.Nc, L.s1.bits);
                    if (L.k2) pre2[i] = load_raw8(row2 + (long long)i * L.s2.stride, L.s2.stride, grp, L.Nc, L.s2.bits);
                }
            }
            for (int rl = 0; rl < nrows; rl++) {
                uint32_t w1[4], w2[4];
                decode8(pre1[0], L.s1.bits, L.k1, w1);
                if (L.k2) decode8(pre2[0], L.s2.bits, L.k2, w2);
#pragma unroll
                for (int i = 0; i + 1 < PF; i++) { pre1[i] = pre1[i + 1]; pre2[i] = pre2[i + 1]; }
                if (rl + PF < nrows) {
                    pre1[PF - 1] = load_raw8(row1 + (long long)(rl + PF) * L.s1.stride, L.s1.stride, grp, L.Nc, L.s1.bits);
                    if (L.k2) pre2[PF - 1] = load_raw8(row2 + (long long)(rl + PF) * L.s2.stride, L.s2.stride, grp, L.Nc, L.s2.bits);
                }
                float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int s = 0; s < 8; s++) {
                    const uint32_t i1 = (w1[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(cb1_addr + i1 * 16u, b0, b1, b2, b3);
                    if (NT == 2) {
                        mma16816(d, A[0][s][0], A[0][s][1], A[0][s][2], A[0][s][3], b0, b1);
                        mma16816(d, A[1][s][0], A[1][s][1], A[1][s][2], A[1][s][3], b2, b3);
                    } else {
                        mma16816(d, A[0][s][0], 0u, A[0][s][1], 0u, b0, b1);
                        mma16816(d, A[1][s][0], 0u, A[1][s][1], 0u, b2, b3);
                    }
                    if (L.k2) {
                        const uint32_t i2 = (w2[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                        ldmatrix_x4_trans(cb2_addr + i2 * 16u, b0, b1, b2, b3);
                        if (NT == 2) {
                            mma16816(d, A[0][s][0], A[0][s][1], A[0][s][2], A[0][s][3], b0, b1);
                            mma16816(d, A[1][s][0], A[1][s][1], A[1][s][2], A[1][s][3], b2, b3);
                        } else {
                            mma16816(d, A[0][s][0], 0u, A[0][s][1], 0u, b0, b1);
                            mma16816(d, A[1][s][0], 0u, A[1][s][1], 0u, b2, b3);
                        }
                    }
                }
                // accumulate into this warp's slot: [rl][token][j]
                float *sl = slots + (((size_t)warp * P.rows_per_pass + rl) * TP) * 8;
                float2 *p = reinterpret_cast<float2 *>(sl + g * 8 + 2 * q);
                float2 v = *p;
                v.x += d[0]; v.y += d[1];
                *p = v;
                if (NT == 2) {
                    float2 *p2 = reinterpret_cast<float2 *>(sl + (g + 8) * 8 + 2 * q);
                    float2 v2 = *p2;
                    v2.x += d[2]; v2.y += d[3];
                    *p2 = v2;
                }
            }
        }
        __syncthreads();

        // ---- reduce the warps' partial sums: fin[ml][t], ml = local output row ---------------------
        const int m_lo = p0 * L.v;
        const int m_hi = min(L.M, p1 * L.v);
        for (int i = threadIdx.x; i < nrows * TP * 8; i += THREADS) {
            const int j = i & 7, t = (i >> 3) % TP, rl = i / (8 * TP);
            float a = 0.f;
#pragma unroll
            for (int w = 0; w < WARPS; w++) a += slots[(((size_t)w * P.rows_per_pass + rl) * TP + t) * 8 + j];
            if (j < L.v) fin[(rl * L.v + j) * TP + t] = a;
        }
        __syncthreads();

        // ---- a5: outlier columns, FP32, centroids gathered from global memory ----------------------
        if (L.n_out > 0) {
            const int q_lo = m_lo / L.v0, q_hi = (m_hi + L.v0 - 1) / L.v0;
            const bool scaled = L.has_scale && !L.scale_rows;
            for (int qq = q_lo + warp; qq < q_hi; qq += WARPS) {
                const uint8_t *row0 = L.s0.ptr + (long long)qq * L.s0.stride;
                for (int t0 = 0; t0 < P.B; t0 += 4) {
                    float acc[8][4];
#pragma unroll
                    for (int j = 0; j < 8; j++)
#pragma unroll
                        for (int t = 0; t < 4; t++) acc[j][t] = 0.f;
                    for (int n = lane; n < L.n_out; n += 32) {
                        const int i0 = clamp_index(load_index(row0, n, L.s0.bits), L.k0);
                        const __half *e = L.c0 + (long long)i0 * L.v0;
                        float sc = scaled ? __half2float(__ldg(L.scale + n)) : 1.f;
                        float xv[4];
#pragma unroll
                        for (int t = 0; t < 4; t++)
                            xv[t] = (t0 + t < P.B) ? load_act(P.x, (long long)(t0 + t) * L.N + (PERM ? in_col(L, n) : n), L.x_bf16) * sc : 0.f;
#pragma unroll
                        for (int j = 0; j < 8; j++) {
                            if (j < L.v0) {
                                float wj = __half2float(__ldg(e + j));
#pragma unroll
                                for (int t = 0; t < 4; t++) acc[j][t] += xv[t] * wj;
                            }
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; j++) {
#pragma unroll
                        for (int t = 0; t < 4; t++) {
                            float a = acc[j][t];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                            const int m = qq * L.v0 + j;
                            if (lane == 0 && j < L.v0 && m >= m_lo && m < m_hi && t0 + t < P.B)
                                fin[(m - m_lo) * TP + t0 + t] += a;
                        }
                    }
                }
            }
            __syncthreads();
        }

        // ---- epilogue: bias term, conversion, store -------------------------------------------------
        const int n_m = m_hi - m_lo;
        for (int i = threadIdx.x; i < n_m * P.B; i += THREADS) {
            const int t = i / n_m, ml = i % n_m;      // consecutive threads -> consecutive m
            const int m = m_lo + ml;
            float y = fin[ml * TP + t];
            if (L.has_scale) {
                if (L.scale_rows) y = y * __half2float(__ldg(L.scale + m)) + __half2float(__ldg(L.bias + m)) * tok[t];
                else y += tok[t];
            }
            store_out(P.out, (long long)t * L.M + m, y, L.out_dtype);
        }
        __syncthreads();
    }
}

int pad16(int x) { return (x + 15) / 16 * 16; }

}  // namespace

bool smem_mma_supported(const LayerView &L, int B)
{
    if (L.G > 1) return false;          // one codebook pair per layer here
    if (B < 1 || B > 16) return false;
    if (L.v > 8 || (L.n_out > 0 && L.v0 > 8)) return false;
    if (L.Nc > 0 && (long long)L.k1 * 16 > 128 * 1024) return false;
    if (L.k2 && (long long)L.k2 * 16 > 32 * 1024) return false;
    return true;
}

namespace {
template <int NT>
cudaError_t launch_variant(const SmemMmaParams &P, bool perm, int grid, size_t smem, cudaStream_t st)
{
    cudaError_t e;
    if (perm) {
        e = cudaFuncSetAttribute(decode_smem_mma_kernel<NT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        decode_smem_mma_kernel<NT, true><<<grid, THREADS, smem, st>>>(P);
    } else {
        e = cudaFuncSetAttribute(decode_smem_mma_kernel<NT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        decode_smem_mma_kernel<NT, false><<<grid, THREADS, smem, st>>>(P);
    }
    return cudaGetLastError();
}
}  // namespace

long long smem_mma_workspace_bytes(const LayerView &L, int B)
{
    return smem_tc_supported(L, B) ? smem_tc_workspace_bytes(L, B) : 0;
}

cudaError_t launch_decode_smem_mma(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st)
{
    // the common kind of layer goes to the row-owner kernel with shared-memory A fragments; per-row scale and
    // all-outlier layers stay here
    if (smem_tc_supported(L, B)) return launch_decode_smem_tc(L, x, B, out, ws, st);
    SmemMmaParams P;
    P.L = L; P.x = x; P.out = out; P.B = B;
    const int NT = B <= 8 ? 1 : 2;
    const int TP = 8 * NT;
    P.cb1_bytes = L.Nc > 0 ? pad16(L.k1 * 16) : 0;
    P.cb2_bytes = L.k2 ? pad16(L.k2 * 16) : 0;
    const int sms = device_sm_count();
    P.rows_per_cta = ceil_div(L.R, sms);
    const int budget = 220 * 1024 - P.cb1_bytes - P.cb2_bytes - (TP + WARPS * TP) * 4;
    const int per_row = (WARPS * TP * 8 + 8 * TP) * 4;
    int rpp = budget / per_row;
    if (rpp < 1) return cudaErrorInvalidConfiguration;
    if (rpp > P.rows_per_cta) rpp = P.rows_per_cta;
    P.rows_per_pass = rpp;
    const int grid = ceil_div(L.R, P.rows_per_cta);
    const size_t smem = (size_t)P.cb1_bytes + P.cb2_bytes + (size_t)rpp * per_row + (TP + WARPS * TP) * 4;
    return NT == 1 ? launch_variant<1>(P, L.perm != nullptr, grid, smem, st)
                   : launch_variant<2>(P, L.perm != nullptr, grid, smem, st);
}

}  // namespace vptq
