// Decode path for codebooks that fit shared memory (k1*16 B <= 64 KB, v <= 8), batch 5..16, tensor cores,
// persistent row-owner grid.
//
// y[t][m] = sum_n (x[t][n]*s[n]) * (C1[i1][j] + C2[i2][j]) + sum_n x[t][n]*b[n]   (a3..a7; App. D.2: the
// lookup is fused with the product, the FP16 weight is never formed).
//
// What bounds it: every index costs one 16-byte shared-memory row (a3, a4), read by ldmatrix, whose 8x8
// matrices take about 3.5 wavefronts each with random rows.  Everything else is arranged so that nothing but
// those reads and the mma stand on the critical path:
//   - one CTA of 32 warps per SM owns whole vector rows; the work is cut into (vector row, 256-column chunk)
//     tasks and every warp owns an equal, contiguous range of them, the packed words of the next two tasks in
//     flight;
//   - the scaled activations of up to 16 tokens are staged per CTA and slab of columns in shared memory, ALREADY
//     IN mma A-FRAGMENT ORDER (one conflict-free 16-byte read per lane and mma), so a warp holds no activations
//     in registers and 32 warps fit; one gathered centroid fragment feeds all 16 tokens;
//   - per step a lane names one main and one residual centroid row; ldmatrix.x4.trans hands the 32 rows out in
//     B-fragment order; the residual fragment is added to the main one in FP16 (one rounding of 2^-11), the
//     residual table is replicated 8 times with a 16-byte skew (conflict free);
//   - two independent FP32 accumulators per warp; partial sums meet in shared memory when the warp's row changes.
// Outlier columns (a5) are a small FP32 pass over activations staged in shared memory.
// The legacy mma.sync form is deliberate: the B operand is a per-lane gather, not a tile TMA could fetch.
#include "common.cuh"
#include "decode.cuh"
#include "index_words.cuh"

namespace vptq {

namespace {

constexpr int TC_WARPS = 32, TC_THREADS = TC_WARPS * 32;
constexpr int TC_SMEM_BUDGET = 224 * 1024;

struct SmemTcParams {
    LayerView L;
    const void *x;
    void *out;
    int B;
    int slab_chunks;     // 256-column chunks per slab
    int n_slabs;
    int cb2_replicated;
    int n_out_pad;
    int rows_cta;        // most vector rows a CTA owns
    int chunks_total;    // 256-column chunks of the main region
    uint8_t *image;      // workspace: [chunks_total][16 steps*mma][32 lanes][FRAG] A fragments of x*s, then
                         // xs_out [TP][n_out_pad] fp16, then tok [TP] floats (written by the pre-pass)
};

__device__ __forceinline__ uint32_t tc_saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void tc_ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void tc_mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t tc_hadd2(uint32_t a, uint32_t b)
{
    const __half2 r = __hadd2(*reinterpret_cast<const __half2 *>(&a), *reinterpret_cast<const __half2 *>(&b));
    return *reinterpret_cast<const uint32_t *>(&r);
}
// Pre-pass (one small launch per call): x*s of all tokens as FP16, written once in the order in which the main
// kernel's mma instructions want their A fragments, so that every CTA fetches its slab with plain 16-byte
// copies instead of re-deriving it; the outlier columns' activations and the bias term sum_n x*b ride along.
// Element (token t, main column c): chunk c / 256, step s = c % 8, lane group l = (c % 256) / 8: mma f = l / 16,
// k = l % 16, quad (k % 8) / 2, half k % 2, register 2 * (k / 8) + t / 8 (NT = 2) or k / 8 (NT = 1), lane
// 4 * (t % 8) + quad.
template <int NT>
__global__ void __launch_bounds__(256)
smem_tc_prepass_kernel(const __grid_constant__ SmemTcParams P)
{
    pdl_launch_dependents();
    const LayerView &L = P.L;
    constexpr int TP = 8 * NT, FRAG = 8 * NT, CHUNK_BYTES = 16 * 32 * FRAG;
    __half *xs_out = reinterpret_cast<__half *>(P.image + (size_t)P.chunks_total * CHUNK_BYTES);
    float *tok = reinterpret_cast<float *>(xs_out + (size_t)TP * P.n_out_pad);
    pdl_wait();                                   // the activations may be the previous kernel's output
    const int n_pad = L.n_out + P.chunks_total * 256;            // stored columns, the last chunk filled up
    __shared__ float red[TP];
    if (threadIdx.x < TP) red[threadIdx.x] = 0.f;
    __syncthreads();
    const int t = threadIdx.x & 15;
    float bacc = 0.f;
    for (int n = blockIdx.x * (blockDim.x >> 4) + (threadIdx.x >> 4); n < n_pad; n += gridDim.x * (blockDim.x >> 4)) {
        if (t >= TP) continue;
        float xv = 0.f, sc = 1.f, bi = 0.f;
        if (n < L.N) {
            if (L.has_scale) { sc = __half2float(__ldg(L.scale + n)); bi = __half2float(__ldg(L.bias + n)); }
            if (t < P.B) xv = load_act(P.x, (long long)t * L.N + in_col(L, n), L.x_bf16);
        }
        bacc += xv * bi;
        const __half hv = __float2half_rn(xv * sc);
        if (n < L.n_out) { xs_out[t * P.n_out_pad + n] = hv; continue; }
        const int c = n - L.n_out, ch = c >> 8, l = (c & 255) >> 3, s = c & 7;
        const int f = l >> 4, k = l & 15, qq = (k & 7) >> 1, hf = k & 1;
        const int reg = NT == 2 ? 2 * (k >> 3) + (t >> 3) : (k >> 3);
        const int ln = 4 * (t & 7) + qq;
        *reinterpret_cast<__half *>(P.image + (size_t)ch * CHUNK_BYTES + ((s * 2 + f) * 32 + ln) * FRAG + reg * 4 + hf * 2) = hv;
    }
    if (t < TP) atomicAdd(&red[t], bacc);
    __syncthreads();
    if (threadIdx.x < TP) atomicAdd(tok + threadIdx.x, red[threadIdx.x]);      // tok is cleared by a memset in front
}

// NT = 1: up to 8 tokens (A fragments of 8 bytes per lane), NT = 2: up to 16 tokens (16 bytes per lane)
template <int NT, bool RES>
__global__ void __launch_bounds__(TC_THREADS, 1)
decode_smem_tc_kernel(const __grid_constant__ SmemTcParams P)
{
    extern __shared__ __align__(16) uint8_t smem[];
    pdl_launch_dependents();
    const LayerView &L = P.L;
    constexpr int TP = 8 * NT;
    constexpr int FRAG = 8 * NT;                                  // bytes of A fragment per lane and mma
    constexpr int CHUNK_BYTES = 16 * 32 * FRAG;                    // 8 steps x 2 mma x 32 lanes
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint4 *cb1 = reinterpret_cast<uint4 *>(smem);                                                        // [k1]
    uint4 *cb2 = cb1 + L.k1;                                                                             // [k2][rep]
    uint8_t *afrag = reinterpret_cast<uint8_t *>(cb2 + (RES ? (size_t)L.k2 * (P.cb2_replicated ? 8 : 1) : 0));   // [slab_chunks][16][32][FRAG]
    __half *xs_out = reinterpret_cast<__half *>(afrag + (size_t)P.slab_chunks * CHUNK_BYTES);            // [TP][n_out_pad]
    float *part = reinterpret_cast<float *>(xs_out + (size_t)TP * P.n_out_pad);                          // [rows_cta][TP][8]
    float *tok = part + (size_t)P.rows_cta * TP * 8;                                                     // [TP] bias term

    const int r0 = (int)((long long)L.R * blockIdx.x / gridDim.x);
    const int r1 = (int)((long long)L.R * (blockIdx.x + 1) / gridDim.x);
    const int m_lo = r0 * L.v, m_hi = min(L.M, r1 * L.v);

    // ---- a2: codebooks -> shared memory as 16-byte rows (4 entries per thread in flight); clear the sums ----
    for (int e0 = threadIdx.x; e0 < L.k1; e0 += 4 * TC_THREADS) {
        uint4 row[4];
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (e0 + u * TC_THREADS < L.k1) row[u] = load_centroid_row(L.c1, e0 + u * TC_THREADS, L.v);
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (e0 + u * TC_THREADS < L.k1) cb1[e0 + u * TC_THREADS] = row[u];
    }
    if (RES) {
        const int n2 = P.cb2_replicated ? L.k2 * 8 : L.k2, sh = P.cb2_replicated ? 3 : 0;
        for (int i = threadIdx.x; i < n2; i += TC_THREADS) cb2[i] = load_centroid_row(L.c2, i >> sh, L.v);
    }
    for (int i = threadIdx.x; i < P.rows_cta * TP * 8; i += TC_THREADS) part[i] = 0.f;
    if (threadIdx.x < TP) tok[threadIdx.x] = 0.f;

    const uint32_t cb1_addr = tc_saddr(cb1);
    const uint32_t cb2_lane = tc_saddr(cb2) + (P.cb2_replicated ? (uint32_t)(lane & 7) * 16u : 0u);
    const uint32_t cb2_shift = P.cb2_replicated ? 7u : 4u;       // bytes per residual entry: 128 (8 copies) or 16
    const uint32_t afrag_lane = tc_saddr(afrag) + (uint32_t)lane * FRAG;
    const int g = lane >> 2, q = lane & 3;

    // the activations may be the previous kernel's output: everything above read weights only
    pdl_wait();
    __syncthreads();

    const __half *img_xs_out = reinterpret_cast<const __half *>(P.image + (size_t)P.chunks_total * CHUNK_BYTES);
    const float *img_tok = reinterpret_cast<const float *>(img_xs_out + (size_t)TP * P.n_out_pad);
    for (int slab = 0; slab < P.n_slabs; slab++) {
        const int c_begin = slab * P.slab_chunks * 256;                 // main-region columns of the slab
        const int c_end = min(L.Nc, c_begin + P.slab_chunks * 256);
        const int chunks = (c_end - c_begin + 255) >> 8;

        // ---- this warp's task range: (row, chunk of the slab), chunk fastest; packed words of its first tasks ----
        const int n_tasks = (r1 - r0) * chunks;
        int tq = (int)((long long)n_tasks * warp / TC_WARPS);
        const int tq_end = (int)((long long)n_tasks * (warp + 1) / TC_WARPS);
        int r_cur = r0 + (chunks ? tq / chunks : 0), ch_cur = chunks ? tq % chunks : 0;     // task tq
        int r_nxt = r_cur, ch_nxt = ch_cur;                                                    // task to load next
        uint4 raw1[2], raw2[2];
#pragma unroll
        for (int d = 0; d < 2; d++) {
            raw1[d] = make_uint4(0, 0, 0, 0); raw2[d] = make_uint4(0, 0, 0, 0);
            if (tq + d < tq_end) {
                const int grp = (c_begin >> 3) + ch_nxt * 32 + lane;
                raw1[d] = load_raw8(L.s1.ptr + (long long)r_nxt * L.s1.stride, L.s1.stride, grp, c_end, L.s1.bits);
                if (RES) raw2[d] = load_raw8(L.s2.ptr + (long long)r_nxt * L.s2.stride, L.s2.stride, grp, c_end, L.s2.bits);
                if (++ch_nxt == chunks) { ch_nxt = 0; r_nxt++; }
            }
        }

        // ---- a6: the slab's A fragments (written by the pre-pass) -> shared memory; slab 0 also takes the outlier
        // columns' activations and the bias term ----
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(P.image + (size_t)slab * P.slab_chunks * CHUNK_BYTES);
            uint4 *dst = reinterpret_cast<uint4 *>(afrag);
            const int n16 = chunks * (CHUNK_BYTES / 16);
            for (int i0 = threadIdx.x; i0 < n16; i0 += 4 * TC_THREADS) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; u++)
                    if (i0 + u * TC_THREADS < n16) v[u] = __ldg(src + i0 + u * TC_THREADS);
#pragma unroll
                for (int u = 0; u < 4; u++)
                    if (i0 + u * TC_THREADS < n16) dst[i0 + u * TC_THREADS] = v[u];
            }
            if (slab == 0) {
                for (int i = threadIdx.x; i < TP * P.n_out_pad; i += TC_THREADS) xs_out[i] = img_xs_out[i];
                if (threadIdx.x < TP) tok[threadIdx.x] = img_tok[threadIdx.x];
            }
        }
        __syncthreads();

        // ---- a5: outlier columns (slab 0 only): FP32.  A warp takes one outlier vector row at a time; 32 columns'
        // indices and centroids are fetched by one lane each (two dependent memory round trips for 32 columns),
        // then broadcast column by column; lane (t, j) owns output component j of token t, so nothing is reduced. ----
        if (slab == 0 && L.n_out > 0) {
            const int q_lo = m_lo / L.v0, q_hi = (m_hi + L.v0 - 1) / L.v0;
            const int ot = lane >> 2, oj = lane & 3;                 // token (and token + 8), components oj and oj + 4
            for (int qq = q_lo + warp; qq < q_hi; qq += TC_WARPS) {
                const uint8_t *row0 = L.s0.ptr + (long long)qq * L.s0.stride;
                float o00 = 0.f, o01 = 0.f, o10 = 0.f, o11 = 0.f;    // [token half][component half]
                for (int nb = 0; nb < L.n_out; nb += 32) {
                    uint4 cw = make_uint4(0, 0, 0, 0);
                    if (nb + lane < L.n_out)
                        cw = load_centroid_row(L.c0, clamp_index(load_index(row0, nb + lane, L.s0.bits), L.k0), L.v0);
                    const int cols = min(32, L.n_out - nb);
                    for (int c = 0; c < cols; c++) {
                        // component oj sits in word oj / 2 (half oj % 2), component oj + 4 two words further
                        const uint32_t wx = __shfl_sync(0xffffffffu, cw.x, c), wy = __shfl_sync(0xffffffffu, cw.y, c);
                        uint32_t wz = 0u, ww = 0u;
                        if (L.v0 > 4) { wz = __shfl_sync(0xffffffffu, cw.z, c); ww = __shfl_sync(0xffffffffu, cw.w, c); }
                        const uint32_t lo = (oj & 2) ? wy : wx, hi = (oj & 2) ? ww : wz;
                        const float2 flo = __half22float2(*reinterpret_cast<const __half2 *>(&lo));
                        const float2 fhi = __half22float2(*reinterpret_cast<const __half2 *>(&hi));
                        const float w0 = (oj & 1) ? flo.y : flo.x, w1 = (oj & 1) ? fhi.y : fhi.x;
                        const float x0 = __half2float(xs_out[ot * P.n_out_pad + nb + c]);
                        o00 += x0 * w0; o01 += x0 * w1;
                        if (NT == 2) {
                            const float x1 = __half2float(xs_out[(ot + 8) * P.n_out_pad + nb + c]);
                            o10 += x1 * w0; o11 += x1 * w1;
                        }
                    }
                }
                const int m0 = qq * L.v0 + oj, m1 = m0 + 4;
                if (oj < L.v0 && m0 >= m_lo && m0 < m_hi) {
                    const int rr = m0 / L.v, jj = m0 - rr * L.v;
                    atomicAdd(part + ((rr - r0) * TP + ot) * 8 + jj, o00);
                    if (NT == 2) atomicAdd(part + ((rr - r0) * TP + ot + 8) * 8 + jj, o10);
                }
                if (oj + 4 < L.v0 && m1 >= m_lo && m1 < m_hi) {
                    const int rr = m1 / L.v, jj = m1 - rr * L.v;
                    atomicAdd(part + ((rr - r0) * TP + ot) * 8 + jj, o01);
                    if (NT == 2) atomicAdd(part + ((rr - r0) * TP + ot + 8) * 8 + jj, o11);
                }
            }
        }

        // ---- main tasks (a3, a4, a7) ----
        float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
        int cur_r = -1;
        auto flush = [&]() {
            if (cur_r < 0) return;
            // this lane holds tokens g (and g + 8), output components 2q, 2q+1
            float *p = part + ((cur_r - r0) * TP + g) * 8 + 2 * q;
            atomicAdd(p, d0[0] + d1[0]);
            atomicAdd(p + 1, d0[1] + d1[1]);
            if (NT == 2) {
                atomicAdd(p + 64, d0[2] + d1[2]);
                atomicAdd(p + 65, d0[3] + d1[3]);
            }
#pragma unroll
            for (int i = 0; i < 4; i++) { d0[i] = 0.f; d1[i] = 0.f; }
        };
        while (tq < tq_end) {
#pragma unroll
            for (int dd = 0; dd < 2; dd++) {
                if (tq < tq_end) {
                    uint32_t w1[4], w2[4] = {0, 0, 0, 0};
                    decode8(raw1[dd], L.s1.bits, L.k1, w1);
                    if (RES) decode8(raw2[dd], L.s2.bits, L.k2, w2);
                    const int r = r_cur, ch = ch_cur;
                    if (++ch_cur == chunks) { ch_cur = 0; r_cur++; }
                    if (tq + 2 < tq_end) {
                        const int grp = (c_begin >> 3) + ch_nxt * 32 + lane;
                        raw1[dd] = load_raw8(L.s1.ptr + (long long)r_nxt * L.s1.stride, L.s1.stride, grp, c_end, L.s1.bits);
                        if (RES) raw2[dd] = load_raw8(L.s2.ptr + (long long)r_nxt * L.s2.stride, L.s2.stride, grp, c_end, L.s2.bits);
                        if (++ch_nxt == chunks) { ch_nxt = 0; r_nxt++; }
                    }
                    if (r != cur_r) { flush(); cur_r = r; }
                    const uint32_t a_base = afrag_lane + (uint32_t)ch * CHUNK_BYTES;
#pragma unroll
                    for (int s = 0; s < 8; s++) {
                        const uint32_t i1 = (w1[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                        uint32_t b0, b1, b2, b3;
                        tc_ldmatrix_x4_trans(cb1_addr + i1 * 16u, b0, b1, b2, b3);
                        if (RES) {
                            const uint32_t i2 = (w2[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                            uint32_t q0, q1, q2, q3;
                            tc_ldmatrix_x4_trans(cb2_lane + (i2 << cb2_shift), q0, q1, q2, q3);
                            b0 = tc_hadd2(b0, q0); b1 = tc_hadd2(b1, q1); b2 = tc_hadd2(b2, q2); b3 = tc_hadd2(b3, q3);
                        }
                        if (NT == 2) {
                            uint4 a0, a1;
                            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a0.x), "=r"(a0.y), "=r"(a0.z), "=r"(a0.w) : "r"(a_base + (uint32_t)(s * 2) * 32u * FRAG));
                            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a1.x), "=r"(a1.y), "=r"(a1.z), "=r"(a1.w) : "r"(a_base + (uint32_t)(s * 2 + 1) * 32u * FRAG));
                            tc_mma16816(d0, a0.x, a0.y, a0.z, a0.w, b0, b1);
                            tc_mma16816(d1, a1.x, a1.y, a1.z, a1.w, b2, b3);
                        } else {
                            uint2 a0, a1;
                            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(a0.x), "=r"(a0.y) : "r"(a_base + (uint32_t)(s * 2) * 32u * FRAG));
                            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(a1.x), "=r"(a1.y) : "r"(a_base + (uint32_t)(s * 2 + 1) * 32u * FRAG));
                            tc_mma16816(d0, a0.x, 0u, a0.y, 0u, b0, b1);
                            tc_mma16816(d1, a1.x, 0u, a1.y, 0u, b2, b3);
                        }
                    }
                    tq++;
                }
            }
        }
        flush();
        __syncthreads();      // the slab's fragments are dead; part[] complete after the last slab
    }

    // ---- bias term, conversion, store ----
    const int n_m = m_hi - m_lo;
    for (int i = threadIdx.x; i < n_m * P.B; i += TC_THREADS) {
        const int t = i / n_m, ml = i % n_m;
        const int m = m_lo + ml;
        const int rr = m / L.v, jj = m - rr * L.v;
        store_out(P.out, (long long)t * L.M + m, part[((rr - r0) * TP + t) * 8 + jj] + tok[t], L.out_dtype);
    }
}

struct SmemTcPlan {
    int slab_chunks, n_slabs, cb2_rep, n_out_pad, rows_cta, grid, chunks_total;
    size_t smem;
    long long ws_bytes, ws_clear_from;      // the workspace image; bytes [ws_clear_from, ws_bytes) start at zero
    bool ok;
};

SmemTcPlan plan_smem_tc(const LayerView &L, int NT)
{
    SmemTcPlan p;
    const int TP = 8 * NT;
    const int G = device_sm_count();
    p.grid = L.R < G ? L.R : G;
    p.rows_cta = ceil_div(L.R, p.grid);
    p.n_out_pad = (L.n_out + 7) / 8 * 8;
    p.cb2_rep = (L.k2 > 0 && L.k2 <= 256) ? 1 : 0;
    const long long fixed = (long long)L.k1 * 16 + (long long)L.k2 * 16 * (p.cb2_rep ? 8 : 1) + (long long)TP * p.n_out_pad * 2 +
                            (long long)p.rows_cta * TP * 8 * 4 + TP * 4 + 64;
    const int chunk_bytes = 16 * 32 * 8 * NT;
    const int n_chunks = (L.Nc + 255) / 256;
    long long room = (TC_SMEM_BUDGET - fixed) / chunk_bytes;
    if (room > n_chunks) room = n_chunks;
    p.ok = room >= 1;
    if (!p.ok) room = 1;
    p.n_slabs = ceil_div(n_chunks, (int)room);
    p.slab_chunks = ceil_div(n_chunks, p.n_slabs);            // equal slabs
    p.smem = (size_t)(fixed + (long long)p.slab_chunks * chunk_bytes);
    p.chunks_total = n_chunks;
    p.ws_clear_from = (long long)n_chunks * chunk_bytes + (long long)TP * p.n_out_pad * 2;
    p.ws_bytes = (p.ws_clear_from + TP * 4 + 255) / 256 * 256;
    return p;
}

}  // namespace

// layers of the common kind: main columns present, per-input-column scale or none, tables that leave room for the
// activations; everything else stays with the register-fragment kernel
bool smem_tc_supported(const LayerView &L, int B)
{
    if (L.G > 1 || B < 1 || B > 16) return false;
    if (L.Nc <= 0 || L.scale_rows) return false;
    if (L.v > 8 || (L.n_out > 0 && L.v0 > 8)) return false;
    if ((long long)L.k1 * 16 > 64 * 1024) return false;
    if (L.k2 && (long long)L.k2 * 16 > 16 * 1024) return false;
    if (L.n_out > 1024) return false;
    return plan_smem_tc(L, B <= 8 ? 1 : 2).ok;
}

long long smem_tc_workspace_bytes(const LayerView &L, int B)
{
    return plan_smem_tc(L, B <= 8 ? 1 : 2).ws_bytes;
}

cudaError_t launch_decode_smem_tc(const LayerView &L, const void *x, int B, void *out, void *ws, cudaStream_t st)
{
    const int NT = B <= 8 ? 1 : 2;
    const SmemTcPlan pl = plan_smem_tc(L, NT);
    SmemTcParams P;
    memset(&P, 0, sizeof(P));
    P.L = L; P.x = x; P.out = out; P.B = B;
    P.slab_chunks = pl.slab_chunks; P.n_slabs = pl.n_slabs; P.cb2_replicated = pl.cb2_rep;
    P.n_out_pad = pl.n_out_pad; P.rows_cta = pl.rows_cta;
    P.chunks_total = pl.chunks_total;
    P.image = reinterpret_cast<uint8_t *>(ws);
    const bool res = L.k2 > 0;
    // the bias terms are summed up by atomics: they start at zero
    cudaError_t e = cudaMemsetAsync(P.image + pl.ws_clear_from, 0, (size_t)(pl.ws_bytes - pl.ws_clear_from), st);
    if (e != cudaSuccess) return e;
    const int pre_grid = (L.n_out + pl.chunks_total * 256 + 15) / 16;
    if (NT == 2) smem_tc_prepass_kernel<2><<<pre_grid, 256, 0, st>>>(P);
    else smem_tc_prepass_kernel<1><<<pre_grid, 256, 0, st>>>(P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (NT == 2) {
        auto kern = res ? decode_smem_tc_kernel<2, true> : decode_smem_tc_kernel<2, false>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
        if (e != cudaSuccess) return e;
        return launch_dependent("smem_tc", kern, pl.grid, TC_THREADS, pl.smem, st, P);
    }
    auto kern = res ? decode_smem_tc_kernel<1, true> : decode_smem_tc_kernel<1, false>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    return launch_dependent("smem_tc", kern, pl.grid, TC_THREADS, pl.smem, st, P);
}

}  // namespace vptq
