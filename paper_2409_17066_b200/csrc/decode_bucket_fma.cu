// Decode path over a PREPARED layer image (format text: include/vptq.h), batch 1.
//
// The canonical decode of a 65536-entry codebook pays one random 16-byte read out of L2 per index, and the
// rate of those reads bounds it (about one per clock and SM).  Here the (main, residual) index pairs of a
// CTA's vector rows arrive bucket by bucket (a bucket = 4096 consecutive main-codebook entries, 64 KB), so
// the CTA keeps the bucket's slice of the codebook in shared memory and every centroid read is a
// conflict-free shared-memory read (App. C.2's argument: lookups are fast while the table fits the
// first-level memory).  Per CTA:
//   - one producer lane streams the 16 slices through two 64 KB buffers with linear bulk copies (no
//     multicast), full/empty mbarriers, every wait bounded;
//   - 31 consumer warps walk their own contiguous run of blocks (four steps of 32 lanes, one 16-byte load
//     per lane and block, three blocks in flight); a quarter warp (8 lanes, one per residue of the main
//     index mod 8, hence 8 different banks) works on one vector row at a time, sums 8 output components per
//     lane and folds them with a three-stage butterfly when its row changes;
//   - an entry is one word: 9 bits of main index, 8 bits of residual index, 15 bits of column; the scaled
//     activation x*s is looked up in shared memory by column (a6 folded into x, bias as one scalar);
//   - products are f16 x f16 accumulated in f32 by the mixed-precision fma of sm_100.
// Shared memory is addressed absolutely so that a table address is (field & mask) | base: the buffers sit at
// 64 KB and 128 KB of the CTA's window, the replicated residual table at 192 KB, the activations below.
#include "common.cuh"
#include "prepared.cuh"
#include "fused_split.cuh"
#include "index_words.cuh"

namespace vptq {

namespace {

constexpr int BK_WARPS = PREP_WARPS + 1, BK_THREADS = BK_WARPS * 32;
constexpr int BK_DEPTH = 2;                                  // blocks in flight per warp
// absolute shared-memory addresses (the window starts with 1 KB the system keeps and the static variables)
constexpr uint32_t XS_ABS = 2048, TAB_ABS = 65536, CB2_ABS = 196608, PART_ABS = CB2_ABS + 32768,
                   RED_ABS = PART_ABS + 64 * 8 * 4, END_ABS = RED_ABS + BK_WARPS * 4;
static_assert(XS_ABS + 2 * (PREP_MAX_N + PREP_PAD_COLS) <= TAB_ABS, "activations must end below the first bucket buffer");
constexpr unsigned long long WAIT_LIMIT_CYCLES = 4000000000ull;      // about two seconds

struct BucketParams {
    LayerView L[MAX_FUSED];
    const uint8_t *image[MAX_FUSED];
    void *out[MAX_FUSED];
    int cta_begin[MAX_FUSED + 1];
    int n_split[MAX_FUSED];            // CTAs that share a group of vector rows, each with a range of buckets
    int n_layers;
    const void *x;
    int *status;                       // may be null; only ever written on an error (the caller clears it)
    int *arrived;                      // [grid] one arrival counter per row group (at its first CTA), zero between launches
    float *slots;                      // [grid][64 * 8] partial sums of a CTA whose row group is split
    unsigned long long wait_limit;     // cycles a device-side wait may take
};

__device__ __forceinline__ uint32_t saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred P1;\n\tmbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\tselp.b32 %0, 1, 0, P1;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when it was abandoned (limit reached here, or the abort flag raised by another waiter).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                          unsigned long long limit)
{
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if ((++spins & 63u) == 0 || limit < 4096ull) {      // a short (test) limit is looked at on every poll
            if (*abort_flag) return false;
            if ((unsigned long long)(clock64() - t0) > limit) {
                *abort_flag = 1;
                if (status) atomicExch(status, VPTQ_E_TIMEOUT);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 lds16(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
// acc[2i] += x * lo(w_i), acc[2i+1] += x * hi(w_i) when `live`: the f16 x f16 product is exact in f32, one
// rounding per fma (fma.rn.f32.f16: f16 factors, f32 addend and result)
__device__ __forceinline__ void fma8(float (&a)[8], uint16_t xh, const uint4 &w, bool live)
{
    asm("{\n\t.reg .b16 l0, h0, l1, h1, l2, h2, l3, h3;\n\t.reg .pred p;\n\tsetp.ne.u32 p, %13, 0;\n\t"
        "mov.b32 {l0, h0}, %9;\n\tmov.b32 {l1, h1}, %10;\n\tmov.b32 {l2, h2}, %11;\n\tmov.b32 {l3, h3}, %12;\n\t"
        "@p fma.rn.f32.f16 %0, %8, l0, %0;\n\t@p fma.rn.f32.f16 %1, %8, h0, %1;\n\t"
        "@p fma.rn.f32.f16 %2, %8, l1, %2;\n\t@p fma.rn.f32.f16 %3, %8, h1, %3;\n\t"
        "@p fma.rn.f32.f16 %4, %8, l2, %4;\n\t@p fma.rn.f32.f16 %5, %8, h2, %5;\n\t"
        "@p fma.rn.f32.f16 %6, %8, l3, %6;\n\t@p fma.rn.f32.f16 %7, %8, h3, %7;\n\t}"
        : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7])
        : "h"(xh), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w), "r"((uint32_t)live));
}

template <bool RES>
__device__ __forceinline__ void slot(uint32_t e, uint32_t pad, uint32_t tab_lane, uint32_t cb2_lane, float (&acc)[8])
{
    uint4 w = lds16(((e << 7) & 0xFF80u) | tab_lane);
    uint16_t xh;
    asm volatile("ld.shared.u16 %0, [%1 + 2048];" : "=h"(xh) : "r"((e >> 16) & 0xFFFEu));
    if (RES) {
        const uint4 rv = lds16(((e >> 2) & 0x7F80u) | cb2_lane);
        __half2 a0 = __hadd2(*reinterpret_cast<__half2 *>(&w.x), *reinterpret_cast<const __half2 *>(&rv.x));
        __half2 a1 = __hadd2(*reinterpret_cast<__half2 *>(&w.y), *reinterpret_cast<const __half2 *>(&rv.y));
        __half2 a2 = __hadd2(*reinterpret_cast<__half2 *>(&w.z), *reinterpret_cast<const __half2 *>(&rv.z));
        __half2 a3 = __hadd2(*reinterpret_cast<__half2 *>(&w.w), *reinterpret_cast<const __half2 *>(&rv.w));
        w.x = *reinterpret_cast<uint32_t *>(&a0); w.y = *reinterpret_cast<uint32_t *>(&a1);
        w.z = *reinterpret_cast<uint32_t *>(&a2); w.w = *reinterpret_cast<uint32_t *>(&a3);
    }
    // a padding entry names a column >= N; it must add nothing even when its table row holds an infinity
    fma8(acc, xh, w, e < pad);
}

// Outlier columns (Sec. 3.2.3: the first n_out stored columns, vectors of v0 rows, codebook c0) of the vector rows
// [r0, r1): their few indices come from the canonical stream, the centroids from global memory, products in
// FP32; every consumer warp takes the outlier rows warp, warp + 31, ...  Sums go to part[row][8].
__device__ __noinline__ void outlier_columns(const LayerView &L, const __half *xs, float *part, int r0, int r1, int warp, int lane)
{
    const int m_lo = r0 * L.v, m_hi = min(L.M, r1 * L.v);
    const int q_lo = m_lo / L.v0, q_hi = (m_hi + L.v0 - 1) / L.v0;
    for (int qq = q_lo + warp; qq < q_hi; qq += PREP_WARPS) {
        const uint8_t *row0 = L.s0.ptr + (long long)qq * L.s0.stride;
        float oacc[8];
#pragma unroll
        for (int j = 0; j < 8; j++) oacc[j] = 0.f;
        for (int n = lane; n < L.n_out; n += 32) {
            const int i0 = clamp_index(load_index(row0, n, L.s0.bits), L.k0);
            const uint4 cw = load_centroid_row(L.c0, i0, L.v0);
            const float2 c01 = __half22float2(*reinterpret_cast<const __half2 *>(&cw.x)), c23 = __half22float2(*reinterpret_cast<const __half2 *>(&cw.y)),
                         c45 = __half22float2(*reinterpret_cast<const __half2 *>(&cw.z)), c67 = __half22float2(*reinterpret_cast<const __half2 *>(&cw.w));
            const float cj[8] = {c01.x, c01.y, c23.x, c23.y, c45.x, c45.y, c67.x, c67.y};
            const float xv = __half2float(xs[n]);
#pragma unroll
            for (int j = 0; j < 8; j++) oacc[j] += xv * cj[j];
        }
#pragma unroll
        for (int j = 0; j < 8; j++) {
            float a = oacc[j];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            const int m = qq * L.v0 + j;
            if (lane == 0 && j < L.v0 && m >= m_lo && m < m_hi) {
                const int rr = m / L.v, jj = m - rr * L.v;
                atomicAdd(part + (rr - r0) * 8 + jj, a);
            }
        }
    }
}

template <bool RES>
__global__ void __launch_bounds__(BK_THREADS, 1)
decode_bucket_fma_kernel(const __grid_constant__ BucketParams P)
{
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t full[2], empty[2];
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // the next kernel of the stream may start its own prologue as soon as SMs free up
    pdl_launch_dependents();

    int li = 0;
    while (li + 1 < P.n_layers && (int)blockIdx.x >= P.cta_begin[li + 1]) li++;
    const LayerView &L = P.L[li];
    const int part_id = (int)blockIdx.x - P.cta_begin[li];
    const int n_parts = P.cta_begin[li + 1] - P.cta_begin[li];
    const uint8_t *img = P.image[li];

    // ---- checks that every thread of the grid answers alike: the shared-memory window and the image header ----
    const uint32_t base = saddr(smem);
    uint32_t dyn;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    const uint32_t *head = reinterpret_cast<const uint32_t *>(img);
    const int all_buckets = (L.k1 + PREP_BUCKET - 1) / PREP_BUCKET;
    const int n_split = P.n_split[li];           // the host derived it from R, k1 and n_parts by the format's rule
    const bool bad = base > XS_ABS || base + dyn < END_ABS ||
                     __ldg(head + 0) != VPTQ_PREPARED_MAGIC || __ldg(head + 1) != 2u || __ldg(head + 2) != (uint32_t)L.M ||
                     __ldg(head + 3) != (uint32_t)L.N || __ldg(head + 4) != (uint32_t)L.k1 || __ldg(head + 5) != (uint32_t)L.k2 ||
                     __ldg(head + 6) != (uint32_t)n_parts || __ldg(head + 7) != (uint32_t)PREP_WARPS ||
                     __ldg(head + 8) != (uint32_t)all_buckets || __ldg(head + 15) != (uint32_t)n_split ||
                     __ldg(head + 16) != (uint32_t)L.v || __ldg(head + 17) != (uint32_t)L.n_out ||
                     n_split < 1 || n_parts % n_split != 0 || n_split > all_buckets ||
                     (L.R + n_parts / n_split - 1) / (n_parts / n_split) > PREP_MAX_ROWS ||
                     (n_split > 1 && (P.arrived == nullptr || P.slots == nullptr)) ||
                     (L.v != 8 && all_buckets != 1) || L.v > 8 || (L.n_out > 0 && L.v0 > 8);
    if (bad) {
        if (threadIdx.x == 0 && P.status) atomicExch(P.status, VPTQ_E_UNSUPPORTED);
        return;
    }
    const uint32_t *woff = reinterpret_cast<const uint32_t *>(img + __ldg(head + 10));
    const uint32_t *hdr = reinterpret_cast<const uint32_t *>(img + __ldg(head + 11));
    const uint4 *entries = reinterpret_cast<const uint4 *>(img + __ldg(head + 12));
    const uint32_t n_blocks = __ldg(head + 9);

    uint8_t *const abs0 = smem - base;                                    // generic pointer of shared address 0
    __half *xs = reinterpret_cast<__half *>(abs0 + XS_ABS);               // [N + 64]
    uint4 *cb2 = reinterpret_cast<uint4 *>(abs0 + CB2_ABS);               // [256][8 replicas]
    float *part = reinterpret_cast<float *>(abs0 + PART_ABS);             // [64][8]
    float *red = reinterpret_cast<float *>(abs0 + RED_ABS);               // [BK_WARPS]
    const PreparedPart pp = prepared_part(L.R, all_buckets, n_parts, n_split, part_id);
    const int r0 = pp.r0, r1 = pp.r1;
    const int b_first = pp.b0, n_buckets = pp.b1 - pp.b0;     // buckets are counted from the partition's first from here on

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; i++) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(saddr(&full[i])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(saddr(&empty[i])), "r"(PREP_WARPS) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        abort_flag = 0;
    }
    __syncthreads();
    // the first two buckets are on their way while the rest of the prologue runs (16-byte rows, v = 8, go by
    // bulk copy; shorter vectors are widened to 16-byte rows by all threads, one bucket at a time)
    const bool bulk = L.v == 8;
    if (bulk && warp == PREP_WARPS && lane == 0) {
        for (int b = 0; b < 2 && b < n_buckets; b++) {
            const uint32_t rows = (uint32_t)min(PREP_BUCKET, L.k1 - (b_first + b) * PREP_BUCKET);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(saddr(&full[b])), "r"(rows * 16u) : "memory");
            for (uint32_t q = 0; q < rows; q += 1024)
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(TAB_ABS + (uint32_t)b * 65536u + q * 16u),
                               "l"(reinterpret_cast<const uint4 *>(L.c1) + (size_t)(b_first + b) * PREP_BUCKET + q),
                               "r"(min(rows - q, 1024u) * 16u), "r"(saddr(&full[b])) : "memory");
        }
    }
    // residual table, eight copies with a 16-byte skew (a4); partial sums
    if (RES)
        for (int i = threadIdx.x; i < L.k2 * 8; i += BK_THREADS) cb2[i] = load_centroid_row(L.c2, i >> 3, L.v);
    if (!bulk) {
        // a layer of short vectors has one bucket (k1 <= 4096), widened to 16-byte rows here
        uint4 *tab0 = reinterpret_cast<uint4 *>(abs0 + TAB_ABS);
        const int rows = min(PREP_BUCKET, L.k1 - b_first * PREP_BUCKET);
        for (int i = threadIdx.x; i < rows; i += BK_THREADS) tab0[i] = load_centroid_row(L.c1, b_first * PREP_BUCKET + i, L.v);
    }
    for (int i = threadIdx.x; i < 64 * 8; i += BK_THREADS) part[i] = 0.f;

    // consumer warps: the first blocks of the run are in flight before the activations are touched (a header
    // word counts its bucket from the partition's first)
    auto load_hdr = [&](const uint32_t *p) { return __ldg(p); };
    int q = 0, qe = 0;
    uint4 eb[BK_DEPTH];
    uint32_t hb[BK_DEPTH];
    if (warp < PREP_WARPS) {
        q = (int)__ldg(woff + part_id * PREP_WARPS + warp);
        qe = (int)__ldg(woff + part_id * PREP_WARPS + warp + 1);
        if ((uint32_t)qe > n_blocks) qe = (int)n_blocks;             // a corrupt table never leads out of the image
        if (q > qe) q = qe;
#pragma unroll
        for (int d = 0; d < BK_DEPTH; d++) {
            eb[d] = make_uint4(0, 0, 0, 0); hb[d] = 0xFFFFFFu;
            if (q + d < qe) { eb[d] = ld_stream16(entries + (size_t)(q + d) * 32 + lane); hb[d] = load_hdr(hdr + q + d); }
        }
    }

    // ---- a6: x*s as FP16 by stored column, bias term sum_n x*b; the activations are the previous kernel's ----
    pdl_wait();
    {
        float bacc = 0.f;
        if ((L.N & 7) == 0 && L.perm == nullptr) {
            for (int n = 8 * threadIdx.x; n < L.N; n += 8 * BK_THREADS) {
                const uint4 xq = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(P.x) + n));
                uint4 sq = make_uint4(0, 0, 0, 0), bq = make_uint4(0, 0, 0, 0);
                if (L.has_scale) {
                    sq = __ldg(reinterpret_cast<const uint4 *>(L.scale + n));
                    bq = __ldg(reinterpret_cast<const uint4 *>(L.bias + n));
                }
                const uint32_t xw[4] = {xq.x, xq.y, xq.z, xq.w}, sw[4] = {sq.x, sq.y, sq.z, sq.w}, bw[4] = {bq.x, bq.y, bq.z, bq.w};
                uint32_t pk[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    float2 xv;
                    if (L.x_bf16) xv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&xw[i]));
                    else xv = __half22float2(*reinterpret_cast<const __half2 *>(&xw[i]));
                    float2 sc = make_float2(1.f, 1.f), bi = make_float2(0.f, 0.f);
                    if (L.has_scale) {
                        sc = __half22float2(*reinterpret_cast<const __half2 *>(&sw[i]));
                        bi = __half22float2(*reinterpret_cast<const __half2 *>(&bw[i]));
                    }
                    const __half2 h = __floats2half2_rn(xv.x * sc.x, xv.y * sc.y);
                    pk[i] = *reinterpret_cast<const uint32_t *>(&h);
                    bacc += xv.x * bi.x + xv.y * bi.y;
                }
                *reinterpret_cast<uint4 *>(xs + n) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        } else {
            for (int n = threadIdx.x; n < L.N; n += BK_THREADS) {
                float sc = 1.f, bi = 0.f;
                if (L.has_scale) { sc = __half2float(__ldg(L.scale + n)); bi = __half2float(__ldg(L.bias + n)); }
                const float xv = load_act(P.x, in_col(L, n), L.x_bf16);
                xs[n] = __float2half_rn(xv * sc);
                bacc += xv * bi;
            }
        }
        // columns N .. N+63 mean "no entry": a zero in every bank, so that the lanes without an entry can all
        // read one word whose bank no other lane of the step uses
        if (threadIdx.x < PREP_PAD_COLS) xs[L.N + threadIdx.x] = __float2half_rn(0.f);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bacc += __shfl_xor_sync(0xffffffffu, bacc, o);
        if (lane == 0) red[warp] = bacc;
    }
    __syncthreads();

    if (warp == PREP_WARPS) {
        // ---- producer: bucket b into buffer b & 1 once every consumer warp has left bucket b - 2 ----
        if (lane == 0) {
            if (!bulk) mbar_arrive(saddr(&full[0]));          // the one bucket was written by all threads above
            bool ok = true;
            int b_stop = min(2, n_buckets);          // buckets issued so far
            for (int b = 2; b < n_buckets && ok; b++) {
                ok = mbar_wait(saddr(&empty[b & 1]), ((b >> 1) - 1) & 1, &abort_flag, P.status, P.wait_limit);
                if (!ok) break;
                b_stop = b + 1;
                const uint32_t rows = (uint32_t)min(PREP_BUCKET, L.k1 - (b_first + b) * PREP_BUCKET);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(saddr(&full[b & 1])), "r"(rows * 16u) : "memory");
                for (uint32_t qq = 0; qq < rows; qq += 1024)
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(TAB_ABS + (uint32_t)(b & 1) * 65536u + qq * 16u),
                                   "l"(reinterpret_cast<const uint4 *>(L.c1) + (size_t)(b_first + b) * PREP_BUCKET + qq),
                                   "r"(min(rows - qq, 1024u) * 16u), "r"(saddr(&full[b & 1])) : "memory");
            }
            // whatever was issued has landed before the CTA ends (bounded): the latest phase of both barriers
            const int issued = ok ? n_buckets : b_stop;
            for (int b = max(0, issued - 2); b < issued; b++) {
                const long long t0 = clock64();
                while (!mbar_try(saddr(&full[b & 1]), (b >> 1) & 1))
                    if ((unsigned long long)(clock64() - t0) > WAIT_LIMIT_CYCLES) break;      // never the shortened test limit
            }
        }
    } else {
        // the row group's outlier columns, once (the partition of its first bucket range)
        if (L.n_out > 0 && part_id % n_split == 0) outlier_columns(L, xs, part, r0, r1, warp, lane);
        const uint32_t rep16 = (uint32_t)(lane & 7) * 16u;
        const uint32_t cb2_lane = CB2_ABS | rep16;
        uint32_t tab_lane = TAB_ABS | rep16;
        const uint32_t pad = (uint32_t)L.N << 17;
        const uint32_t qmask = 0xFFu << (lane & 24);
        // the quarter's row field of a header word, compared in place: all six bits set = no row
        const uint32_t row_mask = 63u << (6 * (lane >> 3));
        uint32_t cur_field = row_mask;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; j++) acc[j] = 0.f;
        int cur_b = -1;
        bool ok = true;

        // the quarter warp's 8 sums per lane -> one output component per lane -> partial sums of the CTA
        auto flush = [&]() {
            if (cur_field == row_mask) {             // no row, or one outside the partition: whatever was summed is dropped
#pragma unroll
                for (int j = 0; j < 8; j++) acc[j] = 0.f;
                return;
            }
            const int cur_row = (int)(cur_field >> (6 * (lane >> 3)));
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; j++) { v[j] = acc[j]; acc[j] = 0.f; }
#pragma unroll
            for (int o = 4, h = 4; o > 0; o >>= 1, h >>= 1) {
                const bool up = (lane & o) != 0;
#pragma unroll
                for (int k = 0; k < 4; k++)
                    if (k < h) {
                        const float send = up ? v[k] : v[k + h], keep = up ? v[k + h] : v[k];
                        v[k] = keep + __shfl_xor_sync(qmask, send, o);
                    }
            }
            atomicAdd(part + cur_row * 8 + (lane & 7), v[0]);
            cur_field = row_mask;
        };
        // every warp visits every bucket in order: wait for it, work, hand its buffer back
        auto enter = [&](int b) {
            while (cur_b < b && ok) {
                if (cur_b >= 0) { __syncwarp(); if (lane == 0) mbar_arrive(saddr(&empty[cur_b & 1])); }
                cur_b++;
                ok = mbar_wait(saddr(&full[cur_b & 1]), (cur_b >> 1) & 1, &abort_flag, P.status, P.wait_limit);
                ok = __all_sync(0xffffffffu, ok);        // one lane giving up ends the warp's work
            }
            tab_lane = (TAB_ABS + (uint32_t)(cur_b & 1) * 65536u) | rep16;
            if (!ok) qe = 0;                              // a wait that gave up ends the warp's run
        };
        uint32_t last_h = 0xFFFFFFFFu;       // no header word has bucket 255 and four idle quarters at once
        // One block: its four entries per lane and its header word are in the registers of slot d; the slot is
        // refilled with the block two ahead at once (the image ends with two spare blocks, so that this needs no
        // bound check: what is fetched beyond the run is never used).
        auto block = [&](const int d) {
            const uint32_t e[4] = {eb[d].x, eb[d].y, eb[d].z, eb[d].w};
            const uint32_t h = hb[d];
            eb[d] = ld_stream16(entries + (size_t)(q + d + BK_DEPTH) * 32 + lane);
            hb[d] = load_hdr(hdr + q + d + BK_DEPTH);
            // most blocks repeat the header word of the one before (same bucket, same rows): nothing to decide then
            if (h != last_h) {
                last_h = h;
                const int b = min((int)(h >> 24), n_buckets - 1);
                if (b > cur_b) {
                    __syncwarp();
                    enter(b);
                    if (!ok) return;
                }
                const uint32_t field = h & row_mask;
                if (field != row_mask && field != cur_field) {
                    flush();
                    // a row outside the partition is ignored
                    cur_field = (int)(field >> (6 * (lane >> 3))) < r1 - r0 ? field : row_mask;
                }
            }
            // a quarter without a row holds entries that name no column: they add nothing, so nobody branches
#pragma unroll
            for (int s = 0; s < 4; s++) slot<RES>(e[s], pad, tab_lane, cb2_lane, acc);
            __syncwarp();
        };
        static_assert(BK_DEPTH == 2, "the loop below takes the blocks in pairs");
        while (q + 1 < qe) {
            block(0);
            block(1);
            q += 2;
        }
        if (q < qe) block(0);
        flush();
        __syncwarp();
        if (ok) enter(n_buckets - 1);                 // the buckets this warp had no blocks in
        if (ok && cur_b >= 0) { __syncwarp(); if (lane == 0) mbar_arrive(saddr(&empty[cur_b & 1])); }
    }
    __syncthreads();

    // ---- bias term, conversion, store (a7 epilogue) ----
    float bterm = 0.f;
    for (int w = 0; w < BK_WARPS; w++) bterm += red[w];
    const int m_lo = r0 * L.v, n_m = min(L.M, r1 * L.v) - m_lo;
    const int vv = L.v;
    if (n_split == 1) {
        for (int i = threadIdx.x; i < n_m; i += BK_THREADS)
            store_out(P.out[li], (long long)m_lo + i, part[(i / vv) * 8 + i % vv] + bterm, L.out_dtype);
        return;
    }
    // The row group's other CTAs hold the sums over their buckets.  Every CTA leaves its sums in its slot and
    // counts itself in; the one that finds all others counted adds the slots up, in slot order whoever it is,
    // and stores.  Nobody waits for anybody, and the counter is back at zero for the next launch.
    const int first_cta = (int)blockIdx.x - part_id % n_split;             // the row group's first CTA
    float *mine = P.slots + (size_t)blockIdx.x * (64 * 8);
    const int n_part = (r1 - r0) * 8;
    for (int i = threadIdx.x; i < n_part; i += BK_THREADS) mine[i] = part[i];
    __threadfence();
    __syncthreads();
    __shared__ int is_last;
    if (threadIdx.x == 0) {
        const int before = atomicAdd(P.arrived + first_cta, 1);
        is_last = before == n_split - 1;
        if (is_last) atomicExch(P.arrived + first_cta, 0);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int i = threadIdx.x; i < n_m; i += BK_THREADS) {
        float y = 0.f;
        for (int h = 0; h < n_split; h++) y += __ldcg(P.slots + (size_t)(first_cta + h) * (64 * 8) + (i / vv) * 8 + i % vv);
        store_out(P.out[li], (long long)m_lo + i, y + bterm, L.out_dtype);
    }
}

size_t bucket_smem_bytes() { return END_ABS - 1024 - 128; }      // dynamic part: the window starts with 1 KB + the static variables

}  // namespace

bool bucket_fma_supported(const LayerView &L, int B)
{
    return B == 1 && prepared_eligible(L);
}

size_t bucket_fma_workspace_bytes(const LayerView *Ls, const int *n_parts, int n)
{
    int grid = 0;
    bool split = false;
    for (int l = 0; l < n; l++) {
        grid += n_parts[l];
        split = split || prepared_split(Ls[l].R, ceil_div(Ls[l].k1, PREP_BUCKET), n_parts[l]) > 1;
    }
    if (!split) return 256;
    return 256 + (size_t)align256(4ull * (unsigned long long)grid) + (size_t)grid * 64 * 8 * 4;
}

cudaError_t launch_decode_bucket_fma(const LayerView *Ls, const void *const *images, const int *n_parts, int n,
                                     const void *x, void *const *outs, void *workspace, unsigned long long wait_limit,
                                     cudaStream_t st)
{
    if (n < 1 || n > MAX_FUSED) return cudaErrorInvalidValue;
    BucketParams P;
    memset(&P, 0, sizeof(P));
    int grid = 0;
    for (int l = 0; l < n; l++) {
        P.L[l] = Ls[l];
        P.image[l] = reinterpret_cast<const uint8_t *>(images[l]);
        P.out[l] = outs[l];
        P.cta_begin[l] = grid;
        P.n_split[l] = prepared_split(Ls[l].R, ceil_div(Ls[l].k1, PREP_BUCKET), n_parts[l]);
        grid += n_parts[l];
    }
    P.cta_begin[n] = grid;
    P.n_layers = n;
    P.x = x;
    P.status = reinterpret_cast<int *>(workspace);
    if (workspace && bucket_fma_workspace_bytes(Ls, n_parts, n) > 256) {
        P.arrived = reinterpret_cast<int *>(reinterpret_cast<uint8_t *>(workspace) + 256);
        P.slots = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(workspace) + 256 + align256(4ull * (unsigned long long)grid));
    }
    P.wait_limit = wait_limit ? wait_limit : WAIT_LIMIT_CYCLES;
    const bool res = Ls[0].k2 > 0;
    const size_t smem = bucket_smem_bytes();
    auto kern = res ? decode_bucket_fma_kernel<true> : decode_bucket_fma_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // programmatic dependent launch: the prologue (barriers, tables, first blocks) runs under the previous kernel's tail
    return launch_dependent("bucket", kern, grid, BK_THREADS, smem, st, P);
}

}  // namespace vptq
