// Decode path for a main codebook too large for shared memory (k1 = 65536, v = 8: 1 MiB),
// batch 1..4 per launch.
//
// The codebook stays in global memory and is served by L2; every index costs one 16-byte random
// read (a3), and the rate of those reads (about one L1-missing request per clock per SM), not
// HBM, bounds the kernel.  It is therefore organised around keeping every SM's read path busy
// all the time:
//   - persistent grid, one CTA per SM; the work is cut into (vector row, 256-column chunk) tasks
//     and every warp owns an equal, contiguous range of them;
//   - per task a lane takes 8 consecutive indices with one 128-bit load (a1; the next task's
//     indices are already in flight), issues its 8 centroid reads back to back and only then
//     consumes them;
//   - the residual codebook (a4) sits in shared memory, replicated 8 times with a 16-byte skew
//     so that the 8 lanes of a quarter warp always hit different banks;
//   - the scaled activations x*s (a6 folded into x) are staged per CTA in shared memory as FP16;
//     the bias becomes one scalar per token.
// A warp accumulates in registers while its tasks stay in one vector row and reduces the 8*B
// partial sums with a halving butterfly at a row change.  Two ways to combine the warps (a7):
//   OWNER    a CTA owns whole vector rows: partial sums meet in shared memory, no scratch;
//            used when the rows divide well over the SMs;
//   balanced tasks are dealt out regardless of rows: partial sums meet in an FP32 scratch array
//            through atomic adds, and a task counter per block of 16 vector rows tells which warp
//            completed the block and so converts and stores it.
// Fused launch (FUSED): up to MAX_FUSED layers that read the same activations (q/k/v, gate/up) in one
// OWNER-mode grid; the CTAs are dealt out to the layers in proportion to their vector rows and each
// CTA works on one layer exactly as in a launch of its own.  Small layers no longer pay a launch,
// a prologue and a ragged tail each.
#include "common.cuh"
#include "decode.cuh"
#include "index_words.cuh"
#include "fused_split.cuh"

namespace vptq {

namespace {

constexpr int RB_ROWS = 16;                 // vector rows per completion counter (balanced mode)
constexpr int XS_BUDGET = 64 * 1024;        // bytes of staged activations per CTA
constexpr int PART_BUDGET = 32 * 1024;      // bytes of per-row partial sums per CTA (OWNER mode)
constexpr int WARPS_TB4 = 16;               // 4 tokens per launch need 128 registers per thread

struct L2FmaParams {
    LayerView L[MAX_FUSED];
    void *out[MAX_FUSED];
    int cta_begin[MAX_FUSED + 1];   // FUSED: layer l is the work of CTAs [cta_begin[l], cta_begin[l + 1])
    int n_layers;
    const void *x;
    int B;                 // tokens in this launch (<= TB)
    int slab_cols;         // columns per slab (multiple of 256); one slab of x*s is staged at a time
    int n_slabs;
    int chunks_total;      // 256-column chunks of a whole row
    int cb2_replicated;    // 1: [k2][8 replicas][16 B], 0: [k2][16 B]
    int part_floats;       // OWNER: floats of the per-row partial sums
    int det;               // OWNER: warp partial sums are kept apart and added in warp order (no atomics)
    int rows_cta;          // OWNER: most vector rows a CTA owns
    float *yacc;           // balanced: [B][M] scratch, zero on entry
    unsigned *counters;    // balanced: [ceil(R / RB_ROWS)] scratch, zero on entry
};

// streaming 128-/64-bit loads of the packed index rows: read once, keep them out of L1
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_stream8(const void *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// 8 consecutive activations (fp16 or bf16 bits in a uint4) -> floats
__device__ __forceinline__ void act8_to_float(uint4 q, int is_bf16, float (&f)[8])
{
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {
        float2 p;
        if (is_bf16) p = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w[i]));
        else p = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        f[2 * i] = p.x; f[2 * i + 1] = p.y;
    }
}

template <int TB, bool RES, bool OWNER, int WARPS, bool FUSED>
__global__ void __launch_bounds__(WARPS * 32, 1)
decode_l2_fma_kernel(const __grid_constant__ L2FmaParams P)
{
    static_assert(!FUSED || OWNER, "a fused launch hands whole vector rows to CTAs");
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

    __half *xs = reinterpret_cast<__half *>(smem);                                   // [TB][slab_cols]
    float *bterm = reinterpret_cast<float *>(smem + (size_t)TB * P.slab_cols * 2);   // [4]
    float *red = bterm + 4;                                                          // [WARPS][4]
    uint4 *cb2 = reinterpret_cast<uint4 *>(red + WARPS * 4);
    float *part = reinterpret_cast<float *>(cb2 + (RES ? (size_t)L.k2 * (P.cb2_replicated ? 8 : 1) : 0));
    float *slots = part + P.part_floats;         // det: [rows_cta + WARPS][TB * 8], slot (row - r0) + warp

    // rows of this CTA (OWNER) / rank among the CTAs of its slab (balanced)
    const int r0 = OWNER ? (int)((long long)L.R * bid / gdim) : 0;
    const int r1 = OWNER ? (int)((long long)L.R * (bid + 1) / gdim) : L.R;
    const int my_slab = OWNER ? 0 : bid % P.n_slabs;
    const int grank = OWNER ? 0 : bid / P.n_slabs;
    const int gsize = OWNER ? 1 : (gdim - my_slab + P.n_slabs - 1) / P.n_slabs;

    // ---- residual codebook -> shared memory; clear the partial sums -----------------------------------
    if (RES) {
        const uint4 *src = reinterpret_cast<const uint4 *>(L.c2);
        if (P.cb2_replicated) {
            for (int i = threadIdx.x; i < L.k2 * 8; i += THREADS) cb2[i] = __ldg(src + (i >> 3));
        } else {
            for (int i = threadIdx.x; i < L.k2; i += THREADS) cb2[i] = __ldg(src + i);
        }
    }
    if (OWNER)
        for (int i = threadIdx.x; i < P.part_floats; i += THREADS) part[i] = 0.f;
    if (threadIdx.x < 4) bterm[threadIdx.x] = 0.f;

    const uint4 *cb1 = reinterpret_cast<const uint4 *>(L.c1);
    const int rep = P.cb2_replicated ? (lane & 7) : 0;
    const int rshift = P.cb2_replicated ? 3 : 0;
    const uint32_t kmax1 = (uint32_t)(L.k1 - 1), kmax2 = RES ? (uint32_t)(L.k2 - 1) : 0u;

    for (int slab = my_slab; slab < (OWNER ? P.n_slabs : my_slab + 1); slab++) {
        const int c_begin = slab * P.slab_cols;
        const int c_end = min(L.N, c_begin + P.slab_cols);
        const int chunks = (c_end - c_begin + 255) >> 8;
        // bias term: over this slab (OWNER walks all slabs) or over all columns (balanced: one slab per CTA)
        const int b_begin = OWNER ? c_begin : 0, b_end = OWNER ? c_end : L.N;

        // ---- this warp's task range: tasks are (row, chunk of the slab), chunk fastest ----------------
        const long long n_tasks = (long long)(r1 - r0) * chunks;
        const long long n_workers = (long long)gsize * WARPS;
        const long long wrank = (long long)grank * WARPS + warp;
        long long q = n_tasks * wrank / n_workers;
        const long long q_end = n_tasks * (wrank + 1) / n_workers;

        int r = r0 + (int)(q / chunks), ch = (int)(q % chunks);
        // packed indices of the first task (a lane's 8 columns: c_begin + 256*ch + 8*lane + s), issued before
        // the staging below so that their DRAM latency overlaps it
        uint4 raw1 = make_uint4(0, 0, 0, 0);
        uint2 raw2 = make_uint2(0, 0);
        if (q < q_end) {
            const int grp = (c_begin >> 3) + ch * 32 + lane;
            if (8 * grp < c_end) {
                raw1 = ld_stream16(L.s1.ptr + (long long)r * L.s1.stride + 16LL * grp);
                if (RES) raw2 = ld_stream8(L.s2.ptr + (long long)r * L.s2.stride + 8LL * grp);
            }
        }

        // ---- stage x*s of the slab (FP16) and accumulate the bias term sum_n x*b ----------------------
        // (the activations may be the previous kernel's output: everything above read weights only)
        pdl_wait();
        {
            float bacc[TB];
#pragma unroll
            for (int t = 0; t < TB; t++) bacc[t] = 0.f;
            if ((L.N & 7) == 0 && L.perm == nullptr) {
                // 8 columns per thread and step, 128-bit loads (rows of x start 16-byte aligned)
                for (int n = b_begin + 8 * threadIdx.x; n < b_end; n += 8 * THREADS) {
                    float sc[8], bi[8];
                    if (L.has_scale) {
                        act8_to_float(__ldg(reinterpret_cast<const uint4 *>(L.scale + n)), 0, sc);
                        act8_to_float(__ldg(reinterpret_cast<const uint4 *>(L.bias + n)), 0, bi);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; i++) { sc[i] = 1.f; bi[i] = 0.f; }
                    }
                    const bool mine = n >= c_begin && n < c_end;
#pragma unroll
                    for (int t = 0; t < TB; t++) {
                        float xv[8];
                        if (t < P.B) {
                            const uint16_t *xp = reinterpret_cast<const uint16_t *>(P.x) + (long long)t * L.N + n;
                            act8_to_float(__ldg(reinterpret_cast<const uint4 *>(xp)), L.x_bf16, xv);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; i++) xv[i] = 0.f;
                        }
                        uint32_t pk[4];
#pragma unroll
                        for (int i = 0; i < 4; i++) {
                            __half2 h = __floats2half2_rn(xv[2 * i] * sc[2 * i], xv[2 * i + 1] * sc[2 * i + 1]);
                            pk[i] = *reinterpret_cast<uint32_t *>(&h);
                            bacc[t] += xv[2 * i] * bi[2 * i] + xv[2 * i + 1] * bi[2 * i + 1];
                        }
                        if (mine)
                            *reinterpret_cast<uint4 *>(xs + t * P.slab_cols + (n - c_begin)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            } else {
                for (int n = b_begin + threadIdx.x; n < b_end; n += THREADS) {
                    float sc = 1.f, bi = 0.f;
                    if (L.has_scale) {
                        sc = __half2float(__ldg(L.scale + n));
                        bi = __half2float(__ldg(L.bias + n));
                    }
                    const bool mine = n >= c_begin && n < c_end;
#pragma unroll
                    for (int t = 0; t < TB; t++) {
                        const float xv = t < P.B ? load_act(P.x, (long long)t * L.N + in_col(L, n), L.x_bf16) : 0.f;
                        if (mine) xs[t * P.slab_cols + (n - c_begin)] = __float2half_rn(xv * sc);
                        bacc[t] += xv * bi;
                    }
                }
            }
            // zero the ragged end of the slab (columns >= N inside the last chunk)
            for (int cl = (c_end - c_begin) + threadIdx.x; cl < chunks * 256; cl += THREADS)
#pragma unroll
                for (int t = 0; t < TB; t++) xs[t * P.slab_cols + cl] = __float2half_rn(0.f);
#pragma unroll
            for (int t = 0; t < TB; t++) {
                float a = bacc[t];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                if (lane == 0) red[warp * 4 + t] = a;
            }
        }
        __syncthreads();
        if (threadIdx.x < TB) {
            float a = bterm[threadIdx.x];
            for (int w = 0; w < WARPS; w++) a += red[w * 4 + threadIdx.x];
            bterm[threadIdx.x] = a;
        }
        if (!OWNER) __syncthreads();     // balanced: a finishing warp reads bterm right away

        float acc[TB][8];
#pragma unroll
        for (int t = 0; t < TB; t++)
#pragma unroll
            for (int j = 0; j < 8; j++) acc[t][j] = 0.f;
        unsigned done_in_row = 0;

        while (q < q_end) {
            const uint32_t w1[4] = {raw1.x, raw1.y, raw1.z, raw1.w};
            const uint2 cur2 = raw2;
            const int cur_r = r, cur_ch = ch;
            const bool cur_live = 8 * ((c_begin >> 3) + cur_ch * 32 + lane) < c_end;
            // next task, and its indices
            q++;
            if (++ch == chunks) { ch = 0; r++; }
            if (q < q_end) {
                const int grp = (c_begin >> 3) + ch * 32 + lane;
                if (8 * grp < c_end) {
                    raw1 = ld_stream16(L.s1.ptr + (long long)r * L.s1.stride + 16LL * grp);
                    if (RES) raw2 = ld_stream8(L.s2.ptr + (long long)r * L.s2.stride + 8LL * grp);
                }
            }
            if (cur_live) {
                // a3: 8 centroid reads in flight
                uint4 cw[8];
#pragma unroll
                for (int s = 0; s < 8; s++) {
                    uint32_t id = (w1[s >> 1] >> (16 * (s & 1))) & 0xFFFFu;
                    id = min(id, kmax1);
                    cw[s] = __ldg(cb1 + id);
                }
                // this lane's 8 scaled activations per token
                uint4 xv4[TB];
#pragma unroll
                for (int t = 0; t < TB; t++)
                    xv4[t] = *reinterpret_cast<const uint4 *>(xs + t * P.slab_cols + cur_ch * 256 + lane * 8);
#pragma unroll
                for (int s = 0; s < 8; s++) {
                    uint4 w = cw[s];
                    if (RES) {
                        // a4: residual centroid from shared memory, summed in FP16 (one rounding of 2^-11)
                        uint32_t id2 = ((s < 4 ? cur2.x : cur2.y) >> (8 * (s & 3))) & 0xFFu;
                        id2 = min(id2, kmax2);
                        const uint4 rv = cb2[(id2 << rshift) + rep];
                        __half2 a0 = __hadd2(*reinterpret_cast<__half2 *>(&w.x), *reinterpret_cast<const __half2 *>(&rv.x));
                        __half2 a1 = __hadd2(*reinterpret_cast<__half2 *>(&w.y), *reinterpret_cast<const __half2 *>(&rv.y));
                        __half2 a2 = __hadd2(*reinterpret_cast<__half2 *>(&w.z), *reinterpret_cast<const __half2 *>(&rv.z));
                        __half2 a3 = __hadd2(*reinterpret_cast<__half2 *>(&w.w), *reinterpret_cast<const __half2 *>(&rv.w));
                        w.x = *reinterpret_cast<uint32_t *>(&a0); w.y = *reinterpret_cast<uint32_t *>(&a1);
                        w.z = *reinterpret_cast<uint32_t *>(&a2); w.w = *reinterpret_cast<uint32_t *>(&a3);
                    }
#pragma unroll
                    for (int t = 0; t < TB; t++) {
                        const uint32_t xw = (s >> 1) == 0 ? xv4[t].x : (s >> 1) == 1 ? xv4[t].y : (s >> 1) == 2 ? xv4[t].z : xv4[t].w;
                        fma_f16x2(acc[t][0], acc[t][1], xw, (s & 1) != 0, w.x);
                        fma_f16x2(acc[t][2], acc[t][3], xw, (s & 1) != 0, w.y);
                        fma_f16x2(acc[t][4], acc[t][5], xw, (s & 1) != 0, w.z);
                        fma_f16x2(acc[t][6], acc[t][7], xw, (s & 1) != 0, w.w);
                    }
                }
            }
            done_in_row++;
            if (q < q_end && r == cur_r) continue;

            // ---- row change (or end of range): halving butterfly, 8*TB partial sums per lane -> one per lane
            constexpr int NV = 8 * TB;
            float v[NV];
#pragma unroll
            for (int t = 0; t < TB; t++)
#pragma unroll
                for (int j = 0; j < 8; j++) { v[t * 8 + j] = acc[t][j]; acc[t][j] = 0.f; }
            const int vi = halving_butterfly<NV>(v, lane);     // index of the value this lane ends up holding
            // lanes that hold a distinct value: NV = 8: (lane & 3) == 0, NV = 16: (lane & 1) == 0, NV = 32: all
            constexpr int dup = 32 / NV;
            const bool holder = (lane & (dup - 1)) == 0;
            const int t = vi >> 3, j = vi & 7;
            if (OWNER) {
                if (P.det) {
                    // a warp meets a row once per slab, and warps meet rows in ascending order: (row, warp) pairs
                    // have slots of their own at row + warp
                    if (holder) slots[((cur_r - r0) + warp) * (TB * 8) + t * 8 + j] = v[0];
                } else if (holder) atomicAdd(part + ((cur_r - r0) * TB + t) * 8 + j, v[0]);
            } else {
                const int m = cur_r * 8 + j;
                if (holder && t < P.B && m < L.M) atomicAdd(P.yacc + (long long)t * L.M + m, v[0]);
                // completion: the warp that brings a row block's task count to its total finishes the block
                __threadfence();
                __syncwarp();
                const int rb = cur_r / RB_ROWS;
                unsigned total = 0, before = 0;
                if (lane == 0) {
                    const int rows_in_rb = min(RB_ROWS, L.R - rb * RB_ROWS);
                    total = (unsigned)rows_in_rb * (unsigned)P.chunks_total;
                    before = atomicAdd(P.counters + rb, done_in_row);
                }
                total = __shfl_sync(0xffffffffu, total, 0);
                before = __shfl_sync(0xffffffffu, before, 0);
                if (before + done_in_row == total) {
                    __threadfence();
                    const int m_lo = rb * RB_ROWS * 8;
                    const int m_hi = min(L.M, m_lo + RB_ROWS * 8);
                    const int n_m = m_hi - m_lo;
                    for (int i = lane; i < n_m * P.B; i += 32) {
                        const int tt = i / n_m, mm = m_lo + i % n_m;
                        const float y = __ldcg(P.yacc + (long long)tt * L.M + mm) + bterm[tt];
                        store_out(out, (long long)tt * L.M + mm, y, L.out_dtype);
                    }
                }
            }
            done_in_row = 0;
        }
        if (OWNER) __syncthreads();      // the slab's xs is dead; part[] complete after the last slab
        if (OWNER && P.det) {
            // one thread per sum adds the slab's warp partial sums in warp order: the warps whose task range
            // [n_tasks*w/WARPS, n_tasks*(w+1)/WARPS) meets the row's tasks [rho*chunks, (rho+1)*chunks)
            for (int i = threadIdx.x; i < (r1 - r0) * TB * 8; i += THREADS) {
                const int rho = i / (TB * 8), e = i % (TB * 8);
                const long long lo = (long long)rho * chunks, hi = lo + chunks;
                float a = part[i];
                for (int w = 0; w < WARPS; w++) {
                    const long long qa = n_tasks * w / WARPS, qb = n_tasks * (w + 1) / WARPS;
                    if (qa < hi && qb > lo) a += slots[(rho + w) * (TB * 8) + e];
                }
                part[i] = a;
            }
            __syncthreads();
        }
    }

    // ---- OWNER: bias term, conversion, store -----------------------------------------------------------
    if (OWNER) {
        const int m_lo = r0 * 8;
        const int m_hi = min(L.M, r1 * 8);
        const int n_m = m_hi - m_lo;
        for (int i = threadIdx.x; i < n_m * P.B; i += THREADS) {
            const int t = i / n_m, ml = i % n_m;       // consecutive threads -> consecutive m
            const float y = part[((ml >> 3) * TB + t) * 8 + (ml & 7)] + bterm[t];
            store_out(out, (long long)t * L.M + m_lo + ml, y, L.out_dtype);
        }
    }
}

struct L2Plan {
    int slab_cols, n_slabs, chunks_total, cb2_rep, grid, owner, part_floats, warps, det, rows_cta;
    size_t smem;
    long long ws_bytes, off_counters;
    int cta_begin[MAX_FUSED + 1];   // fused launches only
};

L2Plan plan_l2(const LayerView &L, int TB)
{
    L2Plan p;
    p.warps = TB == 4 ? WARPS_TB4 : 32;     // 64 registers per thread suffice up to 2 tokens
    const int n_pad = (L.N + 255) / 256 * 256;
    int slab = XS_BUDGET / (2 * TB) / 256 * 256;
    if (slab > n_pad) slab = n_pad;
    p.slab_cols = slab;
    p.n_slabs = (n_pad + slab - 1) / slab;
    p.chunks_total = n_pad / 256;
    const int G = device_sm_count();
    p.cb2_rep = (L.k2 > 0 && L.k2 <= 256) ? 1 : 0;
    // OWNER mode when whole rows divide well over the SMs (and over the warps of a CTA)
    const int rows_cta = ceil_div(L.R, G);
    const double eff_cta = (double)L.R / ((double)(L.R < G ? L.R : G) * rows_cta) * (L.R < G ? (double)L.R / G : 1.0);
    const long long t_cta = (long long)rows_cta * (slab / 256);
    const double eff_warp = (double)t_cta / ((double)p.warps * (double)((t_cta + p.warps - 1) / p.warps));
    p.part_floats = rows_cta * TB * 8;
    p.rows_cta = rows_cta;
    p.det = L.deterministic ? 1 : 0;
    // a deterministic call takes row-owner mode whatever the balance (the other mode adds by global atomics)
    p.owner = ((eff_cta * eff_warp >= 0.80 || p.det) && (long long)p.part_floats * 4 <= PART_BUDGET) ? 1 : 0;
    if (!p.owner) p.part_floats = 0;
    p.grid = p.owner ? (L.R < G ? L.R : G) : (G < p.n_slabs ? p.n_slabs : G);
    p.smem = (size_t)TB * slab * 2 + 4 * 4 + (size_t)p.warps * 4 * 4 + (size_t)L.k2 * 16 * (p.cb2_rep ? 8 : 1) +
             (size_t)p.part_floats * 4 + (p.det && p.owner ? (size_t)(rows_cta + p.warps) * TB * 8 * 4 : 0);
    p.ws_bytes = 0;
    p.off_counters = 0;
    if (!p.owner) {
        p.off_counters = ((long long)TB * L.M * 4 + 255) / 256 * 256;
        p.ws_bytes = p.off_counters + ((long long)ceil_div(L.R, RB_ROWS) * 4 + 255) / 256 * 256;
    }
    return p;
}

int token_group(int B) { return B >= 4 ? 4 : (B >= 2 ? 2 : 1); }

// A fused launch: the SMs are dealt out to the layers in proportion to their vector rows (every layer at
// least one; leftover SMs go where the most rows per CTA remain).  False when the layers cannot share a
// launch or whole rows would leave the SMs unevenly loaded.
bool plan_l2_fused(const LayerView *Ls, int n, int TB, L2Plan *out)
{
    if (n < 2 || n > MAX_FUSED) return false;
    for (int l = 1; l < n; l++)
        if (Ls[l].N != Ls[0].N || Ls[l].x_bf16 != Ls[0].x_bf16 || Ls[l].k2 != Ls[0].k2) return false;
    L2Plan p = plan_l2(Ls[0], TB);          // slab geometry, warps, residual table: functions of N, k2, TB
    const int G = device_sm_count();
    int R[MAX_FUSED], rows_cta = 0;
    long long rows = 0;
    for (int l = 0; l < n; l++) { R[l] = Ls[l].R; rows += Ls[l].R; }
    if (!split_ctas(R, n, G, p.cta_begin, &rows_cta)) return false;
    const double eff_cta = (double)rows / ((double)G * rows_cta);
    const long long t_cta = (long long)rows_cta * (p.slab_cols / 256);
    const double eff_warp = (double)t_cta / ((double)p.warps * (double)((t_cta + p.warps - 1) / p.warps));
    p.part_floats = rows_cta * TB * 8;
    if (eff_cta * eff_warp < 0.80 || (long long)p.part_floats * 4 > PART_BUDGET) return false;
    p.owner = 1;
    p.grid = G;
    p.smem = (size_t)TB * p.slab_cols * 2 + 4 * 4 + (size_t)p.warps * 4 * 4 +
             (size_t)Ls[0].k2 * 16 * (p.cb2_rep ? 8 : 1) + (size_t)p.part_floats * 4;
    p.ws_bytes = 0;
    p.off_counters = 0;
    *out = p;
    return true;
}

template <int TB, bool RES, bool OWNER, int WARPS, bool FUSED>
cudaError_t launch_one(const L2FmaParams &P, const L2Plan &pl, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(decode_l2_fma_kernel<TB, RES, OWNER, WARPS, FUSED>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    // Launched the ordinary way: as a programmatic dependent this kernel measured slower back to back (the
    // 70B-shaped layer 377 us per pass instead of 295 us), although its prologue is short.  It still lets the
    // kernel after it start early (pdl_launch_dependents above), which is where the gain is.
    decode_l2_fma_kernel<TB, RES, OWNER, WARPS, FUSED><<<pl.grid, WARPS * 32, pl.smem, st>>>(P);
    return cudaGetLastError();
}

template <int TB, int WARPS>
cudaError_t launch_group(const LayerView &L, const L2Plan &pl, const void *x, int Bg, void *out,
                         void *ws, cudaStream_t st)
{
    L2FmaParams P;
    memset(&P, 0, sizeof(P));
    P.L[0] = L; P.out[0] = out; P.n_layers = 1; P.cta_begin[1] = pl.grid;
    P.x = x; P.B = Bg;
    P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs; P.chunks_total = pl.chunks_total;
    P.cb2_replicated = pl.cb2_rep; P.part_floats = pl.part_floats;
    P.det = pl.det && pl.owner; P.rows_cta = pl.rows_cta;
    P.yacc = nullptr; P.counters = nullptr;
    if (!pl.owner) {
        P.yacc = reinterpret_cast<float *>(ws);
        P.counters = reinterpret_cast<unsigned *>(reinterpret_cast<uint8_t *>(ws) + pl.off_counters);
        cudaError_t e = cudaMemsetAsync(ws, 0, (size_t)pl.ws_bytes, st);
        if (e != cudaSuccess) return e;
    }
    const bool res = L.k2 > 0;
    if (pl.owner) return res ? launch_one<TB, true, true, WARPS, false>(P, pl, st) : launch_one<TB, false, true, WARPS, false>(P, pl, st);
    return res ? launch_one<TB, true, false, WARPS, false>(P, pl, st) : launch_one<TB, false, false, WARPS, false>(P, pl, st);
}

template <int TB, int WARPS>
cudaError_t launch_group_fused(const LayerView *Ls, int n, const L2Plan &pl, const void *x, int Bg, void *const *outs,
                               cudaStream_t st)
{
    L2FmaParams P;
    memset(&P, 0, sizeof(P));
    for (int l = 0; l < n; l++) { P.L[l] = Ls[l]; P.out[l] = outs[l]; }
    for (int l = 0; l <= n; l++) P.cta_begin[l] = pl.cta_begin[l];
    P.n_layers = n;
    P.x = x; P.B = Bg;
    P.slab_cols = pl.slab_cols; P.n_slabs = pl.n_slabs; P.chunks_total = pl.chunks_total;
    P.cb2_replicated = pl.cb2_rep; P.part_floats = pl.part_floats;
    P.yacc = nullptr; P.counters = nullptr;
    return Ls[0].k2 > 0 ? launch_one<TB, true, true, WARPS, true>(P, pl, st) : launch_one<TB, false, true, WARPS, true>(P, pl, st);
}

}  // namespace

bool l2_fma_supported(const LayerView &L, int B)
{
    if (L.G > 1) return false;          // one codebook pair per layer here
    if (B < 1 || B > 16) return false;
    if (L.v != 8 || L.n_out != 0 || L.scale_rows) return false;
    if (L.s1.bits != 16) return false;
    if (L.k2 && (L.s2.bits != 8 || L.k2 > 2048)) return false;
    return true;
}

bool l2_fma_deterministic_ok(const LayerView &L, int B)
{
    const L2Plan pl = plan_l2(L, token_group(B));
    return pl.owner != 0 && pl.smem <= 200 * 1024;
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
        if (TB == 4) e = launch_group<4, WARPS_TB4>(L, pl, xg, Bg, og, ws, st);
        else if (TB == 2) e = launch_group<2, 32>(L, pl, xg, Bg, og, ws, st);
        else e = launch_group<1, 32>(L, pl, xg, Bg, og, ws, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

bool l2_fma_fused_supported(const LayerView *Ls, int n, int B)
{
    if (B < 1 || B > 16) return false;
    for (int l = 0; l < n; l++)
        if (!l2_fma_supported(Ls[l], B)) return false;
    L2Plan pl;
    return plan_l2_fused(Ls, n, token_group(B), &pl);
}

int l2_fma_fused_launches(int B)
{
    const int TB = token_group(B);
    return (B + TB - 1) / TB;
}

cudaError_t launch_decode_l2_fma_fused(const LayerView *Ls, int n, const void *x, int B, void *const *outs, cudaStream_t st)
{
    const int TB = token_group(B);
    L2Plan pl;
    if (!plan_l2_fused(Ls, n, TB, &pl)) return cudaErrorInvalidValue;
    for (int t0 = 0; t0 < B; t0 += TB) {
        const int Bg = (B - t0 < TB) ? (B - t0) : TB;
        const void *xg = reinterpret_cast<const uint8_t *>(x) + (size_t)t0 * Ls[0].N * 2;
        void *og[MAX_FUSED];
        for (int l = 0; l < n; l++)
            og[l] = reinterpret_cast<uint8_t *>(outs[l]) + (size_t)t0 * Ls[l].M * (Ls[l].out_dtype == VPTQ_DTYPE_FP32 ? 4 : 2);
        cudaError_t e;
        if (TB == 4) e = launch_group_fused<4, WARPS_TB4>(Ls, n, pl, xg, Bg, og, st);
        else if (TB == 2) e = launch_group_fused<2, 32>(Ls, n, pl, xg, Bg, og, st);
        else e = launch_group_fused<1, 32>(Ls, n, pl, xg, Bg, og, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace vptq
