// Helpers shared by the decode kernels that keep codebooks in shared memory or read them per group from global
// memory: the packed words of a lane's 8 consecutive indices (a1), their unpacking with the clamp to k-1 that
// the header promises for corrupt streams, a dense table row as a zero-padded 16-byte row, and the warp-wide
// reduction of the row-owner kernels.
#pragma once
#include "common.cuh"

namespace vptq {

// streaming 32-bit load of packed index words: read once, kept out of L1
__device__ __forceinline__ uint32_t ld_stream4(const void *p)
{
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// Raw packed bits of the 8 indices of lane group g (columns 8g..8g+7) of one packed row.
// Never reads beyond the row: words past row_bytes read as zero.  Widths other than 8, 12 and 16 bits are
// decoded here into eight 16-bit values.
__device__ __forceinline__ uint4 load_raw8(const uint8_t *__restrict__ row, long long row_bytes, int g, int cols, int bits)
{
    uint4 q = make_uint4(0, 0, 0, 0);
    if (8 * g >= cols) return q;
    if (bits == 16) {
        q = __ldg(reinterpret_cast<const uint4 *>(row) + g);
    } else if (bits == 8) {
        const uint2 h = __ldg(reinterpret_cast<const uint2 *>(row) + g);
        q.x = h.x; q.y = h.y;
    } else if (bits == 12) {
        const uint8_t *w = row + 12LL * g;
        const long long off = 12LL * g;
        // three word loads at a 12-byte lane stride: each touches the same 12 sectors of the warp's 384-byte span,
        // so they go through L1 (issued back to back, the second and third merge with the first's misses)
        q.x = __ldg(reinterpret_cast<const uint32_t *>(w));
        q.y = (off + 8 <= row_bytes) ? __ldg(reinterpret_cast<const uint32_t *>(w + 4)) : 0u;
        q.z = (off + 12 <= row_bytes) ? __ldg(reinterpret_cast<const uint32_t *>(w + 8)) : 0u;
    } else {
        uint32_t v[8];
#pragma unroll
        for (int s = 0; s < 8; s++) v[s] = (8 * g + s < cols) ? (uint32_t)load_index(row, 8 * g + s, bits) : 0u;
        q.x = v[0] | (v[1] << 16); q.y = v[2] | (v[3] << 16);
        q.z = v[4] | (v[5] << 16); q.w = v[6] | (v[7] << 16);
    }
    return q;
}

// Raw bits -> eight indices as 16-bit pairs in 4 words, clamped to k-1.
__device__ __forceinline__ void decode8(uint4 q, int bits, int k, uint32_t (&w)[4])
{
    if (bits == 8) {
        w[0] = __byte_perm(q.x, 0, 0x4140); w[1] = __byte_perm(q.x, 0, 0x4342);
        w[2] = __byte_perm(q.y, 0, 0x4140); w[3] = __byte_perm(q.y, 0, 0x4342);
    } else if (bits == 12) {
        const uint32_t a = q.x, b = q.y, c = q.z;
        const uint32_t i0 = a & 0xFFFu, i1 = (a >> 12) & 0xFFFu, i2 = __funnelshift_r(a, b, 24) & 0xFFFu;
        const uint32_t i3 = (b >> 4) & 0xFFFu, i4 = (b >> 16) & 0xFFFu, i5 = __funnelshift_r(b, c, 28) & 0xFFFu;
        const uint32_t i6 = (c >> 8) & 0xFFFu, i7 = c >> 20;
        w[0] = i0 | (i1 << 16); w[1] = i2 | (i3 << 16); w[2] = i4 | (i5 << 16); w[3] = i6 | (i7 << 16);
    } else {
        w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
    }
    const uint32_t lim = (uint32_t)(k - 1) * 0x10001u;
#pragma unroll
    for (int i = 0; i < 4; i++) w[i] = __vminu2(w[i], lim);
}

// One centroid [v] fp16 (dense table, entry e, v <= 8) as a zero-padded 16-byte row.
__device__ __forceinline__ uint4 load_centroid_row(const __half *__restrict__ tab, int e, int v)
{
    if (v == 8) return __ldg(reinterpret_cast<const uint4 *>(tab) + e);
    uint32_t w[4] = {0, 0, 0, 0};
    if ((v & 1) == 0) {
        const uint32_t *p = reinterpret_cast<const uint32_t *>(tab) + (long long)e * (v >> 1);   // tables are 16-byte aligned
#pragma unroll
        for (int i = 0; i < 4; i++)
            if (i < (v >> 1)) w[i] = __ldg(p + i);
    } else {
        const uint16_t *p = reinterpret_cast<const uint16_t *>(tab) + (long long)e * v;
#pragma unroll
        for (int i = 0; i < 8; i++)
            if (i < v) w[i >> 1] |= (uint32_t)__ldg(p + i) << (16 * (i & 1));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Halving butterfly over the warp: every lane holds NV partial sums v[0..NV) of the same NV quantities; after
// the call quantity q's total over the 32 lanes sits in v[k] of the lanes with first = the returned index,
// q = first + k, k < max(1, NV / 32): with NV >= 32 every lane holds NV / 32 distinct totals, with NV < 32 only
// the lanes whose low log2(32 / NV) bits are clear matter (the others hold copies).  31 shuffles' worth of
// additions spread over the lanes instead of 5 * NV.
template <int NV>
__device__ __forceinline__ int halving_butterfly(float (&v)[NV], int lane)
{
    int first = 0, n = NV, o = 16;
#pragma unroll
    for (int step = 0; step < 5; step++) {
        if (n > 1) {
            const bool up = (lane & o) != 0;
            const int h = n / 2;
#pragma unroll
            for (int k = 0; k < NV / 2; k++) {
                if (k < h) {
                    const float send = up ? v[k] : v[k + h];
                    const float keep = up ? v[k + h] : v[k];
                    v[k] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
            }
            first += up ? h : 0;
            n = h;
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
        }
        o >>= 1;
    }
    return first;
}

}  // namespace vptq
