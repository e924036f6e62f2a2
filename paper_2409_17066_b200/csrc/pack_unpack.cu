// Bit-packed index streams: pack (int32 matrix -> stream) and unpack (stream -> int32),
// one thread per 16-byte chunk of a packed row, so that every global access to the
// stream is one aligned 128-bit load or store.
#include "common.cuh"

namespace vptq {

// Thread (row, j) builds bytes [16j, 16j+16) of the row: the 128 stream bits
// [128j, 128j+128) are the OR of every index that overlaps them.
__global__ void __launch_bounds__(256)
pack_kernel(const int32_t *__restrict__ idx, int rows, int cols, int k, int bits,
            int chunks_per_row, uint8_t *__restrict__ packed, int32_t *bad_count)
{
    long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long total = (long long)rows * chunks_per_row;
    if (gid >= total) return;
    int row = (int)(gid / chunks_per_row);
    int j = (int)(gid % chunks_per_row);
    long long bit0 = 128LL * j;
    long long c_lo = bit0 / bits;
    long long c_hi = (bit0 + 127) / bits;
    if (c_hi > cols - 1) c_hi = cols - 1;
    unsigned long long lo = 0ull, hi = 0ull;
    int bad = 0;
    const int32_t *src = idx + (long long)row * cols;
    for (long long c = c_lo; c <= c_hi; c++) {
        int32_t raw = src[c];
        if (raw < 0 || raw >= k) { bad++; raw = 0; }
        unsigned long long val = (unsigned long long)(uint32_t)raw;
        long long p = c * bits - bit0;            // position of the index's bit 0 inside this chunk
        if (p < 0) { val >>= (unsigned)(-p); p = 0; }
        if (p < 64) {
            lo |= val << (unsigned)p;
            if (p + bits > 64) hi |= val >> (unsigned)(64 - p);
        } else {
            hi |= val << (unsigned)(p - 64);       // bits beyond 128 fall off: they belong to the next chunk
        }
    }
    uint4 o;
    o.x = (uint32_t)lo; o.y = (uint32_t)(lo >> 32);
    o.z = (uint32_t)hi; o.w = (uint32_t)(hi >> 32);
    reinterpret_cast<uint4 *>(packed)[gid] = o;
    // count each bad index once: by the chunk that holds its bit 0
    if (bad_count != nullptr && bad) {
        int mine = 0;
        for (long long c = c_lo; c <= c_hi; c++) {
            int32_t raw = src[c];
            if ((raw < 0 || raw >= k) && c * bits >= bit0) mine++;
        }
        if (mine) atomicAdd(bad_count, mine);
    }
}

// Thread (row, j) loads chunk j with one 128-bit load (plus the first word of chunk j+1
// for an index that crosses into it) and decodes every index whose bit 0 lies in the chunk.
__global__ void __launch_bounds__(256)
unpack_kernel(const uint8_t *__restrict__ packed, int rows, int cols, int bits,
              int chunks_per_row, int32_t *__restrict__ idx)
{
    long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long total = (long long)rows * chunks_per_row;
    if (gid >= total) return;
    int row = (int)(gid / chunks_per_row);
    int j = (int)(gid % chunks_per_row);
    const uint4 *src = reinterpret_cast<const uint4 *>(packed);
    uint4 q = __ldg(src + gid);
    uint32_t w4 = (j + 1 < chunks_per_row) ? __ldg(reinterpret_cast<const uint32_t *>(src + gid + 1)) : 0u;
    long long bit0 = 128LL * j;
    long long c_lo = (bit0 + bits - 1) / bits;
    long long c_hi = (bit0 + 127) / bits;
    if (c_hi > cols - 1) c_hi = cols - 1;
    uint32_t mask = (1u << bits) - 1u;
    int32_t *dst = idx + (long long)row * cols;
    for (long long c = c_lo; c <= c_hi; c++) {
        unsigned o = (unsigned)(c * bits - bit0);  // 0..127
        unsigned wi = o >> 5, sh = o & 31u;
        uint32_t lo = wi == 0 ? q.x : wi == 1 ? q.y : wi == 2 ? q.z : q.w;
        uint32_t hi = wi == 0 ? q.y : wi == 1 ? q.z : wi == 2 ? q.w : w4;
        dst[c] = (int32_t)(__funnelshift_r(lo, hi, sh) & mask);
    }
}

cudaError_t launch_pack(const int32_t *idx, int rows, int cols, int k, uint8_t *packed,
                        int32_t *bad_count, cudaStream_t st)
{
    if (rows == 0 || cols == 0) return cudaSuccess;
    int chunks = (int)(row_bytes(cols, k) / 16);
    long long total = (long long)rows * chunks;
    int grid = (int)((total + 255) / 256);
    pack_kernel<<<grid, 256, 0, st>>>(idx, rows, cols, k, index_bits(k), chunks, packed, bad_count);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const uint8_t *packed, int rows, int cols, int k, int32_t *idx,
                          cudaStream_t st)
{
    if (rows == 0 || cols == 0) return cudaSuccess;
    int chunks = (int)(row_bytes(cols, k) / 16);
    long long total = (long long)rows * chunks;
    int grid = (int)((total + 255) / 256);
    unpack_kernel<<<grid, 256, 0, st>>>(packed, rows, cols, index_bits(k), chunks, idx);
    return cudaGetLastError();
}

}  // namespace vptq
