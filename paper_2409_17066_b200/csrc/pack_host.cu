// Host-memory variants of the packer and unpacker (boundary steps for callers that prepare or inspect
// a checkpoint on the CPU): same stream format as the device kernels, no CUDA call.
#include <string.h>

#include "common.cuh"

namespace vptq {

// One row at a time through a 64-bit shift register: indices enter at the top, whole bytes leave at the
// bottom (the format is a little-endian bit stream per row, rows padded with zero bits to 16 bytes).
long long pack_host(const int32_t *idx, int rows, int cols, int k, uint8_t *packed)
{
    const int bits = index_bits(k);
    const long long stride = row_bytes(cols, k);
    long long bad = 0;
    for (int r = 0; r < rows; r++) {
        uint8_t *dst = packed + (long long)r * stride;
        const int32_t *src = idx + (long long)r * cols;
        unsigned long long reg = 0;
        int held = 0;                       // valid bits in reg
        long long o = 0;
        for (int c = 0; c < cols; c++) {
            int32_t val = src[c];
            if (val < 0 || val >= k) { bad++; val = 0; }
            reg |= (unsigned long long)(uint32_t)val << held;
            held += bits;
            while (held >= 8) { dst[o++] = (uint8_t)reg; reg >>= 8; held -= 8; }
        }
        if (held > 0) dst[o++] = (uint8_t)reg;
        if (o < stride) memset(dst + o, 0, (size_t)(stride - o));
    }
    return bad;
}

void unpack_host(const uint8_t *packed, int rows, int cols, int k, int32_t *idx)
{
    const int bits = index_bits(k);
    const long long stride = row_bytes(cols, k);
    const unsigned long long mask = (1ull << bits) - 1ull;
    for (int r = 0; r < rows; r++) {
        const uint8_t *src = packed + (long long)r * stride;
        int32_t *dst = idx + (long long)r * cols;
        unsigned long long reg = 0;
        int held = 0;
        long long o = 0;
        for (int c = 0; c < cols; c++) {
            while (held < bits) { reg |= (unsigned long long)src[o++] << held; held += 8; }
            dst[c] = (int32_t)(reg & mask);
            reg >>= bits;
            held -= bits;
        }
    }
}

}  // namespace vptq
