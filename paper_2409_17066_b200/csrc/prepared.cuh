// Prepared layer image (format text: include/vptq.h): geometry, region offsets, and the launchers of the
// decode kernel that reads it.
#pragma once
#include "common.cuh"

namespace vptq {

constexpr int PREP_WARPS = 31;              // consumer warps of the decode kernel; one more warp loads the buckets
constexpr int PREP_BUCKET = 4096;           // main-codebook entries per bucket (64 KB)
constexpr int PREP_MAX_ROWS = 63;           // vector rows per partition (6-bit row fields; 63 = idle)
constexpr int PREP_SPARE_BLOCKS = 2;         // zero blocks after the last one: a reader may fetch two blocks ahead unchecked
constexpr int PREP_PAD_COLS = 64;           // columns N .. N+63 stand for "no entry" (one per shared-memory bank and half)
constexpr int PREP_MAX_N = 31680;           // the staged activations (N + 64 halves) must fit below the first bucket buffer

struct PreparedGeometry {
    int M, N, v, k1, k2, n_out, Nc, R, n_parts, n_buckets;     // Nc = N - n_out main columns; stored column = n_out + c
    int n_split;                            // partitions that share a group of vector rows, each with a range of buckets
};

// Partition p of an image: row group p / n_split (the groups split the R vector rows evenly, the longer ones first) and the
// h-th of n_split bucket ranges, h = p % n_split.
struct PreparedPart {
    int r0, r1, b0, b1;
};
__host__ __device__ inline PreparedPart prepared_part(int R, int n_buckets, int n_parts, int n_split, int p)
{
    const int groups = n_parts / n_split, g = p / n_split, h = p - g * n_split;
    PreparedPart q;
    // the first R % groups groups hold one row more: CTAs start in index order, a few microseconds apart when the
    // previous kernel's CTAs end one by one, so the longer groups go to the CTAs that start first
    const int base = R / groups, rem = R % groups;
    q.r0 = g * base + (g < rem ? g : rem);
    q.r1 = q.r0 + base + (g < rem ? 1 : 0);
    q.b0 = n_buckets * h / n_split;
    q.b1 = n_buckets * (h + 1) / n_split;
    return q;
}

// The split an image of n_parts partitions gets: the largest of 8, 4, 2, 1 that divides n_parts, leaves every
// partition a bucket, and keeps a row group within PREP_MAX_ROWS rows.  Fewer buckets per CTA mean fewer
// codebook slices to bring in, and more rows per bucket to hide their latency behind.
inline int prepared_split(int R, int n_buckets, int n_parts)
{
    for (int s = 8; s > 1; s >>= 1)
        if (n_parts % s == 0 && s <= n_buckets && ceil_div(R, n_parts / s) <= PREP_MAX_ROWS) return s;
    return 1;
}

struct PreparedLayout {
    unsigned long long off_woff, off_hdr, off_entries, total;
};

inline unsigned long long align256(unsigned long long x) { return (x + 255ull) / 256ull * 256ull; }

inline PreparedLayout prepared_layout(int n_parts, unsigned long long n_blocks)
{
    PreparedLayout l;
    l.off_woff = 256;
    l.off_hdr = align256(l.off_woff + 4ull * ((unsigned long long)n_parts * PREP_WARPS + 1));
    l.off_entries = align256(l.off_hdr + 4ull * n_blocks);
    l.total = align256(l.off_entries + 512ull * (n_blocks + PREP_SPARE_BLOCKS));
    return l;
}

// Layers the prepared path serves (the format text lists them).
inline bool prepared_eligible(const LayerView &L)
{
    // vectors of 8 (16-byte codebook rows, bulk-copied slice by slice), or shorter ones with a main codebook of
    // one bucket (widened to 16-byte rows by the kernel's threads)
    return (L.v == 8 || (L.v < 8 && L.k1 <= PREP_BUCKET)) && L.k1 <= 65536 && (L.k2 == 0 || L.k2 <= 256) &&
           (L.n_out == 0 || L.v0 <= 8) && L.Nc > 0 && L.G == 1 && !L.scale_rows && L.N <= PREP_MAX_N;
}

// n_parts = 0 means one partition per SM; false when a partition would hold more than PREP_MAX_ROWS rows.
inline bool prepared_geometry(const LayerView &L, int n_parts, PreparedGeometry *g)
{
    if (n_parts == 0) n_parts = device_sm_count();
    if (n_parts < 1) return false;
    if (n_parts > L.R) n_parts = L.R;
    g->M = L.M; g->N = L.N; g->v = L.v; g->k1 = L.k1; g->k2 = L.k2; g->n_out = L.n_out; g->Nc = L.Nc; g->R = L.R;
    g->n_parts = n_parts;
    g->n_buckets = (L.k1 + PREP_BUCKET - 1) / PREP_BUCKET;
    g->n_split = prepared_split(L.R, g->n_buckets, n_parts);
    return ceil_div(L.R, n_parts / g->n_split) <= PREP_MAX_ROWS;
}

// capacity handed out by vptq_prepare_bytes: tables for the worst block count that fits, 1.5 x 4 bytes per entry
inline unsigned long long prepared_capacity(const PreparedGeometry &g)
{
    const unsigned long long entries = (unsigned long long)g.R * g.Nc;
    const unsigned long long blocks = (entries * 3 / 2 + 127) / 128 + (unsigned long long)g.n_parts * PREP_WARPS * g.n_buckets;
    return prepared_layout(g.n_parts, blocks).total;
}

int prepare_host(const PreparedGeometry &g, const uint8_t *idx1, const uint8_t *idx2, void *image, size_t image_bytes,
                 size_t *used_bytes);

// decode kernel over prepared images (batch 1): n layers of one launch, CTAs dealt out by the images' n_parts
bool bucket_fma_supported(const LayerView &L, int B);
// Workspace of a launch over these layers: 256 bytes (status word) and, when an image splits its buckets over
// several CTAs, one arrival counter and one block of partial sums per CTA.
size_t bucket_fma_workspace_bytes(const LayerView *Ls, const int *n_parts, int n);
cudaError_t launch_decode_bucket_fma(const LayerView *Ls, const void *const *images, const int *n_parts, int n,
                                     const void *x, void *const *outs, void *workspace, unsigned long long wait_limit,
                                     cudaStream_t st);

}  // namespace vptq
