/*
 * CPU oracle for the inference side of VPTQ (vector post-training quantization).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition of what the
 * vector-quantized linear layer computes.  It is used by the tests, by the smoke
 * check and by the benchmark's CPU-baseline leg; the product path never calls it
 * and it shares no code, header, table or helper with the CUDA library.
 *
 * What is defined here and where the paper states it:
 *   - a weight matrix W (M x N, M = output features, N = input features) is cut
 *     into length-v vectors that run down a column (Sec. 2.2; Sec. 3.1, the
 *     quantized column is a stack of centroids; Algorithm 1 inner loop over
 *     m = 0, V, 2V, ...);
 *   - inference restores the weight from the lookup table by index (Sec. 2.2
 *     "dequantizes the original weight matrix from the lookup table by index and
 *     centroid"; Sec. 4 last sentence);
 *   - residual VQ decode reads one centroid from every table and sums them
 *     (Sec. 3.2.2, last sentence);
 *   - outlier columns use their own table with their own vector length
 *     (Sec. 3.2.3; App. C.1 "Parameter Description"), and have no residual stage
 *     (Algorithm 2 order; index-bit formula of App. C.2);
 *   - which columns are outlier columns is the quantizer's choice (Sec. 3.2.3: the
 *     columns with the largest Hessian diagonal; Algorithm 2 "selects outlier
 *     columns"), so they may lie anywhere in the matrix: the layer may carry a
 *     column order, col_perm, that says which input feature each stored column is;
 *   - the weights are restored to FP16 and then multiplied (App. D.2).
 *   - size accounting: compression ratio / equivalent bit width (Sec. 2.2) and
 *     the index-bit / codebook-bit formulas (App. C.2);
 *   - the quantizer's assignment step (Eq. 2): every vector of the reshaped weight
 *     matrix takes the index of the centroid at the smallest Euclidean distance
 *     (oracle_assign below; the Hessian-driven parts of Algorithms 1 and 2 are not
 *     here).
 *
 * Not stated by the paper, defined by this project (parity unpinned by the
 * paper, consistency-checked only): the per-input-channel scale and bias and
 * their FP32 operation order, the bit-packed index stream, "the first n_out
 * STORED columns are the outlier columns", and the form of the column order
 * (an explicit list of N input-feature numbers; scale and bias follow the
 * stored order), and the arithmetic of the assignment step (Eq. 2 names the
 * Euclidean distance, not its precision, summation order or tie rule: FP32, fused
 * multiply-add, components ascending, lowest index wins).
 *
 * Every function has a pin in tests/test_oracle_pins.py that is not itself: none is
 * "parity unpinned" except in the sense above (choices the paper does not make).
 *
 * Arithmetic: lookup sum, scale and bias in FP32 with three separately rounded
 * operations (build with -ffp-contract=off), result rounded to FP16
 * (round-to-nearest-even), matmul in FP64 over the FP16-rounded weights with n
 * ascending.
 *
 * OpenMP pragmas only split independent output rows across cores for timing;
 * they change no result.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* FP16 / BF16 <-> FP32, written at the bit level (IEEE 754 binary16)   */
/* ------------------------------------------------------------------ */

static float bits_to_float(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static uint32_t float_to_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

float oracle_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) << 31;
    uint32_t e = (h >> 10) & 0x1F;
    uint32_t m = h & 0x3FF;
    if (e == 0) {
        if (m == 0) return bits_to_float(sign);
        /* subnormal: value = m * 2^-24 */
        float v = (float)m * (1.0f / 16777216.0f);
        return (sign ? -v : v);
    }
    if (e == 31) return bits_to_float(sign | 0x7F800000u | (m << 13));
    return bits_to_float(sign | ((e + 112) << 23) | (m << 13));
}

uint16_t oracle_float_to_half(float f)
{
    uint32_t u = float_to_bits(f);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000);
    uint32_t a = u & 0x7FFFFFFFu;
    if (a > 0x7F800000u) return (uint16_t)(sign | 0x7E00 | ((a >> 13) & 0x3FF)); /* NaN */
    if (a >= 0x477FF000u) return (uint16_t)(sign | 0x7C00); /* >= 65520 rounds to inf */
    int32_t e = (int32_t)(a >> 23) - 127;
    if (e >= -14) {
        /* normal half: keep 10 mantissa bits, round to nearest even on the 13 dropped */
        uint32_t mant = a & 0x7FFFFF;
        uint32_t h = ((uint32_t)(e + 15) << 10) | (mant >> 13);
        uint32_t rem = mant & 0x1FFF;
        if (rem > 0x1000 || (rem == 0x1000 && (h & 1))) h++;   /* carry may bump the exponent: still right */
        return (uint16_t)(sign | h);
    }
    if (e < -25) return sign;   /* below half of the smallest subnormal (2^-25 itself handled below) */
    /* subnormal half: value / 2^-24 rounded to nearest even integer */
    uint32_t mant = (a & 0x7FFFFF) | 0x800000;      /* 24-bit significand, value = mant * 2^(e-23) */
    int shift = (-e - 24) + 23;                     /* result = mant >> shift, with e in [-25,-15] -> shift in [14,24] */
    uint32_t h = mant >> shift;
    uint32_t rem = mant & ((1u << shift) - 1);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (h & 1))) h++;
    return (uint16_t)(sign | h);
}

float oracle_bf16_to_float(uint16_t b) { return bits_to_float((uint32_t)b << 16); }

uint16_t oracle_float_to_bf16(float f)
{
    uint32_t u = float_to_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);
    uint32_t lsb = (u >> 16) & 1;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------ */
/* Bit-packed index stream (project-defined format)                    */
/* ------------------------------------------------------------------ */
/* b = max(1, ceil(log2 k)) bits per index.  Every row of the index matrix is its
 * own little-endian bit stream: index c occupies stream bits [c*b, c*b+b), stream
 * bit i is bit (i % 8) of byte (i / 8).  A row occupies ceil(cols*b/8) bytes rounded
 * up to a multiple of 16; pad bits are zero. */

int oracle_index_bits(int32_t k)
{
    int b = 0;
    while (((int64_t)1 << b) < (int64_t)k) b++;
    return b < 1 ? 1 : b;
}

int64_t oracle_row_bytes(int32_t cols, int32_t k)
{
    int64_t bits = (int64_t)cols * oracle_index_bits(k);
    int64_t bytes = (bits + 7) / 8;
    return (bytes + 15) / 16 * 16;
}

int64_t oracle_packed_bytes(int32_t rows, int32_t cols, int32_t k)
{
    return (int64_t)rows * oracle_row_bytes(cols, k);
}

/* returns 0, or -1 when some index lies outside [0, k) (nothing useful is written then) */
int oracle_pack(const int32_t *idx, int32_t rows, int32_t cols, int32_t k, uint8_t *out)
{
    int b = oracle_index_bits(k);
    int64_t stride = oracle_row_bytes(cols, k);
    memset(out, 0, (size_t)(stride * rows));
    for (int32_t r = 0; r < rows; r++) {
        uint8_t *row = out + (int64_t)r * stride;
        for (int32_t c = 0; c < cols; c++) {
            int32_t val = idx[(int64_t)r * cols + c];
            if (val < 0 || val >= k) return -1;
            for (int i = 0; i < b; i++) {
                if ((val >> i) & 1) {
                    int64_t bit = (int64_t)c * b + i;
                    row[bit / 8] |= (uint8_t)(1u << (bit % 8));
                }
            }
        }
    }
    return 0;
}

static int32_t read_index(const uint8_t *row, int64_t c, int b)
{
    int32_t val = 0;
    for (int i = 0; i < b; i++) {
        int64_t bit = c * b + i;
        if ((row[bit / 8] >> (bit % 8)) & 1) val |= (1 << i);
    }
    return val;
}

void oracle_unpack(const uint8_t *packed, int32_t rows, int32_t cols, int32_t k, int32_t *idx)
{
    int b = oracle_index_bits(k);
    int64_t stride = oracle_row_bytes(cols, k);
    for (int32_t r = 0; r < rows; r++)
        for (int32_t c = 0; c < cols; c++)
            idx[(int64_t)r * cols + c] = read_index(packed + (int64_t)r * stride, c, b);
}

/* ------------------------------------------------------------------ */
/* Layer description                                                   */
/* ------------------------------------------------------------------ */

typedef struct oracle_layer {
    int32_t M, N;            /* W is [M][N]: M output features, N input features   */
    int32_t v, k1, k2;       /* main vector length, main / residual table sizes     */
    int32_t n_out, v0, k0;   /* leading outlier columns, their vector length/table  */
    int32_t has_scale;       /* 1: W = t*scale[n] + bias[n]                          */
    int32_t scale_axis;      /* 0: per input column n; 1: per output row m          */
    int32_t n_groups;        /* column groups with codebooks of their own (Sec. 3.1); <= 1: one */
    const uint8_t *idx1;     /* packed [ceil(M/v)][N-n_out], b(k1) bits             */
    const uint16_t *c1;      /* [n_groups][k1][v] fp16 bits                         */
    const uint8_t *idx2;     /* packed, same shape, b(k2) bits (k2 > 0)             */
    const uint16_t *c2;      /* [n_groups][k2][v]                                   */
    const uint8_t *idx0;     /* packed [ceil(M/v0)][n_out], b(k0) bits (n_out > 0)  */
    const uint16_t *c0;      /* [k0][v0]                                            */
    const uint16_t *scale;   /* fp16 bits, [N] (axis 0, stored column order) or [M] (axis 1) */
    const uint16_t *bias;
    const int32_t *col_perm; /* NULL, or [N]: stored column j is input feature col_perm[j]
                                (a permutation of 0..N-1; Sec. 3.2.3)                */
} oracle_layer;

/* Input feature of stored column j; -1 when the list names a feature outside [0,N). */
static int32_t feature_of(const oracle_layer *L, int32_t j)
{
    if (L->col_perm == NULL) return j;
    int32_t f = L->col_perm[j];
    return (f < 0 || f >= L->N) ? -1 : f;
}

/* One restored weight, FP16 bits: row m of STORED column n (its place in W is column
 * feature_of(n)).  Sets *err when an index is out of range (corrupt stream): the tests
 * treat that as a failure. */
static uint16_t restore_weight(const oracle_layer *L, int32_t m, int32_t n, int *err)
{
    float t;
    if (n < L->n_out) {
        /* outlier column: own table, own vector length, no residual stage */
        int64_t stride0 = oracle_row_bytes(L->n_out, L->k0);
        int32_t r0 = m / L->v0, j0 = m % L->v0;
        int32_t i0 = read_index(L->idx0 + (int64_t)r0 * stride0, n, oracle_index_bits(L->k0));
        if (i0 >= L->k0) { *err = 1; return 0; }
        t = oracle_half_to_float(L->c0[(int64_t)i0 * L->v0 + j0]);
    } else {
        int32_t c = n - L->n_out, Nc = L->N - L->n_out;
        int32_t r = m / L->v, j = m % L->v;
        /* Sec. 3.1: the (non-outlier) columns are split into `group num` equal runs of consecutive
         * columns, each with codebooks of its own; the last run is shorter when Nc is not a multiple. */
        int32_t G = L->n_groups > 1 ? L->n_groups : 1;
        int32_t cols_per_group = (Nc + G - 1) / G;
        int32_t g = c / cols_per_group;
        int64_t stride1 = oracle_row_bytes(Nc, L->k1);
        int32_t i1 = read_index(L->idx1 + (int64_t)r * stride1, c, oracle_index_bits(L->k1));
        if (i1 >= L->k1) { *err = 1; return 0; }
        t = oracle_half_to_float(L->c1[((int64_t)g * L->k1 + i1) * L->v + j]);
        if (L->k2 > 0) {
            int64_t stride2 = oracle_row_bytes(Nc, L->k2);
            int32_t i2 = read_index(L->idx2 + (int64_t)r * stride2, c, oracle_index_bits(L->k2));
            if (i2 >= L->k2) { *err = 1; return 0; }
            float t2 = oracle_half_to_float(L->c2[((int64_t)g * L->k2 + i2) * L->v + j]);
            t = t + t2;                     /* rounded FP32 add */
        }
    }
    if (L->has_scale) {
        int32_t a = L->scale_axis ? m : n;
        float s = oracle_half_to_float(L->scale[a]);
        float bb = oracle_half_to_float(L->bias[a]);
        float p = t * s;                    /* rounded FP32 multiply */
        t = p + bb;                         /* rounded FP32 add      */
    }
    return oracle_float_to_half(t);
}

/* Restore the whole matrix: W16 [M][N] FP16 bits.  Returns 0 or -1 (index out of range). */
int oracle_dequant(const oracle_layer *L, uint16_t *W16)
{
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(|:bad)
    for (int32_t m = 0; m < L->M; m++) {
        int err = 0;
        for (int32_t n = 0; n < L->N; n++) {
            int32_t f = feature_of(L, n);
            if (f < 0) { err = 1; continue; }
            W16[(int64_t)m * L->N + f] = restore_weight(L, m, n, &err);
        }
        bad |= err;
    }
    return bad ? -1 : 0;
}

/* Restore selected rows only: rows[i] in [0,M) -> Wrows [n_rows][N]. */
int oracle_dequant_rows(const oracle_layer *L, const int32_t *rows, int32_t n_rows, uint16_t *Wrows)
{
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(|:bad)
    for (int32_t i = 0; i < n_rows; i++) {
        int err = 0;
        for (int32_t n = 0; n < L->N; n++) {
            int32_t f = feature_of(L, n);
            if (f < 0) { err = 1; continue; }
            Wrows[(int64_t)i * L->N + f] = restore_weight(L, rows[i], n, &err);
        }
        bad |= err;
    }
    return bad ? -1 : 0;
}

static double load_x(const uint16_t *x, int64_t i, int x_is_bf16)
{
    return (double)(x_is_bf16 ? oracle_bf16_to_float(x[i]) : oracle_half_to_float(x[i]));
}

/* y[t][i] = sum_n x[t][n] * W16[rows[i]][n] in FP64, n ascending.
 * rows == NULL means all M rows (n_rows must then be M).  y is [B][n_rows]. */
int oracle_linear_rows(const oracle_layer *L, const uint16_t *x, int32_t B, int x_is_bf16,
                       const int32_t *rows, int32_t n_rows, double *y)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 4) reduction(|:bad)
    for (int32_t i = 0; i < n_rows; i++) {
        int err = 0;
        int32_t m = rows ? rows[i] : i;
        uint16_t *w = (uint16_t *)calloc((size_t)L->N, sizeof(uint16_t));
        for (int32_t n = 0; n < L->N; n++) {
            int32_t f = feature_of(L, n);
            if (f < 0) { err = 1; continue; }
            w[f] = restore_weight(L, m, n, &err);          /* row m of W, in input-feature order */
        }
        for (int32_t t = 0; t < B; t++) {
            double acc = 0.0;
            for (int32_t n = 0; n < L->N; n++)
                acc += load_x(x, (int64_t)t * L->N + n, x_is_bf16) * (double)oracle_half_to_float(w[n]);
            y[(int64_t)t * n_rows + i] = acc;
        }
        free(w);
        bad |= err;
    }
    return bad ? -1 : 0;
}

int oracle_linear(const oracle_layer *L, const uint16_t *x, int32_t B, int x_is_bf16, double *y)
{
    return oracle_linear_rows(L, x, B, x_is_bf16, NULL, L->M, y);
}

/* ------------------------------------------------------------------ */
/* Assignment step of the quantizer (Eq. 2)                            */
/* ------------------------------------------------------------------ */

/* Squared Euclidean distance between vector (r, n) of W and centroid i, over the components
 * that exist (the last vector row is short when v does not divide M).
 * Floating point decides an integer here, so the arithmetic is fixed: FP32, components in
 * ascending order, each step d = fma(t, t, d) with t = x_j - c_j rounded to FP32. */
static float sq_distance(const uint16_t *W, int32_t M, int32_t N, int32_t v, int32_t r, int32_t n,
                         const uint16_t *C, int32_t i)
{
    float d = 0.0f;
    for (int32_t j = 0; j < v && r * v + j < M; j++) {
        float x = oracle_half_to_float(W[(int64_t)(r * v + j) * N + n]);
        float c = oracle_half_to_float(C[(int64_t)i * v + j]);
        float t = x - c;
        d = fmaf(t, t, d);
    }
    return d;
}

/* Eq. 2 for one vector: argmin_i || v - C_i ||^2; of equal distances the lowest index wins;
 * a distance that is NaN never wins (all NaN: index 0). */
static int32_t nearest_centroid(const uint16_t *W, int32_t M, int32_t N, int32_t v, int32_t r, int32_t n,
                                const uint16_t *C, int32_t k)
{
    int32_t best = 0;
    float best_d = INFINITY;
    for (int32_t i = 0; i < k; i++) {
        float d = sq_distance(W, M, N, v, r, n, C, i);
        if (d < best_d) { best_d = d; best = i; }
    }
    return best;
}

/* idx [ceil(M/v)][N]: vectors are v consecutive rows of one column (Sec. 3.1, Algorithm 1). */
void oracle_assign(const uint16_t *W, int32_t M, int32_t N, int32_t v, const uint16_t *C, int32_t k, int32_t *idx)
{
    int32_t R = (M + v - 1) / v;
#pragma omp parallel for schedule(static)
    for (int32_t r = 0; r < R; r++)
        for (int32_t n = 0; n < N; n++)
            idx[(int64_t)r * N + n] = nearest_centroid(W, M, N, v, r, n, C, k);
}

/* The same for selected vectors only: vec[i] = r * N + n. */
void oracle_assign_some(const uint16_t *W, int32_t M, int32_t N, int32_t v, const uint16_t *C, int32_t k,
                        const int64_t *vec, int32_t n_vec, int32_t *idx)
{
#pragma omp parallel for schedule(dynamic, 4)
    for (int32_t i = 0; i < n_vec; i++)
        idx[i] = nearest_centroid(W, M, N, v, (int32_t)(vec[i] / N), (int32_t)(vec[i] % N), C, k);
}

/* Centroid update of (weighted) k-means (Sec. 2.2 "k-means ... to build a codebook"; Sec. 3.2.1: the
 * diagonal term of the proxy error, sum_n h_nn ||dW[:,n]||^2, is a weighted k-means problem whose
 * weight is the Hessian diagonal of the vector's column).  With the assignment fixed, the minimiser of
 * sum h_n ||x - C_i||^2 over C_i is the weighted mean of the vectors assigned to i:
 *   C_i[j] = sum h_n x_j / sum h_n   over the vectors (r, n) with idx[r][n] = i that have component j
 * (the short last vector row has no components beyond row M-1).  FP64 sums, result rounded to FP16.
 * h == NULL means all weights 1.  A component that received no weight keeps its old value. */
void oracle_kmeans_update(const uint16_t *W, int32_t M, int32_t N, int32_t v, const int32_t *idx,
                          const float *h, int32_t k, uint16_t *C)
{
    int32_t R = (M + v - 1) / v;
    double *sum = (double *)calloc((size_t)k * v, sizeof(double));
    double *wsum = (double *)calloc((size_t)k * v, sizeof(double));
    for (int32_t r = 0; r < R; r++)
        for (int32_t n = 0; n < N; n++) {
            int32_t i = idx[(int64_t)r * N + n];
            if (i < 0 || i >= k) continue;
            double w = h ? (double)h[n] : 1.0;
            for (int32_t j = 0; j < v && r * v + j < M; j++) {
                sum[(int64_t)i * v + j] += w * (double)oracle_half_to_float(W[(int64_t)(r * v + j) * N + n]);
                wsum[(int64_t)i * v + j] += w;
            }
        }
    for (int64_t e = 0; e < (int64_t)k * v; e++)
        if (wsum[e] > 0.0) C[e] = oracle_float_to_half((float)(sum[e] / wsum[e]));
    free(sum);
    free(wsum);
}

/* Weighted distortion sum_n h_n ||x - C_idx||^2 in FP64 (the quantity a k-means step must not increase). */
double oracle_distortion(const uint16_t *W, int32_t M, int32_t N, int32_t v, const int32_t *idx,
                         const float *h, const uint16_t *C)
{
    int32_t R = (M + v - 1) / v;
    double total = 0.0;
    for (int32_t r = 0; r < R; r++)
        for (int32_t n = 0; n < N; n++) {
            int32_t i = idx[(int64_t)r * N + n];
            double w = h ? (double)h[n] : 1.0, d = 0.0;
            for (int32_t j = 0; j < v && r * v + j < M; j++) {
                double t = (double)oracle_half_to_float(W[(int64_t)(r * v + j) * N + n]) -
                           (double)oracle_half_to_float(C[(int64_t)i * v + j]);
                d += t * t;
            }
            total += w * d;
        }
    return total;
}

/* ------------------------------------------------------------------ */
/* Prepared layer image -> canonical index matrices                    */
/* ------------------------------------------------------------------ */

/* The library can re-order a layer's (main, residual) index pairs into a "prepared image" for its decode
 * kernel.  The image is derived data whose format is stated in the library's header (version 2); this is a
 * decoder written from that statement, used to check that an image says exactly what the canonical streams
 * say.  The paper has no counterpart (it does not describe an inference data layout).
 *
 * Walks every warp's block range of every partition, checks each rule of the format and writes the index
 * pairs back to idx1 / idx2 [ceil(M/v)][N - n_out] (int32; main columns only, the image holds nothing of the
 * outlier columns).  Returns 0, or a positive code naming the first rule
 * that is broken:
 *   1 header magic/version  2 header geometry differs from the arguments, or a split that does not divide the partitions  3 region offsets or sizes
 *   4 block ranges not ascending or not ending at n_blocks  5 bucket outside the partition's range or descending within a warp
 *   6 an entry in a quarter that names no row / a row outside the partition  7 column out of range
 *   8 main or residual index out of range  9 a (row, column) pair occurs twice  10 a pair is missing
 *   11 a partition holds more than 63 vector rows  12 number of real entries differs from the header's */
int oracle_decode_prepared(const uint8_t *image, int64_t image_bytes, int32_t M, int32_t N, int32_t v, int32_t k1, int32_t k2,
                           int32_t n_out, int32_t *idx1, int32_t *idx2)
{
    if (image_bytes < 256) return 3;
    uint32_t head[18];
    memcpy(head, image, sizeof(head));
    if (head[0] != 0x42515056u || head[1] != 2u) return 1;
    if (v < 1 || v > 8 || n_out < 0 || n_out >= N) return 2;
    const int64_t R = (M + v - 1) / v;       /* vector rows */
    const int64_t Nc = N - n_out;            /* main columns; they are stored after the outlier columns */
    const uint32_t n_parts = head[6], n_warps = head[7], n_buckets = head[8], n_blocks = head[9];
    if (head[2] != (uint32_t)M || head[3] != (uint32_t)N || head[4] != (uint32_t)k1 || head[5] != (uint32_t)k2) return 2;
    if (head[16] != (uint32_t)v || head[17] != (uint32_t)n_out) return 2;
    if (n_warps != 31u || n_buckets != (uint32_t)((k1 + 4095) / 4096) || n_parts < 1u || (int64_t)n_parts > R) return 2;
    /* word 15: partitions per row group; each of them holds one range of buckets */
    const uint32_t n_split = head[15];
    if (n_split < 1u || n_parts % n_split != 0u || n_split > n_buckets) return 2;
    const uint32_t n_groups = n_parts / n_split;
    const uint64_t off_woff = head[10], off_hdr = head[11], off_ent = head[12], total = head[13];
    if (off_woff % 256 || off_hdr % 256 || off_ent % 256 || off_woff < 256) return 3;
    if (off_woff + 4ull * ((uint64_t)n_parts * n_warps + 1) > off_hdr) return 3;
    if (off_hdr + 4ull * n_blocks > off_ent) return 3;
    /* two spare blocks follow the last one */
    if (off_ent + 512ull * ((uint64_t)n_blocks + 2u) > total || total > (uint64_t)image_bytes) return 3;
    const uint8_t *woff_b = image + off_woff, *hdr_b = image + off_hdr, *ent_b = image + off_ent;
    for (int64_t i = 0; i < R * Nc; i++) { idx1[i] = -1; idx2[i] = -1; }
    uint64_t real = 0;
    uint32_t prev_end = 0;
    for (uint32_t p = 0; p < n_parts; p++) {
        const uint32_t grp = p / n_split, piece = p % n_split;
        /* R = n_groups * base + rem: the first rem groups hold base + 1 rows, the others base */
        const int64_t base_rows = R / n_groups, rem_rows = R % n_groups;
        const int64_t r0 = grp * base_rows + ((int64_t)grp < rem_rows ? (int64_t)grp : rem_rows);
        const int64_t r1 = r0 + base_rows + ((int64_t)grp < rem_rows ? 1 : 0);
        const uint32_t bucket_lo = n_buckets * piece / n_split, bucket_hi = n_buckets * (piece + 1) / n_split;
        if (r1 - r0 > 63) return 11;
        for (uint32_t w = 0; w < n_warps; w++) {
            uint32_t lo, hi;
            memcpy(&lo, woff_b + 4ull * (p * n_warps + w), 4);
            memcpy(&hi, woff_b + 4ull * (p * n_warps + w + 1), 4);
            if (lo != prev_end || hi < lo || hi > n_blocks) return 4;
            prev_end = hi;
            uint32_t last_bucket = 0;
            for (uint32_t b = lo; b < hi; b++) {
                uint32_t h;
                memcpy(&h, hdr_b + 4ull * b, 4);
                const uint32_t bucket = bucket_lo + (h >> 24);      /* the field counts from the partition's first bucket */
                if (bucket < bucket_lo || bucket >= bucket_hi || bucket < last_bucket) return 5;
                last_bucket = bucket;
                for (int lane = 0; lane < 32; lane++) {
                    const uint32_t rowf = (h >> (6 * (lane / 8))) & 63u;
                    for (int s = 0; s < 4; s++) {
                        uint32_t e;
                        memcpy(&e, ent_b + 4ull * (4ull * (32ull * b + (uint64_t)lane) + (uint64_t)s), 4);
                        const uint32_t col = e >> 17;
                        if (col >= (uint32_t)N && col < (uint32_t)N + 64u) continue;   /* "no entry": columns N .. N+63 */
                        if (col >= (uint32_t)N + 64u) return 7;
                        if (col < (uint32_t)n_out) return 7;          /* outlier columns have no entries here */
                        if (rowf == 63u || (int64_t)rowf >= r1 - r0) return 6;
                        const int64_t main_idx = (int64_t)bucket * 4096 + (int64_t)((e & 0x1FFu) << 3) + (lane % 8);
                        const int64_t res_idx = (e >> 9) & 0xFFu;
                        if (main_idx >= k1) return 8;
                        if (k2 > 0 ? res_idx >= k2 : res_idx != 0) return 8;
                        const int64_t at = (r0 + rowf) * Nc + ((int64_t)col - n_out);
                        if (idx1[at] != -1) return 9;
                        idx1[at] = (int32_t)main_idx;
                        idx2[at] = (int32_t)res_idx;
                        real++;
                    }
                }
            }
        }
    }
    if (prev_end != n_blocks) return 4;
    for (int64_t i = 0; i < R * Nc; i++)
        if (idx1[i] == -1) return 10;
    if (real != (uint64_t)head[14]) return 12;
    return 0;
}

/* ------------------------------------------------------------------ */
/* Size accounting                                                     */
/* ------------------------------------------------------------------ */

/* Codebook bits (App. C.2): (v0*k0 + v1*(k1+k2)) * 16. */
double oracle_codebook_bits(int32_t v, int32_t k1, int32_t k2, int32_t n_out, int32_t v0, int32_t k0)
{
    double e = (double)v * ((double)k1 + (double)(k2 > 0 ? k2 : 0));
    if (n_out > 0) e += (double)v0 * (double)k0;
    return e * 16.0;
}

/* Index bits actually stored for an M x N layer, without row padding:
 * ceil(M/v) * (N - n_out) * (b1 + b2) + ceil(M/v0) * n_out * b0  (App. C.2 with the
 * outlier term read as log2(k0)/v0 per weight). */
double oracle_index_bits_total(int32_t M, int32_t N, int32_t v, int32_t k1, int32_t k2,
                               int32_t n_out, int32_t v0, int32_t k0)
{
    double R = (double)((M + v - 1) / v);
    double bits = R * (double)(N - n_out) *
                  (double)(oracle_index_bits(k1) + (k2 > 0 ? oracle_index_bits(k2) : 0));
    if (n_out > 0) bits += (double)((M + v0 - 1) / v0) * (double)n_out * (double)oracle_index_bits(k0);
    return bits;
}

/* Equivalent bit width (Sec. 2.2): 16 / (16*M*N / (codebook bits + index bits)). */
double oracle_equivalent_bits(int32_t M, int32_t N, int32_t v, int32_t k1, int32_t k2,
                              int32_t n_out, int32_t v0, int32_t k0)
{
    double total = oracle_codebook_bits(v, k1, k2, n_out, v0, k0) +
                   oracle_index_bits_total(M, N, v, k1, k2, n_out, v0, k0);
    return total / ((double)M * (double)N);
}

double oracle_compression_ratio(int32_t M, int32_t N, int32_t v, int32_t k1, int32_t k2,
                                int32_t n_out, int32_t v0, int32_t k0)
{
    return 16.0 / oracle_equivalent_bits(M, N, v, k1, k2, n_out, v0, k0);
}

/* The same with `group num` independent main/residual codebooks (Sec. 3.1; Table of App. B with the
 * parameters of the published 2-bit models): the codebook term grows G-fold, the index term does not. */
double oracle_equivalent_bits_grouped(int32_t M, int32_t N, int32_t v, int32_t k1, int32_t k2,
                                      int32_t n_out, int32_t v0, int32_t k0, int32_t n_groups)
{
    double G = n_groups > 1 ? (double)n_groups : 1.0;
    double codebooks = G * (double)v * ((double)k1 + (double)(k2 > 0 ? k2 : 0)) * 16.0;
    if (n_out > 0) codebooks += (double)v0 * (double)k0 * 16.0;
    return (codebooks + oracle_index_bits_total(M, N, v, k1, k2, n_out, v0, k0)) / ((double)M * (double)N);
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
