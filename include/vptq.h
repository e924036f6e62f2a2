/*
 * vptq.h — C ABI of libvptq: the inference hot path of VPTQ (vector post-training
 * quantization) on NVIDIA B200 (sm_100a).
 *
 * The quantized weight format is the paper's (Sec. 2.2, Sec. 3.1, Sec. 3.2.2-3, App. C.1):
 *   - the weight W_hat is [M][N], M output features, N input features;
 *   - it is cut into length-v vectors that run down a column: vector row r of column n
 *     covers output rows r*v .. r*v+v-1 (Sec. 3.1: a quantized column is a stack of
 *     centroids; Algorithm 1 steps m = 0, V, 2V, ...);
 *   - every vector is stored as an index into a codebook of k1 centroids of length v
 *     (Sec. 2.2); with residual VQ a second index into a codebook of k2 centroids is
 *     stored and decoding sums the two centroids (Sec. 3.2.2);
 *   - n_outlier leading input columns are quantized separately with their own vector
 *     length v0 and codebook of k0 centroids, and have no residual stage (Sec. 3.2.3,
 *     App. C.1, Algorithm 2).
 * Not stated by the paper and fixed by this library: the per-channel scale and bias
 * (W_hat = t*scale + bias, FP32, three separately rounded operations add, multiply, add),
 * the bit-packed index stream below, and "outlier columns come first".
 *
 * Packed index stream.  An index matrix I[rows][cols] with values in [0,k) uses
 * b = max(1, ceil(log2 k)) bits per index.  Each row is its own little-endian bit
 * stream: index c occupies stream bits [c*b, c*b+b); stream bit i is bit (i%8) of
 * byte (i/8).  A row occupies ceil(cols*b/8) bytes rounded up to a multiple of 16; pad
 * bits are zero.  b = 8 is a plain uint8 array, b = 16 a plain little-endian uint16 array.
 *
 * Conventions, unless an entry point says otherwise:
 *   - every data pointer is a DEVICE pointer owned by the caller and must be 16-byte
 *     aligned; the library allocates nothing and keeps no state between calls;
 *   - `stream` is a cudaStream_t passed as void*; calls are asynchronous on it.  It must belong to
 *     the CURRENT device, and so must every pointer: launch plans (grid sizes, row splits, scratch
 *     needs and so the answers of the *_workspace_bytes queries) follow the current device's SM count,
 *     and vptq_linear_noalloc takes the current device's copy of its built-in scratch;
 *   - the return value is 0 (VPTQ_OK) or a negative VPTQ_E_* code; nothing throws,
 *     aborts or traps.  vptq_status_string() names a code; vptq_last_cuda_error()
 *     gives the CUDA runtime's text for the last VPTQ_E_CUDA on this thread.
 */
#ifndef VPTQ_H_
#define VPTQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VPTQ_OK              0
#define VPTQ_E_NULL         -1   /* a required pointer is null                              */
#define VPTQ_E_SHAPE        -2   /* M,N,v,k <= 0, k > 65536, v > 32, n_outlier > N, B <= 0, n_groups < 0 or > N - n_outlier */
#define VPTQ_E_ALIGN        -3   /* a data pointer is not 16-byte aligned                   */
#define VPTQ_E_UNSUPPORTED  -4   /* dtype / flag combination without a kernel               */
#define VPTQ_E_WORKSPACE    -5   /* workspace missing or smaller than the query says        */
#define VPTQ_E_INDEX_RANGE  -6   /* vptq_pack found an index outside [0,k)                  */
#define VPTQ_E_CUDA         -7   /* a CUDA runtime call failed                              */
#define VPTQ_E_TIMEOUT      -8   /* a bounded device-side wait gave up (status word)        */
#define VPTQ_E_SCRATCH_LIMIT -9  /* vptq_linear_noalloc: layer needs more than the built-in scratch */

#define VPTQ_DTYPE_FP16 0
#define VPTQ_DTYPE_BF16 1
#define VPTQ_DTYPE_FP32 2

#define VPTQ_FLAG_SCALE_BIAS   1  /* scale and bias are present                                     */
#define VPTQ_FLAG_SCALE_ROWS   2  /* scale/bias are per OUTPUT row ([M]) instead of per input column */
#define VPTQ_FLAG_FORCE_GENERIC 4 /* use the plain fallback kernels (for testing them)               */
#define VPTQ_FLAG_COL_PERM      8 /* the layer has a stored column order (vptq_layer_ptrs.col_perm)   */
#define VPTQ_FLAG_PREPARED     16 /* vptq_layer_ptrs.prepared holds a prepared image (see vptq_prepare) */
#define VPTQ_FLAG_DETERMINISTIC 64 /* two calls with the same inputs give bit-identical outputs (see vptq_linear)  */
#define VPTQ_FLAG_CONCURRENT   32 /* the call may share the GPU with other work (other streams, other processes,
                                     fewer SMs than the device reports): no CTA waits for another CTA of its grid */

/* Geometry of one quantized linear layer (App. C.1 names: v1,k1,k2 / N%,v0,k0). */
typedef struct vptq_layer_desc {
    int32_t M, N;        /* out_features, in_features: W_hat is [M][N]                       */
    int32_t v;           /* main vector length (1..32)                                       */
    int32_t k1;          /* main codebook size (1..65536)                                    */
    int32_t k2;          /* residual codebook size, 0 = no residual stage                    */
    int32_t n_outlier;   /* columns [0,n_outlier) use the outlier codebook; 0 = none         */
    int32_t v0, k0;      /* outlier vector length / codebook size (ignored if n_outlier = 0) */
    int32_t x_dtype;     /* VPTQ_DTYPE_FP16 or _BF16                                         */
    int32_t out_dtype;   /* VPTQ_DTYPE_FP16, _BF16 or _FP32                                  */
    int32_t flags;       /* VPTQ_FLAG_*                                                      */
    int32_t n_groups;    /* Sec. 3.1: the non-outlier columns are split into this many equal runs of
                            consecutive columns (ceil((N-n_outlier)/n_groups) each, the last one
                            shorter), each with main/residual codebooks of its own; 0 or 1 = one   */
    int32_t prepared_parts; /* with VPTQ_FLAG_PREPARED: the n_parts the image was built with (the number of
                            CTAs that work on the layer); ignored without the flag                   */
} vptq_layer_desc;

/* The format pointers of a layer, in the order of the paper's format statement.
 *   packed_idx       packed [ceil(M/v)][N-n_outlier], b(k1) bits       (required unless n_outlier == N)
 *   codebook         fp16 [n_groups][k1][v]                             (required unless n_outlier == N)
 *   res_idx          packed, same shape, b(k2) bits                     (required iff k2 > 0)
 *   res_codebook     fp16 [n_groups][k2][v]                             (required iff k2 > 0)
 *   outlier_idx      packed [ceil(M/v0)][n_outlier], b(k0) bits         (required iff n_outlier > 0)
 *   outlier_codebook fp16 [k0][v0]                                      (required iff n_outlier > 0)
 *   scale, bias      fp16 [N] (or [M] with VPTQ_FLAG_SCALE_ROWS)        (required iff VPTQ_FLAG_SCALE_BIAS)
 *   col_perm         int32 [N], a permutation of 0..N-1                 (required iff VPTQ_FLAG_COL_PERM)
 *   prepared         image written by vptq_prepare, 256-byte aligned    (required iff VPTQ_FLAG_PREPARED)
 * A pointer that is not required may be null and is never read.
 *
 * col_perm is the stored column order.  The quantizer picks the outlier columns where the Hessian
 * diagonal is largest (Sec. 3.2.3; Algorithm 2 "selects outlier columns"), so they lie anywhere in the
 * matrix, while the format keeps them in front: stored column j (an outlier column for j < n_outlier)
 * is input feature col_perm[j], i.e. W_hat[m][col_perm[j]] = value restored for stored column j, and
 * vptq_linear multiplies stored column j with x[t][col_perm[j]].  scale and bias (per input column)
 * follow the stored order.  Without the flag the order is the identity.  Entries outside [0,N) are clamped to N-1 on the
 * device (like indices beyond a codebook), never dereferenced out of bounds; a list that is not a
 * permutation gives a well-defined but meaningless result. */
typedef struct vptq_layer_ptrs {
    const uint8_t *packed_idx;
    const void    *codebook;
    const uint8_t *res_idx;
    const void    *res_codebook;
    const uint8_t *outlier_idx;
    const void    *outlier_codebook;
    const void    *scale;
    const void    *bias;
    const int32_t *col_perm;
    const void    *prepared;   /* prepared image (device), required iff VPTQ_FLAG_PREPARED */
} vptq_layer_ptrs;

/* ---- format arithmetic (host only, no CUDA call) ---------------------------------- */

/* b = max(1, ceil(log2 k)): bits per index; the index-bit terms log2(k)/v of App. C.2
 * are b/v.  Returns VPTQ_E_SHAPE for k outside [1,65536]. */
int vptq_index_bits(int32_t k);
/* Bytes of one packed row / of the whole packed matrix (16-byte row padding included).
 * Negative (VPTQ_E_SHAPE) on bad arguments. */
int64_t vptq_packed_row_bytes(int32_t n_cols, int32_t k);
int64_t vptq_packed_bytes(int32_t n_rows, int32_t n_cols, int32_t k);
/* Bytes the format of a layer occupies, each stream/table counted once: packed index
 * streams + codebooks (App. C.2 "Codebook bits"/8) + scale and bias.  This is the
 * numerator of "effective weight GB/s". */
int64_t vptq_layer_weight_bytes(const vptq_layer_desc *desc);

/* ---- pack / unpack (boundary steps, not on the timed path) ------------------------ */

/* Pack idx[n_rows][n_cols] (int32, device) into the stream format (device, size
 * vptq_packed_bytes).  Every byte of `packed`, padding included, is written.
 * `bad_count` (device int32, may be null) receives the number of indices outside
 * [0,k); when it is non-null the call synchronises the stream, reads it back and
 * returns VPTQ_E_INDEX_RANGE if it is non-zero (such indices are stored as 0). */
int vptq_pack(const int32_t *idx, int32_t n_rows, int32_t n_cols, int32_t k,
              uint8_t *packed, int32_t *bad_count, void *stream);
/* Inverse of vptq_pack: idx[n_rows][n_cols] (int32, device) from the packed stream,
 * read with 128-bit loads.  Bit-exact inverse for every valid stream. */
int vptq_unpack(const uint8_t *packed, int32_t n_rows, int32_t n_cols, int32_t k,
                int32_t *idx, void *stream);

/* The same two steps on HOST memory, for callers that prepare or inspect a checkpoint on the CPU (the
 * paper does not describe a stream format; this is the format statement at the top of this file applied
 * by plain host code, no CUDA call, synchronous).  idx and packed are host pointers of any alignment.
 * vptq_pack_host writes every byte of `packed` (padding included), stores 0 for an index outside [0,k)
 * and then returns VPTQ_E_INDEX_RANGE; vptq_unpack_host never reads past a row's ceil(cols*b/8) bytes.
 * Byte for byte the streams of vptq_pack / vptq_unpack. */
int vptq_pack_host(const int32_t *idx, int32_t n_rows, int32_t n_cols, int32_t k, uint8_t *packed);
int vptq_unpack_host(const uint8_t *packed, int32_t n_rows, int32_t n_cols, int32_t k, int32_t *idx);

/* ---- dequantisation (Sec. 2.2 "dequantizes the weight matrix from the lookup table by
 *      index and centroid"; Sec. 3.2.2 decode; Sec. 3.2.3; App. D.2 "restore to FP16") -- */

/* W_out[M][N] fp16 (device, row-major) = the restored weight:
 *   n <  n_outlier: t = C0[I0[m/v0][n]][m%v0]
 *   n >= n_outlier: t = C1[I1[m/v][c]][m%v] (+ C2[I2[m/v][c]][m%v]), c = n - n_outlier,
 *                   C1/C2 = the tables of column group c / ceil((N-n_outlier)/n_groups)
 *   W = fp16_rne( fp32(fp32(t*scale) + bias) ) when VPTQ_FLAG_SCALE_BIAS, else fp16(t).
 * Bit-exact by definition (no fused multiply-add, denormals kept).  Indices >= k in a
 * corrupt stream are clamped to k-1, never read out of range. */
int vptq_dequant(const vptq_layer_desc *desc, const vptq_layer_ptrs *p,
                 void *W_out, void *stream);

/* ---- the fused linear layer (App. D.2: dequantisation fused with the product so the
 *      FP16 weight is never written to or read from global memory) ------------------ */

/* Scratch bytes vptq_linear needs for this layer at batch B (0 is possible).  The
 * caller allocates at least this much, 256-byte aligned; contents on entry are
 * irrelevant and undefined on exit.  Negative VPTQ_E_* on a bad descriptor. */
int64_t vptq_linear_workspace_bytes(const vptq_layer_desc *desc, int32_t B);

/* out[B][M] = x[B][N] * W_hat^T, W_hat as defined at vptq_dequant (without the final
 * FP16 rounding of W_hat; FP32 accumulation; the result differs from the FP64 product
 * over the FP16-rounded weights by at most ~1e-3 of max|out|).
 *   x    [B][N] row-major, desc->x_dtype;  out [B][M] row-major, desc->out_dtype.
 * B <= 16 runs the split-K decode kernels; larger B runs the tensor-core path
 * (tcgen05) when the layer qualifies (v = 8, k1 > 8192, x bf16/fp16), otherwise the
 * decode kernels over groups of 16 tokens.  Calls on one stream are ordered; calls
 * on different streams must not share a workspace.
 * The tensor-core path splits the input dimension of some output tiles over CTAs.  With long shares the CTA
 * that holds a tile's last piece stores it and raises a flag, and the CTAs that hold the other pieces wait for
 * that flag (bounded: about two seconds, then VPTQ_E_TIMEOUT in the status word) before they add theirs.  That
 * is only live while every CTA of the grid (one per SM of the current device) is resident at once, i.e. while
 * the call has the GPU to itself.  A call that may overlap other GPU work — another stream, another process, an
 * SM limit — must set VPTQ_FLAG_CONCURRENT: the output is then cleared first and every piece is added, and no
 * CTA waits for another (a few percent slower).
 * Run-to-run differences: the fast kernels combine partial sums with atomic additions, whose order is not
 * fixed, so two calls with the same inputs may differ in the last bits (well inside the tolerance).  With
 * VPTQ_FLAG_DETERMINISTIC every sum is formed in a fixed order: layers on the path "decode_l2_fma" keep their
 * kernel (row-owner mode, warp partial sums kept apart and added in warp order), the batched path gives every
 * CTA whole output tiles (no split of the input dimension), prepared images are not used, and every other
 * layer takes the plain fallback kernel (one warp per output row), which is several times slower. */
int vptq_linear(const vptq_layer_desc *desc, const void *x, int32_t B,
                const vptq_layer_ptrs *p, void *out,
                void *workspace, size_t workspace_bytes, void *stream);

/* Several layers that read the SAME activations in one call (the q/k/v projections of an attention
 * block, the gate/up projections of an MLP; the paper's decode loop, App. D.2, runs them one after
 * the other): out_l = x * W_hat_l^T for l < n_layers <= VPTQ_MAX_FUSED_LAYERS.
 *   descs, ptrs  host arrays of n_layers descriptors / pointer sets; all layers have the same N and
 *                x_dtype (else VPTQ_E_SHAPE); M, codebooks, scale/bias and out_dtype are per layer
 *   outs         host array of n_layers DEVICE pointers, outs[l] = [B][M_l] row-major
 * When every layer takes the same one of the decode paths "decode_l2_fma" (B <= 16), "decode_smem_fma"
 * or "decode_gl_fma" (B <= 4; for these two the layers must also share their format apart from M: v,
 * codebook sizes, outlier columns, groups, scale flag) and whole vector rows of the layers spread evenly
 * over the SMs, one kernel per token group serves all layers (no launch, prologue and ragged tail per
 * layer; no scratch); otherwise the layers run one after the other on `stream`, sharing the workspace.
 * vptq_linear_fused_path() names which: "fused_decode_l2_fma", "fused_decode_smem_fma",
 * "fused_decode_gl_fma" or "one_by_one" ("invalid" for arguments the call would reject).  Each layer's
 * result is the one vptq_linear gives for it (same arithmetic, same summation order within a vector
 * row).  Errors as for vptq_linear; nothing is launched when an argument is rejected. */
#define VPTQ_MAX_FUSED_LAYERS 4
int64_t vptq_linear_fused_workspace_bytes(const vptq_layer_desc *descs, int32_t n_layers, int32_t B);
int vptq_linear_fused(const vptq_layer_desc *descs, const vptq_layer_ptrs *ptrs, int32_t n_layers,
                      const void *x, int32_t B, void *const *outs,
                      void *workspace, size_t workspace_bytes, void *stream);
const char *vptq_linear_fused_path(const vptq_layer_desc *descs, int32_t n_layers, int32_t B);
/* Number of kernels one vptq_linear_fused call launches. */
int vptq_linear_fused_launches(const vptq_layer_desc *descs, int32_t n_layers, int32_t B);

/* Same product with HOST activations and HOST result: copies x_host -> x_dev, runs
 * vptq_linear, copies out_dev -> out_host, all asynchronously on `stream` (the caller
 * synchronises the stream before reading out_host).  x_host/out_host should be pinned
 * host memory; x_dev ([B][N]) and out_dev ([B][M]) are caller-owned device staging
 * buffers.  The weights (p) stay resident on the device.  Pinned activations of at most 256 KB are
 * brought over by a small kernel that reads x_host through the device's address of that buffer (it
 * starts sooner on the stream than a copy); larger or pageable ones by cudaMemcpyAsync.  On the path "decode_bucket_fma", whose
 * kernel stores every output element exactly once, a pinned out_host is written by the kernel
 * itself (through the device's address of that buffer) and out_dev is left untouched: the result
 * crosses the bus once either way, without a copy queued behind the kernel. */
int vptq_linear_host_io(const vptq_layer_desc *desc, const void *x_host, int32_t B,
                        const vptq_layer_ptrs *p, void *out_host,
                        void *x_dev, void *out_dev,
                        void *workspace, size_t workspace_bytes, void *stream);

/* vptq_linear_fused with HOST activations and HOST results: one copy of x_host -> x_dev, the fused
 * call, one copy outs_dev[l] -> outs_host[l] per layer, all asynchronous on `stream` (on the path
 * "fused_decode_bucket_fma" with all outs_host pinned, the kernel writes them itself, as above). */
int vptq_linear_fused_host_io(const vptq_layer_desc *descs, const vptq_layer_ptrs *ptrs, int32_t n_layers,
                              const void *x_host, int32_t B, void *const *outs_host,
                              void *x_dev, void *const *outs_dev,
                              void *workspace, size_t workspace_bytes, void *stream);

/* ---- prepared layer image: the index streams re-ordered for the decode kernel --------------- */

/* Decoding a layer whose main codebook has 65536 entries costs one random 16-byte read of a 1 MiB table per
 * index, and on B200 the rate of such reads out of L2, not HBM, bounds the decode kernels.  The paper's own
 * cache argument (App. C.2: lookups are fast while the table fits the first-level cache) is the way out: a
 * PREPARED IMAGE holds the same (main index, residual index) pairs as the two canonical streams, re-ordered
 * so that the kernel can keep one 4096-entry slice of the main codebook (a "bucket", 64 KB) in shared memory
 * at a time and read every centroid from there.  The image is derived data: it is built once per layer from
 * the canonical streams (vptq_prepare), it can be rebuilt at any time, and the canonical streams stay the
 * interchange format (vptq_dequant and the other paths keep using them).  The paper has no counterpart.
 *
 * Eligible layers: v = 8 with any k1 <= 65536, or v < 8 with k1 <= 4096 (one bucket, which the kernel widens
 * to 16-byte rows itself); k2 = 0 or k2 <= 256; outlier columns with v0 <= 8 (they stay on their canonical
 * stream: the image holds the main columns' entries only); one codebook group; per-input-column scale/bias
 * or none; N <= 31680.  "Vector row" below means v consecutive output rows, R = ceil(M/v) of them.
 *
 * Format (version 2; all fields little-endian; the image is 256-byte aligned):
 *   bytes 0..255  header, uint32 words: [0] 0x42515056 ("VPQB")  [1] version = 2  [2] M  [3] N  [4] k1  [5] k2
 *                 [6] n_parts  [7] n_warps = 31  [8] n_buckets = ceil(k1 / 4096)  [9] n_blocks
 *                 [10] byte offset of woff  [11] byte offset of hdr  [12] byte offset of entries (each a
 *                 multiple of 256)  [13] total bytes  [14] number of real entries = R * (N - n_outlier)
 *                 [15] n_split  [16] v  [17] n_outlier; rest zero
 *   partitions    a partition is the work of one CTA.  The R vector rows are cut into
 *            groups = n_parts / n_split row groups of R / groups rows, the first R % groups of them one row
 *            longer (group g starts at row g * (R / groups) + min(g, R % groups)), at most 63 rows; the
 *            n_split partitions of a group (p = g*n_split + h) each hold the group's entries of one range of
 *            buckets, [n_buckets*h/n_split, n_buckets*(h+1)/n_split).  n_split is the largest of 8, 4, 2, 1
 *            that divides n_parts, does not exceed n_buckets and keeps a group within 63 rows: a CTA then
 *            brings in only its range of the main codebook, and has more rows' work per bucket to hide that
 *            transfer behind.  The CTAs of a group add their partial sums up through the workspace.
 *   woff     uint32 [n_parts * n_warps + 1]: warp w of partition p owns blocks [woff[p*n_warps + w],
 *            woff[p*n_warps + w + 1])
 *   hdr      uint32 [n_blocks]: bits 24..31 = bucket of the block, counted from the first bucket of the
 *            partition's range; bits 6q..6q+5 (q = 0..3) = vector row,
 *            relative to the partition's first row, that the lanes 8q..8q+7 work on in this block, or 63
 *            when those lanes have nothing to do in it.  Buckets ascend within a warp's range and stay
 *            within the partition's range.
 *   entries  uint32 [n_blocks + 2][32][4]: a block is four steps of a warp; the four entries of lane L in block
 *            b are the words 4*(32*b + L) .. + 3; the last two blocks are spare (zero, owned by no warp: a
 *            reader may fetch two blocks ahead of any block without a bound check).  An entry:
 *              bits 0..8    (main index mod 4096) >> 3; the three low bits of the main index are L mod 8
 *                           (so the eight lanes of a quarter warp always read eight different 16-byte banks)
 *                           and its high bits are the block's bucket
 *              bits 9..16   residual index (0 when k2 = 0)
 *              bits 17..31  stored column n of the weight (n_outlier <= n < N: main column n - n_outlier of
 *                           the canonical streams), or one of N .. N+63 for "no entry" (padding; the
 *                           kernel keeps a zero activation for each of these, one per shared-memory bank
 *                           and half word, and the builder names the one whose bank the step's other
 *                           lanes leave free)
 * Every (vector row, main column) pair of the layer occurs exactly once among the entries that are not padding,
 * in a quarter whose header field names that row.
 *
 * vptq_prepare_bytes: capacity to allocate for the image of this layer split into n_parts partitions
 *   (0 = one per SM of the current device): the header and tables plus 4 bytes x 1.5 x the number of
 *   entries.  VPTQ_E_UNSUPPORTED for a layer that is not eligible, or n_parts too small for the 63-row limit
 *   (with the n_split the rule above gives).
 * vptq_prepare_host: packed_idx / res_idx are HOST copies of the canonical streams, `image` is host memory
 *   of `image_bytes` bytes; plain host code, no CUDA call.  *used_bytes (may be null) receives the size of
 *   the image.  VPTQ_E_WORKSPACE when the image does not fit image_bytes: with index histograms far from
 *   uniform (one centroid taking a large share of the vectors) the bank rule above forces much padding, and
 *   such a layer is better left on the canonical streams.
 * vptq_prepare: the same from DEVICE streams into a DEVICE image: copies the streams to the host, builds the
 *   image there and copies it back.  Synchronous; allocates temporary HOST memory; a set-up step, not on
 *   the timed path.
 * Use: set VPTQ_FLAG_PREPARED in desc->flags, desc->prepared_parts to the image's n_parts and
 * vptq_layer_ptrs.prepared to the image.  vptq_linear then takes the path "decode_bucket_fma" for B = 1 when
 * n_parts does not exceed the SM count (other batch sizes use the canonical streams, which must still be
 * valid), and vptq_linear_fused serves prepared layers of one format (N, activation type, residual stage)
 * whose n_parts sum to at most the SM count with one launch ("fused_decode_bucket_fma"); layers meant to
 * share a launch are therefore prepared with n_parts that add up to the SM count (multiples of 4 or 8 where
 * the rows allow, so that n_split can exceed 1).  The path asks for a workspace (vptq_linear_workspace_bytes:
 * 256 bytes, plus 4 bytes and a 2 KB block of partial sums per CTA when an image has n_split > 1) whose
 * first int32 is a status word (vptq_workspace_status): the kernel compares the image header with the
 * descriptor and writes VPTQ_E_UNSUPPORTED there when they disagree (the outputs are then not written), or
 * VPTQ_E_TIMEOUT when a bounded wait gave up.  Unlike the other paths this one needs the WHOLE workspace
 * zero when it is first used: the status word is only ever written on an error and never cleared, and the
 * arrival counters behind it (one per row group; the last CTA to count itself in adds the group's partial
 * sums up in partition order and stores, so no CTA waits for another and the result does not depend on
 * which one was last) are left at zero by every launch that ends without an error.  Consecutive calls
 * therefore need nothing between their kernels: clear the workspace once when it is allocated and after
 * reading an error.  An image that vptq_prepare did not write is outside the contract (its header's sizes
 * are trusted). */
#define VPTQ_PREPARED_MAGIC 0x42515056u
int64_t vptq_prepare_bytes(const vptq_layer_desc *desc, int32_t n_parts);
int vptq_prepare_host(const vptq_layer_desc *desc, const uint8_t *packed_idx, const uint8_t *res_idx,
                      int32_t n_parts, void *image, size_t image_bytes, size_t *used_bytes);
int vptq_prepare(const vptq_layer_desc *desc, const vptq_layer_ptrs *p, int32_t n_parts,
                 void *image, size_t image_bytes, size_t *used_bytes, void *stream);

/* ---- the same product for callers that cannot allocate device memory ---------------- */

/* The paper has no counterpart to this entry point; it exists for integration reasons only.
 *
 * Who needs it: code that runs where a device allocation is not an option — an engine
 * that handed all device memory to its own arena at start-up and gives plug-in operators
 * no way to ask for more, or a latency-critical serving loop in which cudaMalloc (which
 * may synchronise the whole device) is forbidden after initialisation.  vptq_linear
 * asks such a caller for a workspace it cannot provide; this variant brings its own.
 *
 * What it does: the split-K decode kernel of vptq_linear (main codebook in global memory,
 * i.e. v = 8, 16-bit indices, optional 8-bit residual indices, no outlier columns,
 * per-input-column scale/bias) for 1 <= B <= 16, with the FP32 partial-sum scratch taken
 * from an array of VPTQ_NOALLOC_SCRATCH_BYTES that is compiled into the library.  Every GPU
 * that loads the library holds that array until the process exits.  Inputs and outputs
 * are the caller's, exactly as for vptq_linear; the result agrees with vptq_linear's to
 * FP32 summation order.  The call itself allocates nothing: no cudaMalloc, no cudaFree,
 * no allocating library routine.
 *
 * Limits and errors: layers of another geometry return VPTQ_E_UNSUPPORTED.  The kernel
 * needs scratch only when the layer's vector rows do not divide well over the SMs (it then
 * deals the work out regardless of rows and adds partial sums up in scratch): 4 * g * M bytes, g the
 * tokens per launch (4 for B >= 4, 2 for B = 2 or 3, else 1), plus a few KB of counters.  A layer whose need exceeds the array returns
 * VPTQ_E_SCRATCH_LIMIT (M up to about 65000 fits at any B); nothing is launched in either
 * case.  vptq_linear_workspace_bytes() tells the need of a given layer and B.
 *
 * Set-up: the first call on each device looks up the array's device address (with that
 * device current) and remembers it; make that first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same array, and it keeps whatever the previous
 * call left in it.  Each call clears, on `stream`, the part that must start at zero, so
 * back-to-back calls on one stream are safe; two calls that overlap on the GPU (different
 * streams, or different threads without ordering) race on the array and give wrong
 * results. */
#define VPTQ_NOALLOC_SCRATCH_BYTES (1 << 20)
int vptq_linear_noalloc(const vptq_layer_desc *desc, const void *x, int32_t B,
                        const vptq_layer_ptrs *p, void *out, void *stream);

/* ---- the quantizer's assignment step -------------------------------------------------- */

/* Eq. 2: idx[r][n] = argmin_i || W[r*v .. r*v+v-1][n] - C_i ||^2 for every length-v vector of the
 * weight matrix (v consecutive rows of one column: Sec. 3.1, Algorithm 1), i.e. the index matrix that
 * vptq_pack packs and vptq_dequant looks up again.  (With a Hessian-weighted objective the weight of a
 * vector's column is common to all its distances and does not change the argmin: Sec. 3.2.1 moves the
 * weights into the k-means centroid update: vptq_kmeans_update below.)
 *   W        fp16 [M][N] row-major (device)      codebook  fp16 [k][v] (device)
 *   idx      int32 [ceil(M/v)][N] (device, written)
 * Arithmetic, fixed because it decides an integer: FP32, components in ascending order,
 * d = fma(t, t, d) with t = x_j - c_j; of equal distances the lowest index wins; a NaN distance never
 * wins (all NaN: index 0); components beyond row M-1 (short last vector row) are left out.
 * Two kernels give these same indices: "assign_fp32" evaluates the definition for every pair;
 * "assign_tcgen05" (v <= 14, v divides M, k >= 1024, at least 4096 vectors) computes
 * ||c||^2 - 2 x.c on the tensor cores only to find, per vector, the group of 32 centroids that holds
 * the minimum, evaluates that group by the definition, and hands every vector whose candidate group is
 * not clearly the only one (within a bound on the tensor core's rounding) to the first kernel.
 * vptq_assign_path() names the kernel; VPTQ_FLAG_FORCE_GENERIC in `flags` selects "assign_fp32".
 * The tensor-core kernel needs a workspace of vptq_assign_workspace_bytes() bytes (256-byte aligned;
 * its first int32 is a status word read by vptq_workspace_status()); the other needs none.
 * 1 <= v <= 32, 1 <= k <= 65536, else VPTQ_E_SHAPE / VPTQ_E_UNSUPPORTED.  Asynchronous on `stream`. */
const char *vptq_assign_path(int32_t M, int32_t N, int32_t v, int32_t k, int32_t flags);
int64_t vptq_assign_workspace_bytes(int32_t M, int32_t N, int32_t v, int32_t k, int32_t flags);
int vptq_assign(const void *W, int32_t M, int32_t N, int32_t v, const void *codebook, int32_t k,
                int32_t *idx, int32_t flags, void *workspace, size_t workspace_bytes, void *stream);

/* Centroid update of (weighted) k-means (Sec. 2.2: k-means builds the codebook; Sec. 3.2.1: the diagonal
 * term of the proxy error is a weighted k-means problem, the weight of a vector being the Hessian
 * diagonal of its column): with the assignment `idx` fixed,
 *   codebook[i][j] = sum h_n x_j / sum h_n   over the vectors (r, n) with idx[r][n] = i that have
 * component j (x = W[r*v + j][n], h_n = col_weight[n], or 1 when col_weight is null); a component that
 * received no weight keeps its old value, an index outside [0,k) takes no part.  vptq_assign followed
 * by this call is one Lloyd iteration.
 *   W fp16 [M][N], idx int32 [ceil(M/v)][N], col_weight fp32 [N] or null, codebook fp16 [k][v]
 *   (read and written), workspace of vptq_kmeans_update_workspace_bytes(v, k) bytes (all device).
 * Sums are FP32 atomics: the result agrees with the FP64 weighted mean to FP32 summation error (then
 * rounded to FP16), not bit for bit, and may differ from run to run in the last FP16 bit. */
int64_t vptq_kmeans_update_workspace_bytes(int32_t v, int32_t k);
int vptq_kmeans_update(const void *W, int32_t M, int32_t N, int32_t v, const int32_t *idx,
                       const float *col_weight, int32_t k, void *codebook,
                       void *workspace, size_t workspace_bytes, void *stream);

/* ---- diagnostics ------------------------------------------------------------------ */

const char *vptq_status_string(int code);
const char *vptq_last_cuda_error(void);
/* Three paths — vptq_linear on "gemm_tcgen05" and on "decode_bucket_fma" (prepared images), and vptq_assign on
 * "assign_tcgen05" — keep an int32 status word at byte 0 of their workspace; after any other call the workspace holds no status and
 * this call has no meaning.  It synchronises `stream`, reads the word and returns VPTQ_E_TIMEOUT if a
 * bounded device-side wait gave up during the call (the output is then invalid; the context stays
 * usable), VPTQ_E_UNSUPPORTED if the prepared-image kernel refused its image, else VPTQ_OK.  A null
 * workspace returns VPTQ_OK. */
int vptq_workspace_status(const void *workspace, void *stream);
/* For tests of the error path: the kernels' device-side waits (on mbarriers and flags) give up after about
 * two seconds; this sets the limit, in SM clock cycles, for the kernels launched afterwards by any thread
 * (0 restores the default).  With a limit of a few cycles a healthy kernel abandons its first wait that is
 * not already satisfied, reports VPTQ_E_TIMEOUT in its status word, leaves no copy in flight and returns;
 * the context stays usable.  Honoured by the path "decode_bucket_fma".  Process-wide; not for production. */
void vptq_debug_set_wait_limit(uint64_t cycles);
/* 1 when the kernels of vptq_linear for (desc, B) let one CTA wait for a flag that another CTA of the same grid
 * raises, 0 when no CTA waits for another, negative VPTQ_E_* on bad arguments.  Only the batched path does this
 * (see vptq_linear), and VPTQ_FLAG_CONCURRENT switches it off. */
int vptq_linear_waits_between_ctas(const vptq_layer_desc *desc, int32_t B);
/* Name of the kernel family vptq_linear picks for (desc, B): "generic", "decode_smem_fma",
 * "decode_smem_mma", "decode_l2_fma", "decode_gl_fma", "gemm_tcgen05", "decode_bucket_fma".  For tests and
 * benchmark logs. */
const char *vptq_linear_path(const vptq_layer_desc *desc, int32_t B);
/* Number of kernels one vptq_linear call launches (scratch memsets are not counted). */
int vptq_linear_launches(const vptq_layer_desc *desc, int32_t B);

#ifdef __cplusplus
}
#endif
#endif /* VPTQ_H_ */
