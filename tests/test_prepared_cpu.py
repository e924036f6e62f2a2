"""The prepared layer image (the re-ordered index streams the batch-1 decode kernel reads): the library's host
builder against the oracle's own decoder, written from the format statement in include/vptq.h.  No GPU."""
import ctypes as C

import numpy as np
import pytest

from oracle import oracle
from paper_2409_17066_b200 import build as vbuild


@pytest.fixture(scope="module")
def b():
    vbuild.build()
    from paper_2409_17066_b200 import binding
    return binding


def _layer(b, M, N, k1, k2, seed, flags=None, v=8, n_out=0):
    rng = np.random.default_rng(seed)
    R = -(-M // v)
    idx1 = rng.integers(0, k1, (R, N - n_out), dtype=np.int32)
    idx2 = rng.integers(0, k2, (R, N - n_out), dtype=np.int32) if k2 else None
    desc = b.make_desc(M, N, v, k1, k2, n_outlier=n_out, v0=4 if n_out else 0, k0=4096 if n_out else 0,
                       flags=b.FLAG_SCALE_BIAS if flags is None else flags)
    return desc, idx1, idx2


@pytest.mark.parametrize("M,N,v,k1,k2,n_out,n_parts", [
    (1100, 420, 6, 4096, 256, 0, 7),      # vectors of 6 (184 vector rows, the last one ragged), 12-bit main indices
    (1100, 420, 6, 4096, 256, 5, 7),      # the same with 5 outlier columns stored first
    (512, 300, 8, 4096, 0, 3, 4),         # v = 8, one bucket, outlier columns, no residual stage
    (260, 200, 4, 1000, 100, 0, 3),       # vectors of 4, 10-bit main and 7-bit residual indices
    (520, 300, 8, 30000, 256, 2, 8),      # 15-bit main indices, 8 buckets (the last one short), two splits
])
def test_other_formats_decode_back(b, M, N, v, k1, k2, n_out, n_parts):
    desc, idx1, idx2 = _layer(b, M, N, k1, k2, seed=M + N + v, v=v, n_out=n_out)
    image = b.vptq_prepare_host(desc, oracle.pack(idx1, k1), oracle.pack(idx2, k2) if k2 else None, n_parts)
    code, got1, got2 = oracle.decode_prepared(image, M, N, k1, k2, v=v, n_out=n_out)
    assert code == 0
    assert np.array_equal(got1, idx1)
    assert np.array_equal(got2, idx2 if k2 else np.zeros_like(idx1))
    head = image[:72].view(np.uint32)
    assert head[14] == idx1.size and head[16] == v and head[17] == n_out
    # the decoder is told the layer's v and outlier count: other values are a geometry mismatch
    assert oracle.decode_prepared(image, M, N, k1, k2, v=v, n_out=n_out + 1)[0] == 2
    if n_out:
        # an entry that names an outlier column is refused
        off_ent, n_blocks = int(head[12]), int(head[9])
        ent = image[off_ent:off_ent + 512 * n_blocks].view(np.uint32)
        j = int(np.flatnonzero((ent >> 17) < N)[0])
        img = image.copy()
        img[off_ent + 4 * j:off_ent + 4 * j + 4].view(np.uint32)[0] = int(ent[j]) & 0x1FFFF
        assert oracle.decode_prepared(img, M, N, k1, k2, v=v, n_out=n_out)[0] == 7


@pytest.mark.parametrize("M,N,k1,k2,n_parts,n_split", [
    (520, 300, 65536, 256, 7, 1),       # ragged last vector row, several partitions
    (264, 1030, 65536, 256, 33, 1),     # one vector row per partition
    (1024, 256, 65536, 0, 3, 1),        # no residual stage; 43 rows in a partition
    (400, 200, 40000, 200, 5, 1),       # 10 buckets, the last one short; a residual table of 200 entries
    (64, 64, 33000, 256, 1, 1),         # nine buckets, the last one short; a single partition
    (2048, 128, 65536, 256, 148, 4),    # 37 row groups of 6 or 7 rows, four bucket ranges each
    (520, 300, 65536, 256, 8, 4),       # 65 rows: one group of 8 partitions would exceed 63 rows, two groups of 4
    (400, 200, 40000, 200, 8, 8),       # one row group; 10 buckets over 8 partitions (one or two each)
    (1024, 96, 65536, 0, 6, 2),         # three row groups, two bucket ranges each
])
def test_image_decodes_back_to_the_index_matrices(b, M, N, k1, k2, n_parts, n_split):
    desc, idx1, idx2 = _layer(b, M, N, k1, k2, seed=M + N)
    p1 = oracle.pack(idx1, k1)
    p2 = oracle.pack(idx2, k2) if k2 else None
    image = b.vptq_prepare_host(desc, p1, p2, n_parts)
    assert image.size <= b.vptq_prepare_bytes(desc, n_parts) and image.size % 256 == 0
    code, got1, got2 = oracle.decode_prepared(image, M, N, k1, k2)
    assert code == 0
    assert np.array_equal(got1, idx1)
    assert np.array_equal(got2, idx2 if k2 else np.zeros_like(idx1))
    head = image[:64].view(np.uint32)
    assert head[6] == min(n_parts, -(-M // 8)) and head[14] == idx1.size and head[15] == n_split
    # padding stays moderate with uniform indices (bank rule: a quarter warp's 8 lanes take 8 residues mod 8)
    slots = int(head[9]) * 128
    assert slots >= idx1.size
    # the builder is a function of its inputs: the same call gives the same bytes
    assert np.array_equal(image, b.vptq_prepare_host(desc, p1, p2, n_parts))


def test_decoder_names_the_broken_rule(b):
    # mistakes planted in a good image are each reported under their own rule
    M, N, k1, k2 = 264, 300, 65536, 256
    desc, idx1, idx2 = _layer(b, M, N, k1, k2, seed=5)
    image = b.vptq_prepare_host(desc, oracle.pack(idx1, k1), oracle.pack(idx2, k2), 4)
    assert oracle.decode_prepared(image, M, N, k1, k2)[0] == 0
    head = image[:64].view(np.uint32)
    off_woff, off_hdr, off_ent, n_blocks = int(head[10]), int(head[11]), int(head[12]), int(head[9])

    def broken(edit):
        img = image.copy()
        edit(img)
        return oracle.decode_prepared(img, M, N, k1, k2)[0]

    assert broken(lambda im: im[:4].view(np.uint32).__setitem__(0, 0x12345678)) == 1
    assert oracle.decode_prepared(image, M + 8, N, k1, k2)[0] == 2
    assert broken(lambda im: im[40:44].view(np.uint32).__setitem__(0, off_woff + 4)) == 3
    assert broken(lambda im: im[off_woff + 8:off_woff + 12].view(np.uint32).__setitem__(0, n_blocks + 5)) == 4
    ent = image[off_ent:off_ent + 512 * n_blocks].view(np.uint32)
    real = np.flatnonzero((ent >> 17) < N)
    e0 = int(real[0])

    def set_entry(im, i, val):
        im[off_ent + 4 * i:off_ent + 4 * i + 4].view(np.uint32)[0] = val

    assert broken(lambda im: set_entry(im, e0, (int(ent[e0]) & 0x1FFFF) | ((N + 64) << 17))) == 7
    assert broken(lambda im: set_entry(im, e0, int(ent[int(real[1])]))) in (9, 10)        # a pair twice, another missing
    assert broken(lambda im: set_entry(im, e0, N << 17)) == 10                             # an entry turned into padding
    blk = e0 // 128
    hdr = image[off_hdr:off_hdr + 4 * n_blocks].view(np.uint32)

    def set_hdr(im, i, val):
        im[off_hdr + 4 * i:off_hdr + 4 * i + 4].view(np.uint32)[0] = val

    q = (e0 % 128) // 4 // 8
    assert broken(lambda im: set_hdr(im, blk, int(hdr[blk]) | (63 << (6 * q)))) == 6
    assert broken(lambda im: set_hdr(im, blk, (int(hdr[blk]) & 0xFFFFFF) | (200 << 24))) == 5
    # the image has one row group and four bucket ranges: a bucket of another partition's range is refused too
    assert head[15] == 4
    elsewhere = ((int(hdr[blk]) >> 24) + 8) % 16
    assert broken(lambda im: set_hdr(im, blk, (int(hdr[blk]) & 0xFFFFFF) | (elsewhere << 24))) == 5
    assert broken(lambda im: im[60:64].view(np.uint32).__setitem__(0, 3)) == 2             # a split that does not divide 4
    # a residual index beyond the table
    assert oracle.decode_prepared(image, M, N, k1, 256)[0] == 0
    d2, i1, i2 = _layer(b, M, N, k1, 200, seed=6)
    img2 = b.vptq_prepare_host(d2, oracle.pack(i1, k1), oracle.pack(i2, 200), 4)
    e = img2.copy()
    h2 = e[:64].view(np.uint32)
    ent2 = e[int(h2[12]):int(h2[12]) + 512 * int(h2[9])].view(np.uint32)
    j = int(np.flatnonzero((ent2 >> 17) < N)[0])
    ent2[j] = (int(ent2[j]) & ~(0xFF << 9)) | (250 << 9)
    assert oracle.decode_prepared(e, M, N, k1, 200)[0] == 8


def test_indices_beyond_the_codebook_are_clamped_like_everywhere_else(b):
    # k1 = 40000 uses 16-bit indices: values 40000..65535 can occur in a corrupt stream; they become k1 - 1
    M, N, k1 = 64, 96, 40000
    desc = b.make_desc(M, N, 8, k1, 0)
    idx1 = np.full((8, N), 65535, np.int32)
    image = b.vptq_prepare_host(desc, oracle.pack(idx1, 65536), None, 2)
    code, got1, _ = oracle.decode_prepared(image, M, N, k1, 0)
    assert code == 0 and np.all(got1 == k1 - 1)


def test_skewed_histograms_do_not_fit_and_say_so(b):
    # every vector takes the same centroid: one lane of eight does all the work, the image would be ~8x larger
    M, N, k1 = 1024, 2048, 65536
    desc = b.make_desc(M, N, 8, k1, 0)
    idx1 = np.full((128, N), 12345, np.int32)
    cap = b.vptq_prepare_bytes(desc, 4)
    image = np.empty(cap, np.uint8)
    used = C.c_size_t(0)
    p1 = oracle.pack(idx1, k1)
    rc = b.lib.vptq_prepare_host(C.byref(desc), p1.ctypes.data, None, 4, image.ctypes.data, cap, C.byref(used))
    assert rc == b.E_WORKSPACE and used.value > cap
    # with room for it the image is still right
    big = b.vptq_prepare_host(desc, p1, None, 4, capacity=used.value)
    code, got1, _ = oracle.decode_prepared(big, M, N, k1, 0)
    assert code == 0 and np.array_equal(got1, idx1)


def test_eligibility_and_argument_errors(b):
    ok = b.make_desc(4096, 4096, 8, 65536, 256)
    assert b.vptq_prepare_bytes(ok, 148) > 4 * 512 * 4096
    assert b.vptq_prepare_bytes(ok, 0) > 0                                   # one partition per SM
    for good in (b.make_desc(4096, 4096, 8, 4096, 256),                      # one bucket
                 b.make_desc(4096, 4096, 8, 30000, 256),                     # 15-bit main indices
                 b.make_desc(4096, 4096, 6, 4096, 256),                      # shorter vectors, one bucket
                 b.make_desc(4096, 4096, 8, 65536, 256, n_outlier=41, v0=4, k0=4096)):
        assert b.vptq_prepare_bytes(good, 148) > 0
    for bad in (b.make_desc(4096, 4096, 6, 65536, 256),                      # v = 6 with more than one bucket
                b.make_desc(4096, 4096, 8, 65536, 4096),                     # 12-bit residual indices
                b.make_desc(4096, 4096, 8, 65536, 256, n_outlier=41, v0=12, k0=4096),
                b.make_desc(4096, 4096, 8, 65536, 256, n_groups=4),
                b.make_desc(4096, 40000, 8, 65536, 256)):                    # N beyond the staged activations
        assert b.lib.vptq_prepare_bytes(C.byref(bad), 148) == b.E_UNSUPPORTED
    assert b.lib.vptq_prepare_bytes(C.byref(ok), 4) == b.E_UNSUPPORTED       # 128 rows per partition > 63
    assert b.lib.vptq_prepare_bytes(C.byref(ok), -1) == b.E_SHAPE
    img = np.empty(1024, np.uint8)
    assert b.lib.vptq_prepare_host(C.byref(ok), None, None, 148, img.ctypes.data, 1024, None) == b.E_NULL
    # a prepared descriptor needs its image and its partition count
    prep = b.make_desc(4096, 4096, 8, 65536, 256, flags=b.FLAG_SCALE_BIAS | b.FLAG_PREPARED, prepared_parts=148)
    assert b.vptq_linear_path(prep, 1) == "decode_bucket_fma"
    assert b.vptq_linear_path(prep, 2) == "decode_l2_fma"                    # other batch sizes read the canonical streams
    # 512 vector rows over 148 CTAs: 37 row groups of four bucket ranges; a counter and 2 KB of sums per CTA
    assert b.vptq_linear_workspace_bytes(prep, 1) == 256 + 768 + 148 * 2048
    odd = b.make_desc(4096, 4096, 8, 65536, 256, flags=b.FLAG_SCALE_BIAS | b.FLAG_PREPARED, prepared_parts=147)
    assert b.vptq_linear_workspace_bytes(odd, 1) == 256                      # no split: the status word only
    noparts = b.make_desc(4096, 4096, 8, 65536, 256, flags=b.FLAG_SCALE_BIAS | b.FLAG_PREPARED)
    assert b.lib.vptq_linear_workspace_bytes(C.byref(noparts), 1) == b.E_SHAPE
    p = b.LayerPtrs(0x1000, 0x1000, 0x1000, 0x1000, None, None, 0x1000, 0x1000, None, None)
    assert b.lib.vptq_linear(C.byref(prep), 0x1000, 1, C.byref(p), 0x1000, 0x1000, 256, None) == b.E_NULL
    # gate and up prepared for half of the SMs each share a launch
    g = b.make_desc(28672, 8192, 8, 65536, 256, flags=b.FLAG_SCALE_BIAS | b.FLAG_PREPARED, prepared_parts=74)
    assert b.vptq_linear_fused_path([g, g], 1) == "fused_decode_bucket_fma"
    assert b.vptq_linear_fused_launches([g, g], 1) == 1 and b.vptq_linear_fused_workspace_bytes([g, g], 1) == 256
    full = b.make_desc(28672, 8192, 8, 65536, 256, flags=b.FLAG_SCALE_BIAS | b.FLAG_PREPARED, prepared_parts=148)
    assert b.vptq_linear_fused_path([full, full], 1) == "one_by_one"         # 296 partitions do not fit side by side


def test_cta_shares_of_layers_that_share_a_launch(b):
    # q/k/v of the 70B shape: multiples of four, so that every image splits its buckets over four CTAs per row group
    assert b.prepared_shares([1024, 128, 128], 148) == [116, 16, 16]
    # gate/up: 48 or 49 rows per CTA leave no room for a split; the SMs are halved
    assert b.prepared_shares([3584, 3584], 148) == [74, 74]
    # a one-bucket codebook cannot be split whatever the rows would allow
    assert b.prepared_shares([1835, 1835], 148, n_buckets=1) == [74, 74]
    for rows, n_sm, nb in (([125, 65, 33], 148, 16), ([512, 512, 512], 148, 16), ([7, 900], 132, 16), ([40, 40, 40, 40], 148, 2)):
        shares = b.prepared_shares(rows, n_sm, nb)
        assert len(shares) == len(rows) and sum(shares) <= n_sm and all(1 <= s <= r for s, r in zip(shares, rows))
        # what the library makes of them: every image within the 63-row limit, i.e. vptq_prepare_bytes accepts it
        for r, s_ in zip(rows, shares):
            d = b.make_desc(8 * r, 256, 8, 4096 * nb, 0)
            assert b.vptq_prepare_bytes(d, s_) > 0
