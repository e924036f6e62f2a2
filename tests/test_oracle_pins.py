"""Pins for the CPU oracle: each test checks it against something that is not itself —
values the paper prints, closed forms, library routines, a separately written numpy
statement, or brute force on tiny layers.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest

from oracle import mini, oracle
from paper_2409_17066_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


# ---------------------------------------------------------------- converters

def test_half_to_float_exhaustive_vs_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_float_to_half_vs_numpy():
    rng = np.random.default_rng(1)
    # every half value, the midpoints between neighbours, and values a hair off the midpoints
    h = np.arange(0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mids = (h[:-1] + h[1:]) / 2
    cand = np.concatenate([h, mids, np.nextafter(mids.astype(np.float32), np.float32(np.inf)),
                           np.nextafter(mids.astype(np.float32), np.float32(-np.inf)),
                           [65504.0, 65519.99, 65520.0, 65536.0, 1e9, 2.0 ** -24, 2.0 ** -25,
                            np.nextafter(np.float32(2.0 ** -25), np.float32(1)), 2.0 ** -26, 1e-30, 0.0],
                           rng.normal(0, 1, 20000), rng.normal(0, 1e-5, 20000),
                           rng.uniform(-70000, 70000, 20000)]).astype(np.float32)
    cand = np.concatenate([cand, -cand])
    with np.errstate(over="ignore"):
        ref = cand.astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_to_half(float(c)) for c in cand], dtype=np.uint16)
    assert np.array_equal(got, ref)


def _bf16_by_exact_arithmetic(f: np.float32) -> int:
    """Round-to-nearest-even to 8 significant bits, with Python's exact rationals (no bit tricks)."""
    from fractions import Fraction
    f = float(f)
    if f == 0.0:
        return 0x8000 if np.signbit(f) else 0
    sign = 0x8000 if f < 0 else 0
    a = Fraction(abs(f))
    e = int(np.floor(np.log2(float(a))))
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)                                  # subnormal floats share the exponent of 2^-126
    q = a / Fraction(2) ** (e - 7)                    # in units of the last kept bit
    n = int(q)                                        # floor
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    val = Fraction(n) * Fraction(2) ** (e - 7)
    if val >= Fraction(2) ** 128:
        return sign | 0x7F80
    got = np.float32(float(val))                      # exactly representable: 8 bits
    return sign | int(np.array([got], np.float32).view(np.uint32)[0] >> 16)


def test_bf16_converters():
    rng = np.random.default_rng(2)
    f = np.concatenate([rng.normal(0, 1, 3000), rng.normal(0, 1e-20, 100), rng.normal(0, 1e-39, 100),
                        [0.0, 1.0, 3.0e38]]).astype(np.float32)
    # ties: exactly halfway between two bf16 values
    ties = ((rng.integers(0, 2 ** 15, 1000).astype(np.uint32) << 16) | 0x8000).view(np.float32)
    ties = ties[np.isfinite(ties)]
    f = np.concatenate([f, ties, -ties[:100]])
    got = np.array([oracle.float_to_bf16(float(v)) for v in f], dtype=np.uint16)
    want = np.array([_bf16_by_exact_arithmetic(v) for v in f], dtype=np.uint16)
    assert np.array_equal(got, want)
    # the shared input generator rounds the same way (it feeds both sides of the parity tests)
    assert np.array_equal(synth.to_bf16_bits(f), want)
    # a bf16 is the top half of the float: round trip is exact, and widening matches the bit shift
    back = np.array([oracle.bf16_to_float(int(b)) for b in got], dtype=np.float32)
    assert np.array_equal(back.view(np.uint32), got.astype(np.uint32) << 16)
    # values written out by hand
    u = lambda bits: float(np.array([bits], np.uint32).view(np.float32)[0])
    assert oracle.float_to_bf16(1.0 + 2.0 ** -8) == 0x3F80          # tie, lower neighbour even: down
    assert oracle.float_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82      # tie, upper neighbour even: up
    assert oracle.float_to_bf16(-(1.0 + 3 * 2.0 ** -8)) == 0xBF82
    assert oracle.float_to_bf16(u(0x3F808001)) == 0x3F81            # a hair above a tie: up
    assert oracle.float_to_bf16(u(0x3F817FFF)) == 0x3F81            # a hair below a tie: down
    assert oracle.float_to_bf16(u(0x7F7F0000)) == 0x7F7F            # the largest finite bf16 stays
    assert oracle.float_to_bf16(u(0x7F7F7FFF)) == 0x7F7F            # just below the last tie: still finite
    assert oracle.float_to_bf16(u(0x7F7F8000)) == 0x7F80            # the last tie rounds to even = infinity
    assert oracle.float_to_bf16(u(0x7F7FFFFF)) == 0x7F80            # FLT_MAX overflows to +inf
    assert oracle.float_to_bf16(u(0xFF7FFFFF)) == 0xFF80
    assert oracle.float_to_bf16(float("inf")) == 0x7F80 and oracle.float_to_bf16(float("-inf")) == 0xFF80
    assert oracle.float_to_bf16(-0.0) == 0x8000
    for nan_bits in (0x7FC00000, 0x7F800001, 0xFFC00000, 0x7FFFFFFF, 0x7F80FFFF):
        b = oracle.float_to_bf16(u(nan_bits))                       # a NaN stays a NaN (never becomes inf)
        assert (b & 0x7F80) == 0x7F80 and (b & 0x007F) != 0, hex(nan_bits)


# ---------------------------------------------------------------- packed stream

def test_pack_hand_computed_12bit():
    # 2 x 5 matrix at b = 12 (k = 4096).  Row stream is little-endian: index c sits in bits [12c, 12c+12).
    idx = np.array([[0xABC, 0x123, 0xFFF, 0x000, 0x801],
                    [0x001, 0x800, 0x00F, 0xF00, 0x0F0]], dtype=np.int32)
    # row 0 bits: 0xABC | 0x123<<12 | 0xFFF<<24 | 0<<36 | 0x801<<48  -> bytes little-endian
    v0 = 0xABC | (0x123 << 12) | (0xFFF << 24) | (0x000 << 36) | (0x801 << 48)
    v1 = 0x001 | (0x800 << 12) | (0x00F << 24) | (0xF00 << 36) | (0x0F0 << 48)
    exp = np.zeros((2, 16), dtype=np.uint8)
    exp[0, :8] = np.frombuffer(v0.to_bytes(8, "little"), dtype=np.uint8)
    exp[1, :8] = np.frombuffer(v1.to_bytes(8, "little"), dtype=np.uint8)
    # spelled out for row 0: BC 3A 12 FF 0F 00 01 08
    assert list(exp[0, :8]) == [0xBC, 0x3A, 0x12, 0xFF, 0x0F, 0x00, 0x01, 0x08]
    got = oracle.pack(idx, 4096)
    assert got.shape == (2, 16)
    assert np.array_equal(got, exp)
    assert np.array_equal(mini.pack(idx, 4096), exp)


def test_pack_plain_widths_are_plain_arrays():
    rng = np.random.default_rng(3)
    idx = rng.integers(0, 256, size=(3, 32), dtype=np.int32)
    assert np.array_equal(oracle.pack(idx, 256), idx.astype(np.uint8))
    idx = rng.integers(0, 65536, size=(3, 16), dtype=np.int32)
    assert np.array_equal(oracle.pack(idx, 65536).view("<u2"), idx.astype(np.uint16))


@pytest.mark.parametrize("b", list(range(1, 17)))
@pytest.mark.parametrize("cols", [1, 7, 41, 257, 4055])
def test_pack_unpack_round_trip(b, cols):
    k = 1 << b if b > 1 else 2
    if b == 1:
        ks = [1, 2]
    else:
        ks = [k, (1 << (b - 1)) + 1]          # power of two and the smallest k that needs b bits
    rng = np.random.default_rng(100 * b + cols)
    for kk in ks:
        assert oracle.index_bits(kk) == b == mini.index_bits(kk)
        for idx in (rng.integers(0, kk, size=(3, cols), dtype=np.int32),
                    np.zeros((2, cols), np.int32), np.full((2, cols), kk - 1, np.int32)):
            p = oracle.pack(idx, kk)
            assert p.shape[1] % 16 == 0 and p.shape[1] == mini.row_bytes(cols, kk)
            assert p.shape[1] - (cols * b + 7) // 8 < 16
            assert np.array_equal(oracle.unpack(p, idx.shape[0], cols, kk), idx)
            assert np.array_equal(p, mini.pack(idx, kk))
            assert np.array_equal(mini.unpack(p, idx.shape[0], cols, kk), idx)


def test_pack_rejects_out_of_range():
    with pytest.raises(ValueError):
        oracle.pack(np.array([[0, 5]], np.int32), 5)
    with pytest.raises(ValueError):
        oracle.pack(np.array([[-1, 0]], np.int32), 5)


# ---------------------------------------------------------------- size accounting (paper's numbers)

def test_worked_example_ratio_and_bits():
    (M, N, v, k, ratio, bits), = _rows("size_worked_example.txt")
    M, N, v, k = int(M), int(N), int(v), int(k)
    assert round(oracle.compression_ratio(M, N, v, k), 2) == float(ratio)
    assert round(oracle.equivalent_bits(M, N, v, k), 3) == float(bits)
    # and the packed stream really has that many index bits: log2(k)/v per weight
    assert oracle.packed_bytes(M // v, N, k) * 8 == M * N * np.log2(k) / v


def _block_bits(v, k1, k2, pct, v0, k0, G=1, H=5120, F=13824):
    layers = [(H, H)] * 4 + [(F, H), (F, H), (H, F)]
    bits = params = 0.0
    for (M, N) in layers:
        n_out = synth.outlier_columns(N, pct)
        if G == 1:
            bits += oracle.codebook_bits(v, k1, k2, n_out, v0, k0) + \
                oracle.index_bits_total(M, N, v, k1, k2, n_out, v0, k0)
        else:
            bits += oracle.equivalent_bits_grouped(M, N, v, k1, k2, n_out, v0, k0, G) * M * N
        params += M * N
    return bits / params


def test_ablation_table_bit_column():
    seen_grouped = 0
    for row, bit, pct, v0, k0, v1, k1, k2, pin, G in _rows("ablation_bits.txt"):
        got = _block_bits(int(v1), int(k1), max(int(k2), 0), float(pct), int(v0), int(k0), int(G))
        decimals = len(bit.split(".")[1]) if "." in bit else 0
        if pin == "1":
            assert round(got, decimals) == float(bit), (row, got, bit)
        else:
            assert 0 <= float(bit) - got <= 0.015, (row, got, bit)
        seen_grouped += int(G) > 1
    assert seen_grouped == 3            # rows #15-#17 (group num 2, 4, 8) pin the grouped size formula
    # the grouped rows come out only with codebooks per group: one shared codebook misses #17 by 0.24 bit
    assert abs(_block_bits(12, 4096, 4096, 1.0, 4, 4096, 1) - 2.3) > 0.2
    # and the two size routines agree where both apply (one group)
    assert oracle.equivalent_bits_grouped(5120, 13824, 12, 4096, 4096, 138, 4, 4096, 1) == \
        oracle.equivalent_bits(5120, 13824, 12, 4096, 4096, 138, 4, 4096)


def test_codebook_overhead_and_outlier_bits():
    g = dict((k, float(v)) for k, v in _rows("codebook_overhead.txt"))
    params = 4 * 5120 * 5120 + 3 * 5120 * 13824
    over = 7 * oracle.codebook_bits(8, 65536) / params
    assert round(over, 2) in (g["codebook_overhead_v8_k65536"], round(g["codebook_overhead_v8_k65536"] - 0.01, 2))
    assert oracle.index_bits(4096) / 4 == g["outlier_index_bits_v4_k4096"]
    assert oracle.index_bits(4096) / 6 == g["main_index_bits_v6_k4096"]


def test_measured_packed_size_matches_index_bit_formula():
    # App. C.2: average index bits = log2(k1)/v1 + log2(k2)/v1; outlier part log2(k0)/v0.
    for cfg in (1, 2, 3, 4):
        for s in synth.CONFIGS[cfg]["layers"]:
            stored = oracle.packed_bytes(s.R, s.Nc, s.k1) * 8
            if s.k2:
                stored += oracle.packed_bytes(s.R, s.Nc, s.k2) * 8
            if s.n_out:
                stored += oracle.packed_bytes(s.R0, s.n_out, s.k0) * 8
            main = (np.log2(s.k1) + (np.log2(s.k2) if s.k2 else 0)) / s.v
            formula = main * s.M * s.Nc
            if s.n_out:
                formula += np.log2(s.k0) / s.v0 * s.M * s.n_out
            # padding only: ceil(M/v) rows and < 16 bytes per row and stream
            pad_rows = (s.R * s.v - s.M) * s.Nc * main
            pad_bytes = 16 * 8 * (s.R * (2 if s.k2 else 1) + s.R0)
            assert formula <= stored <= formula + pad_rows + pad_bytes
            assert stored / (s.M * s.N) - formula / (s.M * s.N) < 0.01


# ---------------------------------------------------------------- lookup: closed forms and special cases

def _layer(d, **kw):
    return oracle.Layer.from_synth(d, **kw)


def test_single_codebook_no_scale_is_pure_gather():
    spec = synth.LayerSpec("g", 40, 33, v=8, k1=256, has_scale=False)
    d = synth.make_layer(spec, 90, 0, 1)
    W = _layer(d).dequant()
    for m, n in itertools.product(range(spec.M), range(spec.N)):
        assert W[m, n].view(np.uint16) == d["c1"][d["idx1"][m // 8, n], m % 8].view(np.uint16)


def test_k1_closed_form():
    # one centroid: W[m][n] = s[n]*C[0][m%v] + b[n];  y[t][m] = C[0][m%v]*sum(x s) + sum(x b) up to the FP16 rounding of W
    spec = synth.LayerSpec("k1", 21, 64, v=4, k1=1)
    d = synth.make_layer(spec, 91, 0, 3)
    L = _layer(d)
    W = L.dequant()
    c = d["c1"][0].astype(np.float32)
    exp = ((c[np.arange(21) % 4][:, None] * d["scale"].astype(np.float32)[None, :]).astype(np.float32)
           + d["bias"].astype(np.float32)[None, :]).astype(np.float16)
    assert np.array_equal(W.view(np.uint16), exp.view(np.uint16))
    assert oracle.packed_bytes(spec.R, spec.N, 1) == spec.R * 16   # one (wasted) bit per index
    y = L.linear(d["x"])
    x = d["x"].astype(np.float64)
    closed = (x @ d["scale"].astype(np.float64))[:, None] * c.astype(np.float64)[np.arange(21) % 4][None, :] \
        + (x @ d["bias"].astype(np.float64))[:, None]
    assert np.max(np.abs(y - closed)) <= 2.0 ** -11 * np.sum(np.abs(x), axis=1).max() * 0.05


def test_identity_codebook_is_a_histogram():
    # C = I_8: restored W[r*8+j][n] = 1 if I[r][n] == j else 0, so y is a sum of x over matching columns
    v = 8
    spec = synth.LayerSpec("id", 48, 100, v=v, k1=8, has_scale=False)
    d = synth.make_layer(spec, 92, 0, 2)
    d["c1"] = np.eye(8, dtype=np.float16)
    y = _layer(d).linear(d["x"])
    x = d["x"].astype(np.float64)
    exp = np.zeros((2, 48))
    for r in range(6):
        for n in range(100):
            exp[:, r * 8 + d["idx1"][r, n]] += x[:, n]
    assert np.allclose(y, exp, rtol=0, atol=1e-12)


def test_v1_integer_matmul_is_exact():
    spec = synth.LayerSpec("v1", 17, 23, v=1, k1=256, has_scale=False)
    d = synth.make_layer(spec, 93, 0, 2)
    d["c1"] = (np.arange(256, dtype=np.float32) / 256).astype(np.float16).reshape(256, 1)
    d["x"] = np.random.default_rng(5).integers(-8, 9, size=(2, 23)).astype(np.float16)
    L = _layer(d)
    assert np.array_equal(L.dequant().astype(np.float64) * 256, d["idx1"].astype(np.float64))
    y = L.linear(d["x"])
    exp = d["x"].astype(np.int64) @ d["idx1"].astype(np.int64).T
    assert np.array_equal(y * 256, exp.astype(np.float64))


def test_residual_special_cases():
    spec = synth.LayerSpec("r", 32, 40, v=8, k1=256, k2=256)
    d = synth.make_layer(spec, 94, 0, 1)
    single = dict(d, spec=synth.LayerSpec("r1", 32, 40, v=8, k1=256), c2=None, idx2=None)
    # C2 = 0 : same as one codebook
    z = dict(d, c2=np.zeros_like(d["c2"]))
    assert np.array_equal(_layer(z).dequant().view(np.uint16), _layer(single).dequant().view(np.uint16))
    # C2 = -C1, I2 = I1 : the lookup sum cancels, W = bias exactly
    neg = dict(d, c2=(-d["c1"]), idx2=d["idx1"].copy())
    W = _layer(neg).dequant()
    assert np.array_equal(W.view(np.uint16), np.broadcast_to(d["bias"][None, :], W.shape).view(np.uint16))
    # a residual stage really adds: differs from the single-codebook result somewhere
    assert not np.array_equal(_layer(d).dequant().view(np.uint16), _layer(single).dequant().view(np.uint16))


def test_outlier_special_cases():
    base = synth.LayerSpec("o", 24, 30, v=8, k1=256, n_out=30, v0=4, k0=16)
    d = synth.make_layer(base, 95, 0, 1)
    # all columns outliers: equals a plain layer quantized with (v0, k0)
    plain = dict(d, spec=synth.LayerSpec("p", 24, 30, v=4, k1=16), c1=d["c0"], idx1=d["idx0"],
                 c0=None, idx0=None)
    d_all = dict(d, idx1=np.zeros((3, 0), np.int32))
    assert np.array_equal(_layer(d_all).dequant().view(np.uint16), _layer(plain).dequant().view(np.uint16))
    # mixed: outlier columns come from C0 only (no residual added there), the others from C1 + C2
    spec = synth.LayerSpec("m", 24, 30, v=8, k1=256, k2=16, n_out=5, v0=4, k0=16, has_scale=False)
    d = synth.make_layer(spec, 96, 0, 1)
    W = _layer(d).dequant()
    for m in range(24):
        for n in range(5):
            assert W[m, n].view(np.uint16) == d["c0"][d["idx0"][m // 4, n], m % 4].view(np.uint16)
        for n in range(5, 30):
            t = np.float32(d["c1"][d["idx1"][m // 8, n - 5], m % 8]) + np.float32(d["c2"][d["idx2"][m // 8, n - 5], m % 8])
            assert W[m, n].view(np.uint16) == np.float16(t).view(np.uint16)


def test_scale_axis_flag():
    spec = synth.LayerSpec("a", 16, 16, v=8, k1=256)
    d = synth.make_layer(spec, 97, 0, 1)
    W0 = _layer(d, scale_axis=0).dequant()
    W1 = _layer(d, scale_axis=1).dequant()
    assert np.array_equal(W0.view(np.uint16), mini.dequant_from_synth(d, 0).view(np.uint16))
    assert np.array_equal(W1.view(np.uint16), mini.dequant_from_synth(d, 1).view(np.uint16))
    assert not np.array_equal(W0.view(np.uint16), W1.view(np.uint16))


# ---------------------------------------------------------------- brute force and library routines

def test_all_index_combinations_tiny():
    # every index matrix of a 4 x 2 layer with v = 2, k = 3 (3^4 = 81 cases), against the numpy statement
    c1 = np.array([[0.5, -1.25], [2.0, 0.125], [-3.0, 7.0]], dtype=np.float16)
    scale = np.array([1.5, 0.75], np.float16)
    bias = np.array([0.01, -0.02], np.float16)
    x = np.array([[1.0, -2.0]], np.float16)
    for combo in itertools.product(range(3), repeat=4):
        idx = np.array(combo, np.int32).reshape(2, 2)
        L = oracle.Layer(4, 2, 2, 3, c1, oracle.pack(idx, 3), scale=scale, bias=bias)
        W = L.dequant()
        ref = mini.dequant(4, 2, 2, c1, idx, scale=scale, bias=bias)
        assert np.array_equal(W.view(np.uint16), ref.view(np.uint16))
        assert np.allclose(L.linear(x), mini.linear(ref, x.astype(np.float64)), rtol=0, atol=1e-12)


@pytest.mark.parametrize("spec", synth.small_specs(), ids=lambda s: s.name)
def test_small_layers_vs_numpy_statement(spec):
    for seed_layer in range(3):
        d = synth.make_layer(spec, 80, seed_layer, 3)
        L = _layer(d)
        W = L.dequant()
        ref = mini.dequant_from_synth(d)
        assert np.array_equal(W.view(np.uint16), ref.view(np.uint16))
        rows = np.array([0, spec.M - 1, spec.M // 2], np.int32)
        assert np.array_equal(L.dequant_rows(rows).view(np.uint16), ref[rows].view(np.uint16))
        # matmul step reduces to a library routine on the FP16 weights
        y = L.linear(d["x"])
        yr = mini.linear(ref, d["x"].astype(np.float64))
        assert np.max(np.abs(y - yr)) <= 1e-12 * max(1.0, np.max(np.abs(yr)))
        assert np.array_equal(L.linear(d["x"], rows), y[:, rows])


def test_bf16_activations():
    spec = synth.LayerSpec("b", 16, 40, v=8, k1=256, x_dtype="bf16")
    d = synth.make_layer(spec, 81, 0, 2)
    L = _layer(d)
    y = L.linear(d["x"])
    xr = synth.bf16_bits_to_f32(d["x"]).astype(np.float64)
    assert np.allclose(y, mini.linear(L.dequant(), xr), rtol=0, atol=1e-12)


def test_config0_and_ragged_v6_bits():
    # config 0 itself: 1.000 index bit per weight, 1.25 with its codebook
    s = synth.CONFIGS[0]["layers"][0]
    assert oracle.packed_bytes(s.R, s.N, s.k1) * 8 / (s.M * s.N) == 1.0
    assert oracle.equivalent_bits(s.M, s.N, s.v, s.k1) == 1.25
    # the outlier column counts used for the 1 % setting
    assert synth.outlier_columns(4096, 1.0) == 41 and synth.outlier_columns(11008, 1.0) == 110


# ---------------------------------------------------------------- group-wise codebooks (Sec. 3.1)

def test_group_codebook_bits_reproduce_the_published_settings():
    """The "bit" column of the App. B table with the parameters of the published 2-bit models:
    it only comes out when every column group carries codebooks of its own."""
    for model, h, f, kv, bit, pct, v0, k0, v, k1, k2, G in _rows("quant_args_bits.txt"):
        h, f, kv, v0, k0, v, k1, k2, G = map(int, (h, f, kv, v0, k0, v, k1, k2, G))
        linears = [(h, h), (kv, h), (kv, h), (h, h), (f, h), (f, h), (h, f)]
        bits = weights = 0.0
        for M, N in linears:
            n_out = synth.outlier_columns(N, float(pct))
            bits += oracle.equivalent_bits_grouped(M, N, v, k1, k2, n_out, v0, k0, G) * M * N
            weights += M * N
        assert abs(bits / weights - float(bit)) <= 0.011, (model, bit, bits / weights)
    # a single shared codebook would miss the grouped rows by far more than the rounding
    M = N = 4096
    one = oracle.equivalent_bits_grouped(M, N, 12, 4096, 4096, 41, 4, 8192, 1)
    four = oracle.equivalent_bits_grouped(M, N, 12, 4096, 4096, 41, 4, 8192, 4)
    assert four - one == pytest.approx(3 * 12 * 8192 * 16 / (M * N))


def test_groups_with_identical_codebooks_equal_one_codebook():
    spec1 = synth.LayerSpec("g1", 50, 90, v=6, k1=64, k2=16, n_out=5, v0=4, k0=32)
    d1 = synth.make_layer(spec1, 91, 0, 3)
    ref = oracle.Layer.from_synth(d1)
    for G in (2, 3, 7, 85):
        specG = synth.LayerSpec(**{**spec1.__dict__, "n_groups": G})
        dG = dict(d1, spec=specG, c1=np.tile(d1["c1"], (G, 1)), c2=np.tile(d1["c2"], (G, 1)))
        LG = oracle.Layer.from_synth(dG)
        assert np.array_equal(LG.dequant().view(np.uint16), ref.dequant().view(np.uint16))
        assert np.array_equal(LG.linear(d1["x"]), ref.linear(d1["x"]))


@pytest.mark.parametrize("G", [2, 3, 4, 16])
def test_grouped_layers_vs_numpy_statement_and_group_boundaries(G):
    spec = synth.LayerSpec("gg", 44, 101, v=12, k1=32, k2=8, n_out=3, v0=4, k0=16, n_groups=G)
    d = synth.make_layer(spec, 92, G, 2)
    L = oracle.Layer.from_synth(d)
    W = L.dequant()
    assert np.array_equal(W.view(np.uint16), mini.dequant_from_synth(d).view(np.uint16))
    # a column's weights come from its own group's tables: zeroing every other group's tables
    # must leave that group's columns untouched and change nothing but the others
    Nc = spec.N - spec.n_out
    cpg = -(-Nc // G)
    g = G // 2
    d0 = dict(d, c1=d["c1"].copy(), c2=d["c2"].copy())
    keep1 = np.zeros(G * spec.k1, bool); keep1[g * spec.k1:(g + 1) * spec.k1] = True
    keep2 = np.zeros(G * spec.k2, bool); keep2[g * spec.k2:(g + 1) * spec.k2] = True
    d0["c1"][~keep1] = 0
    d0["c2"][~keep2] = 0
    W0 = oracle.Layer.from_synth(d0).dequant()
    cols = spec.n_out + np.arange(g * cpg, min(Nc, (g + 1) * cpg))
    assert np.array_equal(W0[:, cols].view(np.uint16), W[:, cols].view(np.uint16))
    others = np.setdiff1d(np.arange(spec.n_out, spec.N), cols)
    bias = d["bias"].astype(np.float32)[others]
    assert np.array_equal(W0[:, others].astype(np.float32), np.broadcast_to(bias.astype(np.float16).astype(np.float32), (spec.M, others.size)))


# ---------------------------------------------------------------- outlier columns anywhere (Sec. 3.2.3)

def test_column_order_special_cases():
    # Sec. 3.2.3 / Algorithm 2: the quantizer selects the outlier columns, so the stored column order is
    # a list of input features.  Identity order: nothing changes.  Reversed order: the mirror image.
    spec = synth.LayerSpec("p", 24, 30, v=8, k1=256, k2=16, n_out=5, v0=4, k0=16)
    d = synth.make_layer(spec, 98, 0, 2)
    W = _layer(d).dequant()
    ident = dict(d, col_perm=np.arange(30, dtype=np.int32))
    assert np.array_equal(_layer(ident).dequant().view(np.uint16), W.view(np.uint16))
    assert np.array_equal(_layer(ident).linear(d["x"]), _layer(d).linear(d["x"]))
    rev = dict(d, col_perm=np.arange(29, -1, -1, dtype=np.int32))
    assert np.array_equal(_layer(rev).dequant().view(np.uint16), W[:, ::-1].view(np.uint16))
    # the first n_out STORED columns are the outlier columns: they land on the features the list names
    perm = np.random.default_rng(5).permutation(30).astype(np.int32)
    Wp = _layer(dict(d, col_perm=perm)).dequant()
    for j in range(30):
        assert np.array_equal(Wp[:, perm[j]].view(np.uint16), W[:, j].view(np.uint16))
    for m in range(24):
        for j in range(5):      # scale and bias follow the stored order
            t = np.float32(d["c0"][d["idx0"][m // 4, j], m % 4]) * np.float32(d["scale"][j])
            t = np.float32(t) + np.float32(d["bias"][j])
            assert Wp[m, perm[j]].view(np.uint16) == np.float16(t).view(np.uint16)


def test_column_order_is_a_reordering_of_the_activations():
    # y = sum_j x[perm[j]] * W_stored[:, j]: the permuted layer on x equals the plain layer on x[:, perm]
    spec = synth.LayerSpec("q", 40, 52, v=8, k1=256, k2=16, n_out=3, v0=4, k0=16, permuted=True)
    d = synth.make_layer(spec, 99, 0, 3)
    perm = d["col_perm"]
    assert sorted(perm.tolist()) == list(range(52))
    plain = {k: v for k, v in d.items() if k != "col_perm"}
    y = _layer(d).linear(d["x"])
    y_plain = _layer(plain).linear(np.ascontiguousarray(d["x"][:, perm]))
    assert np.max(np.abs(y - y_plain)) <= 1e-12 * np.max(np.abs(y_plain))
    assert np.max(np.abs(y - _layer(plain).linear(d["x"]))) > 1e-3      # and it does matter
    # matmul over the restored matrix (library routine)
    W = _layer(d).dequant()
    assert np.allclose(y, mini.linear(W, d["x"].astype(np.float64)), rtol=0, atol=1e-12)
    # a list that names a feature outside [0, N) is a corrupt layer
    bad = dict(d, col_perm=np.where(np.arange(52) == 7, 52, perm).astype(np.int32))
    with pytest.raises(ValueError):
        _layer(bad).dequant()
    with pytest.raises(ValueError):
        _layer(bad).linear(d["x"])


# ---------------------------------------------------------------- assignment step of the quantizer (Eq. 2)

def _dist64(W, v, C):
    """All squared distances in float64: [R][N][k] (M divisible by v)."""
    M, N = W.shape
    X = W.astype(np.float64).reshape(M // v, v, N).transpose(0, 2, 1)          # [R][N][v]
    return ((X[:, :, None, :] - C.astype(np.float64)[None, None, :, :]) ** 2).sum(axis=3)


def test_assign_is_the_nearest_centroid_brute_force():
    rng = np.random.default_rng(11)
    for v, k, M, N in ((8, 64, 32, 20), (6, 50, 36, 17), (2, 7, 10, 9), (12, 33, 24, 5), (1, 5, 6, 6)):
        W = rng.normal(0, 1, (M, N)).astype(np.float16)
        C = rng.normal(0, 1, (k, v)).astype(np.float16)
        idx = oracle.assign(W, v, C)
        D = _dist64(W, v, C)
        best = D.min(axis=2)
        chosen = np.take_along_axis(D, idx[:, :, None].astype(np.int64), axis=2)[:, :, 0]
        # the chosen centroid is a nearest one (FP32 rounding may only swap near-ties) ...
        assert np.all(chosen <= best * (1 + 1e-5) + 1e-12)
        # ... and THE nearest one wherever the runner-up is clearly farther
        second = np.partition(D, 1, axis=2)[:, :, 1]
        clear = second > best * (1 + 1e-4) + 1e-9
        assert clear.mean() > 0.9
        assert np.array_equal(idx[clear], D.argmin(axis=2)[clear])


def test_assign_special_cases():
    rng = np.random.default_rng(12)
    # every vector IS a centroid: the assignment returns it (distance 0), so assign(dequant(I)) = I
    C = rng.normal(0, 1, (40, 8)).astype(np.float16)
    I = rng.integers(0, 40, (5, 13)).astype(np.int32)
    W = mini.dequant(40, 13, 8, C, I)
    assert np.array_equal(oracle.assign(W, 8, C), I)
    # equal distances: the lowest index wins (a duplicated centroid; a point half way between two)
    C2 = np.concatenate([C[:3], C[:3], C[3:]])
    assert np.array_equal(oracle.assign(W, 8, C2), np.where(I >= 3, I + 3, I))
    mid = oracle.assign(np.zeros((2, 1), np.float16), 2, np.array([[1, 0], [-1, 0], [0, 1]], np.float16))
    assert mid.tolist() == [[0]]
    # v = 1 with a sorted grid of centroids: rounding to the nearest grid point (closed form)
    grid = np.arange(-4, 5, dtype=np.float16).reshape(9, 1)
    x = np.array([[-3.75, -0.25, 0.0, 0.26, 1.49, 1.51, 3.9, 7.0, -9.0]], np.float16)
    want = np.clip(np.rint(x.astype(np.float64)), -4, 4).astype(np.int32) + 4
    assert np.array_equal(oracle.assign(x, 1, grid), want)
    # k = 1: always index 0
    assert not oracle.assign(W, 8, C[:1]).any()


def test_assign_ragged_last_vector_row_ignores_missing_components():
    rng = np.random.default_rng(13)
    v, k, M, N = 8, 30, 21, 11                       # last vector row has 5 of 8 components
    W = rng.normal(0, 1, (M, N)).astype(np.float16)
    C = rng.normal(0, 1, (k, v)).astype(np.float16)
    idx = oracle.assign(W, v, C)
    assert idx.shape == (3, N)
    Wp = np.concatenate([W, np.zeros((3, N), np.float16)])
    assert np.array_equal(idx[:2], oracle.assign(Wp, v, C)[:2])
    # the short row is the assignment against the first 5 components of every centroid
    assert np.array_equal(idx[2:], oracle.assign(W[16:], 5, np.ascontiguousarray(C[:, :5])))
    # selected vectors only
    vec = np.array([0, N - 1, N, 2 * N + 3], np.int64)
    assert np.array_equal(oracle.assign(W, v, C, vec), idx.reshape(-1)[vec])


# ---------------------------------------------------------------- k-means centroid update (Sec. 3.2.1)

def test_kmeans_update_is_the_weighted_mean():
    rng = np.random.default_rng(21)
    v, k, M, N = 4, 6, 16, 9
    W = rng.normal(0, 1, (M, N)).astype(np.float16)
    C = rng.normal(0, 1, (k, v)).astype(np.float16)
    idx = rng.integers(0, k - 1, (M // v, N)).astype(np.int32)        # centroid k-1 gets no vector
    h = rng.uniform(0.1, 3.0, N).astype(np.float32)
    for weights in (None, h):
        new = oracle.kmeans_update(W, v, idx, C, weights)
        X = W.astype(np.float64).reshape(M // v, v, N).transpose(0, 2, 1)          # [R][N][v]
        hw = np.ones(N) if weights is None else weights.astype(np.float64)
        for i in range(k - 1):
            sel = idx == i
            wsel = np.broadcast_to(hw[None, :], idx.shape)[sel]
            want = (X[sel] * wsel[:, None]).sum(0) / wsel.sum()
            assert np.array_equal(new[i].view(np.uint16), want.astype(np.float32).astype(np.float16).view(np.uint16))
        assert np.array_equal(new[k - 1].view(np.uint16), C[k - 1].view(np.uint16))     # empty cluster: unchanged
    # one vector per centroid: the centroid becomes that vector, whatever its weight
    W1 = rng.normal(0, 1, (4, 5)).astype(np.float16)
    new = oracle.kmeans_update(W1, 4, np.arange(5, dtype=np.int32).reshape(1, 5), np.zeros((5, 4), np.float16), h[:5])
    assert np.array_equal(new.view(np.uint16), np.ascontiguousarray(W1.T).view(np.uint16))


def test_distortion_is_the_weighted_sum_of_squared_errors():
    """Sec. 3.2.1: sum over vectors of h_n * ||x - C_idx||^2, written out with numpy in float64 on a case
    with a ragged last vector row, with and without column weights, and a closed form."""
    rng = np.random.default_rng(31)
    v, k, M, N = 4, 7, 14, 9                                         # 14 = 3 * 4 + 2: the last row has 2 components
    W = rng.normal(0, 1, (M, N)).astype(np.float16)
    C = rng.normal(0, 1, (k, v)).astype(np.float16)
    R = -(-M // v)
    idx = rng.integers(0, k, (R, N)).astype(np.int32)
    h = rng.uniform(0.1, 4.0, N).astype(np.float32)
    W64, C64 = W.astype(np.float64), C.astype(np.float64)
    # restored matrix by fancy indexing, cut to the rows that exist
    What = C64[idx].transpose(0, 2, 1).reshape(R * v, N)[:M]          # [R][N][v] -> [R*v][N]
    col_err = ((W64 - What) ** 2).sum(axis=0)                         # per column
    plain, weighted = col_err.sum(), (col_err * h.astype(np.float64)).sum()
    assert oracle.distortion(W, v, idx, C, None) == pytest.approx(plain, rel=1e-13)
    assert oracle.distortion(W, v, idx, C, h) == pytest.approx(weighted, rel=1e-13)
    assert abs(weighted - plain) > 0.05 * plain                       # dropping the weights would show
    # the components of the short last row that do not exist are not counted: counting them would add
    # the squares of the centroids' last two components
    phantom = (C64[idx[R - 1]][:, M - (R - 1) * v:] ** 2).sum()
    assert phantom > 0.05 * plain
    assert abs(oracle.distortion(W, v, idx, C, None) - (plain + phantom)) > 0.04 * plain
    # a transposed operand would show: weights follow columns, not vector rows
    hr = np.resize(h, R).astype(np.float64)
    row_weighted = sum(hr[r] * ((W64 - What)[r * v:min(M, (r + 1) * v)] ** 2).sum() for r in range(R))
    assert abs(oracle.distortion(W, v, idx, C, h) - row_weighted) > 1e-3 * weighted
    # closed form: every vector equals its centroid plus d in every component -> h-weighted count * d^2
    C_exact = np.round(C64 * 4) / 4                                   # quarter steps: +0.5 stays exact in FP16
    Wc = (C_exact[idx].transpose(0, 2, 1).reshape(R * v, N)[:M] + 0.5).astype(np.float16)
    assert oracle.distortion(Wc, v, idx, C_exact.astype(np.float16), h) == \
        pytest.approx(0.25 * M * float(h.astype(np.float64).sum()), rel=1e-13)
    # zero distortion when every vector is its centroid
    Wz = C_exact[idx].transpose(0, 2, 1).reshape(R * v, N)[:M].astype(np.float16)
    assert oracle.distortion(Wz, v, idx, C_exact.astype(np.float16), h) == 0.0


def test_a_kmeans_step_never_increases_the_weighted_distortion():
    # Lloyd iteration on a synthetic matrix with H = diag(h): both half steps are minimisations
    rng = np.random.default_rng(22)
    v, k, M, N = 8, 32, 64, 40
    W = rng.normal(0, 1, (M, N)).astype(np.float16)
    C = W[:v * 4, :8].reshape(4, v, 8).transpose(0, 2, 1).reshape(32, v).copy()       # 32 vectors of W as seeds
    h = rng.uniform(0.2, 5.0, N).astype(np.float32)
    idx = oracle.assign(W, v, C)
    prev = oracle.distortion(W, v, idx, C, h)
    for _ in range(6):
        C = oracle.kmeans_update(W, v, idx, C, h)
        after_update = oracle.distortion(W, v, idx, C, h)
        assert after_update <= prev * (1 + 2e-3)          # centroids are rounded to FP16
        idx = oracle.assign(W, v, C)
        after_assign = oracle.distortion(W, v, idx, C, h)
        assert after_assign <= after_update * (1 + 1e-6)
        prev = after_assign
    # ragged last vector row: components beyond M are neither read nor written
    Wr = W[:61]
    idx_r = oracle.assign(Wr, v, C)
    Cr = oracle.kmeans_update(Wr, v, idx_r, C, h)
    assert oracle.distortion(Wr, v, idx_r, Cr, h) <= oracle.distortion(Wr, v, idx_r, C, h) * (1 + 2e-3)


def test_assign_distances_that_are_not_numbers_never_win():
    # a centroid with a NaN component is never chosen; a vector with a NaN or infinite component gets index 0
    C = np.array([[np.nan, 0.0], [1.0, 1.0], [5.0, 5.0]], np.float16)
    W = np.array([[1.0, 5.0, np.nan, np.inf], [1.25, 4.0, 0.0, 0.0]], np.float16)
    assert oracle.assign(W, 2, C).tolist() == [[1, 2, 0, 0]]

