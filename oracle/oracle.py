"""ctypes wrapper around the C oracle (oracle/vptq_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's
CPU-baseline leg.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_u8p = C.POINTER(C.c_uint8)
_u16p = C.POINTER(C.c_uint16)
_i32p = C.POINTER(C.c_int32)
_f64p = C.POINTER(C.c_double)


class _Layer(C.Structure):
    _fields_ = [("M", C.c_int32), ("N", C.c_int32),
                ("v", C.c_int32), ("k1", C.c_int32), ("k2", C.c_int32),
                ("n_out", C.c_int32), ("v0", C.c_int32), ("k0", C.c_int32),
                ("has_scale", C.c_int32), ("scale_axis", C.c_int32), ("n_groups", C.c_int32),
                ("idx1", C.c_void_p), ("c1", C.c_void_p),
                ("idx2", C.c_void_p), ("c2", C.c_void_p),
                ("idx0", C.c_void_p), ("c0", C.c_void_p),
                ("scale", C.c_void_p), ("bias", C.c_void_p), ("col_perm", C.c_void_p)]


_lib.oracle_half_to_float.restype = C.c_float
_lib.oracle_half_to_float.argtypes = [C.c_uint16]
_lib.oracle_float_to_half.restype = C.c_uint16
_lib.oracle_float_to_half.argtypes = [C.c_float]
_lib.oracle_bf16_to_float.restype = C.c_float
_lib.oracle_bf16_to_float.argtypes = [C.c_uint16]
_lib.oracle_float_to_bf16.restype = C.c_uint16
_lib.oracle_float_to_bf16.argtypes = [C.c_float]
_lib.oracle_index_bits.restype = C.c_int
_lib.oracle_index_bits.argtypes = [C.c_int32]
_lib.oracle_row_bytes.restype = C.c_int64
_lib.oracle_row_bytes.argtypes = [C.c_int32, C.c_int32]
_lib.oracle_packed_bytes.restype = C.c_int64
_lib.oracle_packed_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
_lib.oracle_pack.restype = C.c_int
_lib.oracle_pack.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
_lib.oracle_unpack.restype = None
_lib.oracle_unpack.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
_lib.oracle_dequant.restype = C.c_int
_lib.oracle_dequant.argtypes = [C.POINTER(_Layer), C.c_void_p]
_lib.oracle_dequant_rows.restype = C.c_int
_lib.oracle_dequant_rows.argtypes = [C.POINTER(_Layer), C.c_void_p, C.c_int32, C.c_void_p]
_lib.oracle_linear_rows.restype = C.c_int
_lib.oracle_linear_rows.argtypes = [C.POINTER(_Layer), C.c_void_p, C.c_int32, C.c_int,
                                    C.c_void_p, C.c_int32, C.c_void_p]
for _n in ("oracle_codebook_bits",):
    getattr(_lib, _n).restype = C.c_double
    getattr(_lib, _n).argtypes = [C.c_int32] * 6
_lib.oracle_equivalent_bits_grouped.restype = C.c_double
_lib.oracle_equivalent_bits_grouped.argtypes = [C.c_int32] * 9
for _n in ("oracle_index_bits_total", "oracle_equivalent_bits", "oracle_compression_ratio"):
    getattr(_lib, _n).restype = C.c_double
    getattr(_lib, _n).argtypes = [C.c_int32] * 8
_lib.oracle_assign.restype = None
_lib.oracle_assign.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
_lib.oracle_assign_some.restype = None
_lib.oracle_assign_some.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                    C.c_void_p, C.c_int32, C.c_void_p]
_lib.oracle_kmeans_update.restype = None
_lib.oracle_kmeans_update.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                      C.c_int32, C.c_void_p]
_lib.oracle_distortion.restype = C.c_double
_lib.oracle_distortion.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.oracle_decode_prepared.restype = C.c_int
_lib.oracle_decode_prepared.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int32, C.c_void_p, C.c_void_p]
_lib.oracle_num_threads.restype = C.c_int
_lib.oracle_set_num_threads.argtypes = [C.c_int]


def half_to_float(bits: int) -> float:
    return float(_lib.oracle_half_to_float(int(bits)))


def float_to_half(f: float) -> int:
    return int(_lib.oracle_float_to_half(C.c_float(f)))


def bf16_to_float(bits: int) -> float:
    return float(_lib.oracle_bf16_to_float(int(bits)))


def float_to_bf16(f: float) -> int:
    return int(_lib.oracle_float_to_bf16(C.c_float(f)))


def index_bits(k: int) -> int:
    return int(_lib.oracle_index_bits(k))


def row_bytes(cols: int, k: int) -> int:
    return int(_lib.oracle_row_bytes(cols, k))


def packed_bytes(rows: int, cols: int, k: int) -> int:
    return int(_lib.oracle_packed_bytes(rows, cols, k))


def pack(idx: np.ndarray, k: int) -> np.ndarray:
    """int32 [rows][cols] -> packed bytes [rows][row_bytes]; raises on idx outside [0,k)."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    rows, cols = idx.shape
    out = np.empty((rows, row_bytes(cols, k)), dtype=np.uint8)
    rc = _lib.oracle_pack(idx.ctypes.data, rows, cols, k, out.ctypes.data)
    if rc != 0:
        raise ValueError("index outside [0, k)")
    return out


def unpack(packed: np.ndarray, rows: int, cols: int, k: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    assert packed.size == packed_bytes(rows, cols, k)
    out = np.empty((rows, cols), dtype=np.int32)
    _lib.oracle_unpack(packed.ctypes.data, rows, cols, k, out.ctypes.data)
    return out


class Layer:
    """A quantized layer as the oracle sees it: packed streams + tables (numpy, host)."""

    def __init__(self, M, N, v, k1, c1, idx1_packed, k2=0, c2=None, idx2_packed=None,
                 n_out=0, v0=0, k0=0, c0=None, idx0_packed=None,
                 scale=None, bias=None, scale_axis=0, n_groups=1, col_perm=None):
        def u16(a):
            return None if a is None else np.ascontiguousarray(a).view(np.uint16).reshape(-1).copy()

        def u8(a):
            return None if a is None else np.ascontiguousarray(a, dtype=np.uint8).reshape(-1).copy()

        self.M, self.N, self.v, self.k1, self.k2 = M, N, v, k1, k2
        self.n_out, self.v0, self.k0 = n_out, v0, k0
        self.n_groups = G = max(1, int(n_groups))
        self._keep = dict(idx1=u8(idx1_packed), c1=u16(c1), idx2=u8(idx2_packed), c2=u16(c2),
                          idx0=u8(idx0_packed), c0=u16(c0), scale=u16(scale), bias=u16(bias))
        R, Nc = -(-M // v), N - n_out
        assert self._keep["idx1"].size == packed_bytes(R, Nc, k1) and self._keep["c1"].size == G * k1 * v
        if k2:
            assert self._keep["idx2"].size == packed_bytes(R, Nc, k2) and self._keep["c2"].size == G * k2 * v
        if n_out:
            assert self._keep["idx0"].size == packed_bytes(-(-M // v0), n_out, k0)
            assert self._keep["c0"].size == k0 * v0
        has_scale = scale is not None
        if has_scale:
            assert self._keep["scale"].size == (M if scale_axis else N)
            assert self._keep["bias"].size == (M if scale_axis else N)
        # stored column j is input feature col_perm[j] (Sec. 3.2.3: outlier columns lie where the quantizer found them)
        self._keep["col_perm"] = None if col_perm is None else np.ascontiguousarray(col_perm, dtype=np.int32).copy()
        if col_perm is not None:
            assert self._keep["col_perm"].shape == (N,)
        p = lambda n: (self._keep[n].ctypes.data if self._keep[n] is not None else None)
        self.c = _Layer(M, N, v, k1, k2, n_out, v0, k0, int(has_scale), scale_axis, G,
                        p("idx1"), p("c1"), p("idx2"), p("c2"), p("idx0"), p("c0"),
                        p("scale"), p("bias"), p("col_perm"))

    @classmethod
    def from_synth(cls, d, scale_axis=0):
        """Build from a paper_2409_17066_b200.synth.make_layer dict, packing with the oracle's packer."""
        s = d["spec"]
        return cls(s.M, s.N, s.v, s.k1, d["c1"], pack(d["idx1"], s.k1),
                   k2=s.k2, c2=d["c2"], idx2_packed=pack(d["idx2"], s.k2) if s.k2 else None,
                   n_out=s.n_out, v0=s.v0, k0=s.k0, c0=d["c0"],
                   idx0_packed=pack(d["idx0"], s.k0) if s.n_out else None,
                   scale=d["scale"], bias=d["bias"], scale_axis=scale_axis,
                   n_groups=getattr(s, "n_groups", 1), col_perm=d.get("col_perm"))

    def dequant(self) -> np.ndarray:
        """W16 [M][N] as numpy float16 (bit-exact definition of the restored weight)."""
        W = np.empty((self.M, self.N), dtype=np.uint16)
        if _lib.oracle_dequant(C.byref(self.c), W.ctypes.data) != 0:
            raise ValueError("index out of range in packed stream")
        return W.view(np.float16)

    def dequant_rows(self, rows) -> np.ndarray:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        W = np.empty((rows.size, self.N), dtype=np.uint16)
        if _lib.oracle_dequant_rows(C.byref(self.c), rows.ctypes.data, rows.size, W.ctypes.data) != 0:
            raise ValueError("index out of range in packed stream")
        return W.view(np.float16)

    def linear(self, x: np.ndarray, rows=None) -> np.ndarray:
        """y [B][M] (or [B][len(rows)]) in float64.  x: float16 array or uint16 bf16 bits, [B][N]."""
        is_bf16 = x.dtype == np.uint16
        xb = np.ascontiguousarray(x).view(np.uint16)
        B = xb.shape[0]
        assert xb.shape[1] == self.N
        if rows is None:
            rp, nr = None, self.M
        else:
            rows = np.ascontiguousarray(rows, dtype=np.int32)
            rp, nr = rows.ctypes.data, rows.size
        y = np.empty((B, nr), dtype=np.float64)
        if _lib.oracle_linear_rows(C.byref(self.c), xb.ctypes.data, B, int(is_bf16), rp, nr,
                                   y.ctypes.data) != 0:
            raise ValueError("index out of range in packed stream")
        return y


def assign(W16: np.ndarray, v: int, codebook: np.ndarray, vectors=None) -> np.ndarray:
    """Eq. 2: index of the nearest centroid for every length-v vector (v consecutive rows of a column) of the
    float16 matrix W16 [M][N]; codebook float16 [k][v].  Returns int32 [ceil(M/v)][N], or, with `vectors`
    (flat numbers r * N + n), the indices of those vectors only."""
    Wb = np.ascontiguousarray(W16, dtype=np.float16).view(np.uint16)
    Cb = np.ascontiguousarray(codebook, dtype=np.float16).view(np.uint16)
    M, N = Wb.shape
    k = Cb.shape[0]
    assert Cb.shape == (k, v)
    if vectors is None:
        idx = np.empty((-(-M // v), N), dtype=np.int32)
        _lib.oracle_assign(Wb.ctypes.data, M, N, v, Cb.ctypes.data, k, idx.ctypes.data)
        return idx
    vec = np.ascontiguousarray(vectors, dtype=np.int64)
    idx = np.empty(vec.size, dtype=np.int32)
    _lib.oracle_assign_some(Wb.ctypes.data, M, N, v, Cb.ctypes.data, k, vec.ctypes.data, vec.size, idx.ctypes.data)
    return idx


def kmeans_update(W16: np.ndarray, v: int, idx: np.ndarray, codebook: np.ndarray, h=None) -> np.ndarray:
    """Weighted k-means centroid update (Sec. 3.2.1): the weighted mean of the vectors assigned to every
    centroid (weights h[N] per column, None = 1); components that received no weight keep their old value.
    Returns the new float16 [k][v] codebook."""
    Wb = np.ascontiguousarray(W16, dtype=np.float16).view(np.uint16)
    Cb = np.ascontiguousarray(codebook, dtype=np.float16).view(np.uint16).copy()
    ib = np.ascontiguousarray(idx, dtype=np.int32)
    M, N = Wb.shape
    hb = None if h is None else np.ascontiguousarray(h, dtype=np.float32)
    _lib.oracle_kmeans_update(Wb.ctypes.data, M, N, v, ib.ctypes.data, None if hb is None else hb.ctypes.data,
                              Cb.shape[0], Cb.ctypes.data)
    return Cb.view(np.float16)


def distortion(W16: np.ndarray, v: int, idx: np.ndarray, codebook: np.ndarray, h=None) -> float:
    """sum_n h_n ||x - C_idx||^2 over all vectors, float64."""
    Wb = np.ascontiguousarray(W16, dtype=np.float16).view(np.uint16)
    Cb = np.ascontiguousarray(codebook, dtype=np.float16).view(np.uint16)
    ib = np.ascontiguousarray(idx, dtype=np.int32)
    M, N = Wb.shape
    hb = None if h is None else np.ascontiguousarray(h, dtype=np.float32)
    return float(_lib.oracle_distortion(Wb.ctypes.data, M, N, v, ib.ctypes.data,
                                        None if hb is None else hb.ctypes.data, Cb.ctypes.data))


def decode_prepared(image: np.ndarray, M: int, N: int, k1: int, k2: int, v: int = 8, n_out: int = 0):
    """Index matrices (idx1, idx2), int32 [ceil(M/v)][N - n_out], read back from a prepared layer image by the
    format's rules; returns (code, idx1, idx2) where code = 0 or the number of the first broken rule."""
    img = np.ascontiguousarray(image, dtype=np.uint8)
    R = -(-M // v)
    idx1 = np.empty((R, N - n_out), dtype=np.int32)
    idx2 = np.empty((R, N - n_out), dtype=np.int32)
    code = int(_lib.oracle_decode_prepared(img.ctypes.data, img.size, M, N, v, k1, k2, n_out, idx1.ctypes.data, idx2.ctypes.data))
    return code, idx1, idx2


def codebook_bits(v, k1, k2=0, n_out=0, v0=0, k0=0) -> float:
    return float(_lib.oracle_codebook_bits(v, k1, k2, n_out, v0, k0))


def index_bits_total(M, N, v, k1, k2=0, n_out=0, v0=0, k0=0) -> float:
    return float(_lib.oracle_index_bits_total(M, N, v, k1, k2, n_out, v0, k0))


def equivalent_bits(M, N, v, k1, k2=0, n_out=0, v0=0, k0=0) -> float:
    return float(_lib.oracle_equivalent_bits(M, N, v, k1, k2, n_out, v0, k0))


def equivalent_bits_grouped(M, N, v, k1, k2=0, n_out=0, v0=0, k0=0, n_groups=1) -> float:
    return float(_lib.oracle_equivalent_bits_grouped(M, N, v, k1, k2, n_out, v0, k0, n_groups))


def compression_ratio(M, N, v, k1, k2=0, n_out=0, v0=0, k0=0) -> float:
    return float(_lib.oracle_compression_ratio(M, N, v, k1, k2, n_out, v0, k0))


def num_threads() -> int:
    return int(_lib.oracle_num_threads())


def set_num_threads(n: int) -> None:
    _lib.oracle_set_num_threads(int(n))
