"""Second, separately written statement of the same definitions, in numpy.

TEST INFRASTRUCTURE ONLY.  It exists so that the C oracle can be checked against
something that is not itself: it is written with whole-array numpy operations
(unpackbits, fancy indexing, numpy's own float16 rounding) instead of the C file's
per-element loops and hand-written converters.  It works from the *integer* index
matrices (Sec. 2.2: index + codebook), so the lookup itself does not depend on the
packed format; the packed format has its own decoder below.

Restored weight (Sec. 2.2, Sec. 3.2.2 last sentence, Sec. 3.2.3, App. C.1):
  outlier column n < n_out :  t = C0[I0[m // v0, n], m % v0]
  other columns            :  t = C1[I1[m // v, c], m % v] (+ C2[I2[m // v, c], m % v]),  c = n - n_out
  group-wise (Sec. 3.1)    :  C1, C2 are those of the column group g = c // ceil(Nc / group num)
  (project-defined)           W = fp16( fp32(fp32(t * scale) + bias) )
"""
from __future__ import annotations

import numpy as np


def index_bits(k: int) -> int:
    return max(1, int(np.ceil(np.log2(k)))) if k > 1 else 1


def row_bytes(cols: int, k: int) -> int:
    return -(-(-(-cols * index_bits(k) // 8)) // 16) * 16


def pack(idx: np.ndarray, k: int) -> np.ndarray:
    """[rows][cols] ints -> [rows][row_bytes] uint8; little-endian bit stream per row."""
    idx = np.asarray(idx, dtype=np.int64)
    if idx.min(initial=0) < 0 or idx.max(initial=0) >= k:
        raise ValueError("index outside [0, k)")
    rows, cols = idx.shape
    b = index_bits(k)
    bits = ((idx[:, :, None] >> np.arange(b)[None, None, :]) & 1).astype(np.uint8).reshape(rows, cols * b)
    nbits = row_bytes(cols, k) * 8
    bits = np.concatenate([bits, np.zeros((rows, nbits - cols * b), np.uint8)], axis=1)
    return np.packbits(bits, axis=1, bitorder="little")


def unpack(packed: np.ndarray, rows: int, cols: int, k: int) -> np.ndarray:
    b = index_bits(k)
    packed = np.asarray(packed, dtype=np.uint8).reshape(rows, row_bytes(cols, k))
    bits = np.unpackbits(packed, axis=1, bitorder="little")[:, :cols * b].reshape(rows, cols, b)
    return (bits.astype(np.int64) << np.arange(b)[None, None, :]).sum(axis=2).astype(np.int32)


def dequant(M, N, v, c1, idx1, c2=None, idx2=None, n_out=0, v0=0, c0=None, idx0=None,
            scale=None, bias=None, scale_axis=0, n_groups=1, col_perm=None) -> np.ndarray:
    """float16 [M][N] from integer index matrices and float16 tables.  col_perm (Sec. 3.2.3): stored column j
    is column col_perm[j] of the result."""
    W = np.zeros((M, N), dtype=np.float32)
    m = np.arange(M)
    if n_out < N:
        # one codebook pair per run of consecutive columns: entry i of group g sits at row g*k + i
        G = max(1, int(n_groups))
        Nc = N - n_out
        grp = (np.arange(Nc) // (-(-Nc // G)))[None, :]
        k1 = np.asarray(c1).shape[0] // G
        main = np.asarray(c1, np.float16)[grp * k1 + np.asarray(idx1)[m // v], (m % v)[:, None]].astype(np.float32)
        if c2 is not None:
            k2 = np.asarray(c2).shape[0] // G
            res = np.asarray(c2, np.float16)[grp * k2 + np.asarray(idx2)[m // v], (m % v)[:, None]].astype(np.float32)
            main = (main + res).astype(np.float32)
        W[:, n_out:] = main
    if n_out > 0:
        W[:, :n_out] = np.asarray(c0, np.float16)[np.asarray(idx0)[m // v0], (m % v0)[:, None]].astype(np.float32)
    if scale is not None:
        s = np.asarray(scale, np.float16).astype(np.float32)
        bb = np.asarray(bias, np.float16).astype(np.float32)
        if scale_axis == 0:
            W = (W * s[None, :]).astype(np.float32)
            W = (W + bb[None, :]).astype(np.float32)
        else:
            W = (W * s[:, None]).astype(np.float32)
            W = (W + bb[:, None]).astype(np.float32)
    with np.errstate(over="ignore"):
        W16 = W.astype(np.float16)
    if col_perm is None:
        return W16
    out = np.empty_like(W16)
    out[:, np.asarray(col_perm)] = W16
    return out


def linear(W16: np.ndarray, x_f64: np.ndarray) -> np.ndarray:
    """y = x @ W16^T in float64 (App. D.2: restore to FP16, then matmul)."""
    return np.asarray(x_f64, np.float64) @ np.asarray(W16, np.float16).astype(np.float64).T


def dequant_from_synth(d, scale_axis=0) -> np.ndarray:
    s = d["spec"]
    return dequant(s.M, s.N, s.v, d["c1"], d["idx1"], d["c2"], d["idx2"], s.n_out, s.v0,
                   d["c0"], d["idx0"], d["scale"], d["bias"], scale_axis, getattr(s, "n_groups", 1),
                   d.get("col_perm"))
