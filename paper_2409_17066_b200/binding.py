"""Thin Python binding of libvptq's C ABI (include/vptq.h).

Argument marshalling only: every function here passes device pointers of torch tensors
(and torch's current CUDA stream) straight to the entry point of the same name.  torch is
used for device memory and streams, nothing else; there is no CPU fallback — if the
shared library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvptq.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2409_17066_b200.build` "
        "(there is no CPU fallback)")

lib = C.CDLL(LIB_PATH)

OK = 0
E_NULL, E_SHAPE, E_ALIGN, E_UNSUPPORTED, E_WORKSPACE, E_INDEX_RANGE, E_CUDA, E_TIMEOUT = range(-1, -9, -1)
E_SCRATCH_LIMIT = -9
NOALLOC_SCRATCH_BYTES = 1 << 20
DTYPE_FP16, DTYPE_BF16, DTYPE_FP32 = 0, 1, 2
FLAG_SCALE_BIAS, FLAG_SCALE_ROWS, FLAG_FORCE_GENERIC, FLAG_COL_PERM, FLAG_PREPARED = 1, 2, 4, 8, 16
FLAG_CONCURRENT = 32
FLAG_DETERMINISTIC = 64

_DT = {"fp16": DTYPE_FP16, "bf16": DTYPE_BF16, "fp32": DTYPE_FP32}
_TORCH_DT = {DTYPE_FP16: torch.float16, DTYPE_BF16: torch.bfloat16, DTYPE_FP32: torch.float32}


class LayerDesc(C.Structure):
    """vptq_layer_desc"""
    _fields_ = [("M", C.c_int32), ("N", C.c_int32), ("v", C.c_int32), ("k1", C.c_int32),
                ("k2", C.c_int32), ("n_outlier", C.c_int32), ("v0", C.c_int32), ("k0", C.c_int32),
                ("x_dtype", C.c_int32), ("out_dtype", C.c_int32), ("flags", C.c_int32),
                ("n_groups", C.c_int32), ("prepared_parts", C.c_int32)]


class LayerPtrs(C.Structure):
    """vptq_layer_ptrs"""
    _fields_ = [("packed_idx", C.c_void_p), ("codebook", C.c_void_p),
                ("res_idx", C.c_void_p), ("res_codebook", C.c_void_p),
                ("outlier_idx", C.c_void_p), ("outlier_codebook", C.c_void_p),
                ("scale", C.c_void_p), ("bias", C.c_void_p), ("col_perm", C.c_void_p), ("prepared", C.c_void_p)]


EXPORTS = {
    "vptq_index_bits": (C.c_int, [C.c_int32]),
    "vptq_packed_row_bytes": (C.c_int64, [C.c_int32, C.c_int32]),
    "vptq_packed_bytes": (C.c_int64, [C.c_int32, C.c_int32, C.c_int32]),
    "vptq_layer_weight_bytes": (C.c_int64, [C.POINTER(LayerDesc)]),
    "vptq_pack": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "vptq_unpack": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "vptq_pack_host": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "vptq_unpack_host": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "vptq_prepare_bytes": (C.c_int64, [C.POINTER(LayerDesc), C.c_int32]),
    "vptq_prepare_host": (C.c_int, [C.POINTER(LayerDesc), C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t,
                                    C.POINTER(C.c_size_t)]),
    "vptq_prepare": (C.c_int, [C.POINTER(LayerDesc), C.POINTER(LayerPtrs), C.c_int32, C.c_void_p, C.c_size_t,
                               C.POINTER(C.c_size_t), C.c_void_p]),
    "vptq_dequant": (C.c_int, [C.POINTER(LayerDesc), C.POINTER(LayerPtrs), C.c_void_p, C.c_void_p]),
    "vptq_assign": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32,
                              C.c_void_p, C.c_size_t, C.c_void_p]),
    "vptq_assign_workspace_bytes": (C.c_int64, [C.c_int32] * 5),
    "vptq_assign_path": (C.c_char_p, [C.c_int32] * 5),
    "vptq_kmeans_update_workspace_bytes": (C.c_int64, [C.c_int32, C.c_int32]),
    "vptq_kmeans_update": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "vptq_linear_workspace_bytes": (C.c_int64, [C.POINTER(LayerDesc), C.c_int32]),
    "vptq_linear": (C.c_int, [C.POINTER(LayerDesc), C.c_void_p, C.c_int32, C.POINTER(LayerPtrs),
                              C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "vptq_linear_fused_workspace_bytes": (C.c_int64, [C.POINTER(LayerDesc), C.c_int32, C.c_int32]),
    "vptq_linear_fused": (C.c_int, [C.POINTER(LayerDesc), C.POINTER(LayerPtrs), C.c_int32, C.c_void_p, C.c_int32,
                                    C.POINTER(C.c_void_p), C.c_void_p, C.c_size_t, C.c_void_p]),
    "vptq_linear_fused_path": (C.c_char_p, [C.POINTER(LayerDesc), C.c_int32, C.c_int32]),
    "vptq_linear_fused_launches": (C.c_int, [C.POINTER(LayerDesc), C.c_int32, C.c_int32]),
    "vptq_linear_fused_host_io": (C.c_int, [C.POINTER(LayerDesc), C.POINTER(LayerPtrs), C.c_int32, C.c_void_p, C.c_int32,
                                            C.POINTER(C.c_void_p), C.c_void_p, C.POINTER(C.c_void_p), C.c_void_p,
                                            C.c_size_t, C.c_void_p]),
    "vptq_linear_host_io": (C.c_int, [C.POINTER(LayerDesc), C.c_void_p, C.c_int32, C.POINTER(LayerPtrs),
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                      C.c_void_p]),
    "vptq_linear_noalloc": (C.c_int, [C.POINTER(LayerDesc), C.c_void_p, C.c_int32, C.POINTER(LayerPtrs),
                                      C.c_void_p, C.c_void_p]),
    "vptq_status_string": (C.c_char_p, [C.c_int]),
    "vptq_last_cuda_error": (C.c_char_p, []),
    "vptq_workspace_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "vptq_debug_set_wait_limit": (None, [C.c_uint64]),
    "vptq_linear_waits_between_ctas": (C.c_int, [C.POINTER(LayerDesc), C.c_int32]),
    "vptq_linear_path": (C.c_char_p, [C.POINTER(LayerDesc), C.c_int32]),
    "vptq_linear_launches": (C.c_int, [C.POINTER(LayerDesc), C.c_int32]),
}
for _name, (_res, _args) in EXPORTS.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class VptqError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        msg = lib.vptq_status_string(code).decode()
        if code == E_CUDA:
            msg += ": " + lib.vptq_last_cuda_error().decode()
        super().__init__(f"libvptq error {code}: {msg}")


def _check(code: int) -> None:
    if code != OK:
        raise VptqError(code)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_desc(M, N, v, k1, k2=0, n_outlier=0, v0=0, k0=0, x_dtype="fp16", out_dtype="fp16",
              flags=FLAG_SCALE_BIAS, n_groups=1, prepared_parts=0) -> LayerDesc:
    return LayerDesc(M, N, v, k1, k2, n_outlier, v0, k0, _DT[x_dtype], _DT[out_dtype], flags, n_groups, prepared_parts)


# ---- entry points (same names as the C ABI) -------------------------------------------

def vptq_index_bits(k: int) -> int:
    return lib.vptq_index_bits(k)


def vptq_packed_row_bytes(n_cols: int, k: int) -> int:
    return lib.vptq_packed_row_bytes(n_cols, k)


def vptq_packed_bytes(n_rows: int, n_cols: int, k: int) -> int:
    return lib.vptq_packed_bytes(n_rows, n_cols, k)


def vptq_layer_weight_bytes(desc: LayerDesc) -> int:
    return lib.vptq_layer_weight_bytes(C.byref(desc))


def vptq_pack(idx: torch.Tensor, k: int, check: bool = True) -> torch.Tensor:
    """idx: int32 CUDA tensor [rows][cols] -> uint8 CUDA tensor [rows][row_bytes]."""
    assert idx.is_cuda and idx.dtype == torch.int32 and idx.dim() == 2 and idx.is_contiguous()
    rows, cols = idx.shape
    row_b = lib.vptq_packed_row_bytes(cols, k)
    if row_b < 0:
        raise VptqError(int(row_b))
    packed = torch.empty((rows, row_b), dtype=torch.uint8, device=idx.device)
    bad = torch.zeros(1, dtype=torch.int32, device=idx.device) if check else None
    _check(lib.vptq_pack(_ptr(idx), rows, cols, k, _ptr(packed), _ptr(bad), _stream()))
    return packed


def vptq_unpack(packed: torch.Tensor, rows: int, cols: int, k: int) -> torch.Tensor:
    assert packed.is_cuda and packed.dtype == torch.uint8 and packed.is_contiguous()
    assert packed.numel() == lib.vptq_packed_bytes(rows, cols, k)
    idx = torch.empty((rows, cols), dtype=torch.int32, device=packed.device)
    _check(lib.vptq_unpack(_ptr(packed), rows, cols, k, _ptr(idx), _stream()))
    return idx


def vptq_pack_host(idx: np.ndarray, k: int) -> np.ndarray:
    """Host int32 [rows][cols] -> host uint8 [rows][row_bytes] (no CUDA call)."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    rows, cols = idx.shape
    packed = np.empty((rows, max(0, lib.vptq_packed_row_bytes(cols, k))), dtype=np.uint8)
    _check(lib.vptq_pack_host(idx.ctypes.data, rows, cols, k, packed.ctypes.data))
    return packed


def vptq_unpack_host(packed: np.ndarray, rows: int, cols: int, k: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    assert packed.size == lib.vptq_packed_bytes(rows, cols, k)
    idx = np.empty((rows, cols), dtype=np.int32)
    _check(lib.vptq_unpack_host(packed.ctypes.data, rows, cols, k, idx.ctypes.data))
    return idx


def vptq_prepare_bytes(desc: LayerDesc, n_parts: int = 0) -> int:
    n = lib.vptq_prepare_bytes(C.byref(desc), n_parts)
    if n < 0:
        raise VptqError(int(n))
    return n


def vptq_prepare_host(desc: LayerDesc, packed_idx: np.ndarray, res_idx: Optional[np.ndarray], n_parts: int,
                      capacity: Optional[int] = None) -> np.ndarray:
    """Prepared image (uint8 host array, cut to its size) from HOST copies of the canonical streams; no CUDA call."""
    cap = vptq_prepare_bytes(desc, n_parts) if capacity is None else capacity
    image = np.empty(cap, dtype=np.uint8)
    p1 = np.ascontiguousarray(packed_idx, dtype=np.uint8)
    p2 = None if res_idx is None else np.ascontiguousarray(res_idx, dtype=np.uint8)
    used = C.c_size_t(0)
    _check(lib.vptq_prepare_host(C.byref(desc), p1.ctypes.data, None if p2 is None else p2.ctypes.data, n_parts,
                                 image.ctypes.data, cap, C.byref(used)))
    return image[:used.value]


def vptq_prepare(desc: LayerDesc, ptrs: LayerPtrs, n_parts: int = 0) -> torch.Tensor:
    """Prepared image (uint8 CUDA tensor, cut to its size) from the layer's device streams."""
    cap = vptq_prepare_bytes(desc, n_parts)
    image = torch.empty(cap, dtype=torch.uint8, device="cuda")
    used = C.c_size_t(0)
    _check(lib.vptq_prepare(C.byref(desc), C.byref(ptrs), n_parts, image.data_ptr(), cap, C.byref(used), _stream()))
    return image[:used.value]


def prepared_shares(vector_rows, n_sm: int, n_buckets: int = 16):
    """CTAs for each of several prepared layers that are to share one launch on n_sm SMs (their n_parts): in
    proportion to the layers' vector rows, and in multiples of 8, 4 or 2 where that lets every image split
    its n_buckets = ceil(k1 / 4096) buckets over that many CTAs per row group (at most 63 rows in a group)."""
    rows = [int(r) for r in vector_rows]
    for q in (8, 4, 2, 1):
        if q * len(rows) > n_sm or q > max(1, n_buckets) or (q > 1 and min(rows) < q):
            continue
        share = [q] * len(rows)
        while sum(share) + q <= n_sm:
            i = max(range(len(rows)), key=lambda j: rows[j] / share[j])
            if share[i] + q > rows[i]:                       # never more partitions than rows
                break
            share[i] += q
        if q == 1 or all(-(-r // (s // q)) <= 63 for r, s in zip(rows, share)):
            return share
    return [max(1, n_sm // len(rows))] * len(rows)


def vptq_dequant(desc: LayerDesc, ptrs: LayerPtrs, W_out: torch.Tensor) -> torch.Tensor:
    assert W_out.is_cuda and W_out.dtype == torch.float16 and W_out.is_contiguous()
    assert tuple(W_out.shape) == (desc.M, desc.N)
    _check(lib.vptq_dequant(C.byref(desc), C.byref(ptrs), _ptr(W_out), _stream()))
    return W_out


def vptq_assign_path(M: int, N: int, v: int, k: int, flags: int = 0) -> str:
    return lib.vptq_assign_path(M, N, v, k, flags).decode()


def vptq_assign(W: torch.Tensor, v: int, codebook: torch.Tensor, flags: int = 0,
                workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Eq. 2: int32 [ceil(M/v)][N] index of the nearest centroid of every length-v vector of W (fp16 [M][N]).
    flags = FLAG_FORCE_GENERIC selects the plain FP32 kernel; both kernels give the same indices."""
    assert W.is_cuda and W.dtype == torch.float16 and W.dim() == 2 and W.is_contiguous()
    assert codebook.is_cuda and codebook.dtype == torch.float16 and codebook.is_contiguous()
    M, N = W.shape
    k = codebook.shape[0]
    assert tuple(codebook.shape) == (k, v)
    idx = torch.empty((-(-M // v), N), dtype=torch.int32, device=W.device)
    need = lib.vptq_assign_workspace_bytes(M, N, v, k, flags)
    if need < 0:
        raise VptqError(int(need))
    if need and workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=W.device)
    _check(lib.vptq_assign(_ptr(W), M, N, v, _ptr(codebook), k, _ptr(idx), flags, _ptr(workspace),
                           0 if workspace is None else workspace.numel(), _stream()))
    if need:
        _check(lib.vptq_workspace_status(_ptr(workspace), _stream()))
    return idx


def vptq_kmeans_update(W: torch.Tensor, v: int, idx: torch.Tensor, codebook: torch.Tensor,
                       col_weight: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Weighted k-means centroid update (Sec. 3.2.1), in place on `codebook` (fp16 [k][v])."""
    assert W.is_cuda and W.dtype == torch.float16 and W.is_contiguous()
    assert idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous()
    assert codebook.is_cuda and codebook.dtype == torch.float16 and codebook.is_contiguous()
    assert col_weight is None or (col_weight.is_cuda and col_weight.dtype == torch.float32 and col_weight.is_contiguous())
    M, N = W.shape
    k = codebook.shape[0]
    assert tuple(codebook.shape) == (k, v) and tuple(idx.shape) == (-(-M // v), N)
    need = lib.vptq_kmeans_update_workspace_bytes(v, k)
    ws = torch.empty(need, dtype=torch.uint8, device=W.device)
    _check(lib.vptq_kmeans_update(_ptr(W), M, N, v, _ptr(idx), _ptr(col_weight), k, _ptr(codebook),
                                  _ptr(ws), need, _stream()))
    return codebook


def vptq_linear_workspace_bytes(desc: LayerDesc, B: int) -> int:
    n = lib.vptq_linear_workspace_bytes(C.byref(desc), B)
    if n < 0:
        raise VptqError(int(n))
    return n


def vptq_linear(desc: LayerDesc, x: torch.Tensor, ptrs: LayerPtrs, out: torch.Tensor,
                workspace: Optional[torch.Tensor]) -> torch.Tensor:
    assert x.is_cuda and x.is_contiguous() and out.is_cuda and out.is_contiguous()
    assert x.dtype == _TORCH_DT[desc.x_dtype] and out.dtype == _TORCH_DT[desc.out_dtype]
    B = x.shape[0]
    assert tuple(x.shape) == (B, desc.N) and tuple(out.shape) == (B, desc.M)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vptq_linear(C.byref(desc), _ptr(x), B, C.byref(ptrs), _ptr(out),
                           _ptr(workspace), ws_bytes, _stream()))
    return out


def _desc_array(descs: Sequence[LayerDesc]):
    return (LayerDesc * len(descs))(*descs)


def vptq_linear_fused_workspace_bytes(descs: Sequence[LayerDesc], B: int) -> int:
    n = lib.vptq_linear_fused_workspace_bytes(_desc_array(descs), len(descs), B)
    if n < 0:
        raise VptqError(int(n))
    return n


def vptq_linear_fused(descs: Sequence[LayerDesc], ptrs: Sequence[LayerPtrs], x: torch.Tensor,
                      outs: Sequence[torch.Tensor], workspace: Optional[torch.Tensor]) -> Sequence[torch.Tensor]:
    """Several layers over the same activations in one call (q/k/v, gate/up)."""
    n = len(descs)
    assert len(ptrs) == n and len(outs) == n
    B = x.shape[0]
    assert x.is_cuda and x.is_contiguous() and tuple(x.shape) == (B, descs[0].N)
    for d, o in zip(descs, outs):
        assert o.is_cuda and o.is_contiguous() and tuple(o.shape) == (B, d.M) and o.dtype == _TORCH_DT[d.out_dtype]
    out_ptrs = (C.c_void_p * n)(*[o.data_ptr() for o in outs])
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vptq_linear_fused(_desc_array(descs), (LayerPtrs * n)(*ptrs), n, _ptr(x), B, out_ptrs,
                                 _ptr(workspace), ws_bytes, _stream()))
    return outs


def vptq_linear_fused_path(descs: Sequence[LayerDesc], B: int) -> str:
    return lib.vptq_linear_fused_path(_desc_array(descs), len(descs), B).decode()


def vptq_linear_fused_launches(descs: Sequence[LayerDesc], B: int) -> int:
    return lib.vptq_linear_fused_launches(_desc_array(descs), len(descs), B)


def vptq_linear_host_io(desc: LayerDesc, x_host: torch.Tensor, ptrs: LayerPtrs, out_host: torch.Tensor,
                        x_dev: torch.Tensor, out_dev: torch.Tensor,
                        workspace: Optional[torch.Tensor]) -> torch.Tensor:
    assert not x_host.is_cuda and not out_host.is_cuda and x_dev.is_cuda and out_dev.is_cuda
    B = x_host.shape[0]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.vptq_linear_host_io(C.byref(desc), _ptr(x_host), B, C.byref(ptrs), _ptr(out_host),
                                   _ptr(x_dev), _ptr(out_dev), _ptr(workspace), ws_bytes, _stream()))
    return out_host


def vptq_linear_noalloc(desc: LayerDesc, x: torch.Tensor, ptrs: LayerPtrs, out: torch.Tensor) -> torch.Tensor:
    """vptq_linear for callers that cannot hand over a workspace: the scratch is an array built
    into the library (see include/vptq.h for who needs this, the limits and the sharing rules)."""
    assert x.is_cuda and x.is_contiguous() and out.is_cuda and out.is_contiguous()
    assert x.dtype == _TORCH_DT[desc.x_dtype] and out.dtype == _TORCH_DT[desc.out_dtype]
    B = x.shape[0]
    assert tuple(x.shape) == (B, desc.N) and tuple(out.shape) == (B, desc.M)
    _check(lib.vptq_linear_noalloc(C.byref(desc), _ptr(x), B, C.byref(ptrs), _ptr(out), _stream()))
    return out


def vptq_workspace_status(workspace: Optional[torch.Tensor]) -> int:
    return lib.vptq_workspace_status(_ptr(workspace), _stream())


def vptq_linear_path(desc: LayerDesc, B: int) -> str:
    return lib.vptq_linear_path(C.byref(desc), B).decode()


def vptq_linear_launches(desc: LayerDesc, B: int) -> int:
    return lib.vptq_linear_launches(C.byref(desc), B)


# ---- a quantized layer resident on the device ------------------------------------------

class DeviceLayer:
    """Holds the device tensors of one quantized layer and the desc/ptrs structs over them.

    Built from a synth.make_layer() dict; the index matrices are packed ON THE DEVICE with
    vptq_pack (the product's packer).
    """

    def __init__(self, d: Dict, device="cuda", flags: Optional[int] = None, scale_rows: bool = False):
        s = d["spec"]
        self.spec = s
        dev = torch.device(device)

        def up(a, dt=None):
            if a is None:
                return None
            t = torch.from_numpy(np.ascontiguousarray(a))
            if dt is not None:
                t = t.view(dt)
            return t.to(dev)

        self.idx1 = vptq_pack(up(d["idx1"]), s.k1) if s.Nc > 0 else None
        self.idx2 = vptq_pack(up(d["idx2"]), s.k2) if (s.k2 and s.Nc > 0) else None
        self.idx0 = vptq_pack(up(d["idx0"]), s.k0) if s.n_out else None
        self.c1, self.c2, self.c0 = up(d["c1"]), up(d["c2"]), up(d["c0"])
        self.scale, self.bias = up(d["scale"]), up(d["bias"])
        self.col_perm = up(d.get("col_perm"))          # int32 [N] or None: stored column order
        if flags is None:
            flags = FLAG_SCALE_BIAS if d["scale"] is not None else 0
            if scale_rows:
                flags |= FLAG_SCALE_ROWS
            if self.col_perm is not None:
                flags |= FLAG_COL_PERM
        self.desc = make_desc(s.M, s.N, s.v, s.k1, s.k2, s.n_out, s.v0, s.k0, s.x_dtype, s.out_dtype, flags,
                              getattr(s, "n_groups", 1))
        self.ptrs = LayerPtrs(_ptr(self.idx1), _ptr(self.c1), _ptr(self.idx2), _ptr(self.c2),
                              _ptr(self.idx0), _ptr(self.c0), _ptr(self.scale), _ptr(self.bias),
                              _ptr(self.col_perm))
        self._ws: Dict[int, Optional[torch.Tensor]] = {}
        self.device = dev
        self.image = None

    def with_flags(self, flags: int) -> "DeviceLayer":
        other = object.__new__(DeviceLayer)
        other.__dict__.update(self.__dict__)
        s = self.spec
        other.desc = make_desc(s.M, s.N, s.v, s.k1, s.k2, s.n_out, s.v0, s.k0, s.x_dtype, s.out_dtype, flags,
                               getattr(s, "n_groups", 1))
        other._ws = {}
        return other

    def prepared(self, n_parts: int = 0) -> "DeviceLayer":
        """The same layer with a prepared image (vptq_prepare): batch-1 calls read the image instead of the
        canonical streams.  n_parts = CTAs that will work on the layer (0: one per SM)."""
        other = object.__new__(DeviceLayer)
        other.__dict__.update(self.__dict__)
        other.image = vptq_prepare(self.desc, self.ptrs, n_parts)
        parts = int(other.image[24:28].view(torch.int32).item())           # header word 6
        s = self.spec
        other.desc = make_desc(s.M, s.N, s.v, s.k1, s.k2, s.n_out, s.v0, s.k0, s.x_dtype, s.out_dtype,
                               self.desc.flags | FLAG_PREPARED, getattr(s, "n_groups", 1), parts)
        other.ptrs = LayerPtrs(*[getattr(self.ptrs, f[0]) for f in LayerPtrs._fields_[:-1]], _ptr(other.image))
        other._ws = {}
        return other

    def clone_streams(self) -> "DeviceLayer":
        """A second copy of the packed index streams (codebooks, scale, bias shared): lets a
        benchmark walk more weight bytes than L2 holds."""
        other = object.__new__(DeviceLayer)
        other.__dict__.update(self.__dict__)
        other.idx1 = None if self.idx1 is None else self.idx1.clone()
        other.idx2 = None if self.idx2 is None else self.idx2.clone()
        other.idx0 = None if self.idx0 is None else self.idx0.clone()
        other.image = None if getattr(self, "image", None) is None else self.image.clone()
        other.ptrs = LayerPtrs(_ptr(other.idx1), _ptr(self.c1), _ptr(other.idx2), _ptr(self.c2),
                               _ptr(other.idx0), _ptr(self.c0), _ptr(self.scale), _ptr(self.bias),
                               _ptr(self.col_perm), _ptr(other.image))
        return other

    def weight_bytes(self) -> int:
        return vptq_layer_weight_bytes(self.desc)

    def workspace(self, B: int) -> Optional[torch.Tensor]:
        if B not in self._ws:
            n = vptq_linear_workspace_bytes(self.desc, B)
            self._ws[B] = torch.zeros(n, dtype=torch.uint8, device=self.device) if n > 0 else None
        return self._ws[B]

    def upload_x(self, x_np: np.ndarray) -> torch.Tensor:
        t = torch.from_numpy(np.ascontiguousarray(x_np))
        if self.spec.x_dtype == "bf16":
            t = t.view(torch.bfloat16)
        return t.to(self.device)

    def dequant(self) -> torch.Tensor:
        W = torch.empty((self.spec.M, self.spec.N), dtype=torch.float16, device=self.device)
        return vptq_dequant(self.desc, self.ptrs, W)

    def linear(self, x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = x.shape[0]
        if out is None:
            out = torch.empty((B, self.spec.M), dtype=_TORCH_DT[self.desc.out_dtype], device=self.device)
        return vptq_linear(self.desc, x, self.ptrs, out, self.workspace(B))


class FusedLayers:
    """Several DeviceLayers that read the same activations (q/k/v, gate/up): keeps the argument arrays of
    vptq_linear_fused so that a call costs no more host time than vptq_linear."""

    def __init__(self, dls: Sequence[DeviceLayer]):
        self.dls = list(dls)
        self.n = len(self.dls)
        self.descs = _desc_array([d.desc for d in self.dls])
        self.ptrs = (LayerPtrs * self.n)(*[d.ptrs for d in self.dls])
        self._ws: Dict[int, Optional[torch.Tensor]] = {}

    def path(self, B: int) -> str:
        return lib.vptq_linear_fused_path(self.descs, self.n, B).decode()

    def launches(self, B: int) -> int:
        return lib.vptq_linear_fused_launches(self.descs, self.n, B)

    def workspace(self, B: int) -> Optional[torch.Tensor]:
        if B not in self._ws:
            need = lib.vptq_linear_fused_workspace_bytes(self.descs, self.n, B)
            if need < 0:
                raise VptqError(int(need))
            self._ws[B] = torch.zeros(need, dtype=torch.uint8, device=self.dls[0].device) if need else None
        return self._ws[B]

    def linear(self, x: torch.Tensor, outs: Sequence[torch.Tensor]) -> Sequence[torch.Tensor]:
        B = x.shape[0]
        ws = self.workspace(B)
        out_ptrs = (C.c_void_p * self.n)(*[o.data_ptr() for o in outs])
        _check(lib.vptq_linear_fused(self.descs, self.ptrs, self.n, _ptr(x), B, out_ptrs, _ptr(ws),
                                     0 if ws is None else ws.numel(), _stream()))
        return outs

    def linear_host_io(self, x_host: torch.Tensor, outs_host: Sequence[torch.Tensor], x_dev: torch.Tensor,
                       outs_dev: Sequence[torch.Tensor]) -> Sequence[torch.Tensor]:
        B = x_host.shape[0]
        ws = self.workspace(B)
        oh = (C.c_void_p * self.n)(*[o.data_ptr() for o in outs_host])
        od = (C.c_void_p * self.n)(*[o.data_ptr() for o in outs_dev])
        _check(lib.vptq_linear_fused_host_io(self.descs, self.ptrs, self.n, _ptr(x_host), B, oh, _ptr(x_dev), od,
                                             _ptr(ws), 0 if ws is None else ws.numel(), _stream()))
        return outs_host

