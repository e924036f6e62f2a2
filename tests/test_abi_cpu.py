"""The C-ABI library loads without a GPU and exports every symbol the header declares;
its host-only format arithmetic agrees with the oracle's and with the paper's formulas."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import oracle
from paper_2409_17066_b200 import build as vbuild
from paper_2409_17066_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    vbuild.build()
    from paper_2409_17066_b200 import binding as b
    return b


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "vptq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vptq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(binding.lib, n), n
    # and the binding wraps each of them under the same name
    for n in names:
        assert n in binding.EXPORTS, n


def test_format_arithmetic_matches_oracle(binding):
    for k in [1, 2, 3, 5, 16, 17, 255, 256, 257, 4096, 4097, 8192, 65535, 65536]:
        assert binding.vptq_index_bits(k) == oracle.index_bits(k)
        for cols in [0, 1, 7, 41, 4055, 4096, 10898]:
            assert binding.vptq_packed_row_bytes(cols, k) == oracle.row_bytes(cols, k)
            assert binding.vptq_packed_bytes(13, cols, k) == oracle.packed_bytes(13, cols, k)
    assert binding.vptq_index_bits(0) == binding.E_SHAPE
    assert binding.vptq_index_bits(65537) == binding.E_SHAPE
    assert binding.vptq_packed_bytes(-1, 4, 16) == binding.E_SHAPE


def test_layer_weight_bytes_follow_the_bit_formulas(binding):
    # App. C.2: index bits log2(k)/v per weight and codebook bits (v0*k0 + v1*(k1+k2))*16
    for cfg in sorted(synth.CONFIGS):
        for s in synth.CONFIGS[cfg]["layers"]:
            d = binding.make_desc(s.M, s.N, s.v, s.k1, s.k2, s.n_out, s.v0, s.k0, s.x_dtype, s.out_dtype,
                                  n_groups=s.n_groups)
            got = binding.vptq_layer_weight_bytes(d)
            exp = oracle.packed_bytes(s.R, s.Nc, s.k1) + (oracle.packed_bytes(s.R, s.Nc, s.k2) if s.k2 else 0) \
                + (oracle.packed_bytes(s.R0, s.n_out, s.k0) if s.n_out else 0) \
                + (oracle.codebook_bits(s.v, s.k1, s.k2, 0, 0, 0) * max(1, s.n_groups)
                   + (oracle.codebook_bits(s.v, 0, 0, s.n_out, s.v0, s.k0) if s.n_out else 0)) / 8 + 4 * s.N
            assert got == exp
    # the worked example of Sec. 2.2: 4096 x 4096, v = 8, k = 256, no scale/bias
    d = binding.make_desc(4096, 4096, 8, 256, flags=0)
    assert round(16.0 * 4096 * 4096 / (8 * binding.vptq_layer_weight_bytes(d)), 2) == 15.97


def test_argument_errors_need_no_gpu(binding):
    b = binding
    d = b.make_desc(64, 64, 8, 256)
    p = b.LayerPtrs()
    assert b.lib.vptq_dequant(None, C.byref(p), None, None) == b.E_NULL
    bad = b.make_desc(0, 64, 8, 256)
    assert b.lib.vptq_dequant(C.byref(bad), C.byref(p), None, None) == b.E_SHAPE
    bad = b.make_desc(64, 64, 8, 70000)
    assert b.lib.vptq_linear_workspace_bytes(C.byref(bad), 1) == b.E_SHAPE
    bad = b.make_desc(64, 64, 8, 256, n_outlier=65, v0=4, k0=16)
    assert b.lib.vptq_linear_workspace_bytes(C.byref(bad), 1) == b.E_SHAPE
    bad = b.make_desc(64, 64, 8, 256)
    bad.x_dtype = 2
    assert b.lib.vptq_linear_workspace_bytes(C.byref(bad), 1) == b.E_UNSUPPORTED
    assert b.lib.vptq_linear_workspace_bytes(C.byref(d), 0) == b.E_SHAPE
    # required pointers missing -> E_NULL before any CUDA call
    assert b.lib.vptq_dequant(C.byref(d), C.byref(p), None, None) == b.E_NULL
    assert b.lib.vptq_linear(C.byref(d), None, 1, C.byref(p), None, None, 0, None) == b.E_NULL
    # misaligned pointer -> E_ALIGN (never dereferenced)
    p2 = b.LayerPtrs(0x1008, 0x1000, None, None, None, None, 0x1000, 0x1000)
    assert b.lib.vptq_dequant(C.byref(d), C.byref(p2), 0x1000, None) == b.E_ALIGN
    assert b.lib.vptq_status_string(b.E_ALIGN).decode().startswith("a data pointer")
    assert b.vptq_linear_path(d, 1) in ("generic", "decode_smem_fma", "decode_smem_mma", "decode_l2_fma", "decode_gl_fma", "gemm_tcgen05")
    assert b.vptq_linear_launches(d, 1) >= 1


def test_fused_call_argument_errors_and_path_names(binding):
    b = binding
    q = b.make_desc(8192, 8192, 8, 65536, 256)
    kv = b.make_desc(1024, 8192, 8, 65536, 256)
    arr = (b.LayerDesc * 3)(q, kv, kv)
    assert b.lib.vptq_linear_fused_workspace_bytes(None, 3, 1) == b.E_NULL
    assert b.lib.vptq_linear_fused_workspace_bytes(arr, 0, 1) == b.E_SHAPE
    assert b.lib.vptq_linear_fused_workspace_bytes(arr, 5, 1) == b.E_SHAPE
    assert b.lib.vptq_linear_fused_workspace_bytes(arr, 3, 0) == b.E_SHAPE
    other_n = (b.LayerDesc * 2)(q, b.make_desc(1024, 4096, 8, 65536, 256))
    assert b.lib.vptq_linear_fused_workspace_bytes(other_n, 2, 1) == b.E_SHAPE
    assert b.lib.vptq_linear_fused(arr, None, 3, None, 1, None, None, 0, None) == b.E_NULL
    # three projections of an attention block over the same input: one launch, no scratch
    assert b.vptq_linear_fused_path([q, kv, kv], 1) == "fused_decode_l2_fma"
    assert b.vptq_linear_fused_workspace_bytes([q, kv, kv], 1) == 0
    assert b.vptq_linear_fused_launches([q, kv, kv], 1) == 1
    assert b.vptq_linear_fused_launches([q, kv, kv], 6) == 2          # token groups of 4
    # layers of one format (apart from M) with their codebooks in shared memory are fused as well ...
    small = b.make_desc(11008, 4096, 6, 4096, 256, n_outlier=41, v0=4, k0=4096)
    assert b.vptq_linear_fused_path([small, small], 1) == "fused_decode_smem_fma"
    assert b.vptq_linear_fused_launches([small, small], 1) == 1
    # ... layers of different formats, or of different kernel families, run one after the other and share the scratch
    other = b.make_desc(11008, 4096, 6, 4096, 256, n_outlier=40, v0=4, k0=4096)
    assert b.vptq_linear_fused_path([small, other], 1) == "one_by_one"
    assert b.vptq_linear_fused_launches([small, other], 1) == 2 * b.vptq_linear_launches(small, 1)
    assert b.vptq_linear_fused_path([small, q], 1) == "invalid"            # different N
    assert b.vptq_linear_fused_path([small, small], 8) == "one_by_one"      # 8 tokens: the mma kernel, not fused
    # a single layer, or many tokens, is not fused either
    assert b.vptq_linear_fused_path([q], 1) == "one_by_one"
    assert b.vptq_linear_fused_path([q, kv], 64) == "one_by_one"
    assert b.vptq_linear_fused_workspace_bytes([q, kv], 64) == max(b.vptq_linear_workspace_bytes(q, 64),
                                                                  b.vptq_linear_workspace_bytes(kv, 64))


def test_assign_path_and_workspace_queries(binding):
    b = binding
    assert b.vptq_assign_path(4096, 4096, 8, 65536) == "assign_tcgen05"
    assert b.vptq_assign_path(4096, 4096, 8, 65536, b.FLAG_FORCE_GENERIC) == "assign_fp32"
    assert b.vptq_assign_path(4100, 4096, 8, 65536) == "assign_fp32"        # v does not divide M
    assert b.vptq_assign_path(4096, 4096, 16, 65536) == "assign_fp32"       # two of 16 K columns carry the norm
    assert b.vptq_assign_path(4096, 4096, 8, 256) == "assign_fp32"          # small tables do not pay
    assert b.vptq_assign_path(4096, 4096, 40, 256) == "invalid"
    assert b.lib.vptq_assign_workspace_bytes(4096, 4096, 8, 256, 0) == 0
    need = b.lib.vptq_assign_workspace_bytes(4096, 4096, 8, 65536, 0)
    assert need >= 65536 * 32 + 4 * 512 * 4096
    assert b.lib.vptq_assign(0x1000, 4096, 4096, 8, 0x1000, 65536, 0x1000, 0, None, 0, None) == b.E_WORKSPACE
    assert b.lib.vptq_assign(None, 4096, 4096, 8, 0x1000, 65536, 0x1000, 0, None, 0, None) == b.E_NULL
    assert b.lib.vptq_assign(0x1000, 4096, 4096, 8, 0x1000, 70000, 0x1000, 0, None, 0, None) == b.E_SHAPE



@pytest.mark.parametrize("k", [1, 2, 3, 5, 16, 100, 256, 257, 4096, 5000, 8192, 40000, 65536])
def test_host_pack_and_unpack_write_the_oracle_bytes(binding, k):
    # vptq_pack_host / vptq_unpack_host: plain host code, no CUDA call; byte for byte the oracle's stream
    b = binding
    rng = np.random.default_rng(k)
    for shape in [(1, 1), (3, 7), (5, 41), (4, 257), (2, 4055), (9, 4096)]:
        for idx in (rng.integers(0, k, size=shape, dtype=np.int32), np.full(shape, k - 1, np.int32),
                    np.zeros(shape, np.int32)):
            ref = oracle.pack(idx, k)
            got = b.vptq_pack_host(idx, k)
            assert got.shape == ref.shape and np.array_equal(got, ref)
            # unpack what the ORACLE packed
            assert np.array_equal(b.vptq_unpack_host(ref, shape[0], shape[1], k), idx)


def test_host_pack_argument_errors(binding):
    b = binding
    idx = np.array([[0, 1, 5, 2], [7, 0, -1, 3]], np.int32)
    out = np.full((2, 16), 0xAA, np.uint8)
    assert b.lib.vptq_pack_host(idx.ctypes.data, 2, 4, 5, out.ctypes.data) == b.E_INDEX_RANGE
    # the stream is complete all the same, with 0 stored for the three bad entries
    assert np.array_equal(b.vptq_unpack_host(out, 2, 4, 5), np.array([[0, 1, 0, 2], [0, 0, 0, 3]], np.int32))
    assert b.lib.vptq_pack_host(None, 2, 4, 5, out.ctypes.data) == b.E_NULL
    assert b.lib.vptq_pack_host(idx.ctypes.data, 2, 4, 0, out.ctypes.data) == b.E_SHAPE
    assert b.lib.vptq_pack_host(None, 0, 4, 5, None) == b.OK
    assert b.lib.vptq_unpack_host(out.ctypes.data, 2, 4, 70000, idx.ctypes.data) == b.E_SHAPE
    assert b.lib.vptq_unpack_host(None, 2, 4, 5, idx.ctypes.data) == b.E_NULL


def test_calls_that_share_the_gpu_never_wait_between_ctas(binding):
    # the batched path lets CTAs wait for a flag of another CTA only with long shares of k blocks, and never when
    # the caller says that the call may overlap other GPU work
    b = binding
    down = b.make_desc(4096, 14336, 8, 65536, 256, x_dtype="bf16", out_dtype="fp32")
    assert b.vptq_linear_path(down, 512) == "gemm_tcgen05"
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(down), 512) == 1
    shared = b.make_desc(4096, 14336, 8, 65536, 256, x_dtype="bf16", out_dtype="fp32",
                         flags=b.FLAG_SCALE_BIAS | b.FLAG_CONCURRENT)
    assert b.vptq_linear_path(shared, 512) == "gemm_tcgen05"
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(shared), 512) == 0
    # two layers prepared for two streams: both descriptors carry the flag, neither plan waits
    for d in (shared, b.make_desc(14336, 4096, 8, 65536, 256, x_dtype="bf16", out_dtype="fp32",
                                  flags=b.FLAG_SCALE_BIAS | b.FLAG_CONCURRENT)):
        assert b.lib.vptq_linear_waits_between_ctas(C.byref(d), 512) == 0
    # decode paths and whole-tile outputs never wait
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(down), 1) == 0
    half = b.make_desc(4096, 14336, 8, 65536, 256, x_dtype="bf16", out_dtype="fp16")
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(half), 512) == 0
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(down), 0) == b.E_SHAPE
