"""vptq_linear_noalloc: the decode kernel with its scratch in an array built into the library,
for callers that cannot allocate device memory (an engine whose arena owns all of it, or a
serving loop where cudaMalloc is off limits after start-up).

This file is named so that pytest collects it last: should it fail, every other test has
already run.  It must pass alone in a fresh process and after the rest of the suite: the
built-in array is shared by all calls and keeps the previous call's contents, which is
exactly what the two back-to-back calls below exercise."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2409_17066_b200 import synth

from helpers import TOL, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2409_17066_b200 import build as vbuild
    vbuild.build()
    from paper_2409_17066_b200 import binding
    return binding


@pytest.mark.parametrize("B", [1, 4, 7])
def test_noalloc_matches_vptq_linear_twice_in_a_row(b, B):
    # 65 vector rows do not divide over the SMs: the kernel deals tasks out regardless of rows and
    # really goes through the scratch array
    spec = synth.LayerSpec("na", 520, 2100, v=8, k1=65536, k2=256)
    d = synth.make_layer(spec, 60, B, B)
    dl = b.DeviceLayer(d)
    assert b.vptq_linear_path(dl.desc, B) == "decode_l2_fma"
    assert b.vptq_linear_workspace_bytes(dl.desc, B) > 0
    rng = np.random.default_rng(B)
    x1 = dl.upload_x(d["x"])
    x2_np = rng.normal(0, 1, size=d["x"].shape).astype(np.float16)
    x2 = dl.upload_x(x2_np)
    L = oracle.Layer.from_synth(d)
    for x, x_np in ((x1, d["x"]), (x2, x2_np)):           # two calls in a row on the shared array
        want = dl.linear(x).float().cpu().numpy()          # existing entry point, caller's workspace
        out = torch.full((B, spec.M), float("nan"), dtype=torch.float16, device="cuda")
        got = b.vptq_linear_noalloc(dl.desc, x, dl.ptrs, out).float().cpu().numpy()
        assert np.isfinite(got).all()
        assert rel_err(got, want.astype(np.float64)) <= TOL
        assert rel_err(got, L.linear(x_np)) <= TOL


def test_noalloc_rejects_what_it_cannot_run(b):
    # Argument checks only: every call below must return before anything is launched, so the
    # host-side query is asserted first and the call is made only if it says "too large".
    # so many vector rows per SM that the kernel adds partial sums up in scratch: 4 * 4 * M bytes
    big = b.make_desc(400000, 8192, 8, 65536, 256)
    assert b.vptq_linear_path(big, 4) == "decode_l2_fma"
    assert b.vptq_linear_workspace_bytes(big, 4) > b.NOALLOC_SCRATCH_BYTES
    p = b.LayerPtrs(0x1000, 0x1000, 0x1000, 0x1000, None, None, 0x1000, 0x1000)
    assert b.lib.vptq_linear_noalloc(C.byref(big), 0x1000, 4, C.byref(p), 0x1000, None) == b.E_SCRATCH_LIMIT
    assert "scratch" in b.lib.vptq_status_string(b.E_SCRATCH_LIMIT).decode()
    # a geometry the kernel does not cover (shared-memory codebook path, outlier columns)
    small = b.make_desc(64, 64, 6, 4096, 256, n_outlier=3, v0=4, k0=4096)
    assert b.vptq_linear_path(small, 1) != "decode_l2_fma"
    p2 = b.LayerPtrs(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000)
    assert b.lib.vptq_linear_noalloc(C.byref(small), 0x1000, 1, C.byref(p2), 0x1000, None) == b.E_UNSUPPORTED
    ok = b.make_desc(520, 2100, 8, 65536, 256)
    assert b.lib.vptq_linear_noalloc(C.byref(ok), 0x1000, 17, C.byref(p), 0x1000, None) == b.E_SHAPE
    assert b.lib.vptq_linear_noalloc(C.byref(ok), None, 1, C.byref(p), 0x1000, None) == b.E_NULL
