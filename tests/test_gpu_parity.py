"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer/byte work and the restored FP16 weights must match bit for bit; layer
outputs must satisfy max|y_gpu - y_ref| / max|y_ref| <= 2e-3."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2409_17066_b200 import synth

from helpers import TOL, rel_err, sample_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2409_17066_b200 import build as vbuild
    vbuild.build()
    from paper_2409_17066_b200 import binding
    return binding


# ------------------------------------------------------------------ pack / unpack

@pytest.mark.parametrize("k", [1, 2, 3, 16, 100, 256, 257, 4096, 5000, 8192, 40000, 65536])
@pytest.mark.parametrize("shape", [(1, 1), (3, 7), (5, 41), (4, 257), (2, 4055), (9, 4096)])
def test_pack_unpack_bit_exact(b, k, shape):
    rng = np.random.default_rng(k * 7 + shape[1])
    for idx in (rng.integers(0, k, size=shape, dtype=np.int32), np.full(shape, k - 1, np.int32)):
        ref = oracle.pack(idx, k)
        dev = torch.from_numpy(idx).cuda()
        packed = b.vptq_pack(dev, k)
        assert packed.shape == ref.shape
        assert np.array_equal(packed.cpu().numpy(), ref)
        # unpack what the ORACLE packed (independent of the GPU packer)
        back = b.vptq_unpack(torch.from_numpy(ref).cuda(), shape[0], shape[1], k)
        assert np.array_equal(back.cpu().numpy(), idx)


def test_pack_reports_out_of_range(b):
    idx = torch.tensor([[0, 1, 5, 2], [7, 0, -1, 3]], dtype=torch.int32, device="cuda")
    with pytest.raises(b.VptqError) as e:
        b.vptq_pack(idx, 5)
    assert e.value.code == b.E_INDEX_RANGE
    # without the check the call succeeds and stores 0 for the bad entries
    packed = b.vptq_pack(idx, 5, check=False)
    back = b.vptq_unpack(packed, 2, 4, 5).cpu().numpy()
    assert np.array_equal(back, np.array([[0, 1, 0, 2], [0, 0, 0, 3]], np.int32))


def test_empty_matrices(b):
    assert b.lib.vptq_pack(None, 0, 5, 16, None, None, None) == b.OK
    assert b.lib.vptq_unpack(None, 3, 0, 16, None, None) == b.OK


# ------------------------------------------------------------------ dequant, small layers

@pytest.mark.parametrize("spec", synth.small_specs(), ids=lambda s: s.name)
@pytest.mark.parametrize("scale_rows", [False, True])
def test_dequant_small_bit_exact(b, spec, scale_rows):
    if scale_rows and not spec.has_scale:
        pytest.skip("no scale")
    d = synth.make_layer(spec, 70, 1, 1)
    if scale_rows:   # per-output-row tables have length M
        rng = np.random.default_rng(5)
        d["scale"] = rng.uniform(0.5, 1.5, spec.M).astype(np.float16)
        d["bias"] = rng.normal(0, 0.01, spec.M).astype(np.float16)
    ref = oracle.Layer.from_synth(d, scale_axis=int(scale_rows)).dequant()
    dl = b.DeviceLayer(d, scale_rows=scale_rows)
    got = dl.dequant().cpu().numpy()
    assert np.array_equal(got.view(np.uint16), ref.view(np.uint16))


def test_dequant_extreme_values_bit_exact(b):
    # FP16 subnormals, overflow to inf through the scale, signed zeros
    spec = synth.LayerSpec("x", 32, 64, v=8, k1=256, k2=256)
    d = synth.make_layer(spec, 71, 0, 1)
    bits = np.random.default_rng(9).integers(0, 0x7C00, size=(256, 8)).astype(np.uint16)
    bits[::2] |= 0x8000
    d["c1"] = bits.view(np.float16)
    d["c2"] = (np.random.default_rng(10).integers(0, 0x0400, size=(256, 8)).astype(np.uint16)).view(np.float16)
    d["scale"][:8] = np.float16(1024.0)
    ref = oracle.Layer.from_synth(d).dequant()
    got = b.DeviceLayer(d).dequant().cpu().numpy()
    assert np.array_equal(got.view(np.uint16), ref.view(np.uint16))
    assert np.isinf(ref.astype(np.float32)).any() and (np.abs(ref.astype(np.float32)) < 6e-5).any()


# ------------------------------------------------------------------ linear, small layers

BATCHES = [1, 2, 3, 4, 5, 8, 9, 16, 17, 33]


@pytest.mark.parametrize("spec", synth.small_specs(), ids=lambda s: s.name)
@pytest.mark.parametrize("force_generic", [False, True])
def test_linear_small(b, spec, force_generic):
    for B in BATCHES:
        d = synth.make_layer(spec, 72, 2, B)
        y_ref = oracle.Layer.from_synth(d).linear(d["x"])
        for out_dtype in ("fp32", "fp16"):
            s2 = synth.LayerSpec(**{**spec.__dict__, "out_dtype": out_dtype})
            dl = b.DeviceLayer(dict(d, spec=s2))
            if force_generic:
                dl = dl.with_flags(dl.desc.flags | b.FLAG_FORCE_GENERIC)
            y = dl.linear(dl.upload_x(d["x"])).float().cpu().numpy()
            assert y.shape == y_ref.shape
            assert rel_err(y, y_ref) <= TOL, (spec.name, B, out_dtype, b.vptq_linear_path(dl.desc, B))


@pytest.mark.parametrize("spec", [s for s in synth.small_specs() if s.has_scale][:5], ids=lambda s: s.name)
def test_linear_small_scale_rows_and_bf16(b, spec):
    rng = np.random.default_rng(6)
    for B in (1, 4, 16):
        s2 = synth.LayerSpec(**{**spec.__dict__, "x_dtype": "bf16", "out_dtype": "fp32"})
        d = synth.make_layer(s2, 73, 3, B)
        d["scale"] = rng.uniform(0.5, 1.5, spec.M).astype(np.float16)
        d["bias"] = rng.normal(0, 0.01, spec.M).astype(np.float16)
        y_ref = oracle.Layer.from_synth(d, scale_axis=1).linear(d["x"])
        dl = b.DeviceLayer(d, scale_rows=True)
        y = dl.linear(dl.upload_x(d["x"])).cpu().numpy()
        assert rel_err(y, y_ref) <= TOL, (spec.name, B)
        # bf16 output: equals the fp32 result rounded to bf16, up to one unit in the last place
        s3 = synth.LayerSpec(**{**s2.__dict__, "out_dtype": "bf16"})
        dl3 = b.DeviceLayer(dict(d, spec=s3), scale_rows=True)
        y3 = dl3.linear(dl3.upload_x(d["x"])).float().cpu().numpy()
        assert np.all(np.abs(y3 - y) <= np.abs(y) * 2.0 ** -7 + 1e-30)


def test_linear_is_repeatable_and_leaves_inputs_alone(b):
    spec = synth.small_specs()[3]
    d = synth.make_layer(spec, 74, 0, 4)
    dl = b.DeviceLayer(d)
    x = dl.upload_x(d["x"])
    x0 = x.clone()
    y1 = dl.linear(x).clone()
    y2 = dl.linear(x).clone()
    assert torch.equal(x, x0)
    assert rel_err(y2.float().cpu().numpy(), y1.double().cpu().numpy()) <= 1e-3


DET_CASES = [
    # (path a deterministic call takes, spec, batch)
    ("decode_l2_fma", synth.LayerSpec("d_l2", 1030, 2100, v=8, k1=65536, k2=256), 1),
    ("decode_l2_fma", synth.LayerSpec("d_l2b", 1200, 4360, v=8, k1=65536, k2=256), 7),      # rows that divide badly over the SMs
    ("generic", synth.LayerSpec("d_smem", 520, 700, v=6, k1=4096, k2=256, n_out=7, v0=4, k0=4096), 1),
    ("generic", synth.LayerSpec("d_mma", 520, 700, v=6, k1=4096, k2=256, n_out=7, v0=4, k0=4096), 12),
    ("generic", synth.LayerSpec("d_gl", 600, 134, v=12, k1=4096, k2=4096, n_out=2, v0=4, k0=8192, n_groups=4), 2),
    ("gemm_tcgen05", synth.LayerSpec("d_gemm", 264, 4100, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32"), 40),
]


@pytest.mark.parametrize("path,spec,B", DET_CASES, ids=[c[1].name for c in DET_CASES])
def test_deterministic_calls_repeat_bit_for_bit(b, path, spec, B):
    # VPTQ_FLAG_DETERMINISTIC: every sum in a fixed order; two calls give identical bits, and the right ones
    d = synth.make_layer(spec, 83, 1, B)
    dl = b.DeviceLayer(d)
    det = dl.with_flags(dl.desc.flags | b.FLAG_DETERMINISTIC)
    assert b.vptq_linear_path(det.desc, B) == path
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(det.desc), B) == 0
    x = dl.upload_x(d["x"])
    ys = [det.linear(x).clone() for _ in range(4)]
    for y in ys[1:]:
        assert torch.equal(y, ys[0])
    assert rel_err(ys[0].float().cpu().numpy(), oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
    # and agrees with the fast path to summation order
    assert rel_err(dl.linear(x).float().cpu().numpy(), ys[0].double().cpu().numpy()) <= TOL


def test_deterministic_calls_ignore_prepared_images_and_fused_launches(b):
    spec = synth.LayerSpec("d_prep", 520, 1030, v=8, k1=65536, k2=256)
    d = synth.make_layer(spec, 84, 0, 1)
    dl = b.DeviceLayer(d)
    pl = dl.prepared(7)
    det = pl.with_flags(pl.desc.flags | b.FLAG_DETERMINISTIC)
    det.desc.prepared_parts = pl.desc.prepared_parts
    assert b.vptq_linear_path(det.desc, 1) == "decode_l2_fma"
    x = dl.upload_x(d["x"])
    y1, y2 = det.linear(x).clone(), det.linear(x).clone()
    assert torch.equal(y1, y2)
    assert rel_err(y1.float().cpu().numpy(), oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
    assert b.vptq_linear_fused_path([det.desc, det.desc], 1) == "one_by_one"


def test_linear_argument_errors(b):
    spec = synth.small_specs()[0]
    d = synth.make_layer(spec, 75, 0, 1)
    dl = b.DeviceLayer(d)
    x = dl.upload_x(d["x"])
    out = torch.empty((1, spec.M), dtype=torch.float16, device="cuda")
    lib = b.lib
    assert lib.vptq_linear(C.byref(dl.desc), x.data_ptr(), 0, C.byref(dl.ptrs), out.data_ptr(), None, 0, None) == b.E_SHAPE
    assert lib.vptq_linear(C.byref(dl.desc), x.data_ptr() + 2, 1, C.byref(dl.ptrs), out.data_ptr(), None, 0, None) == b.E_ALIGN
    need = b.vptq_linear_workspace_bytes(dl.desc, 1)
    if need > 0:
        assert lib.vptq_linear(C.byref(dl.desc), x.data_ptr(), 1, C.byref(dl.ptrs), out.data_ptr(), None, 0, None) == b.E_WORKSPACE
    # a corrupt stream (index >= k) is clamped, never read out of range: k = 5 needs 3 bits, store 7 everywhere
    spec5 = synth.LayerSpec("c", 16, 32, v=8, k1=5)
    d5 = synth.make_layer(spec5, 75, 1, 1)
    dl5 = b.DeviceLayer(d5)
    dl5.idx1.fill_(0xFF)
    W = dl5.dequant().cpu().numpy()
    d5c = dict(d5, idx1=np.full_like(d5["idx1"], 4))
    assert np.array_equal(W.view(np.uint16), oracle.Layer.from_synth(d5c).dequant().view(np.uint16))
    y = dl5.linear(dl5.upload_x(d5["x"])).float().cpu().numpy()
    assert rel_err(y, oracle.Layer.from_synth(d5c).linear(d5["x"])) <= TOL


# ------------------------------------------------------------------ batched tensor-core path

@pytest.mark.parametrize("M,N,k2,B,out_dtype", [
    (136, 520, 0, 17, "fp32"),       # ragged rows, ragged last k block, one token half
    (264, 1030, 256, 300, "fp16"),   # residual codebook, both token halves, ragged everything
    (136, 4100, 256, 40, "fp32"),    # few row tiles and many k blocks: K is split, partial sums meet by red.add
    (1024, 512, 256, 1100, "fp32"),  # three token tiles (the last one ragged)
    (1100, 13000, 256, 24, "fp32"),  # long shares of k blocks: the last piece of a split tile stores and raises
                                     # the tile's flag, the other pieces wait for it and reduce-add
])
def test_linear_batched_tcgen05(b, M, N, k2, B, out_dtype):
    spec = synth.LayerSpec("g", M, N, v=8, k1=65536, k2=k2, x_dtype="bf16", out_dtype=out_dtype)
    d = synth.make_layer(spec, 76, B % 7, B)
    dl = b.DeviceLayer(d)
    assert b.vptq_linear_path(dl.desc, B) == "gemm_tcgen05"
    y_ref = oracle.Layer.from_synth(d).linear(d["x"])
    x = dl.upload_x(d["x"])
    for _ in range(2):                                  # twice: the workspace is reused
        y = dl.linear(x)
        assert b.vptq_workspace_status(dl.workspace(B)) == b.OK
        assert rel_err(y.float().cpu().numpy(), y_ref) <= TOL
    # and against the plain fallback kernel (a second CUDA formulation)
    g = dl.with_flags(dl.desc.flags | b.FLAG_FORCE_GENERIC)
    yg = g.linear(x).float().cpu().numpy()
    assert rel_err(y.float().cpu().numpy(), yg.astype(np.float64)) <= TOL


def test_linear_batched_tcgen05_without_waits_between_ctas(b):
    # VPTQ_FLAG_CONCURRENT: the long-share shape whose split tiles otherwise meet by flag order; cleared output,
    # every piece added, no CTA waits for another
    spec = synth.LayerSpec("gc", 1100, 13000, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32")
    B = 24
    d = synth.make_layer(spec, 76, 3, B)
    dl = b.DeviceLayer(d)
    assert b.lib.vptq_linear_waits_between_ctas(C.byref(dl.desc), B) == 1
    sh = dl.with_flags(dl.desc.flags | b.FLAG_CONCURRENT)
    assert b.vptq_linear_path(sh.desc, B) == "gemm_tcgen05" and b.lib.vptq_linear_waits_between_ctas(C.byref(sh.desc), B) == 0
    y_ref = oracle.Layer.from_synth(d).linear(d["x"])
    x = dl.upload_x(d["x"])
    for _ in range(2):
        y = sh.linear(x)
        assert b.vptq_workspace_status(sh.workspace(B)) == b.OK
        assert rel_err(y.float().cpu().numpy(), y_ref) <= TOL


def test_linear_batched_tcgen05_with_a_stored_column_order(b):
    # Sec. 3.2.3: stored column j is input feature col_perm[j]; the pre-pass gathers the activations
    spec = synth.LayerSpec("gp", 264, 1032, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32", permuted=True)
    B = 40
    d = synth.make_layer(spec, 77, 1, B)
    dl = b.DeviceLayer(d)
    assert dl.desc.flags & b.FLAG_COL_PERM and b.vptq_linear_path(dl.desc, B) == "gemm_tcgen05"
    y = dl.linear(dl.upload_x(d["x"])).float().cpu().numpy()
    assert b.vptq_workspace_status(dl.workspace(B)) == b.OK
    assert rel_err(y, oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
    # the same layer without its column order gives another result: the order is really applied
    plain = {k: v for k, v in d.items() if k != "col_perm"}
    assert rel_err(y, oracle.Layer.from_synth(plain).linear(d["x"])) > 100 * TOL


# ------------------------------------------------------------------ several layers over the same activations

def _fused_case(b, specs, B, seed):
    ds = [synth.make_layer(sp, seed + 7 * i, 3, B) for i, sp in enumerate(specs)]
    for d in ds[1:]:
        d["x"] = ds[0]["x"]                                  # the layers of a fused call read the same x
    dls = [b.DeviceLayer(d) for d in ds]
    x = dls[0].upload_x(ds[0]["x"])
    descs = [dl.desc for dl in dls]
    outs = [torch.full((B, dl.spec.M), float("nan"), dtype=b._TORCH_DT[dl.desc.out_dtype], device="cuda") for dl in dls]
    need = b.vptq_linear_fused_workspace_bytes(descs, B)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None
    b.vptq_linear_fused(descs, [dl.ptrs for dl in dls], x, outs, ws)
    return ds, dls, x, outs


@pytest.mark.parametrize("Ms,N,k2,B,out_dtypes", [
    ((4096, 1024, 1024), 4096, 256, 1, ("fp16", "fp16", "fp16")),   # q/k/v shaped
    ((4100, 1000, 1024), 4096, 256, 3, ("fp32", "fp16", "fp16")),   # ragged rows, 3 tokens, mixed output types
    ((2048, 2048), 4096, 0, 5, ("fp16", "fp16")),                   # gate/up shaped, no residual, two token groups
    ((2900, 600), 4360, 256, 2, ("fp16", "fp32")),                  # ragged rows and a ragged last chunk of columns
])
def test_linear_fused_matches_oracle_and_single_calls(b, Ms, N, k2, B, out_dtypes):
    specs = [synth.LayerSpec("f%d" % i, M, N, v=8, k1=65536, k2=k2, x_dtype="bf16", out_dtype=od)
             for i, (M, od) in enumerate(zip(Ms, out_dtypes))]
    ds, dls, x, outs = _fused_case(b, specs, B, 311)
    assert b.vptq_linear_fused_path([dl.desc for dl in dls], B) == "fused_decode_l2_fma"
    tb = 4 if B >= 4 else 2 if B >= 2 else 1                 # tokens per launch
    assert b.vptq_linear_fused_launches([dl.desc for dl in dls], B) == (B + tb - 1) // tb
    for d, dl, y in zip(ds, dls, outs):
        y = y.float().cpu().numpy()
        assert np.isfinite(y).all()
        assert rel_err(y, oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
        y1 = dl.linear(x).float().cpu().numpy()              # the layer's own launch: same arithmetic
        assert rel_err(y, y1.astype(np.float64)) <= 1e-3 * TOL + (4e-3 if dl.desc.out_dtype != b.DTYPE_FP32 else 0)


@pytest.mark.parametrize("family,Ms,kw,B", [
    ("fused_decode_smem_fma", (1200, 1176), dict(N=700, v=6, k1=4096, k2=256, n_out=7, v0=4, k0=4096), 1),
    ("fused_decode_smem_fma", (1200, 900, 1500), dict(N=700, v=6, k1=4096, k2=256, n_out=7, v0=4, k0=4096), 3),
    ("fused_decode_smem_fma", (1600, 1360), dict(N=520, v=8, k1=256), 4),
    ("fused_decode_gl_fma", (1200, 1800), dict(N=134, v=12, k1=4096, k2=4096, n_out=2, v0=4, k0=8192, n_groups=4), 1),
    ("fused_decode_gl_fma", (1200, 1800), dict(N=134, v=12, k1=4096, k2=4096, n_out=2, v0=4, k0=8192, n_groups=4, permuted=True), 2),
])
def test_linear_fused_other_kernel_families(b, family, Ms, kw, B):
    specs = [synth.LayerSpec("f%d" % i, M, **kw) for i, M in enumerate(Ms)]
    ds, dls, x, outs = _fused_case(b, specs, B, 411)
    assert b.vptq_linear_fused_path([dl.desc for dl in dls], B) == family
    assert b.vptq_linear_fused_workspace_bytes([dl.desc for dl in dls], B) == 0
    for d, dl, y in zip(ds, dls, outs):
        y = y.float().cpu().numpy()
        assert np.isfinite(y).all()
        assert rel_err(y, oracle.Layer.from_synth(d).linear(d["x"])) <= TOL


@pytest.mark.parametrize("B", [1, 40])
def test_linear_host_io_matches_the_device_call(b, B):
    # host activations in, host result out (pinned memory), the weights resident: the decode and the batched path
    spec = synth.LayerSpec("hio", 264, 1030, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32")
    d = synth.make_layer(spec, 79, 2, B)
    dl = b.DeviceLayer(d)
    x_host = torch.from_numpy(np.ascontiguousarray(d["x"])).view(torch.bfloat16).pin_memory()
    out_host = torch.empty((B, spec.M), dtype=torch.float32).pin_memory()
    x_dev = torch.empty((B, spec.N), dtype=torch.bfloat16, device="cuda")
    out_dev = torch.empty((B, spec.M), dtype=torch.float32, device="cuda")
    b.vptq_linear_host_io(dl.desc, x_host, dl.ptrs, out_host, x_dev, out_dev, dl.workspace(B))
    torch.cuda.synchronize()
    assert rel_err(out_host.numpy(), oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
    assert torch.equal(out_host, out_dev.cpu())


def test_linear_fused_host_io_matches_the_device_call(b):
    specs = [synth.LayerSpec("h%d" % i, M, 4096, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype=od)
             for i, (M, od) in enumerate(((4096, "fp16"), (1024, "fp32"), (1024, "fp16")))]
    B = 2
    ds, dls, x, outs = _fused_case(b, specs, B, 511)
    fused = b.FusedLayers(dls)
    assert fused.path(B) == "fused_decode_l2_fma"
    x_host = torch.from_numpy(np.ascontiguousarray(ds[0]["x"])).view(torch.bfloat16).pin_memory()
    outs_host = [torch.empty_like(o, device="cpu").pin_memory() for o in outs]
    x_dev = torch.empty_like(x)
    outs_dev = [torch.empty_like(o) for o in outs]
    fused.linear_host_io(x_host, outs_host, x_dev, outs_dev)
    torch.cuda.synchronize()
    for d, oh, o in zip(ds, outs_host, outs):
        assert rel_err(oh.float().numpy(), oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
        assert rel_err(oh.float().numpy(), o.float().cpu().numpy().astype(np.float64)) <= 4e-3


def test_linear_fused_runs_other_kernel_families_one_by_one(b):
    spec = {sp.name: sp for sp in synth.small_specs()}["s_v6_full"]
    specs = [spec, spec]
    B = 2
    ds, dls, x, outs = _fused_case(b, specs, B, 17)
    assert b.vptq_linear_fused_path([dl.desc for dl in dls], B) == "one_by_one"
    for d, y in zip(ds, outs):
        assert rel_err(y.float().cpu().numpy(), oracle.Layer.from_synth(d).linear(d["x"])) <= TOL



# ------------------------------------------------------------------ assignment step of the quantizer (Eq. 2)

@pytest.mark.parametrize("M,N,v,k", [
    (136, 520, 8, 4096),       # several blocks, several codebook chunks
    (130, 333, 6, 4096),       # v = 6 (padded to 8 components), ragged last vector row (130 = 21 * 6 + 4)
    (60, 134, 12, 1000),       # v = 12 (padded to 16), a short last chunk
    (34, 77, 2, 16),
    (9, 17, 1, 1),
    (16, 64, 8, 65536),        # the largest table, few vectors
    (70, 50, 24, 300),         # v > 16
])
def test_assign_is_bit_identical_to_the_oracle(b, M, N, v, k):
    rng = np.random.default_rng(1000 * v + k)
    W = rng.normal(0, 0.02, (M, N)).astype(np.float16)
    Cb = rng.normal(0, 0.02, (k, v)).astype(np.float16)
    idx = b.vptq_assign(torch.from_numpy(W).cuda(), v, torch.from_numpy(Cb).cuda(), b.FLAG_FORCE_GENERIC).cpu().numpy()
    assert np.array_equal(idx, oracle.assign(W, v, Cb))


@pytest.mark.parametrize("M,N,v,k,sigma", [
    (136, 520, 8, 4096, 0.02),     # 35 steps of 256 vectors (the last one ragged), 32 centroid tiles
    (132, 400, 6, 4096, 0.02),     # v = 6
    (120, 500, 12, 2000, 0.02),    # v = 12, a padded last centroid tile
    (64, 600, 8, 65536, 0.02),     # the largest table
    (136, 520, 8, 4096, 30.0),     # large values: norms of about 7000
    (72, 520, 1, 1024, 1.0),       # v = 1
    (136, 520, 8, 4096, 1e-3),     # small values: norms of about 1e-5 (the low half of the FP16 split must not underflow)
    (136, 520, 8, 4096, 1e-4),     # FP16 subnormals throughout
    (136, 520, 8, 4096, 3e-6),     # a few FP16 subnormal steps: many equal vectors and centroids
    (136, 520, 8, 4096, 3000.0),   # near the top of the FP16 range
])
def test_assign_on_tensor_cores_gives_the_same_indices(b, M, N, v, k, sigma):
    rng = np.random.default_rng(77 * v + k)
    W = rng.normal(0, sigma, (M, N)).astype(np.float16)
    Cb = rng.normal(0, sigma, (k, v)).astype(np.float16)
    assert b.vptq_assign_path(M, N, v, k) == "assign_tcgen05"
    assert b.vptq_assign_path(M, N, v, k, b.FLAG_FORCE_GENERIC) == "assign_fp32"
    Wd, Cd = torch.from_numpy(W).cuda(), torch.from_numpy(Cb).cuda()
    idx = b.vptq_assign(Wd, v, Cd).cpu().numpy()
    assert np.array_equal(idx, oracle.assign(W, v, Cb))


def test_assign_on_tensor_cores_with_ties_everywhere(b):
    # every centroid occurs 16 times, 128 apart: equal distances in different candidate groups; the lowest index
    # wins, which only the full FP32 scan of the listed vectors can know
    rng = np.random.default_rng(5)
    M, N, v = 64, 600, 8
    base = rng.normal(0, 0.02, (128, v)).astype(np.float16)
    Cb = np.tile(base, (16, 1))
    W = rng.normal(0, 0.02, (M, N)).astype(np.float16)
    assert b.vptq_assign_path(M, N, v, Cb.shape[0]) == "assign_tcgen05"
    idx = b.vptq_assign(torch.from_numpy(W).cuda(), v, torch.from_numpy(Cb).cuda()).cpu().numpy()
    assert idx.max() < 128
    assert np.array_equal(idx, oracle.assign(W, v, Cb))
    # norms beyond the FP16 range: the filter is meaningless, every vector goes through the full scan
    big = (rng.normal(0, 150.0, (2048, v))).astype(np.float16)
    Wb = rng.normal(0, 150.0, (M, N)).astype(np.float16)
    idx = b.vptq_assign(torch.from_numpy(Wb).cuda(), v, torch.from_numpy(big).cuda()).cpu().numpy()
    assert np.array_equal(idx, oracle.assign(Wb, v, big))


@pytest.mark.parametrize("flags", [0, 4], ids=["tensor_cores", "fp32"])
def test_assign_with_values_that_are_not_numbers(b, flags):
    # NaN and infinite components: such distances never win (oracle rule); the tensor-core filter cannot rank
    # them and sends the vectors (all of them, when the codebook has such an entry) through the full FP32 scan
    rng = np.random.default_rng(31)
    M, N, v, k = 64, 600, 8, 2048
    W = rng.normal(0, 0.02, (M, N)).astype(np.float16)
    W[3, 5] = np.nan
    W[17, 100] = np.inf
    W[40, 7] = -np.inf
    Cb = rng.normal(0, 0.02, (k, v)).astype(np.float16)
    for bad_codebook in (False, True):
        if bad_codebook:
            Cb[77, 2] = np.nan
            Cb[900, 0] = np.inf
        idx = b.vptq_assign(torch.from_numpy(W).cuda(), v, torch.from_numpy(Cb).cuda(), flags).cpu().numpy()
        assert np.array_equal(idx, oracle.assign(W, v, Cb))


def test_assign_then_pack_and_dequant_reproduce_the_matrix(b):
    # a matrix built from centroids goes through assign -> pack -> dequant unchanged
    spec = synth.LayerSpec("enc", 264, 300, v=8, k1=4096, has_scale=False)
    d = synth.make_layer(spec, 78, 0, 1)
    dl = b.DeviceLayer(d)
    W = dl.dequant()
    idx = b.vptq_assign(W, 8, dl.c1)
    again = b.DeviceLayer(dict(d, idx1=idx.cpu().numpy()))
    assert torch.equal(again.dequant(), W)
    # with distinct centroids even the indices come back
    if np.unique(d["c1"].view(np.uint16), axis=0).shape[0] == spec.k1:
        assert torch.equal(b.vptq_pack(idx, spec.k1), dl.idx1)


# ------------------------------------------------------------------ k-means centroid update (Sec. 3.2.1)

@pytest.mark.parametrize("M,N,v,k,weighted", [
    (136, 520, 8, 4096, True),      # sums straight into the workspace
    (130, 333, 6, 300, True),       # shared-memory copy per block, ragged last vector row
    (64, 40, 8, 32, False),         # unweighted
    (60, 134, 12, 5000, True),
])
def test_kmeans_update_matches_the_weighted_mean(b, M, N, v, k, weighted):
    rng = np.random.default_rng(7 * k + v)
    W = rng.normal(0, 0.02, (M, N)).astype(np.float16)
    Cb = rng.normal(0, 0.02, (k, v)).astype(np.float16)
    h = rng.uniform(0.2, 5.0, N).astype(np.float32) if weighted else None
    idx = oracle.assign(W, v, Cb)
    want = oracle.kmeans_update(W, v, idx, Cb, h).astype(np.float64)
    got = b.vptq_kmeans_update(torch.from_numpy(W).cuda(), v, torch.from_numpy(idx).cuda(), torch.from_numpy(Cb).cuda(),
                               None if h is None else torch.from_numpy(h).cuda()).cpu().numpy().astype(np.float64)
    # FP32 atomic sums against the FP64 mean: at most the last FP16 bit
    assert np.all(np.abs(got - want) <= 2.0 ** -10 * np.abs(want) + 1e-7)
    # centroids nobody was assigned to are untouched, bit for bit
    unused = np.setdiff1d(np.arange(k), np.unique(idx))
    assert np.array_equal(got[unused], Cb[unused].astype(np.float64))


def test_lloyd_iterations_on_the_gpu_decrease_the_distortion(b):
    rng = np.random.default_rng(23)
    v, k, M, N = 8, 256, 256, 300
    W = rng.normal(0, 1, (M, N)).astype(np.float16)
    h = rng.uniform(0.2, 5.0, N).astype(np.float32)
    Wd, hd = torch.from_numpy(W).cuda(), torch.from_numpy(h).cuda()
    Cd = torch.from_numpy(rng.normal(0, 1, (k, v)).astype(np.float16)).cuda()
    prev = None
    for _ in range(5):
        idx = b.vptq_assign(Wd, v, Cd)
        b.vptq_kmeans_update(Wd, v, idx, Cd, hd)
        dist = oracle.distortion(W, v, idx.cpu().numpy(), Cd.cpu().numpy(), h)
        assert prev is None or dist <= prev * (1 + 2e-3)
        prev = dist
